// Fused decode GEMV at batch 1, one output channel per lane, V2 and V2a:  y = (D + S) x.
//
// This is the kernel of the single-token decode step ("Fused Decode Kernel", M = 1).  It keeps the decode of
// xfp_gemv_pair.cu -- pair tables in lane-private shared-memory banks, the looked-up half2 used directly as the A
// fragment of mma.sync.m16n8k16, x on the diagonal lanes of the B fragment, fp32 accumulation -- with one channel
// per lane everywhere, so that a CTA is one row-block and launches of any size fill the SMs evenly: one CTA of 16
// warps per SM on matrices with no more row-blocks than SMs, two CTAs of 8 (or 16) warps per SM beyond.
//
// Mapping.  A CTA owns one row-block of 32 channels (lane l = channel l) over all of K or one K slice; its warps
// share K in super-chunks of 128 weights.  One mma covers 8 consecutive k of every channel: the fragment's row g
// carries the lane's weights k..k+3, its row g+8 the weights k+4..k+7; lanes with g == t feed columns 0..3 of the B
// fragment with x[k..k+3], lanes with g == t+4 feed columns 4..7 with x[k+4..k+7]; D[g][n] and D[g+8][4+n] are the
// two halves of channel 4g+n.
//
// Tables, per bit width (V2):
//   N = 2   QUAD table: a byte of the index stream is four indices; entry = the four decoded fp16 (8 bytes per
//           lane, 256 bytes between entries), so one 64-bit load decodes four weights and one PRMT builds its address
//   N = 3   pair table, 64 entries of 4 bytes per lane
//   N = 4   pair table, 256 entries; entries 256 bytes apart so that the index byte is the second byte of the
//           address (one PRMT per look-up)
//   N = 5   pair table, 1024 entries (128 KB, one CTA per SM) or, beyond one round of CTAs, one entry per index
//   N = 6   one entry per index (a pair table would need 16 KB per channel), two look-ups joined by a PRMT
// V2a: the library replicated once per bank -- pair tables of every entry where L * 4^N words fit (N = 2 at L = 32),
// one word per entry otherwise, half a word at N = 6 -- see the kernel's comment.
//
// x is staged once per CTA in shared memory in an order that lets a diagonal lane fetch the B registers of TWO
// mma steps with one 16-byte load: inside every group of 16 k the two middle blocks of four are swapped
// ([0..3][8..11][4..7][12..15]).  Outlier columns are mapped through the same permutation.
//
// Outliers, split-K finish (ticket, fixed order) and the order of work before griddepcontrol.wait are those of
// xfp_gemv_pair.cu.
#include <cstdio>
#include <cstdlib>

#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

namespace {

constexpr int kLaneSlots = 4;   // outlier slots a warp keeps in flight
// smallest N whose codebooks travel through shared memory before the table fill (measured: N = 5 gains 4-8 %,
// N <= 4 loses the extra barrier)
constexpr int kLaneStageCodebooksFrom = 5;

struct LaneArgs {
    Offsets off;
    const void* packed;
    const uint16_t* x;
    void* y;
    // several blobs of one shape in one launch: device pointer lists; the row-blocks of all blobs are numbered
    // through (RB of them per blob) and scheduled as one matrix
    const void* const* packed_list;
    const uint16_t* const* x_list;
    void* const* y_list;
    float* partial;  // [slice][rows_ws]
    int* tickets;    // [blocks of the launch]
    int rows, cols, RB, SC, rows_ws, ell_slots;
    int y_is_fp16;   // type of y: 0 fp32, 1 fp16, 2 bf16
    int x_bf16;      // x holds bf16: converted to fp16 while it is staged
    int tab_bytes;   // shared-memory bytes of the look-up tables
    int L, GH;       // V2a: library size; groups per super-chunk (2 when the format's groups hold 64 weights)
    // schedule tiers: CTAs [tier_cta[i], tier_cta[i+1]) handle blocks from tier_blk[i] on, each cut into
    // tier_kst[i] slices of tier_spp[i] super-chunks
    int tier_cta[5], tier_blk[4], tier_kst[4], tier_spp[4];
#ifdef XFP_TRACE
    unsigned long long* trace;  // timing build only: per CTA 8 globaltimer stamps
#endif
};

// Phase stamps of a timing build (-DXFP_TRACE=1); a normal build has neither the stamps nor their plumbing.
__device__ __forceinline__ void lstamp(const LaneArgs& a, int slot) {
#ifdef XFP_TRACE
    if (a.trace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        a.trace[(size_t)blockIdx.x * 8 + slot] = t;
    }
#else
    (void)a; (void)slot;
#endif
}

// 16 bytes of staged x for the diagonal lanes of the B fragment; the other lanes keep their zeros.  Written as a
// predicated load so that the compiler neither branches around it nor re-zeroes the registers.
__device__ __forceinline__ void ld_x16_if(uint4& v, const unsigned char* p, bool take) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%5];\n\t}"
        : "+r"(v.x), "+r"(v.y), "+r"(v.z), "+r"(v.w)
        : "r"((uint32_t)take), "r"((uint32_t)__cvta_generic_to_shared(p)));
}

// position of activation k in the staged copy: inside every 16 the blocks [4..7] and [8..11] trade places
__device__ __forceinline__ uint32_t xpos(uint32_t k) { return (k & ~12u) | ((k & 4u) << 1) | ((k & 8u) >> 1); }

template <int N, bool SGL, int MODE>
struct LaneCfg {
    static constexpr int E = 1 << N;
    static constexpr bool kQuad = N == 2 && !SGL && MODE == 0;
    static constexpr bool kSingle = SGL;   // one entry per index: N = 6 always, N = 5 on short rows (no 128 KB fill)
    static constexpr int T = kQuad ? 256 : (kSingle ? E : E * E);          // table entries per channel
    static constexpr int kStride = (kQuad || N == 4) ? 256 : 128;            // bytes between entries
    static constexpr int kTabBytes = T * kStride;
};

// Byte offset (q << 6) of index j (compile time) merged with `base`, for tables whose entries are 64 bytes apart
// (two bytes per lane).
template <int N>
__device__ __forceinline__ uint32_t half_addr(const uint32_t* w, int j, uint32_t base) {
    constexpr uint32_t mask = ((1u << N) - 1u) << 6;
    const int bit = j * N, wi = bit >> 5, off = bit & 31;
    uint32_t v;
    if (off + N > 32)
        v = __funnelshift_r(w[wi], w[wi + 1], off - 6);
    else if (off >= 6)
        v = w[wi] >> (off - 6);
    else
        v = w[wi] << (6 - off);
    return (v & mask) | base;
}

// The four A registers of mma step j (weights 8j .. 8j+7 of the lane's channel in this super-chunk).
template <int N, bool SGL, bool HALF, bool QUAD>
__device__ __forceinline__ void lookup8(uint32_t (&f)[4], const uint32_t* w, int j, const unsigned char* tab,
                                        uint32_t base) {
    if (HALF) {
        uint32_t e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = *(const uint16_t*)(tab + half_addr<N>(w, 8 * j + i, base));
        f[0] = __byte_perm(e[0], e[1], 0x5410);
        f[2] = __byte_perm(e[2], e[3], 0x5410);
        f[1] = __byte_perm(e[4], e[5], 0x5410);
        f[3] = __byte_perm(e[6], e[7], 0x5410);
    } else if (QUAD) {
        // bytes 2j and 2j+1 of the stream; base = lane * 8
        const uint32_t a0 = __byte_perm(w[(2 * j) >> 2], base, 0x5504u | ((uint32_t)((2 * j) & 3) << 4));
        const uint32_t a1 = __byte_perm(w[(2 * j + 1) >> 2], base, 0x5504u | ((uint32_t)((2 * j + 1) & 3) << 4));
        const uint2 lo = *(const uint2*)(tab + a0);
        const uint2 hi = *(const uint2*)(tab + a1);
        f[0] = lo.x; f[2] = lo.y; f[1] = hi.x; f[3] = hi.y;
    } else if (SGL) {
        uint32_t e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = *(const uint32_t*)(tab + single_addr<N, 1>(w, 8 * j + i, base));
        f[0] = __byte_perm(e[0], e[1], 0x5410);
        f[2] = __byte_perm(e[2], e[3], 0x5410);
        f[1] = __byte_perm(e[4], e[5], 0x5410);
        f[3] = __byte_perm(e[6], e[7], 0x5410);
    } else {
        constexpr int SL = N == 4 ? 2 : 1;   // N = 4: entries 256 bytes apart
        f[0] = *(const uint32_t*)(tab + pair_addr<N, SL>(w, 4 * j, base));
        f[2] = *(const uint32_t*)(tab + pair_addr<N, SL>(w, 4 * j + 1, base));
        f[1] = *(const uint32_t*)(tab + pair_addr<N, SL>(w, 4 * j + 2, base));
        f[3] = *(const uint32_t*)(tab + pair_addr<N, SL>(w, 4 * j + 3, base));
    }
}

// last mma step of a super-chunk that still reads index vector v (compile time)
template <int N>
__host__ __device__ constexpr int last_step_of_vector(int v) {
    // vector v holds stream bits [128 v, 128 v + 128); step j reads bits [8 j N, 8 (j+1) N)
    return (128 * (v + 1) - 1) / (8 * N);
}

// MODE 0: V2 (the channel's own codebook, tables private to the lane).  MODE 1: V2a -- the whole library replicated
// once per bank (word (id * 2^N + q) * 32 + lane holds lib[id][q]), the table base of a lane follows the library id
// of its channel's current group, the fragment accumulates sum lib * x of ONE group, and after the group's steps the
// sum moves to the lane that owns the channel and is folded into its accumulator with the group's scale and
// mid-point:  acc += scale * G + mid * X_g,  X_g = sum of x over the group ("V2a: Shared Codebook Library").
// TIO instantiations take bf16 x and store bf16 y; compiled into the plain ones the conversion cost the fp16 path 4.5 %
// at 28672 x 8192 through register allocation alone (34.3 against 32.8 us), so only bf16 calls launch them.
template <int N, int W, int MINB, bool SGL, int MODE, bool TIO>
__global__ void __launch_bounds__(W * 32, MINB) gemv_lane_kernel(const LaneArgs a) {
    using C = LaneCfg<N, SGL, MODE>;
    constexpr bool kHalf = MODE == 2;   // V2a with a library too large for one 4-byte word per bank and entry
    constexpr int kEntry = kHalf ? 64 : 128;   // V2a: bytes between library entries
    constexpr int E = C::E;
    // V2a with a small library (L * 4^N words per bank fit): PAIR tables of every library entry, one look-up per two
    // weights as in V2
    constexpr bool kLibPair = MODE == 1 && !SGL;
    constexpr int kIdBytes = (kLibPair ? E * E : E) * kEntry;   // V2a: bytes between the tables of two library entries
    constexpr int T = C::T;
    constexpr int kStride = C::kStride;
    constexpr int kThreads = W * 32;
    extern __shared__ __align__(16) unsigned char smem[];
    // [tables | x fp16 [K] permuted | red [W][32]]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    lstamp(a, 0);
    const int K = a.SC * kSuper;
    unsigned char* tab = smem;
    unsigned char* xs = smem + a.tab_bytes;
    float* red = (float*)(xs + (size_t)K * 2);     // [W][32]
    float* xg = red + W * 32;                      // V2a: [SC][2] sums of x over the halves of every super-chunk
    uint32_t* cbs = (uint32_t*)xg;                 // V2 pair tables: the block's codebooks, word [e / 2][channel]

    // ---- this CTA's block and K slice
    int blk, slice, nslices, sc0, nsc;
    {
        int tier = 0;
#pragma unroll
        for (int i = 1; i < 4; ++i)
            if ((int)blockIdx.x >= a.tier_cta[i]) tier = i;
        const int c = blockIdx.x - a.tier_cta[tier];
        nslices = a.tier_kst[tier];
        blk = a.tier_blk[tier] + c / nslices;
        slice = c - (c / nslices) * nslices;
        sc0 = slice * a.tier_spp[tier];
        nsc = max(0, min(a.SC, sc0 + a.tier_spp[tier]) - sc0);
    }
    const int gw = slice * W + warp, ostride = nslices * W;
    // the blob of this block: `gblk` numbers the row-blocks of the whole launch, `blk` those of its blob
    const int gblk = blk;
    const void* packed = a.packed;
    const uint16_t* xsrc = a.x;
    void* ydst = a.y;
    int ell_slots = a.ell_slots;
    if (a.packed_list) {
        const int prob = blk / a.RB;
        blk -= prob * a.RB;
        packed = a.packed_list[prob];
        xsrc = a.x_list[prob];
        ydst = a.y_list[prob];
        ell_slots = __ldg((const int*)((const char*)packed + a.off.hdr));   // the blobs' outlier counts differ
    }
    const Blob b = blob_at(packed, a.off);

    // ---- loads that do not depend on earlier kernels: first index vectors, outlier slab, codebook
    uint32_t w[4 * N + 1];
    w[4 * N] = 0u;
    const uint4* ip = b.idx + ((size_t)(blk * a.SC + sc0) * N) * 32 + lane;
    if (warp < nsc) {
#pragma unroll
        for (int v = 0; v < N; ++v) {
            const uint4 t = ld_stream(ip + ((size_t)warp * N + v) * 32);
            w[4 * v] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
        }
    }
    // V2a: library id and (scale, mid) of the lane's channel for the two halves of the super-chunk ([1] repeats [0]
    // unless the groups hold 64 weights), current and next
    const int GH = MODE != 0 ? a.GH : 1;
    const size_t m0 = ((size_t)(blk * a.SC + sc0) * GH) * 32 + lane;
    uint32_t gid_c[2] = {0u, 0u}, gsm_c[2] = {0u, 0u}, gid_n[2] = {0u, 0u}, gsm_n[2] = {0u, 0u};
    if (MODE != 0 && warp < nsc) {
        gid_c[0] = b.gid[m0 + (size_t)warp * GH * 32]; gsm_c[0] = b.gsm[m0 + (size_t)warp * GH * 32];
        gid_c[1] = b.gid[m0 + ((size_t)warp * GH + GH - 1) * 32]; gsm_c[1] = b.gsm[m0 + ((size_t)warp * GH + GH - 1) * 32];
    }
    const uint32_t* ell = a.packed_list
        ? (const uint32_t*)((const char*)packed + *(const long long*)((const char*)packed + a.off.hdr + 8)) : b.ell;
    const uint32_t* slab = ell + (size_t)blk * (ell_slots + 1) * 32 + lane;
    uint32_t olen = ell_slots ? __ldg(slab) : 0u;
    uint32_t oe[kLaneSlots];
#pragma unroll
    for (int q = 0; q < kLaneSlots; ++q) {
        const int j = gw + q * ostride;
        oe[q] = j < ell_slots ? __ldg(slab + (size_t)(1 + j) * 32) : 0u;   // every slot below the capacity is readable
    }
    // ---- tables: warp w fills entries [w T / W, (w+1) T / W) of every lane's channel
    if (MODE != 0) {
        if (kHalf) {
            for (int e = warp; e < a.L * E; e += W) *(uint16_t*)(tab + (size_t)e * 64 + lane * 2) = __ldg(b.cb + e);
        } else if (kLibPair) {
            for (int e = warp; e < a.L * E * E; e += W) {
                const uint16_t* cb = b.cb + (size_t)(e >> (2 * N)) * E;
                *(uint32_t*)(tab + (size_t)e * 128 + lane * 4) = (uint32_t)__ldg(cb + (e & (E - 1))) | ((uint32_t)__ldg(cb + ((e >> N) & (E - 1))) << 16);
            }
        } else {
            for (int e = warp; e < a.L * E; e += W) *(uint32_t*)(tab + (size_t)e * 128 + lane * 4) = (uint32_t)__ldg(b.cb + e);
        }
    } else {
        const uint16_t* cb = b.cb + (size_t)(blk * kRowsPerBlock + lane) * E;
        if (C::kQuad) {
            // entry t = (cb[t & 3], cb[t >> 2 & 3], cb[t >> 4 & 3], cb[t >> 6]) as 8 bytes at t * 256 + lane * 8
            const uint2 c4 = __ldg((const uint2*)cb);   // the four entries
            const uint32_t e0 = c4.x & 0xffffu, e1 = c4.x >> 16, e2 = c4.y & 0xffffu, e3 = c4.y >> 16;
            auto ent = [&](int q) { return q == 0 ? e0 : (q == 1 ? e1 : (q == 2 ? e2 : e3)); };
            constexpr int TW = T / W;
#pragma unroll
            for (int i = 0; i < TW; ++i) {
                const int t = warp * TW + i;
                const uint32_t lo = ent(t & 3) | (ent((t >> 2) & 3) << 16);
                const uint32_t hi = ent((t >> 4) & 3) | (ent(t >> 6) << 16);
                *(uint2*)(tab + (size_t)t * kStride + lane * 8) = make_uint2(lo, hi);
            }
        } else if (C::kSingle) {
            constexpr int TW = T / W;   // 4
#pragma unroll
            for (int i = 0; i < TW; ++i) {
                const int t = warp * TW + i;
                *(uint32_t*)(tab + (size_t)t * kStride + lane * 4) = (uint32_t)__ldg(cb + t);
            }
        } else if (T / W >= E) {
            // a warp fills whole rows of the pair matrix: entries (hi, 0..E-1) for its values of hi.  Every warp needs
            // every entry of its lanes' channels: the block's codebooks (32 E fp16, contiguous) are fetched once with
            // coalesced loads and transposed through shared memory, instead of 16-byte loads 2 E bytes apart by every warp.
            constexpr int HW = T / W / E;   // values of the high index per warp
            constexpr bool kStage = N >= kLaneStageCodebooksFrom;
            uint32_t cw[E / 2];
            if (kStage) {
                const uint4* src = (const uint4*)(b.cb + (size_t)blk * kRowsPerBlock * E);
                for (int i = threadIdx.x; i < 4 * E; i += kThreads) {
                    const uint4 t = __ldg(src + i);
                    const int ch = i / (E / 8), w4 = (i % (E / 8)) * 4;
                    cbs[(w4 + 0) * 32 + ch] = t.x; cbs[(w4 + 1) * 32 + ch] = t.y;
                    cbs[(w4 + 2) * 32 + ch] = t.z; cbs[(w4 + 3) * 32 + ch] = t.w;
                }
                __syncthreads();
#pragma unroll
                for (int i = 0; i < E / 2; ++i) cw[i] = cbs[i * 32 + lane];
            } else {
#pragma unroll
                for (int i = 0; i < E / 8; ++i) {
                    const uint4 t = __ldg((const uint4*)cb + i);
                    cw[4 * i] = t.x; cw[4 * i + 1] = t.y; cw[4 * i + 2] = t.z; cw[4 * i + 3] = t.w;
                }
            }
#pragma unroll
            for (int hh = 0; hh < HW; ++hh) {
                const int hi = warp * HW + hh;
                const uint32_t hv = (kStage ? (uint32_t)((const uint16_t*)cbs)[((hi >> 1) * 32 + lane) * 2 + (hi & 1)]
                                            : (uint32_t)__ldg(cb + hi)) << 16;
#pragma unroll
                for (int lo = 0; lo < E; ++lo) {
                    const uint32_t lv = (lo & 1) ? (cw[lo >> 1] >> 16) : (cw[lo >> 1] & 0xffffu);
                    *(uint32_t*)(tab + (size_t)(hi * E + lo) * kStride + lane * 4) = lv | hv;
                }
            }
        } else {
            // few entries per warp (N = 3: 64 entries over 16 warps)
            constexpr int TW = T / W > 0 ? T / W : 1;
#pragma unroll
            for (int i = 0; i < TW; ++i) {
                const int t = warp * TW + i;
                if (t < T) {
                    const uint32_t lv = __ldg(cb + (t & (E - 1))), hv = __ldg(cb + (t >> N));
                    *(uint32_t*)(tab + (size_t)t * kStride + lane * 4) = lv | (hv << 16);
                }
            }
        }
    }

    // ---- x may come from the previous kernel of the stream
    lstamp(a, 1);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    lstamp(a, 2);
    for (int t = threadIdx.x; t < ((K / 8 + 31) & ~31); t += kThreads) {   // whole warps: the sums below shuffle
        const bool in = t < K / 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (in) {
            v = __ldg((const uint4*)(xsrc) + t);
            if (TIO) v = x8_as_f16(v, a.x_bf16);
        }
        if (in) {
            // k = 8t .. 8t+7: its two blocks of four go to positions xpos(8t) and xpos(8t + 4)
            *(uint2*)(xs + xpos(8u * t) * 2) = make_uint2(v.x, v.y);
            *(uint2*)(xs + xpos(8u * t + 4u) * 2) = make_uint2(v.z, v.w);
        }
        if (MODE != 0) {
            // 8 consecutive threads hold 64 consecutive k: sums of x over the halves of the super-chunks, in a fixed order
            const float2 p0 = __half22float2(*(const __half2*)&v.x), p1 = __half22float2(*(const __half2*)&v.y);
            const float2 p2 = __half22float2(*(const __half2*)&v.z), p3 = __half22float2(*(const __half2*)&v.w);
            float sx = ((p0.x + p0.y) + (p1.x + p1.y)) + ((p2.x + p2.y) + (p3.x + p3.y));
            sx += __shfl_xor_sync(0xffffffffu, sx, 1);
            sx += __shfl_xor_sync(0xffffffffu, sx, 2);
            sx += __shfl_xor_sync(0xffffffffu, sx, 4);
            if (in && (t & 7) == 0) xg[t >> 3] = sx;
        }
    }
    __syncthreads();   // tables and x visible
    lstamp(a, 3);

    const int g = lane >> 2, t4 = lane & 3;
    const bool dq = (g == t4) || (g == t4 + 4);
    const uint32_t base = (uint32_t)lane * (C::kQuad ? 8u : (kHalf ? 2u : 4u));
    // a diagonal lane reads 16 bytes per two mma steps: bytes [0,16) of every 32 for g == t, [16,32) for g == t + 4
    const unsigned char* xq = xs + (size_t)sc0 * (kSuper * 2) + ((g == t4 + 4) ? 16 : 0);

    float c[4] = {0.f, 0.f, 0.f, 0.f};
    float oacc = 0.f;   // outliers of the lane's channel; in V2a also the channel's folded group sums
    // V2a: where the two halves of this lane's group sum land in the fragment (see the end of the kernel)
    const int src_a = (lane & ~3) | (t4 >> 1);
    // the rows' slot counts have arrived: outlier rounds of this warp
    int width = (int)olen;
#pragma unroll
    for (int o = 16; o; o >>= 1) width = max(width, __shfl_xor_sync(0xffffffffu, width, o));
    width = min(width, ell_slots);
    const int mine = width > gw ? (width - gw + ostride - 1) / ostride : 0;
    const int nrounds = (mine + kLaneSlots - 1) / kLaneSlots;
    int oround = 0;
    auto consume_slots = [&]() {
#pragma unroll
        for (int q = 0; q < kLaneSlots; ++q) {
            const float v = h2f((uint16_t)(oe[q] >> 16));
            const uint32_t col = oe[q] & 0xffffu;
            oacc = fmaf(v, h2f(*(const uint16_t*)(xs + xpos(col) * 2)), oacc);
        }
    };
    auto fetch_slots = [&](int round) {
#pragma unroll
        for (int q = 0; q < kLaneSlots; ++q) {
            const int j = gw + (round * kLaneSlots + q) * ostride;
            oe[q] = j < width ? __ldg(slab + (size_t)(1 + j) * 32) : 0u;
        }
    };

    // ---- K loop: 16 mma steps per super-chunk, look-ups one step ahead of the tensor pipe; an index vector is
    //      reloaded with the same vector of this warp's next super-chunk as soon as its last step has been looked up
#pragma unroll 1
    for (int s = warp; s < nsc; s += W) {
        if (oround < nrounds) {
            consume_slots();
            if (++oround < nrounds) fetch_slots(oround);
        }
        const bool has_next = s + W < nsc;
        const uint4* nx = ip + (size_t)(s + W) * N * 32;
        const unsigned char* xp = xq + (size_t)s * (kSuper * 2);
        uint32_t fa[4], fb[4];
        uint4 xr = make_uint4(0u, 0u, 0u, 0u);
        uint32_t vbase = base;
        if (MODE != 0) {
            vbase = base + gid_c[0] * (uint32_t)kIdBytes;
            if (has_next) {   // metadata of the next super-chunk travels during this one
                const size_t mn = m0 + (size_t)(s + W) * GH * 32;
                gid_n[0] = b.gid[mn]; gsm_n[0] = b.gsm[mn];
                gid_n[1] = b.gid[mn + (size_t)(GH - 1) * 32]; gsm_n[1] = b.gsm[mn + (size_t)(GH - 1) * 32];
            }
        }
        // V2a: the group's sum leaves the fragment (two halves of the channel's sum sit in two other lanes of the
        // quad) and is folded with the group's scale and mid-point
        auto fold = [&](int h) {
            const float a0 = __shfl_sync(0xffffffffu, c[0], src_a), a1 = __shfl_sync(0xffffffffu, c[1], src_a);
            const float b2 = __shfl_sync(0xffffffffu, c[2], src_a + 2), b3 = __shfl_sync(0xffffffffu, c[3], src_a + 2);
            const float G = (t4 & 1) ? a1 + b3 : a0 + b2;
            const float scale = h2f((uint16_t)(gsm_c[h] & 0xffffu)), mid = h2f((uint16_t)(gsm_c[h] >> 16));
            const float X = GH == 2 ? xg[(sc0 + s) * 2 + h] : xg[(sc0 + s) * 2] + xg[(sc0 + s) * 2 + 1];
            oacc = fmaf(scale, G, fmaf(mid, X, oacc));
            c[0] = c[1] = c[2] = c[3] = 0.f;
        };
        lookup8<N, SGL, kHalf, C::kQuad>(fa, w, 0, tab, vbase);
#pragma unroll
        for (int j = 0; j < kSuper / 8; j += 2) {
            ld_x16_if(xr, xp + j * 16, dq);               // steps j and j + 1
            lookup8<N, SGL, kHalf, C::kQuad>(fb, w, j + 1, tab, vbase);
#pragma unroll
            for (int v = 0; v < N; ++v)
                if ((last_step_of_vector<N>(v) == j || last_step_of_vector<N>(v) == j + 1) && has_next) {
                    const uint4 t = ld_stream(nx + v * 32);
                    w[4 * v] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
                }
            mma16816(c, fa[0], fa[1], fa[2], fa[3], xr.x, xr.y);
            if (MODE != 0 && j + 2 == kSuper / 16) vbase = base + gid_c[1] * (uint32_t)kIdBytes;   // second half's library entry
            if (j + 2 < kSuper / 8) lookup8<N, SGL, kHalf, C::kQuad>(fa, w, j + 2, tab, vbase);
            mma16816(c, fb[0], fb[1], fb[2], fb[3], xr.z, xr.w);
            if (MODE != 0 && j + 2 == kSuper / 16 && GH == 2) fold(0);   // the first group of 64 weights is complete
        }
        if (MODE != 0) {
            fold(1);
            gid_c[0] = gid_n[0]; gid_c[1] = gid_n[1]; gsm_c[0] = gsm_n[0]; gsm_c[1] = gsm_n[1];
        }
    }
    while (oround < nrounds) {   // more outlier rounds than super-chunks
        consume_slots();
        if (++oround < nrounds) fetch_slots(oround);
    }
    // rows that fill their slab continue in the CSR arrays (pathological skew only): warp 0 of the first slice
    if (warp == 0 && slice == 0 && ell_slots && (int)olen >= ell_slots) {
        const int row = blk * kRowsPerBlock + lane;
        const int p1 = __ldg(b.rowptr + row + 1);
        for (int p = __ldg(b.rowptr + row) + ell_slots; p < p1; ++p) {
            const uint32_t e = __ldg(b.oent + p);
            oacc = fmaf(h2f((uint16_t)(e >> 16)), h2f(*(const uint16_t*)(xs + xpos(e & 0xffffu) * 2)), oacc);
        }
    }

    lstamp(a, 4);
    // ---- the two halves of a channel meet: lane (g, t < 2) holds D[g][2t], D[g][2t+1]; lane (g, t + 2) holds
    //      D[g+8][2t+4], D[g+8][2t+5]; then channel order through shared memory
    if (MODE != 0) {
        red[warp * 32 + lane] = oacc;   // every lane already owns its channel's sum
    } else {
        const float h2 = __shfl_xor_sync(0xffffffffu, c[2], 2), h3 = __shfl_xor_sync(0xffffffffu, c[3], 2);
        float* r = red + (size_t)warp * 32;
        if (t4 < 2) *(float2*)(r + 4 * g + 2 * t4) = make_float2(c[0] + h2, c[1] + h3);
        __syncwarp();
        r[lane] += oacc;
    }
    __syncthreads();

    // ---- fixed-order sum over the warps, then store or combine the block's slices
    const int t = threadIdx.x;
    const bool active = t < 32;
    const int row = blk * 32 + t;       // channel inside its blob (y index)
    const int wrow = gblk * 32 + t;     // channel inside the launch (workspace index)
    float total = 0.f;
    if (active) {
#pragma unroll
        for (int ww = 0; ww < W; ++ww) total += red[ww * 32 + t];
    }
    bool writer = true;
    if (nslices > 1) {
        __shared__ int s_last;
        if (active) a.partial[(size_t)slice * a.rows_ws + wrow] = total;
        __threadfence();
        __syncthreads();
        if (t == 0) s_last = (atomicAdd(a.tickets + gblk, 1) == nslices - 1);
        __syncthreads();
        writer = s_last != 0;
        if (writer) {
            __threadfence();
            if (active) {
                total = 0.f;
                for (int k2 = 0; k2 < nslices; ++k2) total += __ldcg(a.partial + (size_t)k2 * a.rows_ws + wrow);
            }
            if (t == 0) a.tickets[gblk] = 0;
        }
    }
        if (writer && active && row < a.rows) store_y<TIO>(ydst, (size_t)row, total, a.y_is_fp16);
    lstamp(a, 5);
}

#ifdef XFP_TRACE
unsigned long long* g_lane_trace = nullptr;
size_t g_lane_trace_calls = 0, g_lane_trace_idx = 0;
#endif

struct LaneSchedule {
    int grid;
    int tier_cta[5], tier_blk[4], tier_kst[4], tier_spp[4];
};

int pow2_floor_(int v) {
    int p = 1;
    while (p * 2 <= v) p *= 2;
    return p;
}

// Whole-K blocks fill whole rounds of CTA slots; the blocks of the last partial round are cut along K in tiers of
// finer slices (the hardware dispatches CTAs in launch order, so the tiers pack the slots largest-first).  A matrix
// with no more blocks than SMs runs one unsplit block per SM and leaves the other half of every SM to the next call.
LaneSchedule lane_schedule(const Layout& l, int blocks, int per_sm, bool tiers) {
    LaneSchedule sc{};
    const int sms = sched_sms();
    const int S = sms * per_sm;
    const int kmax = l.SC / 4 > 1 ? pow2_floor_(l.SC / 4) : 1;   // keep K slices of at least 512 weights
    int nb[4] = {0, 0, 0, 0}, kk[4] = {1, 1, 1, 1};
    int nt = 0;
    if (blocks * 2 <= sms) {
        int kst = 1;
        while (kst < 8 && blocks * kst * 2 <= sms && kst * 2 <= kmax) kst *= 2;
        nb[0] = blocks; kk[0] = kst; nt = 1;
    } else if (blocks <= S || !tiers) {
        // one (partial) round, or a few rounds of unsplit blocks that the hardware deals to the slots as they free up
        nb[0] = blocks; kk[0] = 1; nt = 1;
    } else {
        const int full = (blocks / S) * S;
        int remaining = blocks - full;
        nb[nt] = full; kk[nt] = 1; ++nt;
        int k = 2;
        while (remaining > 0 && nt < 4) {
            if (k > kmax) { nb[nt] = remaining; kk[nt] = kmax; ++nt; remaining = 0; break; }
            const int cap = S / k;   // blocks whose k slices fill one round
            if (remaining <= cap || nt == 3) {
                int kl = pow2_floor_(S / remaining > 1 ? S / remaining : 1);
                if (kl > kmax) kl = kmax;
                if (kl > 64) kl = 64;
                if (kl < k && remaining <= cap) kl = k;
                nb[nt] = remaining; kk[nt] = kl < 1 ? 1 : kl; ++nt; remaining = 0;
            } else {
                nb[nt] = cap; kk[nt] = k; ++nt; remaining -= cap;
                k *= 2;
            }
        }
    }
    int cta = 0, blk = 0;
    for (int i = 0; i < 4; ++i) {
        sc.tier_cta[i] = cta; sc.tier_blk[i] = blk;
        int kst = i < nt ? kk[i] : 1;
        if (kst > l.SC) kst = l.SC;
        const int spp = (l.SC + kst - 1) / kst;
        sc.tier_spp[i] = spp;
        sc.tier_kst[i] = (l.SC + spp - 1) / spp;
        if (i < nt) { cta += nb[i] * sc.tier_kst[i]; blk += nb[i]; }
    }
    sc.tier_cta[4] = cta;
    for (int i = nt; i < 4; ++i) sc.tier_cta[i] = 0x7fffffff;   // unused tiers never match
    sc.grid = cta;
    return sc;
}

// ---- launch configurations: warps per CTA, CTAs per SM (64 registers per thread at 16 x 2), single-entry tables
struct LaneConfig { int W, per_sm; bool sgl; bool off = false; bool tiers = true; };

size_t lane_tab_bytes(const Layout& l, bool sgl) {
    const int bits = l.bits;
    const size_t E = (size_t)1 << bits;
    if (l.mode) {   // the library, one copy per bank: a word per entry (per pair of entries), or half a word when that does not fit
        if (!sgl) return (size_t)l.L * E * E * 128;
        const size_t full = (size_t)l.L * E * 128;
        return full <= 128 * 1024 ? full : full / 2;
    }
    if (bits == 2) return 256 * 256;
    if (sgl) return E * 128;
    return E * E * (bits == 4 ? 256 : 128);
}

size_t lane_smem_bytes(const Layout& l, const LaneConfig& c) {
    // tables | x | red [W][32] | V2a: sums of x per half super-chunk; V2: the block's codebooks for the table fill
    return lane_tab_bytes(l, c.sgl) + (size_t)l.cols * 2 + (size_t)c.W * 32 * 4 + (l.mode ? (size_t)l.SC * 8 : (size_t)l.E * 64);
}

// `RBn`: row-blocks of the launch (all blobs)
LaneConfig lane_config(const Layout& l, int n = 1) {
    const long long RB = (long long)l.RB * n;
#ifdef LANE_TUNE
    if (const char* e = getenv("XFP_LANE_CFG")) {   // tuning build: "W,per_sm,sgl"
        int w = 16, p = 1, g = 0;
        sscanf(e, "%d,%d,%d", &w, &p, &g);
        if (w == 0) return LaneConfig{16, 1, false, true};
        return LaneConfig{w, p > 2 ? 2 : p, l.mode == 1 || l.bits == 6 || (l.bits == 5 && g), false, p <= 2};
    }
#endif
    // Measured on B200 over 4096 x 4096 .. 28672 x 8192 at every bit width (microseconds per call, graph replay):
    //  * no more row-blocks than SMs: one CTA of 16 warps per SM with all 128 registers (the K loop is bound by the
    //    latency of a warp's own look-ups, and two CTAs of one launch on an SM would only serialise)
    //  * more: two CTAs per SM, 8 warps (16 at N = 3, 4 on mid-sized matrices); the blocks of a matrix of up to four
    //    rounds run unsplit (cutting the tail along K cost more than the idle slots), larger ones cut their last round
    //  * N = 5 beyond one round: one entry per index instead of the 128 KB pair table, whose fill per 32 channels
    //    costs as much as 2048 weights of look-ups and cannot overlap anything with one CTA per SM
    const int sms = sched_sms();
    if (l.mode) {
        // V2a: one look-up per weight in the per-bank library.  Up to 64 KB of tables (L * 2^N <= 512) two CTAs fit.
        // Pair tables of the whole library where they fit the same 64 KB (L * 4^N <= 512: N = 2 with the paper's L = 32).
        const bool pairs = (size_t)l.L * l.E * l.E * 128 <= 64 * 1024 && l.bits <= 3;
        const bool two = lane_tab_bytes(l, !pairs) <= 64 * 1024 && RB > sms;
        LaneConfig c{two ? 8 : 16, two ? 2 : 1, !pairs};
        c.tiers = RB > 4 * sms || !two;
        // a 128 KB library (N = 5) leaves one CTA per SM: between one and four rounds the kernel with two channels
        // per lane (xfp_gemv_v2a.cu) measured faster
        const bool half_words = (size_t)l.L * l.E * 128 > 128 * 1024;   // no kernel with two channels per lane for these
        c.off = !two && !half_words && RB > sms && RB <= 4 * sms;
        // the blobs of a routed layer in one launch: the resident CTAs of xfp_gemv_v2a.cu (pair tables built once per
        // SM at N <= 3) measured faster (gate_up 30.7 vs 33.4 us, down 18.7 vs 22.9 us per launch of 8 experts)
        if (n > 1) c.off = true;
        return c;
    }
    if (RB <= sms) return LaneConfig{16, 1, l.bits == 6};
    const bool big = RB > 4 * sms;
    LaneConfig c{(!big && (l.bits == 3 || l.bits == 4)) ? 16 : 8, 2, l.bits >= 5};
    c.off = big && l.bits <= 3;   // the two-channels-per-lane kernel is ahead there
    c.tiers = big;
    return c;
}

template <int N, int W, int MINB, bool SGL, int MODE, bool TIO>
cudaError_t launch_lane_io(const LaneArgs& a, int grid, size_t smem, cudaStream_t s) {
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemv_lane_kernel<N, W, MINB, SGL, MODE, TIO>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             MINB == 1 ? 224 * 1024 : 110 * 1024);
        if (e != cudaSuccess) return e;
        attr_done.set(dev);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(W * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_lane_kernel<N, W, MINB, SGL, MODE, TIO>, a);
}

template <int N, int W, int MINB, bool SGL, int MODE>
cudaError_t launch_lane(const LaneArgs& a, int grid, size_t smem, cudaStream_t s) {
    if (a.x_bf16 || a.y_is_fp16 == 2) return launch_lane_io<N, W, MINB, SGL, MODE, true>(a, grid, smem, s);
    return launch_lane_io<N, W, MINB, SGL, MODE, false>(a, grid, smem, s);
}

template <int N, bool SGL, int MODE>
cudaError_t launch_lane_cfg(const LaneConfig& c, const LaneArgs& a, int grid, size_t smem, cudaStream_t s) {
    if (c.W == 8) return launch_lane<N, 8, 2, SGL, MODE>(a, grid, smem, s);
    if (c.per_sm >= 2) return launch_lane<N, 16, 2, SGL, MODE>(a, grid, smem, s);
    return launch_lane<N, 16, 1, SGL, MODE>(a, grid, smem, s);
}

}  // namespace

// batch 1 (fp16 or bf16 x, any y type), one blob or several, no fused store; x short enough to stage beside the tables
bool lane_supported(const Layout& l, const GemvCall& c) {
    if (c.batch != 1 || c.n < 1 || c.epilogue != 0) return false;
    if ((c.n > 1) != (c.packed_list != nullptr)) return false;
    if (l.bits < 2 || l.bits > 6) return false;
    if (l.mode && (size_t)l.L * l.E * 64 > 128 * 1024) return false;   // V2a: the per-bank library must fit 128 KB
    const LaneConfig cfg = lane_config(l, c.n);
    if (cfg.off) return false;
    return lane_smem_bytes(l, cfg) <= (cfg.per_sm == 1 ? 220u : 110u) * 1024u;
}

cudaError_t launch_gemv_lane(const Layout& l, const GemvCall& c, cudaStream_t s) {
    const LaneConfig cfg = lane_config(l, c.n);
    const LaneSchedule sch = lane_schedule(l, l.RB * c.n, cfg.per_sm, cfg.tiers);
    LaneArgs a{};
    a.off = offsets_of(l);
    a.packed = c.packed; a.x = c.x; a.y = c.y;
    a.packed_list = c.packed_list; a.x_list = c.x_list; a.y_list = c.y_list;
    a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.ell_slots = l.ell_slots;
    a.rows_ws = l.RB * c.n * 32;
    a.y_is_fp16 = c.y_is_fp16; a.x_bf16 = c.x_bf16;
    a.tab_bytes = (int)lane_tab_bytes(l, cfg.sgl);
    a.L = l.L; a.GH = l.GH;
    for (int i = 0; i < 5; ++i) a.tier_cta[i] = sch.tier_cta[i];
    for (int i = 0; i < 4; ++i) { a.tier_blk[i] = sch.tier_blk[i]; a.tier_kst[i] = sch.tier_kst[i]; a.tier_spp[i] = sch.tier_spp[i]; }
    a.tickets = (int*)c.workspace;
    a.partial = (float*)((char*)c.workspace + align256((size_t)l.RB * 4 * c.n));
#ifdef XFP_TRACE
    a.trace = nullptr;
    if (g_lane_trace && g_lane_trace_idx < g_lane_trace_calls) a.trace = g_lane_trace + (g_lane_trace_idx++) * 1024 * 8;
#endif
    const size_t smem = lane_smem_bytes(l, cfg);
    if (l.mode && (size_t)l.L * l.E * 128 > 128 * 1024) {
        // two bytes per lane and entry (lanes 2j and 2j+1 share a bank: a look-up costs two wavefronts when their
        // entries differ): N = 6 with L = 32, which the paper's own V2a kernel does not have
        switch (l.bits) {
            case 4: return launch_lane<4, 16, 1, true, 2>(a, sch.grid, smem, s);
            case 5: return launch_lane<5, 16, 1, true, 2>(a, sch.grid, smem, s);
            case 6: return launch_lane<6, 16, 1, true, 2>(a, sch.grid, smem, s);
            default: return cudaErrorInvalidValue;
        }
    }
    if (l.mode) {
        switch (l.bits) {
            case 2: return cfg.sgl ? launch_lane_cfg<2, true, 1>(cfg, a, sch.grid, smem, s)
                                   : launch_lane_cfg<2, false, 1>(cfg, a, sch.grid, smem, s);
            case 3: return cfg.sgl ? launch_lane_cfg<3, true, 1>(cfg, a, sch.grid, smem, s)
                                   : launch_lane_cfg<3, false, 1>(cfg, a, sch.grid, smem, s);
            case 4: return launch_lane_cfg<4, true, 1>(cfg, a, sch.grid, smem, s);
            default: return launch_lane_cfg<5, true, 1>(cfg, a, sch.grid, smem, s);
        }
    }
    switch (l.bits) {
        case 2: return launch_lane_cfg<2, false, 0>(cfg, a, sch.grid, smem, s);
        case 3: return launch_lane_cfg<3, false, 0>(cfg, a, sch.grid, smem, s);
        case 4: return launch_lane_cfg<4, false, 0>(cfg, a, sch.grid, smem, s);
        case 5: return cfg.sgl ? launch_lane_cfg<5, true, 0>(cfg, a, sch.grid, smem, s)
                               : launch_lane_cfg<5, false, 0>(cfg, a, sch.grid, smem, s);
        default: return launch_lane_cfg<6, true, 0>(cfg, a, sch.grid, smem, s);
    }
}

#ifdef XFP_TRACE
// timing build only: where the next `calls` launches put their stamps (1024 CTAs x 8 stamps each)
extern "C" void xfp_trace_lane(void* p, size_t calls) {
    g_lane_trace = (unsigned long long*)p;
    g_lane_trace_calls = calls;
    g_lane_trace_idx = 0;
}
#endif

}  // namespace xfp
