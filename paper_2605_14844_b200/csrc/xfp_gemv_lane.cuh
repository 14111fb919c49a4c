// The batch-1 decode kernel and its form for several rows of x, shared by xfp_gemv_lane.cu (one row) and
// xfp_gemv_lane_batch.cu (2, 4, 8 rows): kernel template, its arguments and launcher.  See xfp_gemv_lane.cu for
// the design.
#pragma once
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
    int batch;       // rows of x ([batch][cols]) and of y ([batch][rows])
    int y_is_fp16;   // type of y: 0 fp32, 1 fp16, 2 bf16
    int x_bf16;      // x holds bf16: converted to fp16 while it is staged
    int tab_bytes;   // shared-memory bytes of the look-up tables
    int L, GH;       // V2a: library size; groups per super-chunk (2 when the format's groups hold 64 weights)
    // schedule tiers: CTAs [tier_cta[i], tier_cta[i+1]) handle blocks from tier_blk[i] on, each cut into
    // tier_kst[i] slices of tier_spp[i] super-chunks.
    // Kernels for several rows of x keep their CTAs resident instead (x is staged once per CTA): CTA c takes the work
    // items c, c + grid, ...; items below tier_blk[0] are whole blocks, item tier_blk[0] + j < tier_blk[0] + tier_cta[1]
    // is slice j % tier_kst[0] of block tier_blk[0] + j / tier_kst[0].
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

// The four A registers of mma step j (weights 8j .. 8j+7 of the lane's channel in this super-chunk).
template <int N, bool SGL, bool HALF, bool QUAD>
__device__ __forceinline__ void lookup8(uint32_t (&f)[4], const uint32_t* w, int j, const unsigned char* tab,
                                        uint32_t base) {
    if (HALF) {
        // V2a, one entry per index: a word holds the entry of TWO library ids, `base` selects the half
        uint32_t e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = *(const uint16_t*)(tab + single_addr<N, 1>(w, 8 * j + i, base));
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

// V2 tables of one row-block: warp w fills entries [w T / W, (w+1) T / W) of every lane's channel (the table shapes are
// listed at the top of xfp_gemv_lane.cu).  `cbs`: scratch for the block's codebooks (N >= 5).  Every thread of the CTA
// calls it (N >= 5 has a barrier inside).
template <int N, int W, bool SGL>
__device__ __forceinline__ void fill_tables_v2(unsigned char* tab, uint32_t* cbs, const Blob& b, int blk, int warp, int lane) {
    using C = LaneCfg<N, SGL, 0>;
    constexpr int E = C::E;
    constexpr int T = C::T;
    constexpr int kStride = C::kStride;
    constexpr int kThreads = W * 32;
    const uint16_t* cb = b.cb + (size_t)(blk * kRowsPerBlock + lane) * E;
    if constexpr (C::kQuad) {
        // entry t = (cb[t & 3], cb[t >> 2 & 3], cb[t >> 4 & 3], cb[t >> 6]) as 8 bytes at t * 256 + lane * 8
        const uint2 c4 = __ldg((const uint2*)cb);   // the four entries
        const uint32_t e0 = c4.x & 0xffffu, e1 = c4.x >> 16, e2 = c4.y & 0xffffu, e3 = c4.y >> 16;
        auto ent = [&](int q) { return q == 0 ? e0 : (q == 1 ? e1 : (q == 2 ? e2 : e3)); };
        // entries t = 16 h + i: the high half (indices 2, 3 of the byte) is the same for sixteen entries and is
        // picked once; the low half runs over all sixteen pairs with compile-time picks (selecting all four values
        // of every entry at run time made this fill 1.15 us, the longest prologue of all widths)
        const uint32_t eh[4] = {e0 << 16, e1 << 16, e2 << 16, e3 << 16};
        const uint32_t el[4] = {e0, e1, e2, e3};
        constexpr int TW = T / W;
        static_assert(TW % 16 == 0, "a warp fills whole groups of sixteen entries");
#pragma unroll
        for (int gq = 0; gq < TW / 16; ++gq) {
            const int h = warp * (TW / 16) + gq;
            const uint32_t hi = ent(h & 3) | (ent(h >> 2) << 16);
#pragma unroll
            for (int i = 0; i < 16; ++i)
                *(uint2*)(tab + (size_t)(h * 16 + i) * kStride + lane * 8) = make_uint2(el[i & 3] | eh[i >> 2], hi);
        }
    } else if constexpr (C::kSingle && (T / W == 2 || T / W == 4 || T / W == 8)) {
        // a warp's TW consecutive entries of every channel in ONE load per lane (2, 4 or 8 entries: 4, 8 or 16 bytes;
        // one 2-byte load per entry made four requests of 32 sectors each and the fill 1.2 us at N = 6)
        constexpr int TW = T / W;
        uint32_t cw[TW / 2];
        if (TW == 2) {
            cw[0] = __ldg((const uint32_t*)(cb + warp * TW));
        } else if (TW == 4) {
            const uint2 t = __ldg((const uint2*)(cb + warp * TW));
            cw[0] = t.x; cw[TW / 2 - 1] = t.y;
        } else {
            const uint4 t = __ldg((const uint4*)(cb + warp * TW));
            cw[0] = t.x; cw[1 % (TW / 2)] = t.y; cw[2 % (TW / 2)] = t.z; cw[3 % (TW / 2)] = t.w;
        }
#pragma unroll
        for (int i = 0; i < TW; ++i) {
            const int t = warp * TW + i;
            *(uint32_t*)(tab + (size_t)t * kStride + lane * 4) = (i & 1) ? (cw[i >> 1] >> 16) : (cw[i >> 1] & 0xffffu);
        }
    } else if (C::kSingle) {   // (instantiated for V2a widths only, where this branch is never taken)
        constexpr int TW = T / W > 0 ? T / W : 1;
#pragma unroll
        for (int i = 0; i < TW; ++i) {
            const int t = warp * TW + i;
            if (t < T) *(uint32_t*)(tab + (size_t)t * kStride + lane * 4) = (uint32_t)__ldg(cb + t);
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

// V2a tables: every row is one word repeated in the 32 banks -- HALF: row (id / 2) * 2^N + q holds lib[id][q] of ids
// 2m (low half) and 2m + 1 (high half); else the pair table, row id * 4^N + (q1 << N | q0) holds (lib[id][q0],
// lib[id][q1]).  A lane fetches the word of row e0 + lane, then the warp stores the 32 rows one after the other, each word
// handed round by a shuffle (a warp that fetched two halves per row with uniform loads paid their latency once per
// row: 3.9 us for the 1024 rows of N = 6).  Not inlined: inside the kernel the unrolled stores changed the register
// allocation of the K loop (N = 3, 4: 62.2 against 58.3 us at 28672 x 8192).
template <int N, int W, bool HALF>
__device__ __noinline__ void fill_library(unsigned char* tab, const uint16_t* __restrict__ lib, int L, int warp, int lane) {
    constexpr int E = 1 << N;
    const int trows = HALF ? ((L + 1) >> 1) * E : L * E * E;
    if (HALF && trows < 32 * W) {
        // a small table (N = 3, 4 at L = 32): one row per warp and step, so that every warp takes part
        for (int e = warp; e < trows; e += W) {
            const int m = e >> N, q = e & (E - 1);
            const uint32_t lo = __ldg(lib + (size_t)(2 * m) * E + q);
            const uint32_t hi = 2 * m + 1 < L ? (uint32_t)__ldg(lib + (size_t)(2 * m + 1) * E + q) : 0u;
            *(uint32_t*)(tab + (size_t)e * 128 + lane * 4) = lo | (hi << 16);
        }
        return;
    }
    for (int e0 = warp * 32; e0 < trows; e0 += W * 32) {
        const int e = e0 + lane;
        uint32_t word = 0u;
        if (e < trows) {
            if (HALF) {
                const int m = e >> N, q = e & (E - 1);
                word = __ldg(lib + (size_t)(2 * m) * E + q);
                if (2 * m + 1 < L) word |= (uint32_t)__ldg(lib + (size_t)(2 * m + 1) * E + q) << 16;
            } else {
                const uint16_t* cb = lib + (size_t)(e >> (2 * N)) * E;
                word = (uint32_t)__ldg(cb + (e & (E - 1))) | ((uint32_t)__ldg(cb + ((e >> N) & (E - 1))) << 16);
            }
        }
#pragma unroll
        for (int r = 0; r < 32; ++r) {
            const uint32_t v = __shfl_sync(0xffffffffu, word, r);
            if (e0 + r < trows) *(uint32_t*)(tab + (size_t)(e0 + r) * 128 + lane * 4) = v;
        }
    }
}

// MODE 0: V2 (the channel's own codebook, tables private to the lane).  MODE 1: V2a -- the whole library replicated
// once per bank (word ((id / 2) * 2^N + q) * 32 + lane holds lib[id][q] in its half id % 2; pair tables of every
// entry where those fit), the table base of a lane follows the library id
// of its channel's current group, the fragment accumulates sum lib * x of ONE group, and after the group's steps the
// sum moves to the lane that owns the channel and is folded into its accumulator with the group's scale and
// mid-point:  acc += scale * G + mid * X_g,  X_g = sum of x over the group ("V2a: Shared Codebook Library").
// TIO instantiations take bf16 x and store bf16 y; compiled into the plain ones the conversion cost the fp16 path 4.5 %
// at 28672 x 8192 through register allocation alone (34.3 against 32.8 us), so only bf16 calls launch them.  The same
// instantiations serve launches over several blobs (pointer lists): with the list branch compiled into the plain
// ones, the blob's pointers were run-time values instead of kernel parameters and 12288 x 4096 at N = 2 took 11.8
// against 8.4 us.
// NB rows of x (1, 2, 4 or 8): every decoded fragment is multiplied with the B fragment of each row, so the look-ups
// are paid once per weight; a CTA then stays resident and walks several row-blocks with one staged copy of x.
template <int N, int W, int MINB, bool SGL, int MODE, bool TIO, int NB>
__global__ void __launch_bounds__(W * 32, MINB) gemv_lane_kernel(const LaneArgs a) {
    using C = LaneCfg<N, SGL, MODE>;
    constexpr int E = C::E;
    // V2a with a small library (L * 4^N words per bank fit): PAIR tables of every library entry, one look-up per two
    // weights as in V2
    constexpr bool kLibPair = MODE == 1 && !SGL;
    // V2a otherwise: one entry per index, and the word of a bank holds that entry of TWO library ids (2m in the low
    // half, 2m + 1 in the high half): every lane still reads its own bank, whatever ids and indices the lanes hold,
    // and the tables are half as large (64 KB at N = 5, 128 KB at N = 6 with L = 32)
    constexpr bool kHalf = MODE == 1 && SGL;
    constexpr int kIdBytes = (kLibPair ? E * E : E) * 128;   // V2a: bytes between the tables of two ids (kHalf: id pairs)
    constexpr int T = C::T;
    constexpr int kStride = C::kStride;
    constexpr int kThreads = W * 32;
    constexpr bool kMulti = NB > 1;          // resident CTA over several row-blocks
    constexpr int RH = NB < 4 ? NB : 4;      // rows of x whose B registers are live at a time
    static_assert(NB * 32 <= kThreads, "one thread per channel and row of x in the final sum");
    extern __shared__ __align__(16) unsigned char smem[];
    // [tables | x fp16 [NB][K] permuted | red [NB][W][32] | V2a: sums of x; V2: codebooks for the fill]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    lstamp(a, 0);
    const int K = a.SC * kSuper;
    const size_t xrow = (size_t)K * 2;             // bytes of one staged row of x
    unsigned char* tab = smem;
    // V2, N >= 4: a compile-time offset (4096 x 4096, N = 5: 4.70 against 4.86 us; at N = 3 the same change cost 6 % at
    // 12288 x 4096 through register allocation, so N <= 3 keeps the run-time one)
    unsigned char* xs = smem + (MODE == 0 && N >= 4 ? C::kTabBytes : a.tab_bytes);
    float* red = (float*)(xs + NB * xrow);         // [NB][W][32]
    float* xg = red + NB * W * 32;                 // V2a: [NB][SC][2] sums of x over the halves of every super-chunk
    uint32_t* cbs = (uint32_t*)xg;                 // V2 pair tables: the block's codebooks, word [e / 2][channel]
    const int g = lane >> 2, t4 = lane & 3;
    const bool dq = (g == t4) || (g == t4 + 4);
    const uint32_t base = (uint32_t)lane * (C::kQuad ? 8u : 4u);
    // V2a: where the two halves of this lane's group sum land in the fragment (see the end of the kernel)
    const int src_a = (lane & ~3) | (t4 >> 1);
    // V2a: table offset of library id `id`
    auto id_offset = [](uint32_t id) -> uint32_t {
        return kHalf ? (id >> 1) * (uint32_t)kIdBytes + (id & 1u) * 2u : id * (uint32_t)kIdBytes;
    };

#pragma unroll 1
    for (int it = 0;; ++it) {
    // ---- this CTA's block and K slice
    int blk, slice, nslices, sc0, nsc;
    if (kMulti) {
        const int v = it * (int)gridDim.x + (int)blockIdx.x;
        if (v < a.tier_blk[0]) {
            blk = v; slice = 0; nslices = 1; sc0 = 0; nsc = a.SC;
        } else {
            const int c = v - a.tier_blk[0];   // the K slices of the remaining blocks are dealt the same way
            if (c >= a.tier_cta[1]) break;
            nslices = a.tier_kst[0];
            blk = a.tier_blk[0] + c / nslices;
            slice = c - (c / nslices) * nslices;
            sc0 = slice * a.tier_spp[0];
            nsc = max(0, min(a.SC, sc0 + a.tier_spp[0]) - sc0);
        }
        if (it > 0) __syncthreads();   // the previous block's tables and sums are no longer read
    } else {
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
    if (TIO && a.packed_list) {
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
    const uint32_t* ell = (TIO && a.packed_list)
        ? (const uint32_t*)((const char*)packed + *(const long long*)((const char*)packed + a.off.hdr + 8)) : b.ell;
    const uint32_t* slab = ell + (size_t)blk * (ell_slots + 1) * 32 + lane;
    uint32_t olen = ell_slots ? __ldg(slab) : 0u;
    uint32_t oe[kLaneSlots];
#pragma unroll
    for (int q = 0; q < kLaneSlots; ++q) {
        const int j = gw + q * ostride;
        oe[q] = j < ell_slots ? __ldg(slab + (size_t)(1 + j) * 32) : 0u;   // every slot below the capacity is readable
    }
    lstamp(a, 6);
    // ---- tables: warp w fills entries [w T / W, (w+1) T / W) of every lane's channel
    if (MODE != 0) {
        if (!kMulti || it == 0) {   // one library per blob: a resident CTA fills it once
        if constexpr (N >= 5 || kLibPair || W == 8) {
            fill_library<N, W, kHalf>(tab, b.cb, a.L, warp, lane);
        } else {
            // small tables in a CTA that has its SM to itself: inline, so that the index loads issued above stay in
            // flight (registers that are the target of a load are written back around a call, which waits for them:
            // 4096 x 4096, N = 4: 6.99 against 6.66 us)
            if (a.L == 32) {
                // the paper's library size: a known trip count, so that all of a warp's loads are in flight at once
                constexpr int kRows = 16 * E / W;
                uint32_t lo[kRows], hi[kRows];
#pragma unroll
                for (int i = 0; i < kRows; ++i) {
                    const int e = warp + i * W, m = e >> N, q = e & (E - 1);
                    lo[i] = __ldg(b.cb + (size_t)(2 * m) * E + q);
                    hi[i] = __ldg(b.cb + (size_t)(2 * m + 1) * E + q);
                }
#pragma unroll
                for (int i = 0; i < kRows; ++i)
                    *(uint32_t*)(tab + (size_t)(warp + i * W) * 128 + lane * 4) = lo[i] | (hi[i] << 16);
            } else {
                for (int e = warp; e < ((a.L + 1) >> 1) * E; e += W) {
                    const int m = e >> N, q = e & (E - 1);
                    const uint32_t lo = __ldg(b.cb + (size_t)(2 * m) * E + q);
                    const uint32_t hi = 2 * m + 1 < a.L ? (uint32_t)__ldg(b.cb + (size_t)(2 * m + 1) * E + q) : 0u;
                    *(uint32_t*)(tab + (size_t)e * 128 + lane * 4) = lo | (hi << 16);
                }
            }
        }
        }
    } else {
        // inlined: behind a call (as the V2a fill of the 8-warp CTAs is) the same K loops ran 7-11 % slower
        // (28672 x 8192: N = 4 36.9 against 34.1 us, N = 5 55.6 against 49.9 us)
        fill_tables_v2<N, W, SGL>(tab, cbs, b, blk, warp, lane);
    }

    // ---- x may come from the previous kernel of the stream
    lstamp(a, 1);
    if (!kMulti || it == 0) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    lstamp(a, 2);
#pragma unroll 1
    for (int r = 0; r < NB; ++r) {
        const bool have = r < a.batch;   // rows beyond the batch are staged as zeros
        const uint4* xrsrc = (const uint4*)(xsrc + (size_t)r * a.cols);
        unsigned char* xd = xs + r * xrow;
        for (int t = threadIdx.x; t < ((K / 8 + 31) & ~31); t += kThreads) {   // whole warps: the sums below shuffle
            const bool in = t < K / 8;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (in && have) {
                v = __ldg(xrsrc + t);
                if (TIO) v = x8_as_f16(v, a.x_bf16);
            }
            if (in) {
                // k = 8t .. 8t+7: its two blocks of four go to positions xpos(8t) and xpos(8t + 4)
                *(uint2*)(xd + xpos(8u * t) * 2) = make_uint2(v.x, v.y);
                *(uint2*)(xd + xpos(8u * t + 4u) * 2) = make_uint2(v.z, v.w);
            }
            if (MODE != 0) {
                // 8 consecutive threads hold 64 consecutive k: sums of x over the halves of the super-chunks, in a fixed order
                const float2 p0 = __half22float2(*(const __half2*)&v.x), p1 = __half22float2(*(const __half2*)&v.y);
                const float2 p2 = __half22float2(*(const __half2*)&v.z), p3 = __half22float2(*(const __half2*)&v.w);
                float sx = ((p0.x + p0.y) + (p1.x + p1.y)) + ((p2.x + p2.y) + (p3.x + p3.y));
                sx += __shfl_xor_sync(0xffffffffu, sx, 1);
                sx += __shfl_xor_sync(0xffffffffu, sx, 2);
                sx += __shfl_xor_sync(0xffffffffu, sx, 4);
                if (in && (t & 7) == 0) xg[r * a.SC * 2 + (t >> 3)] = sx;
            }
        }
    }
    }
    __syncthreads();   // tables and x visible
    lstamp(a, 3);

    // a diagonal lane reads 16 bytes per two mma steps: bytes [0,16) of every 32 for g == t, [16,32) for g == t + 4
    const unsigned char* xq = xs + (size_t)sc0 * (kSuper * 2) + ((g == t4 + 4) ? 16 : 0);

    float c[NB][4];
    float oacc[NB];   // outliers of the lane's channel; in V2a also the channel's folded group sums
#pragma unroll
    for (int r = 0; r < NB; ++r) { c[r][0] = c[r][1] = c[r][2] = c[r][3] = 0.f; oacc[r] = 0.f; }
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
            const unsigned char* xo = xs + xpos(oe[q] & 0xffffu) * 2;
#pragma unroll
            for (int r = 0; r < NB; ++r) oacc[r] = fmaf(v, h2f(*(const uint16_t*)(xo + r * xrow)), oacc[r]);
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
        uint4 xr[RH];
#pragma unroll
        for (int r = 0; r < RH; ++r) xr[r] = make_uint4(0u, 0u, 0u, 0u);
        uint32_t vbase = base;
        if (MODE != 0) {
            vbase = base + id_offset(gid_c[0]);
            if (has_next) {   // metadata of the next super-chunk travels during this one
                const size_t mn = m0 + (size_t)(s + W) * GH * 32;
                gid_n[0] = b.gid[mn]; gsm_n[0] = b.gsm[mn];
                gid_n[1] = b.gid[mn + (size_t)(GH - 1) * 32]; gsm_n[1] = b.gsm[mn + (size_t)(GH - 1) * 32];
            }
        }
        // V2a: the group's sum leaves the fragment (two halves of the channel's sum sit in two other lanes of the
        // quad) and is folded with the group's scale and mid-point
        auto fold = [&](int h) {
            const float scale = h2f((uint16_t)(gsm_c[h] & 0xffffu)), mid = h2f((uint16_t)(gsm_c[h] >> 16));
#pragma unroll
            for (int r = 0; r < NB; ++r) {
                const float a0 = __shfl_sync(0xffffffffu, c[r][0], src_a), a1 = __shfl_sync(0xffffffffu, c[r][1], src_a);
                const float b2 = __shfl_sync(0xffffffffu, c[r][2], src_a + 2), b3 = __shfl_sync(0xffffffffu, c[r][3], src_a + 2);
                const float G = (t4 & 1) ? a1 + b3 : a0 + b2;
                const float* xgr = xg + (r * a.SC + sc0 + s) * 2;
                const float X = GH == 2 ? xgr[h] : xgr[0] + xgr[1];
                oacc[r] = fmaf(scale, G, fmaf(mid, X, oacc[r]));
                c[r][0] = c[r][1] = c[r][2] = c[r][3] = 0.f;
            }
        };
        lookup8<N, SGL, kHalf, C::kQuad>(fa, w, 0, tab, vbase);
#pragma unroll
        for (int j = 0; j < kSuper / 8; j += 2) {
            if (NB <= RH) {
#pragma unroll
                for (int r = 0; r < NB; ++r) ld_x16_if(xr[r], xp + r * xrow + j * 16, dq);   // steps j and j + 1
            }
            lookup8<N, SGL, kHalf, C::kQuad>(fb, w, j + 1, tab, vbase);
#pragma unroll
            for (int v = 0; v < N; ++v)
                if ((last_step_of_vector<N>(v) == j || last_step_of_vector<N>(v) == j + 1) && has_next) {
                    const uint4 t = ld_stream(nx + v * 32);
                    w[4 * v] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
                }
            if (NB <= RH) {
#pragma unroll
                for (int r = 0; r < NB; ++r) mma16816(c[r], fa[0], fa[1], fa[2], fa[3], xr[r].x, xr[r].y);
                if (MODE != 0 && j + 2 == kSuper / 16) vbase = base + id_offset(gid_c[1]);   // second half's library entry
                if (j + 2 < kSuper / 8) lookup8<N, SGL, kHalf, C::kQuad>(fa, w, j + 2, tab, vbase);
#pragma unroll
                for (int r = 0; r < NB; ++r) mma16816(c[r], fb[0], fb[1], fb[2], fb[3], xr[r].z, xr[r].w);
            } else {
                // more rows than B registers kept live: RH rows at a time through both steps
                uint32_t fn[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int h = 0; h < NB / RH; ++h) {
#pragma unroll
                    for (int r = 0; r < RH; ++r) ld_x16_if(xr[r], xp + (h * RH + r) * xrow + j * 16, dq);
                    if (h == NB / RH - 1) {
                        if (MODE != 0 && j + 2 == kSuper / 16) vbase = base + id_offset(gid_c[1]);
                        if (j + 2 < kSuper / 8) lookup8<N, SGL, kHalf, C::kQuad>(fn, w, j + 2, tab, vbase);
                    }
#pragma unroll
                    for (int r = 0; r < RH; ++r) mma16816(c[h * RH + r], fa[0], fa[1], fa[2], fa[3], xr[r].x, xr[r].y);
#pragma unroll
                    for (int r = 0; r < RH; ++r) mma16816(c[h * RH + r], fb[0], fb[1], fb[2], fb[3], xr[r].z, xr[r].w);
                }
                fa[0] = fn[0]; fa[1] = fn[1]; fa[2] = fn[2]; fa[3] = fn[3];
            }
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
            const float v = h2f((uint16_t)(e >> 16));
            const unsigned char* xo = xs + xpos(e & 0xffffu) * 2;
#pragma unroll
            for (int r = 0; r < NB; ++r) oacc[r] = fmaf(v, h2f(*(const uint16_t*)(xo + r * xrow)), oacc[r]);
        }
    }

    lstamp(a, 4);
    // ---- the two halves of a channel meet: lane (g, t < 2) holds D[g][2t], D[g][2t+1]; lane (g, t + 2) holds
    //      D[g+8][2t+4], D[g+8][2t+5]; then channel order through shared memory
#pragma unroll
    for (int r = 0; r < NB; ++r) {
        float* rr = red + (size_t)(r * W + warp) * 32;
        if (MODE != 0) {
            rr[lane] = oacc[r];   // every lane already owns its channel's sum
        } else {
            const float h2 = __shfl_xor_sync(0xffffffffu, c[r][2], 2), h3 = __shfl_xor_sync(0xffffffffu, c[r][3], 2);
            if (t4 < 2) *(float2*)(rr + 4 * g + 2 * t4) = make_float2(c[r][0] + h2, c[r][1] + h3);
            __syncwarp();
            rr[lane] += oacc[r];
        }
    }
    __syncthreads();

    // ---- fixed-order sum over the warps, then store or combine the block's slices
    const int t = threadIdx.x;
    const int er = t >> 5, ech = t & 31;   // row of x and channel of this thread in the final sum
    const bool active = er < NB;
    const int row = blk * 32 + ech;       // channel inside its blob (y index)
    const int wrow = gblk * 32 + ech;     // channel inside the launch (workspace index)
    float total = 0.f;
    if (active) {
#pragma unroll
        for (int ww = 0; ww < W; ++ww) total += red[(er * W + ww) * 32 + ech];
    }
    bool writer = true;
    if (nslices > 1) {
        __shared__ int s_last;
        if (active) a.partial[((size_t)slice * NB + er) * a.rows_ws + wrow] = total;
        __threadfence();
        __syncthreads();
        if (t == 0) s_last = (atomicAdd(a.tickets + gblk, 1) == nslices - 1);
        __syncthreads();
        writer = s_last != 0;
        if (writer) {
            __threadfence();
            if (active) {
                total = 0.f;
                for (int k2 = 0; k2 < nslices; ++k2) total += __ldcg(a.partial + ((size_t)k2 * NB + er) * a.rows_ws + wrow);
            }
            if (t == 0) a.tickets[gblk] = 0;
        }
    }
    if (writer && active && er < a.batch && row < a.rows) store_y<TIO>(ydst, (size_t)er * a.rows + row, total, a.y_is_fp16);
    lstamp(a, 5);
    if (!kMulti) break;
    }
}

template <int N, int W, int MINB, bool SGL, int MODE, bool TIO, int NB>
cudaError_t launch_lane_io(const LaneArgs& a, int grid, size_t smem, cudaStream_t s) {
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemv_lane_kernel<N, W, MINB, SGL, MODE, TIO, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
    return cudaLaunchKernelEx(&cfg, gemv_lane_kernel<N, W, MINB, SGL, MODE, TIO, NB>, a);
}

// ---- launch configurations: warps per CTA, CTAs per SM (64 registers per thread at 16 x 2), single-entry tables
struct LaneConfig { int W, per_sm; bool sgl; bool off = false; bool tiers = true; };

inline size_t lane_tab_bytes(const Layout& l, bool sgl) {
    const int bits = l.bits;
    const size_t E = (size_t)1 << bits;
    if (l.mode) {   // the library, one copy per bank: a word per entry (per pair of entries), or half a word when that does not fit
        if (!sgl) return (size_t)l.L * E * E * 128;
        return (size_t)((l.L + 1) / 2) * E * 128;   // a word holds one entry of two library ids
    }
    if (bits == 2) return 256 * 256;
    if (sgl) return E * 128;
    return E * E * (bits == 4 ? 256 : 128);
}

// `nb`: rows of x the kernel instantiation stages (1, 2, 4, 8)
inline size_t lane_smem_bytes(const Layout& l, const LaneConfig& c, int nb = 1) {
    // tables | x | red [nb][W][32] | V2a: sums of x per half super-chunk; V2: the block's codebooks for the table fill
    return lane_tab_bytes(l, c.sgl) + (size_t)nb * l.cols * 2 + (size_t)nb * c.W * 32 * 4 +
           (l.mode ? (size_t)nb * l.SC * 8 : (size_t)l.E * 64);
}

// the arguments that do not depend on the schedule
inline LaneArgs lane_args(const Layout& l, const GemvCall& c, bool sgl) {
    LaneArgs a{};
    a.off = offsets_of(l);
    a.packed = c.packed; a.x = c.x; a.y = c.y;
    a.packed_list = c.packed_list; a.x_list = c.x_list; a.y_list = c.y_list;
    a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.ell_slots = l.ell_slots;
    a.rows_ws = l.RB * c.n * 32;
    a.batch = c.batch;
    a.y_is_fp16 = c.y_is_fp16; a.x_bf16 = c.x_bf16;
    a.tab_bytes = (int)lane_tab_bytes(l, sgl);
    a.L = l.L; a.GH = l.GH;
    a.tickets = (int*)c.workspace;
    a.partial = (float*)((char*)c.workspace + align256((size_t)l.RB * 4 * c.n));
    return a;
}

}  // namespace
}  // namespace xfp
