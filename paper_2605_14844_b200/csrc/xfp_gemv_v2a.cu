// Fast fused decode GEMV for V2a blobs (shared codebook library) at batch <= 2:
//     y_i = sum_g [ scale_ig * sum_{k in g} lib[id_ig][q_ik] x_k  +  mid_ig * sum_{k in g} x_k ]  +  (S x)_i
// ("V2a: Shared Codebook Library").  One launch serves one blob or the n blobs of a routed-MoE layer
// (blockIdx.y = blob).
//
// Mapping.  As in the V2 kernel a CTA owns 64 output channels, each lane of a warp two of them
// (lane, lane+32), and the warps share K in super-chunks of 128 weights -- which are exactly the
// format's 128-weight groups, so a lane meets one (id, scale, mid) triple per channel and
// super-chunk.
//
// Look-up.  Every lane may need a different library codebook, so the tables cannot be private to a
// channel as in the V2 kernel.  Two layouts, chosen by the bit width:
//   * N <= 3 (the routed-MoE mode): PAIR tables of the whole library, replicated 16 times: word
//     (id * 4^N + pair) * 16 + (lane & 15) holds the half2 (lib[id][pair & (E-1)], lib[id][pair >> N]).
//     One look-up decodes two weights.  Lanes l and l+16 share a copy; their words fall into the
//     same bank only when their pair indices have the same parity (the bank is
//     16 * (pair & 1) + (lane & 15)), so a look-up costs 1.5 shared-memory wavefronts on average,
//     0.75 per weight.  128 KB at N = 3, L = 32: one CTA of 12 or 16 warps per SM.
//   * N >= 4: the pair tables would not fit, so the library itself is replicated once per bank: word
//     (id * 2^N + q) * 32 + lane holds lib[id][q] (fp16 in the low half).  Lane l only touches bank l;
//     one look-up decodes one weight and a PRMT joins two of them into the half2 the tensor pipe
//     wants.  Two CTAs of 8 warps per SM.
//
// Multiply-accumulate.  The half2 of a lane's two channels form the A fragment of
// mma.sync.m16n8k16 and x sits on the diagonal lanes of the B fragment (see xfp_gemv_pair.cu).  The
// fragment accumulates sum lib*x of ONE group; after the group's 32 mma the sums are moved to the
// lanes that own the channels (two shuffles per channel) and folded into an fp32 accumulator with the
// group's scale and mid-point: acc += scale * G + mid * X_g, X_g = sum of x over the group, computed
// once per CTA.  Products of fp16 numbers are exact in fp32; nothing is rounded to fp16 on the way.
//
// Outliers, schedule, launch overlap: as in the V2 kernel (transposed slabs consumed by the lanes that
// own the rows; whole-K blocks first, the last partial round cut along K with a fixed-order finish
// through the workspace; weights before griddepcontrol.wait, x/y/workspace after it).
#include <algorithm>
#include <utility>

#include "xfp_internal.h"

namespace xfp {

constexpr int kARows = 64;
constexpr int kASlots = 4;

struct V2aArgs {
    Offsets off;
    const void* packed;
    const uint16_t* x;
    void* y;
    const void* const* packed_list;
    const uint16_t* const* x_list;
    void* const* y_list;
    float* partial;  // [blob][KS][NB][rows_ws]
    int* tickets;    // [blob][blocks]
    int rows, cols, RB, SC, rows_ws, ell_slots, L;
    int nb, y_is_fp16, x_bf16;
    int blocks, n_full, kst, sc_per_split;
    int n_a, kst_b, sc_per_split_b;   // of the cut blocks the first n_a use kst slices, the rest kst_b (finer) slices
    int items_x, n;   // work items per blob (whole blocks + K slices), blobs
    int epi;                 // 0 plain store; 1 SiLU(gate) * up inside every 64-channel block; 2 weighted sum over the blobs
    const float* epi_w;      // epi 2: [n] weights
    int comb_G, comb_ng;     // epi 2: runs per block of channels, blobs per run
    int persist;             // per-bank library: resident CTAs walk the items
};

__device__ __forceinline__ void mma16816a(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Byte offset (q << 7) of index j (compile time) of a 128-weight stream, merged with `base`
// (= id * 2^N * 128 + lane * 4; the q field occupies bits 7 .. 7+N, which base leaves clear).
template <int N>
__device__ __forceinline__ uint32_t entry_addr(const uint32_t* w, int j, uint32_t base) {
    constexpr uint32_t mask = ((1u << N) - 1u) << 7;
    const int bit = j * N, wi = bit >> 5, off = bit & 31;
    uint32_t v;
    if (off + N > 32)
        v = __funnelshift_r(w[wi], w[wi + 1], off - 7);   // field straight to bit 7 (off > 7 whenever it straddles)
    else if (off >= 7)
        v = w[wi] >> (off - 7);
    else
        v = w[wi] << (7 - off);
    return (v & mask) | base;
}

// Byte offset (pair << 6) of pair p (compile time) of a 128-weight stream, merged with `base`
// (= id * 4^N * 64 + (lane & 15) * 4; the pair field occupies bits 6 .. 6+2N, which base leaves clear).
template <int N>
__device__ __forceinline__ uint32_t pair_entry_addr(const uint32_t* w, int p, uint32_t base) {
    constexpr uint32_t mask = ((1u << (2 * N)) - 1u) << 6;
    const int bit = p * 2 * N, wi = bit >> 5, off = bit & 31;
    uint32_t v;
    if (off + 2 * N > 32)
        v = __funnelshift_r(w[wi], w[wi + 1], off - 6);   // field straight to bit 6
    else if (off >= 6)
        v = w[wi] >> (off - 6);
    else
        v = w[wi] << (6 - off);
    return (v & mask) | base;
}

// FEAT instantiations carry typed IO (bf16 x, bf16 y) and the fused stores; the plain ones compile them out.
template <int N, int NB, int W, bool PAIR, bool FEAT>
__global__ void __launch_bounds__(W * 32, W == 8 ? 2 : 1) gemv_v2a_kernel(const V2aArgs a) {
    const int epi = FEAT ? a.epi : 0;
    constexpr int E = 1 << N;
    constexpr int kAWarps = W;
    constexpr int kAThreads = W * 32;
    extern __shared__ __align__(16) unsigned char smem[];
    // [library tables | x fp16 [NB][K] | xg fp32 [NB][SC] | red fp32 [W][NB][64] | library copy]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    const int K = a.SC * kSuper;
    const int tab_bytes = PAIR ? a.L * E * E * 64 : a.L * E * 128;
    unsigned char* tab = smem;
    uint16_t* xs = (uint16_t*)(smem + tab_bytes);             // [NB][K]
    float* xg = (float*)(xs + (size_t)NB * K);                // [NB][SC]
    float* red = xg + NB * a.SC;                              // [W][NB][64]
    __shared__ int s_last;

    // the library the tables were built from, on the next 16-byte boundary (NB * SC floats of xg precede red)
    uint4* libcopy = (uint4*)(((uintptr_t)(red + (size_t)kAWarps * NB * kARows) + 15) & ~(uintptr_t)15);
    bool have_tables = false;
    bool waited = false;
    const uint16_t* x_staged = nullptr;

    // ---- work items: (blob, whole block or K slice of a block), dealt round-robin to the CTAs of the launch
    // The weighted sum over the blobs (epi 2) deals RUNS instead: a CTA takes comb_ng consecutive blobs of
    // one block of channels and adds their weighted results in registers; only the comb_G runs of a block
    // meet in the scratch (none when one run covers all blobs).
    const int per = epi == 2 ? a.comb_ng : 1;
    const int nrun = epi == 2 ? a.blocks * a.comb_G : a.items_x * a.n;
    float csum = 0.f;   // epi 2: this thread's channel, weighted sum over the blobs of the run
#pragma unroll 1
    for (int run = blockIdx.x; run < nrun; run += gridDim.x) {
#pragma unroll 1
    for (int jj = 0; jj < per; ++jj) {
    int prob, bx;
    if (epi == 2) {
        bx = run / a.comb_G;
        prob = (run - bx * a.comb_G) * a.comb_ng + jj;
        if (prob >= a.n) break;
        if (jj == 0) csum = 0.f;
    } else {
        prob = run / a.items_x;
        bx = run - prob * a.items_x;
    }
    int blk, ks, KS, spp;
    if (bx < a.n_full) {
        blk = bx; ks = 0; KS = 1; spp = a.SC;
    } else if (bx - a.n_full < a.n_a * a.kst) {
        const int t = bx - a.n_full;
        blk = a.n_full + t / a.kst; ks = t % a.kst; KS = a.kst; spp = a.sc_per_split;
    } else {
        const int t = bx - a.n_full - a.n_a * a.kst;
        blk = a.n_full + a.n_a + t / a.kst_b; ks = t % a.kst_b; KS = a.kst_b; spp = a.sc_per_split_b;
    }
    const float epi_wj = epi == 2 ? __ldg(a.epi_w + prob) : 0.f;   // fetched now, used in the store
    const void* packed = a.packed_list ? a.packed_list[prob] : a.packed;
    const uint16_t* x = a.x_list ? a.x_list[prob] : a.x;
    void* y = a.y_list ? a.y_list[prob] : a.y;
    const Blob b = blob_at(packed, a.off);
    const int sc0 = ks * spp;
    const int nsc = max(0, min(a.SC, sc0 + spp) - sc0);

    const int blk0 = 2 * blk;
    const int blk1 = min(2 * blk + 1, a.RB - 1);              // clamped when RB is odd; its results are dropped

    // ---- (0) start streaming: first super-chunk of this warp (indices and group metadata of both channels)
    uint32_t w0[4 * N + 1], w1[4 * N + 1];
    w0[4 * N] = w1[4 * N] = 0u;
    const uint4* i0 = b.idx + ((size_t)(blk0 * a.SC + sc0) * N) * 32 + lane;
    const uint4* i1 = b.idx + ((size_t)(blk1 * a.SC + sc0) * N) * 32 + lane;
    const size_t m0 = (size_t)(blk0 * a.SC + sc0) * 32 + lane, m1 = (size_t)(blk1 * a.SC + sc0) * 32 + lane;
    uint32_t id0 = 0, id1 = 0, sm0 = 0, sm1 = 0;              // current group: library ids and (scale, mid)
    uint32_t nid0 = 0, nid1 = 0, nsm0 = 0, nsm1 = 0;          // next group
    if (warp < nsc) {
#pragma unroll
        for (int v = 0; v < N; ++v) {
            const uint4 t0 = ld_stream(i0 + ((size_t)warp * N + v) * 32);
            const uint4 t1 = ld_stream(i1 + ((size_t)warp * N + v) * 32);
            w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
            w1[4 * v] = t1.x; w1[4 * v + 1] = t1.y; w1[4 * v + 2] = t1.z; w1[4 * v + 3] = t1.w;
        }
        id0 = b.gid[m0 + (size_t)warp * 32]; id1 = b.gid[m1 + (size_t)warp * 32];
        sm0 = b.gsm[m0 + (size_t)warp * 32]; sm1 = b.gsm[m1 + (size_t)warp * 32];
    }
    // outlier slabs of this CTA's two row-blocks: slots gw, gw + stride, ... belong to this warp.  Launches
    // over several blobs read the slab geometry from each blob (their outlier counts differ).
    int ell_slots = a.ell_slots;
    const uint32_t* ell = b.ell;
    if (a.packed_list) {
        const int* hdr = (const int*)((const char*)packed + a.off.hdr);
        ell_slots = __ldg(hdr);
        ell = (const uint32_t*)((const char*)packed + *(const long long*)(hdr + 2));
    }
    const int gw = ks * kAWarps + warp, ostride = KS * kAWarps;
    const uint32_t* slab[2];
    uint32_t olen[2];
    uint32_t oe[2][kASlots];
    int width[2];
    float acc[NB][2];
    int oround = 0, nrounds = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        slab[h] = ell + (size_t)(h ? blk1 : blk0) * (ell_slots + 1) * 32 + lane;
        width[h] = ell_slots;
        olen[h] = ell_slots ? __ldg(slab[h]) : 0u;
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) acc[bb][h] = 0.f;
    }
    auto fetch_slots = [&](int round) {
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int q = 0; q < kASlots; ++q) {
                const int j = gw + (round * kASlots + q) * ostride;
                oe[h][q] = j < width[h] ? __ldg(slab[h] + (size_t)(1 + j) * 32) : 0u;
            }
    };
    auto consume_slots = [&]() {
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int q = 0; q < kASlots; ++q) {
                const float v = h2f((uint16_t)(oe[h][q] >> 16));
                const uint32_t col = oe[h][q] & 0xffffu;
#pragma unroll
                for (int bb = 0; bb < NB; ++bb) acc[bb][h] = fmaf(v, h2f(xs[(size_t)bb * K + col]), acc[bb][h]);
            }
    };
    if (ell_slots) fetch_slots(0);

    // ---- (1) library tables (after the item's first loads are on their way).  The blobs of a launch normally share one library (one per layer), so the tables are
    //      built once per CTA; a blob whose library differs from the one they were built from rebuilds them.
    {
        const uint4* cb4 = (const uint4*)b.cb;
        const int nvec = a.L * E / 8;   // the library in 16-byte vectors (L * E is a multiple of 8)
        int differs = !have_tables;
        if (have_tables)
            for (int i = threadIdx.x; i < nvec; i += kAThreads) {
                const uint4 u = __ldg(cb4 + i), v = libcopy[i];
                differs |= (u.x != v.x) | (u.y != v.y) | (u.z != v.z) | (u.w != v.w);
            }
        if (__syncthreads_or(differs)) {
            for (int i = threadIdx.x; i < nvec; i += kAThreads) libcopy[i] = __ldg(cb4 + i);
            if (PAIR) {
                // pair tables, 16 copies: words (id * E*E + pair) * 16 .. + 15 hold the same half2.  Four threads per
                // entry, 16 bytes each: a warp's store covers 512 contiguous bytes (one thread writing the entry's 64
                // bytes put a quarter-warp into two bank groups: 4300 wavefronts per fill instead of 1024)
                for (int t = threadIdx.x; t < a.L * E * E * 4; t += kAThreads) {
                    const int e = t >> 2, id = e / (E * E), pr = e % (E * E);
                    const uint32_t v = (uint32_t)__ldg(b.cb + id * E + (pr & (E - 1))) |
                                       ((uint32_t)__ldg(b.cb + id * E + (pr >> N)) << 16);
                    ((uint4*)(tab + (size_t)e * 64))[t & 3] = make_uint4(v, v, v, v);
                }
            } else {
                // one copy per bank: word (e * 32 + lane) = lib[e] for every lane.  A lane fetches entry e0 + lane, the warp
                // stores 32 rows, the entries handed round by shuffle (one uniform load per row paid its latency per row)
                for (int e0 = warp * 32; e0 < a.L * E; e0 += kAWarps * 32) {
                    const uint32_t mine = e0 + lane < a.L * E ? (uint32_t)__ldg(b.cb + e0 + lane) : 0u;
#pragma unroll
                    for (int r = 0; r < 32; ++r) {
                        const uint32_t v = __shfl_sync(0xffffffffu, mine, r);
                        if (e0 + r < a.L * E) *(uint32_t*)(tab + (size_t)(e0 + r) * 128 + lane * 4) = v;
                    }
                }
            }
            have_tables = true;
        }
    }

    // ---- (2) x: wait for the previous kernel, stage fp16 x (all of K) and the group sums X_g -- once per
    //      distinct x of the launch (the experts of a routed layer share it)
    if (!waited) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
    }
    if (x != x_staged) {
        {
            const int nvec = NB * (K / 8);
            for (int t = threadIdx.x; t < nvec; t += kAThreads) {
                const int bb = t / (K / 8), kk = (t - bb * (K / 8)) * 8;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (bb < a.nb) v = __ldg((const uint4*)(x + (size_t)bb * a.cols + kk));
                if (FEAT) v = x8_as_f16(v, a.x_bf16);
                *(uint4*)(xs + (size_t)t * 8) = v;
            }
        }
        __syncthreads();
        for (int u = warp; u < NB * a.SC; u += kAWarps) {   // X_g: 128 values per group, 4 per lane, fixed butterfly
            const uint2 hv = *(const uint2*)(xs + (size_t)u * kSuper + lane * 4);
            const float2 p0 = __half22float2(*(const __half2*)&hv.x), p1 = __half22float2(*(const __half2*)&hv.y);
            float t = (p0.x + p0.y) + (p1.x + p1.y);
#pragma unroll
            for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0) xg[u] = t;
        }
        x_staged = x;
    }
    __syncthreads();   // tables, x and X_g visible
#pragma unroll
    for (int h = 0; h < 2; ++h) {   // the rows' slot counts have arrived: this warp's number of outlier rounds
        int wmax = (int)olen[h];
#pragma unroll
        for (int o = 16; o; o >>= 1) wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
        width[h] = min(wmax, ell_slots);
        const int mine = width[h] > gw ? (width[h] - gw + ostride - 1) / ostride : 0;
        nrounds = max(nrounds, (mine + kASlots - 1) / kASlots);
    }

    // ---- (3) main loop over this warp's groups
    const int g = lane >> 2, t4 = lane & 3;
    const bool diag0 = (g == t4);
    const bool diag1 = (NB > 1) && (g == t4 + 4);
    const bool diag = diag0 || diag1;
    const unsigned char* xrow = (const unsigned char*)xs + (diag1 ? (size_t)K * 2 : 0) + (size_t)sc0 * (kSuper * 2);
    // where this lane's own sums land: D[g][t] sits in lane (g, t >> 1), register t & 1 (batch row 0), and in
    // lane (g, 2 + (t >> 1)) for batch row 1
    const int src0 = (lane & ~3) | (t4 >> 1);
    const bool odd = t4 & 1;

    auto lookup = [&](uint32_t (&f)[4], int m, uint32_t base0, uint32_t base1) {
        if (PAIR) {
            f[0] = *(const uint32_t*)(tab + pair_entry_addr<N>(w0, 2 * m, base0));       // (k, k+1) of channel 0
            f[1] = *(const uint32_t*)(tab + pair_entry_addr<N>(w1, 2 * m, base1));       // (k, k+1) of channel 1
            f[2] = *(const uint32_t*)(tab + pair_entry_addr<N>(w0, 2 * m + 1, base0));   // (k+2, k+3) of channel 0
            f[3] = *(const uint32_t*)(tab + pair_entry_addr<N>(w1, 2 * m + 1, base1));   // (k+2, k+3) of channel 1
            return;
        }
        const uint32_t l00 = *(const uint32_t*)(tab + entry_addr<N>(w0, 4 * m + 0, base0));
        const uint32_t l01 = *(const uint32_t*)(tab + entry_addr<N>(w0, 4 * m + 1, base0));
        const uint32_t l02 = *(const uint32_t*)(tab + entry_addr<N>(w0, 4 * m + 2, base0));
        const uint32_t l03 = *(const uint32_t*)(tab + entry_addr<N>(w0, 4 * m + 3, base0));
        const uint32_t l10 = *(const uint32_t*)(tab + entry_addr<N>(w1, 4 * m + 0, base1));
        const uint32_t l11 = *(const uint32_t*)(tab + entry_addr<N>(w1, 4 * m + 1, base1));
        const uint32_t l12 = *(const uint32_t*)(tab + entry_addr<N>(w1, 4 * m + 2, base1));
        const uint32_t l13 = *(const uint32_t*)(tab + entry_addr<N>(w1, 4 * m + 3, base1));
        f[0] = __byte_perm(l00, l01, 0x5410);   // (k, k+1) of channel 0
        f[1] = __byte_perm(l10, l11, 0x5410);   // (k, k+1) of channel 1
        f[2] = __byte_perm(l02, l03, 0x5410);   // (k+2, k+3) of channel 0
        f[3] = __byte_perm(l12, l13, 0x5410);   // (k+2, k+3) of channel 1
    };

#pragma unroll 1
    for (int s = warp; s < nsc; s += kAWarps) {
        const int sn = s + kAWarps;
        const bool has_next = sn < nsc;
        if (has_next) {   // metadata of the next group travels during this one
            nid0 = b.gid[m0 + (size_t)sn * 32]; nid1 = b.gid[m1 + (size_t)sn * 32];
            nsm0 = b.gsm[m0 + (size_t)sn * 32]; nsm1 = b.gsm[m1 + (size_t)sn * 32];
        }
        if (oround < nrounds) {
            consume_slots();
            if (++oround < nrounds) fetch_slots(oround);
        }
        const uint32_t base0 = PAIR ? id0 * (uint32_t)(E * E * 64) + (uint32_t)(lane & 15) * 4u
                                    : id0 * (uint32_t)(E * 128) + (uint32_t)lane * 4u;
        const uint32_t base1 = PAIR ? id1 * (uint32_t)(E * E * 64) + (uint32_t)(lane & 15) * 4u
                                    : id1 * (uint32_t)(E * 128) + (uint32_t)lane * 4u;
        const unsigned char* xp = xrow + (size_t)s * (kSuper * 2);
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t fa[4], fb[4];
        uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = make_uint4(0u, 0u, 0u, 0u);
        if (diag) xa = *(const uint4*)xp;
        lookup(fa, 0, base0, base1);
        auto reload = [&](int gi) {   // index vectors are reloaded for the next group once fully consumed
#pragma unroll
            for (int v = 0; v < N; ++v) {
                const int jlast = (128 * (v + 1) + N - 1) / N - 1;   // last index touching vector v
                if (jlast / 4 == gi && has_next) {
                    const uint4 t0 = ld_stream(i0 + ((size_t)sn * N + v) * 32);
                    const uint4 t1 = ld_stream(i1 + ((size_t)sn * N + v) * 32);
                    w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
                    w1[4 * v] = t1.x; w1[4 * v + 1] = t1.y; w1[4 * v + 2] = t1.z; w1[4 * v + 3] = t1.w;
                }
            }
        };
#pragma unroll
        for (int m = 0; m < kSuper / 4; m += 4) {   // one mma per 4 consecutive k, look-ups one mma ahead
            if (diag) xb = *(const uint4*)(xp + (m + 2) * 8);
            lookup(fb, m + 1, base0, base1);
            reload(m + 1);
            mma16816a(c0, fa[0], fa[1], fa[2], fa[3], xa.x, xa.y);
            lookup(fa, m + 2, base0, base1);
            reload(m + 2);
            mma16816a(c1, fb[0], fb[1], fb[2], fb[3], xa.z, xa.w);
            if (m + 4 < kSuper / 4) { if (diag) xa = *(const uint4*)(xp + (m + 4) * 8); }
            lookup(fb, m + 3, base0, base1);
            reload(m + 3);
            mma16816a(c0, fa[0], fa[1], fa[2], fa[3], xb.x, xb.y);
            if (m + 4 < kSuper / 4) {
                lookup(fa, m + 4, base0, base1);
                reload(m + 4);
            }
            mma16816a(c1, fb[0], fb[1], fb[2], fb[3], xb.z, xb.w);
        }
        // group sums to their owners, then  acc += scale * G + mid * X_g
        const float d0 = c0[0] + c1[0], d1 = c0[1] + c1[1], d2 = c0[2] + c1[2], d3 = c0[3] + c1[3];
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) {
            const int src = src0 + 2 * bb;
            const float e0 = __shfl_sync(0xffffffffu, d0, src), e1 = __shfl_sync(0xffffffffu, d1, src);
            const float e2 = __shfl_sync(0xffffffffu, d2, src), e3 = __shfl_sync(0xffffffffu, d3, src);
            const float G0 = odd ? e1 : e0, G1 = odd ? e3 : e2;
            const float X = xg[bb * a.SC + sc0 + s];
            acc[bb][0] = fmaf(h2f((uint16_t)(sm0 & 0xffffu)), G0, fmaf(h2f((uint16_t)(sm0 >> 16)), X, acc[bb][0]));
            acc[bb][1] = fmaf(h2f((uint16_t)(sm1 & 0xffffu)), G1, fmaf(h2f((uint16_t)(sm1 >> 16)), X, acc[bb][1]));
        }
        id0 = nid0; id1 = nid1; sm0 = nsm0; sm1 = nsm1;
    }
    while (oround < nrounds) {   // more outlier rounds than groups
        consume_slots();
        if (++oround < nrounds) fetch_slots(oround);
    }
    if (warp == 0 && ks == 0 && ell_slots) {   // rows that overflow their slab finish from the CSR arrays
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if ((int)olen[h] >= ell_slots) {
                const int row = (h ? blk1 : blk0) * kRowsPerBlock + lane;
                const int p1 = __ldg(b.rowptr + row + 1);
                for (int p = __ldg(b.rowptr + row) + ell_slots; p < p1; ++p) {
                    const uint32_t e = __ldg(b.oent + p);
#pragma unroll
                    for (int bb = 0; bb < NB; ++bb)
                        acc[bb][h] = fmaf(h2f((uint16_t)(e >> 16)), h2f(xs[(size_t)bb * K + (e & 0xffffu)]), acc[bb][h]);
                }
            }
        }
    }

    // ---- (4) fixed-order reduction over the warps, store or split-K finish
#pragma unroll
    for (int bb = 0; bb < NB; ++bb) {
        red[((size_t)warp * NB + bb) * kARows + lane] = acc[bb][0];
        red[((size_t)warp * NB + bb) * kARows + 32 + lane] = acc[bb][1];
    }
    __syncthreads();
    const int t = threadIdx.x;
    const int bb = t / kARows, r = t % kARows;
    const bool active = t < NB * kARows;
    const bool dup = (r >= 32) && (2 * blk + 1 >= a.RB);
    const int row = blk * kARows + r;
    float total = 0.f;
    if (active) {
#pragma unroll
        for (int w = 0; w < kAWarps; ++w) total += red[((size_t)w * NB + bb) * kARows + r];
    }
    bool writer = true;
    if (KS > 1) {
        float* part = a.partial + (size_t)prob * 64 * NB * a.rows_ws;
        int* ticket = a.tickets + (size_t)prob * a.blocks + blk;
        if (active) part[((size_t)ks * NB + bb) * a.rows_ws + row] = total;
        __threadfence();
        __syncthreads();
        if (t == 0) s_last = (atomicAdd(ticket, 1) == KS - 1);
        __syncthreads();
        writer = s_last != 0;
        if (writer) {
            __threadfence();
            if (active) {
                total = 0.f;
                for (int k2 = 0; k2 < KS; ++k2) total += __ldcg(part + ((size_t)k2 * NB + bb) * a.rows_ws + row);
            }
            if (t == 0) *ticket = 0;
        }
    }
    if (epi == 0) {
        if (writer && active && !dup && bb < a.nb && row < a.rows) {
            store_y<FEAT>(y, (size_t)bb * a.rows + row, total, a.y_is_fp16);
        }
    } else if (epi == 1) {
        // gated activation of a routed expert: channels 0..31 of the block are gates, 32..63 the matching
        // up channels; the block stores 32 values h = SiLU(gate) * up  (batch 1, rows a multiple of 64)
        if (writer) {
            __syncthreads();   // every thread has read its column of red
            if (t < kARows) red[t] = total;
            __syncthreads();
            if (t < 32) {
                const float g = red[t], u = red[t + 32];
                const float h = g / (1.f + expf(-g)) * u;
                const size_t o = (size_t)blk * 32 + t;
                put_y(y, o, h, a.y_is_fp16);
            }
        }
    } else {
        // weighted sum over the blobs of the launch (the routed experts' down projections)
        if (t < kARows) csum = fmaf(epi_wj, total, csum);
        const bool run_done = jj == per - 1 || prob == a.n - 1;
        if (run_done && a.comb_G == 1) {
            if (t < kARows && !dup && row < a.rows) {
                void* y0 = a.y_list ? a.y_list[0] : a.y;
                put_y(y0, row, csum, a.y_is_fp16);
            }
        } else if (run_done) {
            // the runs of this block leave their sums in the scratch, the last one to arrive adds them in run order
            float* comb = a.partial;            // [run of the block][rows_ws]; the K-split scratch is idle in these launches
            int* ticket = a.tickets + blk;      // one counter per block of channels
            const int g = run - bx * a.comb_G;
            if (t < kARows) comb[(size_t)g * a.rows_ws + row] = csum;
            __threadfence();
            __syncthreads();
            if (t == 0) s_last = (atomicAdd(ticket, 1) == a.comb_G - 1);
            __syncthreads();
            if (s_last) {
                __threadfence();
                if (t < kARows && !dup && row < a.rows) {
                    float sum = 0.f;
                    for (int g2 = 0; g2 < a.comb_G; ++g2) sum += __ldcg(comb + (size_t)g2 * a.rows_ws + row);
                    void* y0 = a.y_list ? a.y_list[0] : a.y;
                    put_y(y0, row, sum, a.y_is_fp16);
                }
                if (t == 0) *ticket = 0;
            }
        }
    }
    if (!PAIR && !a.persist) break;   // the per-bank library is launched with one CTA per item
    __syncthreads();   // red, x and the ticket flag are reused by the CTA's next item
    }
    if (!PAIR && !a.persist) break;
    }
}

// ------------------------------------------------------------------------------------ host side

// Launch configuration of a layout: pair tables (one CTA per SM, 12 or 16 warps) when they fit, else the
// per-bank library (two CTAs of 8 warps per SM, or one of 16 warps when the library is too large for two).
struct V2aConfig { bool pair; int warps, slots; size_t smem; };

static size_t v2a_smem_bytes(const Layout& l, int nb, bool pair, int warps) {
    const size_t tab = pair ? (size_t)l.L * l.E * l.E * 64 : (size_t)l.L * l.E * 128;
    return tab + (size_t)nb * l.cols * 2 + (size_t)nb * l.SC * 4 + (size_t)warps * nb * kARows * 4 +
           (size_t)l.L * l.E * 2 + 16;   // + the copy of the library the tables were built from, 16-byte aligned
}

static V2aConfig v2a_config(const Layout& l, int nb, int n = 1) {
    // Pair tables cost 128 KB of fills per resident CTA and run one CTA of 12 or 16 warps per SM: they pay off
    // when every SM has a few hundred thousand weights to decode and K is long enough to keep those warps busy
    // (measured: 28672 x 8192 53 vs 61 us, 8192 x 8192 18.6 vs 22.9, 12288 x 4096 18.7 vs 20.0 in their favour;
    // 4096 x 4096 10.4 vs 9.1 and the routed experts' 4096 x 1536 down projections 20.6 vs 18.7 against them).
    const bool big = (long long)l.rows * l.cols * n >= 40ll * 1000 * 1000 && l.SC >= 32;
    const int sms = sched_sms();
    if (l.bits <= 3 && big) {
        // K is shared by the warps in super-chunks: 12 warps when that divides the count and 16 does not
        const int warps = (l.SC % 16 != 0 && l.SC % 12 == 0) ? 12 : 16;
        const size_t sm = v2a_smem_bytes(l, nb, true, warps);
        if (sm <= 224u * 1024u) return V2aConfig{true, warps, sms, sm};
    }
    const size_t sm8 = v2a_smem_bytes(l, nb, false, 8);
    if (sm8 <= 110u * 1024u) return V2aConfig{false, 8, 2 * sms, sm8};
    return V2aConfig{false, 16, sms, v2a_smem_bytes(l, nb, false, 16)};   // large library (N = 5): one CTA per SM
}

bool v2a_supported(const Layout& l, int batch) {
    if (l.mode != 1 || l.bits < 2 || l.bits > 5 || batch > 2) return false;
    if (l.GH != 1) return false;   // groups of 64 weights: two table bases per super-chunk, served by the generic kernel
    const V2aConfig cfg = v2a_config(l, batch);
    return cfg.smem <= (cfg.warps == 8 ? 110u : 224u) * 1024u;
}

size_t v2a_workspace_bytes(const Layout& l) {
    const int blocks = (l.RB + 1) / 2;
    // counters first, in the region every GEMV kernel of the library keeps zero-filled: one int per row-block
    return align256((size_t)l.RB * 4) + align256((size_t)64 * 2 * (size_t)blocks * kARows * 4);
}

template <int N, int NB, int W, bool PAIR, bool FEAT>
static cudaError_t launch_v2a_feat(const V2aArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemv_v2a_kernel<N, NB, W, PAIR, FEAT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             W == 8 ? 112 * 1024 : 226 * 1024);
        if (e != cudaSuccess) return e;
        attr_done.set(dev);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(W * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_v2a_kernel<N, NB, W, PAIR, FEAT>, a);
}

template <int N, int NB, int W, bool PAIR>
static cudaError_t launch_v2a(const V2aArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    if (a.epi != 0 || a.x_bf16 || a.y_is_fp16 == 2) return launch_v2a_feat<N, NB, W, PAIR, true>(a, grid, smem, s);
    return launch_v2a_feat<N, NB, W, PAIR, false>(a, grid, smem, s);
}

template <int N, int NB>
static cudaError_t launch_v2a_cfg(const V2aConfig& cfg, const V2aArgs& a, dim3 grid, cudaStream_t s) {
    if (N <= 3 && cfg.pair)
        return cfg.warps == 12 ? launch_v2a<(N <= 3 ? N : 3), NB, 12, true>(a, grid, cfg.smem, s)
                               : launch_v2a<(N <= 3 ? N : 3), NB, 16, true>(a, grid, cfg.smem, s);
    if (cfg.warps == 16) return launch_v2a<N, NB, 16, false>(a, grid, cfg.smem, s);
    return launch_v2a<N, NB, 8, false>(a, grid, cfg.smem, s);
}

cudaError_t launch_gemv_v2a(const Layout& l, const GemvCall& c, cudaStream_t s) {
    const V2aConfig cfg = v2a_config(l, c.batch, c.n);
    V2aArgs a{};
    a.off = offsets_of(l);
    a.packed = c.packed; a.x = c.x; a.y = c.y;
    a.packed_list = c.packed_list; a.x_list = c.x_list; a.y_list = c.y_list;
    a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.ell_slots = l.ell_slots; a.L = l.L;
    a.nb = c.batch; a.y_is_fp16 = c.y_is_fp16; a.x_bf16 = c.x_bf16;
    a.blocks = (l.RB + 1) / 2;
    a.rows_ws = a.blocks * kARows;
    // schedule: whole-K blocks fill whole rounds of CTA slots (all blobs of the launch count); the blocks of
    // the last partial round are cut along K into slices of at least 512 weights
    const long long total = (long long)a.blocks * c.n;
    const int kmax = std::min(64, std::max(1, l.SC / 4));
    auto slices = [&](int want) {   // (slices, super-chunks per slice) for a cut into about `want` pieces
        int k = std::max(1, std::min(want, std::min(kmax, l.SC)));
        const int spp = (l.SC + k - 1) / k;
        k = (l.SC + spp - 1) / spp;
        return std::make_pair(k, spp);
    };
    int rem = 0;
    a.kst = 1; a.sc_per_split = l.SC; a.n_a = 0; a.kst_b = 1; a.sc_per_split_b = l.SC;
    const int tail = (int)(total % cfg.slots);
    if (tail > 0 && c.n == 1 && c.epilogue != 2) {   // the weighted sum uses the K-split scratch for itself
        rem = tail;
        auto ka = slices(cfg.slots / rem);
        if (ka.first > 1) {
            // the whole tail fits one round when cut into ka pieces per block
            a.kst = ka.first; a.sc_per_split = ka.second; a.n_a = rem;
        } else if (kmax >= 2 && total > cfg.slots) {
            // whole rounds came before and more than half a round is left: halves for as many blocks as fill one round, finer slices for the rest
            auto k2 = slices(2);
            a.kst = k2.first; a.sc_per_split = k2.second;
            a.n_a = std::min(rem, cfg.slots / a.kst);
            const int rest = rem - a.n_a;
            if (rest > 0) {
                auto kb = slices(std::max(2, cfg.slots / rest));
                a.kst_b = kb.first; a.sc_per_split_b = kb.second;
            }
            if (a.kst <= 1) { a.n_a = 0; rem = 0; }
        } else {
            rem = 0;
        }
    }
    a.n_full = a.blocks - rem;
    const int n_b = rem - a.n_a;
    a.tickets = (int*)c.workspace;
    a.partial = (float*)((char*)c.workspace + align256((size_t)l.RB * 4 * c.n));   // behind the common counter region
    a.items_x = a.n_full + a.n_a * a.kst + n_b * a.kst_b;
    a.n = c.n;
    a.epi = c.epilogue; a.epi_w = c.epi_weights;
    long long items = (long long)a.items_x * c.n;
    a.comb_G = 1; a.comb_ng = 1;
    if (c.epilogue == 2) {
        // pair tables: as few runs per block as still fill the resident CTAs; per-bank library: one blob per CTA
        int G = cfg.pair ? std::max(1, std::min(c.n, cfg.slots / std::max(1, a.blocks))) : c.n;
        a.comb_ng = (c.n + G - 1) / G;
        a.comb_G = (c.n + a.comb_ng - 1) / a.comb_ng;
        items = (long long)a.blocks * a.comb_G;
    }
    // pair tables are expensive to build: resident CTAs walk the items; the per-bank library launches one CTA per item
    // several blobs on the per-bank library with more items than CTA slots: resident CTAs walk the items, so the
    // tables are not rebuilt for the later rounds (routed experts' down projections: 1 % per token-layer)
    a.persist = (!cfg.pair && c.n > 1 && items > cfg.slots) ? 1 : 0;
    dim3 grid((unsigned)((cfg.pair || a.persist) ? (items < cfg.slots ? items : cfg.slots) : items), 1, 1);
    switch (l.bits * 10 + c.batch) {
        case 21: return launch_v2a_cfg<2, 1>(cfg, a, grid, s);
        case 22: return launch_v2a_cfg<2, 2>(cfg, a, grid, s);
        case 31: return launch_v2a_cfg<3, 1>(cfg, a, grid, s);
        case 32: return launch_v2a_cfg<3, 2>(cfg, a, grid, s);
        case 41: return launch_v2a_cfg<4, 1>(cfg, a, grid, s);
        case 42: return launch_v2a_cfg<4, 2>(cfg, a, grid, s);
        case 51: return launch_v2a_cfg<5, 1>(cfg, a, grid, s);
        case 52: return launch_v2a_cfg<5, 2>(cfg, a, grid, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace xfp
