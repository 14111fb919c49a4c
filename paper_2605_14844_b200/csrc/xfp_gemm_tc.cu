// Prefill form of the fused decode kernel, Y = X (D + S)^T for M >= 1 rows of x ("Fused Decode Kernel", steps
// (1)-(4): depack, codebook gather, outlier scatter-add into the dequantised tile, GEMM on the tensor cores), on
// the fifth-generation tensor cores.  The decoded fp16 tile never touches shared memory: the lane-per-channel
// decode of the GEMV kernels produces exactly the register image of a tensor-memory tile (lane = row, 32-bit
// column = two consecutive k), so it is stored with tcgen05.st and used as the A operand of tcgen05.mma from
// tensor memory; the x tile is the B operand in shared memory, brought there by one bulk tensor copy (TMA) per
// stage; the fp32 accumulator is a second tensor-memory region.
//
//   CTA      128 output channels (four row-blocks) x up to 128 rows of x x one K slice; eight decode warps and a
//            ninth that issues the tensor copies and the products; two CTAs per SM (256 of the 512 tensor-memory
//            columns each: 128 accumulator columns, two A stages of 64).  For many rows of x (see plan_of) the tile
//            is 256 rows: 256 accumulator columns and FOUR A stages, all 512 columns, one CTA per SM (a group of decode
//            warps then stores its next stage while the products of its previous one still run: 28672 x 8192 with
//            0.3 % outliers, 256 rows of x 209 -> 164 us, 512 rows 381 -> 314 us).
//   stage    one super-chunk (128 k): A = W^[128][128] fp16 in tensor memory, B = x[T][128] fp16 in shared memory as
//            two K-major halves of 64 k in the 128-byte swizzle, each written by one tensor copy with the box
//            {64 k, T rows} (128 contiguous bytes per row of x; rows beyond M arrive as zeros).
//   decode   warp (row-block, half of the super-chunk): index vectors prefetched two super-chunks ahead, 64
//            look-ups in one straight block into 32 registers.  V2: per-lane shared-memory tables (pair tables up
//            to N = 3, one entry per index above).  V2a: the library replicated once per bank, then
//            D16 = fp16(fp32(scale * lib[id][q] + mid)) with the group's scale and mid-point.  The outliers of the
//            lane's channel that fall into its half are added to the register that holds them with one correctly
//            rounded fp16 addition each, so the tile is the matrix xfp_dequant writes.  Up to 64 rows of x the
//            outliers stay out of the tile (the walk through a lane's list cost 37 - 50 us of 141 at 28672 x 8192
//            with 0.3 % outliers): the epilogue adds S x^T to the accumulator instead, see below.
//   mma      one thread waits for "A stage stored" (eight arrivals) and "x tile landed" (transaction bytes), issues
//            eight m128 nT k16 instructions and commits them to a "products done" mbarrier; the decode of
//            iteration i waits for the products of iteration i - 2 (i - 4 with four stages), whose A stage it
//            overwrites.  No CTA-wide
//            barrier inside the loop.
//   epilogue tcgen05.ld (lane = channel, registers = rows of x), direct store, or fp32 partials through the
//            workspace when K is cut (few row tiles): the last CTA of a tile adds the slices in slice order.
//            With the sparse outlier product, a thread first walks its channel's outliers inside the K slice and adds
//            value * x[t][column] for its 16 rows of x in fp32, entries in ascending column order; the 16 activations
//            are 32 contiguous bytes of a transposed copy of x that a small kernel writes before the launch.
// Every wait on an mbarrier has an iteration limit; when one runs out the CTA stops issuing work, records it in
// the first word of the workspace and leaves through the common exit that frees its tensor memory.
#include <cuda.h>

#include <cstdlib>

#include <type_traits>

#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

namespace {

constexpr int kTileRows = 128;   // output channels per CTA (the M of the instruction)
constexpr int kSmallT = 128;     // rows of x per CTA (the N of the instruction): 128 with two CTAs per SM, or
constexpr int kBigT = 256;       // 256 with one (more than 128 rows of x: the weights are decoded once per 256 rows)
constexpr int kWarps = 8;        // decode warps of one group (row-block x half); the warp behind the last group issues
                                 // the tensor copies and the products.  256-row tiles (one CTA per SM) run two groups:
                                 // group g decodes the iterations with it % 2 == g, i.e. owns A stage g
constexpr int threads_of(bool big) { return ((big ? 2 : 1) * kWarps + 1) * 32; }
constexpr uint32_t kSpinLimit = 1u << 20;   // polls of a bounded wait, each of at most kPollNs: about a second
constexpr uint32_t kPollNs = 1000;
// tensor memory of a CTA: the accumulator (128 or 256 columns), then the two A stages: 256 or 512 columns
constexpr int kAStageCols = 64;  // 128 k as fp16 pairs
constexpr int kXStages = 3;      // x tiles in flight: the copy of iteration i + 1 is issued at the top of iteration i
constexpr size_t kV2aTabMax = 128 * 1024;   // V2a: the per-bank library (L * 2^N * 128 bytes) must fit beside the x stages
// Up to this many rows of x the outliers are a sparse product in the epilogue.  The product reads 32 bytes of the
// transposed x per outlier and 16 rows, scattered through L2 at about 2.4 TB/s (28672 x 8192, 0.3 %: 13 us at 16 rows,
// 19 at 32, 39 at 64, 78 at 128); the walk through the lists costs about as much per outlier as 64 rows of the product
// whatever the rows (0.3 %: 45 - 50 us, 1 %: 114 us).
constexpr int kSparseRows = 64;
constexpr size_t kMinSmem = 80 * 1024;   // at most two CTAs per SM: each holds half of the tensor memory (a CTA with
                                         // 256-row tiles holds all of it and asks for more than half of the shared memory)

struct GemmArgs {
    Blob b;
    void* y;
    int* ctrl;        // [0] error word, [1 + tile] arrival counters of the K slices
    float* partial;   // [tile][slice][T][128]
    int rows, cols, RB, SC, M, ell_slots, y_kind;
    // schedule: CTAs [tier_cta[i], tier_cta[i+1]) are the K slices of tiles tier_tile[i].., tier_ks[i] slices of
    // tier_spp[i] super-chunks per tile, their partial sums from slot tier_slot[i] on (unused tiers start at INT_MAX)
    int tier_cta[3], tier_tile[3], tier_n[3], tier_ks[3], tier_spp[3], tier_slot[3];   // tier_n: tiles of the tier
    int row_tiles;    // tiles along the output channels; tile = token tile * row_tiles + row tile
    int tstride;      // rows of x per slot of partial sums (the rows of the launch's largest tile)
    int tab_bytes;    // shared-memory bytes of the look-up tables (the x stages follow)
    int L;            // V2a: library size
    int GH;           // V2a: groups per super-chunk (2 when the format's groups hold 64 weights)
    int maxT;         // rows of x per tile: kSmallT or kBigT; the accumulator's columns and the first column of the A stages
    int tmem_cols;    // tensor-memory columns of the CTA: the accumulator (maxT) and the A stages
    int ns_log;       // log2 of the A stages: 1 (two; two CTAs per SM) or 2 (four; the CTA that has the SM to itself)
    int x_stages;     // x tiles in shared memory: kXStages, or 2 when three large ones do not fit
    int b_half;       // bytes of one 64-k half of an x tile: rows of x per tile * 128 (a multiple of 1024)
    // outliers as a sparse product in the epilogue (few rows of x): x transposed, [K][Mp] fp16 with Mp a multiple of 32
    // and zeros behind row M; null: the decode warps add the outliers to the tile instead
    const uint16_t* xT;
    int Mp;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// A poll may suspend the thread for up to kPollNs before it answers (the hint of try_wait): a waiting warp then
// issues a handful of instructions per microsecond instead of competing with the decode for the ALU pipe.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity), "r"(kPollNs) : "memory");
        if (ok) return true;
    }
    return false;
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// Shared-memory operand descriptor (version 1) of a K-major tile in the 128-byte swizzle (rows of 64 fp16 = 128 bytes,
// 16-byte chunk c of row r at chunk c ^ (r & 7), the layout a tensor copy with CU_TENSOR_MAP_SWIZZLE_128B writes; base
// 1024-byte aligned): groups of 8 rows are 1024 bytes apart, the leading offset is not used (1), layout type 2.  A step of 16 k inside
// the 128-byte row advances the start address by 32 bytes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// D[128][T] (+)= A[128][16] B[T][16]^T: A from tensor memory (lane = row, column = two k), B from shared memory.
__device__ __forceinline__ void umma_f16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        :: "r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(acc) : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 16 consecutive columns of the warp's 32 tensor-memory lanes, one lane per thread.
template <int O>
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        :: "r"(taddr), "r"(r[O]), "r"(r[O + 1]), "r"(r[O + 2]), "r"(r[O + 3]), "r"(r[O + 4]), "r"(r[O + 5]),
           "r"(r[O + 6]), "r"(r[O + 7]), "r"(r[O + 8]), "r"(r[O + 9]), "r"(r[O + 10]), "r"(r[O + 11]),
           "r"(r[O + 12]), "r"(r[O + 13]), "r"(r[O + 14]), "r"(r[O + 15])
        : "memory");
}

// lo | hi << 16 for two table words whose upper halves are zero, as a multiply-add: the decode is bound by the ALU
// pipe (PRMT, LOP3, SHF), and this moves one of its operations per two weights to the FMA pipe
__device__ __forceinline__ uint32_t join16(uint32_t lo, uint32_t hi) {
    uint32_t d;
    asm("mad.lo.u32 %0, %1, 65536, %2;" : "=r"(d) : "r"(hi), "r"(lo));
    return d;
}

template <int N>
struct Tab {
    static constexpr int E = 1 << N;
    static constexpr bool kPair = N <= 3;
    static constexpr int T = kPair ? E * E : E;   // words per lane
};

// The 32-bit words [PART*2N, PART*2N + 2N) of the lane's 128*N-bit stream sit in these 16-byte vectors.
template <int N, int PART>
struct Half {
    static constexpr int W0 = PART * 2 * N, W1 = W0 + 2 * N;
    static constexpr int V0 = W0 / 4, V1 = (W1 + 3) / 4, NV = V1 - V0;
};

// A lane's outlier list (transposed slab first, the CSR arrays behind it) with the next four entries in registers:
// an entry is consumed long after its load was issued, so a channel with several outliers close together does not
// stall its warp (and, through the barrier, its CTA) on a chain of dependent loads.
struct Outliers {
    const uint32_t* slab;
    const uint32_t* spill;
    const uint32_t* nextp;      // address of entry cur + 4, the next one to load
    int step;                   // words between consecutive entries at nextp: 32 in the slab, 1 in the CSR arrays
    int nslab, total, cur;
    uint32_t col;               // column of entry cur, 0xffffffff behind the last one
    uint32_t ent, e1, e2, e3;   // entries cur .. cur + 3 (column | fp16 value << 16)
    __device__ __forceinline__ const uint32_t* addr(int j) const {
        return j < nslab ? slab + (size_t)(1 + j) * 32 : spill + j;
    }
    __device__ __forceinline__ uint32_t fetch(int j) const { return __ldg(addr(j)); }
    __device__ __forceinline__ void start(int first) {
        cur = first;
        if (cur < total) { ent = fetch(cur); }
        if (cur + 1 < total) e1 = fetch(cur + 1);
        if (cur + 2 < total) e2 = fetch(cur + 2);
        if (cur + 3 < total) e3 = fetch(cur + 3);
        col = cur < total ? (ent & 0xffffu) : 0xffffffffu;
        nextp = addr(cur + 4);
        step = cur + 4 < nslab ? 32 : 1;
    }
    __device__ __forceinline__ void advance() {
        ++cur;
        ent = e1; e1 = e2; e2 = e3;
        col = cur < total ? (ent & 0xffffu) : 0xffffffffu;
        if (cur + 3 < total) {
            e3 = __ldg(nextp);
            if (cur + 4 == nslab) { nextp = spill + nslab; step = 1; } else nextp += step;
        }
    }
};

// v[0..15] (fp32 bit patterns: the sums of one channel for 16 rows of x) += S x^T over the channel's outliers with
// columns below `kend`, starting at entry o.cur: four entries and their activations in flight at a time, added in
// ascending column order.
__device__ __forceinline__ void sparse_rows(const GemmArgs& a, const Outliers& o, int t, uint32_t kend, uint32_t (&v)[16]) {
    const uint16_t* xt = a.xT + t;
    for (int j = o.cur; j < o.total; j += 4) {
        uint32_t e[4];
        bool ok[4];
        uint4 xa[4], xb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) e[u] = j + u < o.total ? o.fetch(j + u) : 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t col = e[u] & 0xffffu;
            ok[u] = j + u < o.total && col < kend;
            const uint4* p = (const uint4*)(xt + (size_t)(ok[u] ? col : 0u) * a.Mp);
            xa[u] = __ldg(p); xb[u] = __ldg(p + 1);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (!ok[u]) continue;
            const float val = __half2float(__ushort_as_half((uint16_t)(e[u] >> 16)));
            const uint32_t xw[8] = {xa[u].x, xa[u].y, xa[u].z, xa[u].w, xb[u].x, xb[u].y, xb[u].z, xb[u].w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float2 f = __half22float2(*(const __half2*)&xw[i]);
                v[2 * i] = __float_as_uint(fmaf(val, f.x, __uint_as_float(v[2 * i])));
                v[2 * i + 1] = __float_as_uint(fmaf(val, f.y, __uint_as_float(v[2 * i + 1])));
            }
        }
        if (!ok[3]) break;
    }
}

// One K slice of one half of the row-block's super-chunks: the whole main loop of a warp.
// Barriers, with NS A stages: bars[0..NS) "products of iteration i done" (i % NS), bars[NS..NS+3) "x tile landed" (i % 3),
// bars[NS+3..) "A stage
// of iteration i stored by all eight decode warps" (i & 1).  No CTA-wide barrier inside the loop: a decode warp runs
// up to NS iterations ahead of the products.
template <int N, int MODE, int PART>
__device__ __forceinline__ bool main_loop(const GemmArgs& a, int rb, bool rb_ok, int q, int lane, int tid, int Tn,
                                          int t0, int sc0, int sc1, const unsigned char* tab, unsigned char* sB,
                                          uint64_t* bars, uint32_t tmem, Outliers& o, const CUtensorMap* tmap,
                                          int grp, int G) {
    using H = Half<N, PART>;
    const int NS = 1 << a.ns_log;
    // byte offset of the lane inside a table entry; N = 4 (V2): the row-block's half of a 256-byte entry as well
    const uint32_t tbase = (uint32_t)lane * 4u + ((MODE == 0 && N == 4) ? (uint32_t)(q & 1) * 128u : 0u);
    // V2: a row-block's table is aligned to its size in the shared window, so the entry field of an address and the
    // table's own address do not overlap: the look-ups merge them (no addition per look-up) and load from the 32-bit
    // shared address.  N = 4: the high nibble of address byte 1 rides in the index words.  (The same for V2a, whose
    // look-ups are followed by a conversion, a multiply-add and a packing per weight, measured no faster.)
    const uint32_t tabs = smem_u32(tab) + tbase;
    const uint32_t nib = ((tabs >> 12) & 0xfu) * 0x10101010u;
    const uint4* idx = a.b.idx + ((size_t)rb * a.SC + sc0 + grp) * N * 32 + lane;   // advanced by G*N*32 per iteration of this warp
    // index vectors of the next two super-chunks in registers
    uint4 nx[2][H::NV];
    if (rb_ok) {
#pragma unroll
        for (int ahead = 0; ahead < 2; ++ahead) {
            if (sc0 + grp + ahead * G < sc1) {
#pragma unroll
                for (int v = 0; v < H::NV; ++v) nx[ahead][v] = ld_stream(idx + (size_t)ahead * G * N * 32 + (size_t)(H::V0 + v) * 32);
            }
        }
    }
    // V2a: library id, scale and mid-point of the lane's channel for this warp's half of the next super-chunk, one
    // ahead.  A half is 64 weights: a group of its own when the format's groups hold 64 weights (GH = 2), else half
    // of the super-chunk's group.
    const size_t meta0 = (((size_t)rb * a.SC + sc0) * a.GH + (a.GH - 1) * PART) * 32 + lane;
    uint32_t gid_n = 0, gsm_n = 0;
    if (MODE == 1 && rb_ok && sc0 + grp < sc1) {
        gid_n = __ldg(a.b.gid + meta0 + (size_t)grp * a.GH * 32); gsm_n = __ldg(a.b.gsm + meta0 + (size_t)grp * a.GH * 32);
    }
    bool ok = true;
    int it = grp;
    for (int sc = sc0 + grp; sc < sc1; sc += G, it += G) {
        const int s = it & (NS - 1);
        // The A stage written below was read by the products of iteration it - NS.
        if (it >= NS && ok) {
            ok = mbar_wait(smem_u32(&bars[s]), (uint32_t)((it >> a.ns_log) - 1) & 1u);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        if (!ok) break;
        const uint32_t k0 = (uint32_t)sc * kSuper;
        uint32_t d[32];
        if (rb_ok) {
            uint32_t w[4 * N + 1];
#pragma unroll
            for (int i = 0; i <= 4 * N; ++i) w[i] = 0u;
#pragma unroll
            for (int v = 0; v < H::NV; ++v) {
                w[4 * (H::V0 + v)] = nx[0][v].x; w[4 * (H::V0 + v) + 1] = nx[0][v].y;
                w[4 * (H::V0 + v) + 2] = nx[0][v].z; w[4 * (H::V0 + v) + 3] = nx[0][v].w;
                nx[0][v] = nx[1][v];
            }
            idx += G * N * 32;
            if (sc + 2 * G < sc1) {
#pragma unroll
                for (int v = 0; v < H::NV; ++v) nx[1][v] = ld_stream(idx + (size_t)G * N * 32 + (size_t)(H::V0 + v) * 32);
            }
            // 64 look-ups in one straight block (every load can be in flight at once)
            float g_scale = 0.f, g_mid = 0.f;
            uint32_t vbase = tbase;
            if (MODE == 1) {
                // D16 = fp16(fp32(scale * lib[id][q] + mid)): the product of two fp16 values is exact in fp32, so the
                // fused multiply-add rounds once, as the format defines it
                const __half2 sm = *(const __half2*)&gsm_n;
                g_scale = __low2float(sm); g_mid = __high2float(sm);
                vbase = tbase | (gid_n << (7 + N));
                if (sc + G < sc1) {
                    const size_t mi = meta0 + (size_t)(it + G) * a.GH * 32;
                    gid_n = __ldg(a.b.gid + mi); gsm_n = __ldg(a.b.gsm + mi);
                }
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int p = PART * 32 + i;
                if (MODE == 1) {
                    const uint32_t lo = *(const uint32_t*)(tab + single_addr<N, 1>(w, 2 * p, vbase));
                    const uint32_t hi = *(const uint32_t*)(tab + single_addr<N, 1>(w, 2 * p + 1, vbase));
                    const float f0 = __fmaf_rn(g_scale, __half2float(__ushort_as_half((uint16_t)lo)), g_mid);
                    const float f1 = __fmaf_rn(g_scale, __half2float(__ushort_as_half((uint16_t)hi)), g_mid);
                    const __half2 r = __floats2half2_rn(f0, f1);
                    d[i] = *(const uint32_t*)&r;
                } else if (Tab<N>::kPair) {
                    d[i] = lds32(pair_addr<N, 1>(w, p, tabs));
                } else if (N == 4) {
                    // entries 256 bytes apart (two row-blocks share a table): an index, isolated in its own byte,
                    // becomes the second byte of the address with one PRMT.  Pair p = byte p & 3 of word p >> 2.
                    const uint32_t wlo = (w[p >> 2] & 0x0f0f0f0fu) | nib, whi = ((w[p >> 2] >> 4) & 0x0f0f0f0fu) | nib;
                    const uint32_t sel = 0x7604u | ((uint32_t)(p & 3) << 4);   // [tabs.b3, tabs.b2, index byte, tabs.b0]
                    const uint32_t lo = lds32(__byte_perm(wlo, tabs, sel));
                    const uint32_t hi = lds32(__byte_perm(whi, tabs, sel));
                    d[i] = join16(lo, hi);
                } else {
                    const uint32_t lo = lds32(single_addr<N, 1>(w, 2 * p, tabs));
                    const uint32_t hi = lds32(single_addr<N, 1>(w, 2 * p + 1, tabs));
                    d[i] = join16(lo, hi);
                }
            }
            // W^ = fp16(D16 + S) at the outliers of this channel inside this half; the entries of the other half
            // (the other warp's) are passed over.  One loop, one copy of the code that advances the list.
            const uint32_t lo_k = k0 + PART * 64;
            // warp-uniform loop (as many trips as the busiest lane needs, the lanes converged at the top of each)
            while (__any_sync(0xffffffffu, o.col < k0 + kSuper)) {
                const bool mine_now = o.col < k0 + kSuper;
                const uint32_t kk = o.col - lo_k;              // wraps around for entries below this half
                if (mine_now && kk < 64u) {
                    const uint32_t v2 = (o.ent >> 16) << ((kk & 1u) * 16u);
                    // the register that holds weight kk: found by nested tests, not a switch -- the indirect
                    // branch of a jump table inside this divergent loop stalled the warps (176 vs 149 us on
                    // 28672 x 8192 with 0.3 % outliers, same instruction count)
                    const uint32_t r = kk >> 1;
#define XFP_OUT_GROUP(g)                                                                                          \
    if ((r >> 2) == g##u)                                                                                         \
        asm("{\n\t.reg .pred p0, p1, p2, p3;\n\t"                                                                 \
            "setp.eq.u32 p0, %4, 0;\n\tsetp.eq.u32 p1, %4, 1;\n\t"                                                 \
            "setp.eq.u32 p2, %4, 2;\n\tsetp.eq.u32 p3, %4, 3;\n\t"                                                 \
            "@p0 add.rn.f16x2 %0, %0, %5;\n\t@p1 add.rn.f16x2 %1, %1, %5;\n\t"                                     \
            "@p2 add.rn.f16x2 %2, %2, %5;\n\t@p3 add.rn.f16x2 %3, %3, %5;\n\t}"                                    \
            : "+r"(d[4 * g]), "+r"(d[4 * g + 1]), "+r"(d[4 * g + 2]), "+r"(d[4 * g + 3])                          \
            : "r"(r & 3u), "r"(v2));
                    if (r < 16u) {
                        if (r < 8u) { XFP_OUT_GROUP(0) XFP_OUT_GROUP(1) } else { XFP_OUT_GROUP(2) XFP_OUT_GROUP(3) }
                    } else {
                        if (r < 24u) { XFP_OUT_GROUP(4) XFP_OUT_GROUP(5) } else { XFP_OUT_GROUP(6) XFP_OUT_GROUP(7) }
                    }
#undef XFP_OUT_GROUP
                }
                if (mine_now) o.advance();
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) d[i] = 0u;
        }
        const uint32_t ta = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(a.maxT + s * kAStageCols + PART * 32);
        tmem_st16<0>(ta, d);
        tmem_st16<16>(ta + 16, d);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(&bars[NS + kXStages + s])) : "memory");
    }
    // all products of this CTA are complete when the last commit has arrived
    // this warp's last iteration: its commit is on the barrier this warp has followed (the other group's is not);
    // the CTA-wide vote behind the loops then covers the very last commit through the warps that waited for it
    const int lastit = it - G;
    if (lastit < 0) return ok;
    return ok && mbar_wait(smem_u32(&bars[lastit & (NS - 1)]), (uint32_t)(lastit >> a.ns_log) & 1u);
}

// The ninth warp (one thread): x tiles by tensor copy one iteration ahead, the eight products of every stage.
__device__ __forceinline__ bool mma_loop(const GemmArgs& a, int Tn, int t0, int sc0, int sc1, unsigned char* sB,
                                         uint64_t* bars, uint32_t tmem, const CUtensorMap* tmap) {
    const uint32_t idesc = (1u << 4) | ((uint32_t)(Tn >> 3) << 17) | ((uint32_t)(kTileRows >> 4) << 24);
    const int NS = 1 << a.ns_log;
    const int b_stage = 2 * a.b_half;
    const uint32_t x_bytes = (uint32_t)b_stage;
    auto stage_x = [&](int sc, int xs) {
        // two tensor copies, one per 64-k half: box {64 k, rows of x} of x [M][K], 128-byte rows in the 128-byte swizzle;
        // rows beyond M arrive as zeros
        const uint32_t bar = smem_u32(&bars[NS + xs]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(x_bytes) : "memory");
#pragma unroll
        for (int h = 0; h < 2; ++h)
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                :: "r"(smem_u32(sB + xs * b_stage + h * a.b_half)), "l"(tmap), "r"(sc * kSuper + h * 64), "r"(t0), "r"(bar)
                : "memory");
    };
    stage_x(sc0, 0);
    int it = 0, xs = 0;                       // xs = it % x_stages
    uint32_t xuse = 0;                        // it / x_stages
    for (int sc = sc0; sc < sc1; ++sc, ++it) {
        const int s = it & (NS - 1);
        const int xn = xs + 1 == a.x_stages ? 0 : xs + 1;
        // the x stage refilled now was read by the products of iteration it + 1 - x_stages
        const int jf = it + 1 - a.x_stages;
        if (jf >= 0 && !mbar_wait(smem_u32(&bars[jf & (NS - 1)]), (uint32_t)(jf >> a.ns_log) & 1u)) return false;
        if (sc + 1 < sc1) stage_x(sc + 1, xn);
        if (!mbar_wait(smem_u32(&bars[NS + kXStages + s]), (uint32_t)(it >> a.ns_log) & 1u)) return false;   // A stage stored
        if (!mbar_wait(smem_u32(&bars[NS + xs]), xuse & 1u)) return false;   // x tile landed
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t b0 = smem_u32(sB + xs * b_stage);
#pragma unroll
        for (int ks = 0; ks < kSuper / 16; ++ks) {
            const uint64_t db = smem_desc_sw128(b0 + (uint32_t)(ks >> 2) * (uint32_t)a.b_half + (uint32_t)(ks & 3) * 32u);
            umma_f16_ts(tmem, tmem + (uint32_t)(a.maxT + s * kAStageCols + ks * 8), db, idesc, (it > 0 || ks > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&bars[s]));
        xs = xn;
        if (xn == 0) ++xuse;
    }
    const int lastit = it - 1;
    return mbar_wait(smem_u32(&bars[lastit & (NS - 1)]), (uint32_t)(lastit >> a.ns_log) & 1u);
}

// A CTA's place in the schedule: its tile, its K slice of `spp` super-chunks, the slices of the tile and the first
// slot of their partial sums.
struct Work { int tile, slice, ks, spp, slot0; };
__device__ __forceinline__ Work work_of(const GemmArgs& a, int cta) {
    int tier = 0;
#pragma unroll
    for (int i = 1; i < 3; ++i)
        if (cta >= a.tier_cta[i]) tier = i;
    // inside a tier the tiles run fastest: the CTAs of one K slice are neighbours in launch order
    const int ks = a.tier_ks[tier], n = a.tier_n[tier], cl = cta - a.tier_cta[tier], slice = cl / n, ti = cl - slice * n;
    return Work{a.tier_tile[tier] + ti, slice, ks, a.tier_spp[tier], a.tier_slot[tier] + ti * ks};
}

template <int N, int MODE, bool BIG>
__global__ void __launch_bounds__(threads_of(BIG), BIG ? 1 : 2) gemm_tc_kernel(const GemmArgs a, const __grid_constant__ CUtensorMap tmap) {
    constexpr int E = Tab<N>::E;
    constexpr int TW = Tab<N>::T;
    extern __shared__ __align__(1024) unsigned char smem[];
    // V2: [4 row-blocks][TW][32] words, the start rounded up to 8 KB in the shared window (the size of the largest
    // row-block table; the host leaves that much room); V2a: [L * E][32] words
    unsigned char* sTab = smem + (MODE == 0 ? (8192u - (smem_u32(smem) & 8191u)) & 8191u : 0u);
    unsigned char* sB = smem + a.tab_bytes;           // the x stages, two swizzled halves each (1024-byte aligned)
    __shared__ __align__(8) uint64_t bars[8 + kXStages];
    __shared__ uint32_t s_tmem;
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int G = BIG ? 2 : 1, DW = G * kWarps;            // groups, decode warps
    const int q = warp & 3, part = (warp >> 2) & 1, grp = warp >> 3;   // row-block of the tile, half of the super-chunk, group
    const Work wk = work_of(a, (int)blockIdx.x);
    const int tile = wk.tile, slice = wk.slice;
    const int tile_x = tile % a.row_tiles, tile_y = tile / a.row_tiles;
    const int rb = tile_x * 4 + q;
    const bool rb_ok = rb < a.RB && warp < DW;
    const int row = rb * kRowsPerBlock + lane;
    const int t0 = tile_y * a.maxT;
    const int Tn = min(a.maxT, (a.M - t0 + 15) & ~15);          // rows of x of this tile, rounded up to 16
    const int sc0 = slice * wk.spp;
    const int sc1 = min(a.SC, sc0 + wk.spp);

    // ---- set-up: barriers, tensor memory, tables ----
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < 8 + kXStages; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bars[i])), "r"(i >= (1 << a.ns_log) + kXStages ? kWarps : 1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&s_tmem)), "r"(a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (MODE == 1) {
        // the library, every entry replicated once per bank: word (id * E + q) * 32 + lane
        const int n = a.L * E;
        for (int i = warp; i < n; i += DW + 1) ((uint32_t*)sTab)[i * 32 + lane] = (uint32_t)__ldg(a.b.cb + i);
    } else {
        // codebooks -> one word per (entry, lane); pair tables are built from a copy staged in the x stages
        uint32_t* one = Tab<N>::kPair ? (uint32_t*)sB : (uint32_t*)sTab;
        for (int i = warp; i < 4 * E; i += DW + 1) {
            const int qq = i / E, e = i % E, r = (tile_x * 4 + qq) * kRowsPerBlock + lane;
            const int slot = N == 4 ? ((qq >> 1) * E + e) * 64 + (qq & 1) * 32 : (qq * E + e) * 32;   // N = 4: see the look-ups
            one[slot + lane] = (tile_x * 4 + qq) < a.RB ? (uint32_t)__ldg(a.b.cb + (size_t)r * E + e) : 0u;
        }
        if (Tab<N>::kPair) {
            __syncthreads();
            uint32_t* tab = (uint32_t*)sTab;
            for (int i = warp; i < 4 * TW; i += DW + 1) {
                const int qq = i / TW, t = i % TW;
                tab[(qq * TW + t) * 32 + lane] =
                    one[(qq * E + (t & (E - 1))) * 32 + lane] | (one[(qq * E + (t >> N)) * 32 + lane] << 16);
            }
        }
    }
    // the tables were written through the generic proxy where the first tensor copy (async proxy) lands
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    // ---- the lane's outlier list: transposed slab first, the CSR arrays behind it ----
    Outliers o{nullptr, nullptr, nullptr, 1, 0, 0, 0, 0xffffffffu, 0u, 0u, 0u, 0u};
    if (rb_ok && a.ell_slots) {
        o.slab = a.b.ell + (size_t)rb * (a.ell_slots + 1) * 32 + lane;
        const int olen = (int)__ldg(o.slab);
        o.nslab = min(olen, a.ell_slots);
        o.total = o.nslab;
        if (olen >= a.ell_slots && row < a.rows) {
            const int p0 = __ldg(a.b.rowptr + row);
            o.total = __ldg(a.b.rowptr + row + 1) - p0;
            o.spill = a.b.oent + p0;
        }
        // first entry of this K slice: the list ascends, so count the entries below the slice, sixteen
        // independent loads at a time (a coarse pass over every 16th entry, then the 15 before the first hit)
        int first = 0;
        if (sc0 > 0 && o.total) {
            const uint32_t kb = (uint32_t)sc0 * kSuper;
            int coarse = 0;
            for (int j = 15; j < o.total; j += 16) coarse += (o.fetch(j) & 0xffffu) < kb;
            first = coarse * 16;
            int fine = 0;
#pragma unroll
            for (int j = 0; j < 15; ++j) fine += (first + j < o.total) && (o.fetch(min(first + j, o.total - 1)) & 0xffffu) < kb;
            first += fine;
        }
        if (a.xT) { o.cur = first; o.col = 0xffffffffu; }   // the epilogue walks the list from `first`
        else o.start(first);
    }

    const unsigned char* tab = MODE == 1 ? sTab : N == 4 ? sTab + (size_t)(q >> 1) * TW * 256 : sTab + (size_t)q * TW * 128;
    bool done;
    if (warp == DW) {
        done = lane != 0 || mma_loop(a, Tn, t0, sc0, sc1, sB, bars, tmem, &tmap);
        __syncwarp();
    } else {
        done = part == 0
            ? main_loop<N, MODE, 0>(a, rb, rb_ok, q, lane, tid, Tn, t0, sc0, sc1, tab, sB, bars, tmem, o, &tmap, grp, G)
            : main_loop<N, MODE, 1>(a, rb, rb_ok, q, lane, tid, Tn, t0, sc0, sc1, tab, sB, bars, tmem, o, &tmap, grp, G);
    }
    // what the finish needs of the schedule is worked out again from a fresh read of the CTA index, so that it does
    // not occupy registers through the main loop
    uint32_t cta_again;
    asm volatile("mov.u32 %0, %%ctaid.x;" : "=r"(cta_again));
    const Work wf = work_of(a, (int)cta_again);
    const int ks = wf.ks, slot0 = wf.slot0;
    const bool failed = __syncthreads_or(!done) != 0;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (failed) {
        if (tid == 0) atomicExch(a.ctrl, 1);
    } else {
        // lane = channel (tensor-memory lane 32*(warp%4) + lane), registers = 16 consecutive rows of x
        const int r = q * 32 + lane;
        float* part_out = a.partial + (size_t)(slot0 + slice) * a.tstride * kTileRows;
        for (int cc = part + 2 * grp; warp < DW && cc * 16 < Tn; cc += 2 * G) {
            uint32_t v[16];
            tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 16), v);
            if (a.xT && rb_ok) sparse_rows(a, o, t0 + cc * 16, (uint32_t)sc1 * kSuper, v);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int t = cc * 16 + j;
                if (ks > 1) part_out[t * kTileRows + r] = __uint_as_float(v[j]);
                else if (t0 + t < a.M && row < a.rows) put_y(a.y, (size_t)(t0 + t) * a.rows + row, __uint_as_float(v[j]), a.y_kind);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(a.tmem_cols) : "memory");
    if (failed || ks == 1) return;

    // ---- K slices: the last CTA of the tile to arrive adds the slices in slice order ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(a.ctrl + 1 + tile, 1);
        s_last = ticket == ks - 1;
        if (s_last) a.ctrl[1 + tile] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // four consecutive channels of one row of x per thread and step: 16-byte loads, all slices of a step in flight
    const float4* p0 = (const float4*)(a.partial + (size_t)slot0 * a.tstride * kTileRows);
    constexpr int kQuads = kTileRows / 4;
    for (int i = tid; i < Tn * kQuads; i += (DW + 1) * 32) {
        const int t = i / kQuads, r = (i % kQuads) * 4;
        const int orow = tile_x * kTileRows + r;
        if (t0 + t >= a.M || orow >= a.rows) continue;
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int z = 0; z < ks; ++z) {
            const float4 v = __ldcg(p0 + (size_t)z * (a.tstride * kQuads) + i);
            sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
        const size_t o0 = (size_t)(t0 + t) * a.rows + orow;
        put_y(a.y, o0, sum.x, a.y_kind);
        if (orow + 1 < a.rows) put_y(a.y, o0 + 1, sum.y, a.y_kind);
        if (orow + 2 < a.rows) put_y(a.y, o0 + 2, sum.z, a.y_kind);
        if (orow + 3 < a.rows) put_y(a.y, o0 + 3, sum.w, a.y_kind);
    }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (the library does not link libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
        return nullptr;
    return (EncodeTiledFn)fn;
}

// x [M][K] fp16 -> xT [K][Mp] fp16 (zeros behind row M): tiles of 32 rows x 64 k through shared memory.
__global__ void __launch_bounds__(256) x_transpose_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ xT,
                                                          int M, int K, int Mp) {
    __shared__ uint16_t tile[64][34];   // [k][t]
    const int tid = threadIdx.x, k0 = blockIdx.x * 64, t0 = blockIdx.y * 32;
    for (int r = tid >> 5; r < 32; r += 8) {
        const int t = t0 + r, kk = 2 * (tid & 31);
        const uint32_t w = t < M ? __ldg((const uint32_t*)(x + (size_t)t * K + k0 + kk)) : 0u;
        tile[kk][r] = (uint16_t)w; tile[kk + 1][r] = (uint16_t)(w >> 16);
    }
    __syncthreads();
    for (int kk = tid >> 4; kk < 64; kk += 16) {
        const int tt = 2 * (tid & 15);
        *(uint32_t*)(xT + (size_t)(k0 + kk) * Mp + t0 + tt) = (uint32_t)tile[kk][tt] | ((uint32_t)tile[kk][tt + 1] << 16);
    }
}

struct Plan {
    int row_tiles, tok_tiles;
    // K slices in up to three tiers of tiles (see schedule_tiles); slots: (tile, slice) pairs that store partial sums
    int tier_cta[3], tier_tile[3], tier_n[3], tier_ks[3], tier_spp[3], tier_slot[3];
    int grid, slots;
    int maxT, x_stages;
    bool lone;        // the CTA with 16 decode warps, alone on its SM (else 8 decode warps, two CTAs per SM)
    size_t tab_bytes, smem;
};

constexpr size_t kSmemLimit = 227 * 1024 - 1024;   // dynamic shared memory a CTA may ask for, less the static part

// Which tiles are cut along K, and how finely, so that every SM gets about the same number of super-chunks.  The two
// CTAs of an SM share its throughput (148 tiles, one per SM: 41.5 us; 296 tiles: 72.9 us; and 224 whole tiles took as
// long as 296, the SMs with two of them setting the time), so what counts is the work per SM, not per CTA slot:
//   * at most half as many tiles as slots: every tile in the same number of slices;
//   * else the whole rounds of slots run whole tiles, and so does one tile per SM of the last partial round (two
//     CTAs per SM only); what remains of that round is cut to fill the remaining slots, in tiers of finer slices
//     (74 tiles in halves fill 148 slots, the last 2 tiles go in 32 slices each), CTAs in launch order.
// A slice holds at least two super-chunks, and a tile at most 32 slices (fewer for many rows of x).  Slices store fp32 partial sums; the last CTA of a tile adds them.
void schedule_tiles(Plan& p, int tiles, int SC, int sms, int tmax) {
    const int S = p.lone ? sms : 2 * sms;
    const int kfine = SC / 2 > 1 ? SC / 2 : 1;     // a slice holds at least two super-chunks
    // the tail of a large matrix: the CTA that adds a tile's slices reads slices x rows of x x 512 bytes at the very
    // end of the launch, at most 256 KB of them (32 slices at 16 rows of x, 4 at 128)
    const int kcap = 512 / tmax > 2 ? 512 / tmax : 2;
    const int kmax = kfine < kcap ? kfine : kcap;
    int nb[3] = {0, 0, 0}, kk[3] = {1, 1, 1}, nt = 0;
    if (tiles * 2 <= S) {
        // powers of two while the slices fill at most the slots (more, finer slices cost more in set-up and sums than
        // the idle slots: 4096 x 4096 at 16 rows of x, 4 slices 27.3 us, 8 slices 29.7), or three where two leave a
        // third of the slots idle (12288 x 4096: 58.4 -> 52.6 us)
        int k = 1;
        while (tiles * k * 2 <= S && k * 2 <= kfine) k *= 2;
        if (k == 2 && tiles * 3 <= S && 3 <= kfine) k = 3;
        nb[0] = tiles; kk[0] = k; nt = 1;
    } else {
        int whole = (tiles / S) * S, rem = tiles - whole, S2 = S;
        if (!p.lone && rem > sms) { whole += sms; rem -= sms; S2 = S - sms; }
        if (whole) { nb[nt] = whole; kk[nt] = 1; ++nt; }
        int k = 2;
        while (rem > 0) {
            const int cap = S2 / k;
            if (k >= kmax || rem <= cap || nt == 2) {
                int kl = S2 / rem;                     // as many slices as fill the slots once
                if (kl < 1) kl = 1;
                if (kl > kmax) kl = kmax;
                nb[nt] = rem; kk[nt] = kl; ++nt; rem = 0;
            } else {
                nb[nt] = cap; kk[nt] = k; ++nt; rem -= cap;
                k *= 2;
            }
        }
    }
    int cta = 0, tile = 0, slot = 0;
    for (int i = 0; i < 3; ++i) {
        const int k = i < nt ? kk[i] : 1;
        const int spp = (SC + k - 1) / k, ks = (SC + spp - 1) / spp;
        p.tier_cta[i] = i < nt ? cta : 0x7fffffff;
        p.tier_tile[i] = tile; p.tier_n[i] = i < nt ? nb[i] : 1; p.tier_ks[i] = ks; p.tier_spp[i] = spp; p.tier_slot[i] = slot;
        if (i < nt) { cta += nb[i] * ks; tile += nb[i]; if (ks > 1) slot += nb[i] * ks; }
    }
    p.grid = cta; p.slots = slot;
}

// `sms`: SMs to plan for (kSizingSMs when sizing the workspace, the device's own count, capped by it, at launch)
Plan plan_of(const Layout& l, int M, int sms) {
    Plan p;
    p.tab_bytes = l.mode == 1 ? (size_t)l.L * l.E * 128 : (size_t)4 * (l.bits <= 3 ? l.E * l.E : l.E) * 128;
    if (l.mode == 0) p.tab_bytes += 8192;                    // room to align the tables to 8 KB in the shared window
    p.tab_bytes = (p.tab_bytes + 1023) & ~size_t(1023);      // the x stages behind the tables are 1024-byte aligned
    // More than 128 rows of x: tiles of 256 rows (one CTA per SM with two groups of decode warps, all 512 tensor-memory
    // columns), which decode the weights once per 256 rows -- 28672 x 8192, M = 512: 555 -> 450 us; 4096 x 4096,
    // M = 512: 80 -> 72 us -- when their x stages fit beside the tables.
    p.maxT = kSmallT; p.x_stages = kXStages; p.lone = false;
    // the same CTA shape (16 decode warps, alone on its SM) also serves fewer rows of x when the tables leave no room
    // for two CTAs of 128-row tiles on an SM (V2a from N = 4: a 64 KB library; 28672 x 8192, M = 128: 274 us with one
    // CTA of 8 decode warps per SM)
    const int tsmall = M >= kSmallT ? kSmallT : (M + 15) & ~15;
    const bool lone_anyway = p.tab_bytes + (size_t)2 * tsmall * 256 > 113 * 1024;
    if (M > kSmallT || lone_anyway) {
        for (int xs = kXStages; xs >= 2; --xs) {
            const int tbig = M >= kBigT ? kBigT : (M + 15) & ~15;    // rows of x its largest tile would hold
            if (p.tab_bytes + (size_t)xs * tbig * 256 <= kSmemLimit) { p.maxT = kBigT; p.x_stages = xs; p.lone = true; break; }
        }
        // tables too large for 256-row x stages (V2a, N = 5: 128 KB): the lone CTA with 128-row tiles
        if (!p.lone && lone_anyway) { p.lone = true; p.x_stages = 2; }
    }
    const int tmax = M >= p.maxT ? p.maxT : (M + 15) & ~15;    // rows of x in the largest tile of this launch
    // 128-row tiles: two x stages instead of three where that keeps two CTAs on an SM (N = 3 pair tables and N = 6
    // tables are 32 KB: 28672 x 8192, M = 128, N = 3: 216 us with one CTA per SM)
    if (!p.lone && p.tab_bytes + (size_t)kXStages * tmax * 256 > 113 * 1024 &&
        p.tab_bytes + (size_t)2 * tmax * 256 <= 113 * 1024)
        p.x_stages = 2;
    p.smem = p.tab_bytes + (size_t)p.x_stages * 16 * tmax * 16;
    if (p.smem < kMinSmem) p.smem = kMinSmem;
    if (p.lone && p.smem < 120 * 1024) p.smem = 120 * 1024;   // alone on its SM: it may hold all 512 columns
    p.row_tiles = (l.RB + 3) / 4;
    p.tok_tiles = (M + p.maxT - 1) / p.maxT;
    schedule_tiles(p, p.row_tiles * p.tok_tiles, l.SC, sms, tmax);
    return p;
}

size_t partial_offset(const Layout& l, int M);
size_t partial_bytes(const Plan& p, int M);

template <int N, int MODE>
cudaError_t launch_n(const Layout& l, const GemmCall& c, cudaStream_t s) {
    Plan p = plan_of(l, c.M, sched_sms());
    // workspaces are sized for kSizingSMs: a device with fewer SMs whose own schedule wants more slots takes that one
    if (partial_bytes(p, c.M) > partial_bytes(plan_of(l, c.M, kSizingSMs), c.M)) p = plan_of(l, c.M, kSizingSMs);
    const int tmax = c.M >= p.maxT ? p.maxT : (c.M + 15) & ~15;  // rows of x in the largest tile of this launch
    const int b_half = tmax * 128;
    const size_t tab_bytes = p.tab_bytes, smem = p.smem;
    // x [M][K] fp16: a box of 64 k x tmax rows lands as 128-byte rows in the 128-byte swizzle, the B operand's layout
    static const EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    CUtensorMap tmap;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)l.cols, (cuuint64_t)c.M};
        const cuuint64_t strides[1] = {(cuuint64_t)l.cols * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)tmax};
        const cuuint32_t estr[2] = {1, 1};
        if (encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<uint16_t*>(c.x), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<N, MODE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemLimit);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(gemm_tc_kernel<N, MODE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kSmemLimit);
        if (e != cudaSuccess) return e;
        attr_done.set(dev);
    }
    GemmArgs a;
    a.b = blob_at(c.packed, offsets_of(l));
    a.y = c.y;
    a.ctrl = (int*)c.workspace;
    a.partial = (float*)((char*)c.workspace + partial_offset(l, c.M));
    a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.M = c.M; a.ell_slots = l.ell_slots;
    a.GH = l.GH;
    a.y_kind = c.y_kind; a.b_half = b_half;
    for (int i = 0; i < 3; ++i) {
        a.tier_cta[i] = p.tier_cta[i]; a.tier_tile[i] = p.tier_tile[i]; a.tier_n[i] = p.tier_n[i]; a.tier_ks[i] = p.tier_ks[i];
        a.tier_spp[i] = p.tier_spp[i]; a.tier_slot[i] = p.tier_slot[i];
    }
    a.row_tiles = p.row_tiles; a.tstride = tmax;
    a.tab_bytes = (int)tab_bytes; a.L = l.L;
    // two A stages beside the accumulator; the CTA that has its SM to itself takes all 512 columns and four stages, so
    // that a group of decode warps does not wait for the products of its previous iteration before it stores the next
    a.maxT = p.maxT; a.x_stages = p.x_stages;
    a.ns_log = p.lone ? 2 : 1;
    a.tmem_cols = p.lone ? 512 : 2 * p.maxT;
    a.xT = nullptr; a.Mp = (c.M + 31) & ~31;
    const size_t xt_off = gemm_xt_offset(l, c.M), xt_bytes = gemm_xt_bytes(l, c.M);
    if (xt_bytes && c.workspace_bytes >= xt_off + xt_bytes) {
        uint16_t* xT = (uint16_t*)((char*)c.workspace + xt_off);
        x_transpose_kernel<<<dim3((unsigned)(l.cols / 64), (unsigned)(a.Mp / 32)), 256, 0, s>>>(c.x, xT, c.M, l.cols, a.Mp);
        a.xT = xT;
    }
    const dim3 grid((unsigned)p.grid, 1, 1);
    if (p.lone)
        gemm_tc_kernel<N, MODE, true><<<grid, threads_of(true), smem, s>>>(a, tmap);
    else
        gemm_tc_kernel<N, MODE, false><<<grid, threads_of(false), smem, s>>>(a, tmap);
    return cudaGetLastError();
}

}  // namespace

bool gemm_tc_supported(const Layout& l, int M) {
    if (M < 1 || (long long)((M + kSmallT - 1) / kSmallT) > 65535) return false;
    return l.mode == 0 || (size_t)l.L * l.E * 128 <= kV2aTabMax;
}

size_t gemm_ctrl_bytes(const Layout& l, int M) {
    const Plan p = plan_of(l, M, kSizingSMs);
    return align256((size_t)(1 + p.row_tiles * p.tok_tiles) * 4);
}

namespace {
// Partial sums start behind the counters, and behind the counter region that the GEMV kernels want left zero-filled (a
// batch sent here by xfp_gemv brings the GEMV's workspace).
size_t partial_offset(const Layout& l, int M) {
    const size_t ctrl = gemm_ctrl_bytes(l, M), tickets = align256((size_t)l.RB * 4);
    return ctrl > tickets ? ctrl : tickets;
}
size_t partial_bytes(const Plan& p, int M) {
    const int tmax = M >= p.maxT ? p.maxT : (M + 15) & ~15;      // rows of x in the largest tile: the rows of a slot
    return (size_t)p.slots * tmax * kTileRows * 4;
}
}  // namespace

size_t gemm_core_bytes(const Layout& l, int M) {
    const Plan p = plan_of(l, M, kSizingSMs);
    return p.slots ? partial_offset(l, M) + partial_bytes(p, M) : gemm_ctrl_bytes(l, M);
}

// the transposed copy of x for the sparse outlier product: up to kSparseRows rows of x on a matrix with outliers
size_t gemm_xt_bytes(const Layout& l, int M) {
    if (l.nnz == 0 || M > kSparseRows) return 0;
    return align256((size_t)l.cols * ((M + 31) & ~31) * 2);
}

// where the transposed copy starts: behind the counters and partial sums, and behind the GEMV kernels' counter region
size_t gemm_xt_offset(const Layout& l, int M) {
    const size_t core = align256(gemm_core_bytes(l, M)), tickets = align256((size_t)l.RB * 4);
    return core > tickets ? core : tickets;
}

size_t gemm_workspace_bytes(const Layout& l, int M) {
    const size_t xt = gemm_xt_bytes(l, M);
    return xt ? gemm_xt_offset(l, M) + xt : gemm_core_bytes(l, M);
}

namespace {
// bf16 rows of x -> fp16 (round to nearest even, clamped to the finite fp16 range), eight values per thread and step
__global__ void x_to_f16_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n8) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = x8_as_f16(__ldg(src + i), 1);
}
}  // namespace

size_t gemm_x_scratch_bytes(const Layout& l, int M) { return align256((size_t)M * l.cols * 2); }

cudaError_t launch_x_to_f16(const void* x_bf16, void* x_f16, size_t elems, cudaStream_t s) {
    const size_t n8 = elems / 8;     // cols is a multiple of 128
    const size_t cap = (size_t)sm_count() * 8;
    const unsigned grid = (unsigned)((n8 + 255) / 256 < cap ? (n8 + 255) / 256 : cap);
    x_to_f16_kernel<<<grid ? grid : 1, 256, 0, s>>>((const uint4*)x_bf16, (uint4*)x_f16, n8);
    return cudaGetLastError();
}

cudaError_t launch_gemm_tc(const Layout& l, const GemmCall& c, cudaStream_t s) {
    if (l.mode == 1) {
        switch (l.bits) {
            case 2: return launch_n<2, 1>(l, c, s);
            case 3: return launch_n<3, 1>(l, c, s);
            case 4: return launch_n<4, 1>(l, c, s);
            case 5: return launch_n<5, 1>(l, c, s);
            default: return launch_n<6, 1>(l, c, s);
        }
    }
    switch (l.bits) {
        case 2: return launch_n<2, 0>(l, c, s);
        case 3: return launch_n<3, 0>(l, c, s);
        case 4: return launch_n<4, 0>(l, c, s);
        case 5: return launch_n<5, 0>(l, c, s);
        default: return launch_n<6, 0>(l, c, s);
    }
}

}  // namespace xfp
