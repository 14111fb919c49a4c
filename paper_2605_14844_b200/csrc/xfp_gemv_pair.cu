// Fast fused decode GEMV for V2 blobs at batch <= 2:  y = (D + S) x.
//
// Mapping.  A CTA works on blocks of 32*RPL output channels (RPL = rows per lane: 2 for N <= 4,
// 1 for N = 5 and for matrices with few rows).  Each lane of a warp owns RPL channels (lane, lane+32
// of the block) and the warps of the CTA share K in super-chunks of 128 weights.  The channels'
// codebooks are expanded once per block into PAIR tables in shared memory: entry
// t = (cb[t & (E-1)], cb[t >> N]) as a half2, so one 32-bit shared-memory load decodes two weights
// ("codebook gather from shared memory", step 2 of the fused kernel).  The tables are laid out so
// that lane l only ever touches bank l: byte address
//     t * (128 * RPL) + channel_half * 128 + lane * 4
// hence any index pattern is bank-conflict free.
//
// Multiply-accumulate (step 4).  The looked-up half2 of a lane's channels are exactly the A
// fragment of mma.sync.m16n8k16 (f16 x f16 -> f32): fragment rows g and g+8 of lane (g, t) are that
// lane's two channels (the second is zero when RPL = 1), and its k slots are four consecutive k.
// The B fragment carries x on the "diagonal" lanes only (column n = t gets the k slots of
// lane-group t), so D[g][t] accumulates the dot product of lane (g,t)'s own channel: every lane
// keeps its own rows although the fragment nominally shares a row between four lanes.  Products
// of two fp16 numbers are exact in fp32 and the accumulation is fp32.  Columns 4..7 carry a second
// batch row.  (The scalar route, one mixed-precision FMA per weight, needs the halves unpacked
// first and measured ~8 issue slots per pair against ~3 here; that is why the dot product runs on
// the tensor pipe even at batch 1.)
//
// Outliers (step 3) ride in the same pass: xfp_pack stores every 32-row block's outliers as a
// transposed slab (slot j of channel l at slab + (1+j)*32 + l), so a warp reads one slot of all 32
// channels with one coalesced load and every lane adds val * x[col] (x gathered from the staged
// copy in shared memory) to an accumulator of its own channel.  Slots are dealt round-robin to the
// warps and consumed between super-chunks, their loads issued one iteration ahead, the first round
// before the rows' lengths are known.  Rows longer than the slab (pathological skew) finish from
// the CSR arrays.  The order of additions is fixed by the schedule, so results are reproducible.
//
// Schedule.  A CTA handles one block over all of K, or one K slice of a block.  Blocks that fill whole
// rounds of CTA slots run unsplit; the blocks of the last, partial round are cut into 2 slices, and
// what still does not fit into finer slices (tiers of decreasing piece size: the hardware
// dispatches CTAs in launch order, so the tiers pack the slots largest-first).  Partial sums of a
// cut block go through the workspace and the last CTA to arrive adds them in slice order (an atomic
// ticket, no waiting, no atomics on data).  With fewer blocks than half the slots every block is
// cut into 2, 4 or 8 slices that form a thread-block cluster and reduce through distributed shared
// memory.
//
// Launch overlap.  Weights do not depend on earlier kernels, so a CTA first issues its index,
// codebook and outlier loads and fills its pair tables, and only then executes
// griddepcontrol.wait (programmatic dependent launch) before it touches x, y or the workspace.
#include <cooperative_groups.h>

#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

constexpr int kSlotsPerRound = 4;  // outlier slots a warp keeps in flight per channel half

struct PairArgs {
    Offsets off;
    const void* packed;
    const uint16_t* x;
    void* y;
    // several blobs of one shape in one launch (typed-IO instantiations only): device pointer lists; the
    // blocks of all blobs are numbered through, blocks_per of them belong to each blob
    const void* const* packed_list;
    const uint16_t* const* x_list;
    void* const* y_list;
    int blocks_per, prob0;   // blocks per blob; first blob of this launch
    float* partial;  // [slice][NB][rows_ws]
    int* tickets;    // [blocks]
    int rows, cols, RB, SC, rows_ws, ell_slots;
    int nb, y_is_fp16, x_bf16;
    int blocks;      // blocks of 32*RPL channels
    // schedule tiers: CTAs [tier_cta[i], tier_cta[i+1]) handle blocks from tier_blk[i] on, each cut into
    // tier_kst[i] slices of tier_spp[i] super-chunks
    int tier_cta[5], tier_blk[4], tier_kst[4], tier_spp[4];
    int cluster;     // single tier with kst > 1: the kst CTAs of a block form a cluster and reduce through DSMEM
#ifdef XFP_TRACE
    unsigned long long* trace;  // timing build only: per CTA 8 globaltimer stamps
#endif
};

// Phase stamps of a timing build (-DXFP_TRACE=1); a normal build has neither the stamps nor their plumbing.
__device__ __forceinline__ void stamp(const PairArgs& a, int slot) {
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

template <int N, int NB, int RPL, int W, bool TIO>
__global__ void __launch_bounds__(W * 32, W == 8 ? 2 : 1) gemv_pair_kernel(const PairArgs a) {
    constexpr int E = 1 << N;
    constexpr bool kSingle = N > 5;            // N = 6: a pair table (4096 entries) does not fit, one entry per index
    constexpr int T = kSingle ? E : E * E;     // table entries per channel
    constexpr int ROWS = 32 * RPL;             // channels per block
    // bytes between consecutive entries: 128 per channel half; N = 4 keeps 256 also with one channel per lane,
    // so that an index byte is the table offset's second byte and one PRMT builds the address
    constexpr int SL = (RPL == 2 || N == 4) ? 2 : 1;
    constexpr int kStride = 128 * SL;
    // one channel per lane at batch 1: the fragment's second row slot carries the channel's NEXT four weights
    // and columns 4..7 of the B fragment their x, so one mma covers 8 consecutive k
    constexpr bool kDual = (RPL == 1 && NB == 1 && !kSingle);
    constexpr int kTabBytes = T * kStride;
    constexpr int kThreads = W * 32;
    constexpr int TW = T / W;                  // table entries a warp fills per channel half
    extern __shared__ __align__(16) unsigned char smem[];
    // [tables | x fp16 [NB][K] | red[W][NB][ROWS]]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    stamp(a, 0);
    Blob b = blob_at(a.packed, a.off);
    const int K = a.SC * kSuper;

    unsigned char* tab = smem;
    uint16_t* xs = (uint16_t*)(smem + kTabBytes);               // [NB][K]
    float* red = (float*)(xs + (size_t)NB * K);                 // [W][NB][ROWS]

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
        slice = c % nslices;
        sc0 = slice * a.tier_spp[tier];
        nsc = max(0, min(a.SC, sc0 + a.tier_spp[tier]) - sc0);
    }
    // the blob of this block: `blk` numbers the blocks of the whole launch, `lblk` those of its blob
    int lblk = blk;
    const uint16_t* xsrc = a.x;
    void* ydst = a.y;
    int ell_slots = a.ell_slots;
    const uint32_t* ell = b.ell;
    if (TIO && a.packed_list) {
        const int pj = blk / a.blocks_per;
        const int prob = a.prob0 + pj;
        lblk = blk - pj * a.blocks_per;
        const void* packed = a.packed_list[prob];
        xsrc = a.x_list[prob]; ydst = a.y_list[prob];
        b = blob_at(packed, a.off);
        // the blobs' outlier counts differ: slab geometry from each blob's header
        const int* hdr = (const int*)((const char*)packed + a.off.hdr);
        ell_slots = __ldg(hdr);
        ell = (const uint32_t*)((const char*)packed + *(const long long*)(hdr + 2));
    }
    const int blk0 = RPL * lblk;
    const int blk1 = min(RPL * lblk + (RPL - 1), a.RB - 1);   // clamped when RB is odd; its results are dropped
    const int gw = slice * W + warp, ostride = nslices * W;

    // per-thread state
    uint32_t w0[4 * N + 1], w1[RPL == 2 ? 4 * N + 1 : 1];
    w0[4 * N] = 0u;
    if (RPL == 2) w1[4 * N] = 0u;
    const uint4 *i0 = nullptr, *i1 = nullptr;
    const uint32_t* slab[RPL];
    int width[RPL];
    uint32_t olen[RPL];
    uint32_t oe[RPL][kSlotsPerRound];
    uint32_t cbw[RPL][TW >= E ? E / 2 : 1];
    uint32_t cbh[RPL][TW >= E ? TW / E : 1];
    auto fetch_slots = [&](int round) {
#pragma unroll
        for (int h = 0; h < RPL; ++h)
#pragma unroll
            for (int q = 0; q < kSlotsPerRound; ++q) {
                const int j = gw + (round * kSlotsPerRound + q) * ostride;
                oe[h][q] = j < width[h] ? __ldg(slab[h] + (size_t)(1 + j) * 32) : 0u;
            }
    };
    // everything the CTA reads from the blob before it can start: first super-chunk of this warp,
    // slab lengths and first round of outlier slots, the channels' codebooks
    auto issue_loads = [&]() {
        i0 = b.idx + ((size_t)(blk0 * a.SC + sc0) * N) * 32 + lane;
        i1 = b.idx + ((size_t)(blk1 * a.SC + sc0) * N) * 32 + lane;
        if (warp < nsc) {
#pragma unroll
            for (int v = 0; v < N; ++v) {
                const uint4 t0 = ld_stream(i0 + ((size_t)warp * N + v) * 32);
                w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
                if (RPL == 2) {
                    const uint4 t1 = ld_stream(i1 + ((size_t)warp * N + v) * 32);
                    w1[4 * v] = t1.x; w1[4 * v + 1] = t1.y; w1[4 * v + 2] = t1.z; w1[4 * v + 3] = t1.w;
                }
            }
        }
#pragma unroll
        for (int h = 0; h < RPL; ++h) {
            slab[h] = ell + (size_t)(h ? blk1 : blk0) * (ell_slots + 1) * 32 + lane;
            width[h] = ell_slots;   // capacity: every slot below it is readable
            olen[h] = ell_slots ? __ldg(slab[h]) : 0u;
        }
        if (ell_slots) fetch_slots(0);
        if (TW >= E) {
#pragma unroll
            for (int half = 0; half < RPL; ++half) {
                const uint16_t* cb = b.cb + (size_t)((half ? blk1 : blk0) * kRowsPerBlock + lane) * E;
#pragma unroll
                for (int i = 0; i < E / 8; ++i) {
                    const uint4 t = __ldg((const uint4*)cb + i);
                    cbw[half][4 * i] = t.x; cbw[half][4 * i + 1] = t.y; cbw[half][4 * i + 2] = t.z; cbw[half][4 * i + 3] = t.w;
                }
#pragma unroll
                for (int hh = 0; hh < TW / E; ++hh) cbh[half][hh] = __ldg(cb + warp * (TW / E) + hh);
            }
        }
    };
    // pair tables: warp w fills entries t in [w*T/W, (w+1)*T/W) of every channel half
    auto fill_tables = [&]() {
#pragma unroll
        for (int half = 0; half < RPL; ++half) {
            unsigned char* dst = tab + half * 128 + lane * 4;
            if (TW >= E) {
#pragma unroll
                for (int hh = 0; hh < TW / E; ++hh) {
                    const int hi = warp * (TW / E) + hh;
                    const uint32_t hv = cbh[half][hh];
#pragma unroll
                    for (int lo = 0; lo < E; ++lo) {
                        const uint32_t lv = (lo & 1) ? (cbw[half][lo >> 1] >> 16) : (cbw[half][lo >> 1] & 0xffffu);
                        *(uint32_t*)(dst + (size_t)(hi * E + lo) * kStride) = lv | (hv << 16);
                    }
                }
            } else {
                // small tables (N = 2): at most a few entries per warp
                const uint16_t* cb = b.cb + (size_t)((half ? blk1 : blk0) * kRowsPerBlock + lane) * E;
#pragma unroll
                for (int i = 0; i < (TW > 0 ? TW : 1); ++i) {
                    const int t = TW > 0 ? warp * TW + i : warp;
                    if (t < T) {
                        const uint32_t lv = __ldg(cb + (t & (E - 1))), hv = kSingle ? 0u : (uint32_t)__ldg(cb + (t >> N));
                        *(uint32_t*)(dst + (size_t)t * kStride) = lv | (hv << 16);
                    }
                }
            }
        }
    };

    // ---- loads and tables overlap the previous kernel's tail
    issue_loads();
    fill_tables();
    stamp(a, 1);
    // ---- x (fp16 bits, all of K: outlier columns are gathered from it) may come from the previous kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");
    stamp(a, 2);
    for (int t = threadIdx.x; t < NB * (K / 8); t += kThreads) {
        const int bb = t / (K / 8), kk = (t - bb * (K / 8)) * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (bb < a.nb) v = __ldg((const uint4*)(xsrc + (size_t)bb * a.cols + kk));
        if (TIO) v = x8_as_f16(v, a.x_bf16);
        *(uint4*)(xs + (size_t)t * 8) = v;
    }
    __syncthreads();   // tables and x visible
    stamp(a, 3);

    const uint32_t base0 = (uint32_t)lane * 4u, base1 = base0 | 128u;
    const int g = lane >> 2, t4 = lane & 3;
    // B fragment: lane (g', t') feeds column n = g' with the k slots of group t'.  Column t' of
    // batch row 0 is fed by g' == t'; column 4 + t' of batch row 1 by g' == t' + 4.
    const bool diag0 = (g == t4);
    const bool diag1 = (NB > 1) && (g == t4 + 4);
    const bool diag = diag0 || diag1;
    const unsigned char* xbase = (const unsigned char*)xs + (diag1 ? (size_t)K * 2 : 0);

    auto lookup = [&](uint32_t (&f)[4], int m) {
        if (kSingle) {
            // one entry per index; a PRMT joins two of them into the half2 of the fragment
            const uint32_t a0 = *(const uint32_t*)(tab + single_addr<N, RPL>(w0, 4 * m + 0, base0));
            const uint32_t a1 = *(const uint32_t*)(tab + single_addr<N, RPL>(w0, 4 * m + 1, base0));
            const uint32_t a2 = *(const uint32_t*)(tab + single_addr<N, RPL>(w0, 4 * m + 2, base0));
            const uint32_t a3 = *(const uint32_t*)(tab + single_addr<N, RPL>(w0, 4 * m + 3, base0));
            f[0] = __byte_perm(a0, a1, 0x5410);
            f[2] = __byte_perm(a2, a3, 0x5410);
            if (RPL == 2) {
                const uint32_t b0 = *(const uint32_t*)(tab + single_addr<N, RPL>(w1, 4 * m + 0, base1));
                const uint32_t b1 = *(const uint32_t*)(tab + single_addr<N, RPL>(w1, 4 * m + 1, base1));
                const uint32_t b2 = *(const uint32_t*)(tab + single_addr<N, RPL>(w1, 4 * m + 2, base1));
                const uint32_t b3 = *(const uint32_t*)(tab + single_addr<N, RPL>(w1, 4 * m + 3, base1));
                f[1] = __byte_perm(b0, b1, 0x5410);
                f[3] = __byte_perm(b2, b3, 0x5410);
            } else {
                f[1] = 0u; f[3] = 0u;
            }
            return;
        }
        f[0] = *(const uint32_t*)(tab + pair_addr<N, SL>(w0, 2 * m, base0));
        f[2] = *(const uint32_t*)(tab + pair_addr<N, SL>(w0, 2 * m + 1, base0));
        if (RPL == 2) {
            f[1] = *(const uint32_t*)(tab + pair_addr<N, SL>(w1, 2 * m, base1));
            f[3] = *(const uint32_t*)(tab + pair_addr<N, SL>(w1, 2 * m + 1, base1));
        } else {
            f[1] = 0u; f[3] = 0u;
        }
    };

    {
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
        float oacc[NB][RPL];
        int oround = 0, nrounds = 0;
#pragma unroll
        for (int h = 0; h < RPL; ++h) {
            // the rows' slot counts have arrived: this warp's number of outlier rounds
            int wmax = (int)olen[h];
#pragma unroll
            for (int o = 16; o; o >>= 1) wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
            width[h] = min(wmax, ell_slots);
            const int mine = width[h] > gw ? (width[h] - gw + ostride - 1) / ostride : 0;
            nrounds = max(nrounds, (mine + kSlotsPerRound - 1) / kSlotsPerRound);
#pragma unroll
            for (int bb = 0; bb < NB; ++bb) oacc[bb][h] = 0.f;
        }
        auto consume_slots = [&]() {
#pragma unroll
            for (int h = 0; h < RPL; ++h)
#pragma unroll
                for (int q = 0; q < kSlotsPerRound; ++q) {
                    const float v = h2f((uint16_t)(oe[h][q] >> 16));
                    const uint32_t col = oe[h][q] & 0xffffu;
#pragma unroll
                    for (int bb = 0; bb < NB; ++bb) oacc[bb][h] = fmaf(v, h2f(xs[(size_t)bb * K + col]), oacc[bb][h]);
                }
        };

        // ---- K loop.  Look-ups run one mma ahead of the tensor pipe; as soon as the last pair of a 16-byte
        //      vector has been looked up, its registers are reloaded with the same vector of this warp's
        //      next super-chunk (the index stream needs 4 * N * RPL registers).
#pragma unroll 1
        for (int s = warp; s < nsc; s += W) {
            if (oround < nrounds) {
                consume_slots();
                if (++oround < nrounds) fetch_slots(oround);
            }
            const bool has_next = s + W < nsc;
            const int snext = s + W;
            auto reload = [&](int gi) {   // gi: group whose look-ups were just issued (compile time)
#pragma unroll
                for (int v = 0; v < N; ++v) {
                    const int plast = (128 * (v + 1) + 2 * N - 1) / (2 * N) - 1;   // last pair touching vector v
                    if (plast / 2 == gi && has_next) {
                        const uint4 t0 = ld_stream(i0 + ((size_t)snext * N + v) * 32);
                        w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
                        if (RPL == 2) {
                            const uint4 t1 = ld_stream(i1 + ((size_t)snext * N + v) * 32);
                            w1[4 * v] = t1.x; w1[4 * v + 1] = t1.y; w1[4 * v + 2] = t1.z; w1[4 * v + 3] = t1.w;
                        }
                    }
                }
            };
            const unsigned char* xp = xbase + (size_t)(sc0 + s) * (kSuper * 2);
            uint32_t fa[4], fb[4];
            if (kDual) {
                // 16 mma of 8 consecutive k: pairs 4j, 4j+1 in the fragment's g rows, pairs 4j+2, 4j+3 in its g+8
                // rows; lanes g == t feed columns 0..3 with x[8j .. 8j+3], lanes g == t+4 columns 4..7 with
                // x[8j+4 .. 8j+7].  D[g][n] and D[g+8][4+n] are the two halves of channel lane 4g+n.
                const bool dq = diag0 || (g == t4 + 4);
                const unsigned char* xq = xp + ((g == t4 + 4) ? 8 : 0);
                auto lookup2 = [&](uint32_t (&f)[4], int j) {
                    f[0] = *(const uint32_t*)(tab + pair_addr<N, SL>(w0, 4 * j, base0));
                    f[2] = *(const uint32_t*)(tab + pair_addr<N, SL>(w0, 4 * j + 1, base0));
                    f[1] = *(const uint32_t*)(tab + pair_addr<N, SL>(w0, 4 * j + 2, base0));
                    f[3] = *(const uint32_t*)(tab + pair_addr<N, SL>(w0, 4 * j + 3, base0));
                };
                auto reload2 = [&](int gi) {   // gi: mma whose look-ups were just issued (compile time)
#pragma unroll
                    for (int v = 0; v < N; ++v) {
                        const int plast = (128 * (v + 1) + 2 * N - 1) / (2 * N) - 1;   // last pair touching vector v
                        if (plast / 4 == gi && has_next) {
                            const uint4 t0 = ld_stream(i0 + ((size_t)snext * N + v) * 32);
                            w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
                        }
                    }
                };
                uint2 xa = make_uint2(0u, 0u), xb = make_uint2(0u, 0u);
                if (dq) xa = *(const uint2*)xq;
                lookup2(fa, 0);
#pragma unroll
                for (int j = 0; j < kSuper / 8; j += 2) {
                    if (dq) xb = *(const uint2*)(xq + (j + 1) * 16);
                    lookup2(fb, j + 1);
                    reload2(j + 1);
                    mma16816(c0, fa[0], fa[1], fa[2], fa[3], xa.x, xa.y);
                    if (j + 2 < kSuper / 8) {
                        if (dq) xa = *(const uint2*)(xq + (j + 2) * 16);
                        lookup2(fa, j + 2);
                        reload2(j + 2);
                    }
                    mma16816(c1, fb[0], fb[1], fb[2], fb[3], xb.x, xb.y);
                }
                continue;
            }
            uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = make_uint4(0u, 0u, 0u, 0u);
            if (diag) xa = *(const uint4*)xp;
            lookup(fa, 0);
#pragma unroll
            for (int m = 0; m < kSuper / 4; m += 4) {   // one mma per 4 consecutive k
                if (diag) xb = *(const uint4*)(xp + (m + 2) * 8);
                lookup(fb, m + 1);
                reload(m + 1);
                mma16816(c0, fa[0], fa[1], fa[2], fa[3], xa.x, xa.y);
                lookup(fa, m + 2);
                reload(m + 2);
                mma16816(c1, fb[0], fb[1], fb[2], fb[3], xa.z, xa.w);
                if (m + 4 < kSuper / 4) { if (diag) xa = *(const uint4*)(xp + (m + 4) * 8); }
                lookup(fb, m + 3);
                reload(m + 3);
                mma16816(c0, fa[0], fa[1], fa[2], fa[3], xb.x, xb.y);
                if (m + 4 < kSuper / 4) {
                    lookup(fa, m + 4);
                    reload(m + 4);
                }
                mma16816(c1, fb[0], fb[1], fb[2], fb[3], xb.z, xb.w);
            }
        }
        while (oround < nrounds) {   // more outlier rounds than super-chunks
            consume_slots();
            if (++oround < nrounds) fetch_slots(oround);
        }
        // Rows that fill their slab may continue in the CSR arrays (pathological skew only): warp 0 of
        // the block's first slice finishes them, one lane per row.
        if (warp == 0 && slice == 0 && ell_slots) {
#pragma unroll
            for (int h = 0; h < RPL; ++h) {
                if ((int)olen[h] >= ell_slots) {
                    const int row = (h ? blk1 : blk0) * kRowsPerBlock + lane;
                    const int p1 = __ldg(b.rowptr + row + 1);
                    for (int p = __ldg(b.rowptr + row) + ell_slots; p < p1; ++p) {
                        const uint32_t e = __ldg(b.oent + p);
#pragma unroll
                        for (int bb = 0; bb < NB; ++bb)
                            oacc[bb][h] = fmaf(h2f((uint16_t)(e >> 16)), h2f(xs[(size_t)bb * K + (e & 0xffffu)]), oacc[bb][h]);
                    }
                }
            }
        }
        stamp(a, 4);
        const int cur_blk = blk, cur_slice = slice, cur_nslices = nslices;
        // ---- scatter the fragment to channel order: lane (g, t) holds D[g][2t], D[g][2t+1], D[g+8][..];
        //      column n < 4: batch 0 of lane 4g + n; column n >= 4: batch 1 of lane 4g + n - 4
        {
            const float v0 = c0[0] + c1[0], v1 = c0[1] + c1[1], v2 = c0[2] + c1[2], v3 = c0[3] + c1[3];
            const int bb = t4 >> 1;                  // batch row held by this lane's columns
            const int l0 = 4 * g + 2 * (t4 & 1);     // channel lane of column 2t
            if (bb < NB) {
                float* r = red + ((size_t)warp * NB + bb) * ROWS;
                r[l0] = v0; r[l0 + 1] = v1;
                if (RPL == 2) { r[32 + l0] = v2; r[32 + l0 + 1] = v3; }
            }
            __syncwarp();
            if (kDual) {   // the second halves sit in rows g+8, columns 4..7: lanes t >= 2 add them
                if (t4 >= 2) {
                    float* r = red + (size_t)warp * ROWS;
                    r[l0] += v2; r[l0 + 1] += v3;
                }
                __syncwarp();
            }
#pragma unroll
            for (int bb2 = 0; bb2 < NB; ++bb2)
#pragma unroll
                for (int h = 0; h < RPL; ++h) red[((size_t)warp * NB + bb2) * ROWS + 32 * h + lane] += oacc[bb2][h];
        }
        __syncthreads();   // partial sums of all warps are in red

        // ---- fixed-order reduction over the warps, then store or combine the block's slices
        const int t = threadIdx.x;
        const int bb = t / ROWS, r = t % ROWS;
        const bool active = t < NB * ROWS;
        const bool dup = (r >= 32) && (RPL * lblk + 1 >= a.RB);
        const int row = lblk * ROWS + r;               // channel inside its blob (y index)
        const int wrow = cur_blk * ROWS + r;           // channel inside the launch (workspace index)
        float total = 0.f;
        if (active) {
#pragma unroll
            for (int w = 0; w < W; ++w) total += red[((size_t)w * NB + bb) * ROWS + r];
        }
        bool writer = true;
        if (cur_nslices > 1 && a.cluster) {
            // the slices of a block are the CTAs of one cluster: rank 0 adds the partial sums of its peers
            // straight out of their shared memory, in rank order
            namespace cg = cooperative_groups;
            cg::cluster_group cl = cg::this_cluster();
            if (active) red[t] = total;          // slot t of red is read by thread t only
            cl.sync();
            if (cur_slice == 0 && active) {
                for (int k2 = 1; k2 < cur_nslices; ++k2) total += *cl.map_shared_rank(red + t, k2);
            }
            cl.sync();                            // peers keep their shared memory alive until rank 0 has read it
            writer = cur_slice == 0;
        } else if (cur_nslices > 1) {
            __shared__ int s_last;
            if (active) a.partial[((size_t)cur_slice * NB + bb) * a.rows_ws + wrow] = total;
            __threadfence();
            __syncthreads();
            if (t == 0) s_last = (atomicAdd(a.tickets + cur_blk, 1) == cur_nslices - 1);
            __syncthreads();
            writer = s_last != 0;
            if (writer) {
                __threadfence();
                if (active) {
                    total = 0.f;
                    for (int k2 = 0; k2 < cur_nslices; ++k2)
                        total += __ldcg(a.partial + ((size_t)k2 * NB + bb) * a.rows_ws + wrow);
                }
                if (t == 0) a.tickets[cur_blk] = 0;
            }
        }
        if (writer && active && !dup && bb < a.nb && row < a.rows) {
            store_y<TIO>(ydst, (size_t)bb * a.rows + row, total, a.y_is_fp16);
        }
        stamp(a, 5);
    }
}

// ------------------------------------------------------------------------------------ host side

#ifdef XFP_TRACE
// timing build only: where the next `calls` launches put their stamps (1024 CTAs x 8 stamps each)
static unsigned long long* g_pair_trace = nullptr;
static size_t g_pair_trace_calls = 0, g_pair_trace_idx = 0;
extern "C" void xfp_trace_pair(void* p, size_t calls) {
    g_pair_trace = (unsigned long long*)p;
    g_pair_trace_calls = calls;
    g_pair_trace_idx = 0;
}
#endif

struct PairConfig { int rpl, warps, slots; };

static PairConfig pair_config(const Layout& l, int n = 1) {
    // N <= 4: two rows per lane, 8 warps, two CTAs per SM.  N = 5: the pair table of a row is 4 KB, so
    // one row per lane (128 KB of tables), 16 warps, one CTA per SM.  Matrices with no more row-blocks than
    // the device has SMs also take one row per lane: twice the CTAs and no cut along K.
    const int sms = sched_sms();
    if (l.bits == 5) return PairConfig{1, 16, sms};
    if ((long long)l.RB * n <= sms && l.bits >= 3) return PairConfig{1, 16, sms};
    return PairConfig{2, 8, 2 * sms};
}

struct PairSchedule {
    int blocks, grid, cluster, ntiers;
    int tier_cta[5], tier_blk[4], tier_kst[4], tier_spp[4];
};

static int pow2_floor(int v) {
    int p = 1;
    while (p * 2 <= v) p *= 2;
    return p;
}

static PairSchedule pair_schedule(const Layout& l, int n = 1) {
    const PairConfig cfg = pair_config(l, n);
    PairSchedule sc{};
    sc.blocks = ((l.RB + cfg.rpl - 1) / cfg.rpl) * n;   // the blocks of all blobs of the launch
    const int S = cfg.slots;
    const int kmax = l.SC / 4 > 1 ? pow2_floor(l.SC / 4) : 1;   // keep K slices of at least 512 weights
    int nb[4] = {0, 0, 0, 0}, kk[4] = {1, 1, 1, 1};
    int nt = 0;
    if (sc.blocks * 2 <= S) {
        // fewer blocks than half the CTA slots: cut every block into 2, 4 or 8 K slices that form a cluster
        int kst = 1;
        while (kst < 8 && sc.blocks * kst * 2 <= S && kst * 2 <= kmax) kst *= 2;
        nb[0] = sc.blocks; kk[0] = kst; nt = 1;
        sc.cluster = kst > 1;
    } else {
        // whole rounds unsplit, then tiers of finer slices for the blocks of the last, partial round
        const int full = (sc.blocks / S) * S;
        int remaining = sc.blocks - full;
        if (full > 0) { nb[nt] = full; kk[nt] = 1; ++nt; }
        if (full == 0) { nb[nt] = remaining; kk[nt] = 1; ++nt; remaining = 0; }   // a single partial round
        int k = 2;
        while (remaining > 0 && nt < 4) {
            if (k > kmax) { nb[nt] = remaining; kk[nt] = kmax; ++nt; remaining = 0; break; }
            const int cap = S / k;   // blocks whose k slices fill one round
            if (remaining <= cap || nt == 3) {
                int kl = pow2_floor(S / remaining > 1 ? S / remaining : 1);
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
    sc.ntiers = nt;
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
    if (sc.cluster && (sc.tier_kst[0] == 1 || (sc.tier_kst[0] & (sc.tier_kst[0] - 1)))) sc.cluster = 0;
    return sc;
}

static size_t pair_smem_bytes(const Layout& l, int nb, int n = 1) {
    const PairConfig cfg = pair_config(l, n);
    const int rows = 32 * cfg.rpl;
    const size_t T = l.bits > 5 ? (size_t)l.E : (size_t)l.E * l.E;   // N = 6: one entry per index
    const int sl = (cfg.rpl == 2 || l.bits == 4) ? 2 : 1;              // entry stride in units of 128 bytes
    return T * 128 * sl + (size_t)nb * l.cols * 2 + (size_t)cfg.warps * nb * rows * 4;
}

bool pair_supported(const Layout& l, int batch, int n_problems) {
    if (l.mode != 0 || l.bits < 2 || l.bits > 6 || batch > 2 || n_problems < 1) return false;
    if (n_problems > 1 && batch != 1) return false;
    return pair_smem_bytes(l, batch, n_problems) <= (pair_config(l, n_problems).warps == 8 ? 110u : 220u) * 1024u;
}

size_t pair_workspace_bytes(const Layout& l) {
    const int ksmax = 64 < l.SC ? 64 : l.SC;
    return align256((size_t)l.RB * 4) + align256((size_t)ksmax * 2 * (size_t)(l.RB + 1) * 32 * 4);
}

template <int N, int NB, int RPL, int W, bool TIO>
static cudaError_t launch_pair_io(const PairArgs& a, int grid, size_t smem, cudaStream_t s) {
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemv_pair_kernel<N, NB, RPL, W, TIO>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return e;
        attr_done.set(dev);
    }
    const int cluster = a.cluster ? a.tier_kst[0] : 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(W * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cluster > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, gemv_pair_kernel<N, NB, RPL, W, TIO>, a);
}

// bf16 activations or bf16 outputs take the typed-IO instantiation; everything else the plain one
template <int N, int NB, int RPL, int W>
static cudaError_t launch_pair(const PairArgs& a, int grid, size_t smem, cudaStream_t s) {
    if (a.x_bf16 || a.y_is_fp16 == 2 || a.packed_list) return launch_pair_io<N, NB, RPL, W, true>(a, grid, smem, s);
    return launch_pair_io<N, NB, RPL, W, false>(a, grid, smem, s);
}

static cudaError_t launch_gemv_pair_n(const Layout& l, const GemvCall& c, int prob0, cudaStream_t s);

cudaError_t launch_gemv_pair(const Layout& l, const GemvCall& c, cudaStream_t s) {
    // N >= 5 (large tables: one CTA per SM, or two channels per lane at N = 6) gains nothing from a common schedule
    // once the blocks exceed one round: one launch per blob, read through the same lists.
    if (c.n > 1) {
        const PairConfig one_cfg = pair_config(l, 1);
        if (l.bits >= 5 && (long long)((l.RB + one_cfg.rpl - 1) / one_cfg.rpl) * c.n > one_cfg.slots) {
            GemvCall one = c;
            one.n = 1;
            for (int j = 0; j < c.n; ++j) {
                const cudaError_t e = launch_gemv_pair_n(l, one, j, s);
                if (e != cudaSuccess) return e;
            }
            return cudaSuccess;
        }
    }
    return launch_gemv_pair_n(l, c, 0, s);
}

static cudaError_t launch_gemv_pair_n(const Layout& l, const GemvCall& c, int prob0, cudaStream_t s) {
    const PairConfig cfg = pair_config(l, c.n);
    const PairSchedule sch = pair_schedule(l, c.n);
    PairArgs a{};
    a.off = offsets_of(l);
    a.packed = c.packed; a.x = c.x; a.y = c.y;
    a.packed_list = c.packed_list; a.x_list = c.x_list; a.y_list = c.y_list;
    a.blocks_per = sch.blocks / c.n;
    a.prob0 = prob0;
    a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.ell_slots = l.ell_slots;
    a.blocks = sch.blocks;
    a.rows_ws = sch.blocks * 32 * cfg.rpl;
    for (int i = 0; i < 5; ++i) a.tier_cta[i] = sch.tier_cta[i];
    for (int i = 0; i < 4; ++i) { a.tier_blk[i] = sch.tier_blk[i]; a.tier_kst[i] = sch.tier_kst[i]; a.tier_spp[i] = sch.tier_spp[i]; }
    a.cluster = sch.cluster;
    a.nb = c.batch; a.y_is_fp16 = c.y_is_fp16; a.x_bf16 = c.x_bf16;
#ifdef XFP_TRACE
    a.trace = nullptr;
    if (g_pair_trace && g_pair_trace_idx < g_pair_trace_calls) a.trace = g_pair_trace + (g_pair_trace_idx++) * 1024 * 8;
#endif
    a.tickets = (int*)c.workspace;
    a.partial = (float*)((char*)c.workspace + align256((size_t)l.RB * 4 * c.n));
    const size_t smem = pair_smem_bytes(l, c.batch, c.n);
    if (cfg.rpl == 1) {
        switch (l.bits * 10 + c.batch) {
            case 31: return launch_pair<3, 1, 1, 16>(a, sch.grid, smem, s);
            case 32: return launch_pair<3, 2, 1, 16>(a, sch.grid, smem, s);
            case 41: return launch_pair<4, 1, 1, 16>(a, sch.grid, smem, s);
            case 42: return launch_pair<4, 2, 1, 16>(a, sch.grid, smem, s);
            case 51: return launch_pair<5, 1, 1, 16>(a, sch.grid, smem, s);
            case 52: return launch_pair<5, 2, 1, 16>(a, sch.grid, smem, s);
            case 61: return launch_pair<6, 1, 1, 16>(a, sch.grid, smem, s);
            case 62: return launch_pair<6, 2, 1, 16>(a, sch.grid, smem, s);
        }
        return cudaErrorInvalidValue;
    }
    switch (l.bits * 10 + c.batch) {
        case 21: return launch_pair<2, 1, 2, 8>(a, sch.grid, smem, s);
        case 22: return launch_pair<2, 2, 2, 8>(a, sch.grid, smem, s);
        case 31: return launch_pair<3, 1, 2, 8>(a, sch.grid, smem, s);
        case 32: return launch_pair<3, 2, 2, 8>(a, sch.grid, smem, s);
        case 41: return launch_pair<4, 1, 2, 8>(a, sch.grid, smem, s);
        case 42: return launch_pair<4, 2, 2, 8>(a, sch.grid, smem, s);
        case 61: return launch_pair<6, 1, 2, 8>(a, sch.grid, smem, s);
        case 62: return launch_pair<6, 2, 2, 8>(a, sch.grid, smem, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace xfp
