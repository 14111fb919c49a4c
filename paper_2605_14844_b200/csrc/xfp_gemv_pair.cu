// Fast fused decode GEMV for V2 blobs at batch <= 2:  y = (D + S) x.
//
// Mapping.  A CTA owns a block of 32*RPL output channels (RPL = rows per lane: 2 for N <= 4,
// 1 for N = 5) and all of K, or a slice of K for the blocks of the last scheduling round.  Each
// lane of a dense warp owns RPL channels (lane, lane+32 of the block) and the warps of the CTA
// share K in super-chunks of 128 weights.  The channels' codebooks are expanded once per CTA into
// PAIR tables in shared memory: entry t = (cb[t & (E-1)], cb[t >> N]) as a half2, so one 32-bit
// shared-memory load decodes two weights ("codebook gather from shared memory", step 2 of the
// fused kernel).  The tables are laid out so that lane l only ever touches bank l: byte address
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
// transposed slab (slot j of channel l at slab + j*32 + l), so a warp reads one slot of all 32
// channels with one coalesced load and every lane adds val * x[col] (x gathered from the staged
// copy in shared memory) to an accumulator of its own channel.  Slots are dealt round-robin to the
// dense warps and consumed between super-chunks, their loads issued one iteration ahead.  Rows
// longer than the slab (pathological skew) finish from the CSR arrays.  The order of additions is
// fixed by the schedule, so results are reproducible.
//
// Schedule.  Blocks that fill whole rounds of CTA slots run over all of K; the blocks of the last,
// partial round are cut along K so that they occupy the idle slots, and their partial sums are
// combined by the last CTA of a block in fixed order (no waiting, no atomics on data).
//
// Launch overlap.  Weights do not depend on earlier kernels, so every CTA first issues its index,
// codebook and row-pointer loads and fills its pair tables, and only then executes
// griddepcontrol.wait (programmatic dependent launch) before it touches x, y or the workspace.
// Back-to-back calls on one stream therefore overlap the next call's weight streaming with the
// current call's tail.
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
    float* partial;  // [KS][NB][rows_ws]
    int* tickets;    // [blocks]
    int rows, cols, RB, SC, rows_ws, ell_slots;
    int nb, y_is_fp16;
    // schedule: work items [0, n_full) are whole blocks; the remaining blocks are cut into kst
    // K-slices of sc_per_split super-chunks each
    int n_full, kst, sc_per_split;
    int pf_dist;  // L2 prefetch distance in warp iterations (0 = off)
    int cluster;  // 1: the kst CTAs of a block form a thread-block cluster and reduce through DSMEM
    int dbg;      // timing probes only: 1 = return after the dependency wait, 2 = skip the main loop, 3 = no PDL
    unsigned long long* trace;  // timing probes only: per CTA 8 globaltimer stamps
};

__device__ __forceinline__ void stamp(const PairArgs& a, int slot) {
    if (a.trace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        a.trace[(size_t)blockIdx.x * 8 + slot] = t;
    }
}

template <int N, int NB, int RPL, int W>
__global__ void __launch_bounds__(W * 32, W == 8 ? 2 : 1) gemv_pair_kernel(const PairArgs a) {
    constexpr int E = 1 << N;
    constexpr int T = E * E;                   // pair-table entries per channel
    constexpr int ROWS = 32 * RPL;             // channels per CTA
    constexpr int kStride = 128 * RPL;         // bytes between consecutive entries
    constexpr int kTabBytes = T * kStride;
    constexpr int kDense = W * 32;
    extern __shared__ __align__(16) unsigned char smem[];
    // [tables | x fp16 [NB][K] | red[W][NB][ROWS]]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    stamp(a, 0);
    if (a.dbg == 1) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    int blk, ks, KS, spp;
    if ((int)blockIdx.x < a.n_full) {
        blk = blockIdx.x; ks = 0; KS = 1; spp = a.SC;
    } else {
        const int t = blockIdx.x - a.n_full;
        blk = a.n_full + t / a.kst; ks = t % a.kst; KS = a.kst; spp = a.sc_per_split;
    }
    const Blob b = blob_at(a.packed, a.off);
    const int sc0 = ks * spp;
    const int nsc = max(0, min(a.SC, sc0 + spp) - sc0);
    const int K = a.SC * kSuper;

    unsigned char* tab = smem;
    uint16_t* xs = (uint16_t*)(smem + kTabBytes);               // [NB][K]
    float* red = (float*)(xs + (size_t)NB * K);                 // [W][NB][ROWS]

    // the 32-row blocks of this CTA (the second is clamped when RB is odd; its results are dropped)
    const int blk0 = RPL * blk;
    const int blk1 = min(RPL * blk + (RPL - 1), a.RB - 1);

    {
        // ------------------------------------------------ dense warps
        // (0) start streaming this warp's first super-chunk before anything else
        uint32_t w0[4 * N + 1], w1[RPL == 2 ? 4 * N + 1 : 1];
        w0[4 * N] = 0u;
        if (RPL == 2) w1[4 * N] = 0u;
        const uint4* i0 = b.idx + ((size_t)(blk0 * a.SC + sc0) * N) * 32 + lane;
        const uint4* i1 = b.idx + ((size_t)(blk1 * a.SC + sc0) * N) * 32 + lane;
        auto prefetch_sc = [&](int sidx) {   // the RPL * N * 512 bytes of a super-chunk are RPL * 4N lines
            if (lane < RPL * 4 * N) {
                const int half = lane / (4 * N), line = lane % (4 * N);
                const char* p = (const char*)((half ? i1 : i0) - lane + (size_t)sidx * N * 32) + line * 128;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
            }
        };
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
        // one row per lane leaves registers for a second super-chunk in flight (short K loops are
        // otherwise a chain of DRAM round trips)
        constexpr bool kTwoDeep = (RPL == 1);
        uint32_t z0[kTwoDeep ? 4 * N + 1 : 1];
        if (kTwoDeep) {
            z0[4 * N] = 0u;
            if (warp + W < nsc) {
#pragma unroll
                for (int v = 0; v < N; ++v) {
                    const uint4 t0 = ld_stream(i0 + ((size_t)(warp + W) * N + v) * 32);
                    z0[4 * v] = t0.x; z0[4 * v + 1] = t0.y; z0[4 * v + 2] = t0.z; z0[4 * v + 3] = t0.w;
                }
            }
        }
        if (a.pf_dist > 0)
            for (int r = 1; r <= a.pf_dist; ++r)
                if (warp + r * W < nsc) prefetch_sc(warp + r * W);
        // outlier slabs of this CTA's row-blocks: slots gw, gw + stride, ... belong to this warp.  The first
        // round is fetched before the rows' lengths are known (any slot below the capacity is readable).
        const int gw = ks * W + warp, ostride = KS * W;
        const uint32_t* slab[RPL];
        int width[RPL];
        uint32_t olen[RPL];
        uint32_t oe[RPL][kSlotsPerRound];
        float oacc[NB][RPL];
        int oround = 0, nrounds = 0;
#pragma unroll
        for (int h = 0; h < RPL; ++h) {
            slab[h] = b.ell + (size_t)(h ? blk1 : blk0) * (a.ell_slots + 1) * 32 + lane;
            width[h] = a.ell_slots;
            olen[h] = a.ell_slots ? __ldg(slab[h]) : 0u;
#pragma unroll
            for (int bb = 0; bb < NB; ++bb) oacc[bb][h] = 0.f;
        }
        auto fetch_slots = [&](int round) {
#pragma unroll
            for (int h = 0; h < RPL; ++h)
#pragma unroll
                for (int q = 0; q < kSlotsPerRound; ++q) {
                    const int j = gw + (round * kSlotsPerRound + q) * ostride;
                    oe[h][q] = j < width[h] ? __ldg(slab[h] + (size_t)(1 + j) * 32) : 0u;
                }
        };
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
        if (a.ell_slots) fetch_slots(0);
        // codebooks of this lane's channels (for the table fill below)
        constexpr int TW = T / W;  // table entries per warp
        uint32_t cbw[RPL][TW >= E ? E / 2 : 1];
        uint32_t cbh[RPL][TW >= E ? TW / E : 1];
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
        // (1) pair tables: warp w fills entries t in [w*T/W, (w+1)*T/W) of every channel half
        {
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
                    // small tables (N = 2): TW < E entries per warp
                    const uint16_t* cb = b.cb + (size_t)((half ? blk1 : blk0) * kRowsPerBlock + lane) * E;
#pragma unroll
                    for (int i = 0; i < TW; ++i) {
                        const int t = warp * TW + i;
                        const uint32_t lv = __ldg(cb + (t & (E - 1))), hv = __ldg(cb + (t >> N));
                        *(uint32_t*)(dst + (size_t)t * kStride) = lv | (hv << 16);
                    }
                }
            }
        }
        // x may come from the previous kernel: everything above overlaps that kernel's tail
        stamp(a, 1);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        stamp(a, 2);
        constexpr int XV = 4;                       // uint4 of x per thread per pass
        const int nvec = NB * (K / 8);
        uint4 xv[XV];
#pragma unroll
        for (int i = 0; i < XV; ++i) {
            const int t = threadIdx.x + i * kDense;
            xv[i] = make_uint4(0u, 0u, 0u, 0u);
            if (t < nvec) {
                const int bb = t / (K / 8), kk = (t - bb * (K / 8)) * 8;
                if (bb < a.nb) xv[i] = __ldg((const uint4*)(a.x + (size_t)bb * a.cols + kk));
            }
        }

        stamp(a, 3);
        // (2) x (fp16 bits, all of K: outlier columns are gathered from it) -> shared memory
#pragma unroll
        for (int i = 0; i < XV; ++i) {
            const int t = threadIdx.x + i * kDense;
            if (t < nvec) *(uint4*)(xs + (size_t)t * 8) = xv[i];
        }
        for (int t = threadIdx.x + XV * kDense; t < nvec; t += kDense) {   // K beyond XV passes
            const int bb = t / (K / 8), kk = (t - bb * (K / 8)) * 8;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (bb < a.nb) v = __ldg((const uint4*)(a.x + (size_t)bb * a.cols + kk));
            *(uint4*)(xs + (size_t)t * 8) = v;
        }
        // the rows' slot counts are here by now: this warp's number of outlier rounds
#pragma unroll
        for (int h = 0; h < RPL; ++h) {
            int wmax = (int)olen[h];
#pragma unroll
            for (int o = 16; o; o >>= 1) wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
            width[h] = min(wmax, a.ell_slots);
            const int mine = width[h] > gw ? (width[h] - gw + ostride - 1) / ostride : 0;
            nrounds = max(nrounds, (mine + kSlotsPerRound - 1) / kSlotsPerRound);
        }
        __syncthreads();  // tables and x visible
        stamp(a, 4);

        // (3) main loop
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t base0 = (uint32_t)lane * 4u, base1 = base0 | 128u;
        const int g = lane >> 2, t4 = lane & 3;
        // B fragment: lane (g', t') feeds column n = g' with the k slots of group t'.  Column t' of
        // batch row 0 is fed by g' == t'; column 4 + t' of batch row 1 by g' == t' + 4.
        const bool diag0 = (g == t4);
        const bool diag1 = (NB > 1) && (g == t4 + 4);
        const bool diag = diag0 || diag1;
        const unsigned char* xrow =
            (const unsigned char*)xs + (diag1 ? (size_t)K * 2 : 0) + (size_t)sc0 * (kSuper * 2);

        auto lookup = [&](uint32_t (&f)[4], const uint32_t* u0, const uint32_t* u1, int m) {
            f[0] = *(const uint32_t*)(tab + pair_addr<N, RPL>(u0, 2 * m, base0));
            f[2] = *(const uint32_t*)(tab + pair_addr<N, RPL>(u0, 2 * m + 1, base0));
            if (RPL == 2) {
                f[1] = *(const uint32_t*)(tab + pair_addr<N, RPL>(u1, 2 * m, base1));
                f[3] = *(const uint32_t*)(tab + pair_addr<N, RPL>(u1, 2 * m + 1, base1));
            } else {
                f[1] = 0u; f[3] = 0u;
            }
        };
        // One super-chunk.  Look-ups run one mma ahead of the tensor pipe; as soon as the last pair of
        // a 16-byte vector has been looked up, the vector's registers are reloaded with the same
        // vector of this warp's next super-chunk (the index stream needs 4 * N * RPL registers).
        auto compute_sc = [&](uint32_t* u0, uint32_t* u1, int sidx, bool has_next, int snext) {
            const unsigned char* xp = xrow + (size_t)sidx * (kSuper * 2);
            uint32_t fa[4], fb[4];
            uint4 xa = make_uint4(0u, 0u, 0u, 0u), xb = make_uint4(0u, 0u, 0u, 0u);
            if (diag) xa = *(const uint4*)xp;
            lookup(fa, u0, u1, 0);
            auto reload = [&](int gi) {   // gi: group whose look-ups were just issued (compile time)
#pragma unroll
                for (int v = 0; v < N; ++v) {
                    const int plast = (128 * (v + 1) + 2 * N - 1) / (2 * N) - 1;   // last pair touching vector v
                    if (plast / 2 == gi && has_next) {
                        const uint4 t0 = ld_stream(i0 + ((size_t)snext * N + v) * 32);
                        u0[4 * v] = t0.x; u0[4 * v + 1] = t0.y; u0[4 * v + 2] = t0.z; u0[4 * v + 3] = t0.w;
                        if (RPL == 2) {
                            const uint4 t1 = ld_stream(i1 + ((size_t)snext * N + v) * 32);
                            u1[4 * v] = t1.x; u1[4 * v + 1] = t1.y; u1[4 * v + 2] = t1.z; u1[4 * v + 3] = t1.w;
                        }
                    }
                }
            };
#pragma unroll
            for (int m = 0; m < kSuper / 4; m += 4) {   // one mma per 4 consecutive k
                if (diag) xb = *(const uint4*)(xp + (m + 2) * 8);
                lookup(fb, u0, u1, m + 1);
                reload(m + 1);
                mma16816(c0, fa[0], fa[1], fa[2], fa[3], xa.x, xa.y);
                lookup(fa, u0, u1, m + 2);
                reload(m + 2);
                mma16816(c1, fb[0], fb[1], fb[2], fb[3], xa.z, xa.w);
                if (m + 4 < kSuper / 4) { if (diag) xa = *(const uint4*)(xp + (m + 4) * 8); }
                lookup(fb, u0, u1, m + 3);
                reload(m + 3);
                mma16816(c0, fa[0], fa[1], fa[2], fa[3], xb.x, xb.y);
                if (m + 4 < kSuper / 4) {
                    lookup(fa, u0, u1, m + 4);
                    reload(m + 4);
                }
                mma16816(c1, fb[0], fb[1], fb[2], fb[3], xb.z, xb.w);
            }
        };
        if (kTwoDeep) {
#pragma unroll 1
            for (int s = warp; s < (a.dbg == 2 ? 0 : nsc); s += 2 * W) {
                if (oround < nrounds) {
                    consume_slots();
                    if (++oround < nrounds) fetch_slots(oround);
                }
                compute_sc(w0, w1, s, s + 2 * W < nsc, s + 2 * W);
                if (s + W < nsc) {
                    if (oround < nrounds) {
                        consume_slots();
                        if (++oround < nrounds) fetch_slots(oround);
                    }
                    compute_sc(z0, w1, s + W, s + 3 * W < nsc, s + 3 * W);
                }
            }
        } else {
#pragma unroll 1
            for (int s = warp; s < (a.dbg == 2 ? 0 : nsc); s += W) {
                if (a.pf_dist > 0 && s + (a.pf_dist + 1) * W < nsc) prefetch_sc(s + (a.pf_dist + 1) * W);
                if (oround < nrounds) {
                    consume_slots();
                    if (++oround < nrounds) fetch_slots(oround);
                }
                compute_sc(w0, w1, s, s + W < nsc, s + W);
            }
        }
        while (oround < nrounds) {   // more outlier rounds than super-chunks
            consume_slots();
            if (++oround < nrounds) fetch_slots(oround);
        }
        // Rows that fill their slab may continue in the CSR arrays (pathological skew only): warp 0 of
        // the first K slice finishes them, one lane per row.
        if (warp == 0 && ks == 0 && a.ell_slots) {
#pragma unroll
            for (int h = 0; h < RPL; ++h) {
                if ((int)olen[h] >= a.ell_slots) {
                    const int row = (h ? blk1 : blk0) * kRowsPerBlock + lane;
                    const int p1 = __ldg(b.rowptr + row + 1);
                    for (int p = __ldg(b.rowptr + row) + a.ell_slots; p < p1; ++p) {
                        const uint32_t e = __ldg(b.oent + p);
#pragma unroll
                        for (int bb = 0; bb < NB; ++bb)
                            oacc[bb][h] = fmaf(h2f((uint16_t)(e >> 16)), h2f(xs[(size_t)bb * K + (e & 0xffffu)]), oacc[bb][h]);
                    }
                }
            }
        }
        stamp(a, 5);
        // (4) scatter the fragment to channel order: lane (g, t) holds D[g][2t], D[g][2t+1], D[g+8][..]
        //     column n < 4: batch 0 of lane 4g + n; column n >= 4: batch 1 of lane 4g + n - 4
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
#pragma unroll
            for (int bb2 = 0; bb2 < NB; ++bb2)
#pragma unroll
                for (int h = 0; h < RPL; ++h) red[((size_t)warp * NB + bb2) * ROWS + 32 * h + lane] += oacc[bb2][h];
        }
        __syncthreads();
    }

    // ---------------------------------------------------- fixed-order reduction, store / split-K finish
    const int t = threadIdx.x;
    const int bb = t / ROWS, r = t % ROWS;
    const bool active = t < NB * ROWS;
    // channel r of the block: rows of blk0 for r < 32, of blk1 for r >= 32
    const bool dup = (r >= 32) && (RPL * blk + 1 >= a.RB);
    const int row = blk * ROWS + r;
    float total = 0.f;
    if (active) {
#pragma unroll
        for (int w = 0; w < W; ++w) total += red[((size_t)w * NB + bb) * ROWS + r];
    }
    if (KS > 1 && a.cluster) {
        // K slices of one block are the CTAs of one cluster: rank 0 adds the partial sums of its peers
        // straight out of their shared memory, in rank order.
        namespace cg = cooperative_groups;
        cg::cluster_group cl = cg::this_cluster();
        if (active) red[t] = total;          // slot t of red is read by thread t only
        cl.sync();
        if (ks == 0 && active) {
            for (int k2 = 1; k2 < KS; ++k2) total += *cl.map_shared_rank(red + t, k2);
        }
        cl.sync();                            // peers keep their shared memory alive until rank 0 has read it
        if (ks != 0) return;
    } else if (KS > 1) {
        __shared__ int s_last;
        if (active) a.partial[((size_t)ks * NB + bb) * a.rows_ws + row] = total;
        __threadfence();
        __syncthreads();
        if (t == 0) s_last = (atomicAdd(a.tickets + blk, 1) == KS - 1);
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        if (active) {
            total = 0.f;
            for (int k2 = 0; k2 < KS; ++k2) total += __ldcg(a.partial + ((size_t)k2 * NB + bb) * a.rows_ws + row);
        }
        if (t == 0) a.tickets[blk] = 0;
    }
    if (active && !dup && bb < a.nb && row < a.rows) {
        if (a.y_is_fp16)
            ((uint16_t*)a.y)[(size_t)bb * a.rows + row] = f2h(total);
        else
            ((float*)a.y)[(size_t)bb * a.rows + row] = total;
    }
    stamp(a, 6);
}

// ------------------------------------------------------------------------------------ host side

static int g_pair_ks_override = 0;  // 0 = policy below
static unsigned long long* g_pair_trace = nullptr;
static size_t g_pair_trace_calls = 0, g_pair_trace_idx = 0;
void pair_set_trace(void* p, size_t calls) { g_pair_trace = (unsigned long long*)p; g_pair_trace_calls = calls; g_pair_trace_idx = 0; }
static int g_pair_dbg = 0;
void pair_set_debug(int m) { g_pair_dbg = m; }
static int g_pair_pf_dist = 0;  // L2 prefetch measured slower than none on B200

void pair_set_ksplit_override(int ks) { g_pair_ks_override = ks; }
void pair_set_prefetch(int d) { g_pair_pf_dist = d; }

struct PairConfig { int rpl, warps, slots; };

static int g_pair_small = 1;   // probe switch: one row per lane for matrices with few row blocks
void pair_set_small(int v) { g_pair_small = v; }

static PairConfig pair_config(const Layout& l) {
    // N <= 4: two rows per lane, 8 dense warps, two CTAs per SM.  N = 5: the pair table of a row is
    // 4 KB, so one row per lane (128 KB of tables), 16 dense warps, one CTA per SM.  Matrices with
    // fewer 64-row blocks than SMs also take one row per lane: twice the CTAs, no split along K.
    if (l.bits == 5) return PairConfig{1, 16, 148};
    if (g_pair_small == 1 && l.RB <= 148 && l.bits >= 3) return PairConfig{1, 16, 148};
    if (g_pair_small == 2 && l.RB <= 148 && l.bits >= 3 && l.bits <= 4) return PairConfig{1, 8, 148};
    return PairConfig{2, 8, 296};
}

struct PairSchedule { int blocks, n_full, kst, sc_per_split, grid, cluster; };

static PairSchedule pair_schedule(const Layout& l) {
    const PairConfig cfg = pair_config(l);
    PairSchedule sc{};
    sc.blocks = (l.RB + cfg.rpl - 1) / cfg.rpl;
    int rem = sc.blocks % cfg.slots;
    int kst = 1;
    const int kmax = l.SC / 4 > 1 ? l.SC / 4 : 1;   // keep K slices of at least 512 weights
    if (g_pair_ks_override > 0) {
        rem = sc.blocks; kst = g_pair_ks_override;
    } else if (sc.blocks < cfg.slots) {
        // fewer blocks than CTA slots: cut every block into 2, 4 or 8 K slices that form a cluster
        kst = 1;
        while (kst < 8 && sc.blocks * kst * 2 <= cfg.slots && kst * 2 <= kmax) kst *= 2;
        sc.cluster = kst > 1;
    } else if (rem > 0) {
        // blocks of the last, partial round: cut along K so that the pieces fit the slots of one round
        kst = cfg.slots / rem;
        if (kst > kmax) kst = kmax;
        if (kst > 64) kst = 64;
    }
    if (kst > l.SC) kst = l.SC;
    if (kst <= 1) { rem = 0; kst = 1; sc.cluster = 0; }
    sc.n_full = sc.blocks - rem;
    sc.sc_per_split = (l.SC + kst - 1) / kst;
    sc.kst = (l.SC + sc.sc_per_split - 1) / sc.sc_per_split;
    if (sc.cluster && (sc.kst & (sc.kst - 1))) sc.cluster = 0;   // cluster sizes are powers of two
    sc.grid = sc.n_full + rem * sc.kst;
    return sc;
}

static size_t pair_smem_bytes(const Layout& l, int nb) {
    const PairConfig cfg = pair_config(l);
    const int rows = 32 * cfg.rpl;
    const size_t T = (size_t)l.E * l.E;
    return T * 128 * cfg.rpl + (size_t)nb * l.cols * 2 + (size_t)cfg.warps * nb * rows * 4;
}

bool pair_supported(const Layout& l, int batch, int n_problems) {
    if (l.mode != 0 || l.bits < 2 || l.bits > 5 || batch > 2 || n_problems != 1) return false;
    return pair_smem_bytes(l, batch) <= (pair_config(l).rpl == 2 ? 110u : 220u) * 1024u;
}

size_t pair_workspace_bytes(const Layout& l) {
    const int ksmax = 64 < l.SC ? 64 : l.SC;
    return align256((size_t)l.RB * 4) + align256((size_t)ksmax * 2 * (size_t)(l.RB + 1) * 32 * 4);
}

template <int N, int NB, int RPL, int W>
static cudaError_t launch_pair(const PairArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    const int cluster = a.cluster ? a.kst : 1;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemv_pair_kernel<N, NB, RPL, W>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
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
    if (a.dbg == 3) {   // probe: plain stream order
        attr[0] = attr[1];
        cfg.numAttrs = cluster > 1 ? 1 : 0;
    }
    return cudaLaunchKernelEx(&cfg, gemv_pair_kernel<N, NB, RPL, W>, a);
}

cudaError_t launch_gemv_pair(const Layout& l, const GemvCall& c, cudaStream_t s) {
    const PairConfig cfg = pair_config(l);
    const PairSchedule sch = pair_schedule(l);
    PairArgs a{};
    a.off = offsets_of(l);
    a.packed = c.packed; a.x = c.x; a.y = c.y;
    a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.ell_slots = l.ell_slots;
    a.rows_ws = sch.blocks * 32 * cfg.rpl;
    a.n_full = sch.n_full; a.kst = sch.kst; a.sc_per_split = sch.sc_per_split;
    a.nb = c.batch; a.y_is_fp16 = c.y_is_fp16;
    a.pf_dist = g_pair_pf_dist;
    a.cluster = sch.cluster && g_pair_ks_override == 0;
    a.dbg = g_pair_dbg;
    a.trace = nullptr;
    if (g_pair_trace && g_pair_trace_idx < g_pair_trace_calls) a.trace = g_pair_trace + (g_pair_trace_idx++) * 1024 * 8;
    a.tickets = (int*)c.workspace;
    a.partial = (float*)((char*)c.workspace + align256((size_t)l.RB * 4));
    const size_t smem = pair_smem_bytes(l, c.batch);
    dim3 grid((unsigned)sch.grid, 1, 1);
    if (cfg.rpl == 1 && cfg.warps == 8) {
        switch (l.bits * 10 + c.batch) {
            case 31: return launch_pair<3, 1, 1, 8>(a, grid, smem, s);
            case 32: return launch_pair<3, 2, 1, 8>(a, grid, smem, s);
            case 41: return launch_pair<4, 1, 1, 8>(a, grid, smem, s);
            case 42: return launch_pair<4, 2, 1, 8>(a, grid, smem, s);
        }
        return cudaErrorInvalidValue;
    }
    if (cfg.rpl == 1) {
        switch (l.bits * 10 + c.batch) {
            case 31: return launch_pair<3, 1, 1, 16>(a, grid, smem, s);
            case 32: return launch_pair<3, 2, 1, 16>(a, grid, smem, s);
            case 41: return launch_pair<4, 1, 1, 16>(a, grid, smem, s);
            case 42: return launch_pair<4, 2, 1, 16>(a, grid, smem, s);
            case 51: return launch_pair<5, 1, 1, 16>(a, grid, smem, s);
            case 52: return launch_pair<5, 2, 1, 16>(a, grid, smem, s);
        }
        return cudaErrorInvalidValue;
    }
    switch (l.bits * 10 + c.batch) {
        case 21: return launch_pair<2, 1, 2, 8>(a, grid, smem, s);
        case 22: return launch_pair<2, 2, 2, 8>(a, grid, smem, s);
        case 31: return launch_pair<3, 1, 2, 8>(a, grid, smem, s);
        case 32: return launch_pair<3, 2, 2, 8>(a, grid, smem, s);
        case 41: return launch_pair<4, 1, 2, 8>(a, grid, smem, s);
        case 42: return launch_pair<4, 2, 2, 8>(a, grid, smem, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace xfp
