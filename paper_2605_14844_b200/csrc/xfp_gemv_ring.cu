// Persistent fused decode GEMV for V2 blobs at batch 1:  y = (D + S) x, one or several problems per launch.
//
// Same arithmetic as the pair-table kernel (xfp_gemv_pair.cu): the channels' codebooks are expanded into
// per-lane pair tables in shared memory ("codebook gather from shared memory", one 32-bit load decodes
// two weights, bank = lane, no conflicts), the looked-up half2 are the A fragment of mma.sync.m16n8k16
// with x on the diagonal of the B fragment, fp32 accumulation, outliers from the transposed slabs in the
// same pass.  What differs is how the index stream reaches the SM and how work is dealt out:
//
//  * One CTA of 16 warps per SM stays resident and walks a list of work items (a block of 32*RPL
//    channels x a range of super-chunks).  The warps of the CTA share an item's super-chunks round-robin.
//  * Every warp owns a small ring of shared-memory stages.  Lane 0 issues a bulk asynchronous copy
//    (cp.async.bulk, completion on an mbarrier) of the warp's next super-chunk -- N*512 contiguous bytes
//    per 32-channel row-block -- as soon as a stage has been read out, so each warp keeps `stages`
//    super-chunks in flight, across item boundaries, with no registers tied up and no load instructions
//    in the decode loop.  The stream does not stall while a CTA rebuilds its tables for the next block.
//  * The schedule is a table in the kernel parameters: CTA c works on the pooled units
//    [seg[c], seg[c+1]); a unit is (pooled block, super-chunk).
//    The host cuts the pooled unit space by cost (bytes), so a block may be shared by several CTAs; their
//    partial sums go through the workspace and the last CTA to arrive adds them in slice order (atomic
//    ticket, no waiting, fixed order -> reproducible results).
//
// Waits are bounded: a warp that does not see its copy complete within kWaitPolls polls raises the
// status word, the CTA writes NaN to the channels it owns and leaves after a second bounded wait for
// the copies still in flight.
//
// Launch overlap as in the pair kernel: index copies, codebooks, outlier slabs and tables are started
// before griddepcontrol.wait; x, y and the workspace are touched after it.
#include <algorithm>
#include <cstddef>

#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

constexpr int kRingMaxProblems = 8;
constexpr int kRingMaxCtas = 160;
constexpr int kRingSlots = 4;                // outlier slots a warp keeps in flight per channel half
constexpr uint32_t kWaitPolls = 1u << 20;
constexpr int kPosShift = 12;                // position = pooled block << 12 | super-chunk
constexpr uint32_t kPosMask = (1u << kPosShift) - 1u;

struct RingProblem {
    Offsets off;
    const void* packed;
    const uint16_t* x;
    void* y;
    float* partial;   // [slice][rows_ws]
    int* tickets;     // [blocks]
    int rows, cols, RB, SC, ell_slots, bits, rpl;
    int blocks;       // blocks of 32*rpl channels
    int blk_begin;    // pooled index of the first block
    int rows_ws;
};

struct RingArgs {
    int n, y_is_fp16;
    int stage_shift, stage_stride;     // ring: log2 of the stages per warp, bytes between stages
    int off_x, off_red, off_ring, off_misc;   // shared-memory layout behind the tables
    int fault;                         // test hook: withhold this CTA-0 warp-0 copy so that its wait runs out (0 = off)
    int zero;                          // always 0 (an operand the compiler cannot fold, see ring_issue)
    int* status;
    unsigned long long* trace;         // timing probe: per CTA 8 globaltimer stamps (null in normal use)
    RingProblem p[kRingMaxProblems];
    uint32_t seg[kRingMaxCtas + 1];    // CTA c works on the pooled units [seg[c], seg[c+1])
};

struct WarpRing {
    uint32_t ring, bar;        // shared-window addresses of this warp's first stage and first barrier
    uint32_t taken, issued;    // units taken out of the ring / copies started (stage = count mod stages)
    // producer cursor: the warp's next unit to copy
    const unsigned char* psrc; // its bytes (first row-block of the item)
    uint32_t pvb, pdelta;      // bytes of one row-block's unit; offset of the second row-block's unit
    int prpl;                  // row-blocks per unit of the producer's item
    int prem;                  // units of this warp left in the producer's item (0: no more work)
    int pgb;                   // the producer's item (pooled block)
    int dead;
};

__device__ __forceinline__ unsigned long long ring_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// probe: add the time since *t0 to trace slot `slot` of this CTA and restart the clock (thread 0 only)
__device__ __forceinline__ void ring_lap(const RingArgs& a, int slot, unsigned long long* t0) {
    if (a.trace && threadIdx.x == 0) {
        const unsigned long long t = ring_now();
        a.trace[(size_t)blockIdx.x * 8 + slot] += t - *t0;
        *t0 = t;
    }
}
__device__ __forceinline__ void ring_stamp(const RingArgs& a, int slot) {
    if (a.trace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        a.trace[(size_t)blockIdx.x * 8 + slot] = t;
    }
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for a phase of an mbarrier: 1 when the phase completed, 0 after kWaitPolls polls.
__device__ __forceinline__ uint32_t mbar_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .u32 i;\n\t"
        "mov.u32 i, 0;\n\t"
        "WAIT_LOOP:\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "@p bra WAIT_DONE;\n\t"
        "add.u32 i, i, 1;\n\t"
        "setp.lt.u32 p, i, %3;\n\t"
        "@p bra WAIT_LOOP;\n\t"
        "mov.u32 %0, 0;\n\t"
        "bra WAIT_END;\n\t"
        "WAIT_DONE:\n\t"
        "mov.u32 %0, 1;\n\t"
        "WAIT_END:\n\t"
        "}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "n"(kWaitPolls)
        : "memory");
    return done;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// The pair tables sit at the start of the dynamic shared memory, which on this architecture begins at
// shared address 1024 when the kernel has no static shared memory (the kernel checks it).  Spelling the
// address out as an immediate keeps the base out of the look-up's address arithmetic: the table offset
// built by pair_addr is the whole register operand.
constexpr uint32_t kTabShared = 1024;
__device__ __forceinline__ uint32_t lds_tab(uint32_t off) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+1024];" : "=r"(v) : "r"(off));
    return v;
}

template <bool kSingle>
__device__ __forceinline__ int problem_of(const RingArgs& a, int gb) {
    int j = 0;
    if (!kSingle) {
#pragma unroll
        for (int i = 1; i < kRingMaxProblems; ++i)
            if (i < a.n && gb >= a.p[i].blk_begin) j = i;
    }
    return j;
}

// Super-chunk range [sa, sb) of pooled block gb inside this CTA's range, and the block's problem.
template <bool kSingle>
__device__ __forceinline__ void seg_item(const RingArgs& a, int gb, int& sa, int& sb, int& j) {
    const uint32_t p0 = a.seg[blockIdx.x], p1 = a.seg[blockIdx.x + 1];
    j = problem_of<kSingle>(a, gb);
    sa = gb == (int)(p0 >> kPosShift) ? (int)(p0 & kPosMask) : 0;
    sb = gb == (int)(p1 >> kPosShift) ? (int)(p1 & kPosMask) : a.p[j].SC;
}

// Point the producer cursor at the first unit of this warp in pooled block r.pgb or a later block of the
// CTA's range (prem = 0 when there is none).  Runs once per item and warp; the per-unit path is ring_issue.
template <bool kSingle, int W>
__device__ __forceinline__ void producer_seek(const RingArgs& a, WarpRing& r, int warp) {
    const int gb1 = (int)(a.seg[blockIdx.x + 1] >> kPosShift);
    r.prem = 0;
    for (; r.pgb <= gb1; ++r.pgb) {
        int sa, sb, j;
        seg_item<kSingle>(a, r.pgb, sa, sb, j);
        const int n = sb - sa;
        if (warp >= n) continue;
        const RingProblem& P = a.p[j];
        const int rb0 = P.rpl * (r.pgb - P.blk_begin), rb1 = min(rb0 + P.rpl - 1, P.RB - 1);
        r.pvb = (uint32_t)P.bits * 512u;
        r.prpl = P.rpl;
        r.pdelta = (uint32_t)(rb1 - rb0) * (uint32_t)P.SC * r.pvb;
        r.psrc = (const unsigned char*)P.packed + P.off.idx + ((size_t)rb0 * P.SC + sa + warp) * r.pvb;
        r.prem = (n - warp + W - 1) / W;
        return;
    }
}

// Start the copy of the warp's next unit into its next free stage (lane 0 issues; every lane tracks the cursor).
// `dep`: a value computed from what the warp last read out of the stage (0 for a fresh stage).  The copy's
// byte count is made to depend on it, so the copy cannot be issued before those reads have returned.
template <bool kSingle, int W>
__device__ __forceinline__ void ring_issue(const RingArgs& a, WarpRing& r, int warp, int lane, uint32_t dep) {
    if (r.prem == 0) return;
    if (lane == 0) {
        const uint32_t st = r.issued & ((1u << a.stage_shift) - 1u);
        const uint32_t dst = r.ring + st * (uint32_t)a.stage_stride, bar = r.bar + st * 8u;
        mbar_expect(bar, r.pvb * (uint32_t)r.prpl + (dep & (uint32_t)a.zero));
        const bool withhold = a.fault && blockIdx.x == 0 && warp == 0 && (int)r.issued + 1 == a.fault;
        if (!withhold) {
            bulk_load(dst, r.psrc, r.pvb, bar);
            if (r.prpl == 2) bulk_load(dst + r.pvb, r.psrc + r.pdelta, r.pvb, bar);
        }
    }
    ++r.issued;
    r.psrc += (size_t)W * r.pvb;
    if (--r.prem == 0) {
        ++r.pgb;
        producer_seek<kSingle, W>(a, r, warp);
    }
}

// One work item: super-chunks [sa, sb) of block lb (32*RPL channels) of problem P; this CTA is slice
// `slice` of the `nslices` CTAs that share the block.
template <int N, int RPL, int W, bool kSingle>
__device__ __forceinline__ void ring_item(const RingArgs& a, const RingProblem& P, WarpRing& r, const int lb,
                                          const int sa, const int sb, const int slice, const int nslices,
                                          bool& waited, const uint16_t*& x_staged, int* s_flags,
                                          const unsigned char* zeros) {
    constexpr int E = 1 << N;
    constexpr int T = E * E;
    constexpr int ROWS = 32 * RPL;
    constexpr int kStride = 128 * RPL;
    constexpr int TW = T / W;
    constexpr int kThreads = W * 32;
    // look-up steps in flight ahead of the tensor pipe: with few warps the latency of the table look-ups is
    // covered inside the warp
    constexpr int kAhead = W == 16 ? 1 : (RPL == 2 ? 3 : 5);
    constexpr int kAcc = W == 16 ? 2 : 4;   // independent accumulator chains
    extern __shared__ __align__(128) unsigned char smem[];   // [tables | x | zeros | red | ring]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const char* blob = (const char*)P.packed;
    unsigned char* tab = smem;
    uint16_t* xs = (uint16_t*)(smem + a.off_x);
    float* red = (float*)(smem + a.off_red);   // [W][ROWS]

    const int blk0 = RPL * lb;
    const int blk1 = min(RPL * lb + (RPL - 1), P.RB - 1);   // clamped when RB is odd; its results are dropped
    const int gw = slice * W + warp, ostride = nslices * W;
    const int C = P.ell_slots;
    unsigned long long lap = a.trace ? ring_now() : 0;

    // ---- loads that do not depend on earlier kernels: slab lengths, first round of outlier slots, codebooks.
    //      Round `ocur` holds slots ocur + q * ostride (q < 4) of this warp; it is fetched one round ahead, the
    //      first before the rows' lengths are known (every slot below the capacity C is readable).
    const uint32_t* slab[RPL];
    int width[RPL];
    uint32_t olen[RPL];
    uint32_t oe[RPL][kRingSlots];
    int ocur = gw;
    auto fetch_slots = [&]() {
#pragma unroll
        for (int h = 0; h < RPL; ++h)
#pragma unroll
            for (int q = 0; q < kRingSlots; ++q) {
                const int j = ocur + q * ostride;
                oe[h][q] = j < width[h] ? __ldg(slab[h] + (1 + j) * 32) : 0u;
            }
    };
#pragma unroll
    for (int h = 0; h < RPL; ++h) {
        slab[h] = (const uint32_t*)(blob + P.off.ell) + (size_t)((h ? blk1 : blk0) * (C + 1)) * 32 + lane;
        width[h] = C;
        olen[h] = C ? __ldg(slab[h]) : 0u;
    }
    if (C) fetch_slots();

    // ---- pair tables: warp w fills entries t in [w*T/W, (w+1)*T/W) of every channel half
#pragma unroll
    for (int half = 0; half < RPL; ++half) {
        const uint16_t* cb = (const uint16_t*)(blob + P.off.cb) + (size_t)((half ? blk1 : blk0) * kRowsPerBlock + lane) * E;
        unsigned char* dst = tab + half * 128 + lane * 4;
        if (TW >= E) {
            uint32_t cbw[E / 2];
#pragma unroll
            for (int i = 0; i < E / 8; ++i) {
                const uint4 t = __ldg((const uint4*)cb + i);
                cbw[4 * i] = t.x; cbw[4 * i + 1] = t.y; cbw[4 * i + 2] = t.z; cbw[4 * i + 3] = t.w;
            }
#pragma unroll
            for (int hh = 0; hh < TW / E; ++hh) {
                const int hi = warp * (TW / E) + hh;
                const uint32_t hv = (uint32_t)__ldg(cb + hi) << 16;
#pragma unroll
                for (int lo = 0; lo < E; ++lo) {
                    const uint32_t lv = (lo & 1) ? (cbw[lo >> 1] >> 16) : (cbw[lo >> 1] & 0xffffu);
                    *(uint32_t*)(dst + (size_t)(hi * E + lo) * kStride) = lv | hv;
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < (TW > 0 ? TW : 1); ++i) {
                const int t = TW > 0 ? warp * TW + i : warp;
                if (t < T) {
                    const uint32_t lv = __ldg(cb + (t & (E - 1))), hv = __ldg(cb + (t >> N));
                    *(uint32_t*)(dst + (size_t)t * kStride) = lv | (hv << 16);
                }
            }
        }
    }
    // ---- x (fp16 bits, all of K: outlier columns are gathered from it) may come from the previous kernel
    if (!waited) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
        ring_stamp(a, 2);
    }
    if (x_staged != P.x) {
        for (int t = threadIdx.x; t < P.SC * (kSuper / 8); t += kThreads)
            *(uint4*)(xs + (size_t)t * 8) = __ldg((const uint4*)P.x + t);
        x_staged = P.x;
    }
    __syncthreads();   // tables and x visible
    ring_lap(a, 1, &lap);

    const uint32_t base0 = (uint32_t)lane * 4u, base1 = base0 | 128u;
    const int g = lane >> 2, t4 = lane & 3;
    const bool diag = (g == t4);   // B fragment: lane (g, t) with g == t feeds column t with the k slots of group t

    float c[kAcc][4];
#pragma unroll
    for (int i = 0; i < kAcc; ++i) { c[i][0] = 0.f; c[i][1] = 0.f; c[i][2] = 0.f; c[i][3] = 0.f; }
    float oacc[RPL];
    int wany = 0;   // slots any channel of this warp uses: rounds at or beyond it are empty
#pragma unroll
    for (int h = 0; h < RPL; ++h) {
        int wmax = (int)olen[h];
#pragma unroll
        for (int o = 16; o; o >>= 1) wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
        width[h] = min(wmax, C);
        wany = max(wany, width[h]);
        oacc[h] = 0.f;
    }
    auto outlier_round = [&]() {
#pragma unroll
        for (int h = 0; h < RPL; ++h)
#pragma unroll
            for (int q = 0; q < kRingSlots; ++q)
                oacc[h] = fmaf(h2f((uint16_t)(oe[h][q] >> 16)), h2f(xs[oe[h][q] & 0xffffu]), oacc[h]);
        ocur += kRingSlots * ostride;
        if (ocur < wany) fetch_slots();
    };

    const uint32_t smask = (1u << a.stage_shift) - 1u;
    uint4 xq[2];
    // ---- K loop: one unit (super-chunk of the block) per iteration, taken from the warp's ring
#pragma unroll 1
    for (int sc = sa + warp; sc < sb; sc += W) {
        if (ocur < wany) outlier_round();
        uint32_t w0[4 * N + 1], w1[RPL == 2 ? 4 * N + 1 : 1];
        w0[4 * N] = 0u;
        if (RPL == 2) w1[4 * N] = 0u;
        const uint32_t st = r.taken & smask;
        if (!r.dead && !mbar_wait(r.bar + st * 8u, (r.taken >> a.stage_shift) & 1u)) {
            r.dead = 1;
            r.prem = 0;
            s_flags[1] = 1;
            if (lane == 0 && a.status) atomicExch(a.status, 1);
        }
        ++r.taken;
        const unsigned char* sp = smem + a.off_ring + (warp << a.stage_shift) * a.stage_stride + st * a.stage_stride + lane * 16;

        // The unit is 32 mma steps of 4 consecutive k.  The table look-ups of step q are issued kAhead
        // steps before its mma.  Vector v of the index stream is first touched by step 32 v / N and is
        // read from the stage two steps before that; once the last vector has come back the stage is
        // handed to the next copy.
        auto load_vec = [&](int v) {
            const uint4 t0 = *(const uint4*)(sp + v * 512);
            w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
            if (RPL == 2) {
                const uint4 t1 = *(const uint4*)(sp + (N + v) * 512);
                w1[4 * v] = t1.x; w1[4 * v + 1] = t1.y; w1[4 * v + 2] = t1.z; w1[4 * v + 3] = t1.w;
            }
        };
        auto lookup = [&](uint32_t (&f)[4], int m) {
            f[0] = lds_tab(pair_addr<N, RPL>(w0, 2 * m, base0));
            f[2] = lds_tab(pair_addr<N, RPL>(w0, 2 * m + 1, base0));
            if (RPL == 2) {
                f[1] = lds_tab(pair_addr<N, RPL>(w1, 2 * m, base1));
                f[3] = lds_tab(pair_addr<N, RPL>(w1, 2 * m + 1, base1));
            } else {
                f[1] = 0u; f[3] = 0u;
            }
        };
        auto issue_step = [&](uint32_t (&f)[4], int q) {   // everything that belongs to look-up step q (compile time)
#pragma unroll
            for (int v = 0; v < N; ++v) {
                const int at = (32 * v) / N - 2;
                if ((at < 0 ? 0 : at) == q) load_vec(v);
            }
            lookup(f, q);
            if (q == (32 * (N - 1)) / N) {
                // the look-ups above consumed the last vector: every read of the stage has returned
                const uint32_t dep = w0[4 * N - 1] ^ (RPL == 2 ? w1[4 * N - 1] : 0u);
                __syncwarp();
                ring_issue<kSingle, W>(a, r, warp, lane, dep);
            }
        };
        constexpr int STEPS = kSuper / 4;
        // B fragments: the diagonal lanes read x, the others a block of zeros (no predicates in the loop; the
        // zeros sit 64 bytes off the 128-byte phase of x, so the two addresses of a load never share a bank)
        const unsigned char* xp = diag ? (const unsigned char*)xs + sc * (kSuper * 2) : zeros + 64;
        uint32_t f[kAhead + 1][4];
        xq[0] = *(const uint4*)xp;   // x of steps 0, 1
#pragma unroll
        for (int q = 0; q < kAhead; ++q) issue_step(f[q], q);
#pragma unroll
        for (int m = 0; m < STEPS; ++m) {
            if (m + kAhead < STEPS) issue_step(f[(m + kAhead) % (kAhead + 1)], m + kAhead);
            if ((m & 1) == 0 && m / 2 + 1 < STEPS / 2) xq[(m / 2 + 1) & 1] = *(const uint4*)(xp + (m / 2 + 1) * 16);
            uint32_t(&fm)[4] = f[m % (kAhead + 1)];
            const uint4 xv = xq[(m / 2) & 1];
            if (m & 1) mma16816(c[m % kAcc], fm[0], fm[1], fm[2], fm[3], xv.z, xv.w);
            else mma16816(c[m % kAcc], fm[0], fm[1], fm[2], fm[3], xv.x, xv.y);
        }
    }
    ring_lap(a, 3, &lap);
    while (ocur < wany) outlier_round();   // more outlier rounds than super-chunks
    // Rows that fill their slab continue in the CSR arrays (pathological skew only): warp 0 of the
    // block's first slice finishes them, one lane per row.
    if (warp == 0 && slice == 0 && C) {
#pragma unroll
        for (int h = 0; h < RPL; ++h) {
            if ((int)olen[h] >= C) {
                const int* rowptr = (const int*)(blob + P.off.rowptr);
                const uint32_t* oent = (const uint32_t*)(blob + P.off.oent);
                const int row = (h ? blk1 : blk0) * kRowsPerBlock + lane;
                const int p1 = __ldg(rowptr + row + 1);
                for (int p = __ldg(rowptr + row) + C; p < p1; ++p) {
                    const uint32_t e = __ldg(oent + p);
                    oacc[h] = fmaf(h2f((uint16_t)(e >> 16)), h2f(xs[e & 0xffffu]), oacc[h]);
                }
            }
        }
    }
    // ---- scatter the fragment to channel order: lane (g, t) holds D[g][2t], D[g][2t+1], D[g+8][..];
    //      column n < 4 belongs to channel lane 4g + n
    if (t4 < 2) {
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[e] = c[0][e] + c[1][e];
            if (kAcc == 4) v[e] += c[2][e] + c[3][e];
        }
        float* rr = red + warp * ROWS;
        const int l0 = 4 * g + 2 * t4;
        rr[l0] = v[0]; rr[l0 + 1] = v[1];
        if (RPL == 2) { rr[32 + l0] = v[2]; rr[32 + l0 + 1] = v[3]; }
    }
    __syncwarp();
#pragma unroll
    for (int h = 0; h < RPL; ++h) red[warp * ROWS + 32 * h + lane] += oacc[h];
    __syncthreads();   // partial sums of all warps are in red; tables and x are free for the next item
    ring_lap(a, 4, &lap);

    // ---- fixed-order reduction over the warps (threads 0..ROWS-1), then store or combine the block's slices
    if (threadIdx.x < ROWS) {
        const int t = threadIdx.x;
        const bool dup = (t >= 32) && (RPL * lb + 1 >= P.RB);
        const int row = lb * ROWS + t;
        float total = 0.f;
#pragma unroll
        for (int w = 0; w < W; ++w) total += red[w * ROWS + t];
        bool writer = true;
        if (nslices > 1) {
            P.partial[(size_t)slice * P.rows_ws + row] = total;
            __threadfence();
            asm volatile("bar.sync 1, %0;" ::"n"(ROWS));
            if (t == 0) s_flags[0] = (atomicAdd(P.tickets + lb, 1) == nslices - 1);
            asm volatile("bar.sync 1, %0;" ::"n"(ROWS));
            writer = s_flags[0] != 0;
            if (writer) {
                __threadfence();
                total = 0.f;
                for (int k2 = 0; k2 < nslices; ++k2) total += __ldcg(P.partial + (size_t)k2 * P.rows_ws + row);
                if (t == 0) P.tickets[lb] = 0;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(ROWS));   // s_flags[0] is rewritten by the next item
        }
        if (s_flags[1]) total = __int_as_float(0x7fc00000);
        if (writer && !dup && row < P.rows) {
            if (a.y_is_fp16)
                ((uint16_t*)P.y)[row] = f2h(total);
            else
                ((float*)P.y)[row] = total;
        }
    }
    ring_lap(a, 6, &lap);
}

template <int NS, int RS, int W>   // NS = 0: bit width and rows per lane taken from each problem
__global__ void __launch_bounds__(W * 32, 1) gemv_ring_kernel(const __grid_constant__ RingArgs a) {
    constexpr bool kSingle = NS != 0;
    extern __shared__ __align__(128) unsigned char smem[];
    // behind the ring: 384 bytes of zeros (for the idle B-fragment lanes), the warps' barriers, two flags
    uint32_t* s_zero = (uint32_t*)(smem + a.off_misc);
    unsigned long long* s_bar = (unsigned long long*)(smem + a.off_misc + 384);          // [W][4]
    int* s_flags = (int*)(smem + a.off_misc + 384 + 512);   // [0] last-arriver flag of the ticket, [1] a wait ran out
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    {
        // The parameters arrive through the constant cache, one miss per 64-byte line on first touch: touch
        // the lines this CTA will need from different warps at once instead of one after the other.
        const uint32_t* pw = (const uint32_t*)&a;
        const int head = (int)((offsetof(RingArgs, p) + sizeof(RingProblem) * (kSingle ? 1 : a.n) + 63) / 64);
        int word = -1;
        if (warp < head && warp < W - 2) word = warp * 16;
        else if (warp == W - 2) word = (int)(offsetof(RingArgs, seg) / 4) + blockIdx.x;
        else if (warp == W - 1) word = (int)(offsetof(RingArgs, seg) / 4) + blockIdx.x + 1;
        if (word >= 0) {
            const uint32_t v = pw[word];
            asm volatile("" ::"r"(v));
        }
    }
    ring_stamp(a, 0);
    if ((uint32_t)__cvta_generic_to_shared(smem) != kTabShared) {   // layout assumption of lds_tab broken: refuse to run
        if (threadIdx.x == 0 && a.status) atomicExch(a.status, 2);
        return;
    }
    if (threadIdx.x == 0) { s_flags[0] = 0; s_flags[1] = 0; }
    if (threadIdx.x < 96) s_zero[threadIdx.x] = 0u;

    WarpRing r;
    r.ring = (uint32_t)__cvta_generic_to_shared(smem + a.off_ring) + (uint32_t)((warp << a.stage_shift) * a.stage_stride);
    r.bar = (uint32_t)__cvta_generic_to_shared(s_bar + warp * 4);
    r.taken = 0; r.issued = 0; r.dead = 0;
    if (lane == 0) {
        for (int s = 0; s < (1 << a.stage_shift); ++s) mbar_init(r.bar + 8u * s, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    r.pgb = (int)(a.seg[blockIdx.x] >> kPosShift);
    producer_seek<kSingle, W>(a, r, warp);
    for (int s = 0; s < (1 << a.stage_shift); ++s) ring_issue<kSingle, W>(a, r, warp, lane, 0u);

    bool waited = false;
    const uint16_t* x_staged = nullptr;
    {
        const uint32_t p0 = a.seg[blockIdx.x], p1 = a.seg[blockIdx.x + 1];
        const int gb0 = (int)(p0 >> kPosShift), gb1 = (int)(p1 >> kPosShift);
#pragma unroll 1
        for (int gb = gb0; gb <= gb1; ++gb) {
            int sa, sb, j;
            seg_item<kSingle>(a, gb, sa, sb, j);
            if (sa >= sb) continue;
            const RingProblem& P = a.p[j];
            int slice = 0, nslices = 1;
            if (sa > 0 || sb < P.SC) {
                // the CTAs that share the block: cf .. cl
                int cf = blockIdx.x, cl = blockIdx.x;
                const uint32_t bpos = (uint32_t)gb << kPosShift, epos = (uint32_t)(gb + 1) << kPosShift;
                while (cf > 0 && a.seg[cf] > bpos) --cf;
                while (cl + 1 < (int)gridDim.x && a.seg[cl + 1] < epos) ++cl;
                slice = blockIdx.x - cf;
                nslices = cl - cf + 1;
            }
            const int lb = gb - P.blk_begin;
            if (kSingle) {
                ring_item<NS ? NS : 4, RS ? RS : 1, W, kSingle>(a, P, r, lb, sa, sb, slice, nslices, waited, x_staged, s_flags, (const unsigned char*)s_zero);
            } else {
                switch (P.bits * 2 + P.rpl) {
                    case 7:  ring_item<3, 1, W, kSingle>(a, P, r, lb, sa, sb, slice, nslices, waited, x_staged, s_flags, (const unsigned char*)s_zero); break;
                    case 8:  ring_item<3, 2, W, kSingle>(a, P, r, lb, sa, sb, slice, nslices, waited, x_staged, s_flags, (const unsigned char*)s_zero); break;
                    case 9:  ring_item<4, 1, W, kSingle>(a, P, r, lb, sa, sb, slice, nslices, waited, x_staged, s_flags, (const unsigned char*)s_zero); break;
                    case 10: ring_item<4, 2, W, kSingle>(a, P, r, lb, sa, sb, slice, nslices, waited, x_staged, s_flags, (const unsigned char*)s_zero); break;
                    default: ring_item<5, 1, W, kSingle>(a, P, r, lb, sa, sb, slice, nslices, waited, x_staged, s_flags, (const unsigned char*)s_zero); break;
                }
            }
        }
    }
    // A wait ran out somewhere: give the copies that may still be in flight a bounded chance to land
    // before the shared memory is released.
    __syncthreads();
    if (s_flags[1]) {
        for (; r.taken != r.issued; ++r.taken)
            mbar_wait(r.bar + (r.taken & ((1u << a.stage_shift) - 1u)) * 8u, (r.taken >> a.stage_shift) & 1u);
    }
    ring_stamp(a, 5);
}

// ------------------------------------------------------------------------------------ host side

static int g_ring_enable = 0;     // probe switch: 1 routes eligible calls to this kernel
static int g_ring_policy = 0;     // probe switch: schedule policy
static int g_ring_fault = 0;
static int g_ring_stages = 0;     // probe: cap on stages (0 = as many as fit, at most 4)
static int g_ring_warps = 16;     // probe: warps per CTA (8 or 16)
static unsigned long long* g_ring_trace = nullptr;   // probe: calls write their stamps to consecutive slices of 1024 CTAs x 8
static long long g_ring_trace_calls = 0, g_ring_trace_idx = 0;
void ring_set(int what, long long v) {
    if (what == 0) g_ring_enable = (int)v;
    if (what == 1) g_ring_policy = (int)v;
    if (what == 2) g_ring_fault = (int)v;
    if (what == 3) g_ring_stages = (int)v;
    if (what == 4) { g_ring_trace = (unsigned long long*)(uintptr_t)v; g_ring_trace_idx = 0; }
    if (what == 5) g_ring_trace_calls = v;
    if (what == 6) g_ring_warps = (int)v;
}

static int ring_rpl(const Layout& l, int pooled_rb) {
    // two channels per lane halve the x-fragment loads, but need 64-row blocks: only when that still
    // leaves at least two blocks per SM
    if (l.bits == 5) return 1;
    return pooled_rb >= 4 * 148 ? 2 : 1;
}

size_t ring_workspace_bytes(const Layout& l) {
    return align256((size_t)(l.RB + 1) * 4) + align256((size_t)64 * (l.RB + 1) * 32 * 4);
}

struct RingPlan {
    RingArgs args;
    int grid;
    size_t smem;
    int ns, rs;   // template selection (0, 0 = per-problem switch)
    int warps;
};

static bool ring_plan(int n, const Layout* ls, const GemvCall* cs, RingPlan& pl) {
    if (!g_ring_enable || n < 1 || n > kRingMaxProblems) return false;
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return false;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
        if (sms > kRingMaxCtas) sms = kRingMaxCtas;
    }
    int pooled_rb = 0;
    for (int j = 0; j < n; ++j) {
        const Layout& l = ls[j];
        if (l.mode != 0 || cs[j].batch != 1 || l.bits < 2 || l.bits > 5 || l.SC > (int)kPosMask || l.SC < 1) return false;
        if (n > 1 && l.bits < 3) return false;
        if (cs[j].y_is_fp16 != cs[0].y_is_fp16 || cs[j].packed_list) return false;
        pooled_rb += l.RB;
    }
    RingArgs& a = pl.args;
    a = RingArgs{};
    a.n = n;
    a.y_is_fp16 = cs[0].y_is_fp16;
    const int kRW = g_ring_warps == 8 ? 8 : 16;
    pl.warps = kRW;
    size_t tab = 0, xb = 0, red = 0, stride = 0;
    long long total_cost = 0, total_units = 0;
    int blocks = 0, max_block_cost = 0;
    for (int j = 0; j < n; ++j) {
        const Layout& l = ls[j];
        RingProblem& P = a.p[j];
        P.off = offsets_of(l);
        P.packed = cs[j].packed; P.x = cs[j].x; P.y = cs[j].y;
        P.rows = l.rows; P.cols = l.cols; P.RB = l.RB; P.SC = l.SC; P.ell_slots = l.ell_slots; P.bits = l.bits;
        P.rpl = ring_rpl(l, pooled_rb);
        P.blocks = (l.RB + P.rpl - 1) / P.rpl;
        P.blk_begin = blocks;
        P.rows_ws = P.blocks * 32 * P.rpl;
        P.tickets = (int*)cs[j].workspace;
        P.partial = (float*)((char*)cs[j].workspace + align256((size_t)(l.RB + 1) * 4));
        blocks += P.blocks;
        const size_t T = (size_t)l.E * l.E;
        tab = std::max(tab, T * 128 * P.rpl);
        xb = std::max(xb, (size_t)l.cols * 2);
        red = std::max(red, (size_t)kRW * 32 * P.rpl * 4);
        stride = std::max(stride, (size_t)P.rpl * l.bits * 512);
        const int c = P.rpl * l.bits;
        total_cost += (long long)P.blocks * l.SC * c;
        total_units += (long long)P.blocks * l.SC;
        max_block_cost = std::max(max_block_cost, l.SC * c);
    }
    if (blocks >= (1 << (31 - kPosShift))) return false;
    a.status = (int*)((char*)cs[0].workspace + status_offset(ls[0]));
    a.fault = g_ring_fault;
    a.trace = nullptr;
    // shared memory: [tables | x | red | ring]
    const size_t budget = 226 * 1024;   // ring and everything before it; 1 KB of barriers, flags and zeros follows
    const size_t fixed = tab + align256(xb) + align256(red);
    if (fixed + 2 * kRW * stride > budget) return false;
    int stages = (budget - fixed) / (kRW * stride) >= 4 ? 4 : 2;
    if (g_ring_stages > 0 && stages > g_ring_stages) stages = g_ring_stages >= 4 ? 4 : 2;
    a.stage_shift = stages == 4 ? 2 : 1;
    a.stage_stride = (int)stride;
    a.off_x = (int)tab;
    a.off_red = (int)(tab + align256(xb));
    a.off_ring = (int)fixed;
    a.off_misc = (int)(fixed + (size_t)stages * kRW * stride);
    pl.smem = a.off_misc + 1024;

    // ---- schedule
    int G = sms;
    if (total_units < G) G = (int)total_units;
    // a block may be shared by at most 64 CTAs (rows of the partial-sum workspace)
    while (G > 1 && (max_block_cost + total_cost / G - 1) / (total_cost / G) + 1 > 64) --G;
    auto pos_of_unit = [&](int j, long long u) -> uint32_t {   // unit u of problem j (block-major)
        const RingProblem& P = a.p[j];
        return (uint32_t)((P.blk_begin + u / P.SC) << kPosShift) | (uint32_t)(u % P.SC);
    };
    const uint32_t end_pos = (uint32_t)blocks << kPosShift;
    if (blocks <= G && 2 * blocks > G && g_ring_policy != 1) {
        // one whole block per CTA
        G = blocks;
        for (int c = 0; c <= G; ++c) a.seg[c] = (uint32_t)c << kPosShift;
    } else {
        // cost-balanced cut of the pooled unit space; CTA c owns the units whose start cost lies in
        // [c*C/G, (c+1)*C/G).  Every CTA must own at least one unit: retry with fewer CTAs otherwise.
        for (;; --G) {
            for (int c = 0; c <= G; ++c) {
                const long long start = total_cost * c / G;
                long long prefix = 0;
                uint32_t pos = end_pos;
                for (int j = 0; j < n; ++j) {
                    const RingProblem& P = a.p[j];
                    const long long cj = (long long)P.rpl * P.bits, uj = (long long)P.blocks * P.SC;
                    if (start < prefix + uj * cj) {
                        const long long u = start <= prefix ? 0 : (start - prefix + cj - 1) / cj;
                        pos = u >= uj ? (j + 1 < n ? pos_of_unit(j + 1, 0) : end_pos) : pos_of_unit(j, u);
                        break;
                    }
                    prefix += uj * cj;
                }
                a.seg[c] = pos;
            }
            a.seg[0] = 0;
            a.seg[G] = end_pos;
            bool ok = true;
            for (int c = 0; c < G; ++c) ok = ok && a.seg[c] < a.seg[c + 1];
            if (ok || G == 1) break;
        }
    }
    pl.grid = G;
    if (n == 1) { pl.ns = a.p[0].bits; pl.rs = a.p[0].rpl; } else { pl.ns = 0; pl.rs = 0; }
    return true;
}

template <int NS, int RS, int W>
static cudaError_t ring_launch_t(const RingPlan& pl, cudaStream_t s) {
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemv_ring_kernel<NS, RS, W>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             227 * 1024);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)pl.grid, 1, 1);
    cfg.blockDim = dim3(W * 32, 1, 1);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_ring_kernel<NS, RS, W>, pl.args);
}

template <int W>
static cudaError_t ring_launch_w(const RingPlan& pl, cudaStream_t s) {
    switch (pl.ns * 4 + pl.rs) {
        case 0:  return ring_launch_t<0, 0, W>(pl, s);
        case 9:  return ring_launch_t<2, 1, W>(pl, s);
        case 10: return ring_launch_t<2, 2, W>(pl, s);
        case 13: return ring_launch_t<3, 1, W>(pl, s);
        case 14: return ring_launch_t<3, 2, W>(pl, s);
        case 17: return ring_launch_t<4, 1, W>(pl, s);
        case 18: return ring_launch_t<4, 2, W>(pl, s);
        case 21: return ring_launch_t<5, 1, W>(pl, s);
        default: return cudaErrorInvalidValue;
    }
}

bool ring_supported(int n, const Layout* ls, const GemvCall* cs) {
    RingPlan pl;
    return ring_plan(n, ls, cs, pl);
}

cudaError_t launch_gemv_ring(int n, const Layout* ls, const GemvCall* cs, cudaStream_t s) {
    RingPlan pl;
    if (!ring_plan(n, ls, cs, pl)) return cudaErrorInvalidValue;
    if (g_ring_trace && g_ring_trace_idx < g_ring_trace_calls) pl.args.trace = g_ring_trace + (size_t)(g_ring_trace_idx++) * 1024 * 8;
    return pl.warps == 8 ? ring_launch_w<8>(pl, s) : ring_launch_w<16>(pl, s);
}

}  // namespace xfp
