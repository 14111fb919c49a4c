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
// otherwise one entry per index with the entries of two library ids sharing a word -- see the kernel's comment.
//
// x is staged once per CTA in shared memory in an order that lets a diagonal lane fetch the B registers of TWO
// mma steps with one 16-byte load: inside every group of 16 k the two middle blocks of four are swapped
// ([0..3][8..11][4..7][12..15]).  Outlier columns are mapped through the same permutation.
//
// Outliers, split-K finish (ticket, fixed order) and the order of work before griddepcontrol.wait are those of
// xfp_gemv_pair.cu.
#include <cstdio>
#include <cstdlib>

#include "xfp_gemv_lane.cuh"

namespace xfp {

namespace {

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

// `RBn`: row-blocks of the launch (all blobs)
LaneConfig lane_config(const Layout& l, int n = 1) {
    const long long RB = (long long)l.RB * n;
#ifdef LANE_TUNE
    if (const char* e = getenv("XFP_LANE_CFG")) {   // tuning build: "W,per_sm,sgl"
        int w = 16, p = 1, g = 0, t = -1;
        sscanf(e, "%d,%d,%d,%d", &w, &p, &g, &t);
        if (w == 0) return LaneConfig{16, 1, false, true};
        const bool pairs = l.mode == 1 && (size_t)l.L * l.E * l.E * 128 <= 64 * 1024 && l.bits <= 3;
        return LaneConfig{w, p > 2 ? 2 : p, l.mode == 1 ? !pairs : (l.bits == 6 || (l.bits == 5 && g)), false, t < 0 ? p <= 2 : t != 0};
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
        // (pair tables between two and four rounds: 16 warps, 12288 x 4096 at N = 2 13.8 against 14.4 us)
        LaneConfig c{two && !(pairs && RB > 2 * sms && RB <= 4 * sms) ? 8 : 16, two ? 2 : 1, !pairs};
        c.tiers = RB > 4 * sms;   // up to four rounds unsplit, as in V2 (N = 6, one CTA per SM: 12288 x 4096 33.6 -> 26.6 us)
        c.off = false;
        // the blobs of a routed layer in one launch: the resident CTAs of xfp_gemv_v2a.cu (pair tables built once per
        // SM at N <= 3) measured faster (gate_up 30.7 vs 33.4 us, down 18.7 vs 22.9 us per launch of 8 experts)
        if (n > 1) c.off = true;
        return c;
    }
    if (RB <= sms) return LaneConfig{16, 1, l.bits == 6};
    const bool big = RB > 4 * sms;
    // 16 warps at N = 3, 4 only beyond one round of slots: in a single round 8 warps measured faster (8192 x 8192,
    // N = 4: 10.7 against 11.5 us)
    // N = 2 on short rows in a single round: the 64 KB fill dominates and 16 warps share it (8192 x 4096: 5.8 against 7.7 us)
    const bool w16 = !big && (RB > 2 * sms ? (l.bits == 3 || l.bits == 4) : (l.bits == 2 && l.SC <= 32));
    LaneConfig c{w16 ? 16 : 8, 2, l.bits >= 5};
    c.off = big && l.bits <= 3;   // the two-channels-per-lane kernel is ahead there
    c.tiers = big;
    return c;
}

template <int N, int W, int MINB, bool SGL, int MODE>
cudaError_t launch_lane(const LaneArgs& a, int grid, size_t smem, cudaStream_t s) {
    if (a.x_bf16 || a.y_is_fp16 == 2 || a.packed_list) return launch_lane_io<N, W, MINB, SGL, MODE, true, 1>(a, grid, smem, s);
    return launch_lane_io<N, W, MINB, SGL, MODE, false, 1>(a, grid, smem, s);
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
    if (l.mode && (size_t)((l.L + 1) / 2) * l.E * 128 > 128 * 1024) return false;   // V2a: the per-bank library must fit 128 KB
    const LaneConfig cfg = lane_config(l, c.n);
    if (cfg.off) return false;
    return lane_smem_bytes(l, cfg) <= (cfg.per_sm == 1 ? 220u : 110u) * 1024u;
}

cudaError_t launch_gemv_lane(const Layout& l, const GemvCall& c, cudaStream_t s) {
    const LaneConfig cfg = lane_config(l, c.n);
    const LaneSchedule sch = lane_schedule(l, l.RB * c.n, cfg.per_sm, cfg.tiers);
    LaneArgs a = lane_args(l, c, cfg.sgl);
    for (int i = 0; i < 5; ++i) a.tier_cta[i] = sch.tier_cta[i];
    for (int i = 0; i < 4; ++i) { a.tier_blk[i] = sch.tier_blk[i]; a.tier_kst[i] = sch.tier_kst[i]; a.tier_spp[i] = sch.tier_spp[i]; }
#ifdef XFP_TRACE
    a.trace = nullptr;
    if (g_lane_trace && g_lane_trace_idx < g_lane_trace_calls) a.trace = g_lane_trace + (g_lane_trace_idx++) * 1024 * 8;
#endif
    const size_t smem = lane_smem_bytes(l, cfg);
    if (l.mode) {
        switch (l.bits) {
            case 2: return cfg.sgl ? launch_lane_cfg<2, true, 1>(cfg, a, sch.grid, smem, s)
                                   : launch_lane_cfg<2, false, 1>(cfg, a, sch.grid, smem, s);
            case 3: return cfg.sgl ? launch_lane_cfg<3, true, 1>(cfg, a, sch.grid, smem, s)
                                   : launch_lane_cfg<3, false, 1>(cfg, a, sch.grid, smem, s);
            case 4: return launch_lane_cfg<4, true, 1>(cfg, a, sch.grid, smem, s);
            case 5: return launch_lane_cfg<5, true, 1>(cfg, a, sch.grid, smem, s);
            default: return launch_lane_cfg<6, true, 1>(cfg, a, sch.grid, smem, s);
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
