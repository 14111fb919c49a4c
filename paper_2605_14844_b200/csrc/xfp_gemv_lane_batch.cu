// The one-channel-per-lane decode kernel (xfp_gemv_lane.cu) for 2..8 rows of x, V2 and V2a:  Y = X (D + S)^T.
//
// Every decoded A fragment is multiplied with one B fragment per row of x (x on the diagonal lanes, as at batch 1),
// so the look-ups -- the cost that bounds the decode -- are paid once per weight whatever the batch; a row of x adds
// half a shared-memory wavefront and one mma per 256 weights.  The tensor pipe (one m16n8k16 per two clocks and SM)
// becomes the bound near 8 rows.
//
// A CTA stays resident and walks the row-blocks c, c + grid, ... with ONE staged copy of x (staging 8 rows of
// K = 8192 per row-block would move as many bytes as the weights); the row-blocks of the last partial round are cut
// along K so that every CTA gets a slice, and meet through the workspace in slice order (ticket, no waiting).
// V2a fills its library tables once per CTA, V2 its row-block's tables once per row-block.
#include <cstdlib>

#include "xfp_gemv_lane.cuh"

namespace xfp {

namespace {

struct BatchPlan {
    int NB;          // rows of x per launch (2, 4, 8)
    LaneConfig cfg;
    size_t smem;
};

int pow2_floor_b(int v) {
    int p = 1;
    while (p * 2 <= v) p *= 2;
    return p;
}

// The launch for `rows_x` (2..8) rows of x: the smallest tile that holds them, else the largest that fits shared memory.
bool batch_plan(const Layout& l, int rows_x, BatchPlan& p) {
    if (l.bits < 2 || l.bits > 6) return false;
    const int sms = sched_sms();
    if (l.RB * 2 <= sms) return false;   // tiny matrices cut every block along K: the kernels with clusters do that
    bool sgl;
    if (l.mode) {
        if ((size_t)((l.L + 1) / 2) * l.E * 128 > 128 * 1024) return false;
        sgl = !((size_t)l.L * l.E * l.E * 128 <= 64 * 1024 && l.bits <= 3);
    } else {
        sgl = l.bits >= 5;   // the 128 KB pair table of N = 5 leaves no room for several rows of x
    }
    for (int nb = 8; nb >= 2; nb /= 2) {
        if (nb >= 2 * rows_x && nb > 2) continue;   // a smaller tile holds the rows
        LaneConfig two{8, 2, sgl}, one{16, 1, sgl};
        if (l.RB > sms && lane_smem_bytes(l, two, nb) <= 110u * 1024u) {
            p = BatchPlan{nb, two, lane_smem_bytes(l, two, nb)};
            return true;
        }
        if (lane_smem_bytes(l, one, nb) <= 220u * 1024u) {
            p = BatchPlan{nb, one, lane_smem_bytes(l, one, nb)};
            return true;
        }
    }
    return false;
}

template <int N, bool SGL, int MODE, int NB>
cudaError_t launch_nb(const LaneConfig& c, const LaneArgs& a, int grid, size_t smem, cudaStream_t s) {
    if (c.W == 8) return launch_lane_io<N, 8, 2, SGL, MODE, false, NB>(a, grid, smem, s);
    return launch_lane_io<N, 16, 1, SGL, MODE, false, NB>(a, grid, smem, s);
}

template <int N, bool SGL, int MODE>
cudaError_t launch_tile(const BatchPlan& p, const LaneArgs& a, int grid, cudaStream_t s) {
    switch (p.NB) {
        case 2: return launch_nb<N, SGL, MODE, 2>(p.cfg, a, grid, p.smem, s);
        case 4: return launch_nb<N, SGL, MODE, 4>(p.cfg, a, grid, p.smem, s);
        default: return launch_nb<N, SGL, MODE, 8>(p.cfg, a, grid, p.smem, s);
    }
}

}  // namespace

// Where this kernel measured faster than the kernels with two channels per lane (xfp_gemv_pair.cu at 2 rows,
// xfp_gemv_batch.cu, xfp_gemv_v2a.cu), the general kernel and, from 9 rows (5 for V2a and N >= 5 on large blobs), the tcgen05 kernel; sweep over
// 4096 x 4096 .. 28672 x 8192, every bit width, 2 / 4 / 8 rows, 1 % outliers on a B200 (us per call, this kernel
// against the other):
//   * V2 N = 6 (the other kernel is the general one): everywhere (28672 x 8192, 4 rows: 78 against 240) except 2 rows
//     on matrices of one round (pair kernel 7.2 against 7.6)
//   * V2 N = 5 (the others keep one channel per lane there too): beyond one round (28672 x 8192, 8 rows: 114 against
//     160), and on one round where the batched kernel does not fit its shared memory (4096 x 12288, 4 rows: 19 against 54)
//   * V2 N <= 4: matrices of one round at 3 or 4 rows (4096 x 4096, 4 rows: 7.1 against 8.2); everywhere else two
//     channels per lane halve the mma count per weight and stay ahead (8192 x 8192, 4 rows: 16.4 against 19.9;
//     28672 x 8192, 8 rows: 80 against 105)
//   * V2a: up to 4 rows on matrices of one round (4096 x 4096, 2 rows: 7.9 against 11.2), N = 2 up to 4 rows
//     everywhere, N = 4 at 2 rows and on large matrices up to 4 rows (28672 x 8192: 86 against 92), N = 5 on large
//     matrices (8 rows: 158 against 198), N = 3 only at 3..4 rows on large matrices (its pair tables of the whole
//     library serve the other kernel), N = 6 everywhere (28672 x 8192, 8 rows: 193 against 766)
//   * many rows on a large matrix with few outliers stay on the tcgen05 kernel (28672 x 8192, 16 rows, 0.3 %: V2a 159
//     against 246)
static bool lane_batch_preferred(const Layout& l, int batch) {
    const int sms = sched_sms();
    const bool small = l.RB <= sms, big = l.RB > 4 * sms;
    if (batch_prefers_gemm(l, batch) && big) return false;
    const bool many = batch > 4;   // tiles of 8 rows
    if (l.mode == 0) {
        if (l.bits == 6) return !(small && batch == 2);
        if (l.bits == 5) return small ? (batch >= 3 && !batch_supported(l, batch)) : true;
        return small && batch >= 3 && !many;
    }
    if ((size_t)l.L * l.E * 128 > 128 * 1024) return true;   // N = 6 at L = 32: the other kernel is the general one
    if (small) return !many || !batch_supported(l, batch);
    switch (l.bits) {
        case 2: return !many;
        case 3: return big && batch >= 3 && !many;
        case 4: return batch == 2 || (big && !many);
        default: return big || (!many && l.RB > 2 * sms);
    }
}

// 2..16 rows of fp16 x, one blob, fp32 or fp16 y, no fused store
bool lane_batch_supported(const Layout& l, const GemvCall& c) {
    if (c.batch < 2 || c.n != 1 || c.packed_list || c.epilogue != 0) return false;
    if (c.x_bf16 || c.y_is_fp16 == 2) return false;
#ifdef LANE_TUNE
    if (const char* e = getenv("XFP_LANE_BATCH")) {   // tuning build: largest batch this kernel takes, whatever the rule
        if (c.batch > atoi(e)) return false;
    } else
#endif
    if (!lane_batch_preferred(l, c.batch)) return false;
    BatchPlan p;
    return batch_plan(l, c.batch < 8 ? c.batch : 8, p);
}

cudaError_t launch_gemv_lane_batch(const Layout& l, const GemvCall& c, cudaStream_t s) {
    const int sms = sched_sms();
    for (int b0 = 0; b0 < c.batch;) {
        const int left = c.batch - b0;
        BatchPlan p;
        if (!batch_plan(l, left < 8 ? left : 8, p)) return cudaErrorInvalidValue;
        GemvCall t = c;
        t.x = c.x + (size_t)b0 * l.cols;
        t.y = (char*)c.y + (size_t)b0 * l.rows * (c.y_is_fp16 ? 2 : 4);
        t.batch = left < p.NB ? left : p.NB;
        LaneArgs a = lane_args(l, t, p.cfg.sgl);
        // resident CTAs: whole blocks in whole rounds, the blocks of the last partial round in K slices
        const int G = l.RB < sms * p.cfg.per_sm ? l.RB : sms * p.cfg.per_sm;
        const int full = (l.RB / G) * G, tail = l.RB - full;
        // K slices per remaining block: as many as give every CTA at most one slice.  More, finer slices in several
        // waves measured slower whenever the tail is a large part of a round (8192 x 8192, 4 rows: 19.9 us unsplit, 26.4 us
        // with two waves of halves): a slice pays its own table fill, first loads and the finish through the workspace.
        int kst = 1;
        if (tail > 0) {
            const int kmax = l.SC / 4 > 1 ? pow2_floor_b(l.SC / 4) : 1;          // slices of at least 512 weights
            const int cap = 2 * (l.SC < 64 ? l.SC : 64) / p.NB;                    // partial sums the workspace holds
            kst = pow2_floor_b(G / tail);
            if (kst > kmax) kst = kmax;
            if (kst > cap) kst = cap;
            if (kst < 1) kst = 1;
        }
#ifdef LANE_TUNE
        if (const char* e = getenv("XFP_LANE_KST")) kst = atoi(e) < 1 ? 1 : atoi(e);
#endif
        const int spp = (l.SC + kst - 1) / kst;
        for (int i = 0; i < 5; ++i) a.tier_cta[i] = 0;
        for (int i = 0; i < 4; ++i) { a.tier_blk[i] = 0; a.tier_kst[i] = 1; a.tier_spp[i] = l.SC; }
        a.tier_blk[0] = full;
        a.tier_kst[0] = (l.SC + spp - 1) / spp;
        a.tier_spp[0] = spp;
        a.tier_cta[1] = tail * a.tier_kst[0];
        cudaError_t e;
        if (l.mode) {
            switch (l.bits) {
                case 2: e = p.cfg.sgl ? launch_tile<2, true, 1>(p, a, G, s) : launch_tile<2, false, 1>(p, a, G, s); break;
                case 3: e = p.cfg.sgl ? launch_tile<3, true, 1>(p, a, G, s) : launch_tile<3, false, 1>(p, a, G, s); break;
                case 4: e = launch_tile<4, true, 1>(p, a, G, s); break;
                case 5: e = launch_tile<5, true, 1>(p, a, G, s); break;
                default: e = launch_tile<6, true, 1>(p, a, G, s); break;
            }
        } else {
            switch (l.bits) {
                case 2: e = launch_tile<2, false, 0>(p, a, G, s); break;
                case 3: e = launch_tile<3, false, 0>(p, a, G, s); break;
                case 4: e = launch_tile<4, false, 0>(p, a, G, s); break;
                case 5: e = launch_tile<5, true, 0>(p, a, G, s); break;
                default: e = launch_tile<6, true, 0>(p, a, G, s); break;
            }
        }
        if (e != cudaSuccess) return e;
        b0 += t.batch;
    }
    return cudaSuccess;
}

}  // namespace xfp
