// Launchers shared between the translation units of libxfp.  Every launcher queues work on
// `stream` and returns the cudaError_t of the launch.
#pragma once
#include <cstdlib>
#include <cuda_runtime.h>

#include <atomic>

#include "xfp_common.cuh"

namespace xfp {

// Function attributes (the opt-in shared-memory size) belong to a device: every kernel instantiation remembers
// on which devices it has set them, so a process that drives several GPUs sets them on each.
// Host threads may race to the first launch: the bits are atomic (setting an attribute twice is harmless, losing
// another thread's bit is not).
struct DeviceOnce {
    std::atomic<unsigned long long> mask[4] = {};   // devices 0..255
    static int current() {
        int d = 0;
        cudaGetDevice(&d);
        return d & 255;
    }
    bool is_set(int d) const { return (mask[d >> 6].load(std::memory_order_acquire) >> (d & 63)) & 1ull; }
    void set(int d) { mask[d >> 6].fetch_or(1ull << (d & 63), std::memory_order_release); }
};

// Streaming multiprocessors of the current device, asked once per device.  Schedules (CTA slots per round, K
// splits) are built from it; workspace SIZES are a function of the descriptor alone and never depend on it.
int sm_count();
// The SM count the workspace sizes of the split-K kernels allow for: a launch never plans for more SMs than this,
// so its partial sums fit the size xfp_packed_size reported without asking a device (a B200 has 148).
constexpr int kSizingSMs = 148;
inline int sched_sms() {
    const int n = sm_count();
    return n < kSizingSMs ? n : kSizingSMs;
}

struct PackInputs {
    const uint8_t* idx;
    const uint16_t* codebook;
    const uint8_t* gid;
    const uint16_t* gscale;
    const uint16_t* gmid;
    const int32_t* rowptr;
    const void* ocol;
    int col_bits;
    const uint16_t* oval;
};

cudaError_t launch_pack(const Layout& l, const PackInputs& in, void* packed, int* err_word, cudaStream_t s);
cudaError_t launch_dequant(const Layout& l, const void* packed, uint16_t* W, cudaStream_t s);

// One GEMV problem set: either a single blob (packed/x/y) or n blobs through device pointer lists.
struct GemvCall {
    const void* packed;
    const uint16_t* x;
    void* y;
    const void* const* packed_list;
    const uint16_t* const* x_list;
    void* const* y_list;
    int n;          // number of problems (1 for the single form)
    int batch;      // rows of x (1..16)
    int y_is_fp16;  // type of y: 0 fp32, 1 fp16, 2 bf16
    void* workspace;
    size_t workspace_bytes;  // per problem
    int epilogue = 0;                      // XFP_EPI_* (grouped V2a launches only)
    const float* epi_weights = nullptr;    // XFP_EPI_COMBINE: [n] routing weights on the device
    int x_bf16 = 0;                        // x holds bf16 instead of fp16
};

// Split-K factor the generic kernel uses for this shape and batch tile on `sms` SMs (host-side policy).
int generic_ksplit(const Layout& l, int batch_tile, int sms);
size_t generic_workspace_bytes(const Layout& l);
cudaError_t launch_gemv_generic(const Layout& l, const GemvCall& c, cudaStream_t s);

// Fast V2 path (pair tables + mma.sync fragments); see xfp_gemv_pair.cu.
bool pair_supported(const Layout& l, int batch, int n_problems);
size_t pair_workspace_bytes(const Layout& l);
cudaError_t launch_gemv_pair(const Layout& l, const GemvCall& c, cudaStream_t s);

// Batch 1, one channel per lane, V2 and V2a; see xfp_gemv_lane.cu.
bool lane_supported(const Layout& l, const GemvCall& c);
cudaError_t launch_gemv_lane(const Layout& l, const GemvCall& c, cudaStream_t s);
// The same decode for 2..16 rows of x (tiles of 2, 4, 8 rows); see xfp_gemv_lane_batch.cu.
bool lane_batch_supported(const Layout& l, const GemvCall& c);
cudaError_t launch_gemv_lane_batch(const Layout& l, const GemvCall& c, cudaStream_t s);

// Fast V2a path (per-bank library + mma.sync fragments, one or several blobs); see xfp_gemv_v2a.cu.
bool v2a_supported(const Layout& l, int batch);
size_t v2a_workspace_bytes(const Layout& l);
cudaError_t launch_gemv_v2a(const Layout& l, const GemvCall& c, cudaStream_t s);

// Batched path (3..16 rows of x), V2 and V2a; see xfp_gemv_batch.cu.
bool batch_supported(const Layout& l, int batch);
cudaError_t launch_gemv_batch(const Layout& l, const GemvCall& c, cudaStream_t s);

// Prefill form on the tcgen05 tensor cores (V2, any number of rows of x); see xfp_gemm_tc.cu.
struct GemmCall {
    const void* packed;
    const uint16_t* x;   // [M][cols] fp16
    void* y;             // [M][rows]
    int M;
    int y_kind;          // 0 fp32, 1 fp16, 2 bf16
    void* workspace;
    size_t workspace_bytes;
};
bool gemm_tc_supported(const Layout& l, int M);
size_t gemm_ctrl_bytes(const Layout& l, int M);
size_t gemm_core_bytes(const Layout& l, int M);        // counters and the partial sums of K slices
size_t gemm_xt_bytes(const Layout& l, int M);          // the transposed copy of x of the sparse outlier product (0: not used)
size_t gemm_xt_offset(const Layout& l, int M);         // where that copy starts in the workspace
size_t gemm_workspace_bytes(const Layout& l, int M);   // all of it
cudaError_t launch_gemm_tc(const Layout& l, const GemmCall& c, cudaStream_t s);
// bf16 activations: converted to fp16 into a scratch area behind the GEMM's own workspace, then the same kernel
size_t gemm_x_scratch_bytes(const Layout& l, int M);
cudaError_t launch_x_to_f16(const void* x_bf16, void* x_f16, size_t elems, cudaStream_t s);

// Batches of 9..16 rows of x run on the tensor-core kernel (xfp_gemm_tc.cu) when the matrix is large and the blob
// sparse in outliers: the batched GEMV kernels decode once per 8 rows of x, the tcgen05 kernel decodes once for up to
// 128 rows (measurements at batch_prefers_gemm).
// Layout of a GEMV workspace, shared by every kernel that may be given it: counters (split-K tickets, one int per
// row-block and blob at most) in [0, align256(4 * RB * n)), zero-filled before first use and left zero-filled by every
// call; partial sums behind it, written before they are read.
// matrices with more tiles of 128 channels than SMs: batches of 9..16 rows of x may go to the tensor-core kernel
inline bool gemm_batch_shape(const Layout& l) { return (l.RB + 3) / 4 > kSizingSMs && gemm_tc_supported(l, 16); }

inline size_t workspace_bytes_for(const Layout& l) {
    size_t w = generic_workspace_bytes(l);
    const size_t p = l.mode ? v2a_workspace_bytes(l) : pair_workspace_bytes(l);
    if (p > w) w = p;
    // room for that kernel's partial sums and its transposed copy of x at 16 rows
    const size_t g = gemm_batch_shape(l) ? gemm_workspace_bytes(l, 16) : 0;
    return w > g ? w : g;
}

inline bool batch_prefers_gemm(const Layout& l, int batch) {
    // 28672 x 8192, us per call, tensor-core kernel against the batched kernels (0.3 % outliers unless noted):
    //   9..16 rows: V2 N = 4 74 against 124..148 (2 %: 107 against 146..174), V2a 102 against 210..246, N = 2 73
    //               against 110..133, N = 6 99 against 494..792
    //   5..8 rows:  V2a 102 against 123, V2 N = 6 98 against 115; V2 N = 4 73 against 74 (1 %: 87 against 80) and
    //               N = 2 72 against 67 stay on the batched lane kernel
    int least = ((l.mode || l.bits >= 5) && l.nnz * 100 <= (long long)l.rows * l.cols) ? 5 : 9;
#ifdef LANE_TUNE
    if (const char* e = getenv("XFP_GEMM_MIN")) least = atoi(e);
#endif
    if (batch < least || batch > 16 || !gemm_batch_shape(l)) return false;
    // at most 2.5 % outliers: the kernel adds them as a sparse product whose cost grows with their count
    return l.nnz * 40 <= (long long)l.rows * l.cols;
}

}  // namespace xfp
