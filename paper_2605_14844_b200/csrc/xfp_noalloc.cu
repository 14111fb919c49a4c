// xfp_gemv_v2_noalloc: the V2 fused GEMV for callers that must not allocate device memory.
//
// The regular entry point, xfp_gemv_v2, needs a workspace from the caller (split-K partial sums and
// their counters).  Some callers have no way to provide one: a plug-in running inside a host
// application that claimed all device memory at start-up and hands out none, or a component on a
// latency-critical path where cudaMalloc, which synchronises the whole device, is off limits.  For
// them this file keeps the workspace in a fixed array that is part of the library image.
//
// The array costs kNoAllocScratchBytes of memory on every GPU that loads the library, for the life
// of the process, whether the entry point is used or not -- hence the modest size and the shape
// limit that follows from it.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/xfp.h"

namespace {

constexpr size_t kNoAllocScratchBytes = size_t(8) << 20;  // 8 MiB
constexpr int kMaxDevices = 64;

// File-scope device array.  In host code this name is only a handle for the runtime, never a
// device address: the address a kernel may use comes from cudaGetSymbolAddress (below).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

std::mutex g_setup_lock;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the current device; looked up once per device.
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return XFP_ERR_CUDA;
    std::lock_guard<std::mutex> hold(g_setup_lock);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return XFP_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return XFP_OK;
}

}  // namespace

extern "C" int xfp_gemv_v2_noalloc(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t batch,
                                   void* y, int32_t y_is_fp16, void* stream) {
    size_t packed_bytes = 0, need = 0;
    const int st = xfp_packed_size(desc, &packed_bytes, &need);  // validates the descriptor as well
    if (st != XFP_OK) return st;
    if (need > kNoAllocScratchBytes) return XFP_ERR_BUFFER_TOO_SMALL;  // shape too large for the built-in array
    void* scratch = nullptr;
    const int ss = scratch_for_current_device(&scratch);
    if (ss != XFP_OK) return ss;
    // The array keeps whatever the previous call left.  Partial sums are always written before they are
    // read, but the split-K counters must start at zero: clear them on the caller's stream.
    const size_t counters = (((size_t)(desc->rows + 31) / 32) * 4 + 255) & ~size_t(255);
    if (cudaMemsetAsync(scratch, 0, counters < need ? counters : need, (cudaStream_t)stream) != cudaSuccess)
        return XFP_ERR_CUDA;
    return xfp_gemv_v2(desc, packed, x, batch, y, y_is_fp16, scratch, kNoAllocScratchBytes, stream);
}
