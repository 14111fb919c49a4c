// extern "C" boundary of libxfp: host-side validation, layout computation, kernel selection.
#include <cstdlib>

#include "../../include/xfp.h"
#include "xfp_internal.h"

using namespace xfp;

namespace xfp {

int sm_count() {
    static std::atomic<int> cache[256] = {};
    const int dev = DeviceOnce::current();
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = kSizingSMs;   // no device to ask (host-only use of the library)
        }
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

}  // namespace xfp

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_desc(const xfp_desc* d) {
    if (!d) return XFP_ERR_NULL;
    if (d->mode != 0 && d->mode != 1) return XFP_ERR_SHAPE;
    if (d->rows <= 0 || d->cols <= 0) return XFP_ERR_SHAPE;
    if (d->bits < 2 || d->bits > 6) return XFP_ERR_SHAPE;
    if (d->group_size <= 0) return XFP_ERR_SHAPE;
    if (d->group_size != 64 && d->group_size != 128 && d->group_size != 256) return XFP_ERR_UNSUPPORTED;
    // the device layout walks K in super-chunks of 128 weights, whatever the group size
    if (d->cols % d->group_size || d->cols % 128) return XFP_ERR_SHAPE;
    if (d->cols > 65536) return XFP_ERR_UNSUPPORTED;
    if (d->mode == 1 && (d->lib_size < 1 || d->lib_size > 256)) return XFP_ERR_SHAPE;
    if (d->mode == 0 && d->lib_size != 0) return XFP_ERR_SHAPE;
    if (d->col_bits != 16 && d->col_bits != 32) return XFP_ERR_SHAPE;
    if (d->nnz < 0 || d->nnz >= (int64_t(1) << 31)) return XFP_ERR_SHAPE;
    if (d->nnz > (int64_t)d->rows * d->cols) return XFP_ERR_SHAPE;
    if ((int64_t)d->rows > (int64_t(1) << 24)) return XFP_ERR_UNSUPPORTED;
    return XFP_OK;
}

Layout layout_of(const xfp_desc* d) {
    return make_layout(d->mode, d->rows, d->cols, d->bits, d->lib_size, d->nnz, d->group_size);
}

int gemv_common(const xfp_desc* desc, int want_mode, const GemvCall& c, void* stream) {
    int st = check_desc(desc);
    if (st) return st;
    if (desc->mode != want_mode) return XFP_ERR_SHAPE;
    if (c.batch < 1 || c.batch > 16) return XFP_ERR_SHAPE;
    if (c.n == 1 && !c.packed_list) {
        if (!c.packed || !c.x || !c.y) return XFP_ERR_NULL;
        if (!aligned16(c.packed) || !aligned16(c.x) || !aligned16(c.y)) return XFP_ERR_ALIGN;
    } else {
        if (!c.packed_list || !c.x_list || !c.y_list) return XFP_ERR_NULL;
    }
    const Layout l = layout_of(desc);
    const size_t need = workspace_bytes_for(l);
    if (!c.workspace) return XFP_ERR_NULL;
    if (!aligned16(c.workspace)) return XFP_ERR_ALIGN;
    if (c.workspace_bytes < need) return XFP_ERR_BUFFER_TOO_SMALL;
    GemvCall cc = c;
    cc.workspace_bytes = need;
    cudaError_t e;
    if (c.epilogue != 0) {
        // fused epilogues exist in the V2a kernel only (batch 1)
        if (!v2a_supported(l, c.batch) || c.batch != 1) return XFP_ERR_UNSUPPORTED;
        e = launch_gemv_v2a(l, cc, (cudaStream_t)stream);
        return e == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
    }
    if (lane_supported(l, cc))
        e = launch_gemv_lane(l, cc, (cudaStream_t)stream);
    else if (lane_batch_supported(l, cc))
        e = launch_gemv_lane_batch(l, cc, (cudaStream_t)stream);
    else if (!c.packed_list && !c.x_bf16 && batch_prefers_gemm(l, c.batch)
#ifdef LANE_TUNE
             && !getenv("XFP_NO_GEMM")   // tuning build: keep batches off the tensor-core kernel
#endif
    ) {
        // many rows of x, few outliers: one decode for all rows on the tensor cores (y = x W^T with W the matrix
        // xfp_dequant writes; inside the GEMV's bound)
        GemmCall g{c.packed, c.x, c.y, c.batch, c.y_is_fp16, c.workspace, need};
        e = launch_gemm_tc(l, g, (cudaStream_t)stream);
    }
    else if (pair_supported(l, c.batch, c.n))
        e = launch_gemv_pair(l, cc, (cudaStream_t)stream);
    else if (!c.packed_list && batch_supported(l, c.batch))
        e = launch_gemv_batch(l, cc, (cudaStream_t)stream);
    else if (v2a_supported(l, c.batch))
        e = launch_gemv_v2a(l, cc, (cudaStream_t)stream);
    else
        e = launch_gemv_generic(l, cc, (cudaStream_t)stream);
    return e == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

// Device alias of a pinned, mapped host pointer; null for anything else (pageable memory, device memory).
const void* mapped_alias(const void* p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        cudaGetLastError();   // pageable memory may report an error on older runtimes: not ours to keep
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

// x from mapped host memory to its device staging buffer.  The host loads are issued before the dependency
// wait (x_host is not written by earlier kernels of the stream; the staging buffer may still be read by one).
__global__ void __launch_bounds__(256) host_in_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int n) {
    asm volatile("griddepcontrol.launch_dependents;");
    const int i = blockIdx.x * 1024 + threadIdx.x;
    uint4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (i + j * 256 < n) v[j] = src[i + j * 256];
    asm volatile("griddepcontrol.wait;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (i + j * 256 < n) dst[i + j * 256] = v[j];
}

cudaError_t launch_host_in(const void* src, void* dst, size_t bytes, cudaStream_t s) {
    const int n = (int)(bytes / 16);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((n + 1023) / 1024), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, host_in_kernel, (const uint4*)src, (uint4*)dst, n);
}

}  // namespace

extern "C" {

int xfp_packed_size(const xfp_desc* desc, size_t* packed_bytes, size_t* workspace_bytes) {
    int st = check_desc(desc);
    if (st) return st;
    const Layout l = layout_of(desc);
    if (packed_bytes) *packed_bytes = l.total;
    if (workspace_bytes) *workspace_bytes = workspace_bytes_for(l);
    return XFP_OK;
}

int xfp_pack(const xfp_desc* desc, const uint8_t* idx, const uint16_t* codebook, const uint8_t* group_id,
             const uint16_t* group_scale, const uint16_t* group_mid, const int32_t* out_rowptr, const void* out_col,
             const uint16_t* out_val, void* packed, size_t packed_bytes, int32_t* err_word, void* stream) {
    int st = check_desc(desc);
    if (st) return st;
    if (!idx || !codebook || !packed) return XFP_ERR_NULL;
    if (desc->mode == 1 && (!group_id || !group_scale || !group_mid)) return XFP_ERR_NULL;
    if (desc->nnz > 0 && (!out_rowptr || !out_col || !out_val)) return XFP_ERR_NULL;
    if (!aligned16(idx) || !aligned16(codebook) || !aligned16(packed)) return XFP_ERR_ALIGN;
    if (err_word && (reinterpret_cast<uintptr_t>(err_word) & 3u)) return XFP_ERR_ALIGN;
    const Layout l = layout_of(desc);
    if (packed_bytes < l.total) return XFP_ERR_BUFFER_TOO_SMALL;
    PackInputs in{idx, codebook, group_id, group_scale, group_mid, out_rowptr, out_col, desc->col_bits, out_val};
    return launch_pack(l, in, packed, err_word, (cudaStream_t)stream) == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_gemv_v2(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t batch, void* y,
                int32_t y_is_fp16, void* workspace, size_t workspace_bytes, void* stream) {
    GemvCall c{packed, x, y, nullptr, nullptr, nullptr, 1, batch, y_is_fp16 ? 1 : 0, workspace, workspace_bytes};
    return gemv_common(desc, 0, c, stream);
}

int xfp_gemv_v2a(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t batch, void* y,
                 int32_t y_is_fp16, void* workspace, size_t workspace_bytes, void* stream) {
    GemvCall c{packed, x, y, nullptr, nullptr, nullptr, 1, batch, y_is_fp16 ? 1 : 0, workspace, workspace_bytes};
    return gemv_common(desc, 1, c, stream);
}

int xfp_gemv_typed(const xfp_desc* desc, const void* packed, const void* x, int32_t x_type, int32_t batch, void* y,
                   int32_t y_type, void* workspace, size_t workspace_bytes, void* stream) {
    if (!desc) return XFP_ERR_NULL;
    if (x_type != XFP_T_F16 && x_type != XFP_T_BF16) return XFP_ERR_SHAPE;
    if (y_type != XFP_T_F32 && y_type != XFP_T_F16 && y_type != XFP_T_BF16) return XFP_ERR_SHAPE;
    GemvCall c{packed, (const uint16_t*)x, y, nullptr, nullptr, nullptr, 1, batch, y_type, workspace, workspace_bytes};
    c.x_bf16 = x_type == XFP_T_BF16;
    return gemv_common(desc, desc->mode, c, stream);
}

int xfp_gemv_grouped(const xfp_desc* desc, int32_t n, const void* const* packed, const uint16_t* const* x,
                     void* const* y, int32_t y_is_fp16, void* workspace, size_t workspace_bytes, void* stream) {
    if (!desc) return XFP_ERR_NULL;
    if (n < 1 || n > 65535) return XFP_ERR_SHAPE;
    if (!packed || !x || !y) return XFP_ERR_NULL;
    int st = check_desc(desc);
    if (st) return st;
    const Layout l = layout_of(desc);
    const size_t need = workspace_bytes_for(l);
    if (workspace_bytes < need * (size_t)n) return XFP_ERR_BUFFER_TOO_SMALL;
    GemvCall c{nullptr, nullptr, nullptr, packed, x, y, n, 1, y_is_fp16 ? 1 : 0, workspace, need};
    return gemv_common(desc, desc->mode, c, stream);
}

static int grouped_common(const xfp_desc* desc, int32_t n, const void* const* packed, const uint16_t* const* x,
                          int32_t x_bf16, void* const* y, int32_t y_type, int32_t epilogue, const float* weights,
                          void* workspace, size_t workspace_bytes, void* stream) {
    if (!desc) return XFP_ERR_NULL;
    if (n < 1 || n > 65535) return XFP_ERR_SHAPE;
    if (!packed || !x || !y) return XFP_ERR_NULL;
    if (epilogue != XFP_EPI_NONE && epilogue != XFP_EPI_SWIGLU && epilogue != XFP_EPI_COMBINE) return XFP_ERR_SHAPE;
    if (epilogue == XFP_EPI_COMBINE && !weights) return XFP_ERR_NULL;
    int st = check_desc(desc);
    if (st) return st;
    if (epilogue == XFP_EPI_SWIGLU && desc->rows % 64 != 0) return XFP_ERR_SHAPE;
    const Layout l = layout_of(desc);
    const size_t need = workspace_bytes_for(l);
    if (workspace_bytes < need * (size_t)n) return XFP_ERR_BUFFER_TOO_SMALL;
    GemvCall c{nullptr, nullptr, nullptr, packed, x, y, n, 1, y_type, workspace, need};
    c.epilogue = epilogue;
    c.epi_weights = weights;
    c.x_bf16 = x_bf16;
    return gemv_common(desc, desc->mode, c, stream);
}

int xfp_gemv_grouped_epilogue(const xfp_desc* desc, int32_t n, const void* const* packed, const uint16_t* const* x,
                              void* const* y, int32_t y_is_fp16, int32_t epilogue, const float* weights,
                              void* workspace, size_t workspace_bytes, void* stream) {
    return grouped_common(desc, n, packed, x, 0, y, y_is_fp16 ? 1 : 0, epilogue, weights, workspace, workspace_bytes, stream);
}

int xfp_gemv_grouped_typed(const xfp_desc* desc, int32_t n, const void* const* packed, const void* const* x,
                           int32_t x_type, void* const* y, int32_t y_type, int32_t epilogue, const float* weights,
                           void* workspace, size_t workspace_bytes, void* stream) {
    if (x_type != XFP_T_F16 && x_type != XFP_T_BF16) return XFP_ERR_SHAPE;
    if (y_type != XFP_T_F32 && y_type != XFP_T_F16 && y_type != XFP_T_BF16) return XFP_ERR_SHAPE;
    return grouped_common(desc, n, packed, (const uint16_t* const*)x, x_type == XFP_T_BF16, y, y_type, epilogue, weights,
                          workspace, workspace_bytes, stream);
}

int xfp_gemm_workspace_size(const xfp_desc* desc, int32_t m, size_t* workspace_bytes) {
    int st = check_desc(desc);
    if (st) return st;
    if (!workspace_bytes) return XFP_ERR_NULL;
    if (m < 1) return XFP_ERR_SHAPE;
    const Layout l = layout_of(desc);
    if (!gemm_tc_supported(l, m)) return XFP_ERR_UNSUPPORTED;
    *workspace_bytes = gemm_workspace_bytes(l, m);
    return XFP_OK;
}

int xfp_gemm(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t m, void* y, int32_t y_type,
             void* workspace, size_t workspace_bytes, void* stream) {
    int st = check_desc(desc);
    if (st) return st;
    if (m < 1 || y_type < 0 || y_type > 2) return XFP_ERR_SHAPE;
    if (!packed || !x || !y || !workspace) return XFP_ERR_NULL;
    if (!aligned16(packed) || !aligned16(x) || !aligned16(y) || !aligned16(workspace)) return XFP_ERR_ALIGN;
    const Layout l = layout_of(desc);
    if (!gemm_tc_supported(l, m)) return XFP_ERR_UNSUPPORTED;
    if (workspace_bytes < gemm_workspace_bytes(l, m)) return XFP_ERR_BUFFER_TOO_SMALL;
    GemmCall c{packed, x, y, m, y_type, workspace, workspace_bytes};
    return launch_gemm_tc(l, c, (cudaStream_t)stream) == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_gemm_typed_workspace_size(const xfp_desc* desc, int32_t m, int32_t x_type, size_t* workspace_bytes) {
    if (x_type != XFP_T_F16 && x_type != XFP_T_BF16) return XFP_ERR_SHAPE;
    int st = xfp_gemm_workspace_size(desc, m, workspace_bytes);
    if (st) return st;
    if (x_type == XFP_T_BF16) {
        const Layout l = layout_of(desc);
        *workspace_bytes = align256(*workspace_bytes) + gemm_x_scratch_bytes(l, m);
    }
    return XFP_OK;
}

int xfp_gemm_typed(const xfp_desc* desc, const void* packed, const void* x, int32_t x_type, int32_t m, void* y,
                   int32_t y_type, void* workspace, size_t workspace_bytes, void* stream) {
    if (x_type == XFP_T_F16) return xfp_gemm(desc, packed, (const uint16_t*)x, m, y, y_type, workspace, workspace_bytes, stream);
    if (x_type != XFP_T_BF16) return XFP_ERR_SHAPE;
    size_t need = 0;
    int st = xfp_gemm_typed_workspace_size(desc, m, x_type, &need);
    if (st) return st;
    if (!packed || !x || !y || !workspace) return XFP_ERR_NULL;
    if (!aligned16(x) || !aligned16(workspace)) return XFP_ERR_ALIGN;
    if (workspace_bytes < need) return XFP_ERR_BUFFER_TOO_SMALL;
    const Layout l = layout_of(desc);
    const size_t own = align256(gemm_workspace_bytes(l, m));
    uint16_t* x16 = (uint16_t*)((char*)workspace + own);
    if (launch_x_to_f16(x, x16, (size_t)m * l.cols, (cudaStream_t)stream) != cudaSuccess) return XFP_ERR_CUDA;
    return xfp_gemm(desc, packed, x16, m, y, y_type, workspace, own, stream);
}

int xfp_dequant(const xfp_desc* desc, const void* packed, uint16_t* W, void* stream) {
    int st = check_desc(desc);
    if (st) return st;
    if (!packed || !W) return XFP_ERR_NULL;
    if (!aligned16(packed) || !aligned16(W)) return XFP_ERR_ALIGN;
    return launch_dequant(layout_of(desc), packed, W, (cudaStream_t)stream) == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_gemv_host(const xfp_desc* desc, const void* packed, const uint16_t* x_host, uint16_t* x_dev, int32_t batch,
                  void* y_host, void* y_dev, int32_t y_is_fp16, void* workspace, size_t workspace_bytes,
                  void* stream) {
    int st = check_desc(desc);
    if (st) return st;
    if (!x_host || !x_dev || !y_host || !y_dev) return XFP_ERR_NULL;
    if (batch < 1 || batch > 16) return XFP_ERR_SHAPE;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t xbytes = (size_t)batch * desc->cols * 2, ybytes = (size_t)batch * desc->rows * (y_is_fp16 ? 2 : 4);
    // Pinned, device-mapped host buffers are used in place: a small kernel fetches x over the bus (its loads
    // overlap the tail of the previous kernel) and the GEMV stores y straight into host memory.  Two DMA
    // copies of a few KB cost more than the GEMV itself.  Pageable or unmapped buffers take the copies.
    const void* xmap = mapped_alias(x_host);
    void* ymap = (void*)mapped_alias(y_host);
    if (xmap && aligned16(xmap) && aligned16(x_dev) && xbytes % 16 == 0) {
        if (launch_host_in(xmap, x_dev, xbytes, s) != cudaSuccess) return XFP_ERR_CUDA;
    } else if (cudaMemcpyAsync(x_dev, x_host, xbytes, cudaMemcpyHostToDevice, s) != cudaSuccess) {
        return XFP_ERR_CUDA;
    }
    void* y = (ymap && aligned16(ymap)) ? ymap : y_dev;
    st = desc->mode ? xfp_gemv_v2a(desc, packed, x_dev, batch, y, y_is_fp16, workspace, workspace_bytes, stream)
                    : xfp_gemv_v2(desc, packed, x_dev, batch, y, y_is_fp16, workspace, workspace_bytes, stream);
    if (st) return st;
    if (y == y_dev && cudaMemcpyAsync(y_host, y_dev, ybytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return XFP_ERR_CUDA;
    return XFP_OK;
}

const char* xfp_status_str(int status) {
    switch (status) {
        case XFP_OK: return "ok";
        case XFP_ERR_NULL: return "null pointer";
        case XFP_ERR_ALIGN: return "pointer not 16-byte aligned";
        case XFP_ERR_SHAPE: return "shape or parameter outside the domain";
        case XFP_ERR_UNSUPPORTED: return "not supported by this build";
        case XFP_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case XFP_ERR_BAD_DATA: return "bad data";
        case XFP_ERR_CUDA: return "CUDA runtime error";
    }
    return "unknown status";
}

}  // extern "C"
