/*
 * xfp.h -- C ABI of the B200 (sm_100a) XFP decode library.
 *
 * XFP stores a weight matrix W [rows = output channels][cols = input features K] as
 *     W  ~=  S + Codebook[Q]                                   (paper Eq. 1, "Decomposition")
 * Q: dense N-bit indices (N in 2..6, "Sub-Byte Packing"); S: sparse fp16 outlier residual.
 * Two codebook storage modes ("The XFP Format"):
 *   V2  : one fp16 codebook of 2^N entries per output channel:  D_ik = codebook_i[q_ik]
 *   V2a : a per-layer library of L codebooks; every group of G consecutive k of one channel (G = 128 in the
 *         paper, which leaves the size open: 64, 128 and 256 are built) carries a library id, an fp16 scale and an
 *         fp16 mid-point ("V2a: Shared Codebook Library"):  D_ik = mid_ig + scale_ig * lib[id_ig][q_ik],  g = k / G
 * The hot path is the fused decode kernel y = (D + S) x of "Fused Decode Kernel": depack, codebook
 * gather, outlier add and multiply-accumulate in one launch, fp32 accumulation.
 *
 * Conventions
 *  - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller and
 *    16-byte aligned.  fp16 values travel as uint16_t bit patterns.
 *  - The library allocates no memory, creates no streams and never synchronises; work is queued
 *    on `stream` (a cudaStream_t passed as void*, NULL = the legacy default stream).
 *  - The return value (xfp_status) is the only error channel.  Problems the host can see (NULL or
 *    misaligned pointers, unsupported shapes, small buffers, mode mismatch) are rejected before any
 *    launch.  Problems in the data are found by xfp_pack on the device and reported through
 *    err_word; GEMV and dequant trust a packed blob (xfp_pack clamps bad values so that a blob
 *    packed from bad data is still safe to read).
 *  - `packed` is opaque, position independent (may be copied with cudaMemcpy) and fully
 *    determined by the descriptor; keep the descriptor with it.
 *  - Thread safety: calls from several host threads are safe as long as they do not share a workspace
 *    (or the built-in scratch of xfp_gemv_v2_noalloc); the library keeps no mutable state besides
 *    per-device caches that are filled once.
 *  - Stream capture: the first call of an entry point that launches kernels (gemv, gemm, dequant, pack and
 *    their variants) on each device sets kernel attributes and asks the device for its properties.  Make one
 *    call per kernel variant you will use (same mode, bits and batch class) on each device BEFORE you begin a
 *    stream capture; later calls with those variants only launch.
 *  - Programmatic dependent launch: the GEMV kernels start before the previous kernel of the stream has
 *    finished and read the packed blob -- and, for the grouped calls, the device pointer lists and the
 *    routing weights -- BEFORE they wait for it; x, y and the workspace are touched only after the wait.
 *    Blobs, pointer lists and routing weights must therefore be complete when the call is made: do not
 *    produce them with a kernel that itself releases its dependents early (a plain kernel, a copy or a memset
 *    on the same stream is fine).
 */
#ifndef XFP_H
#define XFP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    XFP_OK = 0,
    XFP_ERR_NULL = 1,             /* a required pointer is NULL                         */
    XFP_ERR_ALIGN = 2,            /* a pointer is not 16-byte aligned                   */
    XFP_ERR_SHAPE = 3,            /* rows/cols/bits/group/lib/batch outside the domain  */
    XFP_ERR_UNSUPPORTED = 4,      /* valid in the format, not built (e.g. cols > 65536) */
    XFP_ERR_BUFFER_TOO_SMALL = 5, /* packed_bytes / workspace_bytes too small           */
    XFP_ERR_BAD_DATA = 6,         /* reserved for callers that decode err_word          */
    XFP_ERR_CUDA = 7              /* a CUDA runtime call failed (launch, copy)          */
} xfp_status;

/* bits of *err_word written by xfp_pack (0 = the data were clean) */
#define XFP_BAD_INDEX 1u    /* an index >= 2^bits                                  */
#define XFP_BAD_GROUP_ID 2u /* a V2a group id >= lib_size                          */
#define XFP_BAD_ROWPTR 4u   /* rowptr not monotone, rowptr[0] != 0 or rowptr[rows] != nnz */
#define XFP_BAD_COLUMN 8u   /* an outlier column >= cols                           */
#define XFP_BAD_ORDER 16u   /* outlier columns of a row not strictly ascending     */

typedef struct {
    int32_t mode;       /* 0 = V2 (per-channel codebook), 1 = V2a (library + per-group id)          */
    int32_t rows, cols; /* output channels; input features K, a multiple of group_size and of 128, <= 65536 */
    int32_t bits;       /* N in {2,3,4,5,6}, both modes (the paper's own V2a kernel: {2,4} only)    */
    int32_t group_size; /* 64, 128 or 256 (others: XFP_ERR_UNSUPPORTED).  V2a: weights per (id, scale, mid);
                           V2 has no per-group data and only the divisibility of cols is checked.  Groups of
                           64 run on the general kernels (GEMV, dequant, GEMM), not on the fast V2a GEMV paths */
    int32_t lib_size;   /* V2a: L in 1..256 (paper default 32); V2: 0                               */
    int32_t col_bits;   /* width of the CSR column indices handed to xfp_pack: 16 or 32             */
    int64_t nnz;        /* number of outliers, 0 <= nnz < 2^31                                      */
} xfp_desc;

/* Size of the packed blob and of the GEMV workspace for this descriptor (host call, no GPU work).
 * The workspace holds split-K partial sums and counters; it must be zero-filled once before its
 * first use and is left zero-filled in its counter part by every call.  One workspace serves any
 * batch and either GEMV entry point for this shape, but not two calls that overlap in time. */
int xfp_packed_size(const xfp_desc* desc, size_t* packed_bytes, size_t* workspace_bytes);

/* Re-tile the unpacked tensors (the last stage of the encoder, "Sub-Byte Packing") into the
 * device layout read by the decode kernels, validating value ranges on the device.
 *   idx        [rows][cols] one index per byte
 *   codebook   V2: [rows][2^bits] fp16;  V2a: [lib_size][2^bits] fp16
 *   group_id   V2a: [rows][cols/group_size] u8;  V2: NULL
 *   group_scale, group_mid   V2a: [rows][cols/group_size] fp16;  V2: NULL
 *   out_rowptr [rows+1] int32, monotone, out_rowptr[rows] == nnz   (may be NULL when nnz == 0)
 *   out_col    [nnz] uint16 or int32 (desc->col_bits), strictly ascending inside a row
 *   out_val    [nnz] fp16
 *   packed     receives packed_bytes (>= xfp_packed_size) bytes
 *   err_word   optional int32 on the device: OR of XFP_BAD_* bits; the caller zeroes it before the
 *              call and reads it after its own synchronisation */
int xfp_pack(const xfp_desc* desc, const uint8_t* idx, const uint16_t* codebook, const uint8_t* group_id,
             const uint16_t* group_scale, const uint16_t* group_mid, const int32_t* out_rowptr,
             const void* out_col, const uint16_t* out_val, void* packed, size_t packed_bytes,
             int32_t* err_word, void* stream);

/* Fused decode GEMV for a V2 blob ("Fused Decode Kernel"):  y[b][i] = sum_k (D_ik + S_ik) x[b][k].
 *   x  [batch][cols] fp16, batch in 1..16
 *   y  [batch][rows] fp32, or fp16 (round to nearest even of the fp32 sum) when y_is_fp16 != 0
 * Products are exact in fp32 and accumulated in fp32; the summation order is fixed, so repeated
 * calls give identical bits.  workspace/workspace_bytes as returned by xfp_packed_size.
 * Which kernel serves a call depends on shape, bit width, batch and outlier count only (never on the data): batch 1
 * runs on a kernel with one channel per lane, 2..8 rows of x on kernels that decode once per 8 rows, and from 9
 * rows (5 for V2a and for N >= 5) a large blob with at most 2.5 % outliers may run on the tensor-core kernel of
 * xfp_gemm (D16 on the tensor cores, S as a sparse product, both accumulated in fp32); every kernel lies inside the
 * bound the tests hold them to
 * (|y - y_ref| <= 1e-3 * sum_k |W_ik x_k|). */
int xfp_gemv_v2(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t batch, void* y,
                int32_t y_is_fp16, void* workspace, size_t workspace_bytes, void* stream);

/* Same for a V2a blob ("V2a: Shared Codebook Library"). */
int xfp_gemv_v2a(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t batch, void* y,
                 int32_t y_is_fp16, void* workspace, size_t workspace_bytes, void* stream);

/* The fused GEMV of desc->mode with bf16 activations and/or outputs (bf16 is the paper's native activation
 * type; its kernel "outputs bf16 natively").
 *   x  [batch][cols] of x_type: XFP_T_F16, or XFP_T_BF16 -- converted to fp16 while the kernel stages it
 *      (round to nearest even, clamped to +-65504; a bf16 value with 2^-14 <= |x| <= 65504 converts
 *      exactly, smaller ones land on the fp16 subnormal grid, absolute error <= 2^-25)
 *   y  [batch][rows] of y_type: XFP_T_F32, XFP_T_F16 or XFP_T_BF16 (one rounding of the fp32 sum)
 * Everything else as xfp_gemv_v2 / xfp_gemv_v2a. */
#define XFP_T_F32 0
#define XFP_T_F16 1
#define XFP_T_BF16 2
int xfp_gemv_typed(const xfp_desc* desc, const void* packed, const void* x, int32_t x_type, int32_t batch, void* y,
                   int32_t y_type, void* workspace, size_t workspace_bytes, void* stream);

/* Materialise W^ = fp16(D16 + S) as fp16 [rows][cols] ("Reconstruct" in Algorithm 1; Eq. 1).
 * D16 is the fp16 value the index decodes to: the codebook entry (V2), or
 * fp16(fp32(scale * lib + mid)) (V2a, one fp32 rounding then one fp16 rounding).  The sum with an
 * outlier is rounded once.  Bit-exact and unique. */
int xfp_dequant(const xfp_desc* desc, const void* packed, uint16_t* W, void* stream);

/* n independent GEMVs of one shape in one launch (the active experts of a routed-MoE layer,
 * "MoE-native" dispatch): packed[j], x[j] ([cols] fp16, batch 1), y[j] ([rows]) are DEVICE arrays of
 * n device pointers.  All blobs share `desc` (same mode, shape, bits, lib_size; nnz is the largest
 * of the group and sizes nothing at run time).  The workspace must hold n * workspace_bytes. */
int xfp_gemv_grouped(const xfp_desc* desc, int32_t n, const void* const* packed, const uint16_t* const* x,
                     void* const* y, int32_t y_is_fp16, void* workspace, size_t workspace_bytes, void* stream);

/* xfp_gemv_grouped with the element-wise step that follows it in a routed expert's feed-forward block fused
 * into the store, so that one token-layer is two launches ("MoE-native" dispatch; the paper blames the
 * launch count of the unfused expert path for its power plateau).  V2a blobs the fast kernel supports
 * (bits 2..5), batch 1; anything else returns XFP_ERR_UNSUPPORTED.
 *   XFP_EPI_NONE     y[j][rows] as xfp_gemv_grouped.
 *   XFP_EPI_SWIGLU   the blob is a gate_up projection whose channels were ordered, before quantisation, in
 *                    blocks of 64: 32 gate channels followed by the 32 matching up channels.  y[j] receives
 *                    rows/2 values h = SiLU(gate) * up, SiLU(g) = g / (1 + exp(-g)), evaluated in fp32 on
 *                    the fp32 sums.  rows must be a multiple of 64.
 *   XFP_EPI_COMBINE  y[0][rows] = sum_j weights[j] * (W_j x[j]) added in blob order in fp32 (the routing
 *                    weights of the token, `weights` [n] floats on the device); y[1..] are not used. */
#define XFP_EPI_NONE 0
#define XFP_EPI_SWIGLU 1
#define XFP_EPI_COMBINE 2
int xfp_gemv_grouped_epilogue(const xfp_desc* desc, int32_t n, const void* const* packed, const uint16_t* const* x,
                              void* const* y, int32_t y_is_fp16, int32_t epilogue, const float* weights,
                              void* workspace, size_t workspace_bytes, void* stream);

/* The grouped launch with typed activations and outputs (x_type, y_type as for xfp_gemv_typed) and an optional fused
 * store (epilogue, weights as for xfp_gemv_grouped_epilogue; XFP_EPI_NONE for none): a routed expert block of a
 * bf16 model in two launches.  Fused stores and grouped V2 blobs run on the kernels that carry typed IO; the same
 * restrictions as xfp_gemv_grouped_epilogue apply when epilogue != XFP_EPI_NONE. */
int xfp_gemv_grouped_typed(const xfp_desc* desc, int32_t n, const void* const* packed, const void* const* x,
                           int32_t x_type, void* const* y, int32_t y_type, int32_t epilogue, const float* weights,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Prefill form of the fused kernel ("Fused Decode Kernel": depack, codebook gather, outlier scatter-add into the
 * dequantised tile, GEMM on the tensor cores; the paper's split-M path for many rows of x):
 *     y[t][i] = sum_k W^[i][k] * x[t][k],   W^ = fp16(D16 + S), the matrix xfp_dequant writes,
 * for m >= 1 rows of x in one launch on the tcgen05 tensor cores (fp16 x fp16 products, fp32 accumulation in tensor
 * memory, one rounding of the sum to y_type).  Up to 64 rows of x the outliers are not added to the decoded tile:
 * the tensor cores multiply D16 and the kernel adds sum_k S_ik x[t][k] to the accumulator in fp32, entries in
 * ascending column order (y = (D16 + S) x without the fp16 rounding of the sum, as in xfp_gemv; the activations of
 * that sparse product come from a transposed copy of x which a small kernel writes into the workspace first).
 * V2 blobs, every N; V2a blobs whose library, replicated once per
 * shared-memory bank, fits 128 KB (lib_size * 2^bits <= 1024: L = 32 up to N = 5), else XFP_ERR_UNSUPPORTED.
 *   x  [m][cols] fp16;  y  [m][rows] of y_type (XFP_T_F32, XFP_T_F16 or XFP_T_BF16)
 *   workspace  xfp_gemm_workspace_size(desc, m) bytes, zero-filled once before first use; its counter part is left
 *              zero-filled by every call.  Its first 32-bit word is an error flag: the kernel sets it to 1 if one of
 *              its bounded waits ran out (y is then not written); the caller may read it after synchronising.
 *              The library never clears the flag, and a call that set it may leave tile counters behind: a
 *              workspace whose flag reads 1 must be zero-filled again before it is reused.
 * Results are deterministic (K slices, when the matrix has few rows, are added in slice order). */
int xfp_gemm_workspace_size(const xfp_desc* desc, int32_t m, size_t* workspace_bytes);
int xfp_gemm(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t m, void* y, int32_t y_type,
             void* workspace, size_t workspace_bytes, void* stream);

/* xfp_gemm with typed activations: x_type XFP_T_F16 (the call above) or XFP_T_BF16, the paper's native type.  bf16
 * rows of x are first converted to fp16 (round to nearest even, clamped to +-65504: exact for 2^-14 <= |x| <= 65504)
 * by a small kernel into a scratch area behind the GEMM's own workspace, then multiplied by the same kernel.
 *   workspace  xfp_gemm_typed_workspace_size(desc, m, x_type) bytes, zero-filled once before first use. */
int xfp_gemm_typed_workspace_size(const xfp_desc* desc, int32_t m, int32_t x_type, size_t* workspace_bytes);
int xfp_gemm_typed(const xfp_desc* desc, const void* packed, const void* x, int32_t x_type, int32_t m, void* y,
                   int32_t y_type, void* workspace, size_t workspace_bytes, void* stream);

/* Convenience for callers whose activations live in host memory: brings x_host to x_dev, runs the GEMV for
 * desc->mode and delivers y in y_host, all on `stream` (the host sees y once the stream reached this point).
 * x_dev [batch][cols] fp16 and y_dev [batch][rows] are device staging buffers of the caller.  Pinned,
 * device-mapped host buffers (cudaHostAlloc / cudaHostRegister under unified addressing) are used in
 * place: a small kernel reads x_host and the GEMV stores into y_host directly (y_dev is then not
 * touched); other host memory goes through cudaMemcpyAsync in both directions. */
int xfp_gemv_host(const xfp_desc* desc, const void* packed, const uint16_t* x_host, uint16_t* x_dev,
                  int32_t batch, void* y_host, void* y_dev, int32_t y_is_fp16, void* workspace,
                  size_t workspace_bytes, void* stream);

/* xfp_gemv_v2 for callers that cannot allocate device memory.  The paper has no counterpart: this is a
 * packaging variant of the same GEMV, not another operation.
 * Who needs it: code that is handed a fixed set of buffers and may not ask the driver for more -- for
 * instance a plug-in inside a host application that reserved the whole GPU at start-up, or a component
 * on a latency-critical path where cudaMalloc (which synchronises the device) is forbidden.  Such a
 * caller cannot supply the split-K workspace xfp_gemv_v2 asks for, so the library keeps one in a
 * built-in device array of 8 MiB (present on every GPU that loads the library, until the process exits).
 *   desc, packed, x, batch, y, y_is_fp16, stream: as for xfp_gemv_v2; the caller still owns inputs and outputs.
 * Limits and behaviour:
 *   - shapes whose workspace (see xfp_packed_size) exceeds 8 MiB return XFP_ERR_BUFFER_TOO_SMALL;
 *     roughly: (rows / 32) * min(64, cols / 128) <= 32k, e.g. anything up to 8192 x 8192.
 *   - the first call on each device looks up the array's device address (once per device, with that
 *     device current); make that first call before starting any stream capture.
 *   - no cudaMalloc, cudaFree or other allocating call is made; the only extra work is a small
 *     cudaMemsetAsync on `stream` that zeroes the workspace counters, because the array keeps the
 *     previous call's contents.
 *   - all calls share the one array: two calls that may run at the same time on the GPU (different
 *     streams, or different host threads without ordering) race on it and give wrong results.  Order
 *     them on one stream, or use xfp_gemv_v2 with separate workspaces. */
int xfp_gemv_v2_noalloc(const xfp_desc* desc, const void* packed, const uint16_t* x, int32_t batch, void* y,
                        int32_t y_is_fp16, void* stream);

const char* xfp_status_str(int status);

#ifdef __cplusplus
}
#endif
#endif /* XFP_H */
