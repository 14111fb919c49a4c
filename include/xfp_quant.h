/*
 * xfp_quant.h -- C ABI of the B200 (sm_100a) XFP encoder: the stages of the paper's "Quantization"
 * section that turn a float matrix into the unpacked tensors xfp_pack (xfp.h) consumes.
 *
 *   Outlier Extraction                     xfp_quant_stats, xfp_quant_outliers
 *   Learned Codebook via Lloyd Iteration   xfp_quant_lloyd            (V2: one codebook per channel)
 *   V2a: Shared Codebook Library (LibFit)  xfp_quant_libfit_library, xfp_quant_libfit_assign
 *   residual S of Eq. 1                    xfp_quant_residual
 *   Algorithm 1 (cosine gate, auto-select) xfp_quant_cosine, xfp_quant_median, xfp_quantize
 *
 * Conventions are those of xfp.h: device pointers unless a parameter says "host", 16-byte aligned,
 * fp16 as uint16_t bit patterns, the status code is the only error channel, nothing is allocated.
 * Every stage queues its kernels on `stream` and returns without synchronising, except
 * xfp_quantize, which has to read one number per candidate bit width to take Algorithm 1's branch.
 *
 * Arithmetic.  Decisions that produce integers (which weights are extracted, where a Lloyd cell
 * ends, which codebook entry or library entry is nearest) are taken in IEEE fp64 on the fp32
 * weights, operation by operation in a fixed order, so a stage's integer and fp16 outputs are a
 * function of its inputs alone.  Only the two statistics (mu, sigma) and the cosines are sums
 * whose order is the kernel's own (fixed, but a tree): they are reproducible, and equal to a
 * serial fp64 evaluation to about 1e-13 relative.
 */
#ifndef XFP_QUANT_H
#define XFP_QUANT_H

#include "xfp.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int32_t sigma_mode;   /* 0: population standard deviation of the whole matrix (the paper's);
                             1: 1.4826 * median|w - mu| (for matrices whose tail inflates sigma)      */
    int32_t outlier_mode; /* 0: extract |w - mu| > k_sigma * sigma, at most floor(cap_frac * n), the
                                largest |w - mu| first (ties: lower flat index);
                             1: extract exactly the floor(rate * n) largest |w - mu|                  */
    double k_sigma;       /* paper default 4                                                          */
    double cap_frac;      /* paper default 0.02                                                       */
    double rate;          /* outlier_mode 1 only                                                      */
    int32_t lloyd_iters;  /* rounds of Lloyd (paper: 20; its V2 default elsewhere: 5)                 */
    int32_t group_size;   /* V2a: weights per (id, scale, mid) group: 64, 128 or 256; 0 means 128, the paper's
                             default (the paper leaves the size open)                                 */
} xfp_quant_params;

typedef struct {
    int32_t bits;      /* the bit width the tensors were produced with                                */
    int32_t fallback;  /* 1: no candidate reached tau, the largest candidate was kept                 */
    int32_t tried;     /* how many candidates were quantised                                          */
    int32_t reserved;
    int64_t nnz;       /* number of extracted weights = out_rowptr[rows]                              */
    double mu, sigma;  /* statistics of the matrix                                                    */
    double median_cos; /* median per-channel cosine of the returned quantisation                      */
} xfp_quant_result;

/* Bytes of scratch the calls below need for a rows x cols matrix (host call). */
int xfp_quant_workspace_size(int32_t rows, int32_t cols, size_t* bytes);

/* "Outlier Extraction": mu_sigma[0] = mean, mu_sigma[1] = sigma of the n = rows*cols weights. */
int xfp_quant_stats(const float* W, int64_t n, int32_t sigma_mode, double* mu_sigma, void* workspace,
                    size_t workspace_bytes, void* stream);

/* "Outlier Extraction": mask[t] = 1 where weight t is extracted, else 0; *count = how many.
 * outlier_mode 0: k_or_rate = k (threshold k * mu_sigma[1]) with the cap cap_frac; mode 1: k_or_rate = rate. */
int xfp_quant_outliers(const float* W, int64_t n, const double* mu_sigma, int32_t outlier_mode, double k_or_rate,
                       double cap_frac, uint8_t* mask, int64_t* count, void* workspace, size_t workspace_bytes,
                       void* stream);

/* "Learned Codebook via Lloyd Iteration", one channel per thread block: the bulk values of the channel
 * (extracted positions hold mu) are sorted; 2^bits entries start at the (j + 1/2) / 2^bits quantiles;
 * `iters` rounds of nearest-entry cells (a tie goes to the lower entry) and cell means (an empty cell
 * keeps its entry), stopping early when nothing moves; the entries are rounded to fp16 and every
 * weight is re-assigned to its nearest STORED entry.  mask may be NULL (nothing extracted).
 *   codebook [rows][2^bits] fp16, idx [rows][cols] one index per byte.
 * Channels of up to 16384 weights are sorted in shared memory and need no workspace (NULL is accepted); longer
 * ones (up to the format's 65536) use the workspace of xfp_quant_workspace_size for their arrays. */
int xfp_quant_lloyd(const float* W, const uint8_t* mask, const double* mu_sigma, int32_t rows, int32_t cols,
                    int32_t bits, int32_t iters, uint16_t* codebook, uint8_t* idx, void* workspace,
                    size_t workspace_bytes, void* stream);

/* LibFit, first half: a second Lloyd pass over the per-channel codebooks.  Each codebook is normalised to
 * (c - m) / s, m and s the middle and half-width of its range; k-means with L centroids, started from L
 * evenly spaced channels after ordering by squared norm, `iters` rounds; lib [L][2^bits] fp16, each
 * entry ascending. */
int xfp_quant_libfit_library(const uint16_t* codebook, int32_t rows, int32_t bits, int32_t L, int32_t iters,
                             uint16_t* lib, void* workspace, size_t workspace_bytes, void* stream);

/* LibFit, second half: every group of group_size (64, 128 or 256) consecutive weights of a channel gets
 * mid = fp16((max+min)/2), scale = fp16((max-min)/2) of its bulk values, the library entry with the least squared
 * error under nearest-value assignment (ties: lower entry) and the indices of the nearest decoded values.
 *   idx [rows][cols], gid / gscale / gmid [rows][cols/group_size]; cols a multiple of group_size. */
int xfp_quant_libfit_assign(const float* W, const uint8_t* mask, const double* mu_sigma, int32_t rows, int32_t cols,
                            int32_t bits, int32_t L, int32_t group_size, const uint16_t* lib, uint8_t* idx, uint8_t* gid,
                            uint16_t* gscale, uint16_t* gmid, void* stream);

/* The residual of Eq. 1 at the extracted positions, S = fp16(w - D16), as CSR with int32 columns.
 * desc gives mode, rows, cols, bits, group_size, lib_size (nnz is ignored); codebook is the V2 table or the
 * V2a library; gid/gscale/gmid are NULL for V2.  out_col/out_val hold `capacity` entries: entries beyond
 * it are dropped, out_rowptr always holds the true counts, so out_rowptr[rows] > capacity tells the
 * caller to retry with larger buffers. */
int xfp_quant_residual(const xfp_desc* desc, const float* W, const uint8_t* mask, const uint8_t* idx,
                       const uint16_t* codebook, const uint8_t* gid, const uint16_t* gscale, const uint16_t* gmid,
                       int32_t* out_rowptr, int32_t* out_col, uint16_t* out_val, int64_t capacity, void* workspace,
                       size_t workspace_bytes, void* stream);

/* Algorithm 1's gate: cos[i] = <W_i, W^_i> / (|W_i| |W^_i|) in fp64, W^ = fp16(D16 + S) the
 * reconstruction xfp_dequant would give (a zero row gives 1).  cos [rows] doubles. */
int xfp_quant_cosine(const xfp_desc* desc, const float* W, const uint8_t* mask, const uint8_t* idx,
                     const uint16_t* codebook, const uint8_t* gid, const uint16_t* gscale, const uint16_t* gmid,
                     double* cos, void* stream);

/* Median of n doubles (even n: mean of the two middle values); *median on the device. */
int xfp_quant_median(const double* v, int64_t n, double* median, void* workspace, size_t workspace_bytes,
                     void* stream);

/* Algorithm 1, two-threshold auto-select: extract the outliers once, then for each candidate bit width
 * in ascending order quantise (mode 0: xfp_quant_lloyd; mode 1: Lloyd, LibFit library, LibFit assign),
 * take the residual and the median per-channel cosine, and stop at the first candidate whose median
 * reaches tau; if none does the largest candidate stays (result->fallback = 1).
 *   candidates  host array, ascending, each in 2..6
 *   codebook    [rows][2^max candidate] fp16: the V2 codebooks (for V2a: scratch for the per-channel books)
 *   lib, gid, gscale, gmid   V2a outputs (lib [lib_size][2^bits]); NULL for V2
 *   cos         [rows] doubles, left holding the cosines of the returned quantisation
 *   result      host
 * SYNCHRONISES `stream` once per candidate.  The outputs are ready for xfp_pack with col_bits = 32. */
int xfp_quantize(int32_t mode, const float* W, int32_t rows, int32_t cols, const xfp_quant_params* params,
                 const int32_t* candidates, int32_t n_candidates, double tau, int32_t lib_size, uint8_t* mask,
                 uint8_t* idx, uint16_t* codebook, uint16_t* lib, uint8_t* gid, uint16_t* gscale, uint16_t* gmid,
                 int32_t* out_rowptr, int32_t* out_col, uint16_t* out_val, int64_t capacity, double* cos,
                 xfp_quant_result* result, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* XFP_QUANT_H */
