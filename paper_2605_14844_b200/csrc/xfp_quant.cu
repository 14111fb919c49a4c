// The XFP encoder on the GPU ("Quantization": Outlier Extraction, Learned Codebook via Lloyd Iteration,
// V2a LibFit, the residual of Eq. 1, Algorithm 1's cosine gate and auto-select).
//
// Every decision that yields an integer or an fp16 value is taken in IEEE fp64 with explicit
// round-to-nearest intrinsics (no fused multiply-add), in the order the method states: a Lloyd cell
// boundary is the midpoint of two entries, a cell mean is a difference of two SERIAL prefix sums over
// the sorted channel divided by the count, a nearest entry is found by a linear scan with a strict
// "less than", a group's squared error is summed value by value.  The serial parts are short (one
// channel, one group) and the parallelism is across channels, groups and library entries.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "../../include/xfp_quant.h"
#include "xfp_internal.h"   // sm_count()

namespace xq {

constexpr int kRedBlocks = 1024;   // partial sums of a whole-matrix reduction
constexpr int kRedThreads = 256;
constexpr int kTieChunk = 4096;    // elements per block in the ordered tie pass (256 threads x 16)
constexpr int kTiePer = 16;

__device__ __forceinline__ double h2d(uint16_t h) { return (double)__half2float(__ushort_as_half(h)); }
__device__ __forceinline__ uint16_t d2h(double d) { return __half_as_ushort(__double2half(d)); }

// D16 of a V2a weight: one fp32 rounding of scale*lib + mid (the product of two fp16 is exact in fp32),
// then one fp16 rounding ("V2a: Shared Codebook Library").
__device__ __forceinline__ uint16_t v2a_value16(uint16_t scale, uint16_t lib, uint16_t mid) {
    const float r = __fmaf_rn(__half2float(__ushort_as_half(scale)), __half2float(__ushort_as_half(lib)),
                              __half2float(__ushort_as_half(mid)));
    return __half_as_ushort(__float2half_rn(r));
}

// Index of the entry nearest to x among e[0..E), ties to the lower index: the answer of a linear scan that keeps an
// entry only when it is strictly nearer.  When the entries ascend (codebooks and decoded library entries do) x is
// bracketed by bisection and only its two neighbours are measured; the scan's answer is the nearer of the two
// (the lower on an exact tie: fp64 rounding is monotone and distinct fp16 values are too far apart to round to
// the same distance), moved down over duplicates of its value.
__device__ __forceinline__ int nearest_entry(const double* e, int E, double x, bool ascending) {
    if (!ascending) {
        int best = 0;
        double bd = fabs(__dsub_rn(x, e[0]));
        for (int j = 1; j < E; ++j) {
            const double d = fabs(__dsub_rn(x, e[j]));
            if (d < bd) { bd = d; best = j; }
        }
        return best;
    }
    int lo = 0, hi = E;   // first index whose entry is >= x
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (e[mid] < x) lo = mid + 1; else hi = mid;
    }
    int best;
    if (lo == 0) best = 0;
    else if (lo == E) best = E - 1;
    else best = fabs(__dsub_rn(x, e[lo - 1])) <= fabs(__dsub_rn(x, e[lo])) ? lo - 1 : lo;
    while (best > 0 && e[best - 1] == e[best]) --best;
    return best;
}

// Sum over the block in a fixed tree order; every thread gets the result.
__device__ double block_sum(double v, double* sh) {
    sh[threadIdx.x] = v;
    __syncthreads();
    for (int s = blockDim.x >> 1; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) sh[threadIdx.x] = __dadd_rn(sh[threadIdx.x], sh[threadIdx.x + s]);
        __syncthreads();
    }
    const double r = sh[0];
    __syncthreads();
    return r;
}

// Exclusive scan of one int per thread over the block (blockDim.x <= 1024, a multiple of 32); returns
// the thread's offset and leaves the block total in *total.
__device__ int block_excl_scan(int v, int* sh_warp, int* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += t;
    }
    if (lane == 31) sh_warp[w] = inc;
    __syncthreads();
    if (w == 0) {
        int x = lane < nw ? sh_warp[lane] : 0;
        int xi = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, xi, d);
            if (lane >= d) xi += t;
        }
        if (lane < nw) sh_warp[lane] = xi - x;
        if (lane == 31) *total = xi;
    }
    __syncthreads();
    const int r = sh_warp[w] + inc - v;
    __syncthreads();
    return r;
}

// ------------------------------------------------------------------ statistics

// PASS 0: sum of w.  PASS 1: sum of (w - mu)^2.
template <int PASS>
__global__ void __launch_bounds__(kRedThreads) stats_partial(const float* __restrict__ W, int64_t n,
                                                              const double* __restrict__ ms, double* part) {
    __shared__ double sh[kRedThreads];
    const int64_t per = (n + gridDim.x - 1) / gridDim.x;
    const int64_t b0 = (int64_t)blockIdx.x * per;
    const int64_t b1 = b0 + per < n ? b0 + per : n;
    const double mu = PASS ? ms[0] : 0.0;
    double acc = 0.0;
    for (int64_t t = b0 + threadIdx.x; t < b1; t += kRedThreads) {
        const double w = (double)W[t];
        if (PASS) {
            const double d = __dsub_rn(w, mu);
            acc = __dadd_rn(acc, __dmul_rn(d, d));
        } else {
            acc = __dadd_rn(acc, w);
        }
    }
    const double r = block_sum(acc, sh);
    if (threadIdx.x == 0) part[blockIdx.x] = r;
}

template <int PASS>
__global__ void __launch_bounds__(kRedThreads) stats_final(const double* part, int64_t n, double* ms) {
    __shared__ double sh[kRedThreads];
    double acc = 0.0;
    for (int t = threadIdx.x; t < kRedBlocks; t += kRedThreads) acc = __dadd_rn(acc, part[t]);
    const double r = block_sum(acc, sh);
    if (threadIdx.x == 0) {
        if (PASS == 0) ms[0] = __ddiv_rn(r, (double)n);
        else ms[1] = __dsqrt_rn(__ddiv_rn(r, (double)n));
    }
}

// ------------------------------------------------------------------ exact selection by radix descent

// State of one selection: after eight 8-bit passes `prefix` is the key of the wanted element and `k`
// its rank among the elements with that key (in scan direction).
struct SelState {
    unsigned long long prefix;
    long long k;
    long long count;   // candidates (threshold mode: weights above the threshold)
    long long keep;    // entries to keep
    int shift;
    int descending;
    int skip;          // 1: nothing to select (all candidates are kept, or none)
    int pad;
    double value[2];   // selected values (median passes)
    unsigned int hist[256];
};

// |w - mu| of weight t as an order-preserving key (non-negative doubles order like their bit patterns).
struct SrcAbsDev {
    const float* W;
    const double* ms;
    const uint8_t* mask;  // candidates only where mask != 0 (NULL: every weight)
    __device__ bool valid(int64_t t) const { return mask == nullptr || mask[t] != 0; }
    __device__ unsigned long long key(int64_t t, double mu) const {
        return (unsigned long long)__double_as_longlong(fabs(__dsub_rn((double)W[t], mu)));
    }
    __device__ double mu() const { return ms[0]; }
};

// Any doubles: flip so that unsigned order equals numeric order.
struct SrcDouble {
    const double* v;
    __device__ bool valid(int64_t) const { return true; }
    __device__ unsigned long long key(int64_t t, double) const {
        const unsigned long long b = (unsigned long long)__double_as_longlong(v[t]);
        return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
    }
    __device__ double mu() const { return 0.0; }
};
__device__ __forceinline__ double unflip(unsigned long long k) {
    const unsigned long long b = (k >> 63) ? (k & 0x7fffffffffffffffull) : ~k;
    return __longlong_as_double((long long)b);
}

template <class Src>
__global__ void __launch_bounds__(256) sel_hist(Src src, int64_t n, SelState* st) {
    __shared__ unsigned int h[256];
    if (st->skip) return;
    h[threadIdx.x] = 0;
    __syncthreads();
    const int shift = st->shift;
    const unsigned long long prefix = st->prefix;
    const double mu = src.mu();
    // runs of one digit (the high bytes of similar magnitudes) are counted in a register first
    unsigned int run_bin = 0, run = 0;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < n; t += (int64_t)gridDim.x * 256) {
        if (!src.valid(t)) continue;
        const unsigned long long key = src.key(t, mu);
        if (shift == 56 || ((key ^ prefix) >> (shift + 8)) == 0) {
            const unsigned int bin = (unsigned int)(key >> shift) & 255u;
            if (bin != run_bin && run) { atomicAdd(&h[run_bin], run); run = 0; }
            run_bin = bin;
            ++run;
        }
    }
    if (run) atomicAdd(&h[run_bin], run);
    __syncthreads();
    if (h[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], h[threadIdx.x]);
}

__global__ void sel_pick(SelState* st) {
    if (st->skip) return;
    long long k = st->k;
    const int shift = st->shift;
    int d;
    if (st->descending) {
        for (d = 255; d > 0; --d) {
            const long long c = st->hist[d];
            if (k < c) break;
            k -= c;
        }
    } else {
        for (d = 0; d < 255; ++d) {
            const long long c = st->hist[d];
            if (k < c) break;
            k -= c;
        }
    }
    st->k = k;
    st->prefix |= (unsigned long long)d << shift;
    st->shift = shift - 8;
    for (int j = 0; j < 256; ++j) st->hist[j] = 0;
}

__global__ void sel_begin(SelState* st, long long k, int descending) {
    st->prefix = 0;
    st->k = k;
    st->shift = 56;
    st->descending = descending;
    st->skip = 0;
    for (int j = 0; j < 256; ++j) st->hist[j] = 0;
}

// value[slot] = the selected double (SrcDouble keys)
__global__ void sel_store_double(SelState* st, int slot) { st->value[slot] = unflip(st->prefix); }
// value[slot] = the selected |w - mu|
__global__ void sel_store_absdev(SelState* st, int slot) { st->value[slot] = __longlong_as_double((long long)st->prefix); }

__global__ void median_finish(const SelState* st, int64_t n, double scale, double* out) {
    const double m = (n & 1) ? st->value[1] : __dmul_rn(0.5, __dadd_rn(st->value[0], st->value[1]));
    *out = scale == 1.0 ? m : __dmul_rn(scale, m);
}

// The same descent for a short array of doubles (the per-channel cosines), one block, one launch.
__global__ void __launch_bounds__(1024) median_small_kernel(const double* __restrict__ v, int n, double* out) {
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ long long s_k;
    __shared__ double val[2];
    const SrcDouble src{v};
    for (int slot = 0; slot < 2; ++slot) {
        if (threadIdx.x == 0) { s_prefix = 0; s_k = slot == 0 ? (n - 1) / 2 : n / 2; }
        for (int shift = 56; shift >= 0; shift -= 8) {
            if (threadIdx.x < 256) hist[threadIdx.x] = 0;
            __syncthreads();
            const unsigned long long prefix = s_prefix;
            for (int t = threadIdx.x; t < n; t += 1024) {
                const unsigned long long key = src.key(t, 0.0);
                if (shift == 56 || ((key ^ prefix) >> (shift + 8)) == 0) atomicAdd(&hist[(key >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                long long k = s_k;
                int d;
                for (d = 0; d < 255; ++d) {
                    const long long c = hist[d];
                    if (k < c) break;
                    k -= c;
                }
                s_k = k;
                s_prefix = prefix | ((unsigned long long)d << shift);
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) val[slot] = unflip(s_prefix);
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = (n & 1) ? val[1] : __dmul_rn(0.5, __dadd_rn(val[0], val[1]));
}

template <class Src>
static cudaError_t run_select(Src src, int64_t n, SelState* st, cudaStream_t s) {
    int blocks = (int)((n + 256 * 16 - 1) / (256 * 16));
    if (blocks < 1) blocks = 1;
    const int cap = xfp::sm_count() * 8;
    if (blocks > cap) blocks = cap;
    for (int p = 0; p < 8; ++p) {
        sel_hist<Src><<<blocks, 256, 0, s>>>(src, n, st);
        sel_pick<<<1, 1, 0, s>>>(st);
    }
    return cudaGetLastError();
}

// median of the keys of src (even n: mean of the two middle ones), times `scale`, to *out
template <class Src>
static cudaError_t run_median(Src src, int64_t n, double scale, bool absdev, double* out, SelState* st,
                              cudaStream_t s) {
    for (int slot = 0; slot < 2; ++slot) {
        const long long k = slot == 0 ? (n - 1) / 2 : n / 2;
        sel_begin<<<1, 1, 0, s>>>(st, k, 0);
        cudaError_t e = run_select(src, n, st, s);
        if (e != cudaSuccess) return e;
        if (absdev) sel_store_absdev<<<1, 1, 0, s>>>(st, slot);
        else sel_store_double<<<1, 1, 0, s>>>(st, slot);
    }
    // odd n: both passes chose the same element and value[1] is used
    median_finish<<<1, 1, 0, s>>>(st, n, scale, out);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ outlier mask

__global__ void __launch_bounds__(256) mask_threshold(const float* __restrict__ W, int64_t n,
                                                       const double* __restrict__ ms, double k, uint8_t* mask,
                                                       SelState* st) {
    __shared__ int warp_cnt[8];
    const double mu = ms[0];
    const double thresh = __dmul_rn(k, ms[1]);
    int c = 0;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < n; t += (int64_t)gridDim.x * 256) {
        const int m = fabs(__dsub_rn((double)W[t], mu)) > thresh;
        mask[t] = (uint8_t)m;
        c += m;
    }
    for (int d = 16; d > 0; d >>= 1) c += __shfl_xor_sync(0xffffffffu, c, d);
    if ((threadIdx.x & 31) == 0) warp_cnt[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < 8; ++w) tot += warp_cnt[w];
        if (tot) atomicAdd((unsigned long long*)&st->count, (unsigned long long)tot);
    }
}

__global__ void outlier_zero(SelState* st) { st->count = 0; }

// Decide what the selection has to do.  mode 0: keep = floor(cap*n), select only when more qualified.
// mode 1: keep = floor(rate*n) of all weights.
__global__ void outlier_plan(SelState* st, int64_t n, int mode, double frac, int64_t* count_out) {
    const long long keep = (long long)floor(__dmul_rn(frac, (double)n));
    st->keep = keep;
    st->prefix = 0;
    st->shift = 56;
    st->descending = 1;
    for (int j = 0; j < 256; ++j) st->hist[j] = 0;
    if (mode == 0) {
        st->skip = st->count <= keep;
        st->k = keep - 1;
        *count_out = st->skip ? st->count : keep;
    } else {
        st->skip = keep <= 0;
        st->count = n;
        st->k = keep - 1;
        *count_out = keep > 0 ? keep : 0;
    }
}

__global__ void __launch_bounds__(256) mask_clear(uint8_t* mask, int64_t n) {
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < n; t += (int64_t)gridDim.x * 256) mask[t] = 0;
}

// Ties of the selected key are kept in position order: count them per chunk ...
template <class Src>
__global__ void __launch_bounds__(256) tie_count(Src src, int64_t n, const SelState* st, int* blockcnt) {
    __shared__ int sh[8];
    __shared__ int total;
    if (st->skip) return;
    const unsigned long long T = st->prefix;
    const double mu = src.mu();
    const int64_t base = (int64_t)blockIdx.x * kTieChunk + (int64_t)threadIdx.x * kTiePer;
    int c = 0;
    for (int e = 0; e < kTiePer; ++e) {
        const int64_t t = base + e;
        if (t < n && src.valid(t) && src.key(t, mu) == T) ++c;
    }
    block_excl_scan(c, sh, &total);
    if (threadIdx.x == 0) blockcnt[blockIdx.x] = total;
}

// ... turn the chunk counts into offsets ...
__global__ void __launch_bounds__(1024) tie_scan(int* blockcnt, int nblk, const SelState* st) {
    __shared__ int sh[32];
    __shared__ int total;
    if (st->skip) return;
    int carry = 0;
    for (int b0 = 0; b0 < nblk; b0 += 1024) {
        const int b = b0 + threadIdx.x;
        const int v = b < nblk ? blockcnt[b] : 0;
        const int off = block_excl_scan(v, sh, &total);
        if (b < nblk) blockcnt[b] = carry + off;
        carry += total;
        __syncthreads();
    }
}

// ... and write the final mask: above the selected key, or one of its first k+1 ties.
template <class Src>
__global__ void __launch_bounds__(256) tie_apply(Src src, int64_t n, const SelState* st, const int* blockcnt,
                                                 uint8_t* mask) {
    __shared__ int sh[8];
    __shared__ int total;
    if (st->skip) return;
    const unsigned long long T = st->prefix;
    const long long need = st->k + 1;
    const double mu = src.mu();
    const int64_t base = (int64_t)blockIdx.x * kTieChunk + (int64_t)threadIdx.x * kTiePer;
    unsigned long long keys[kTiePer];
    int c = 0;
#pragma unroll
    for (int e = 0; e < kTiePer; ++e) {
        const int64_t t = base + e;
        const bool ok = t < n && src.valid(t);
        keys[e] = ok ? src.key(t, mu) : 0ull;
        if (ok && keys[e] == T) ++c;   // slots that are no candidates never count, whatever T is
    }
    long long rank = (long long)blockcnt[blockIdx.x] + block_excl_scan(c, sh, &total);
#pragma unroll
    for (int e = 0; e < kTiePer; ++e) {
        const int64_t t = base + e;
        if (t >= n) break;
        if (!src.valid(t)) continue;   // not a candidate: its mask byte is already 0
        int m = 0;
        if (keys[e] > T) m = 1;
        else if (keys[e] == T) m = rank++ < need;
        mask[t] = (uint8_t)m;
    }
}

// ------------------------------------------------------------------ Lloyd, one channel per block

constexpr int kLloydThreads = 256;

#ifdef XFP_TRACE
// phase boundaries of block 0 (clock64), read back by xfp_debug_lloyd_phases: a timing probe
__device__ long long g_lloyd_phase[8];
#define LLOYD_STAMP(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) g_lloyd_phase[i] = clock64(); } while (0)
#else
#define LLOYD_STAMP(i) do { } while (0)
#endif

__device__ __forceinline__ double bulk_value(const float* __restrict__ W, const uint8_t* __restrict__ mask,
                                             int64_t t, double mu) {
    return (mask != nullptr && mask[t]) ? mu : (double)W[t];
}

// Compare-exchange of the bitonic network: after it a <= b when `asc`, a >= b otherwise; equal keys stay put.
__device__ __forceinline__ void cswap(float& a, float& b, bool asc) {
    const bool sw = (a > b) == asc;
    const float x = sw ? b : a, y = sw ? a : b;
    a = x;
    b = y;
}
// the stages with partner distance 4, 2, 1 on eight consecutive elements
__device__ __forceinline__ void last3(float (&v)[8], bool asc) {
    cswap(v[0], v[4], asc); cswap(v[1], v[5], asc); cswap(v[2], v[6], asc); cswap(v[3], v[7], asc);
    cswap(v[0], v[2], asc); cswap(v[1], v[3], asc); cswap(v[4], v[6], asc); cswap(v[5], v[7], asc);
    cswap(v[0], v[1], asc); cswap(v[2], v[3], asc); cswap(v[4], v[5], asc); cswap(v[6], v[7], asc);
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    const float4 a = *(const float4*)p, b = *(const float4*)(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
    *(float4*)p = make_float4(v[0], v[1], v[2], v[3]);
    *(float4*)(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}

// The channel's bulk values in ascending order without storing them as doubles: the weights that were not
// extracted, sorted as floats, with the m copies of mu (one per extracted position) inserted at p0.
struct SortedBulk {
    const float* r;
    int p0, m;
    double mu;
    __device__ __forceinline__ double at(int t) const {   // one load, then a select: no branch
        const int u = t < p0 ? t : (t - m > 0 ? t - m : 0);
        const double v = (double)r[u];
        return (t >= p0 && t < p0 + m) ? mu : v;
    }
};

// LONG = false: one channel per CTA, its two arrays in shared memory (channels of up to 16384 weights).
// LONG = true: the arrays live in a slice of global scratch owned by the CTA (L1/L2 resident; the CTA's own
// writes are ordered by its barriers) and the resident CTAs walk the channels; any length the format allows.
template <bool LONG>
__global__ void __launch_bounds__(kLloydThreads, 4) lloyd_kernel(const float* __restrict__ W,
                                                               const uint8_t* __restrict__ mask,
                                                               const double* __restrict__ ms, int rows, int K, int Kp2,
                                                               int bits, int iters, uint16_t* __restrict__ cb16,
                                                               uint8_t* __restrict__ idx, double* scratch,
                                                               size_t slice_doubles) {
    extern __shared__ __align__(16) double sm[];
    double* base = LONG ? scratch + (size_t)blockIdx.x * slice_doubles : sm;
    double* pre = base;                      // [K + 1] serial prefix sums of the sorted bulk values
    float* r = (float*)(base + ((K + 2) & ~1));   // [Kp2] kept weights, ascending (extracted slots and padding = +inf); 16-byte aligned
    __shared__ double c[64];
    __shared__ double e16[64];
    __shared__ int cut[65];
    __shared__ int s_m, s_p0;
    const int tid = threadIdx.x;
    const int E = 1 << bits;
    const double mu = ms[0];

#pragma unroll 1
    for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    const int64_t row0 = (int64_t)row * K;
    LLOYD_STAMP(0);
    if (tid == 0) s_m = 0;
    __syncthreads();
    int extracted = 0;
    for (int kb = tid; kb < Kp2; kb += 8 * kLloydThreads) {   // eight loads in flight per thread
        float v[8];
        uint8_t x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int k = kb + e * kLloydThreads;
            v[e] = k < K ? W[row0 + k] : INFINITY;
            x[e] = (k < K && mask != nullptr) ? mask[row0 + k] : (uint8_t)0;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int k = kb + e * kLloydThreads;
            if (k < Kp2) r[k] = x[e] ? INFINITY : v[e];
            extracted += x[e] != 0;
        }
    }
    if (extracted) atomicAdd(&s_m, extracted);
    __syncthreads();
    LLOYD_STAMP(1);
    // bitonic sort, ascending.  The stages with partner distance 4, 2, 1 stay inside blocks of 8 consecutive
    // elements and run in registers (one pass per step instead of three trips through the array); the wider
    // stages go through the array, a thread's eight pairs loaded before any is written back.
    const int half = Kp2 >> 1, nblk8 = Kp2 >> 3;
    for (int b8 = tid; b8 < nblk8; b8 += kLloydThreads) {   // steps 2, 4 and 8 entirely in registers
        float v[8];
        load8(r + 8 * b8, v);
        cswap(v[0], v[1], true); cswap(v[2], v[3], false); cswap(v[4], v[5], true); cswap(v[6], v[7], false);
        cswap(v[0], v[2], true); cswap(v[1], v[3], true); cswap(v[4], v[6], false); cswap(v[5], v[7], false);
        cswap(v[0], v[1], true); cswap(v[2], v[3], true); cswap(v[4], v[5], false); cswap(v[6], v[7], false);
        last3(v, ((8 * b8) & 8) == 0);
        store8(r + 8 * b8, v);
    }
    __syncthreads();
    for (int size = 16; size <= Kp2; size <<= 1) {
        for (int j = size >> 1; j >= 8; j >>= 1) {
            for (int pb = tid; pb < half; pb += 8 * kLloydThreads) {
                int ia[8];
                float a[8], b[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int p = pb + e * kLloydThreads;
                    ia[e] = p < half ? (((p & ~(j - 1)) << 1) | (p & (j - 1))) : -1;
                    if (ia[e] >= 0) { a[e] = r[ia[e]]; b[e] = r[ia[e] + j]; }
                }
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (ia[e] >= 0 && (a[e] > b[e]) == ((ia[e] & size) == 0)) { r[ia[e]] = b[e]; r[ia[e] + j] = a[e]; }
            }
            __syncthreads();
        }
        for (int b8 = tid; b8 < nblk8; b8 += kLloydThreads) {
            float v[8];
            load8(r + 8 * b8, v);
            last3(v, ((8 * b8) & size) == 0);
            store8(r + 8 * b8, v);
        }
        __syncthreads();
    }
    LLOYD_STAMP(2);
    if (tid == 0) {   // where mu sits among the kept weights
        int lo = 0, hi = K - s_m;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if ((double)r[mid] <= mu) lo = mid + 1; else hi = mid;
        }
        s_p0 = lo;
    }
    __syncthreads();
    SortedBulk s{r, s_p0, s_m, mu};
    // serial prefix sums: cell sums below are differences of these, as in a one-pass CPU evaluation.
    // All threads first lay the sorted values out as doubles in pre[1..K]; one thread then scans in place,
    // fetching the next eight values before it starts the current chain of eight dependent adds.
    for (int t = tid; t < K; t += kLloydThreads) pre[t + 1] = s.at(t);
    __syncthreads();
    if (tid == 0) {
        double run = 0.0;
        double f[8], g[8];
        pre[0] = 0.0;
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = pre[1 + e];
        for (int t = 0; t < K; t += 8) {   // K is a multiple of 128
            if (t + 8 < K) {
#pragma unroll
                for (int e = 0; e < 8; ++e) g[e] = pre[t + 9 + e];
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                run = __dadd_rn(run, f[e]);
                f[e] = run;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) pre[t + 1 + e] = f[e];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = g[e];
        }
    }
    if (tid >= 32 && tid < 32 + E) {   // a warp other than the one that runs the prefix
        const int j = tid - 32;
        long long q = (long long)floor(__ddiv_rn(__dmul_rn(__dadd_rn((double)j, 0.5), (double)K), (double)E));
        if (q >= K) q = K - 1;
        c[j] = s.at((int)q);
    }
    if (tid == 32) { cut[0] = 0; cut[E] = K; }
    __syncthreads();
    LLOYD_STAMP(3);

    // P lanes share one boundary search (P = 256 / 2^N, at most a warp): each round probes P positions of
    // the remaining range at once, so 4096 values take three rounds at N = 4 instead of twelve steps.
    const int P = (kLloydThreads >> bits) > 32 ? 32 : (kLloydThreads >> bits);
    const int jb = tid / P, sub = tid % P;
    const unsigned gmask = (P == 32 ? 0xffffffffu : ((1u << P) - 1u)) << ((tid & 31) & ~(P - 1));
    for (int it = 0; it < iters; ++it) {
        // cell j = (b_{j-1}, b_j], b_j the midpoint of entries j and j+1: cut[j+1] = #{t : s[t] <= b_j}
        {
            const bool mine = jb < E - 1;
            const double b = mine ? __dmul_rn(0.5, __dadd_rn(c[jb], c[jb + 1])) : 0.0;
            int lo = 0, hi = mine ? K : 0;   // every t < lo has s[t] <= b, every t >= hi has s[t] > b
            while (__any_sync(0xffffffffu, lo < hi)) {
                const int step = (hi - lo + P - 1) / P;
                const int pos = lo + (sub + 1) * step - 1;
                const bool below = lo < hi && pos < hi && s.at(pos) <= b;
                const int cnt = __popc(__ballot_sync(0xffffffffu, below) & gmask);   // the probes are ordered
                if (lo < hi) {
                    const int nlo = lo + cnt * step;
                    const int nhi = cnt < P ? lo + (cnt + 1) * step - 1 : hi;
                    lo = nlo < hi ? nlo : hi;
                    hi = nhi < hi ? nhi : hi;
                    if (hi < lo) hi = lo;
                }
            }
            if (mine && sub == 0) cut[jb + 1] = lo;
        }
        __syncthreads();
        int changed = 0;
        if (tid < E) {
            const int n = cut[tid + 1] - cut[tid];
            if (n > 0) {
                const double mean = __ddiv_rn(__dsub_rn(pre[cut[tid + 1]], pre[cut[tid]]), (double)n);
                if (mean != c[tid]) { c[tid] = mean; changed = 1; }
            }
        }
        if (!__syncthreads_or(changed)) break;
    }
    LLOYD_STAMP(4);
    if (tid < E) {
        const uint16_t h = d2h(c[tid]);
        cb16[(int64_t)row * E + tid] = h;
        e16[tid] = h2d(h);
    }
    __syncthreads();
    // every weight goes to the nearest STORED entry (ties: lower index), four weights per thread at a time.  Up to
    // 16 entries the plain scan with four chains of compares in flight is the faster form; above, bisection.
    bool e_asc = E > 16;
    for (int j = 1; j < E && e_asc; ++j) e_asc = e16[j] >= e16[j - 1];
    for (int kb = tid; kb < K; kb += 4 * kLloydThreads) {
        double v[4], bd[4];
        int best[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int k = kb + e * kLloydThreads;
            v[e] = k < K ? bulk_value(W, mask, row0 + k, mu) : 0.0;
        }
        if (e_asc) {
#pragma unroll
            for (int e = 0; e < 4; ++e) best[e] = nearest_entry(e16, E, v[e], true);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) { bd[e] = fabs(__dsub_rn(v[e], e16[0])); best[e] = 0; }
            for (int j = 1; j < E; ++j) {
                const double ej = e16[j];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const double d = fabs(__dsub_rn(v[e], ej));
                    if (d < bd[e]) { bd[e] = d; best[e] = j; }
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int k = kb + e * kLloydThreads;
            if (k < K) idx[row0 + k] = (uint8_t)best[e];
        }
    }
    LLOYD_STAMP(5);
    if (!LONG) break;  // one channel per CTA
    __syncthreads();   // the arrays and the small tables are reused by the CTA's next channel
    }
}

// ------------------------------------------------------------------ decoded value of a stored index

struct Unpacked {
    const uint8_t* idx;
    const uint16_t* cb;
    const uint8_t* gid;
    const uint16_t* gscale;
    const uint16_t* gmid;
    int mode, K, E, G, group;
};
__device__ __forceinline__ uint16_t decode16(const Unpacked& u, int row, int k) {
    const int q = u.idx[(int64_t)row * u.K + k];
    if (u.mode == 0) return u.cb[(int64_t)row * u.E + q];
    const int64_t g = (int64_t)row * u.G + k / u.group;
    return v2a_value16(u.gscale[g], u.cb[(int)u.gid[g] * u.E + q], u.gmid[g]);
}

// ------------------------------------------------------------------ residual (CSR)

__global__ void __launch_bounds__(256) row_count_kernel(const uint8_t* __restrict__ mask, int K, int* cnt) {
    __shared__ int sh[8];
    __shared__ int total;
    const uint8_t* m = mask + (int64_t)blockIdx.x * K;
    int c = 0;
    for (int k = threadIdx.x; k < K; k += 256) c += m[k] != 0;
    block_excl_scan(c, sh, &total);
    if (threadIdx.x == 0) cnt[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) rowptr_scan(const int* cnt, int rows, int32_t* rowptr) {
    __shared__ int sh[32];
    __shared__ int total;
    int carry = 0;
    for (int b0 = 0; b0 < rows; b0 += 1024) {
        const int b = b0 + threadIdx.x;
        const int v = b < rows ? cnt[b] : 0;
        const int off = block_excl_scan(v, sh, &total);
        if (b < rows) rowptr[b] = carry + off;
        carry += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) rowptr[rows] = carry;
}

__global__ void __launch_bounds__(256) residual_kernel(const float* __restrict__ W, const uint8_t* __restrict__ mask,
                                                        Unpacked u, const int32_t* __restrict__ rowptr,
                                                        int32_t* ocol, uint16_t* oval, int64_t capacity) {
    __shared__ int sh[8];
    __shared__ int total;
    const int row = blockIdx.x;
    int64_t p = rowptr[row];
    if (rowptr[row + 1] == p) return;
    for (int k0 = 0; k0 < u.K; k0 += 256) {
        const int k = k0 + threadIdx.x;
        const int64_t t = (int64_t)row * u.K + k;
        const int f = k < u.K && mask[t] != 0;
        const int off = block_excl_scan(f, sh, &total);
        if (f && p + off < capacity) {
            ocol[p + off] = k;
            oval[p + off] = d2h(__dsub_rn((double)W[t], h2d(decode16(u, row, k))));
        }
        p += total;
        __syncthreads();
    }
}

// ------------------------------------------------------------------ per-channel cosine

__global__ void __launch_bounds__(256) cosine_kernel(const float* __restrict__ W, const uint8_t* __restrict__ mask,
                                                      Unpacked u, double* cosv) {
    __shared__ double sh[256];
    const int row = blockIdx.x;
    double ab = 0.0, aa = 0.0, bb = 0.0;
    for (int k = threadIdx.x; k < u.K; k += 256) {
        const int64_t t = (int64_t)row * u.K + k;
        const double a = (double)W[t];
        const uint16_t d16 = decode16(u, row, k);
        double b = h2d(d16);
        if (mask != nullptr && mask[t]) {
            const uint16_t s16 = d2h(__dsub_rn(a, b));           // the stored residual
            b = h2d(d2h(__dadd_rn(b, h2d(s16))));                // W^ = fp16(D16 + S), one rounding
        }
        ab = __dadd_rn(ab, __dmul_rn(a, b));
        aa = __dadd_rn(aa, __dmul_rn(a, a));
        bb = __dadd_rn(bb, __dmul_rn(b, b));
    }
    ab = block_sum(ab, sh);
    aa = block_sum(aa, sh);
    bb = block_sum(bb, sh);
    if (threadIdx.x == 0)
        cosv[row] = (aa == 0.0 || bb == 0.0) ? 1.0 : __ddiv_rn(ab, __dmul_rn(__dsqrt_rn(aa), __dsqrt_rn(bb)));
}

// ------------------------------------------------------------------ LibFit: the library

// u[i][j] = (c_ij - m_i) / s_i and nn[i] = |u_i|^2, one thread per channel
__global__ void libfit_normalise(const uint16_t* __restrict__ cb, int rows, int E, double* u, double* nn) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    double lo = INFINITY, hi = -INFINITY;
    for (int j = 0; j < E; ++j) {
        const double c = h2d(cb[(int64_t)i * E + j]);
        if (c < lo) lo = c;
        if (c > hi) hi = c;
    }
    const double m = __dmul_rn(0.5, __dadd_rn(hi, lo));
    double s = __dmul_rn(0.5, __dsub_rn(hi, lo));
    if (s == 0.0) s = 1.0;
    double acc = 0.0;
    for (int j = 0; j < E; ++j) {
        const double v = __ddiv_rn(__dsub_rn(h2d(cb[(int64_t)i * E + j]), m), s);
        u[(int64_t)i * E + j] = v;
        acc = __dadd_rn(acc, __dmul_rn(v, v));
    }
    nn[i] = acc;
}

// order[r] = the channel of rank r by (nn, channel): rank by counting, exact and order independent
__global__ void __launch_bounds__(256) libfit_rank(const double* __restrict__ nn, int rows, int* order) {
    const int i = blockIdx.x * 256 + threadIdx.x;
    __shared__ double tile[256];
    const double mine = i < rows ? nn[i] : 0.0;
    int r = 0;
    for (int j0 = 0; j0 < rows; j0 += 256) {
        __syncthreads();
        tile[threadIdx.x] = j0 + threadIdx.x < rows ? nn[j0 + threadIdx.x] : INFINITY;
        __syncthreads();
        const int lim = rows - j0 < 256 ? rows - j0 : 256;
        for (int j = 0; j < lim; ++j) {
            const double o = tile[j];
            r += (o < mine) || (o == mine && j0 + j < i);
        }
    }
    if (i < rows) order[r] = i;
}

__global__ void libfit_seed(const double* __restrict__ u, const int* __restrict__ order, int rows, int E, int L,
                            double* cen) {
    const int l = blockIdx.x, j = threadIdx.x;
    if (j >= E) return;
    long long t = rows >= L ? (long long)floor(__ddiv_rn(__dmul_rn(__dadd_rn((double)l, 0.5), (double)rows), (double)L))
                            : (long long)(l % rows);
    if (t >= rows) t = rows - 1;
    cen[l * E + j] = u[(int64_t)order[t] * E + j];
}

// asg[i] = nearest centroid (squared distance summed entry by entry; ties: lower centroid).  One warp per channel,
// lane = centroid (32 at a time): every lane sums its distance in entry order, the warp keeps the smallest
// (distance, centroid) pair -- the answer of a scan over the centroids with a strict "less than".
__global__ void __launch_bounds__(256) libfit_assign_rows(const double* __restrict__ u, const double* __restrict__ cen,
                                                           int rows, int E, int L, int* asg, const int* done) {
    if (*done) return;
    const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (i >= rows) return;
    int best = 0;
    double bd = INFINITY;
    for (int l0 = 0; l0 < L; l0 += 32) {
        const int l = l0 + lane;
        double d = INFINITY;
        if (l < L) {
            d = 0.0;
            for (int j = 0; j < E; ++j) {
                const double t = __dsub_rn(u[(int64_t)i * E + j], cen[l * E + j]);
                d = __dadd_rn(d, __dmul_rn(t, t));
            }
        }
        int bl = l;
#pragma unroll
        for (int o = 16; o; o >>= 1) {   // smallest distance, lower centroid on a tie
            const double od = __shfl_xor_sync(0xffffffffu, d, o);
            const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
            if (od < d || (od == d && ol < bl)) { d = od; bl = ol; }
        }
        if (d < bd) { bd = d; best = bl; }   // a later group of 32 wins only when strictly nearer
    }
    if (lane == 0) asg[i] = best;
}

// centroid l <- mean of its members, every entry summed in channel order.  One block per centroid: the
// members of each tile of 1024 channels are compacted in order, then thread j adds them to entry j.
__global__ void __launch_bounds__(1024) libfit_update(const double* __restrict__ u, const int* __restrict__ asg,
                                                       int rows, int E, int L, double* cen, int* changed,
                                                       const int* done) {
    __shared__ int sh[32];
    __shared__ int total;
    __shared__ int member[1024];
    if (*done) return;
    const int l = blockIdx.x, j = threadIdx.x;
    double acc = 0.0;
    long long cnt = 0;
    for (int i0 = 0; i0 < rows; i0 += 1024) {
        const int i = i0 + threadIdx.x;
        const int f = i < rows && asg[i] == l;
        const int off = block_excl_scan(f, sh, &total);
        if (f) member[off] = i;
        __syncthreads();
        const int n = total;
        if (j < E)
            for (int m = 0; m < n; ++m) acc = __dadd_rn(acc, u[(int64_t)member[m] * E + j]);
        cnt += n;
        __syncthreads();
    }
    if (j < E && cnt > 0) {
        const double m = __ddiv_rn(acc, (double)cnt);
        if (m != cen[l * E + j]) { cen[l * E + j] = m; *changed = 1; }
    }
}

// done |= !changed; changed = 0
__global__ void libfit_round_end(int* changed, int* done) {
    if (!*done && !*changed) *done = 1;
    *changed = 0;
}
__global__ void libfit_flags_init(int* changed, int* done) { *changed = 0; *done = 0; }

// lib[l] = the centroid's entries in ascending order, fp16
__global__ void libfit_store(const double* __restrict__ cen, int E, uint16_t* lib) {
    const int l = blockIdx.x;
    if (threadIdx.x != 0) return;
    double tmp[64];
    for (int j = 0; j < E; ++j) tmp[j] = cen[l * E + j];
    for (int a = 1; a < E; ++a) {   // insertion sort
        const double v = tmp[a];
        int b = a - 1;
        while (b >= 0 && tmp[b] > v) { tmp[b + 1] = tmp[b]; --b; }
        tmp[b + 1] = v;
    }
    for (int j = 0; j < E; ++j) lib[l * E + j] = d2h(tmp[j]);
}

// ------------------------------------------------------------------ LibFit: per-group assignment

// A block of GS threads takes `gpb` consecutive groups of GS weights (4 when L <= 32; GS = 64, 128 or 256, the
// group size of the format).  Thread (s, l) scores library entry l on group s serially over the GS values; one
// thread per group picks the winner; then the GS threads index each group against its winner.
template <int GS>
__global__ void __launch_bounds__(GS) libfit_group_kernel(const float* __restrict__ W,
                                                            const uint8_t* __restrict__ mask,
                                                            const double* __restrict__ ms, int64_t groups, int bits,
                                                            int L, int gpb, const uint16_t* __restrict__ lib,
                                                            uint8_t* idx, uint8_t* gid, uint16_t* gscale,
                                                            uint16_t* gmid) {
    constexpr int NW = GS / 32;
    __shared__ double gv[4][GS];
    __shared__ double red_lo[4][NW], red_hi[4][NW];
    __shared__ double sse[256];
    __shared__ double dec[4][64];
    __shared__ uint16_t s_mid[4], s_sc[4];
    __shared__ int s_best[4], s_const[4];
    const int E = 1 << bits;
    const int tid = threadIdx.x;
    const int lw = GS / gpb;                   // threads per group while scoring
    const double mu = ms[0];
    const int64_t g0 = (int64_t)blockIdx.x * gpb;
    for (int s = 0; s < gpb; ++s) {
        const int64_t grp = g0 + s;
        if (grp >= groups) break;
        const double v = bulk_value(W, mask, grp * GS + tid, mu);
        gv[s][tid] = v;
        double lo = v, hi = v;
        for (int d = 16; d > 0; d >>= 1) {
            lo = fmin(lo, __shfl_xor_sync(0xffffffffu, lo, d));
            hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, d));
        }
        if ((tid & 31) == 0) { red_lo[s][tid >> 5] = lo; red_hi[s][tid >> 5] = hi; }
    }
    __syncthreads();
    if (tid < gpb && g0 + tid < groups) {
        double lo = red_lo[tid][0], hi = red_hi[tid][0];
#pragma unroll
        for (int w = 1; w < NW; ++w) { lo = fmin(lo, red_lo[tid][w]); hi = fmax(hi, red_hi[tid][w]); }
        s_mid[tid] = d2h(__dmul_rn(0.5, __dadd_rn(hi, lo)));
        s_sc[tid] = d2h(__dmul_rn(0.5, __dsub_rn(hi, lo)));
        s_const[tid] = hi == lo;
    }
    __syncthreads();
    {
        const int s = tid / lw;
        const int64_t grp = g0 + s;
        if (grp < groups && !s_const[s]) {
            const uint16_t mid16 = s_mid[s], sc16 = s_sc[s];
            for (int l = tid % lw; l < L; l += lw) {
                double d16[64];
                bool asc = true;
                for (int j = 0; j < E; ++j) {
                    d16[j] = h2d(v2a_value16(sc16, lib[l * E + j], mid16));
                    if (j && d16[j] < d16[j - 1]) asc = false;
                }
                double acc = 0.0;
                for (int t = 0; t < GS; t += 4) {   // four searches in flight, the sum stays in value order
                    double d[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const double x = gv[s][t + e];
                        d[e] = __dsub_rn(x, d16[nearest_entry(d16, E, x, asc)]);
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc = __dadd_rn(acc, __dmul_rn(d[e], d[e]));
                }
                sse[s * L + l] = acc;   // gpb * L <= 256
            }
        }
    }
    __syncthreads();
    if (tid < gpb && g0 + tid < groups) {
        const int64_t grp = g0 + tid;
        int best = 0;
        if (!s_const[tid]) {
            double b = INFINITY;
            for (int l = 0; l < L; ++l) {
                const double e = sse[tid * L + l];
                if (e < b) { b = e; best = l; }
            }
        }
        s_best[tid] = best;
        gid[grp] = (uint8_t)best;
        gscale[grp] = s_const[tid] ? (uint16_t)0 : s_sc[tid];   // a constant group: scale 0, entry 0, indices 0
        gmid[grp] = s_mid[tid];
    }
    __syncthreads();
    for (int e = tid; e < gpb * E; e += GS) {
        const int s = e / E, j = e % E;
        if (g0 + s < groups) dec[s][j] = h2d(v2a_value16(s_sc[s], lib[s_best[s] * E + j], s_mid[s]));
    }
    __syncthreads();
    for (int s = 0; s < gpb; ++s) {
        const int64_t grp = g0 + s;
        if (grp >= groups) break;
        int bj = 0;
        if (!s_const[s]) {
            bool asc = true;
            for (int j = 1; j < E; ++j) asc = asc && dec[s][j] >= dec[s][j - 1];
            bj = nearest_entry(dec[s], E, gv[s][tid], asc);
        }
        idx[grp * GS + tid] = (uint8_t)bj;
    }
}

// ------------------------------------------------------------------ host side

struct Workspace {
    double* part;      // [kRedBlocks]
    SelState* sel;
    int* flags;        // [2] LibFit changed / done
    int* tie;          // [ceil(n / kTieChunk)]
    int* rowcnt;       // [rows]
    double* u;         // [rows][64]
    double* nn;        // [rows]
    int* order;        // [rows]
    int* asg;          // [rows]
    double* cen;       // [256][64]
    size_t bytes;
};

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

static Workspace carve(void* base, int64_t rows, int64_t cols) {
    Workspace w;
    char* p = (char*)base;
    size_t o = 0;
    auto take = [&](size_t bytes) { char* r = p + o; o += align256(bytes); return r; };
    const int64_t n = rows * cols;
    w.part = (double*)take(sizeof(double) * kRedBlocks);
    w.sel = (SelState*)take(sizeof(SelState));
    w.flags = (int*)take(sizeof(int) * 2);
    w.tie = (int*)take(sizeof(int) * (size_t)((n + kTieChunk - 1) / kTieChunk + 1));
    w.rowcnt = (int*)take(sizeof(int) * (size_t)rows);
    w.u = (double*)take(sizeof(double) * (size_t)rows * 64);
    w.nn = (double*)take(sizeof(double) * (size_t)rows);
    w.order = (int*)take(sizeof(int) * (size_t)rows);
    w.asg = (int*)take(sizeof(int) * (size_t)rows);
    w.cen = (double*)take(sizeof(double) * 256 * 64);
    if (cols > 16384) {   // channels too long for shared memory: the Lloyd kernel's arrays (it uses the scratch from its start)
        size_t kp2 = 1;
        while ((int64_t)kp2 < cols) kp2 <<= 1;
        const size_t slice = (((size_t)cols + 2) & ~(size_t)1) + kp2 / 2;
        const size_t need = slice * sizeof(double) * (size_t)(rows < 2 * xfp::kSizingSMs ? rows : 2 * xfp::kSizingSMs);
        if (o < need) o = align256(need);
    }
    w.bytes = o;
    return w;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

static int shape_status(int64_t rows, int64_t cols) {
    if (rows < 1 || cols < 128 || cols % 128 != 0) return XFP_ERR_SHAPE;
    if (cols > 65536 || rows > (1 << 24)) return XFP_ERR_UNSUPPORTED;
    return XFP_OK;
}

static int lloyd_smem(int cols, int* kp2_out) {
    int kp2 = 1;
    while (kp2 < cols) kp2 <<= 1;
    *kp2_out = kp2;
    return (int)(sizeof(double) * (((size_t)cols + 2) & ~(size_t)1) + sizeof(float) * (size_t)kp2);
}

static Unpacked unpacked_of(const xfp_desc* d, const uint8_t* idx, const uint16_t* cb, const uint8_t* gid,
                            const uint16_t* gscale, const uint16_t* gmid) {
    Unpacked u;
    u.idx = idx; u.cb = cb; u.gid = gid; u.gscale = gscale; u.gmid = gmid;
    u.mode = d->mode; u.K = d->cols; u.E = 1 << d->bits; u.group = d->group_size; u.G = d->cols / d->group_size;
    return u;
}

static int desc_status(const xfp_desc* d) {
    if (!d) return XFP_ERR_NULL;
    if (d->mode != 0 && d->mode != 1) return XFP_ERR_SHAPE;
    if (d->bits < 2 || d->bits > 6) return XFP_ERR_SHAPE;
    if (d->group_size != 64 && d->group_size != 128 && d->group_size != 256)
        return d->group_size > 0 ? XFP_ERR_UNSUPPORTED : XFP_ERR_SHAPE;
    if (d->cols > 0 && d->cols % d->group_size) return XFP_ERR_SHAPE;
    if (d->mode == 1 && (d->lib_size < 1 || d->lib_size > 256)) return XFP_ERR_SHAPE;
    return shape_status(d->rows, d->cols);
}

}  // namespace xq

using namespace xq;

extern "C" {

int xfp_quant_workspace_size(int32_t rows, int32_t cols, size_t* bytes) {
    if (!bytes) return XFP_ERR_NULL;
    const int st = shape_status(rows, cols);
    if (st) return st;
    *bytes = carve(nullptr, rows, cols).bytes;
    return XFP_OK;
}

int xfp_quant_stats(const float* W, int64_t n, int32_t sigma_mode, double* mu_sigma, void* workspace,
                    size_t workspace_bytes, void* stream) {
    if (!W || !mu_sigma || !workspace) return XFP_ERR_NULL;
    if (!aligned16(W) || !aligned16(mu_sigma) || !aligned16(workspace)) return XFP_ERR_ALIGN;
    if (n < 1 || (sigma_mode != 0 && sigma_mode != 1)) return XFP_ERR_SHAPE;
    if (workspace_bytes < carve(nullptr, 1, 128).bytes) return XFP_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(workspace, 1, 128);
    stats_partial<0><<<kRedBlocks, kRedThreads, 0, s>>>(W, n, mu_sigma, w.part);
    stats_final<0><<<1, kRedThreads, 0, s>>>(w.part, n, mu_sigma);
    if (sigma_mode == 0) {
        stats_partial<1><<<kRedBlocks, kRedThreads, 0, s>>>(W, n, mu_sigma, w.part);
        stats_final<1><<<1, kRedThreads, 0, s>>>(w.part, n, mu_sigma);
    } else {
        SrcAbsDev src{W, mu_sigma, nullptr};
        if (run_median(src, n, 1.4826, true, mu_sigma + 1, w.sel, s) != cudaSuccess) return XFP_ERR_CUDA;
    }
    return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_quant_outliers(const float* W, int64_t n, const double* mu_sigma, int32_t outlier_mode, double k_or_rate,
                       double cap_frac, uint8_t* mask, int64_t* count, void* workspace, size_t workspace_bytes,
                       void* stream) {
    if (!W || !mu_sigma || !mask || !count || !workspace) return XFP_ERR_NULL;
    if (!aligned16(W) || !aligned16(mask) || !aligned16(workspace)) return XFP_ERR_ALIGN;
    if (n < 1 || (outlier_mode != 0 && outlier_mode != 1)) return XFP_ERR_SHAPE;
    if (!(k_or_rate >= 0.0) || (outlier_mode == 0 && !(cap_frac >= 0.0 && cap_frac <= 1.0)) ||
        (outlier_mode == 1 && k_or_rate > 1.0))
        return XFP_ERR_SHAPE;
    const int64_t nblk = (n + kTieChunk - 1) / kTieChunk;
    // the tie counters are the only part of the scratch that grows with n; they start where the smallest layout puts them
    const size_t tie_offset = (size_t)((char*)carve(nullptr, 1, 128).tie - (char*)nullptr);
    if (workspace_bytes < tie_offset + (size_t)nblk * sizeof(int)) return XFP_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(workspace, 1, 128);   // part, sel, flags, then the tie counters
    const int64_t sweep_cap = (int64_t)xfp::sm_count() * 8;
    const int sweep = (int)(nblk < sweep_cap ? (nblk < 1 ? 1 : nblk) : sweep_cap);
    if (outlier_mode == 0) {
        outlier_zero<<<1, 1, 0, s>>>(w.sel);
        mask_threshold<<<sweep, 256, 0, s>>>(W, n, mu_sigma, k_or_rate, mask, w.sel);
        outlier_plan<<<1, 1, 0, s>>>(w.sel, n, 0, cap_frac, count);
        SrcAbsDev src{W, mu_sigma, mask};
        if (run_select(src, n, w.sel, s) != cudaSuccess) return XFP_ERR_CUDA;
        tie_count<SrcAbsDev><<<(unsigned)nblk, 256, 0, s>>>(src, n, w.sel, w.tie);
        tie_scan<<<1, 1024, 0, s>>>(w.tie, (int)nblk, w.sel);
        tie_apply<SrcAbsDev><<<(unsigned)nblk, 256, 0, s>>>(src, n, w.sel, w.tie, mask);
    } else {
        mask_clear<<<sweep, 256, 0, s>>>(mask, n);
        outlier_plan<<<1, 1, 0, s>>>(w.sel, n, 1, k_or_rate, count);
        SrcAbsDev src{W, mu_sigma, nullptr};
        if (run_select(src, n, w.sel, s) != cudaSuccess) return XFP_ERR_CUDA;
        tie_count<SrcAbsDev><<<(unsigned)nblk, 256, 0, s>>>(src, n, w.sel, w.tie);
        tie_scan<<<1, 1024, 0, s>>>(w.tie, (int)nblk, w.sel);
        tie_apply<SrcAbsDev><<<(unsigned)nblk, 256, 0, s>>>(src, n, w.sel, w.tie, mask);
    }
    return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

// long channels: resident CTAs, each with a slice of scratch for its two arrays
// (the scratch is sized for two CTAs on each of kSizingSMs SMs; a launch never uses more)
static size_t lloyd_slice_doubles(int cols, int kp2) { return (((size_t)cols + 2) & ~(size_t)1) + (size_t)kp2 / 2; }

int xfp_quant_lloyd(const float* W, const uint8_t* mask, const double* mu_sigma, int32_t rows, int32_t cols,
                    int32_t bits, int32_t iters, uint16_t* codebook, uint8_t* idx, void* workspace,
                    size_t workspace_bytes, void* stream) {
    if (!W || !mu_sigma || !codebook || !idx) return XFP_ERR_NULL;
    if (!aligned16(W) || !aligned16(codebook) || !aligned16(idx) || (mask && !aligned16(mask))) return XFP_ERR_ALIGN;
    const int st = shape_status(rows, cols);
    if (st) return st;
    if (bits < 2 || bits > 6 || iters < 0) return XFP_ERR_SHAPE;
    int kp2;
    const int smem = lloyd_smem(cols, &kp2);
    if (smem <= 227 * 1024 - 2048) {
        if (cudaFuncSetAttribute(lloyd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
            cudaFuncSetAttribute(lloyd_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout, 100) != cudaSuccess)
            return XFP_ERR_CUDA;
        lloyd_kernel<false><<<rows, kLloydThreads, smem, (cudaStream_t)stream>>>(W, mask, mu_sigma, rows, cols, kp2, bits,
                                                                                 iters, codebook, idx, nullptr, 0);
    } else {
        if (!workspace) return XFP_ERR_NULL;
        if (!aligned16(workspace)) return XFP_ERR_ALIGN;
        const size_t slice = lloyd_slice_doubles(cols, kp2);
        const int want = 2 * xfp::sched_sms();   // two resident CTAs per SM
        const int ctas = rows < want ? rows : want;
        if (workspace_bytes < slice * sizeof(double) * (size_t)ctas) return XFP_ERR_BUFFER_TOO_SMALL;
        lloyd_kernel<true><<<ctas, kLloydThreads, 0, (cudaStream_t)stream>>>(W, mask, mu_sigma, rows, cols, kp2, bits, iters,
                                                                             codebook, idx, (double*)workspace, slice);
    }
    return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_quant_libfit_library(const uint16_t* codebook, int32_t rows, int32_t bits, int32_t L, int32_t iters,
                             uint16_t* lib, void* workspace, size_t workspace_bytes, void* stream) {
    if (!codebook || !lib || !workspace) return XFP_ERR_NULL;
    if (!aligned16(codebook) || !aligned16(lib) || !aligned16(workspace)) return XFP_ERR_ALIGN;
    if (rows < 1 || bits < 2 || bits > 6 || L < 1 || L > 256 || iters < 0) return XFP_ERR_SHAPE;
    if (rows > (1 << 24)) return XFP_ERR_UNSUPPORTED;
    if (workspace_bytes < carve(nullptr, rows, 128).bytes) return XFP_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(workspace, rows, 128);
    const int E = 1 << bits;
    const int rb = (rows + 255) / 256;
    libfit_normalise<<<rb, 256, 0, s>>>(codebook, rows, E, w.u, w.nn);
    libfit_rank<<<rb, 256, 0, s>>>(w.nn, rows, w.order);
    libfit_seed<<<L, 64, 0, s>>>(w.u, w.order, rows, E, L, w.cen);
    libfit_flags_init<<<1, 1, 0, s>>>(w.flags, w.flags + 1);
    for (int it = 0; it < iters; ++it) {
        libfit_assign_rows<<<(rows + 7) / 8, 256, 0, s>>>(w.u, w.cen, rows, E, L, w.asg, w.flags + 1);
        libfit_update<<<L, 1024, 0, s>>>(w.u, w.asg, rows, E, L, w.cen, w.flags, w.flags + 1);
        libfit_round_end<<<1, 1, 0, s>>>(w.flags, w.flags + 1);
    }
    libfit_store<<<L, 32, 0, s>>>(w.cen, E, lib);
    return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_quant_libfit_assign(const float* W, const uint8_t* mask, const double* mu_sigma, int32_t rows, int32_t cols,
                            int32_t bits, int32_t L, int32_t group_size, const uint16_t* lib, uint8_t* idx, uint8_t* gid,
                            uint16_t* gscale, uint16_t* gmid, void* stream) {
    if (!W || !mu_sigma || !lib || !idx || !gid || !gscale || !gmid) return XFP_ERR_NULL;
    if (!aligned16(W) || !aligned16(lib) || !aligned16(idx) || !aligned16(gid) || !aligned16(gscale) ||
        !aligned16(gmid) || (mask && !aligned16(mask)))
        return XFP_ERR_ALIGN;
    const int st = shape_status(rows, cols);
    if (st) return st;
    if (bits < 2 || bits > 6 || L < 1 || L > 256) return XFP_ERR_SHAPE;
    if (group_size != 64 && group_size != 128 && group_size != 256) return group_size > 0 ? XFP_ERR_UNSUPPORTED : XFP_ERR_SHAPE;
    if (cols % group_size) return XFP_ERR_SHAPE;
    const int64_t groups = (int64_t)rows * (cols / group_size);
    if (groups > 0x7fffffff) return XFP_ERR_UNSUPPORTED;
    const int gpb = L <= 32 ? 4 : (L <= 64 ? 2 : 1);
    const unsigned grid = (unsigned)((groups + gpb - 1) / gpb);
    cudaStream_t s = (cudaStream_t)stream;
    if (group_size == 64)
        libfit_group_kernel<64><<<grid, 64, 0, s>>>(W, mask, mu_sigma, groups, bits, L, gpb, lib, idx, gid, gscale, gmid);
    else if (group_size == 128)
        libfit_group_kernel<128><<<grid, 128, 0, s>>>(W, mask, mu_sigma, groups, bits, L, gpb, lib, idx, gid, gscale, gmid);
    else
        libfit_group_kernel<256><<<grid, 256, 0, s>>>(W, mask, mu_sigma, groups, bits, L, gpb, lib, idx, gid, gscale, gmid);
    return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

static int unpacked_args_status(const xfp_desc* desc, const float* W, const uint8_t* idx, const uint16_t* codebook,
                                const uint8_t* gid, const uint16_t* gscale, const uint16_t* gmid) {
    const int st = desc_status(desc);
    if (st) return st;
    if (!W || !idx || !codebook) return XFP_ERR_NULL;
    if (desc->mode == 1 && (!gid || !gscale || !gmid)) return XFP_ERR_NULL;
    if (!aligned16(W) || !aligned16(idx) || !aligned16(codebook)) return XFP_ERR_ALIGN;
    return XFP_OK;
}

int xfp_quant_residual(const xfp_desc* desc, const float* W, const uint8_t* mask, const uint8_t* idx,
                       const uint16_t* codebook, const uint8_t* gid, const uint16_t* gscale, const uint16_t* gmid,
                       int32_t* out_rowptr, int32_t* out_col, uint16_t* out_val, int64_t capacity, void* workspace,
                       size_t workspace_bytes, void* stream) {
    const int st = unpacked_args_status(desc, W, idx, codebook, gid, gscale, gmid);
    if (st) return st;
    if (!mask || !out_rowptr || !workspace || (capacity > 0 && (!out_col || !out_val))) return XFP_ERR_NULL;
    if (!aligned16(mask) || !aligned16(out_rowptr) || !aligned16(workspace)) return XFP_ERR_ALIGN;
    if (capacity < 0) return XFP_ERR_SHAPE;
    if (workspace_bytes < carve(nullptr, desc->rows, desc->cols).bytes) return XFP_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(workspace, desc->rows, desc->cols);
    row_count_kernel<<<desc->rows, 256, 0, s>>>(mask, desc->cols, w.rowcnt);
    rowptr_scan<<<1, 1024, 0, s>>>(w.rowcnt, desc->rows, out_rowptr);
    residual_kernel<<<desc->rows, 256, 0, s>>>(W, mask, unpacked_of(desc, idx, codebook, gid, gscale, gmid), out_rowptr,
                                               out_col, out_val, capacity);
    return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_quant_cosine(const xfp_desc* desc, const float* W, const uint8_t* mask, const uint8_t* idx,
                     const uint16_t* codebook, const uint8_t* gid, const uint16_t* gscale, const uint16_t* gmid,
                     double* cos, void* stream) {
    const int st = unpacked_args_status(desc, W, idx, codebook, gid, gscale, gmid);
    if (st) return st;
    if (!cos) return XFP_ERR_NULL;
    if (!aligned16(cos) || (mask && !aligned16(mask))) return XFP_ERR_ALIGN;
    cosine_kernel<<<desc->rows, 256, 0, (cudaStream_t)stream>>>(W, mask, unpacked_of(desc, idx, codebook, gid, gscale, gmid),
                                                                cos);
    return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_quant_median(const double* v, int64_t n, double* median, void* workspace, size_t workspace_bytes,
                     void* stream) {
    if (!v || !median || !workspace) return XFP_ERR_NULL;
    if (!aligned16(v) || !aligned16(workspace)) return XFP_ERR_ALIGN;
    if (n < 1) return XFP_ERR_SHAPE;
    if (workspace_bytes < carve(nullptr, 1, 128).bytes) return XFP_ERR_BUFFER_TOO_SMALL;
    if (n <= (1 << 16)) {
        median_small_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(v, (int)n, median);
        return cudaGetLastError() == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
    }
    Workspace w = carve(workspace, 1, 128);
    SrcDouble src{v};
    return run_median(src, n, 1.0, false, median, w.sel, (cudaStream_t)stream) == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}

int xfp_quantize(int32_t mode, const float* W, int32_t rows, int32_t cols, const xfp_quant_params* p,
                 const int32_t* candidates, int32_t n_candidates, double tau, int32_t lib_size, uint8_t* mask,
                 uint8_t* idx, uint16_t* codebook, uint16_t* lib, uint8_t* gid, uint16_t* gscale, uint16_t* gmid,
                 int32_t* out_rowptr, int32_t* out_col, uint16_t* out_val, int64_t capacity, double* cos,
                 xfp_quant_result* result, void* workspace, size_t workspace_bytes, void* stream) {
    if (!W || !p || !candidates || !mask || !idx || !codebook || !out_rowptr || !cos || !result || !workspace)
        return XFP_ERR_NULL;
    if (mode != 0 && mode != 1) return XFP_ERR_SHAPE;
    if (mode == 1 && (!lib || !gid || !gscale || !gmid)) return XFP_ERR_NULL;
    if (n_candidates < 1 || n_candidates > 5) return XFP_ERR_SHAPE;
    for (int c = 0; c < n_candidates; ++c) {
        if (candidates[c] < 2 || candidates[c] > 6) return XFP_ERR_SHAPE;
        if (c && candidates[c] <= candidates[c - 1]) return XFP_ERR_SHAPE;
    }
    int st = shape_status(rows, cols);
    if (st) return st;
    size_t need;
    xfp_quant_workspace_size(rows, cols, &need);
    // two doubles (mu, sigma), the median and the count live behind the carved scratch
    if (workspace_bytes < need + 256) return XFP_ERR_BUFFER_TOO_SMALL;
    cudaStream_t s = (cudaStream_t)stream;
    double* ms = (double*)((char*)workspace + need);
    double* med_dev = ms + 2;
    int64_t* cnt_dev = (int64_t*)(ms + 4);
    const int64_t n = (int64_t)rows * cols;

    st = xfp_quant_stats(W, n, p->sigma_mode, ms, workspace, need, stream);
    if (st) return st;
    st = xfp_quant_outliers(W, n, ms, p->outlier_mode, p->outlier_mode ? p->rate : p->k_sigma, p->cap_frac, mask,
                            cnt_dev, workspace, need, stream);
    if (st) return st;
    double host_ms[2];
    int64_t host_cnt = 0;
    if (cudaMemcpyAsync(host_ms, ms, sizeof(host_ms), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(&host_cnt, cnt_dev, sizeof(host_cnt), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return XFP_ERR_CUDA;
    if (host_cnt > capacity) return XFP_ERR_BUFFER_TOO_SMALL;

    xfp_desc d;
    d.mode = mode; d.rows = rows; d.cols = cols; d.group_size = p->group_size ? p->group_size : 128;
    d.lib_size = mode ? lib_size : 0;
    if (d.group_size != 64 && d.group_size != 128 && d.group_size != 256) return d.group_size > 0 ? XFP_ERR_UNSUPPORTED : XFP_ERR_SHAPE;
    if (cols % d.group_size) return XFP_ERR_SHAPE;
    d.col_bits = 32; d.nnz = host_cnt;
    result->mu = host_ms[0]; result->sigma = host_ms[1]; result->nnz = host_cnt;
    result->fallback = 1; result->tried = 0; result->reserved = 0;
    for (int c = 0; c < n_candidates; ++c) {
        d.bits = candidates[c];
        st = xfp_quant_lloyd(W, mask, ms, rows, cols, d.bits, p->lloyd_iters, codebook, idx, workspace, need, stream);
        if (st) return st;
        const uint16_t* table = codebook;
        if (mode == 1) {
            st = xfp_quant_libfit_library(codebook, rows, d.bits, lib_size, p->lloyd_iters, lib, workspace, need, stream);
            if (st) return st;
            st = xfp_quant_libfit_assign(W, mask, ms, rows, cols, d.bits, lib_size, d.group_size, lib, idx, gid, gscale, gmid,
                                         stream);
            if (st) return st;
            table = lib;
        }
        st = xfp_quant_cosine(&d, W, mask, idx, table, gid, gscale, gmid, cos, stream);
        if (st) return st;
        st = xfp_quant_median(cos, rows, med_dev, workspace, need, stream);
        if (st) return st;
        double med = 0.0;
        if (cudaMemcpyAsync(&med, med_dev, sizeof(med), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess)
            return XFP_ERR_CUDA;
        result->bits = d.bits;
        result->median_cos = med;
        result->tried = c + 1;
        if (med >= tau) { result->fallback = 0; break; }
    }
    return xfp_quant_residual(&d, W, mask, idx, mode ? lib : codebook, gid, gscale, gmid, out_rowptr, out_col, out_val,
                              capacity, workspace, need, stream);
}

#ifdef XFP_TRACE
/* timing probe: clock64 at the six phase boundaries of block 0 of the last xfp_quant_lloyd launch (host array) */
int xfp_debug_lloyd_phases(long long* out) {
    return cudaMemcpyFromSymbol(out, g_lloyd_phase, sizeof(long long) * 8) == cudaSuccess ? XFP_OK : XFP_ERR_CUDA;
}
#endif

}  // extern "C"
