/*
 * XFP oracle: a plain, slow CPU statement of what the XFP format decodes to and of the
 * encoder that produces it.  TEST INFRASTRUCTURE ONLY: nothing on the product path may
 * link, import or call this file.  It shares no code with the CUDA library.
 *
 * Half 1 (format semantics; defines parity for the GPU library)
 *   - own fp16 <-> fp64 conversion (round to nearest even, subnormals, inf/nan)
 *   - Table 1 sub-byte packing of the paper (interchange words, LSB first)
 *   - dequantisation  W^ = fp16(D16 + S)          (Eq. 1, "The XFP Format / Decomposition")
 *       V2 : D16_ik = codebook_i[q_ik]                         (per-channel codebook)
 *       V2a: D16_ik = fp16(fp32(scale_ig * lib[id_ig][q_ik] + mid_ig)),  g = k / group
 *   - fp64 GEMV  y_b,i = sum_k (D_ik + S_ik) x_b,k  and the bound term sum_k |W_ik x_b,k|
 *
 * Half 2 (the encoder of "Encoding and Auto-Selection")
 *   - matrix statistics and outlier extraction        ("Outlier Extraction")
 *   - per-channel Lloyd with CDF-quantile initialisation ("Learned Codebook via Lloyd Iteration")
 *   - per-channel cosine                              (Algorithm 1, cos_sim line)
 *   - LibFit for V2a                                  ("V2a: Shared Codebook Library / Library learning")
 *     LibFit: the paper gives one sentence and no reconstruction figure for it, so the READING is this
 *     file's own (parity with the paper unpinned); what the functions compute is pinned: the group
 *     assignment against exhaustive search, the library against the fixed-point properties of k-means.
 *
 * Arithmetic is fp64 except the one V2a step the format fixes to fp32 (see xo_v2a_value16).
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ fp16 */

double xo_half_to_double(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 31;
    int m = h & 1023;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24); /* subnormal or zero */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp((double)(1024 + m), e - 25);
    return sign ? -v : v;
}

/* One rounding, to nearest, ties to even (the C default rounding mode drives nearbyint). */
uint16_t xo_double_to_half(double d) {
    uint16_t sign = signbit(d) ? 0x8000u : 0u;
    double a = fabs(d);
    if (isnan(d)) return (uint16_t)(sign | 0x7e00u);
    if (isinf(d)) return (uint16_t)(sign | 0x7c00u);
    if (a < ldexp(1.0, -14)) {
        /* subnormal range: units of 2^-24; 1024 units carries into the first normal */
        double q = nearbyint(ldexp(a, 24));
        return (uint16_t)(sign | (uint16_t)q);
    }
    int e;
    double m = frexp(a, &e);              /* a = m * 2^e, m in [0.5, 1) */
    double n = nearbyint(ldexp(m, 11));   /* 11-bit significand, in [1024, 2048] */
    int E = e - 1;
    if (n >= 2048.0) { n = 1024.0; E += 1; }
    if (E > 15) return (uint16_t)(sign | 0x7c00u);
    return (uint16_t)(sign | ((uint16_t)(E + 15) << 10) | ((uint16_t)n - 1024u));
}

uint16_t xo_float_to_half(float f) { return xo_double_to_half((double)f); }

void xo_halfs_to_doubles(int64_t n, const uint16_t* h, double* d) {
    for (int64_t t = 0; t < n; ++t) d[t] = xo_half_to_double(h[t]);
}

void xo_doubles_to_halfs(int64_t n, const double* d, uint16_t* h) {
    for (int64_t t = 0; t < n; ++t) h[t] = xo_double_to_half(d[t]);
}

/* ------------------------------------------------------------------ Table 1 packing */

/* Table 1: N -> values per word, word width.  Returns 0 on success. */
int xo_table1(int bits, int* vals_per_word, int* word_bits) {
    switch (bits) {
        case 2: *vals_per_word = 16; *word_bits = 32; return 0;
        case 3: *vals_per_word = 10; *word_bits = 32; return 0;
        case 4: *vals_per_word = 8;  *word_bits = 32; return 0;
        case 5: *vals_per_word = 3;  *word_bits = 16; return 0;
        case 6: *vals_per_word = 5;  *word_bits = 32; return 0;
    }
    return -1;
}

int64_t xo_table1_words(int bits, int64_t cols) {
    int v, w;
    if (xo_table1(bits, &v, &w)) return -1;
    return (cols + v - 1) / v;
}

/* value j of a word sits at bits [j*N, (j+1)*N), reserve bits zero, tail padded with index 0 */
void xo_table1_pack_row(int bits, const uint8_t* idx, int64_t cols, void* words) {
    int v, wb;
    if (xo_table1(bits, &v, &wb)) return;
    int64_t nw = (cols + v - 1) / v;
    for (int64_t w = 0; w < nw; ++w) {
        uint32_t word = 0;
        for (int j = 0; j < v; ++j) {
            int64_t k = w * v + j;
            uint32_t q = (k < cols) ? idx[k] : 0u;
            word |= q << (j * bits);
        }
        if (wb == 32) ((uint32_t*)words)[w] = word;
        else ((uint16_t*)words)[w] = (uint16_t)word;
    }
}

void xo_table1_unpack_row(int bits, const void* words, int64_t cols, uint8_t* idx) {
    int v, wb;
    if (xo_table1(bits, &v, &wb)) return;
    uint32_t mask = (1u << bits) - 1u;
    for (int64_t k = 0; k < cols; ++k) {
        int64_t w = k / v;
        int j = (int)(k % v);
        uint32_t word = (wb == 32) ? ((const uint32_t*)words)[w] : ((const uint16_t*)words)[w];
        idx[k] = (uint8_t)((word >> (j * bits)) & mask);
    }
}

/* ------------------------------------------------------------------ the quantised matrix */

typedef struct {
    int32_t mode;       /* 0 = V2, 1 = V2a */
    int32_t rows, cols; /* output channels, input features K */
    int32_t bits;       /* N */
    int32_t group_size; /* 128 */
    int32_t lib_size;   /* V2a: L */
    const uint8_t* idx;       /* [rows][cols] */
    const uint16_t* codebook; /* V2: [rows][2^N]; V2a: [L][2^N] (fp16 bits) */
    const uint8_t* gid;       /* V2a: [rows][cols/group] */
    const uint16_t* gscale;   /* V2a: [rows][cols/group] fp16 */
    const uint16_t* gmid;     /* V2a: [rows][cols/group] fp16 */
    const int32_t* rowptr;    /* [rows+1] */
    const int32_t* ocol;      /* [nnz] */
    const uint16_t* oval;     /* [nnz] fp16 */
} xo_matrix;

/* V2a, one value: the product of two fp16 numbers is exact in fp32, so the fp32 sum below is
 * the single fp32 rounding of scale*lib + mid; a second rounding takes it to fp16. */
uint16_t xo_v2a_value16(uint16_t scale, uint16_t lib, uint16_t mid) {
    volatile float p = (float)xo_half_to_double(scale) * (float)xo_half_to_double(lib);
    volatile float d = p + (float)xo_half_to_double(mid);
    return xo_float_to_half(d);
}

static uint16_t bulk16(const xo_matrix* m, int64_t i, int64_t k) {
    int E = 1 << m->bits;
    uint8_t q = m->idx[i * m->cols + k];
    if (m->mode == 0) return m->codebook[i * E + q];
    int64_t G = m->cols / m->group_size;
    int64_t g = k / m->group_size;
    uint8_t id = m->gid[i * G + g];
    return xo_v2a_value16(m->gscale[i * G + g], m->codebook[(int64_t)id * E + q], m->gmid[i * G + g]);
}

/* unrounded bulk value used by the GEMV reference */
static double bulk64(const xo_matrix* m, int64_t i, int64_t k) {
    int E = 1 << m->bits;
    uint8_t q = m->idx[i * m->cols + k];
    if (m->mode == 0) return xo_half_to_double(m->codebook[i * E + q]);
    int64_t G = m->cols / m->group_size;
    int64_t g = k / m->group_size;
    uint8_t id = m->gid[i * G + g];
    return xo_half_to_double(m->gmid[i * G + g]) +
           xo_half_to_double(m->gscale[i * G + g]) * xo_half_to_double(m->codebook[(int64_t)id * E + q]);
}

/* W^[i][k] = fp16(D16 + S); the fp64 sum of two fp16 numbers is exact, so one rounding. */
void xo_dequant(const xo_matrix* m, uint16_t* W) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m->rows; ++i) {
        for (int64_t k = 0; k < m->cols; ++k) W[i * m->cols + k] = bulk16(m, i, k);
        if (m->rowptr)
            for (int32_t p = m->rowptr[i]; p < m->rowptr[i + 1]; ++p) {
                int64_t k = m->ocol[p];
                double s = xo_half_to_double(W[i * m->cols + k]) + xo_half_to_double(m->oval[p]);
                W[i * m->cols + k] = xo_double_to_half(s);
            }
    }
}

/* y[b][i] = sum_k (D_ik + S_ik) x[b][k] in fp64, k ascending; absum[b][i] = sum_k |(D_ik+S_ik) x[b][k]|.
 * Rows [row0, row1) only (lets a caller sample rows of a large matrix).  x as doubles: any activation type
 * (fp16, or the paper's native bf16) is exact in fp64. */
void xo_gemv_rows_x64(const xo_matrix* m, const double* xd, int32_t batch, int64_t row0, int64_t row1,
                      double* y, double* absum) {
    int64_t K = m->cols;
#pragma omp parallel
    {
        double* w = (double*)malloc(sizeof(double) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t i = row0; i < row1; ++i) {
            for (int64_t k = 0; k < K; ++k) w[k] = bulk64(m, i, k);
            if (m->rowptr)
                for (int32_t p = m->rowptr[i]; p < m->rowptr[i + 1]; ++p)
                    w[m->ocol[p]] += xo_half_to_double(m->oval[p]);
            for (int32_t b = 0; b < batch; ++b) {
                double s = 0.0, a = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    double t = w[k] * xd[(int64_t)b * K + k];
                    s += t;
                    a += fabs(t);
                }
                y[(int64_t)b * m->rows + i] = s;
                if (absum) absum[(int64_t)b * m->rows + i] = a;
            }
        }
        free(w);
    }
}

/* the same with x as fp16 bit patterns */
void xo_gemv_rows(const xo_matrix* m, const uint16_t* x, int32_t batch, int64_t row0, int64_t row1,
                  double* y, double* absum) {
    int64_t K = m->cols;
    double* xd = (double*)malloc(sizeof(double) * (size_t)batch * (size_t)K);
    for (int64_t t = 0; t < (int64_t)batch * K; ++t) xd[t] = xo_half_to_double(x[t]);
    xo_gemv_rows_x64(m, xd, batch, row0, row1, y, absum);
    free(xd);
}

int xo_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void xo_set_threads(int n) {
#ifdef _OPENMP
    omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ================================================================== Half 2: the encoder */

/* mean and population standard deviation of the whole matrix, fp64, two passes */
void xo_stats(const float* W, int64_t n, double* mu, double* sigma) {
    double s = 0.0;
    for (int64_t t = 0; t < n; ++t) s += (double)W[t];
    double m = s / (double)n;
    double v = 0.0;
    for (int64_t t = 0; t < n; ++t) {
        double d = (double)W[t] - m;
        v += d * d;
    }
    *mu = m;
    *sigma = sqrt(v / (double)n);
}

static int cmp_double(const void* a, const void* b) {
    double x = *(const double*)a, y = *(const double*)b;
    return (x > y) - (x < y);
}

/* robust scale 1.4826 * median|w - mu| (not in the paper; used by the synthetic config whose
 * "sigma" means the bulk sigma, not one inflated by the planted tail) */
double xo_robust_sigma(const float* W, int64_t n, double mu) {
    double* a = (double*)malloc(sizeof(double) * (size_t)n);
    for (int64_t t = 0; t < n; ++t) a[t] = fabs((double)W[t] - mu);
    qsort(a, (size_t)n, sizeof(double), cmp_double);
    double med = (n & 1) ? a[n / 2] : 0.5 * (a[n / 2 - 1] + a[n / 2]);
    free(a);
    return 1.4826 * med;
}

typedef struct { double key; int64_t pos; } keyed;
static int cmp_keyed_desc(const void* a, const void* b) {
    const keyed* x = (const keyed*)a; const keyed* y = (const keyed*)b;
    if (x->key != y->key) return (x->key < y->key) - (x->key > y->key); /* larger key first */
    return (x->pos > y->pos) - (x->pos < y->pos);                       /* tie: lower flat index */
}

/* mask[t] = 1 where |w - mu| > thresh; if more than cap_frac*n qualify keep the largest
 * |w - mu| (ties: lower flat index).  Returns the number kept. */
int64_t xo_outlier_mask(const float* W, int64_t n, double mu, double thresh, double cap_frac, uint8_t* mask) {
    int64_t cnt = 0;
    for (int64_t t = 0; t < n; ++t) {
        mask[t] = fabs((double)W[t] - mu) > thresh;
        cnt += mask[t];
    }
    int64_t cap = (int64_t)floor(cap_frac * (double)n);
    if (cnt <= cap) return cnt;
    keyed* c = (keyed*)malloc(sizeof(keyed) * (size_t)cnt);
    int64_t j = 0;
    for (int64_t t = 0; t < n; ++t)
        if (mask[t]) { c[j].key = fabs((double)W[t] - mu); c[j].pos = t; ++j; }
    qsort(c, (size_t)cnt, sizeof(keyed), cmp_keyed_desc);
    for (int64_t t = cap; t < cnt; ++t) mask[c[t].pos] = 0;
    free(c);
    return cap;
}

/* exactly the floor(rate*n) entries with the largest |w - mu| (ties: lower flat index) */
int64_t xo_outlier_top_rate(const float* W, int64_t n, double mu, double rate, uint8_t* mask) {
    int64_t keep = (int64_t)floor(rate * (double)n);
    memset(mask, 0, (size_t)n);
    if (keep <= 0) return 0;
    keyed* c = (keyed*)malloc(sizeof(keyed) * (size_t)n);
    for (int64_t t = 0; t < n; ++t) { c[t].key = fabs((double)W[t] - mu); c[t].pos = t; }
    qsort(c, (size_t)n, sizeof(keyed), cmp_keyed_desc);
    for (int64_t t = 0; t < keep; ++t) mask[c[t].pos] = 1;
    free(c);
    return keep;
}

/* index of the entry nearest to v among the fp16 values e16[0..E) (ties: lower index) */
static int nearest16(const double* e, int E, double v) {
    int best = 0;
    double bd = fabs(v - e[0]);
    for (int j = 1; j < E; ++j) {
        double d = fabs(v - e[j]);
        if (d < bd) { bd = d; best = j; }
    }
    return best;
}

/*
 * Lloyd on one channel ("Learned Codebook via Lloyd Iteration"): 2^N entries start at
 * CDF-uniform quantiles of the channel's bulk values, then `iters` rounds of nearest-neighbour
 * assignment and conditional-mean update.  v[0..K) are the bulk values (extracted positions
 * already hold mu).  Outputs the fp16 codebook and, for every k, the index of the nearest
 * STORED (fp16) entry.  trace, if given, receives the mean squared error of the fp64
 * codebook before each round and after the last (iters+1 numbers; entries after an early
 * stop repeat the last value).  Returns the number of rounds run.
 */
int xo_lloyd_row(const double* v, int64_t K, int bits, int iters, uint16_t* cb16, uint8_t* idx, double* trace) {
    int E = 1 << bits;
    double* s = (double*)malloc(sizeof(double) * (size_t)K);
    double* pre = (double*)malloc(sizeof(double) * (size_t)(K + 1));
    double* pre2 = (double*)malloc(sizeof(double) * (size_t)(K + 1));
    double c[64], e16[64];
    int64_t cut[65];
    memcpy(s, v, sizeof(double) * (size_t)K);
    qsort(s, (size_t)K, sizeof(double), cmp_double);
    pre[0] = 0.0; pre2[0] = 0.0;
    for (int64_t t = 0; t < K; ++t) { pre[t + 1] = pre[t] + s[t]; pre2[t + 1] = pre2[t] + s[t] * s[t]; }
    for (int j = 0; j < E; ++j) {
        int64_t q = (int64_t)floor(((double)j + 0.5) * (double)K / (double)E);
        if (q >= K) q = K - 1;
        c[j] = s[q];
    }
    int done = 0;
    for (int it = 0; it <= iters; ++it) {
        /* cell j = (b_{j-1}, b_j], b_j the midpoint of c_j and c_{j+1}: a tie goes to the lower j */
        cut[0] = 0;
        int64_t t = 0;
        for (int j = 0; j < E - 1; ++j) {
            double b = 0.5 * (c[j] + c[j + 1]);
            while (t < K && s[t] <= b) ++t;
            cut[j + 1] = t;
        }
        cut[E] = K;
        if (trace) {
            double sse = 0.0;
            for (int j = 0; j < E; ++j) {
                double n = (double)(cut[j + 1] - cut[j]);
                double s1 = pre[cut[j + 1]] - pre[cut[j]], s2 = pre2[cut[j + 1]] - pre2[cut[j]];
                sse += s2 - 2.0 * c[j] * s1 + n * c[j] * c[j];
            }
            trace[it] = sse / (double)K;
        }
        if (it == iters) break;
        int changed = 0;
        for (int j = 0; j < E; ++j) {
            int64_t n = cut[j + 1] - cut[j];
            if (n > 0) {
                double mean = (pre[cut[j + 1]] - pre[cut[j]]) / (double)n;
                if (mean != c[j]) { c[j] = mean; changed = 1; }
            } /* an empty cell keeps its entry */
        }
        ++done;
        if (!changed) {
            if (trace) for (int r = it + 1; r <= iters; ++r) trace[r] = trace[it];
            break;
        }
    }
    for (int j = 0; j < E; ++j) { cb16[j] = xo_double_to_half(c[j]); e16[j] = xo_half_to_double(cb16[j]); }
    for (int64_t k = 0; k < K; ++k) idx[k] = (uint8_t)nearest16(e16, E, v[k]);
    free(s); free(pre); free(pre2);
    return done;
}

/* bulk row: W with extracted positions replaced by mu ("Outlier Extraction") */
static void bulk_row(const float* W, const uint8_t* mask, double mu, int64_t i, int64_t K, double* out) {
    for (int64_t k = 0; k < K; ++k)
        out[k] = (mask && mask[i * K + k]) ? mu : (double)W[i * K + k];
}

/* V2: one Lloyd codebook per output channel */
void xo_quantize_v2(const float* W, int64_t rows, int64_t K, const uint8_t* mask, double mu, int bits, int iters,
                    uint8_t* idx, uint16_t* cb) {
    int E = 1 << bits;
#pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * (size_t)K);
#pragma omp for schedule(dynamic, 8)
        for (int64_t i = 0; i < rows; ++i) {
            bulk_row(W, mask, mu, i, K, v);
            xo_lloyd_row(v, K, bits, iters, cb + i * E, idx + i * K, NULL);
        }
        free(v);
    }
}

/* residual at the extracted positions: S = fp16(w - D16); D16 is what the bulk index decodes to */
void xo_residual(const float* W, const uint16_t* D16, const uint8_t* mask, int64_t rows, int64_t K,
                 int32_t* rowptr, int32_t* ocol, uint16_t* oval) {
    int32_t p = 0;
    for (int64_t i = 0; i < rows; ++i) {
        rowptr[i] = p;
        for (int64_t k = 0; k < K; ++k)
            if (mask[i * K + k]) {
                ocol[p] = (int32_t)k;
                oval[p] = xo_double_to_half((double)W[i * K + k] - xo_half_to_double(D16[i * K + k]));
                ++p;
            }
    }
    rowptr[rows] = p;
}

/* per-channel cosine between the original row and its reconstruction (Algorithm 1); a zero row gives 1 */
void xo_row_cosine(const float* W, const uint16_t* What, int64_t rows, int64_t K, double* cosv) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double ab = 0.0, aa = 0.0, bb = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double a = (double)W[i * K + k], b = xo_half_to_double(What[i * K + k]);
            ab += a * b; aa += a * a; bb += b * b;
        }
        cosv[i] = (aa == 0.0 || bb == 0.0) ? 1.0 : ab / (sqrt(aa) * sqrt(bb));
    }
}

/* ------------------------------------------------------------------ LibFit (V2a) */

typedef struct { double key; int64_t pos; } normed;
static int cmp_normed(const void* a, const void* b) {
    const normed* x = (const normed*)a; const normed* y = (const normed*)b;
    if (x->key != y->key) return (x->key > y->key) - (x->key < y->key);
    return (x->pos > y->pos) - (x->pos < y->pos);
}

/*
 * Library learning: a second Lloyd (k-means) pass over the per-channel codebooks.
 * cb[rows][E] are the V2 codebooks (fp16).  Each is normalised to u = (c - m)/s with
 * m = (max+min)/2, s = (max-min)/2 (s = 0 -> 1); k-means in R^E to L centroids, started
 * from L evenly spaced members after ordering the channels by |u|^2; `iters` rounds;
 * an empty cluster keeps its centroid.  lib[L][E] is stored fp16.
 */
void xo_libfit_library(const uint16_t* cb, int64_t rows, int bits, int L, int iters, uint16_t* lib) {
    int E = 1 << bits;
    double* u = (double*)malloc(sizeof(double) * (size_t)rows * E);
    normed* ord = (normed*)malloc(sizeof(normed) * (size_t)rows);
    for (int64_t i = 0; i < rows; ++i) {
        double lo = INFINITY, hi = -INFINITY;
        for (int j = 0; j < E; ++j) {
            double c = xo_half_to_double(cb[i * E + j]);
            if (c < lo) lo = c;
            if (c > hi) hi = c;
        }
        double m = 0.5 * (hi + lo), s = 0.5 * (hi - lo);
        if (s == 0.0) s = 1.0;
        double nn = 0.0;
        for (int j = 0; j < E; ++j) {
            u[i * E + j] = (xo_half_to_double(cb[i * E + j]) - m) / s;
            nn += u[i * E + j] * u[i * E + j];
        }
        ord[i].key = nn; ord[i].pos = i;
    }
    qsort(ord, (size_t)rows, sizeof(normed), cmp_normed);
    double* cen = (double*)malloc(sizeof(double) * (size_t)L * E);
    for (int l = 0; l < L; ++l) {
        int64_t t = (rows >= L) ? (int64_t)floor(((double)l + 0.5) * (double)rows / (double)L) : (l % rows);
        if (t >= rows) t = rows - 1;
        memcpy(cen + (int64_t)l * E, u + ord[t].pos * E, sizeof(double) * (size_t)E);
    }
    int* asg = (int*)malloc(sizeof(int) * (size_t)rows);
    double* acc = (double*)malloc(sizeof(double) * (size_t)L * E);
    int64_t* cnt = (int64_t*)malloc(sizeof(int64_t) * (size_t)L);
    for (int it = 0; it < iters; ++it) {
        for (int64_t i = 0; i < rows; ++i) {
            int best = 0; double bd = INFINITY;
            for (int l = 0; l < L; ++l) {
                double d = 0.0;
                for (int j = 0; j < E; ++j) { double t = u[i * E + j] - cen[(int64_t)l * E + j]; d += t * t; }
                if (d < bd) { bd = d; best = l; }
            }
            asg[i] = best;
        }
        memset(acc, 0, sizeof(double) * (size_t)L * E);
        memset(cnt, 0, sizeof(int64_t) * (size_t)L);
        for (int64_t i = 0; i < rows; ++i) {
            cnt[asg[i]]++;
            for (int j = 0; j < E; ++j) acc[(int64_t)asg[i] * E + j] += u[i * E + j];
        }
        int changed = 0;
        for (int l = 0; l < L; ++l)
            if (cnt[l] > 0)
                for (int j = 0; j < E; ++j) {
                    double m = acc[(int64_t)l * E + j] / (double)cnt[l];
                    if (m != cen[(int64_t)l * E + j]) { cen[(int64_t)l * E + j] = m; changed = 1; }
                }
        if (!changed) break;
    }
    for (int l = 0; l < L; ++l) {
        double tmp[64];
        memcpy(tmp, cen + (int64_t)l * E, sizeof(double) * (size_t)E);
        qsort(tmp, (size_t)E, sizeof(double), cmp_double);
        for (int j = 0; j < E; ++j) lib[(int64_t)l * E + j] = xo_double_to_half(tmp[j]);
    }
    free(u); free(ord); free(cen); free(asg); free(acc); free(cnt);
}

/*
 * Re-index every 128-weight group to its closest library entry under a per-group scale and
 * mid-point: mid = fp16((max+min)/2), scale = fp16((max-min)/2) of the group's bulk values;
 * for each library entry the squared error of nearest-value assignment against the decoded
 * fp16 values; keep the smallest (ties: lower entry); indices point at the nearest decoded
 * value (ties: lower index).  A constant group gets scale 0, id 0, indices 0.
 */
void xo_libfit_assign(const float* W, int64_t rows, int64_t K, const uint8_t* mask, double mu, int bits, int L,
                      int group, const uint16_t* lib, uint8_t* idx, uint8_t* gid, uint16_t* gscale, uint16_t* gmid) {
    int E = 1 << bits;
    int64_t G = K / group;
#pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * (size_t)K);
        double dec[64];
#pragma omp for schedule(dynamic, 8)
        for (int64_t i = 0; i < rows; ++i) {
            bulk_row(W, mask, mu, i, K, v);
            for (int64_t g = 0; g < G; ++g) {
                const double* gv = v + g * group;
                double lo = gv[0], hi = gv[0];
                for (int t = 1; t < group; ++t) { if (gv[t] < lo) lo = gv[t]; if (gv[t] > hi) hi = gv[t]; }
                uint16_t mid16 = xo_double_to_half(0.5 * (hi + lo));
                uint16_t sc16 = xo_double_to_half(0.5 * (hi - lo));
                gmid[i * G + g] = mid16;
                gscale[i * G + g] = sc16;
                if (hi == lo) {
                    gscale[i * G + g] = 0; gid[i * G + g] = 0;
                    memset(idx + i * K + g * group, 0, (size_t)group);
                    continue;
                }
                int best = 0; double bsse = INFINITY;
                for (int l = 0; l < L; ++l) {
                    for (int j = 0; j < E; ++j)
                        dec[j] = xo_half_to_double(xo_v2a_value16(sc16, lib[(int64_t)l * E + j], mid16));
                    double sse = 0.0;
                    for (int t = 0; t < group; ++t) {
                        int j = nearest16(dec, E, gv[t]);
                        double d = gv[t] - dec[j];
                        sse += d * d;
                    }
                    if (sse < bsse) { bsse = sse; best = l; }
                }
                gid[i * G + g] = (uint8_t)best;
                for (int j = 0; j < E; ++j)
                    dec[j] = xo_half_to_double(xo_v2a_value16(sc16, lib[(int64_t)best * E + j], mid16));
                for (int t = 0; t < group; ++t) idx[i * K + g * group + t] = (uint8_t)nearest16(dec, E, gv[t]);
            }
        }
        free(v);
    }
}
