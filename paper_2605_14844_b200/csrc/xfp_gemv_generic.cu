// Generic fused decode GEMV  y = (D + S) x : every N in 2..6, V2 and V2a, batch tiles of 1/2/4/8,
// split-K with a fixed-order finish.  One warp lane owns one output channel (row); a warp walks
// super-chunks of 128 weights; x is broadcast from shared memory; the codebook sits in a
// per-lane shared-memory bank so that look-ups never conflict.
//
//   steps of "Fused Decode Kernel": (1) depack  -> field<N>()
//                                   (2) codebook gather from shared memory -> tab[]
//                                   (3) sparse outlier add -> CSR rows of the row-block
//                                   (4) multiply-accumulate, fp32
#include "xfp_internal.h"

namespace xfp {

constexpr int kGenericThreads = 256;
constexpr int kGenericWarps = kGenericThreads / 32;
constexpr int kMaxXFloats = 16384;  // fp32 activations staged per CTA (64 KB)

struct GenericArgs {
    Offsets off;
    const void* packed;
    const uint16_t* x;
    void* y;
    const void* const* packed_list;
    const uint16_t* const* x_list;
    void* const* y_list;
    float* partial;  // [problem][KS][BT][rows_pad]
    int* tickets;    // [problem][RB]
    int rows, cols, RB, SC, rows_pad;
    int KS, sc_per_split, nb, y_is_fp16, L, rep;
};

template <int N, int MODE, int BT>
__global__ void __launch_bounds__(kGenericThreads) gemv_generic_kernel(const GenericArgs a) {
    constexpr int E = 1 << N;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rb = blockIdx.x, ks = blockIdx.y, prob = blockIdx.z;
    const void* packed = a.packed_list ? a.packed_list[prob] : a.packed;
    const uint16_t* x = a.x_list ? a.x_list[prob] : a.x;
    void* y = a.y_list ? a.y_list[prob] : a.y;
    const Blob b = blob_at(packed, a.off);

    const int sc0 = ks * a.sc_per_split;
    const int nsc = min(a.SC, sc0 + a.sc_per_split) - sc0;
    const int kseg = a.sc_per_split * kSuper;

    const int tab_floats = MODE == 0 ? E * 32 : a.L * E * a.rep;
    float* tab = smem;
    float* xs = tab + tab_floats;                   // [BT][kseg]
    float* xg = xs + BT * kseg;                     // [BT][sc_per_split]   (V2a group sums of x)
    float* red = xg + BT * a.sc_per_split;          // [warps][BT][32]
    float* osum = red + kGenericWarps * BT * 32;    // [BT][32]

    // ---- stage the codebook (per-lane bank) or the library
    if (MODE == 0) {
        for (int t = threadIdx.x; t < E * 32; t += kGenericThreads) {
            const int e = t >> 5, l = t & 31;
            tab[t] = h2f(b.cb[(size_t)(rb * kRowsPerBlock + l) * E + e]);
        }
    } else {
        for (int t = threadIdx.x; t < tab_floats; t += kGenericThreads) tab[t] = h2f(b.cb[a.rep == 32 ? (t >> 5) : t]);
    }
    // ---- stage this split's slice of x as fp32
    for (int t = threadIdx.x; t < BT * kseg; t += kGenericThreads) {
        const int bb = t / kseg, kk = t - bb * kseg;
        float v = 0.f;
        if (bb < a.nb && kk < nsc * kSuper) v = h2f(x[(size_t)bb * a.cols + (size_t)sc0 * kSuper + kk]);
        xs[t] = v;
    }
    for (int t = threadIdx.x; t < BT * 32; t += kGenericThreads) osum[t] = 0.f;
    __syncthreads();
    if (MODE == 1) {
        for (int u = warp; u < BT * nsc; u += kGenericWarps) {
            const int bb = u / nsc, s = u - bb * nsc;
            const float4 v = *(const float4*)(xs + bb * kseg + s * kSuper + lane * 4);
            float t = (v.x + v.y) + (v.z + v.w);
#pragma unroll
            for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0) xg[bb * a.sc_per_split + s] = t;
        }
    }

    // ---- outliers of this row-block (first split only): a warp per row, lanes stride the row
    if (ks == 0) {
        for (int r = warp; r < 32; r += kGenericWarps) {
            const int row = rb * kRowsPerBlock + r;
            const int p0 = b.rowptr[row], p1 = b.rowptr[row + 1];
            if (p1 <= p0) continue;
            float oa[BT];
#pragma unroll
            for (int bb = 0; bb < BT; ++bb) oa[bb] = 0.f;
            for (int p = p0 + lane; p < p1; p += 32) {
                const uint32_t e = __ldg(b.oent + p);
                const float v = h2f((uint16_t)(e >> 16));
                const uint32_t col = e & 0xffffu;
#pragma unroll
                for (int bb = 0; bb < BT; ++bb)
                    if (bb < a.nb) oa[bb] = fmaf(v, h2f(__ldg(x + (size_t)bb * a.cols + col)), oa[bb]);
            }
#pragma unroll
            for (int bb = 0; bb < BT; ++bb) {
                float t = oa[bb];
#pragma unroll
                for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                if (lane == 0) osum[bb * 32 + r] = t;
            }
        }
    }
    if (MODE == 1) __syncthreads();  // xg visible to every warp

    // ---- dense part
    float acc[BT];
#pragma unroll
    for (int bb = 0; bb < BT; ++bb) acc[bb] = 0.f;

    uint32_t cur[4 * N + 1], nxt[4 * N + 1];
    cur[4 * N] = nxt[4 * N] = 0u;
    const uint4* ibase = b.idx + ((size_t)(rb * a.SC + sc0) * N) * 32 + lane;
    if (warp < nsc) {
#pragma unroll
        for (int v = 0; v < N; ++v) {
            const uint4 t = ld_stream(ibase + ((size_t)warp * N + v) * 32);
            cur[4 * v] = t.x; cur[4 * v + 1] = t.y; cur[4 * v + 2] = t.z; cur[4 * v + 3] = t.w;
        }
    }
#pragma unroll 1
    for (int s = warp; s < nsc; s += kGenericWarps) {
        const int sn = s + kGenericWarps;
        if (sn < nsc) {
#pragma unroll
            for (int v = 0; v < N; ++v) {
                const uint4 t = ld_stream(ibase + ((size_t)sn * N + v) * 32);
                nxt[4 * v] = t.x; nxt[4 * v + 1] = t.y; nxt[4 * v + 2] = t.z; nxt[4 * v + 3] = t.w;
            }
        }
        const float* xrow = xs + s * kSuper;
        if (MODE == 0) {
#pragma unroll
            for (int j4 = 0; j4 < kSuper / 4; ++j4) {
                float4 xv[BT];
#pragma unroll
                for (int bb = 0; bb < BT; ++bb) xv[bb] = *(const float4*)(xrow + bb * kseg + j4 * 4);
                const float w0 = tab[field<N>(cur, j4 * 4 + 0) * 32 + lane];
                const float w1 = tab[field<N>(cur, j4 * 4 + 1) * 32 + lane];
                const float w2 = tab[field<N>(cur, j4 * 4 + 2) * 32 + lane];
                const float w3 = tab[field<N>(cur, j4 * 4 + 3) * 32 + lane];
#pragma unroll
                for (int bb = 0; bb < BT; ++bb) {
                    acc[bb] = fmaf(w0, xv[bb].x, acc[bb]);
                    acc[bb] = fmaf(w1, xv[bb].y, acc[bb]);
                    acc[bb] = fmaf(w2, xv[bb].z, acc[bb]);
                    acc[bb] = fmaf(w3, xv[bb].w, acc[bb]);
                }
            }
        } else {
            const size_t unit = (size_t)(rb * a.SC + sc0 + s) * 32 + lane;
            const uint32_t id = b.gid[unit];
            const uint32_t sm = b.gsm[unit];
            const float scale = h2f((uint16_t)(sm & 0xffffu)), mid = h2f((uint16_t)(sm >> 16));
            const float* t = tab + (size_t)id * E * a.rep + (a.rep == 32 ? lane : 0);
            float gs[BT];
#pragma unroll
            for (int bb = 0; bb < BT; ++bb) gs[bb] = 0.f;
#pragma unroll
            for (int j4 = 0; j4 < kSuper / 4; ++j4) {
                float4 xv[BT];
#pragma unroll
                for (int bb = 0; bb < BT; ++bb) xv[bb] = *(const float4*)(xrow + bb * kseg + j4 * 4);
                const float w0 = t[field<N>(cur, j4 * 4 + 0) * a.rep];
                const float w1 = t[field<N>(cur, j4 * 4 + 1) * a.rep];
                const float w2 = t[field<N>(cur, j4 * 4 + 2) * a.rep];
                const float w3 = t[field<N>(cur, j4 * 4 + 3) * a.rep];
#pragma unroll
                for (int bb = 0; bb < BT; ++bb) {
                    gs[bb] = fmaf(w0, xv[bb].x, gs[bb]);
                    gs[bb] = fmaf(w1, xv[bb].y, gs[bb]);
                    gs[bb] = fmaf(w2, xv[bb].z, gs[bb]);
                    gs[bb] = fmaf(w3, xv[bb].w, gs[bb]);
                }
            }
            // sum_k (mid + scale*lib) x = scale * sum lib*x + mid * sum x
#pragma unroll
            for (int bb = 0; bb < BT; ++bb)
                acc[bb] = fmaf(scale, gs[bb], fmaf(mid, xg[bb * a.sc_per_split + s], acc[bb]));
        }
#pragma unroll
        for (int i = 0; i < 4 * N; ++i) cur[i] = nxt[i];
    }

    // ---- fixed-order reduction over the CTA's warps, then over the K splits
#pragma unroll
    for (int bb = 0; bb < BT; ++bb) red[(warp * BT + bb) * 32 + lane] = acc[bb];
    __syncthreads();
    const int t = threadIdx.x;
    const int bb = t >> 5, l = t & 31;
    const int row = rb * kRowsPerBlock + l;
    float total = 0.f;
    if (t < BT * 32) {
        total = osum[bb * 32 + l];
#pragma unroll
        for (int w = 0; w < kGenericWarps; ++w) total += red[(w * BT + bb) * 32 + l];
    }
    if (a.KS > 1) {
        __shared__ int s_last;
        float* part = a.partial + ((size_t)prob * a.KS) * BT * a.rows_pad;
        if (t < BT * 32) part[((size_t)ks * BT + bb) * a.rows_pad + row] = total;
        __threadfence();
        __syncthreads();
        if (t == 0) s_last = (atomicAdd(a.tickets + (size_t)prob * a.RB + rb, 1) == a.KS - 1);
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        if (t < BT * 32) {
            total = 0.f;
            for (int k2 = 0; k2 < a.KS; ++k2) total += __ldcg(part + ((size_t)k2 * BT + bb) * a.rows_pad + row);
        }
        if (t == 0) a.tickets[(size_t)prob * a.RB + rb] = 0;
    }
    if (t < BT * 32 && bb < a.nb && row < a.rows) {
        if (a.y_is_fp16)
            ((uint16_t*)y)[(size_t)bb * a.rows + row] = f2h(total);
        else
            ((float*)y)[(size_t)bb * a.rows + row] = total;
    }
}

// ------------------------------------------------------------------------------------ host side

static int next_pow2(int v) {
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

int generic_ksplit(const Layout& l, int batch_tile) {
    // enough CTAs for about two per SM, never more splits than super-chunks, and a slice of x
    // that fits the shared-memory budget
    int ks = 1;
    while ((long long)l.RB * ks < 2 * 148 && ks * 2 <= l.SC && ks < 32) ks *= 2;
    while ((long long)((l.SC + ks - 1) / ks) * kSuper * batch_tile > kMaxXFloats && ks < l.SC) ks *= 2;
    if (ks > l.SC) ks = l.SC;
    return ks;
}

size_t generic_workspace_bytes(const Layout& l) {
    int ksmax = 1;
    for (int bt = 1; bt <= 8; bt *= 2) {
        const int k = generic_ksplit(l, bt);
        const int spp = (l.SC + k - 1) / k;
        const int keff = (l.SC + spp - 1) / spp;
        if (keff * bt > ksmax) ksmax = keff * bt;
    }
    return align256((size_t)l.RB * 4) + align256((size_t)ksmax * l.rows_pad * 4);
}

template <int N, int MODE, int BT>
static cudaError_t launch_one(const GenericArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemv_generic_kernel<N, MODE, BT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    gemv_generic_kernel<N, MODE, BT><<<grid, kGenericThreads, smem, s>>>(a);
    return cudaGetLastError();
}

template <int N, int MODE>
static cudaError_t launch_bt(int bt, const GenericArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    switch (bt) {
        case 1: return launch_one<N, MODE, 1>(a, grid, smem, s);
        case 2: return launch_one<N, MODE, 2>(a, grid, smem, s);
        case 4: return launch_one<N, MODE, 4>(a, grid, smem, s);
        default: return launch_one<N, MODE, 8>(a, grid, smem, s);
    }
}

template <int MODE>
static cudaError_t launch_n(int bits, int bt, const GenericArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    switch (bits) {
        case 2: return launch_bt<2, MODE>(bt, a, grid, smem, s);
        case 3: return launch_bt<3, MODE>(bt, a, grid, smem, s);
        case 4: return launch_bt<4, MODE>(bt, a, grid, smem, s);
        case 5: return launch_bt<5, MODE>(bt, a, grid, smem, s);
        default: return launch_bt<6, MODE>(bt, a, grid, smem, s);
    }
}

cudaError_t launch_gemv_generic(const Layout& l, const GemvCall& c, cudaStream_t s) {
    const size_t ticket_bytes = align256((size_t)l.RB * 4);
    const size_t per_problem = c.workspace_bytes;
    for (int b0 = 0; b0 < c.batch; b0 += 8) {
        const int nb = c.batch - b0 < 8 ? c.batch - b0 : 8;
        const int bt = next_pow2(nb);
        GenericArgs a{};
        a.off = offsets_of(l);
        a.packed = c.packed;
        a.x = c.x ? c.x + (size_t)b0 * l.cols : nullptr;
        a.y = c.y ? (void*)((char*)c.y + (size_t)b0 * l.rows * (c.y_is_fp16 ? 2 : 4)) : nullptr;
        a.packed_list = c.packed_list; a.x_list = c.x_list; a.y_list = c.y_list;
        a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.rows_pad = l.rows_pad;
        const int ks = generic_ksplit(l, bt);
        a.sc_per_split = (l.SC + ks - 1) / ks;
        a.KS = (l.SC + a.sc_per_split - 1) / a.sc_per_split;
        a.nb = nb; a.y_is_fp16 = c.y_is_fp16; a.L = l.L;
        // V2a: a per-bank copy of the library when it fits, else a single copy (bank conflicts)
        a.rep = (l.mode && (size_t)l.L * l.E * 32 * 4 <= 128 * 1024) ? 32 : 1;
        // grouped calls stride the workspace by the per-problem size the caller was told
        a.tickets = (int*)c.workspace;
        a.partial = (float*)((char*)c.workspace + align256(ticket_bytes * (size_t)c.n));
        (void)per_problem;
        const size_t tab = l.mode ? (size_t)l.L * l.E * a.rep : (size_t)l.E * 32;
        const size_t smem = 4 * (tab + (size_t)bt * a.sc_per_split * kSuper + (size_t)bt * a.sc_per_split +
                                 (size_t)kGenericWarps * bt * 32 + (size_t)bt * 32);
        dim3 grid((unsigned)l.RB, (unsigned)a.KS, (unsigned)c.n);
        cudaError_t e = l.mode ? launch_n<1>(l.bits, bt, a, grid, smem, s) : launch_n<0>(l.bits, bt, a, grid, smem, s);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace xfp
