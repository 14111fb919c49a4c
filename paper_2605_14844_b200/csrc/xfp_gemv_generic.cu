// Generic fused decode GEMV  y = (D + S) x : every N in 2..6, V2 and V2a, batch tiles of 1/2/4/8,
// split-K with a fixed-order finish.  One warp lane owns one output channel (row); a warp walks
// super-chunks of 128 weights; x is broadcast from shared memory; the codebook sits in a
// per-lane shared-memory bank so that look-ups never conflict.
//
//   steps of "Fused Decode Kernel": (1) depack  -> field<N>()
//                                   (2) codebook gather from shared memory -> tab[]
//                                   (3) sparse outlier add -> the row-block's transposed slab, one slot of
//                                       all 32 channels per coalesced load, each lane adding to its own row
//                                   (4) multiply-accumulate, fp32
// Index vectors and V2a group metadata of the next super-chunk are fetched while the current one is
// decoded.  Weights are loaded before griddepcontrol.wait (programmatic dependent launch); x, y and
// the workspace are touched after it.
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
    int KS, sc_per_split, nb, y_is_fp16, L, rep, ell_slots, x_bf16;
    int GH;   // V2a: groups per super-chunk (2 when the format's groups hold 64 weights)
};

template <int N, int MODE, int BT>
__global__ void __launch_bounds__(kGenericThreads) gemv_generic_kernel(const GenericArgs a) {
    constexpr int E = 1 << N;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rb = blockIdx.x, ks = blockIdx.y, prob = blockIdx.z;
    asm volatile("griddepcontrol.launch_dependents;");
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
    float* xg = xs + BT * kseg;                     // [BT][sc_per_split][2]   (V2a: sums of x over the halves of a super-chunk)
    float* red = xg + BT * a.sc_per_split * 2;      // [warps][BT][32]

    // ---- start streaming: first super-chunk of this warp, its group metadata, first outlier slots
    uint32_t cur[4 * N + 1], nxt[4 * N + 1];
    cur[4 * N] = nxt[4 * N] = 0u;
    const uint4* ibase = b.idx + ((size_t)(rb * a.SC + sc0) * N) * 32 + lane;
    // group metadata of the current and the next super-chunk; [1] is the second half's group when GH = 2, else a copy
    uint32_t gid_c[2] = {0, 0}, gsm_c[2] = {0, 0}, gid_n[2] = {0, 0}, gsm_n[2] = {0, 0};
    const int GH = MODE == 1 ? a.GH : 1;
    if (warp < nsc) {
#pragma unroll
        for (int v = 0; v < N; ++v) {
            const uint4 t = ld_stream(ibase + ((size_t)warp * N + v) * 32);
            cur[4 * v] = t.x; cur[4 * v + 1] = t.y; cur[4 * v + 2] = t.z; cur[4 * v + 3] = t.w;
        }
        if (MODE == 1) {
            const size_t unit = (size_t)(rb * a.SC + sc0 + warp) * GH;
            gid_c[0] = b.gid[unit * 32 + lane];
            gsm_c[0] = b.gsm[unit * 32 + lane];
            gid_c[1] = b.gid[(unit + GH - 1) * 32 + lane];
            gsm_c[1] = b.gsm[(unit + GH - 1) * 32 + lane];
        }
    }
    // outlier slab of this row-block: slots gw, gw + stride, ... belong to this warp (first round fetched
    // before the rows' lengths are known: every slot below the capacity is readable)
    constexpr int kSlots = 4;
    const int gw = ks * kGenericWarps + warp, ostride = a.KS * kGenericWarps;
    // launches over several blobs read the slab geometry from each blob (their outlier counts differ)
    int ell_slots = a.ell_slots;
    const uint32_t* ell = b.ell;
    if (a.packed_list) {
        const int* hdr = (const int*)((const char*)packed + a.off.hdr);
        ell_slots = __ldg(hdr);
        ell = (const uint32_t*)((const char*)packed + *(const long long*)(hdr + 2));
    }
    const uint32_t* slab = ell + (size_t)rb * (ell_slots + 1) * 32 + lane;
    const uint32_t olen = ell_slots ? __ldg(slab) : 0u;
    uint32_t oe[kSlots];
    int width = ell_slots, oround = 0, nrounds = 0;
    auto fetch_slots = [&](int round) {
#pragma unroll
        for (int q = 0; q < kSlots; ++q) {
            const int j = gw + (round * kSlots + q) * ostride;
            oe[q] = j < width ? __ldg(slab + (size_t)(1 + j) * 32) : 0u;
        }
    };
    if (ell_slots) fetch_slots(0);

    // ---- stage the codebook (per-lane bank) or the library
    if (MODE == 0) {
        for (int t = threadIdx.x; t < E * 32; t += kGenericThreads) {
            const int e = t >> 5, l = t & 31;
            tab[t] = h2f(b.cb[(size_t)(rb * kRowsPerBlock + l) * E + e]);
        }
    } else {
        for (int t = threadIdx.x; t < tab_floats; t += kGenericThreads) tab[t] = h2f(b.cb[t / a.rep]);
    }
    // ---- x may come from the previous kernel: stage this split's slice as fp32
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int t = threadIdx.x; t < BT * kseg; t += kGenericThreads) {
        const int bb = t / kseg, kk = t - bb * kseg;
        float v = 0.f;
        if (bb < a.nb && kk < nsc * kSuper) v = x_as_float(x[(size_t)bb * a.cols + (size_t)sc0 * kSuper + kk], a.x_bf16);
        xs[t] = v;
    }
    __syncthreads();
    if (MODE == 1) {
        for (int u = warp; u < BT * nsc; u += kGenericWarps) {
            const int bb = u / nsc, s = u - bb * nsc;
            const float4 v = *(const float4*)(xs + bb * kseg + s * kSuper + lane * 4);
            float t = (v.x + v.y) + (v.z + v.w);
#pragma unroll
            for (int o = 8; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);   // lanes 0 and 16: the two halves
            if ((lane & 15) == 0) xg[(bb * a.sc_per_split + s) * 2 + (lane >> 4)] = t;
        }
        __syncthreads();  // xg visible to every warp
    }

    float acc[BT];
#pragma unroll
    for (int bb = 0; bb < BT; ++bb) acc[bb] = 0.f;

    // ---- outliers: every lane adds the slots of its own channel (x gathered from global memory:
    //      the staged copy only covers this split's slice of K)
    {
        int wmax = (int)olen;
#pragma unroll
        for (int o = 16; o; o >>= 1) wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
        width = min(wmax, ell_slots);
        const int mine = width > gw ? (width - gw + ostride - 1) / ostride : 0;
        nrounds = (mine + kSlots - 1) / kSlots;
    }
    auto consume_slots = [&]() {
#pragma unroll
        for (int q = 0; q < kSlots; ++q) {
            const float v = h2f((uint16_t)(oe[q] >> 16));
            const uint32_t col = oe[q] & 0xffffu;
#pragma unroll
            for (int bb = 0; bb < BT; ++bb)
                if (bb < a.nb) acc[bb] = fmaf(v, x_as_float(__ldg(x + (size_t)bb * a.cols + col), a.x_bf16), acc[bb]);
        }
    };

    // ---- dense part
#pragma unroll 1
    for (int s = warp; s < nsc; s += kGenericWarps) {
        const int sn = s + kGenericWarps;
        if (sn < nsc) {
#pragma unroll
            for (int v = 0; v < N; ++v) {
                const uint4 t = ld_stream(ibase + ((size_t)sn * N + v) * 32);
                nxt[4 * v] = t.x; nxt[4 * v + 1] = t.y; nxt[4 * v + 2] = t.z; nxt[4 * v + 3] = t.w;
            }
            if (MODE == 1) {
                const size_t unit_n = (size_t)(rb * a.SC + sc0 + sn) * GH;
                gid_n[0] = b.gid[unit_n * 32 + lane];
                gsm_n[0] = b.gsm[unit_n * 32 + lane];
                gid_n[1] = b.gid[(unit_n + GH - 1) * 32 + lane];
                gsm_n[1] = b.gsm[(unit_n + GH - 1) * 32 + lane];
            }
        }
        if (oround < nrounds) {
            consume_slots();
            if (++oround < nrounds) fetch_slots(oround);
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
            // the two halves of the super-chunk: one group each when GH = 2, the same group otherwise
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t id = gid_c[h];
                const uint32_t sm = gsm_c[h];
                const float scale = h2f((uint16_t)(sm & 0xffffu)), mid = h2f((uint16_t)(sm >> 16));
                const float* t = tab + (size_t)id * E * a.rep + (lane & (a.rep - 1));
                float gs[BT];
#pragma unroll
                for (int bb = 0; bb < BT; ++bb) gs[bb] = 0.f;
#pragma unroll
                for (int j4 = h * (kSuper / 8); j4 < (h + 1) * (kSuper / 8); ++j4) {
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
                // sum_k (mid + scale*lib) x = scale * sum lib*x + mid * sum x, over this half
#pragma unroll
                for (int bb = 0; bb < BT; ++bb)
                    acc[bb] = fmaf(scale, gs[bb], fmaf(mid, xg[(bb * a.sc_per_split + s) * 2 + h], acc[bb]));
            }
        }
#pragma unroll
        for (int i = 0; i < 4 * N; ++i) cur[i] = nxt[i];
        gid_c[0] = gid_n[0]; gid_c[1] = gid_n[1];
        gsm_c[0] = gsm_n[0]; gsm_c[1] = gsm_n[1];
    }
    while (oround < nrounds) {   // more outlier rounds than super-chunks
        consume_slots();
        if (++oround < nrounds) fetch_slots(oround);
    }
    // rows that fill their slab may continue in the CSR arrays (pathological skew): warp 0 of the first split
    if (warp == 0 && ks == 0 && ell_slots && (int)olen >= ell_slots) {
        const int row = rb * kRowsPerBlock + lane;
        const int p1 = __ldg(b.rowptr + row + 1);
        for (int p = __ldg(b.rowptr + row) + ell_slots; p < p1; ++p) {
            const uint32_t e = __ldg(b.oent + p);
#pragma unroll
            for (int bb = 0; bb < BT; ++bb)
                if (bb < a.nb)
                    acc[bb] = fmaf(h2f((uint16_t)(e >> 16)), x_as_float(__ldg(x + (size_t)bb * a.cols + (e & 0xffffu)), a.x_bf16), acc[bb]);
        }
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
        put_y(y, (size_t)bb * a.rows + row, total, a.y_is_fp16);
    }
}

// ------------------------------------------------------------------------------------ host side

static int next_pow2(int v) {
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

int generic_ksplit(const Layout& l, int batch_tile, int sms) {
    // enough CTAs for about two per SM, never more splits than super-chunks, and a slice of x
    // that fits the shared-memory budget
    int ks = 1;
    while ((long long)l.RB * ks < 2 * sms && ks * 2 <= l.SC && ks < 32) ks *= 2;
    while ((long long)((l.SC + ks - 1) / ks) * kSuper * batch_tile > kMaxXFloats && ks < l.SC) ks *= 2;
    if (ks > l.SC) ks = l.SC;
    return ks;
}

size_t generic_workspace_bytes(const Layout& l) {
    int ksmax = 1;
    for (int bt = 1; bt <= 8; bt *= 2) {
        const int k = generic_ksplit(l, bt, kSizingSMs);
        const int spp = (l.SC + k - 1) / k;
        const int keff = (l.SC + spp - 1) / spp;
        if (keff * bt > ksmax) ksmax = keff * bt;
    }
    return align256((size_t)l.RB * 4) + align256((size_t)ksmax * l.rows_pad * 4);
}

template <int N, int MODE, int BT>
static cudaError_t launch_one(const GenericArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemv_generic_kernel<N, MODE, BT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        attr_done.set(dev);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kGenericThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_generic_kernel<N, MODE, BT>, a);
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
        const int ks = generic_ksplit(l, bt, sched_sms());
        a.sc_per_split = (l.SC + ks - 1) / ks;
        a.KS = (l.SC + a.sc_per_split - 1) / a.sc_per_split;
        a.nb = nb; a.y_is_fp16 = c.y_is_fp16; a.x_bf16 = c.x_bf16; a.L = l.L; a.ell_slots = l.ell_slots;
        a.GH = l.GH;
        // V2a: a per-bank copy of the library when it fits, else a single copy (bank conflicts)
        a.rep = (l.mode && (size_t)l.L * l.E * 32 * 4 <= 128 * 1024) ? 32 : 1;
        // grouped calls stride the workspace by the per-problem size the caller was told
        a.tickets = (int*)c.workspace;
        a.partial = (float*)((char*)c.workspace + align256(ticket_bytes * (size_t)c.n));
        (void)per_problem;
        const size_t tab = l.mode ? (size_t)l.L * l.E * a.rep : (size_t)l.E * 32;
        const size_t smem = 4 * (tab + (size_t)bt * a.sc_per_split * kSuper + (size_t)bt * a.sc_per_split * 2 +
                                 (size_t)kGenericWarps * bt * 32);
        dim3 grid((unsigned)l.RB, (unsigned)a.KS, (unsigned)c.n);
        cudaError_t e = l.mode ? launch_n<1>(l.bits, bt, a, grid, smem, s) : launch_n<0>(l.bits, bt, a, grid, smem, s);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace xfp
