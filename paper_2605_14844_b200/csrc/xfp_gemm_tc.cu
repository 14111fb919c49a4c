// Prefill form of the fused decode kernel, Y = X (D + S)^T for M >= 1 rows of x ("Fused Decode Kernel", steps
// (1)-(4): depack, codebook gather, outlier scatter-add into the dequantised tile, GEMM on the tensor cores), on
// the fifth-generation tensor cores: the decoded fp16 tile is the A operand of tcgen05.mma in shared memory, the
// x tile the B operand, the fp32 accumulator lives in tensor memory.
//
//   CTA      128 output channels (four row-blocks) x up to 128 rows of x x one K slice; 8 warps.
//   stage    one super-chunk (128 k): A = W^[128][128] fp16, B = x[T][128] fp16, both K-major in the plain
//            (unswizzled) core-matrix layout: element (r, k) at (k/8)*LBO + r*16 + (k%8)*2 bytes, so the 32 lanes
//            of a warp (one channel each) write 512 contiguous bytes per 8 decoded weights.  Two stages: the
//            tensor pipe multiplies stage s while the warps decode stage s^1.
//   decode   warp (row-block, half of the super-chunk): look-ups in per-lane shared-memory tables (pair tables
//            up to N = 3, one entry per index above), then the outliers of the lane's channel that fall into
//            the tile are added with one correctly rounded fp16 addition each: the tile holds exactly the
//            weights xfp_dequant writes.
//   mma      one thread issues eight m128 nT k16 instructions per stage and commits them to the stage's
//            mbarrier, which frees the stage for the decode two iterations later.
//   epilogue tcgen05.ld (lane = channel, registers = rows of x), direct store, or fp32 partials through the
//            workspace when K is cut (few row tiles): the last CTA of a tile adds the slices in slice order.
// Every wait on an mbarrier has an iteration limit; when one runs out the CTA stops issuing work, records it in
// the first word of the workspace and leaves through the common exit that frees its tensor memory.
#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

namespace {

constexpr int kTileRows = 128;   // output channels per CTA (the M of the instruction)
constexpr int kMaxT = 128;       // rows of x per CTA (the N of the instruction), a multiple of 16
constexpr int kWarps = 8;
constexpr int kALbo = kTileRows * 16;         // bytes between consecutive 8-k chunks of the A tile
constexpr int kAStage = 16 * kALbo;           // 32 KB
constexpr int kBLbo = (kMaxT + 1) * 16;       // one padding row: the x staging writes hit distinct banks
constexpr int kBStage = 16 * kBLbo;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kTmemCols = 128;

struct GemmArgs {
    Blob b;
    const uint16_t* x;
    void* y;
    int* ctrl;        // [0] error word, [1 + tile] arrival counters of the K slices
    float* partial;   // [tile][slice][T][128]
    int rows, cols, RB, SC, M, ell_slots, ks, sc_per_slice, y_kind;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

// Shared-memory operand descriptor, K-major, no swizzle: start address, byte distance between the two 8-k core
// matrices of one instruction (leading), byte distance between groups of 8 rows (stride), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3fffu) << 32) | (1ull << 46);
}

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int N>
struct Tab {
    static constexpr int E = 1 << N;
    static constexpr bool kPair = N <= 3;
    static constexpr int T = kPair ? E * E : E;   // words per lane
};

// One half (64 weights) of the lane's super-chunk: look-ups, eight 16-byte stores into the A tile.
template <int N, int PART>
__device__ __forceinline__ void decode_half(const uint4* src, const unsigned char* tab, uint32_t tbase,
                                            unsigned char* arow) {
    constexpr int W0 = PART * 2 * N, W1 = W0 + 2 * N;     // 32-bit words of this half of the bit stream
    constexpr int V0 = W0 / 4, V1 = (W1 + 3) / 4;
    uint32_t w[4 * N + 1];
#pragma unroll
    for (int i = 0; i <= 4 * N; ++i) w[i] = 0u;
#pragma unroll
    for (int v = V0; v < V1; ++v) {
        const uint4 t = ld_stream(src + (size_t)v * 32);
        w[4 * v] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t o[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int p = PART * 32 + c * 4 + h;
            if (Tab<N>::kPair) {
                o[h] = *(const uint32_t*)(tab + pair_addr<N, 1>(w, p, tbase));
            } else {
                const uint32_t lo = *(const uint32_t*)(tab + single_addr<N, 1>(w, 2 * p, tbase));
                const uint32_t hi = *(const uint32_t*)(tab + single_addr<N, 1>(w, 2 * p + 1, tbase));
                o[h] = lo | (hi << 16);
            }
        }
        *(uint4*)(arow + (PART * 8 + c) * kALbo) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

template <int N>
__global__ void __launch_bounds__(kWarps * 32, 1) gemm_tc_kernel(const GemmArgs a) {
    constexpr int E = Tab<N>::E;
    constexpr int TW = Tab<N>::T;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sA = smem;                                  // two A stages
    unsigned char* sB = smem + 2 * kAStage;                    // two B stages
    unsigned char* sTab = sB + 2 * kBStage;                    // [4 row-blocks][TW][32] words
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = warp & 3, part = warp >> 2;                  // row-block of the tile, half of the super-chunk
    const int rb = blockIdx.x * 4 + q;
    const bool rb_ok = rb < a.RB;
    const int row = rb * kRowsPerBlock + lane;
    const int t0 = blockIdx.y * kMaxT;
    const int Tn = min(kMaxT, (a.M - t0 + 15) & ~15);          // rows of x of this tile, rounded up to 16
    const int sc0 = blockIdx.z * a.sc_per_slice;
    const int sc1 = min(a.SC, sc0 + a.sc_per_slice);
    const int tile = blockIdx.y * gridDim.x + blockIdx.x;

    // ---- set-up: barriers, tensor memory, tables ----
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&bars[0])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&bars[1])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    {
        // codebooks -> one word per (entry, lane); pair tables are built from a copy staged in the first A stage
        uint32_t* one = Tab<N>::kPair ? (uint32_t*)sA : (uint32_t*)sTab;
        for (int i = warp; i < 4 * E; i += kWarps) {
            const int qq = i / E, e = i % E, r = (blockIdx.x * 4 + qq) * kRowsPerBlock + lane;
            one[(qq * E + e) * 32 + lane] = (blockIdx.x * 4 + qq) < a.RB ? (uint32_t)__ldg(a.b.cb + (size_t)r * E + e) : 0u;
        }
        if (Tab<N>::kPair) {
            __syncthreads();
            uint32_t* tab = (uint32_t*)sTab;
            for (int i = warp; i < 4 * TW; i += kWarps) {
                const int qq = i / TW, t = i % TW;
                tab[(qq * TW + t) * 32 + lane] =
                    one[(qq * E + (t & (E - 1))) * 32 + lane] | (one[(qq * E + (t >> N)) * 32 + lane] << 16);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    // rows of the tile beyond the matrix decode to zero, once, in both stages
    if (!rb_ok) {
        for (int s = 0; s < 2; ++s)
            for (int c = 0; c < 8; ++c)
                *(uint4*)(sA + s * kAStage + (part * 8 + c) * kALbo + (q * 32 + lane) * 16) = make_uint4(0, 0, 0, 0);
    }

    // ---- the lane's outlier list: transposed slab first, the CSR arrays behind it ----
    const uint32_t* slab = nullptr;
    const uint32_t* spill = nullptr;
    int nslab = 0, total = 0, cur = 0;
    uint32_t ent = 0;
    if (rb_ok && a.ell_slots) {
        slab = a.b.ell + (size_t)rb * (a.ell_slots + 1) * 32 + lane;
        const int olen = (int)__ldg(slab);
        nslab = min(olen, a.ell_slots);
        total = nslab;
        if (olen >= a.ell_slots && row < a.rows) {
            const int p0 = __ldg(a.b.rowptr + row);
            total = __ldg(a.b.rowptr + row + 1) - p0;
            spill = a.b.oent + p0;
        }
    }
    auto fetch = [&](int j) { return j < nslab ? __ldg(slab + (size_t)(1 + j) * 32) : __ldg(spill + j); };
    if (total) {
        ent = fetch(0);
        const uint32_t kb = (uint32_t)sc0 * kSuper;
        while ((ent & 0xffffu) < kb && ++cur < total) ent = fetch(cur);
    }

    const uint32_t idesc = (1u << 4) | ((uint32_t)(Tn >> 3) << 17) | ((uint32_t)(kTileRows >> 4) << 24);
    const unsigned char* tab = sTab + (size_t)q * TW * 128;
    const uint32_t tbase = (uint32_t)lane * 4u;
    bool failed = false;
    int it = 0;
    for (int sc = sc0; sc < sc1; ++sc, ++it) {
        const int s = it & 1, use = it >> 1;
        bool ok = true;
        if (use >= 1) ok = mbar_wait(smem_u32(&bars[s]), (uint32_t)(use - 1) & 1u);
        unsigned char* As = sA + s * kAStage;
        unsigned char* Bs = sB + s * kBStage;
        if (ok) {
            // x tile: thread -> (row of x, 16-byte chunk); rows beyond M are zero
            const int k0 = sc * kSuper;
            for (int i = tid; i < Tn * 16; i += kWarps * 32) {
                const int c = i & 15, t = i >> 4;
                const uint32_t dst = smem_u32(Bs + c * kBLbo + t * 16);
                const uint16_t* src = a.x + (size_t)(t0 + t) * a.cols + k0 + c * 8;
                const int bytes = (t0 + t) < a.M ? 16 : 0;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst), "l"(bytes ? src : a.x), "r"(bytes) : "memory");
            }
            if (rb_ok) {
                const uint4* src = a.b.idx + ((size_t)rb * a.SC + sc) * N * 32 + lane;
                unsigned char* arow = As + (q * 32 + lane) * 16;
                if (part == 0) decode_half<N, 0>(src, tab, tbase, arow);
                else decode_half<N, 1>(src, tab, tbase, arow);
                // W^ = fp16(D16 + S) at the outliers of this channel inside the tile
                const uint32_t kend = (uint32_t)k0 + kSuper;
                while (cur < total && (ent & 0xffffu) < kend) {
                    const uint32_t kk = (ent & 0xffffu) - (uint32_t)k0;
                    if ((int)(kk >> 6) == part) {
                        const uint32_t ha = smem_u32(arow + (kk >> 3) * kALbo + (kk & 7u) * 2u);
                        uint16_t hv;
                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(hv) : "r"(ha) : "memory");
                        hv = __half_as_ushort(__hadd(__ushort_as_half(hv), __ushort_as_half((uint16_t)(ent >> 16))));
                        asm volatile("st.shared.u16 [%0], %1;" :: "r"(ha), "h"(hv) : "memory");
                    }
                    if (++cur < total) ent = fetch(cur);
                }
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        if (__syncthreads_or(!ok)) { failed = true; break; }
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_u32(As), b0 = smem_u32(Bs);
#pragma unroll
            for (int ks = 0; ks < kSuper / 16; ++ks) {
                const uint64_t da = smem_desc(a0 + 2 * ks * kALbo, kALbo, 128);
                const uint64_t db = smem_desc(b0 + 2 * ks * kBLbo, kBLbo, 128);
                umma_f16(tmem, da, db, idesc, (it > 0 || ks > 0) ? 1u : 0u);
            }
            umma_commit(smem_u32(&bars[s]));
        }
    }
    // ---- all products of this CTA are complete when the last commit has arrived ----
    if (!failed && it > 0) {
        const int lastit = it - 1;
        const bool ok = mbar_wait(smem_u32(&bars[lastit & 1]), (uint32_t)(lastit >> 1) & 1u);
        if (__syncthreads_or(!ok)) failed = true;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (failed) {
        if (tid == 0) atomicExch(a.ctrl, 1);
    } else {
        // lane = channel (tensor-memory lane 32*(warp%4) + lane), registers = 16 consecutive rows of x
        const int r = q * 32 + lane;
        float* part_out = a.partial + ((size_t)tile * a.ks + blockIdx.z) * kMaxT * kTileRows;
        for (int cc = part; cc * 16 < Tn; cc += 2) {
            uint32_t v[16];
            if (it > 0) {
                tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 16), v);
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = 0u;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int t = cc * 16 + j;
                if (a.ks > 1) part_out[t * kTileRows + r] = __uint_as_float(v[j]);
                else if (t0 + t < a.M && row < a.rows) put_y(a.y, (size_t)(t0 + t) * a.rows + row, __uint_as_float(v[j]), a.y_kind);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kTmemCols) : "memory");
    if (failed || a.ks == 1) return;

    // ---- K slices: the last CTA of the tile to arrive adds the slices in slice order ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(a.ctrl + 1 + tile, 1);
        s_last = ticket == a.ks - 1;
        if (s_last) a.ctrl[1 + tile] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const float* p0 = a.partial + (size_t)tile * a.ks * kMaxT * kTileRows;
    for (int i = tid; i < Tn * kTileRows; i += kWarps * 32) {
        const int t = i / kTileRows, r = i % kTileRows;
        const int orow = blockIdx.x * kTileRows + r;
        if (t0 + t >= a.M || orow >= a.rows) continue;
        float sum = 0.f;
        for (int z = 0; z < a.ks; ++z) sum += __ldcg(p0 + (size_t)z * kMaxT * kTileRows + i);
        put_y(a.y, (size_t)(t0 + t) * a.rows + orow, sum, a.y_kind);
    }
}

struct Plan {
    int row_tiles, tok_tiles, ks, sc_per_slice;
};

Plan plan_of(const Layout& l, int M) {
    Plan p;
    p.row_tiles = (l.RB + 3) / 4;
    p.tok_tiles = (M + kMaxT - 1) / kMaxT;
    const int tiles = p.row_tiles * p.tok_tiles;
    int ks = 1;
    // fewer tiles than SMs: cut K, at least two super-chunks per slice
    while (tiles * ks * 2 <= 148 && l.SC / (ks * 2) >= 2) ks *= 2;
    p.sc_per_slice = (l.SC + ks - 1) / ks;
    p.ks = (l.SC + p.sc_per_slice - 1) / p.sc_per_slice;
    return p;
}

template <int N>
cudaError_t launch_n(const Layout& l, const GemmCall& c, cudaStream_t s) {
    const size_t smem = 2 * kAStage + 2 * kBStage + (size_t)4 * Tab<N>::T * 128;
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done.set(dev);
    }
    const Plan p = plan_of(l, c.M);
    GemmArgs a;
    a.b = blob_at(c.packed, offsets_of(l));
    a.x = c.x; a.y = c.y;
    a.ctrl = (int*)c.workspace;
    a.partial = (float*)((char*)c.workspace + gemm_ctrl_bytes(l, c.M));
    a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.M = c.M; a.ell_slots = l.ell_slots;
    a.ks = p.ks; a.sc_per_slice = p.sc_per_slice; a.y_kind = c.y_kind;
    gemm_tc_kernel<N><<<dim3((unsigned)p.row_tiles, (unsigned)p.tok_tiles, (unsigned)p.ks), kWarps * 32, smem, s>>>(a);
    return cudaGetLastError();
}

}  // namespace

bool gemm_tc_supported(const Layout& l, int M) {
    return l.mode == 0 && M >= 1 && (long long)((M + kMaxT - 1) / kMaxT) <= 65535;
}

size_t gemm_ctrl_bytes(const Layout& l, int M) {
    const Plan p = plan_of(l, M);
    return align256((size_t)(1 + p.row_tiles * p.tok_tiles) * 4);
}

size_t gemm_workspace_bytes(const Layout& l, int M) {
    const Plan p = plan_of(l, M);
    const size_t partial = p.ks > 1 ? (size_t)p.row_tiles * p.tok_tiles * p.ks * kMaxT * kTileRows * 4 : 0;
    return gemm_ctrl_bytes(l, M) + partial;
}

cudaError_t launch_gemm_tc(const Layout& l, const GemmCall& c, cudaStream_t s) {
    switch (l.bits) {
        case 2: return launch_n<2>(l, c, s);
        case 3: return launch_n<3>(l, c, s);
        case 4: return launch_n<4>(l, c, s);
        case 5: return launch_n<5>(l, c, s);
        default: return launch_n<6>(l, c, s);
    }
}

}  // namespace xfp
