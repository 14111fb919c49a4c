// xfp_pack: unpacked tensors -> device layout (with range validation and clamping);
// xfp_dequant: device layout -> fp16 matrix W^ = fp16(D16 + S), bit-exact.
#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

// ------------------------------------------------------------------------------------ pack

// One thread per (row-block, super-chunk, lane): 128 byte-indices of one channel -> N uint4.
template <int N>
__global__ void __launch_bounds__(128) pack_idx_kernel(const uint8_t* __restrict__ idx, uint4* __restrict__ out,
                                                       int rows, int cols, int RB, int SC, int* err_word) {
    constexpr uint32_t E = 1u << N;
    const int lane = threadIdx.x & 31;
    const long long unit = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (unit >= (long long)RB * SC) return;
    const int rb = (int)(unit / SC), sc = (int)(unit % SC);
    const int row = rb * kRowsPerBlock + lane;
    uint32_t w[4 * N + 1];
#pragma unroll
    for (int i = 0; i < 4 * N + 1; ++i) w[i] = 0u;
    bool bad = false;
    if (row < rows) {
        const uint4* src = (const uint4*)(idx + (size_t)row * cols + (size_t)sc * kSuper);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint4 t = __ldg(src + i);
            const uint32_t tw[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                uint32_t q = (tw[b >> 2] >> ((b & 3) * 8)) & 0xffu;
                bad |= (q >= E);
                q &= E - 1u;
                const int j = i * 16 + b;
                const int bit = j * N, wi = bit >> 5, off = bit & 31;
                w[wi] |= q << off;
                if (off + N > 32) w[wi + 1] |= q >> (32 - off);
            }
        }
    }
    if (bad && err_word) atomicOr(err_word, 1);
    uint4* dst = out + ((size_t)unit * N) * 32 + lane;
#pragma unroll
    for (int v = 0; v < N; ++v) dst[(size_t)v * 32] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
}

__global__ void pack_codebook_kernel(const uint16_t* __restrict__ cb, uint16_t* __restrict__ out, long long n_src,
                                     long long n_dst) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n_dst) out[t] = t < n_src ? cb[t] : (uint16_t)0;
}

__global__ void pack_group_kernel(const uint8_t* __restrict__ gid, const uint16_t* __restrict__ gscale,
                                  const uint16_t* __restrict__ gmid, uint8_t* __restrict__ out_gid,
                                  uint32_t* __restrict__ out_gsm, int rows, int RB, int SC, int L, int G, int GH,
                                  int* err_word) {
    // one thread per (row-block, super-chunk, part of the super-chunk, lane); the group that holds the part's first
    // weight supplies its metadata (a group of 256 weights is stored with both of its super-chunks)
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (long long)RB * SC * GH * 32) return;
    const int lane = (int)(t & 31);
    const long long part = t >> 5;
    const long long unit = part / GH;
    const int h = (int)(part % GH);
    const int rb = (int)(unit / SC), sc = (int)(unit % SC);
    const int row = rb * kRowsPerBlock + lane;
    const int groups = SC * kSuper / G;                        // groups per channel
    const int grp = (sc * kSuper + h * (kSuper / GH)) / G;
    uint32_t id = 0, sm = 0;
    if (row < rows) {
        id = gid[(size_t)row * groups + grp];
        if ((int)id >= L) {
            if (err_word) atomicOr(err_word, 2);
            id = (uint32_t)(L - 1);
        }
        sm = (uint32_t)gscale[(size_t)row * groups + grp] | ((uint32_t)gmid[(size_t)row * groups + grp] << 16);
    }
    out_gid[t] = (uint8_t)id;
    out_gsm[t] = sm;
}

__device__ __forceinline__ int clampi(long long v, long long lo, long long hi) {
    return (int)(v < lo ? lo : (v > hi ? hi : v));
}

// rowptr -> clamped copy (padding rows empty); checks monotonicity and the end points;
// each thread also checks that its row's columns ascend strictly.
__global__ void pack_rowptr_kernel(const int32_t* __restrict__ rowptr, const void* __restrict__ ocol, int col_bits,
                                   int* __restrict__ out, int rows, int rows_pad, long long nnz, int* err_word) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t > rows_pad) return;
    if (rowptr == nullptr) {  // nnz == 0
        out[t] = 0;
        return;
    }
    int bad = 0;
    long long v = t <= rows ? (long long)rowptr[t] : nnz;
    if (t == 0 && v != 0) bad |= 4;
    if (t == rows && v != nnz) bad |= 4;
    if (v < 0 || v > nnz) bad |= 4;
    if (t < rows) {
        long long nx = rowptr[t + 1];
        if (nx < v) bad |= 4;
        const int p0 = clampi(v, 0, nnz), p1 = clampi(nx, 0, nnz);
        long long prev = -1;
        for (int p = p0; p < p1; ++p) {
            const long long c = col_bits == 16 ? (long long)((const uint16_t*)ocol)[p] : (long long)((const int32_t*)ocol)[p];
            if (c <= prev) bad |= 16;
            prev = c;
        }
    }
    out[t] = clampi(v, 0, nnz);
    if (bad && err_word) atomicOr(err_word, bad);
}

__global__ void pack_entries_kernel(const void* __restrict__ ocol, int col_bits, const uint16_t* __restrict__ oval,
                                    uint32_t* __restrict__ out, long long nnz, int cols, int* err_word) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= nnz) return;
    long long c = col_bits == 16 ? (long long)((const uint16_t*)ocol)[p] : (long long)((const int32_t*)ocol)[p];
    uint32_t v = oval[p];
    if (c < 0 || c >= cols) {  // neutralise: column 0, value +0
        if (err_word) atomicOr(err_word, 8);
        c = 0;
        v = 0;
    }
    out[p] = (uint32_t)c | (v << 16);
}

// Transposed outlier slab of row-block b (one CTA of 8 warps per block, the slots dealt to the warps): word [0][lane]
// = slots used by channel b*32+lane, word [1+j][lane] = its j-th outlier or the neutral entry (column 0, value +0).
__global__ void __launch_bounds__(256) ell_fill_kernel(const int* __restrict__ rp, const uint32_t* __restrict__ oent,
                                                       uint32_t* __restrict__ ell, int RB, int C) {
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (b >= RB) return;
    const int p0 = rp[b * 32 + lane], p1 = rp[b * 32 + lane + 1];
    const int len = p1 > p0 ? min(p1 - p0, C) : 0;
    uint32_t* slab = ell + (size_t)b * (C + 1) * 32 + lane;
    if (warp == 0) slab[0] = (uint32_t)len;
    for (int j = warp; j < C; j += 8) slab[(size_t)(1 + j) * 32] = j < len ? oent[p0 + j] : 0u;
}

__global__ void pack_header_kernel(int* hdr, int ell_slots, long long off_ell) {
    if (threadIdx.x == 0) {
        hdr[0] = ell_slots;
        hdr[1] = 0;
        *(long long*)(hdr + 2) = off_ell;
    }
}

template <int N>
static void launch_pack_idx(const Layout& l, const uint8_t* idx, uint4* out, int* err, cudaStream_t s) {
    const long long units = (long long)l.RB * l.SC;
    const unsigned grid = (unsigned)((units + 3) / 4);
    pack_idx_kernel<N><<<grid, 128, 0, s>>>(idx, out, l.rows, l.cols, l.RB, l.SC, err);
}

cudaError_t launch_pack(const Layout& l, const PackInputs& in, void* packed, int* err_word, cudaStream_t s) {
    char* base = (char*)packed;
    uint4* oidx = (uint4*)(base + l.off_idx);
    switch (l.bits) {
        case 2: launch_pack_idx<2>(l, in.idx, oidx, err_word, s); break;
        case 3: launch_pack_idx<3>(l, in.idx, oidx, err_word, s); break;
        case 4: launch_pack_idx<4>(l, in.idx, oidx, err_word, s); break;
        case 5: launch_pack_idx<5>(l, in.idx, oidx, err_word, s); break;
        default: launch_pack_idx<6>(l, in.idx, oidx, err_word, s); break;
    }
    const long long n_src = (long long)(l.mode ? l.L : l.rows) * l.E;
    const long long n_dst = (long long)(l.mode ? l.L : l.rows_pad) * l.E;
    pack_codebook_kernel<<<(unsigned)((n_dst + 255) / 256), 256, 0, s>>>(in.codebook, (uint16_t*)(base + l.off_cb), n_src,
                                                                        n_dst);
    if (l.mode) {
        const long long n = (long long)l.RB * l.SC * l.GH * 32;
        pack_group_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(in.gid, in.gscale, in.gmid,
                                                                     (uint8_t*)(base + l.off_gid),
                                                                     (uint32_t*)(base + l.off_gsm), l.rows, l.RB, l.SC,
                                                                     l.L, l.G, l.GH, err_word);
    }
    pack_rowptr_kernel<<<(unsigned)((l.rows_pad + 1 + 255) / 256), 256, 0, s>>>(
        l.nnz ? in.rowptr : nullptr, in.ocol, in.col_bits, (int*)(base + l.off_rowptr), l.rows, l.rows_pad, l.nnz,
        err_word);
    pack_header_kernel<<<1, 32, 0, s>>>((int*)(base + l.off_hdr), l.ell_slots, (long long)l.off_ell);
    if (l.nnz) {
        pack_entries_kernel<<<(unsigned)((l.nnz + 255) / 256), 256, 0, s>>>(in.ocol, in.col_bits, in.oval,
                                                                           (uint32_t*)(base + l.off_oent), l.nnz,
                                                                           l.cols, err_word);
        ell_fill_kernel<<<(unsigned)l.RB, 256, 0, s>>>((const int*)(base + l.off_rowptr),
                                                                   (const uint32_t*)(base + l.off_oent),
                                                                   (uint32_t*)(base + l.off_ell), l.RB, l.ell_slots);
    }
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ dequant

constexpr int kTileStride = 130;  // halves per tile row: 65 words, so 32 lanes hit 32 banks

// One warp per (row-block, super-chunk): each lane decodes the 128 values of its channel into a
// shared tile, then the warp writes the tile row by row (256 contiguous bytes per row).
template <int N, int MODE>
__global__ void __launch_bounds__(128) dequant_kernel(Blob b, uint16_t* __restrict__ W, int rows, int cols, int RB,
                                                      int SC, int GH) {
    constexpr int E = 1 << N;
    __shared__ uint16_t tile[4][32 * kTileStride];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long unit = (long long)blockIdx.x * 4 + warp;
    if (unit >= (long long)RB * SC) return;
    const int rb = (int)(unit / SC), sc = (int)(unit % SC);
    const int row = rb * kRowsPerBlock + lane;
    uint32_t w[4 * N + 1];
    const uint4* src = b.idx + ((size_t)unit * N) * 32 + lane;
#pragma unroll
    for (int v = 0; v < N; ++v) {
        const uint4 t = ld_stream(src + (size_t)v * 32);
        w[4 * v] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
    }
    w[4 * N] = 0u;
    uint16_t* trow = &tile[warp][lane * kTileStride];
    if (MODE == 0) {
        const uint16_t* cb = b.cb + (size_t)row * E;  // padding rows exist in the blob
#pragma unroll
        for (int j = 0; j < kSuper; ++j) trow[j] = __ldg(cb + field<N>(w, j));
    } else {
        // one group per super-chunk, or two groups of 64 weights (GH = 2)
        const size_t m0 = ((size_t)unit * GH) * 32 + lane, m1 = ((size_t)unit * GH + (GH - 1)) * 32 + lane;
        const uint32_t id0 = b.gid[m0], sm0 = b.gsm[m0], id1 = b.gid[m1], sm1 = b.gsm[m1];
#pragma unroll
        for (int j = 0; j < kSuper; ++j) {
            const uint32_t id = j < kSuper / 2 ? id0 : id1, sm = j < kSuper / 2 ? sm0 : sm1;
            const float scale = h2f((uint16_t)(sm & 0xffffu)), mid = h2f((uint16_t)(sm >> 16));
            // scale*lib is exact in fp32; one fp32 rounding for the sum, one fp16 rounding after it
            const float d = __fmaf_rn(scale, h2f(__ldg(b.cb + (size_t)id * E + field<N>(w, j))), mid);
            trow[j] = f2h(d);
        }
    }
    __syncwarp();
    for (int r = 0; r < 32; ++r) {
        const int orow = rb * kRowsPerBlock + r;
        if (orow >= rows) break;
        const uint32_t* srow = (const uint32_t*)&tile[warp][r * kTileStride];
        uint32_t* drow = (uint32_t*)(W + (size_t)orow * cols + (size_t)sc * kSuper);
        drow[lane] = srow[lane];
        drow[lane + 32] = srow[lane + 32];
    }
}

// The same for V2 blobs with the codebooks in shared memory.  The kernel above looks every weight up in global
// memory, one 2-byte load per lane with 32 distinct sectors per request, and that is what it is bound by (ncu: 49 M
// LSU wavefronts, the pipe 98 % busy, 183 us at 28672 x 8192).  Here a CTA of 8 warps takes one row-block and a
// range of super-chunks and stages the block's codebooks once, one word per lane and entry so that every look-up is
// conflict free: up to N = 3 as tables indexed by a PAIR of indices (one look-up yields the two fp16 values of a
// 4-byte tile store), above as one entry per index.  (A V2a variant with the library replicated per bank measured
// slower than the kernel above -- 64 KB of table fill per CTA, one CTA per SM -- and is not kept.)
template <int N>
__global__ void __launch_bounds__(256) dequant_lut_kernel(Blob b, uint16_t* W, int rows, int cols, int RB, int SC,
                                                          int sc_per_cta, int ell_slots) {
    constexpr int E = 1 << N;
    constexpr bool kPair = N <= 3;   // at N = 4 the 32 KB pair table costs a CTA per SM: slower than one entry per index
    constexpr int T = kPair ? E * E : E;
    constexpr int kWarps = 8;
    constexpr int kStrideW = 65;   // words per tile row: 32 lanes hit 32 banks
    extern __shared__ __align__(16) uint32_t dq_smem[];
    uint32_t* tab = dq_smem;                                        // [T][32]
    uint32_t* tiles = dq_smem + T * 32;                             // [kWarps][32 * kStrideW]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rb = blockIdx.x % RB, part = blockIdx.x / RB;
    const int sc_begin = part * sc_per_cta;
    const int sc_end = min(SC, sc_begin + sc_per_cta);
    {
        // the lane's codebook goes through the first tile (one word per entry), the pair table is built from there
        const uint16_t* cb = b.cb + (size_t)(rb * kRowsPerBlock + lane) * E;   // padding rows exist in the blob
        uint32_t* one = kPair ? tiles : tab;
        for (int e = warp; e < E; e += kWarps) one[e * 32 + lane] = __ldg(cb + e);
        if (kPair) {
            __syncthreads();
            for (int t = warp; t < T; t += kWarps)
                tab[t * 32 + lane] = one[(t & (E - 1)) * 32 + lane] | (one[(t >> N) * 32 + lane] << 16);
        }
    }
    __syncthreads();
    const uint32_t base = (uint32_t)lane * 4u;
    uint32_t* tile = tiles + warp * 32 * kStrideW;
    for (int sc = sc_begin + warp; sc < sc_end; sc += kWarps) {
        const size_t unit = (size_t)rb * SC + sc;
        uint32_t w[4 * N + 1];
        const uint4* src = b.idx + (unit * N) * 32 + lane;
#pragma unroll
        for (int v = 0; v < N; ++v) {
            const uint4 t = ld_stream(src + (size_t)v * 32);
            w[4 * v] = t.x; w[4 * v + 1] = t.y; w[4 * v + 2] = t.z; w[4 * v + 3] = t.w;
        }
        w[4 * N] = 0u;
        uint32_t* trow = tile + lane * kStrideW;
#pragma unroll
        for (int p = 0; p < kSuper / 2; ++p) {
            if (kPair) {
                trow[p] = *(const uint32_t*)((const unsigned char*)tab + pair_addr<N, 1>(w, p, base));
            } else {
                const uint32_t lo = *(const uint32_t*)((const unsigned char*)tab + single_addr<N, 1>(w, 2 * p, base));
                const uint32_t hi = *(const uint32_t*)((const unsigned char*)tab + single_addr<N, 1>(w, 2 * p + 1, base));
                trow[p] = lo | (hi << 16);
            }
        }
        __syncwarp();
#pragma unroll 4
        for (int r = 0; r < 32; ++r) {
            const int orow = rb * kRowsPerBlock + r;
            if (orow >= rows) break;
            const uint32_t* srow = tile + r * kStrideW;
            uint32_t* drow = (uint32_t*)(W + (size_t)orow * cols + (size_t)sc * kSuper);
            drow[lane] = srow[lane];
            drow[lane + 32] = srow[lane + 32];
        }
        __syncwarp();   // the tile is rewritten for the warp's next super-chunk
    }
    // W^ += S for the outliers of this row-block that fall into this CTA's columns: one correctly rounded fp16
    // addition each, on values this CTA has just written (ordered by the barrier).  Lane = channel; the slots of the
    // transposed slab are dealt to the warps; channels that overflow their slab finish from the CSR arrays.
    if (ell_slots == 0) return;
    __syncthreads();
    {
        const int row = rb * kRowsPerBlock + lane;
        const uint32_t* slab = b.ell + (size_t)rb * (ell_slots + 1) * 32 + lane;
        const int olen = (int)__ldg(slab);
        const uint32_t k0 = (uint32_t)sc_begin * kSuper, k1 = (uint32_t)sc_end * kSuper;
        auto add = [&](uint32_t e) {
            const uint32_t col = e & 0xffffu;
            if (row < rows && col >= k0 && col < k1) {
                uint16_t* dst = W + (size_t)row * cols + col;
                *dst = __half_as_ushort(__hadd(__ushort_as_half(*dst), __ushort_as_half((uint16_t)(e >> 16))));
            }
        };
        const int n_slab = min(olen, ell_slots);
        for (int j = warp; j < n_slab; j += kWarps) add(__ldg(slab + (size_t)(1 + j) * 32));
        if (warp == 0 && olen >= ell_slots && row < rows) {
            const int p1 = __ldg(b.rowptr + row + 1);
            for (int p = __ldg(b.rowptr + row) + ell_slots; p < p1; ++p) add(__ldg(b.oent + p));
        }
    }
}

// W^ += S at the outlier positions: one correctly rounded fp16 addition per outlier.
__global__ void dequant_outlier_kernel(Blob b, uint16_t* __restrict__ W, int rows, int cols) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const int p0 = b.rowptr[row], p1 = b.rowptr[row + 1];
    for (int p = p0 + lane; p < p1; p += 32) {
        const uint32_t e = b.oent[p];
        uint16_t* dst = W + (size_t)row * cols + (e & 0xffffu);
        const __half s = __hadd(__ushort_as_half(*dst), __ushort_as_half((uint16_t)(e >> 16)));
        *dst = __half_as_ushort(s);
    }
}

template <int N>
static bool launch_dequant_lut(const Layout& l, const Blob& b, uint16_t* W, cudaStream_t s, bool* outliers_done) {
    const size_t tab_bytes = (size_t)(N <= 3 ? l.E * l.E : l.E) * 128;
    const size_t smem = tab_bytes + (size_t)8 * 32 * 65 * 4;
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        if (cudaFuncSetAttribute(dequant_lut_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024) != cudaSuccess)
            return false;
        attr_done.set(dev);
    }
    // a CTA per row-block; row-blocks too few to fill the GPU are cut along K (at least 8 super-chunks per CTA)
    int parts = 1;
    const int sms = sm_count();
    while (l.RB * parts < 2 * sms && l.SC / (parts * 2) >= 8) parts *= 2;
    const int sc_per_cta = (l.SC + parts - 1) / parts;
    parts = (l.SC + sc_per_cta - 1) / sc_per_cta;
    // The outliers are added by the same kernel on small matrices (one launch less: 25.6 -> 23.5 us at 4096 x 4096);
    // on large ones the pass at the end of every CTA is a chain of dependent read-modify-writes and the separate
    // kernel, which spreads them over the whole GPU, is faster (181 against 191 us at 28672 x 8192, 0.3 %).
    const bool fuse_outliers = (long long)l.RB * l.SC <= (long long)sms * 64;
    dequant_lut_kernel<N><<<(unsigned)(l.RB * parts), 256, smem, s>>>(b, W, l.rows, l.cols, l.RB, l.SC, sc_per_cta,
                                                                      fuse_outliers ? l.ell_slots : 0);
    *outliers_done = fuse_outliers;
    return true;
}

// returns true when the kernel has added the outliers itself
template <int N>
static bool launch_dequant_n(const Layout& l, const Blob& b, uint16_t* W, cudaStream_t s) {
    bool done = false;
    if (l.mode == 0 && launch_dequant_lut<N>(l, b, W, s, &done)) return done;
    const long long units = (long long)l.RB * l.SC;
    const unsigned grid = (unsigned)((units + 3) / 4);
    if (l.mode == 0)
        dequant_kernel<N, 0><<<grid, 128, 0, s>>>(b, W, l.rows, l.cols, l.RB, l.SC, 1);
    else
        dequant_kernel<N, 1><<<grid, 128, 0, s>>>(b, W, l.rows, l.cols, l.RB, l.SC, l.GH);
    return false;
}

cudaError_t launch_dequant(const Layout& l, const void* packed, uint16_t* W, cudaStream_t s) {
    const Blob b = blob_at(packed, offsets_of(l));
    bool outliers_done = false;
    switch (l.bits) {
        case 2: outliers_done = launch_dequant_n<2>(l, b, W, s); break;
        case 3: outliers_done = launch_dequant_n<3>(l, b, W, s); break;
        case 4: outliers_done = launch_dequant_n<4>(l, b, W, s); break;
        case 5: outliers_done = launch_dequant_n<5>(l, b, W, s); break;
        default: outliers_done = launch_dequant_n<6>(l, b, W, s); break;
    }
    if (l.nnz && !outliers_done) dequant_outlier_kernel<<<(unsigned)((l.rows + 7) / 8), 256, 0, s>>>(b, W, l.rows, l.cols);
    return cudaGetLastError();
}

}  // namespace xfp
