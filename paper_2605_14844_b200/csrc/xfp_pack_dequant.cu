// xfp_pack: unpacked tensors -> device layout (with range validation and clamping);
// xfp_dequant: device layout -> fp16 matrix W^ = fp16(D16 + S), bit-exact.
#include <cstdlib>

#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

// ------------------------------------------------------------------------------------ pack
//
// One launch: the blocks of the grid are dealt to the six parts of the blob (index stream, codebooks, group
// metadata, row pointers, outlier entries, transposed slabs) by block index.  Every part reads the caller's tensors
// only -- the slabs apply the same clamping and neutralisation as the row pointers and entries they mirror -- so no
// part waits for another.  (As seven launches the small parts cost 28 of 94 us at 28672 x 8192 and set a floor of
// ~32 us on small matrices.)

constexpr int kPackThreads = 256;
constexpr int kPackWarps = kPackThreads / 32;

struct PackArgs {
    PackInputs in;
    char* base;             // the blob
    Layout l;
    int* err_word;
    // first block of every part, in this order: slabs, entries, rowptr, group, codebook, idx; [6] = grid.  (Spreading
    // the blocks of the small parts evenly among those of the index part measured the same: 110.6 against 106.5 us at
    // 28672 x 8192 with 2 % outliers.)
    unsigned first[7];
};

__device__ __forceinline__ int clampi(long long v, long long lo, long long hi) {
    return (int)(v < lo ? lo : (v > hi ? hi : v));
}

__device__ __forceinline__ long long col_at(const void* ocol, int col_bits, long long p) {
    return col_bits == 16 ? (long long)((const uint16_t*)ocol)[p] : (long long)((const int32_t*)ocol)[p];
}

// outlier p as the blob stores it: column | fp16 value << 16; a column outside the matrix becomes column 0, value +0
__device__ __forceinline__ uint32_t entry_at(const PackInputs& in, long long p, int cols, bool* bad) {
    long long c = col_at(in.ocol, in.col_bits, p);
    uint32_t v = in.oval[p];
    if (c < 0 || c >= cols) { *bad = true; c = 0; v = 0; }
    return (uint32_t)c | (v << 16);
}

// One warp per (row-block, super-chunk): 128 byte-indices of every channel -> N uint4 per lane.  The warp fetches its
// 32 x 128-byte tile of indices with whole 128-byte lines per quarter-warp and hands every lane its channel's row through
// shared memory (a lane reading its own row from global memory made every 16-byte load a line of its own: 16.3 M
// wavefronts on the L1 data pipe at 28672 x 8192 against 7.6 M this way).
template <int N>
__device__ __forceinline__ void pack_idx_block(const PackArgs& a, unsigned vblk, unsigned char* tiles) {
    constexpr uint32_t E = 1u << N;
    constexpr int kRowB = 144;   // bytes per tile row: 16-byte aligned, the lanes of a quarter-warp in distinct banks
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long unit = (long long)vblk * kPackWarps + warp;
    if (unit >= (long long)a.l.RB * a.l.SC) return;
    const int rb = (int)(unit / a.l.SC), sc = (int)(unit % a.l.SC);
    unsigned char* tile = tiles + warp * 32 * kRowB;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + (lane >> 3), c = lane & 7;   // rows 4i .. 4i+3 of the tile, 16-byte chunk c
        const int row_g = rb * kRowsPerBlock + r;
        uint4 t = make_uint4(0u, 0u, 0u, 0u);
        if (row_g < a.l.rows) t = __ldg((const uint4*)(a.in.idx + (size_t)row_g * a.l.cols + (size_t)sc * kSuper) + c);
        *(uint4*)(tile + r * kRowB + c * 16) = t;
    }
    __syncwarp();
    uint32_t w[4 * N + 1];
#pragma unroll
    for (int i = 0; i < 4 * N + 1; ++i) w[i] = 0u;
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint4 t = *(const uint4*)(tile + lane * kRowB + i * 16);
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
    if (bad && a.err_word) atomicOr(a.err_word, 1);
    uint4* dst = (uint4*)(a.base + a.l.off_idx) + ((size_t)unit * N) * 32 + lane;
#pragma unroll
    for (int v = 0; v < N; ++v) dst[(size_t)v * 32] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
}

__device__ __forceinline__ void pack_codebook_block(const PackArgs& a, unsigned vblk) {
    const long long n_src = (long long)(a.l.mode ? a.l.L : a.l.rows) * a.l.E;
    const long long n_dst = (long long)(a.l.mode ? a.l.L : a.l.rows_pad) * a.l.E;
    const long long t = (long long)vblk * kPackThreads + threadIdx.x;
    uint16_t* out = (uint16_t*)(a.base + a.l.off_cb);
    if (t < n_dst) out[t] = t < n_src ? a.in.codebook[t] : (uint16_t)0;
}

__device__ __forceinline__ void pack_group_block(const PackArgs& a, unsigned vblk) {
    // one thread per (row-block, super-chunk, part of the super-chunk, lane); the group that holds the part's first
    // weight supplies its metadata (a group of 256 weights is stored with both of its super-chunks)
    const Layout& l = a.l;
    const long long t = (long long)vblk * kPackThreads + threadIdx.x;
    if (t >= (long long)l.RB * l.SC * l.GH * 32) return;
    const int lane = (int)(t & 31);
    const long long part = t >> 5;
    const long long unit = part / l.GH;
    const int h = (int)(part % l.GH);
    const int rb = (int)(unit / l.SC), sc = (int)(unit % l.SC);
    const int row = rb * kRowsPerBlock + lane;
    const int groups = l.SC * kSuper / l.G;                        // groups per channel
    const int grp = (sc * kSuper + h * (kSuper / l.GH)) / l.G;
    uint32_t id = 0, sm = 0;
    if (row < l.rows) {
        id = a.in.gid[(size_t)row * groups + grp];
        if ((int)id >= l.L) {
            if (a.err_word) atomicOr(a.err_word, 2);
            id = (uint32_t)(l.L - 1);
        }
        sm = (uint32_t)a.in.gscale[(size_t)row * groups + grp] | ((uint32_t)a.in.gmid[(size_t)row * groups + grp] << 16);
    }
    ((uint8_t*)(a.base + l.off_gid))[t] = (uint8_t)id;
    ((uint32_t*)(a.base + l.off_gsm))[t] = sm;
}

// rowptr -> clamped copy (padding rows empty); checks monotonicity and the end points (that the columns of a row
// ascend strictly is checked where the entries are read in order, in ell_fill_block).  The first thread writes the
// header words.
__device__ __forceinline__ void pack_rowptr_block(const PackArgs& a, unsigned vblk) {
    const Layout& l = a.l;
    const int t = (int)(vblk * kPackThreads + threadIdx.x);
    if (t == 0) {
        int* hdr = (int*)(a.base + l.off_hdr);
        hdr[0] = l.ell_slots;
        hdr[1] = 0;
        *(long long*)(hdr + 2) = (long long)l.off_ell;
    }
    if (t > l.rows_pad) return;
    int* out = (int*)(a.base + l.off_rowptr);
    if (l.nnz == 0) {
        out[t] = 0;
        return;
    }
    const long long nnz = l.nnz;
    int bad = 0;
    long long v = t <= l.rows ? (long long)a.in.rowptr[t] : nnz;
    if (t == 0 && v != 0) bad |= 4;
    if (t == l.rows && v != nnz) bad |= 4;
    if (v < 0 || v > nnz) bad |= 4;
    if (t < l.rows) {
        long long nx = a.in.rowptr[t + 1];
        if (nx < v) bad |= 4;
    }
    out[t] = clampi(v, 0, nnz);
    if (bad && a.err_word) atomicOr(a.err_word, bad);
}

__device__ __forceinline__ void pack_entries_block(const PackArgs& a, unsigned vblk) {
    const long long p = (long long)vblk * kPackThreads + threadIdx.x;
    if (p >= a.l.nnz) return;
    bool bad = false;
    ((uint32_t*)(a.base + a.l.off_oent))[p] = entry_at(a.in, p, a.l.cols, &bad);
    if (bad && a.err_word) atomicOr(a.err_word, 8);
}

// Transposed outlier slab of row-block b: word [0][lane] = slots used by channel b*32+lane, word [1+j][lane] = its
// j-th outlier or the neutral entry (column 0, value +0).  Reads the caller's row pointers and entries with the
// clamping of pack_rowptr_block and pack_entries_block.  The block's entries are one contiguous range of the CSR
// arrays: a warp takes a channel and reads its entries in order (coalesced), each entry goes to its slot of a copy of
// the slab in shared memory (windows of 256 slots), which is then written out in whole lines.  (Every lane walking its
// own row -- 32 scattered sectors per load --, scattered 4-byte stores into the slab, and a binary search of every
// entry for its channel each made this part 50-60 us at 2 % outliers on 28672 x 8192.)  The same pass checks that the
// columns of a row ascend strictly.  Row pointers that do not ascend (reported by pack_rowptr_block) leave slots
// neutral, never an access outside the arrays.
constexpr int kEllWindow = 256;   // slots of the slab held in shared memory at a time
__device__ __forceinline__ void ell_fill_block(const PackArgs& a, unsigned b, unsigned char* smem) {
    const Layout& l = a.l;
    uint32_t* sl = (uint32_t*)smem;                       // [kEllWindow][33]: consecutive slots of one channel in consecutive banks
    int* rp = (int*)(smem + kEllWindow * 33 * 4);         // [33]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int C = l.ell_slots;
    const long long nnz = l.nnz;
    if (threadIdx.x < 33) {
        const int row = (int)b * 32 + (int)threadIdx.x;
        rp[threadIdx.x] = row <= l.rows ? clampi(a.in.rowptr[row], 0, nnz) : (int)nnz;
    }
    __syncthreads();
    uint32_t* slab = (uint32_t*)(a.base + l.off_ell) + (size_t)b * (C + 1) * 32;
    if (warp == 0) {
        const int p0 = rp[lane], p1 = rp[lane + 1];
        slab[lane] = (uint32_t)(p1 > p0 ? min(p1 - p0, C) : 0);
    }
    int bad = 0;   // a column outside the matrix is reported by pack_entries_block
    for (int j0 = 0; j0 < C; j0 += kEllWindow) {
        const int nj = min(kEllWindow, C - j0);
        for (int i = threadIdx.x; i < nj * 33; i += kPackThreads) sl[i] = 0u;
        __syncthreads();
        for (int r = warp; r < 32; r += kPackWarps) {   // a warp per channel, its lanes along the channel's entries
            const int p0 = rp[r], n = rp[r + 1] - p0;   // n <= 0: an empty channel, or row pointers that descend
            for (int jj = lane; jj < n; jj += 32) {
                const int p = p0 + jj;
                if (j0 == 0 && jj > 0 && col_at(a.in.ocol, a.in.col_bits, p) <= col_at(a.in.ocol, a.in.col_bits, p - 1)) bad = 16;
                bool outside = false;
                if (jj >= j0 && jj < j0 + nj) sl[(jj - j0) * 33 + r] = entry_at(a.in, p, l.cols, &outside);
            }
        }
        __syncthreads();
        for (int i = threadIdx.x; i < nj * 32; i += kPackThreads) slab[(size_t)(1 + j0) * 32 + i] = sl[(i >> 5) * 33 + (i & 31)];
        __syncthreads();
    }
    if (bad && a.err_word) atomicOr(a.err_word, bad);
}

template <int N>
__global__ void __launch_bounds__(kPackThreads) pack_kernel(const PackArgs a) {
    __shared__ __align__(16) unsigned char tiles[kPackWarps * 32 * 144];   // 36864 bytes; the slab part uses 33792 + 132
    static_assert(kPackWarps * 32 * 144 >= kEllWindow * 33 * 4 + 33 * 4, "slab window and row pointers fit the tile area");
    const unsigned b = blockIdx.x;
    if (b < a.first[1]) ell_fill_block(a, b, tiles);
    else if (b < a.first[2]) pack_entries_block(a, b - a.first[1]);
    else if (b < a.first[3]) pack_rowptr_block(a, b - a.first[2]);
    else if (b < a.first[4]) pack_group_block(a, b - a.first[3]);
    else if (b < a.first[5]) pack_codebook_block(a, b - a.first[4]);
    else pack_idx_block<N>(a, b - a.first[5], tiles);
}

cudaError_t launch_pack(const Layout& l, const PackInputs& in, void* packed, int* err_word, cudaStream_t s) {
    PackArgs a;
    a.in = in; a.base = (char*)packed; a.l = l; a.err_word = err_word;
    auto blocks = [](long long n, int per) { return (unsigned)((n + per - 1) / per); };
    const long long n_cb = (long long)(l.mode ? l.L : l.rows_pad) * l.E;
    unsigned n[6];
    n[0] = l.nnz ? (unsigned)l.RB : 0u;
    n[1] = l.nnz ? blocks(l.nnz, kPackThreads) : 0u;
    n[2] = blocks((long long)l.rows_pad + 1, kPackThreads);
    n[3] = l.mode ? blocks((long long)l.RB * l.SC * l.GH * 32, kPackThreads) : 0u;
    n[4] = blocks(n_cb, kPackThreads);
    n[5] = blocks((long long)l.RB * l.SC, kPackWarps);
#ifdef LANE_TUNE
    if (const char* e = getenv("XFP_PACK_SKIP"))   // tuning build: leave parts out (bit i = part i) to time the others
        for (int i = 0; i < 6; ++i)
            if ((atoi(e) >> i) & 1) n[i] = 0;
#endif
    a.first[0] = 0;
    for (int i = 0; i < 6; ++i) a.first[i + 1] = a.first[i] + n[i];
    switch (l.bits) {
        case 2: pack_kernel<2><<<a.first[6], kPackThreads, 0, s>>>(a); break;
        case 3: pack_kernel<3><<<a.first[6], kPackThreads, 0, s>>>(a); break;
        case 4: pack_kernel<4><<<a.first[6], kPackThreads, 0, s>>>(a); break;
        case 5: pack_kernel<5><<<a.first[6], kPackThreads, 0, s>>>(a); break;
        default: pack_kernel<6><<<a.first[6], kPackThreads, 0, s>>>(a); break;
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
    // the index vectors of a warp's next super-chunk travel while it decodes the current one
    uint4 nx[N];
    if (sc_begin + warp < sc_end) {
        const uint4* src = b.idx + (((size_t)rb * SC + sc_begin + warp) * N) * 32 + lane;
#pragma unroll
        for (int v = 0; v < N; ++v) nx[v] = ld_stream(src + (size_t)v * 32);
    }
    for (int sc = sc_begin + warp; sc < sc_end; sc += kWarps) {
        uint32_t w[4 * N + 1];
#pragma unroll
        for (int v = 0; v < N; ++v) { w[4 * v] = nx[v].x; w[4 * v + 1] = nx[v].y; w[4 * v + 2] = nx[v].z; w[4 * v + 3] = nx[v].w; }
        w[4 * N] = 0u;
        if (sc + kWarps < sc_end) {
            const uint4* src = b.idx + (((size_t)rb * SC + sc + kWarps) * N) * 32 + lane;
#pragma unroll
            for (int v = 0; v < N; ++v) nx[v] = ld_stream(src + (size_t)v * 32);
        }
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
