// Batched fused decode, 3..16 rows of x, for V2 and V2a blobs:  y[b] = (D + S) x[b].
//
// Same decode as xfp_gemv_pair.cu (tables in per-lane shared-memory banks, looked-up half2 used directly as the A
// fragment of mma.sync.m16n8k16, x on the diagonal lanes of the B fragment), but every decoded fragment is
// multiplied with NB/2 B fragments, one per pair of batch rows: the look-ups, which bound the kernel, are paid
// once per weight whatever the batch.  Here the tensor pipe does real work (NB/2 mma per 8 weights of a lane),
// the reason the paper's step 4 is a tensor core GEMM.
//
// MODE 0 (V2): pair tables of the lanes' own channels.  MODE 1 (V2a, "V2a: Shared Codebook Library"):
//     y[b][i] = sum_g [ scale_ig * sum_{k in g} lib[id_ig][q_ik] x[b][k]  +  mid_ig * sum_{k in g} x[b][k] ]  +  (S x[b])_i
// with the library replicated once per shared-memory bank (word (id * 2^N + q) * 32 + lane), one look-up per weight
// and a PRMT joining two of them into a half2; the fragments accumulate the sums of ONE 128-weight group, which
// then move to the lanes that own the channels and are folded into fp32 accumulators with the group's scale and
// mid-point, acc[b] += scale * G[b] + mid * X_g[b] (X_g[b]: sum of x[b] over the group, computed once per CTA from
// the staged copy of x).  Nothing is rounded to fp16 on the way.
//
// x is staged in shared memory as 16-byte chunks ordered [k / 8][batch row], so the two diagonal lane groups of a
// batch pair read adjacent chunks (one wavefront) and outlier columns are gathered from the same copy.  One CTA
// per SM (16 warps): tables + x take up to ~200 KB.  After the K loop the x area is reused for the cross-warp
// reduction.  Batches above 8 run as two tiles.
#include "xfp_internal.h"
#include "xfp_pair_common.cuh"

namespace xfp {

constexpr int kBWarps = 16;
constexpr int kBThreads = kBWarps * 32;
constexpr int kBSlots = 4;

struct BatchArgs {
    Offsets off;
    const void* packed;
    const uint16_t* x;
    void* y;
    float* partial;  // [KS][NB][rows_ws]
    int* tickets;    // [blocks]
    int rows, cols, RB, SC, rows_ws, ell_slots, L;
    int nb, y_is_fp16, x_bf16;
    int n_full, kst, sc_per_split;
};

// byte offset of x[bb][k] in the staged copy: chunk (k / 8) * NB + (bb ^ (k / 8 mod NB)), 8 halves per chunk.  The
// swizzle of the row inside a chunk group lets eight consecutive lanes stage eight consecutive chunks of ONE row
// (one 128-byte line per quarter-warp instead of eight) without meeting in the same banks when they store.
template <int NB>
__device__ __forceinline__ uint32_t xoff(int bb, uint32_t k) {
    const uint32_t k8 = k >> 3;
    return ((k8 * NB + ((uint32_t)bb ^ (k8 & (uint32_t)(NB - 1)))) << 4) + ((k & 7u) << 1);
}

// Byte offset (q << 7) of index j (compile time) of a 128-weight stream, merged with `base`
// (= id * 2^N * 128 + lane * 4; the q field occupies bits 7 .. 7+N, which base leaves clear).
template <int N>
__device__ __forceinline__ uint32_t lib_entry_addr(const uint32_t* w, int j, uint32_t base) {
    constexpr uint32_t mask = ((1u << N) - 1u) << 7;
    const int bit = j * N, wi = bit >> 5, off = bit & 31;
    uint32_t v;
    if (off + N > 32)
        v = __funnelshift_r(w[wi], w[wi + 1], off - 7);   // field straight to bit 7 (off > 7 whenever it straddles)
    else if (off >= 7)
        v = w[wi] >> (off - 7);
    else
        v = w[wi] << (7 - off);
    return (v & mask) | base;
}

template <int N, int NB, int RPL, bool TIO, int MODE>
__global__ void __launch_bounds__(kBThreads, 1) gemv_batch_kernel(const BatchArgs a) {
    static_assert(MODE == 0 || RPL == 2, "V2a blocks hold two channels per lane");
    constexpr int E = 1 << N;
    constexpr int T = E * E;
    constexpr int ROWS = 32 * RPL;
    constexpr int kStride = 128 * RPL;
    constexpr int NBP = NB / 2;   // batch pairs
    constexpr int W = kBWarps;
    extern __shared__ __align__(16) unsigned char smem[];
    // V2:  [pair tables | x chunks (NB * K * 2 bytes), later red[W][NB][ROWS] fp32]
    // V2a: [library L*E*128 bytes | xg fp32 [NB][SC] | x chunks, later red]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    int blk, ks, KS, spp;
    if ((int)blockIdx.x < a.n_full) {
        blk = blockIdx.x; ks = 0; KS = 1; spp = a.SC;
    } else {
        const int t = blockIdx.x - a.n_full;
        blk = a.n_full + t / a.kst; ks = t % a.kst; KS = a.kst; spp = a.sc_per_split;
    }
    const Blob b = blob_at(a.packed, a.off);
    const int sc0 = ks * spp;
    const int nsc = max(0, min(a.SC, sc0 + spp) - sc0);
    const int K = a.SC * kSuper;

    const int tab_bytes = MODE == 1 ? a.L * E * 128 : T * kStride;
    unsigned char* tab = smem;
    float* xg = (float*)(smem + tab_bytes);                                  // V2a: [NB][SC]
    unsigned char* xs = smem + tab_bytes + (MODE == 1 ? (((size_t)NB * a.SC * 4 + 15) & ~(size_t)15) : 0);
    float* red = (float*)xs;

    const int blk0 = RPL * blk;
    const int blk1 = min(RPL * blk + (RPL - 1), a.RB - 1);

    // ---- (0) first super-chunk of this warp, first outlier slots
    uint32_t w0[4 * N + 1], w1[RPL == 2 ? 4 * N + 1 : 1];
    w0[4 * N] = 0u;
    if (RPL == 2) w1[4 * N] = 0u;
    const uint4* i0 = b.idx + ((size_t)(blk0 * a.SC + sc0) * N) * 32 + lane;
    const uint4* i1 = b.idx + ((size_t)(blk1 * a.SC + sc0) * N) * 32 + lane;
    // V2a: library ids and (scale, mid) of the two channels' current and next group
    const size_t m0 = (size_t)(blk0 * a.SC + sc0) * 32 + lane, m1 = (size_t)(blk1 * a.SC + sc0) * 32 + lane;
    uint32_t id0 = 0, id1 = 0, sm0 = 0, sm1 = 0, nid0 = 0, nid1 = 0, nsm0 = 0, nsm1 = 0;
    if (warp < nsc) {
#pragma unroll
        for (int v = 0; v < N; ++v) {
            const uint4 t0 = ld_stream(i0 + ((size_t)warp * N + v) * 32);
            w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
            if (RPL == 2) {
                const uint4 t1 = ld_stream(i1 + ((size_t)warp * N + v) * 32);
                w1[4 * v] = t1.x; w1[4 * v + 1] = t1.y; w1[4 * v + 2] = t1.z; w1[4 * v + 3] = t1.w;
            }
        }
        if (MODE == 1) {
            id0 = b.gid[m0 + (size_t)warp * 32]; id1 = b.gid[m1 + (size_t)warp * 32];
            sm0 = b.gsm[m0 + (size_t)warp * 32]; sm1 = b.gsm[m1 + (size_t)warp * 32];
        }
    }
    const int gw = ks * W + warp, ostride = KS * W;
    const uint32_t* slab[RPL];
    int width[RPL];
    uint32_t olen[RPL];
    uint32_t oe[RPL][kBSlots];
    float oacc[NB][RPL];
    int oround = 0, nrounds = 0;
#pragma unroll
    for (int h = 0; h < RPL; ++h) {
        slab[h] = b.ell + (size_t)(h ? blk1 : blk0) * (a.ell_slots + 1) * 32 + lane;
        width[h] = a.ell_slots;
        olen[h] = a.ell_slots ? __ldg(slab[h]) : 0u;
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) oacc[bb][h] = 0.f;
    }
    auto fetch_slots = [&](int round) {
#pragma unroll
        for (int h = 0; h < RPL; ++h)
#pragma unroll
            for (int q = 0; q < kBSlots; ++q) {
                const int j = gw + (round * kBSlots + q) * ostride;
                oe[h][q] = j < width[h] ? __ldg(slab[h] + (size_t)(1 + j) * 32) : 0u;
            }
    };
    auto consume_slots = [&]() {
#pragma unroll
        for (int h = 0; h < RPL; ++h)
#pragma unroll
            for (int q = 0; q < kBSlots; ++q) {
                const float v = h2f((uint16_t)(oe[h][q] >> 16));
                const uint32_t col = oe[h][q] & 0xffffu;
#pragma unroll
                for (int bb = 0; bb < NB; ++bb)
                    oacc[bb][h] = fmaf(v, h2f(*(const uint16_t*)(xs + xoff<NB>(bb, col))), oacc[bb][h]);
            }
    };
    if (a.ell_slots) fetch_slots(0);

    // ---- (1) tables.  V2a: the library, one copy per bank (word e * 32 + lane = lib[e] for every lane).
    //      V2: pair tables, warp w fills entries [w*T/W, (w+1)*T/W) of every channel half
    if (MODE == 1) {
        for (int e = warp; e < a.L * E; e += W)
            *(uint32_t*)(tab + (size_t)e * 128 + lane * 4) = (uint32_t)__ldg(b.cb + e);
    } else {
        constexpr int TW = T / W;
#pragma unroll
        for (int half = 0; half < RPL; ++half) {
            const uint16_t* cb = b.cb + (size_t)((half ? blk1 : blk0) * kRowsPerBlock + lane) * E;
            unsigned char* dst = tab + half * 128 + lane * 4;
            if (TW >= E) {
                uint32_t c[E / 2];
#pragma unroll
                for (int i = 0; i < E / 8; ++i) {
                    const uint4 t = __ldg((const uint4*)cb + i);
                    c[4 * i] = t.x; c[4 * i + 1] = t.y; c[4 * i + 2] = t.z; c[4 * i + 3] = t.w;
                }
#pragma unroll
                for (int hh = 0; hh < TW / E; ++hh) {
                    const int hi = warp * (TW / E) + hh;
                    const uint32_t hv = __ldg(cb + hi);
#pragma unroll
                    for (int lo = 0; lo < E; ++lo) {
                        const uint32_t lv = (lo & 1) ? (c[lo >> 1] >> 16) : (c[lo >> 1] & 0xffffu);
                        *(uint32_t*)(dst + (size_t)(hi * E + lo) * kStride) = lv | (hv << 16);
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < (TW > 0 ? TW : 1); ++i) {
                    const int t = TW > 0 ? warp * TW + i : warp;
                    if (t < T) {
                        const uint32_t lv = __ldg(cb + (t & (E - 1))), hv = __ldg(cb + (t >> N));
                        *(uint32_t*)(dst + (size_t)t * kStride) = lv | (hv << 16);
                    }
                }
            }
        }
    }
    // ---- (2) x: chunk t = (k / 8) * NB + bb  <-  x[bb][8 (k/8) .. +8]
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int t = threadIdx.x; t < NB * (K / 8); t += kBThreads) {
        // eight consecutive lanes: eight consecutive chunks of one row (K / 8 is a multiple of 16)
        const int grp = t >> 3, bb = grp % NB, k8 = (grp / NB) * 8 + (t & 7);
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (bb < a.nb) v = __ldg((const uint4*)(a.x + (size_t)bb * a.cols + (size_t)k8 * 8));
        if (TIO) v = x8_as_f16(v, a.x_bf16);
        *(uint4*)(xs + xoff<NB>(bb, (uint32_t)k8 * 8u)) = v;
    }
#pragma unroll
    for (int h = 0; h < RPL; ++h) {
        int wmax = (int)olen[h];
#pragma unroll
        for (int o = 16; o; o >>= 1) wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
        width[h] = min(wmax, a.ell_slots);
        const int mine = width[h] > gw ? (width[h] - gw + ostride - 1) / ostride : 0;
        nrounds = max(nrounds, (mine + kBSlots - 1) / kBSlots);
    }
    __syncthreads();
    if (MODE == 1) {
        // X_g[bb]: the 128 values of group u are 16 chunks of 8; lane l sums 4 of them, then a fixed butterfly
        for (int u = warp; u < NB * a.SC; u += W) {
            const int bb = u / a.SC, gq = u - bb * a.SC;
            const uint2 hv = *(const uint2*)(xs + xoff<NB>(bb, (uint32_t)(16 * gq + (lane >> 1)) * 8u) + (lane & 1) * 8);
            const float2 p0 = __half22float2(*(const __half2*)&hv.x), p1 = __half22float2(*(const __half2*)&hv.y);
            float t = (p0.x + p0.y) + (p1.x + p1.y);
#pragma unroll
            for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0) xg[u] = t;
        }
        __syncthreads();
    }

    // ---- (3) main loop (V2a: over this warp's groups, the fragments restart with every group)
    float c[NBP][4];
#pragma unroll
    for (int p = 0; p < NBP; ++p) c[p][0] = c[p][1] = c[p][2] = c[p][3] = 0.f;
    uint32_t base0 = (uint32_t)lane * 4u, base1 = MODE == 1 ? base0 : (base0 | 128u);
    const uint32_t lane4 = (uint32_t)lane * 4u;
    const int g = lane >> 2, t4 = lane & 3;
    const bool diag0 = (g == t4), diag1 = (g == t4 + 4);
    const bool diag = diag0 || diag1;
    const int b2 = diag1 ? 1 : 0;
    // staged x of the lane's batch row of a pair, for chunk groups whose swizzle flips the row's low bit or not
    const unsigned char* xrow[2] = {xs + b2 * 16, xs + (b2 ^ 1) * 16};

    // V2a: where this lane's own sums land: D[g][t] sits in lane (g, t >> 1), register t & 1 (even batch row of the
    // pair), and in lane (g, 2 + (t >> 1)) for the odd one
    const int src0 = (lane & ~3) | (t4 >> 1);
    const bool odd = t4 & 1;
    auto lookup = [&](uint32_t (&f)[4], int m) {
        if (MODE == 1) {
            const uint32_t l00 = *(const uint32_t*)(tab + lib_entry_addr<N>(w0, 4 * m + 0, base0));
            const uint32_t l01 = *(const uint32_t*)(tab + lib_entry_addr<N>(w0, 4 * m + 1, base0));
            const uint32_t l02 = *(const uint32_t*)(tab + lib_entry_addr<N>(w0, 4 * m + 2, base0));
            const uint32_t l03 = *(const uint32_t*)(tab + lib_entry_addr<N>(w0, 4 * m + 3, base0));
            const uint32_t l10 = *(const uint32_t*)(tab + lib_entry_addr<N>(w1, 4 * m + 0, base1));
            const uint32_t l11 = *(const uint32_t*)(tab + lib_entry_addr<N>(w1, 4 * m + 1, base1));
            const uint32_t l12 = *(const uint32_t*)(tab + lib_entry_addr<N>(w1, 4 * m + 2, base1));
            const uint32_t l13 = *(const uint32_t*)(tab + lib_entry_addr<N>(w1, 4 * m + 3, base1));
            f[0] = __byte_perm(l00, l01, 0x5410);   // (k, k+1) of channel 0
            f[1] = __byte_perm(l10, l11, 0x5410);   // (k, k+1) of channel 1
            f[2] = __byte_perm(l02, l03, 0x5410);   // (k+2, k+3) of channel 0
            f[3] = __byte_perm(l12, l13, 0x5410);   // (k+2, k+3) of channel 1
            return;
        }
        f[0] = *(const uint32_t*)(tab + pair_addr<N, RPL>(w0, 2 * m, base0));
        f[2] = *(const uint32_t*)(tab + pair_addr<N, RPL>(w0, 2 * m + 1, base0));
        if (RPL == 2) {
            f[1] = *(const uint32_t*)(tab + pair_addr<N, RPL>(w1, 2 * m, base1));
            f[3] = *(const uint32_t*)(tab + pair_addr<N, RPL>(w1, 2 * m + 1, base1));
        } else {
            f[1] = 0u; f[3] = 0u;
        }
    };
#pragma unroll 1
    for (int s = warp; s < nsc; s += W) {
        if (oround < nrounds) {
            consume_slots();
            if (++oround < nrounds) fetch_slots(oround);
        }
        const bool has_next = s + W < nsc;
        const int snext = s + W;
        if (MODE == 1) {
            if (has_next) {   // metadata of the next group travels during this one
                nid0 = b.gid[m0 + (size_t)snext * 32]; nid1 = b.gid[m1 + (size_t)snext * 32];
                nsm0 = b.gsm[m0 + (size_t)snext * 32]; nsm1 = b.gsm[m1 + (size_t)snext * 32];
            }
            base0 = id0 * (uint32_t)(E * 128) + lane4;
            base1 = id1 * (uint32_t)(E * 128) + lane4;
#pragma unroll
            for (int p = 0; p < NBP; ++p) c[p][0] = c[p][1] = c[p][2] = c[p][3] = 0.f;
        }
        auto reload = [&](int gi) {
#pragma unroll
            for (int v = 0; v < N; ++v) {
                // last look-up group (of 4 weights per channel) that still reads index vector v
                const int plast = MODE == 1 ? ((128 * (v + 1) + N - 1) / N - 1) / 2 : (128 * (v + 1) + 2 * N - 1) / (2 * N) - 1;
                if (plast / 2 == gi && has_next) {
                    const uint4 t0 = ld_stream(i0 + ((size_t)snext * N + v) * 32);
                    w0[4 * v] = t0.x; w0[4 * v + 1] = t0.y; w0[4 * v + 2] = t0.z; w0[4 * v + 3] = t0.w;
                    if (RPL == 2) {
                        const uint4 t1 = ld_stream(i1 + ((size_t)snext * N + v) * 32);
                        w1[4 * v] = t1.x; w1[4 * v + 1] = t1.y; w1[4 * v + 2] = t1.z; w1[4 * v + 3] = t1.w;
                    }
                }
            }
        };
        const uint32_t kbase = (uint32_t)(sc0 + s) * kSuper;
        uint32_t fa[4], fb[4];
        lookup(fa, 0);
#pragma unroll
        for (int m = 0; m < kSuper / 4; m += 2) {   // two mma groups (8 consecutive k) per step
            uint4 xq[NBP];
#pragma unroll
            for (int p = 0; p < NBP; ++p) {
                xq[p] = make_uint4(0u, 0u, 0u, 0u);
                // chunk k / 8 = 16 (sc0 + s) + m / 2: its swizzle (m / 2) mod NB is known at compile time
                constexpr int kSw = NB - 1;
                const int c8 = (m >> 1) & kSw;
                if (diag) xq[p] = *(const uint4*)(xrow[c8 & 1] + (size_t)(kbase >> 3) * (NB * 16) +
                                                  (((m >> 1) * NB + ((2 * p) ^ (c8 & ~1))) << 4) + (((m * 4) & 7) << 1));
            }
            lookup(fb, m + 1);
            reload(m + 1);
#pragma unroll
            for (int p = 0; p < NBP; ++p) mma16816(c[p], fa[0], fa[1], fa[2], fa[3], xq[p].x, xq[p].y);
            if (m + 2 < kSuper / 4) {
                lookup(fa, m + 2);
                reload(m + 2);
            }
#pragma unroll
            for (int p = 0; p < NBP; ++p) mma16816(c[p], fb[0], fb[1], fb[2], fb[3], xq[p].z, xq[p].w);
        }
        if (MODE == 1) {
            // group sums to their owners, then  acc += scale * G + mid * X_g  (oacc doubles as the accumulator)
            const float sc_0 = h2f((uint16_t)(sm0 & 0xffffu)), md_0 = h2f((uint16_t)(sm0 >> 16));
            const float sc_1 = h2f((uint16_t)(sm1 & 0xffffu)), md_1 = h2f((uint16_t)(sm1 >> 16));
#pragma unroll
            for (int bb = 0; bb < NB; ++bb) {
                const int src = src0 + 2 * (bb & 1);
                const float e0 = __shfl_sync(0xffffffffu, c[bb >> 1][0], src), e1 = __shfl_sync(0xffffffffu, c[bb >> 1][1], src);
                const float e2 = __shfl_sync(0xffffffffu, c[bb >> 1][2], src), e3 = __shfl_sync(0xffffffffu, c[bb >> 1][3], src);
                const float G0 = odd ? e1 : e0, G1 = odd ? e3 : e2;
                const float X = xg[bb * a.SC + sc0 + s];
                oacc[bb][0] = fmaf(sc_0, G0, fmaf(md_0, X, oacc[bb][0]));
                oacc[bb][RPL - 1] = fmaf(sc_1, G1, fmaf(md_1, X, oacc[bb][RPL - 1]));
            }
            id0 = nid0; id1 = nid1; sm0 = nsm0; sm1 = nsm1;
        }
    }
    while (oround < nrounds) {
        consume_slots();
        if (++oround < nrounds) fetch_slots(oround);
    }
    if (warp == 0 && ks == 0 && a.ell_slots) {   // rows that overflow their slab finish from the CSR arrays
#pragma unroll
        for (int h = 0; h < RPL; ++h) {
            if ((int)olen[h] >= a.ell_slots) {
                const int row = (h ? blk1 : blk0) * kRowsPerBlock + lane;
                const int p1 = __ldg(b.rowptr + row + 1);
                for (int p = __ldg(b.rowptr + row) + a.ell_slots; p < p1; ++p) {
                    const uint32_t e = __ldg(b.oent + p);
#pragma unroll
                    for (int bb = 0; bb < NB; ++bb)
                        oacc[bb][h] = fmaf(h2f((uint16_t)(e >> 16)), h2f(*(const uint16_t*)(xs + xoff<NB>(bb, e & 0xffffu))),
                                           oacc[bb][h]);
                }
            }
        }
    }

    // ---- (4) the x area becomes red[W][NB][ROWS]; fragment lanes scatter to channel order, owners add outliers
    __syncthreads();   // every warp is done reading x
    if (MODE == 1) {   // every lane already owns its two channels' sums
#pragma unroll
        for (int bb = 0; bb < NB; ++bb)
#pragma unroll
            for (int h = 0; h < RPL; ++h) red[((size_t)warp * NB + bb) * ROWS + 32 * h + lane] = oacc[bb][h];
    } else {
        const int l0 = 4 * g + 2 * (t4 & 1);
#pragma unroll
        for (int p = 0; p < NBP; ++p) {
            const int bb = 2 * p + (t4 >> 1);
            float* r = red + ((size_t)warp * NB + bb) * ROWS;
            r[l0] = c[p][0]; r[l0 + 1] = c[p][1];
            if (RPL == 2) { r[32 + l0] = c[p][2]; r[32 + l0 + 1] = c[p][3]; }
        }
        __syncwarp();
#pragma unroll
        for (int bb = 0; bb < NB; ++bb)
#pragma unroll
            for (int h = 0; h < RPL; ++h) red[((size_t)warp * NB + bb) * ROWS + 32 * h + lane] += oacc[bb][h];
    }
    __syncthreads();

    // ---- (5) fixed-order reduction over the warps, store or split-K finish
    for (int t = threadIdx.x; t < NB * ROWS; t += kBThreads) {
        const int bb = t / ROWS, r = t % ROWS;
        float total = 0.f;
#pragma unroll
        for (int w = 0; w < W; ++w) total += red[((size_t)w * NB + bb) * ROWS + r];
        red[t] = total;   // slot t is read by this thread only (w = 0 term)
    }
    __syncthreads();
    if (KS > 1) {
        __shared__ int s_last;
        for (int t = threadIdx.x; t < NB * ROWS; t += kBThreads) {
            const int bb = t / ROWS, r = t % ROWS;
            a.partial[((size_t)ks * NB + bb) * a.rows_ws + blk * ROWS + r] = red[t];
        }
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) s_last = (atomicAdd(a.tickets + blk, 1) == KS - 1);
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        for (int t = threadIdx.x; t < NB * ROWS; t += kBThreads) {
            const int bb = t / ROWS, r = t % ROWS;
            float total = 0.f;
            for (int k2 = 0; k2 < KS; ++k2) total += __ldcg(a.partial + ((size_t)k2 * NB + bb) * a.rows_ws + blk * ROWS + r);
            red[t] = total;
        }
        if (threadIdx.x == 0) a.tickets[blk] = 0;
        __syncthreads();
    }
    for (int t = threadIdx.x; t < NB * ROWS; t += kBThreads) {
        const int bb = t / ROWS, r = t % ROWS;
        const int row = blk * ROWS + r;
        const bool dup = (r >= 32) && (RPL * blk + 1 >= a.RB);
        if (!dup && bb < a.nb && row < a.rows) {
            store_y<TIO>(a.y, (size_t)bb * a.rows + row, red[t], a.y_is_fp16);
        }
    }
}

// ------------------------------------------------------------------------------------ host side

static int batch_rpl(const Layout& l) { return (l.mode == 0 && l.bits == 5) ? 1 : 2; }

static size_t batch_smem_bytes(const Layout& l, int nbt) {
    const int rpl = batch_rpl(l);
    const size_t x = (size_t)nbt * l.cols * 2, red = (size_t)kBWarps * nbt * 32 * rpl * 4;
    const size_t tab = l.mode ? (size_t)l.L * l.E * 128 + (((size_t)nbt * l.SC * 4 + 15) & ~(size_t)15)
                              : (size_t)l.E * l.E * 128 * rpl;
    return tab + (x > red ? x : red);
}

// batch tile (4 or 8 rows of x per launch) that fits one CTA per SM, 0 if none does
static int batch_tile(const Layout& l, int batch) {
    if (l.bits < 2 || l.bits > 5) return 0;
    if (batch > 4 && batch_smem_bytes(l, 8) <= 220u * 1024u) return 8;
    if (batch_smem_bytes(l, 4) <= 220u * 1024u) return 4;
    return 0;
}

// V2 blobs, and V2a blobs whose groups are whole super-chunks (groups of 64 weights go to the generic kernel)
bool batch_supported(const Layout& l, int batch) {
    return batch > 2 && (l.mode == 0 || l.GH == 1) && batch_tile(l, batch) != 0;
}

template <int N, int NB, int RPL, bool TIO, int MODE>
static cudaError_t launch_batch_io(const BatchArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    static DeviceOnce attr_done;
    const int dev = DeviceOnce::current();
    if (!attr_done.is_set(dev)) {
        cudaError_t e = cudaFuncSetAttribute(gemv_batch_kernel<N, NB, RPL, TIO, MODE>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return e;
        attr_done.set(dev);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kBThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_batch_kernel<N, NB, RPL, TIO, MODE>, a);
}

template <int N, int NB, int RPL, int MODE>
static cudaError_t launch_batch(const BatchArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    if (a.x_bf16 || a.y_is_fp16 == 2) return launch_batch_io<N, NB, RPL, true, MODE>(a, grid, smem, s);
    return launch_batch_io<N, NB, RPL, false, MODE>(a, grid, smem, s);
}

template <int N, int NB>
static cudaError_t launch_batch_mode(int mode, const BatchArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
    if (mode) return launch_batch<N, NB, 2, 1>(a, grid, smem, s);
    return launch_batch<N, NB, (N == 5 ? 1 : 2), 0>(a, grid, smem, s);
}

cudaError_t launch_gemv_batch(const Layout& l, const GemvCall& c, cudaStream_t s) {
    const int rpl = batch_rpl(l);
    const int blocks = (l.RB + rpl - 1) / rpl;
    const int slots = sched_sms();   // one CTA per SM
    for (int b0 = 0; b0 < c.batch; b0 += 8) {
        const int nb = c.batch - b0 < 8 ? c.batch - b0 : 8;
        const int nbt = batch_tile(l, nb);
        if (nbt == 0) return cudaErrorInvalidValue;
        // a tile of 4 serves up to 4 rows: split an 8-row step in two when only the small tile fits
        for (int b1 = 0; b1 < nb; b1 += nbt) {
            const int n1 = nb - b1 < nbt ? nb - b1 : nbt;
            BatchArgs a{};
            a.off = offsets_of(l);
            a.packed = c.packed;
            a.x = c.x + (size_t)(b0 + b1) * l.cols;
            a.y = (void*)((char*)c.y + (size_t)(b0 + b1) * l.rows * (c.y_is_fp16 ? 2 : 4));
            a.rows = l.rows; a.cols = l.cols; a.RB = l.RB; a.SC = l.SC; a.ell_slots = l.ell_slots; a.L = l.L;
            a.rows_ws = blocks * 32 * rpl;
            a.nb = n1; a.y_is_fp16 = c.y_is_fp16; a.x_bf16 = c.x_bf16;
            // schedule: whole-K blocks in whole rounds of slots; the last partial round cut along K (<= 16 slices)
            int rem = blocks % slots, kst = 1;
            if (rem > 0) {
                kst = slots / rem;
                const int kmax = l.SC / 4 > 1 ? l.SC / 4 : 1;
                if (kst > kmax) kst = kmax;
                if (kst > 16) kst = 16;
                if (kst > l.SC) kst = l.SC;
            }
            if (kst <= 1) { kst = 1; rem = 0; }
            a.n_full = blocks - rem;
            a.sc_per_split = (l.SC + kst - 1) / kst;
            a.kst = (l.SC + a.sc_per_split - 1) / a.sc_per_split;
            if (a.kst <= 1) { a.kst = 1; a.n_full = blocks; rem = 0; }
            a.tickets = (int*)c.workspace;
            a.partial = (float*)((char*)c.workspace + align256((size_t)l.RB * 4));   // behind the common counter region
            const size_t smem = batch_smem_bytes(l, nbt);
            dim3 grid((unsigned)(a.n_full + rem * a.kst), 1, 1);
            cudaError_t e = cudaErrorInvalidValue;
            switch (l.bits * 10 + nbt) {
                case 24: e = launch_batch_mode<2, 4>(l.mode, a, grid, smem, s); break;
                case 28: e = launch_batch_mode<2, 8>(l.mode, a, grid, smem, s); break;
                case 34: e = launch_batch_mode<3, 4>(l.mode, a, grid, smem, s); break;
                case 38: e = launch_batch_mode<3, 8>(l.mode, a, grid, smem, s); break;
                case 44: e = launch_batch_mode<4, 4>(l.mode, a, grid, smem, s); break;
                case 48: e = launch_batch_mode<4, 8>(l.mode, a, grid, smem, s); break;
                case 54: e = launch_batch_mode<5, 4>(l.mode, a, grid, smem, s); break;
                case 58: e = launch_batch_mode<5, 8>(l.mode, a, grid, smem, s); break;
            }
            if (e != cudaSuccess) return e;
        }
    }
    return cudaSuccess;
}

}  // namespace xfp
