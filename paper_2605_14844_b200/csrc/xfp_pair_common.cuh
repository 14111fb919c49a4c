// Device helpers shared by the pair-table GEMV kernels (xfp_gemv_pair.cu, xfp_gemv_batch.cu).
#pragma once
#include "xfp_common.cuh"

namespace xfp {

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Byte offset of the table entry of pair p (compile time) of a 128-weight stream w[4N]:
// t * 128 * RPL merged with `base` (= channel_half * 128 + lane * 4, below the t field).
template <int N, int RPL>
__device__ __forceinline__ uint32_t pair_addr(const uint32_t* w, int p, uint32_t base) {
    constexpr int SH = RPL == 2 ? 8 : 7;  // log2 of the entry stride
    if (N == 4 && RPL == 2) {
        // pair p is byte (p & 3) of word p >> 2: one PRMT builds [base.b0, byte, 0, 0]
        return __byte_perm(w[p >> 2], base, 0x5504u | ((uint32_t)(p & 3) << 4));
    } else {
        constexpr uint32_t mask = ((1u << (2 * N)) - 1u) << SH;
        const int bit = p * 2 * N, wi = bit >> 5, off = bit & 31;
        uint32_t v;
        if (off + 2 * N > 32)
            v = __funnelshift_r(w[wi], w[wi + 1], off - SH);   // field straight to bit SH (off > SH whenever it straddles)
        else if (off >= SH)
            v = w[wi] >> (off - SH);
        else
            v = w[wi] << (SH - off);
        return (v & mask) | base;
    }
}

// Byte offset of the table entry of index j (compile time) for tables that hold one entry per index
// (N = 6): q * 128 * RPL merged with `base`.
template <int N, int RPL>
__device__ __forceinline__ uint32_t single_addr(const uint32_t* w, int j, uint32_t base) {
    constexpr int SH = RPL == 2 ? 8 : 7;
    constexpr uint32_t mask = ((1u << N) - 1u) << SH;
    const int bit = j * N, wi = bit >> 5, off = bit & 31;
    uint32_t v;
    if (off + N > 32)
        v = __funnelshift_r(w[wi], w[wi + 1], off - SH);   // field straight to bit SH (off > SH whenever it straddles)
    else if (off >= SH)
        v = w[wi] >> (off - SH);
    else
        v = w[wi] << (SH - off);
    return (v & mask) | base;
}

}  // namespace xfp
