// Shared device helpers of the XFP kernels: bit-field extraction from a lane's index stream,
// cache-hinted loads, fp16 bit casts.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "xfp_layout.h"

namespace xfp {

// Index j (compile-time after unrolling) of a lane's 128*N-bit stream held in w[4*N].
template <int N>
__device__ __forceinline__ uint32_t field(const uint32_t* w, int j) {
    const int bit = j * N;
    const int wi = bit >> 5;
    const int off = bit & 31;
    uint32_t v;
    if (off + N > 32)
        v = __funnelshift_r(w[wi], w[wi + 1], off);
    else
        v = w[wi] >> off;
    return v & ((1u << N) - 1u);
}

// Streaming 16-byte load of packed indices: read-only path, no L1 allocation (touched once).
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ float h2f(uint16_t b) { return __half2float(__ushort_as_half(b)); }
__device__ __forceinline__ uint16_t f2h(float f) { return __half_as_ushort(__float2half_rn(f)); }

// Activations may arrive as bf16 (the paper's native type): they are converted to fp16 while they are staged,
// round to nearest even, clamped to the finite fp16 range.  A bf16 value with |x| in [2^-14, 65504] has 8
// significant bits and converts exactly; smaller ones land on the fp16 subnormal grid (absolute error <= 2^-25).
// NaN stays NaN (the clamp is applied to ordered values only; fminf/fmaxf would return the bound instead), so a
// NaN activation poisons y under bf16 exactly as it does under fp16.
__device__ __forceinline__ float clamp_f16_range(float v) {
    return (v != v) ? v : fminf(fmaxf(v, -65504.f), 65504.f);
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v) {
    const float lo = clamp_f16_range(__uint_as_float(v << 16));
    const float hi = clamp_f16_range(__uint_as_float(v & 0xffff0000u));
    const __half2 h = __floats2half2_rn(lo, hi);
    return *(const uint32_t*)&h;
}
__device__ __forceinline__ uint4 x8_as_f16(uint4 v, int x_bf16) {
    if (x_bf16) {
        v.x = bf16x2_to_f16x2(v.x); v.y = bf16x2_to_f16x2(v.y);
        v.z = bf16x2_to_f16x2(v.z); v.w = bf16x2_to_f16x2(v.w);
    }
    return v;
}
// One activation as the float the kernels multiply with: a bf16 value takes the same route as in the staged
// kernels (clamp, round to fp16), so that every kernel sees the same x whatever the dispatcher picked.
__device__ __forceinline__ float x_as_float(uint16_t bits, int x_bf16) {
    if (!x_bf16) return h2f(bits);
    return __half2float(__float2half_rn(clamp_f16_range(__uint_as_float((uint32_t)bits << 16))));
}
// Output element i of y: fp32 (kind 0), fp16 (1) or bf16 (2), one rounding of the fp32 sum.
__device__ __forceinline__ void put_y(void* y, size_t i, float v, int kind) {
    if (kind == 1) ((uint16_t*)y)[i] = f2h(v);
    else if (kind == 2) ((uint16_t*)y)[i] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
    else ((float*)y)[i] = v;
}

// TIO (typed IO) instantiations take bf16 x and store any y type; the plain ones keep the two-way store so that
// the code of the fp16 path is what it was before typed IO existed.
template <bool TIO>
__device__ __forceinline__ void store_y(void* y, size_t i, float v, int kind) {
    if (TIO) {
        put_y(y, i, v, kind);
    } else if (kind) {
        ((uint16_t*)y)[i] = f2h(v);
    } else {
        ((float*)y)[i] = v;
    }
}

// Pointers of one packed blob.
struct Blob {
    const uint4* idx;
    const uint16_t* cb;
    const uint8_t* gid;
    const uint32_t* gsm;  // half2 bits: scale | mid << 16
    const int* rowptr;
    const uint32_t* oent;
    const uint32_t* ell;
};

struct Offsets {
    size_t idx, cb, gid, gsm, rowptr, hdr, oent, ell;
};

__host__ __device__ inline Blob blob_at(const void* packed, const Offsets& o) {
    const char* b = (const char*)packed;
    Blob r;
    r.idx = (const uint4*)(b + o.idx);
    r.cb = (const uint16_t*)(b + o.cb);
    r.gid = (const uint8_t*)(b + o.gid);
    r.gsm = (const uint32_t*)(b + o.gsm);
    r.rowptr = (const int*)(b + o.rowptr);
    r.oent = (const uint32_t*)(b + o.oent);
    r.ell = (const uint32_t*)(b + o.ell);
    return r;
}

inline Offsets offsets_of(const Layout& l) {
    return Offsets{l.off_idx, l.off_cb, l.off_gid, l.off_gsm, l.off_rowptr, l.off_hdr, l.off_oent, l.off_ell};
}

}  // namespace xfp
