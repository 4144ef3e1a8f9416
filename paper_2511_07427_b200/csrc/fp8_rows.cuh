// FP8 storage of K/V rows (the precision the paper evaluates in: arXiv 2511.07427, Section 8.1).
//
// Format.  A row of d elements is stored as d bytes in the OCP e4m3 format (1 sign, 4 exponent bits with bias 7,
// 3 mantissa bits, largest finite value 448, no infinities) plus ONE power-of-two scale per row, kept as its
// exponent e in a signed byte: element = e4m3 value * 2^e.  e is the smallest integer with max|x| / 2^e <= 448
// (0 for an all-zero row), clamped to [-120, 120]; elements are rounded to nearest-even.  Because the scale is a
// power of two and e4m3 has four significant bits, every stored value is exactly representable in bf16, so the
// rest of the library (k-means, representatives, statistics, splits) works on bf16 rows that already lie on this
// grid: keys and values are rounded to it once, where they enter the library, and the gather-attention kernel reads
// the one-byte pages.  No wider copy of a row is kept: the paths that re-read keys (splits, statistics, export)
// decode the bytes through load_key below, which gives the rounded values back exactly.
//
// The helpers below do the rounding for the register layouts the kernels use.  Conversions go through the
// conversion intrinsics of cuda_fp8.h.
#pragma once

#include <cuda_fp8.h>

#include "common.cuh"

namespace dkv {

// Exponent of the row's power-of-two scale from the row's largest magnitude.
__device__ __forceinline__ int fp8_row_exp(float amax) {
    if (!(amax > 0.f)) return 0;
    int ex;
    const float m = frexpf(amax, &ex);                 // amax = m * 2^ex, m in [0.5, 1)
    const int e = (m <= 0.875f) ? ex - 9 : ex - 8;     // 448 = 0.875 * 2^9
    return max(-120, min(120, e));
}
__device__ __forceinline__ float pow2f(int e) { return __int_as_float((e + 127) << 23); }     // e in [-126, 127]

// Two values scaled by 2^-e to two e4m3 bytes (low byte = x).
__device__ __forceinline__ unsigned short fp8_pack2(float x, float y, float inv_scale) {
    return (unsigned short)__nv_cvt_float2_to_fp8x2(make_float2(x * inv_scale, y * inv_scale), __NV_SATFINITE, __NV_E4M3);
}
// Two e4m3 bytes (low byte first) to two floats, times the row's scale.
__device__ __forceinline__ float2 fp8_unpack2(unsigned short b, float scale) {
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)b, __NV_E4M3);
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h));
    return make_float2(f.x * scale, f.y * scale);
}
// x rounded to the row's grid.
__device__ __forceinline__ float2 fp8_round2(float x, float y, float inv_scale, float scale) {
    return fp8_unpack2(fp8_pack2(x, y, inv_scale), scale);
}

// Largest magnitude over the lanes that share a row: `group` consecutive lanes (a power of two, 8 or 32).
__device__ __forceinline__ float group_max(float v, int group) {
    for (int o = group >> 1; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// N consecutive elements (logical index e0; N = 1, 2 or 4, inside one 4-element group) of the K row in global slot
// `gslot` (its index in the whole page pool), as floats: from the row's bf16 / fp32 page, or -- FP8 storage, which keeps
// no such page -- decoded from the row's bytes and scale exponent (exact).
template <typename KV, int HD, int N>
__device__ __forceinline__ void load_key(const Tables& t, size_t gslot, int e0, float (&x)[N]) {
    if (t.fp8) {
        if constexpr (HD == 128 && sizeof(KV) == 2) {
            const unsigned char* p = t.k8 + gslot * HD + row_pos<16>(gslot, e0);
            const float sc = pow2f(t.k8e[gslot]);
            if constexpr (N == 4) {
                const unsigned w = *reinterpret_cast<const unsigned*>(p);
                const float2 a = fp8_unpack2((unsigned short)(w & 0xffffu), sc), b = fp8_unpack2((unsigned short)(w >> 16), sc);
                x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
            } else {
#pragma unroll
                for (int i = 0; i < N; i++) x[i] = fp8_unpack2((unsigned short)p[i], sc).x;
            }
        }
        return;
    }
    const KV* k = reinterpret_cast<const KV*>(t.kpages) + gslot * HD + row_pos<Epc<KV>::v>(gslot, e0);
#pragma unroll
    for (int i = 0; i < N; i++) x[i] = to_f(k[i]);
}

}  // namespace dkv
