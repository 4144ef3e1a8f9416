// Per-row arithmetic of the centroid pass (arXiv 2511.07427, Section 4.1: similarity of the query to
// every representative; Algorithm 1: distance of the new key to every representative), shared by the
// stand-alone pass (k_front) and by the pass fused into the tail of a loop iteration, so that both give
// the same bits.  Eight lanes share one representative row: lane l8 of a row group holds elements
// 4*l8 + 32*i .. +3 (i < HD/32) of the row, of the summed query heads and of the new key.
#pragma once

#include "common.cuh"
#include "fp8_rows.cuh"

namespace dkv {

// Partial sum of the unit's query heads: the four row groups of a warp take heads sub and sub + 4.
// front_qsum_finish() exchanges the partial sums, after which every lane holds the sum over all heads.
template <int HD>
__device__ __forceinline__ void front_qsum_load(const float* __restrict__ q, int G, int lane, float (&qs)[HD / 32][4]) {
    static_assert(MAX_G <= 8, "two heads per row group");
    const int sub = lane >> 3, l8 = lane & 7;
#pragma unroll
    for (int i = 0; i < HD / 32; i++)
#pragma unroll
        for (int e = 0; e < 4; e++) qs[i][e] = 0.f;
#pragma unroll
    for (int h = 0; h < 2; h++) {
        const int g = sub + 4 * h;
        if (g < G) {
#pragma unroll
            for (int i = 0; i < HD / 32; i++) {
                const float4 v = *reinterpret_cast<const float4*>(q + g * HD + l8 * 4 + 32 * i);
                qs[i][0] += v.x; qs[i][1] += v.y; qs[i][2] += v.z; qs[i][3] += v.w;
            }
        }
    }
}
template <int HD>
__device__ __forceinline__ void front_qsum_finish(float (&qs)[HD / 32][4]) {
#pragma unroll
    for (int i = 0; i < HD / 32; i++)
#pragma unroll
        for (int e = 0; e < 4; e++) {
            qs[i][e] += __shfl_xor_sync(0xffffffffu, qs[i][e], 8);
            qs[i][e] += __shfl_xor_sync(0xffffffffu, qs[i][e], 16);
        }
}

// fp8: the key is rounded to the FP8 storage grid first (the eight lanes of a row group hold the whole row).
template <typename KV, int HD>
__device__ __forceinline__ void front_key_load(const KV* __restrict__ k, int lane, float (&kk)[HD / 32][4], int fp8 = 0) {
    const int l8 = lane & 7;
#pragma unroll
    for (int i = 0; i < HD / 32; i++) {
        const float4 v = ld4(k, l8 * 4 + 32 * i);
        kk[i][0] = v.x; kk[i][1] = v.y; kk[i][2] = v.z; kk[i][3] = v.w;
    }
    if (fp8) {
        float am = 0.f;
#pragma unroll
        for (int i = 0; i < HD / 32; i++)
#pragma unroll
            for (int e = 0; e < 4; e++) am = fmaxf(am, fabsf(kk[i][e]));
        const int ex = fp8_row_exp(group_max(am, 8));
        const float sc = pow2f(ex), inv = pow2f(-ex);
#pragma unroll
        for (int i = 0; i < HD / 32; i++) {
            const float2 a = fp8_round2(kk[i][0], kk[i][1], inv, sc), b = fp8_round2(kk[i][2], kk[i][3], inv, sc);
            kk[i][0] = a.x; kk[i][1] = a.y; kk[i][2] = b.x; kk[i][3] = b.y;
        }
    }
}

// s = (sum of heads) . r and dd = |k - r|^2 of one row, complete in every lane of the row group.
template <int HD>
__device__ __forceinline__ void front_row(const float4 (&r)[HD / 32], const float (&qs)[HD / 32][4], const float (&kk)[HD / 32][4],
                                          float& s, float& dd) {
    s = 0.f; dd = 0.f;
#pragma unroll
    for (int i = 0; i < HD / 32; i++) {
        const float4 r4 = r[i];
        s = fmaf(qs[i][0], r4.x, s); s = fmaf(qs[i][1], r4.y, s); s = fmaf(qs[i][2], r4.z, s); s = fmaf(qs[i][3], r4.w, s);
        float a = kk[i][0] - r4.x, b = kk[i][1] - r4.y, c = kk[i][2] - r4.z, e = kk[i][3] - r4.w;
        dd = fmaf(a, a, dd); dd = fmaf(b, b, dd); dd = fmaf(c, c, dd); dd = fmaf(e, e, dd);
    }
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) { s += __shfl_xor_sync(0xffffffffu, s, o); dd += __shfl_xor_sync(0xffffffffu, dd, o); }
}

}  // namespace dkv
