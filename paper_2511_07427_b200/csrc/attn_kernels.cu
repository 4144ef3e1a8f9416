// Gather-attention over the selected clusters' pages for bf16 K/V: attention restricted to
// the retrieved entries (arXiv 2511.07427, Section 2.1 / 4.1), G query heads sharing every
// K/V row that is read.
//
// Each warp owns whole pages.  K and V rows go from HBM straight into mma.sync operand
// registers with 128-bit loads (no shared-memory staging): the contraction index of
// Q.K^T is permuted so that the 16 bytes a thread loads from a K row are exactly its B
// fragments of two k-steps, and the output columns of P.V are permuted so that the 16
// bytes a thread loads from each of its four V rows become, after one byte-permute per
// register, its B fragments of eight n-tiles.  Q (pre-scaled by log2(e)/sqrt(d)) and the
// softmax weights P are each split into bf16 hi + lo parts that sit in rows r and r+8 of
// the 16-row MMA tile, which the same thread accumulates, so fp32 queries and weights
// lose nothing that matters (2^-17 relative) and no cross-lane traffic is needed.
#include <float.h>

#include "common.cuh"

namespace dkv {

__device__ __forceinline__ void mma_bf16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (hi, lo) bf16 split of two floats packed as bf16x2 (first value in the low half).
__device__ __forceinline__ void split2(float x, float y, unsigned& hi, unsigned& lo) {
    __nv_bfloat16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
    __nv_bfloat16 xl = __float2bfloat16_rn(x - __bfloat162float(xh)), yl = __float2bfloat16_rn(y - __bfloat162float(yh));
    hi = (unsigned)__bfloat16_as_ushort(xh) | ((unsigned)__bfloat16_as_ushort(yh) << 16);
    lo = (unsigned)__bfloat16_as_ushort(xl) | ((unsigned)__bfloat16_as_ushort(yl) << 16);
}

__device__ __forceinline__ uint4 ldg16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

constexpr int AT_WARPS = 4;

template <int HD>
__global__ void __launch_bounds__(AT_WARPS * 32, 2) k_gather_attn_mma(Tables t, StepPtr qp) {
    constexpr int KS = HD / 16;       // k-steps of Q.K^T
    constexpr int KJ = KS / 2;        // 16-byte chunks a thread loads per K row
    constexpr int NT = HD / 8;        // n-tiles of P.V
    constexpr int VI = HD / 64;       // 16-byte chunks a thread loads per V row
    const int s = blockIdx.x, u = blockIdx.y, S = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, c = lane & 3;
    const int G = t.G;
    const float* q = reinterpret_cast<const float*>(qp.get()) + (size_t)u * G * HD;
    const float scale = rsqrtf((float)HD) * 1.4426950408889634f;

    // Q fragments: rows 0..7 = hi part of head r, rows 8..15 = lo part of head r
    unsigned qa[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ks++) {
        const int base = 8 * (c + 4 * (ks >> 1)) + 4 * (ks & 1);
        float x0 = 0.f, x1 = 0.f, x2 = 0.f, x3 = 0.f;
        if (r < G) {
            const float4 v = *reinterpret_cast<const float4*>(q + r * HD + base);
            x0 = v.x * scale; x1 = v.y * scale; x2 = v.z * scale; x3 = v.w * scale;
        }
        split2(x0, x1, qa[ks][0], qa[ks][1]);
        split2(x2, x3, qa[ks][2], qa[ks][3]);
    }
    float o[NT][4];
#pragma unroll
    for (int x = 0; x < NT; x++) { o[x][0] = 0.f; o[x][1] = 0.f; o[x][2] = 0.f; o[x][3] = 0.f; }
    float m = -INFINITY, l = 0.f;

    const int nw = t.n_work[u];
    const int per = (nw + S - 1) / S;
    const int w0 = s * per, w1 = min(nw, w0 + per);
    const int2* work = t.work + (size_t)u * t.W;
    const __nv_bfloat16* kpg = reinterpret_cast<const __nv_bfloat16*>(t.kpages) + (size_t)u * t.P * PAGE * HD;
    const __nv_bfloat16* vpg = reinterpret_cast<const __nv_bfloat16*>(t.vpages) + (size_t)u * t.P * PAGE * HD;

    for (int w = w0 + warp; w < w1; w += AT_WARPS) {
        const int2 ent = work[w];
        for (int half = 0; half < 2; half++) {
            const int nvalid = ent.y - half * 16;
            if (nvalid <= 0) break;
            const size_t row0 = (size_t)ent.x * PAGE + half * 16;
            // ---- loads: K rows (tile*8 + r), chunks c + 4j; V rows 2c, 2c+1, 2c+8, 2c+9, chunks r + 8i
            uint4 kw[2][KJ];
#pragma unroll
            for (int tile = 0; tile < 2; tile++) {
                const bool ok = tile * 8 + r < nvalid;
                const __nv_bfloat16* kr = kpg + (row0 + tile * 8 + r) * HD;
#pragma unroll
                for (int j = 0; j < KJ; j++) kw[tile][j] = ok ? ldg16(kr + 8 * (c + 4 * j)) : make_uint4(0, 0, 0, 0);
            }
            uint4 vw[4][VI];
#pragma unroll
            for (int rr = 0; rr < 4; rr++) {
                const int tok = 2 * c + (rr & 1) + 8 * (rr >> 1);
                const bool ok = tok < nvalid;
                const __nv_bfloat16* vr = vpg + (row0 + tok) * HD;
#pragma unroll
                for (int i = 0; i < VI; i++) vw[rr][i] = ok ? ldg16(vr + 8 * (r + 8 * i)) : make_uint4(0, 0, 0, 0);
            }
            // ---- S = Q K^T for the two 8-token tiles
            float sc[2][4];
#pragma unroll
            for (int tile = 0; tile < 2; tile++) {
                sc[tile][0] = 0.f; sc[tile][1] = 0.f; sc[tile][2] = 0.f; sc[tile][3] = 0.f;
#pragma unroll
                for (int j = 0; j < KJ; j++) {
                    mma_bf16(sc[tile], qa[2 * j][0], qa[2 * j][1], qa[2 * j][2], qa[2 * j][3], kw[tile][j].x, kw[tile][j].y);
                    mma_bf16(sc[tile], qa[2 * j + 1][0], qa[2 * j + 1][1], qa[2 * j + 1][2], qa[2 * j + 1][3], kw[tile][j].z, kw[tile][j].w);
                }
            }
            // logits of head r for tokens tile*8 + 2c + {0,1}: hi row + lo row
            float lg[4];
#pragma unroll
            for (int tile = 0; tile < 2; tile++) {
                const int tok = tile * 8 + 2 * c;
                lg[tile * 2 + 0] = tok < nvalid ? sc[tile][0] + sc[tile][2] : -INFINITY;
                lg[tile * 2 + 1] = tok + 1 < nvalid ? sc[tile][1] + sc[tile][3] : -INFINITY;
            }
            float mx = fmaxf(fmaxf(lg[0], lg[1]), fmaxf(lg[2], lg[3]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float mn = fmaxf(m, mx);                 // finite: token 0 of the half page is valid
            const float corr = exp2f(m - mn);
            m = mn;
            float p[4];
#pragma unroll
            for (int e = 0; e < 4; e++) p[e] = exp2f(lg[e] - mn);
            l = l * corr + (p[0] + p[1]) + (p[2] + p[3]);
            unsigned pa[4];
            split2(p[0], p[1], pa[0], pa[1]);   // a0 = hi(tile 0), a1 = lo(tile 0)
            split2(p[2], p[3], pa[2], pa[3]);   // a2 = hi(tile 1), a3 = lo(tile 1)
#pragma unroll
            for (int x = 0; x < NT; x++) { o[x][0] *= corr; o[x][1] *= corr; o[x][2] *= corr; o[x][3] *= corr; }
            // ---- O += P V : n-tile (i, e) takes element e of chunk i of the thread's four rows
#pragma unroll
            for (int i = 0; i < VI; i++) {
                const unsigned* a0 = reinterpret_cast<const unsigned*>(&vw[0][i]);
                const unsigned* a1 = reinterpret_cast<const unsigned*>(&vw[1][i]);
                const unsigned* a2 = reinterpret_cast<const unsigned*>(&vw[2][i]);
                const unsigned* a3 = reinterpret_cast<const unsigned*>(&vw[3][i]);
#pragma unroll
                for (int e = 0; e < 8; e++) {
                    const unsigned sel = (e & 1) ? 0x7632u : 0x5410u;
                    const unsigned b0 = __byte_perm(a0[e >> 1], a1[e >> 1], sel);
                    const unsigned b1 = __byte_perm(a2[e >> 1], a3[e >> 1], sel);
                    mma_bf16(o[i * 8 + e], pa[0], pa[1], pa[2], pa[3], b0, b1);
                }
            }
        }
    }
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);

    // ---- merge the warps of the block, write the partial (acc, m, l) of split s
    __shared__ float sm_m[AT_WARPS][8], sm_l[AT_WARPS][8];
    __shared__ float sm_o[AT_WARPS][8][HD];
    if (c == 0) { sm_m[warp][r] = m; sm_l[warp][r] = l; }
#pragma unroll
    for (int x = 0; x < NT; x++) {
        const int i = x >> 3, e = x & 7;
        sm_o[warp][r][8 * (2 * c + 8 * i) + e] = o[x][0] + o[x][2];
        sm_o[warp][r][8 * (2 * c + 1 + 8 * i) + e] = o[x][1] + o[x][3];
    }
    __syncthreads();
    float* part = t.part + (((size_t)u * S + s) * G) * (HD + 2);
    for (int idx = threadIdx.x; idx < G * HD; idx += AT_WARPS * 32) {
        const int g = idx / HD, e = idx % HD;
        float mm = sm_m[0][g];
#pragma unroll
        for (int w = 1; w < AT_WARPS; w++) mm = fmaxf(mm, sm_m[w][g]);
        float a = 0.f, ll = 0.f;
        if (mm != -INFINITY) {
#pragma unroll
            for (int w = 0; w < AT_WARPS; w++) {
                const float f = exp2f(sm_m[w][g] - mm);
                a += sm_o[w][g][e] * f; ll += sm_l[w][g] * f;
            }
        }
        part[g * (HD + 2) + e] = a;
        if (e == 0) { part[g * (HD + 2) + HD] = mm; part[g * (HD + 2) + HD + 1] = ll; }
    }
}

void launch_gather_attn_mma(const Tables& t, StepPtr q, cudaStream_t s, long long* launches) {
    dim3 grid(t.n_splits_attn, t.U);
    if (t.d == 64) k_gather_attn_mma<64><<<grid, AT_WARPS * 32, 0, s>>>(t, q);
    else k_gather_attn_mma<128><<<grid, AT_WARPS * 32, 0, s>>>(t, q);
    (*launches)++;
}

}  // namespace dkv
