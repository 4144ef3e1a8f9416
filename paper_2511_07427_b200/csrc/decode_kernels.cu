// Plain fp32 gather-attention over the selected clusters' pages (any K/V dtype; the path
// for fp32 K/V) and the split-K combine shared by both attention kernels
// (arXiv 2511.07427, Section 2.1 / 4.1: attention over the retrieved entries only).
#include <float.h>

#include "common.cuh"
#include "fp8_rows.cuh"

namespace dkv {

// ------------------------------------------------------------------ gather attention (baseline)

// Grid (S, U), 4 warps.  Split s of unit u owns a contiguous range of the unit's work
// list; its warps take entries round-robin, one token at a time with the head dimension
// spread over the lanes, and keep an online-softmax state (m, l, acc) per query head.
// The block merges its warps and writes the unnormalised partial to t.part.
template <typename KV, int HD, int G>
__global__ void __launch_bounds__(128) k_gather_attn_v1(Tables t, StepPtr qp) {
    constexpr int EPL = HD / 32;
    const int s = blockIdx.x, u = blockIdx.y, S = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* q = reinterpret_cast<const float*>(qp.get()) + (size_t)u * G * HD;
    const float scale = rsqrtf((float)HD) * 1.4426950408889634f;   // fold log2(e): exp(x) = exp2(x * log2 e)
    float qr[G][EPL];
#pragma unroll
    for (int g = 0; g < G; g++)
#pragma unroll
        for (int e = 0; e < EPL; e++) qr[g][e] = q[g * HD + lane * EPL + e] * scale;
    float m[G], l[G], acc[G][EPL];
#pragma unroll
    for (int g = 0; g < G; g++) {
        m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; e++) acc[g][e] = 0.f;
    }
    const int nw = t.n_work[u];
    const int per = (nw + S - 1) / S;
    const int w0 = s * per, w1 = min(nw, w0 + per);
    const int2* work = t.work + (size_t)u * t.W;
    const KV* kp = reinterpret_cast<const KV*>(t.kpages);
    const KV* vp = reinterpret_cast<const KV*>(t.vpages);
    for (int w = w0 + warp; w < w1; w += 4) {
        int2 ent = work[w];
        if (!DKV_IN(t, SITE_PLAIN_ENTRY, ent.y, 1, ENTRY_ROWS + 1) || !DKV_IN(t, SITE_PLAIN_ENTRY, ent.x, 0, (long long)t.P * PAGE - ent.y + 1)) continue;
        size_t pbase = ((size_t)u * t.P * PAGE + ent.x) * HD;
        for (int r = 0; r < ent.y; r++) {
            const int pos = row_pos<Epc<KV>::v>((size_t)(ent.x + r), lane * EPL);      // the row's stored chunk order
            const KV* k = kp + pbase + (size_t)r * HD + pos;
            const KV* v = vp + pbase + (size_t)r * HD + pos;
            float kk[EPL], vv[EPL];
            if (t.fp8) {
                // FP8 mode: the row's one-byte copy (four bytes per lane) and its two scale exponents
                if constexpr (EPL == 4) {
                    const size_t slot = (size_t)u * t.P * PAGE + ent.x + r;
                    const unsigned kb = *reinterpret_cast<const unsigned*>(t.k8 + slot * HD + row_pos<16>(slot, lane * 4));
                    const unsigned vb = *reinterpret_cast<const unsigned*>(t.v8 + slot * HD + row_pos<16>(slot, lane * 4));
                    const float ks = pow2f(t.k8e[slot]), vs = pow2f(t.v8e[slot]);
                    float2 a = fp8_unpack2((unsigned short)(kb & 0xffffu), ks), b = fp8_unpack2((unsigned short)(kb >> 16), ks);
                    kk[0] = a.x; kk[1] = a.y; kk[2] = b.x; kk[3] = b.y;
                    a = fp8_unpack2((unsigned short)(vb & 0xffffu), vs); b = fp8_unpack2((unsigned short)(vb >> 16), vs);
                    vv[0] = a.x; vv[1] = a.y; vv[2] = b.x; vv[3] = b.y;
                }
            } else {
#pragma unroll
            for (int e = 0; e < EPL; e++) { kk[e] = to_f(k[e]); vv[e] = to_f(v[e]); }
            }
#pragma unroll
            for (int g = 0; g < G; g++) {
                float p = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; e++) p = fmaf(qr[g][e], kk[e], p);
                p = warp_sum(p);
                float mn = fmaxf(m[g], p);
                float corr = exp2f(m[g] - mn), w8 = exp2f(p - mn);
                l[g] = l[g] * corr + w8;
#pragma unroll
                for (int e = 0; e < EPL; e++) acc[g][e] = fmaf(w8, vv[e], acc[g][e] * corr);
                m[g] = mn;
            }
        }
    }
    // merge the 4 warps
    __shared__ float sm_m[4][G], sm_l[4][G];
    __shared__ float sm_acc[4][G][HD];
#pragma unroll
    for (int g = 0; g < G; g++) {
        if (lane == 0) { sm_m[warp][g] = m[g]; sm_l[warp][g] = l[g]; }
#pragma unroll
        for (int e = 0; e < EPL; e++) sm_acc[warp][g][lane * EPL + e] = acc[g][e];
    }
    __syncthreads();
    float* part = t.part + (((size_t)u * S + s) * G) * (HD + 2);
    for (int idx = threadIdx.x; idx < G * HD; idx += 128) {
        int g = idx / HD, e = idx % HD;
        float mm = fmaxf(fmaxf(sm_m[0][g], sm_m[1][g]), fmaxf(sm_m[2][g], sm_m[3][g]));
        float a = 0.f, ll = 0.f;
        if (mm != -INFINITY) {
#pragma unroll
            for (int w = 0; w < 4; w++) {
                float f = exp2f(sm_m[w][g] - mm);
                a += sm_acc[w][g][e] * f; ll += sm_l[w][g] * f;
            }
        }
        part[g * (HD + 2) + e] = a;
        if (e == 0) { part[g * (HD + 2) + HD] = mm; part[g * (HD + 2) + HD + 1] = ll; }
    }
}

// One block per unit: merge the S partials of every head and normalise.
template <int HD>
__global__ void __launch_bounds__(256) k_attn_combine(Tables t, StepPtrW outp, int S) {
    const int u = blockIdx.x;
    float* out = reinterpret_cast<float*>(outp.get()) + (size_t)u * t.G * HD;
    const float* part = t.part + ((size_t)u * S * t.G) * (HD + 2);
    for (int idx = threadIdx.x; idx < t.G * HD; idx += blockDim.x) {
        int g = idx / HD, e = idx % HD;
        float mm = -INFINITY;
        for (int s = 0; s < S; s++) mm = fmaxf(mm, part[((size_t)s * t.G + g) * (HD + 2) + HD]);
        float a = 0.f, ll = 0.f;
        if (mm != -INFINITY) {
            for (int s = 0; s < S; s++) {
                const float* ps = part + ((size_t)s * t.G + g) * (HD + 2);
                float f = exp2f(ps[HD] - mm);
                a += ps[e] * f; ll += ps[HD + 1] * f;
            }
        }
        out[idx] = ll > 0.f ? a / ll : 0.f;
    }
}

// ------------------------------------------------------------------ launchers

template <typename KV, int HD>
static void gather_attn_t(const Tables& t, StepPtr q, cudaStream_t s, long long* launches) {
    dim3 grid(t.n_splits_attn, t.U);
    switch (t.G) {
        case 1: k_gather_attn_v1<KV, HD, 1><<<grid, 128, 0, s>>>(t, q); break;
        case 2: k_gather_attn_v1<KV, HD, 2><<<grid, 128, 0, s>>>(t, q); break;
        case 3: k_gather_attn_v1<KV, HD, 3><<<grid, 128, 0, s>>>(t, q); break;
        case 4: k_gather_attn_v1<KV, HD, 4><<<grid, 128, 0, s>>>(t, q); break;
        case 5: k_gather_attn_v1<KV, HD, 5><<<grid, 128, 0, s>>>(t, q); break;
        case 6: k_gather_attn_v1<KV, HD, 6><<<grid, 128, 0, s>>>(t, q); break;
        case 7: k_gather_attn_v1<KV, HD, 7><<<grid, 128, 0, s>>>(t, q); break;
        default: k_gather_attn_v1<KV, HD, 8><<<grid, 128, 0, s>>>(t, q); break;
    }
    (*launches)++;
}

void launch_gather_attn_v1(const Tables& t, StepPtr q, cudaStream_t s, long long* launches) {
    if (t.kv_dtype == DYNAKV_F32) {
        if (t.d == 64) gather_attn_t<float, 64>(t, q, s, launches); else gather_attn_t<float, 128>(t, q, s, launches);
    } else {
        if (t.d == 64) gather_attn_t<__nv_bfloat16, 64>(t, q, s, launches); else gather_attn_t<__nv_bfloat16, 128>(t, q, s, launches);
    }
}

void launch_attn_combine(const Tables& t, StepPtrW out, cudaStream_t s, long long* launches) {
    if (t.d == 64) k_attn_combine<64><<<t.U, 256, 0, s>>>(t, out, t.n_splits_attn);
    else k_attn_combine<128><<<t.U, 256, 0, s>>>(t, out, t.n_splits_attn);
    (*launches)++;
}

}  // namespace dkv
