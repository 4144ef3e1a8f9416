// dynakv_attend_rows_noalloc: softmax attention of every unit's G query heads over ALL n rows of
// that unit's K/V, for callers that must not allocate device memory.
//
// Who needs this.  Code that runs where cudaMalloc is off limits: inside a region that a memory
// pool or a serving framework has frozen (every byte of the device already handed out), inside
// latency-critical loops where an allocation's implicit synchronisation is not acceptable, or
// in processes that are only allowed to launch kernels on buffers somebody else gave them.  The
// regular entry points allocate their arenas and scratch in dynakv_create / dynakv_build_index;
// this one allocates nothing at all.
//
// How.  It is a variant of the plain gather-attention kernel and its split-K combine
// (decode_kernels.cu): the rows are read in place from the caller's contiguous [U][n][d] arrays
// instead of from cluster pages, and the split-K partial records (acc, m, l) -- the scratch
// memory of that kernel pair -- live in a file-scope __device__ array of fixed size that every
// GPU loading the library carries until the process exits.
#include <atomic>
#include <float.h>

#include "common.cuh"

namespace dkv {

constexpr int NA_SPLITS = 16;                                  // split-K pieces per unit
constexpr size_t NA_SCRATCH_FLOATS = DYNAKV_NOALLOC_SCRATCH_BYTES / sizeof(float);

// The scratch.  In host code this name is only a stand-in (taking its address there does not yield
// a device address); the host obtains the real address once per device with cudaGetSymbolAddress.
static __device__ __align__(256) float g_noalloc_scratch[NA_SCRATCH_FLOATS];

// Grid (NA_SPLITS, U), 4 warps.  Split s of unit u owns rows [s*per, (s+1)*per); its warps take rows
// round-robin with the head dimension spread over the lanes and keep an online-softmax state per
// query head.  The block merges its warps and writes one unnormalised partial (acc[d], m, l) per head.
// Every record of the scratch that the combine reads is written here, empty splits included, so
// nothing in the scratch has to be cleared between calls.
template <typename KV, int HD, int G>
__global__ void __launch_bounds__(128) k_na_attend(const float* __restrict__ q_all, const KV* __restrict__ K,
                                                   const KV* __restrict__ V, long long n, float* __restrict__ part_all) {
    constexpr int EPL = HD / 32;
    const int s = blockIdx.x, u = blockIdx.y, S = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* q = q_all + (size_t)u * G * HD;
    const float scale = rsqrtf((float)HD) * 1.4426950408889634f;   // exp(x) = exp2(x * log2 e)
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
    const long long per = (n + S - 1) / S;
    const long long r0 = (long long)s * per, r1 = min(n, r0 + per);
    const KV* Ku = K + (size_t)u * n * HD;
    const KV* Vu = V + (size_t)u * n * HD;
    for (long long r = r0 + warp; r < r1; r += 4) {
        float kk[EPL], vv[EPL];
#pragma unroll
        for (int e = 0; e < EPL; e++) { kk[e] = to_f(Ku[(size_t)r * HD + lane * EPL + e]); vv[e] = to_f(Vu[(size_t)r * HD + lane * EPL + e]); }
#pragma unroll
        for (int g = 0; g < G; g++) {
            float p = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; e++) p = fmaf(qr[g][e], kk[e], p);
            p = warp_sum(p);
            const float mn = fmaxf(m[g], p);
            const float corr = exp2f(m[g] - mn), w = exp2f(p - mn);
            l[g] = l[g] * corr + w;
#pragma unroll
            for (int e = 0; e < EPL; e++) acc[g][e] = fmaf(w, vv[e], acc[g][e] * corr);
            m[g] = mn;
        }
    }
    __shared__ float sm_m[4][G], sm_l[4][G];
    __shared__ float sm_acc[4][G][HD];
#pragma unroll
    for (int g = 0; g < G; g++) {
        if (lane == 0) { sm_m[warp][g] = m[g]; sm_l[warp][g] = l[g]; }
#pragma unroll
        for (int e = 0; e < EPL; e++) sm_acc[warp][g][lane * EPL + e] = acc[g][e];
    }
    __syncthreads();
    float* part = part_all + (((size_t)u * S + s) * G) * (HD + 2);
    for (int idx = threadIdx.x; idx < G * HD; idx += 128) {
        const int g = idx / HD, e = idx % HD;
        const float mm = fmaxf(fmaxf(sm_m[0][g], sm_m[1][g]), fmaxf(sm_m[2][g], sm_m[3][g]));
        float a = 0.f, ll = 0.f;
        if (mm != -INFINITY) {
#pragma unroll
            for (int w = 0; w < 4; w++) {
                const float f = exp2f(sm_m[w][g] - mm);
                a += sm_acc[w][g][e] * f; ll += sm_l[w][g] * f;
            }
        }
        part[g * (HD + 2) + e] = a;
        if (e == 0) { part[g * (HD + 2) + HD] = mm; part[g * (HD + 2) + HD + 1] = ll; }
    }
}

// One block per unit: merge the S partials of every head and normalise (zeros when n == 0).
template <int HD>
__global__ void __launch_bounds__(256) k_na_combine(const float* __restrict__ part_all, int S, int G, float* __restrict__ out_all) {
    const int u = blockIdx.x;
    float* out = out_all + (size_t)u * G * HD;
    const float* part = part_all + ((size_t)u * S * G) * (HD + 2);
    for (int idx = threadIdx.x; idx < G * HD; idx += blockDim.x) {
        const int g = idx / HD, e = idx % HD;
        float mm = -INFINITY;
        for (int s = 0; s < S; s++) mm = fmaxf(mm, part[((size_t)s * G + g) * (HD + 2) + HD]);
        float a = 0.f, ll = 0.f;
        if (mm != -INFINITY) {
            for (int s = 0; s < S; s++) {
                const float* ps = part + ((size_t)s * G + g) * (HD + 2);
                const float f = exp2f(ps[HD] - mm);
                a += ps[e] * f; ll += ps[HD + 1] * f;
            }
        }
        out[idx] = ll > 0.f ? a / ll : 0.f;
    }
}

template <typename KV, int HD>
static void na_launch(const float* q, const void* K, const void* V, int U, long long n, int G, float* scratch, float* out,
                      cudaStream_t st) {
    dim3 grid(NA_SPLITS, U);
    const KV* k = reinterpret_cast<const KV*>(K);
    const KV* v = reinterpret_cast<const KV*>(V);
    switch (G) {
        case 1: k_na_attend<KV, HD, 1><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
        case 2: k_na_attend<KV, HD, 2><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
        case 3: k_na_attend<KV, HD, 3><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
        case 4: k_na_attend<KV, HD, 4><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
        case 5: k_na_attend<KV, HD, 5><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
        case 6: k_na_attend<KV, HD, 6><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
        case 7: k_na_attend<KV, HD, 7><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
        default: k_na_attend<KV, HD, 8><<<grid, 128, 0, st>>>(q, k, v, n, scratch); break;
    }
    k_na_combine<HD><<<U, 256, 0, st>>>(scratch, NA_SPLITS, G, out);
}

}  // namespace dkv

using namespace dkv;

// Device address of the scratch array, looked up once per device (with that device current).
static float* na_scratch_for_current_device(int* rc) {
    constexpr int MAX_DEV = 64;
    // threads may race to fill a device's slot; they all store the same address, and the slot is atomic
    static std::atomic<float*> ptr[MAX_DEV];
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= MAX_DEV) {
        *rc = DYNAKV_ERR_CUDA;
        return nullptr;
    }
    float* p = ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            *rc = DYNAKV_ERR_CUDA;
            return nullptr;
        }
        ptr[dev].store(p, std::memory_order_release);
    }
    *rc = DYNAKV_OK;
    return p;
}

extern "C" int dynakv_attend_rows_noalloc(const float* q, const void* K, const void* V, int32_t n_units, int64_t n,
                                          int32_t gqa_group, int32_t d, int32_t kv_dtype, float* out, void* cuda_stream) {
    if (!q || !K || !V || !out || n_units < 1 || n < 0 || gqa_group < 1 || gqa_group > MAX_G || (d != 64 && d != 128) ||
        (kv_dtype != DYNAKV_F32 && kv_dtype != DYNAKV_BF16)) {
        return DYNAKV_ERR_ARG;
    }
    const size_t need = (size_t)n_units * NA_SPLITS * gqa_group * (size_t)(d + 2);
    if (need > NA_SCRATCH_FLOATS || n_units > 65535) return DYNAKV_ERR_TOO_LARGE;   // more partial records than the fixed scratch holds
    int rc = DYNAKV_OK;
    float* scratch = na_scratch_for_current_device(&rc);
    if (!scratch) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    // an error left behind by an earlier, unrelated call on this thread must not be reported as this call's
    cudaGetLastError();
    if (kv_dtype == DYNAKV_F32) {
        if (d == 64) na_launch<float, 64>(q, K, V, n_units, n, gqa_group, scratch, out, st);
        else na_launch<float, 128>(q, K, V, n_units, n, gqa_group, scratch, out, st);
    } else {
        if (d == 64) na_launch<__nv_bfloat16, 64>(q, K, V, n_units, n, gqa_group, scratch, out, st);
        else na_launch<__nv_bfloat16, 128>(q, K, V, n_units, n, gqa_group, scratch, out, st);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        return DYNAKV_ERR_CUDA;
    }
    return DYNAKV_OK;
}
