// Prefill kernels: seeded initial centres, fp32 nearest-centre assignment, centroid
// reduction, and the layout step that stores each cluster's members contiguously in pages
// (arXiv 2511.07427: NewCluster of Algorithm 1, Eq. 3-4, Section 5.1 placement).
#include <float.h>

#include "common.cuh"
#include "fp8_rows.cuh"

namespace dkv {

// ------------------------------------------------------------------ FP8 mode: rows rounded where they enter

// One warp per row of 128 bf16 elements: the row rounded to e4m3 values times the row's power-of-two scale, written
// back as bf16 (exact).  Every later kernel of the build works on these rows.
__global__ void __launch_bounds__(256) k_fp8_round_rows(const __nv_bfloat16* __restrict__ X, __nv_bfloat16* __restrict__ Y, long long rows) {
    const int lane = threadIdx.x & 31;
    long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nw = ((long long)gridDim.x * blockDim.x) >> 5;
    for (; w < rows; w += nw) {
        const float4 v = ld4(X + (size_t)w * 128, lane * 4);
        const float amax = group_max(fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))), 32);
        const int e = fp8_row_exp(amax);
        const float sc = pow2f(e), inv = pow2f(-e);
        const float2 a = fp8_round2(v.x, v.y, inv, sc), b = fp8_round2(v.z, v.w, inv, sc);
        __nv_bfloat162 o0 = __floats2bfloat162_rn(a.x, a.y), o1 = __floats2bfloat162_rn(b.x, b.y);
        uint2 pk;
        pk.x = *reinterpret_cast<unsigned*>(&o0); pk.y = *reinterpret_cast<unsigned*>(&o1);
        *reinterpret_cast<uint2*>(Y + (size_t)w * 128 + lane * 4) = pk;
    }
}

void launch_fp8_round_rows(const void* X, void* Y, long long rows, cudaStream_t s, long long* launches) {
    long long blocks = (rows + 7) / 8;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    k_fp8_round_rows<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(X), reinterpret_cast<__nv_bfloat16*>(Y), rows);
    (*launches)++;
}

// ------------------------------------------------------------------ init: k-means++

// One block per unit.  Exponential-race form of D^2 sampling: round 0 picks
// argmin_i E_i, round r picks argmax_i D2_i / E_i with E_i = -ln u(seed, unit, r, i);
// ties go to the lowest index.
template <typename KV, int HD>
__global__ void __launch_bounds__(1024) k_init_kmeanspp(const KV* __restrict__ K, int n, int M,
                                                        unsigned long long seed, float* __restrict__ C,
                                                        float* __restrict__ D2, int* __restrict__ picks) {
    const int u = blockIdx.x, tid = threadIdx.x;
    const KV* Ku = K + (size_t)u * n * HD;
    float* D2u = D2 + (size_t)u * n;
    __shared__ float cen[HD];
    __shared__ float red_v[32];
    __shared__ int red_i[32];
    __shared__ int s_pick;
    for (int r = 0; r < M; r++) {
        float bv = -FLT_MAX; int bi = 0x7fffffff;
        for (int i = tid; i < n; i += blockDim.x) {
            float uu = ((float)hash23(seed, u, r, i) + 0.5f) * (1.0f / 8388608.0f);
            float E = -logf(uu);
            float v;
            if (r == 0) v = -E;
            else {
                const KV* k = Ku + (size_t)i * HD;
                float dist = 0.f;
#pragma unroll 4
                for (int e = 0; e < HD; e += 4) {
                    float4 kk = ld4(k, e);
                    float a = kk.x - cen[e], b = kk.y - cen[e + 1], c = kk.z - cen[e + 2], dd = kk.w - cen[e + 3];
                    dist = fmaf(a, a, dist); dist = fmaf(b, b, dist); dist = fmaf(c, c, dist); dist = fmaf(dd, dd, dist);
                }
                float d2 = (r == 1) ? dist : fminf(D2u[i], dist);
                D2u[i] = d2;
                v = d2 / E;
            }
            if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o); int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if ((tid & 31) == 0) { red_v[tid >> 5] = bv; red_i[tid >> 5] = bi; }
        __syncthreads();
        if (tid < 32) {
            int nw = blockDim.x >> 5;
            bv = tid < nw ? red_v[tid] : -FLT_MAX; bi = tid < nw ? red_i[tid] : 0x7fffffff;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                float ov = __shfl_xor_sync(0xffffffffu, bv, o); int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (tid == 0) { s_pick = bi; picks[(size_t)u * M + r] = bi; }
        }
        __syncthreads();
        for (int e = tid; e < HD; e += blockDim.x) {
            float x = to_f(Ku[(size_t)s_pick * HD + e]);
            cen[e] = x;
            C[((size_t)u * M + r) * HD + e] = x;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ init: random distinct

// One block per unit.  Selects the M keys with the smallest (hash23, index) and lists
// them in index order: two histogram passes find the boundary hash value, a chunked
// ordered compaction writes the picks.
template <typename KV, int HD>
__global__ void __launch_bounds__(1024) k_init_random(const KV* __restrict__ K, int n, int M,
                                                      unsigned long long seed, float* __restrict__ C,
                                                      int* __restrict__ picks) {
    const int u = blockIdx.x, tid = threadIdx.x;
    __shared__ int hist[4096];
    __shared__ int sh[33];
    __shared__ int s_bin, s_before;
    // pass 1: top 12 bits
    for (int b = tid; b < 4096; b += blockDim.x) hist[b] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += blockDim.x) atomicAdd(&hist[hash23(seed, u, 0, i) >> 11], 1);
    __syncthreads();
    if (tid == 0) {
        int cum = 0, b = 0;
        for (; b < 4096; b++) { if (cum + hist[b] >= M) break; cum += hist[b]; }
        s_bin = b; s_before = cum;
    }
    __syncthreads();
    const int bin1 = s_bin; const int need1 = M - s_before;
    __syncthreads();
    // pass 2: low 11 bits inside the boundary bin
    for (int b = tid; b < 2048; b += blockDim.x) hist[b] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += blockDim.x) {
        unsigned int h = hash23(seed, u, 0, i);
        if ((int)(h >> 11) == bin1) atomicAdd(&hist[h & 2047], 1);
    }
    __syncthreads();
    if (tid == 0) {
        int cum = 0, b = 0;
        for (; b < 2048; b++) { if (cum + hist[b] >= need1) break; cum += hist[b]; }
        s_bin = b; s_before = cum;
    }
    __syncthreads();
    const unsigned int hstar = ((unsigned int)bin1 << 11) | (unsigned int)s_bin;
    const int need_eq = need1 - s_before;   // how many keys with hash == hstar are taken (lowest indices first)
    int eq_seen = 0, out_pos = 0;
    for (int base = 0; base < n; base += blockDim.x) {
        int i = base + tid;
        unsigned int h = i < n ? hash23(seed, u, 0, i) : 0xffffffffu;
        int is_eq = (i < n && h == hstar) ? 1 : 0;
        int tot_eq, tot_sel;
        int eq_rank = eq_seen + block_scan_excl(is_eq, sh, &tot_eq);
        int sel = (i < n && (h < hstar || (is_eq && eq_rank < need_eq))) ? 1 : 0;
        int pos = out_pos + block_scan_excl(sel, sh, &tot_sel);
        if (sel && pos < M) picks[(size_t)u * M + pos] = i;
        eq_seen += tot_eq; out_pos += tot_sel;
    }
    __syncthreads();
    const KV* Ku = K + (size_t)u * n * HD;
    for (int idx = tid; idx < M * HD; idx += blockDim.x) {
        int j = idx / HD, e = idx % HD;
        C[((size_t)u * M + j) * HD + e] = to_f(Ku[(size_t)picks[(size_t)u * M + j] * HD + e]);
    }
}

// ------------------------------------------------------------------ assign (fp32, direct form)

// a_i = argmin_j sum_t (k_it - c_jt)^2, ties to the lowest j.  Block tile: 128 keys x 64
// centres, whole head dimension staged in shared memory (transposed, so the inner loop
// reads 3 vectors per t); thread tile 8 keys x 4 centres.
constexpr int AS_BK = 128, AS_BC = 64, AS_THREADS = 256;
template <int HD> struct AssignSmem {
    static constexpr int KS = AS_BK + 4, CS = AS_BC + 4;
    static constexpr size_t bytes = sizeof(float) * ((size_t)HD * KS + (size_t)HD * CS);
};

// With `list` given (per unit: list[u][0 .. counts[u]) are key indices), only the listed keys are assigned.
template <typename KV, int HD>
__global__ void __launch_bounds__(AS_THREADS) k_assign_f32(const KV* __restrict__ K, int n, int M,
                                                           const float* __restrict__ C, int* __restrict__ assign,
                                                           const int* __restrict__ list, const unsigned* __restrict__ counts,
                                                           unsigned long long* __restrict__ listed_total) {
    extern __shared__ __align__(16) float smem[];
    constexpr int KS = AssignSmem<HD>::KS, CS = AssignSmem<HD>::CS;
    float* keysT = smem;                 // [HD][KS]
    float* centT = smem + (size_t)HD * KS;  // [HD][CS]
    const int u = blockIdx.y, tid = threadIdx.x;
    const KV* Ku = K + (size_t)u * n * HD;
    const float* Cu = C + (size_t)u * M * HD;
    const int ty = tid >> 4, tx = tid & 15;
    const int n_here = list ? (int)counts[u] : n;          // keys this unit has to assign
    const int* lu = list ? list + (size_t)u * n : nullptr;
    if (list && blockIdx.x == 0 && tid == 0 && n_here > 0) atomicAdd(listed_total, (unsigned long long)n_here);

    // the grid covers every 128-key tile of a full assignment; in list mode it is a few blocks per unit, each taking
    // the tiles of the (short, device-side) list in turn
    for (int key0 = blockIdx.x * AS_BK; key0 < n_here; key0 += gridDim.x * AS_BK) {
    for (int idx = tid; idx < AS_BK * (HD / 4); idx += AS_THREADS) {
        int key = idx % AS_BK, t4 = idx / AS_BK;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (key0 + key < n_here) v = ld4(Ku + (size_t)(lu ? lu[key0 + key] : key0 + key) * HD, t4 * 4);
        keysT[(t4 * 4 + 0) * KS + key] = v.x; keysT[(t4 * 4 + 1) * KS + key] = v.y;
        keysT[(t4 * 4 + 2) * KS + key] = v.z; keysT[(t4 * 4 + 3) * KS + key] = v.w;
    }
    float best[8]; int bj[8];
#pragma unroll
    for (int i = 0; i < 8; i++) { best[i] = FLT_MAX; bj[i] = 0x7fffffff; }

    for (int c0 = 0; c0 < M; c0 += AS_BC) {
        __syncthreads();
        for (int idx = tid; idx < AS_BC * (HD / 4); idx += AS_THREADS) {
            int c = idx % AS_BC, t4 = idx / AS_BC;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c0 + c < M) v = ld4(Cu + (size_t)(c0 + c) * HD, t4 * 4);
            centT[(t4 * 4 + 0) * CS + c] = v.x; centT[(t4 * 4 + 1) * CS + c] = v.y;
            centT[(t4 * 4 + 2) * CS + c] = v.z; centT[(t4 * 4 + 3) * CS + c] = v.w;
        }
        __syncthreads();
        float acc[8][4];
#pragma unroll
        for (int i = 0; i < 8; i++)
#pragma unroll
            for (int j = 0; j < 4; j++) acc[i][j] = 0.f;
#pragma unroll 4
        for (int t = 0; t < HD; t++) {
            float4 k0 = *reinterpret_cast<const float4*>(keysT + t * KS + ty * 8);
            float4 k1 = *reinterpret_cast<const float4*>(keysT + t * KS + ty * 8 + 4);
            float4 cc = *reinterpret_cast<const float4*>(centT + t * CS + tx * 4);
            float kk[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
            float cv[4] = {cc.x, cc.y, cc.z, cc.w};
#pragma unroll
            for (int i = 0; i < 8; i++)
#pragma unroll
                for (int j = 0; j < 4; j++) { float df = kk[i] - cv[j]; acc[i][j] = fmaf(df, df, acc[i][j]); }
        }
#pragma unroll
        for (int i = 0; i < 8; i++)
#pragma unroll
            for (int j = 0; j < 4; j++) {
                int cj = c0 + tx * 4 + j;
                if (cj < M && (acc[i][j] < best[i] || (acc[i][j] == best[i] && cj < bj[i]))) { best[i] = acc[i][j]; bj[i] = cj; }
            }
    }
#pragma unroll
    for (int i = 0; i < 8; i++) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, best[i], o); int oj = __shfl_xor_sync(0xffffffffu, bj[i], o);
            if (ov < best[i] || (ov == best[i] && oj < bj[i])) { best[i] = ov; bj[i] = oj; }
        }
        int key = key0 + ty * 8 + i;
        if (tx == 0 && key < n_here) assign[(size_t)u * n + (lu ? lu[key] : key)] = bj[i];
    }
    __syncthreads();          // the next tile's keys overwrite the staging area
    }
}

// ------------------------------------------------------------------ update (centroid reduction)

// One warp per key: add the key into its cluster's fp32 sum with vector atomics, count it.
template <typename KV, int HD>
__global__ void __launch_bounds__(256) k_update_sums(const KV* __restrict__ K, long long n_total, int n, int M,
                                                      const int* __restrict__ assign, float* __restrict__ sums,
                                                      int* __restrict__ counts) {
    const int lane = threadIdx.x & 31;
    long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (; w < n_total; w += nwarps) {
        int u = (int)(w / n);
        int j = assign[w];
        const KV* k = K + (size_t)w * HD;
        float* dst = sums + ((size_t)u * M + j) * HD;
        if (lane * 4 < HD) {
            float4 v = ld4(k, lane * 4);
            atomicAdd(reinterpret_cast<float4*>(dst + lane * 4), v);
        }
        if (lane == 0) atomicAdd(&counts[(size_t)u * M + j], 1);
    }
}

// Eq. 4 by member lists instead of atomic sums: count the members of every cluster, lay the key indices out cluster by
// cluster (a counting sort of the assignment), and let one warp per cluster add its members' rows in registers and
// write the new centre.  The keys are read once, as whole rows; the only atomics are the two integer ones per key.
__global__ void __launch_bounds__(256) k_upd_hist(const int* __restrict__ assign, long long n_total, int n, int M,
                                                   int* __restrict__ counts) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x; w < n_total; w += stride) {
        const int j = assign[w];
        if (j >= 0 && j < M) atomicAdd(&counts[(w / n) * M + j], 1);
    }
}
// One block per unit: exclusive prefix of the counts.
__global__ void __launch_bounds__(1024) k_upd_scan(const int* __restrict__ counts, int M, int* __restrict__ offset,
                                                    int* __restrict__ cursor) {
    __shared__ int sh[33];
    const int u = blockIdx.x;
    int run = 0;
    for (int base = 0; base < M; base += 1024) {
        const int j = base + threadIdx.x;
        const int c = j < M ? counts[(size_t)u * M + j] : 0;
        int tot;
        const int at = run + block_scan_excl(c, sh, &tot);
        if (j < M) { offset[(size_t)u * M + j] = at; cursor[(size_t)u * M + j] = at; }
        run += tot;
        __syncthreads();
    }
}
__global__ void __launch_bounds__(256) k_upd_scatter(const int* __restrict__ assign, long long n_total, int n, int M,
                                                      int* __restrict__ cursor, int* __restrict__ order) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x; w < n_total; w += stride) {
        const int j = assign[w];
        if (j < 0 || j >= M) continue;
        const long long u = w / n;
        const int pos = atomicAdd(&cursor[u * M + j], 1);
        if (pos >= 0 && pos < n) order[u * n + pos] = (int)(w - u * n);
    }
}
// One warp per (unit, cluster), the grid looping: the members' rows are added in list order, 4 elements per lane; an
// empty cluster keeps its centre.
template <typename KV, int HD>
__global__ void __launch_bounds__(256) k_upd_reduce(const KV* __restrict__ K, int U, int n, int M,
                                                     const int* __restrict__ counts, const int* __restrict__ offset,
                                                     const int* __restrict__ order, float* __restrict__ C) {
    const int lane = threadIdx.x & 31;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < (long long)U * M; w += nwarps) {
        const int u = (int)(w / M);
        const int c = counts[w];
        if (c <= 0) continue;
        const int* ord = order + (size_t)u * n + offset[w];
        const KV* Ku = K + (size_t)u * n * HD;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int m0 = 0; m0 < c; m0 += 32) {
            const int mine = (m0 + lane < c) ? ord[m0 + lane] : 0;         // 32 member indices with one load
            const int rows = min(32, c - m0);
#pragma unroll 8
            for (int r = 0; r < rows; r++) {
                const int i = __shfl_sync(0xffffffffu, mine, r);
                if (lane * 4 < HD) {
                    const float4 v = ld4(Ku + (size_t)i * HD, lane * 4);
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
            }
        }
        if (lane * 4 < HD) {
            const float fc = (float)c;
            *reinterpret_cast<float4*>(C + (size_t)w * HD + lane * 4) = make_float4(acc.x / fc, acc.y / fc, acc.z / fc, acc.w / fc);
        }
    }
}

// The same with sums that do not depend on the order of arrival: every element is rounded to a multiple of 2^-24 and
// added as a 64-bit integer.  Elements of 2^18 or more are clamped and reported.
constexpr float DET_SCALE = 16777216.f;     // 2^24
template <typename KV, int HD>
__global__ void __launch_bounds__(256) k_update_sums_det(const KV* __restrict__ K, long long n_total, int n, int M,
                                                          const int* __restrict__ assign, long long* __restrict__ sums,
                                                          int* __restrict__ counts, unsigned int* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (; w < n_total; w += nwarps) {
        int u = (int)(w / n);
        int j = assign[w];
        const KV* k = K + (size_t)w * HD;
        unsigned long long* dst = reinterpret_cast<unsigned long long*>(sums + ((size_t)u * M + j) * HD);
        if (lane * 4 < HD) {
            float4 v = ld4(k, lane * 4);
            const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; e++) {
                float xe = x[e];
                if (!(fabsf(xe) < 262144.f)) { atomicOr(status, DYNAKV_ST_INTERNAL); xe = xe != xe ? 0.f : copysignf(262143.f, xe); }
                atomicAdd(dst + lane * 4 + e, (unsigned long long)__float2ll_rn(xe * DET_SCALE));
            }
        }
        if (lane == 0) atomicAdd(&counts[(size_t)u * M + j], 1);
    }
}
__global__ void k_centroid_div_det(float* __restrict__ C, const long long* __restrict__ sums, const int* __restrict__ counts,
                                   long long total, int d) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    int c = counts[i / d];
    if (c > 0) C[i] = (float)(((double)sums[i] * (1.0 / 16777216.0)) / (double)c);
}

// c_j = sum_j / count_j; an empty cluster keeps its previous centre.
// (four elements per thread and a grid that loops: d is a multiple of 4, so a vector never straddles two clusters)
__global__ void __launch_bounds__(256) k_centroid_div(float* __restrict__ C, const float* __restrict__ sums,
                                                      const int* __restrict__ counts, long long total, int d) {
    const long long stride = (long long)gridDim.x * blockDim.x * 4;
    for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < total; i += stride) {
        const int c = counts[i / d];
        if (c > 0) {
            const float4 v = *reinterpret_cast<const float4*>(sums + i);
            const float fc = (float)c;
            *reinterpret_cast<float4*>(C + i) = make_float4(v.x / fc, v.y / fc, v.z / fc, v.w / fc);
        }
    }
}

// ------------------------------------------------------------------ finalize: layout

// One block per unit: page chains for every non-empty cluster (consecutive pages at build
// time), per-unit counters, cursors zeroed.
// `order` (optional, [U][M]): the clusters of the build in the order in which their pages follow one another in the
// pool (correlation-aware placement, Section 5.1); without it they follow one another by id.
__global__ void __launch_bounds__(1024) k_fin_layout(Tables t, int n, int M, const int* __restrict__ counts,
                                                     int* __restrict__ cursor, const int* __restrict__ order) {
    const int u = blockIdx.x, tid = threadIdx.x;
    __shared__ int sh[33];
    __shared__ int s_live;
    if (tid == 0) s_live = 0;
    __syncthreads();
    int page_base = 0, live = 0;
    for (int base = 0; base < t.max_clusters; base += blockDim.x) {
        const int pos = base + tid;                                   // position in the pool's order
        int j = (order && pos < M) ? order[(size_t)u * M + pos] : pos;
        int c = (j < M) ? counts[(size_t)u * M + j] : 0;
        int np = (c + PAGE - 1) / PAGE;
        int tot;
        int first = page_base + block_scan_excl(np, sh, &tot);
        if (j < t.max_clusters) {
            size_t cj = (size_t)u * t.max_clusters + j;
            t.cl_n[cj] = c;
            t.cl_flags[cj] = 0; t.cl_buf[cj] = 0;
            t.cl_M2[cj] = 0.f;
            t.cl_head[cj] = c > 0 ? first : -1;
            t.cl_tail[cj] = c > 0 ? first + np - 1 : -1;
            if (j < M) cursor[(size_t)u * M + j] = 0;
            for (int p = 0; p < np; p++) t.page_next[(size_t)u * t.P + first + p] = (p + 1 < np) ? first + p + 1 : -1;
            if (c > 0) live++;
        }
        page_base += tot;
    }
    atomicAdd(&s_live, live);
    __syncthreads();
    if (tid == 0) {
        t.u_N[u] = n; t.u_M[u] = M; t.u_Mlive[u] = s_live; t.u_page_top[u] = page_base; t.u_free_cnt[u] = 0;
        t.u_scan[u] = 1; t.u_last[u] = -1;
    }
    for (int i = n + tid; i < t.max_tokens; i += blockDim.x) t.tok_cluster[(size_t)u * t.max_tokens + i] = -1;
}

template <int BYTES> struct VecOf;
template <> struct VecOf<4> { using type = unsigned int; };
template <> struct VecOf<8> { using type = uint2; };
template <> struct VecOf<16> { using type = uint4; };

// One warp per token: claim the next slot of the token's cluster and copy its K, V rows.
template <typename KV, int HD>
__global__ void __launch_bounds__(256) k_fin_scatter(Tables t, const KV* __restrict__ K, const KV* __restrict__ V,
                                                      long long n_total, int n, int M, const int* __restrict__ assign,
                                                      int* __restrict__ cursor) {
    const int lane = threadIdx.x & 31;
    long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    KV* kp = reinterpret_cast<KV*>(t.kpages);
    KV* vp = reinterpret_cast<KV*>(t.vpages);
    for (; w < n_total; w += nwarps) {
        int u = (int)(w / n), i = (int)(w % n);
        int j = assign[w];
        int slot = 0;
        if (lane == 0) slot = atomicAdd(&cursor[(size_t)u * M + j], 1);
        slot = __shfl_sync(0xffffffffu, slot, 0);
        int page = t.cl_head[(size_t)u * t.max_clusters + j] + slot / PAGE, row = slot % PAGE;
        if (!DKV_IN(t, SITE_LAYOUT_PAGE, page, 0, t.P) || !DKV_IN(t, SITE_LAYOUT_PAGE, i, 0, t.max_tokens)) continue;
        const size_t dslot = ((size_t)u * t.P + page) * PAGE + row;
        size_t dst = dslot * HD;
        constexpr int EPL = HD / 32;   // elements per lane
        const int pos = row_pos<Epc<KV>::v>(dslot, lane * EPL);      // EPL elements stay inside one chunk
        const KV* ks = K + (size_t)w * HD + lane * EPL;
        const KV* vs = V + (size_t)w * HD + lane * EPL;
        if (!t.fp8) {
            // one store per lane and row (the EPL elements are contiguous on both sides and aligned to their total size)
            using Vec = typename VecOf<sizeof(KV) * EPL>::type;
            *reinterpret_cast<Vec*>(kp + dst + pos) = *reinterpret_cast<const Vec*>(ks);
            *reinterpret_cast<Vec*>(vp + dst + pos) = *reinterpret_cast<const Vec*>(vs);
        }
        if (t.fp8) {
            // the one-byte copy of the row (the rows are on the grid already, so this conversion is exact)
            if constexpr (HD == 128 && sizeof(KV) == 2) {
                const size_t slot = ((size_t)u * t.P + page) * PAGE + row;
#pragma unroll
                for (int side = 0; side < 2; side++) {
                    const KV* src = side == 0 ? ks : vs;
                    const float x0 = to_f(src[0]), x1 = to_f(src[1]), x2 = to_f(src[2]), x3 = to_f(src[3]);
                    const int ex = fp8_row_exp(group_max(fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3))), 32));
                    const float inv = pow2f(-ex);
                    const unsigned pk = (unsigned)fp8_pack2(x0, x1, inv) | ((unsigned)fp8_pack2(x2, x3, inv) << 16);
                    *reinterpret_cast<unsigned*>((side == 0 ? t.k8 : t.v8) + slot * HD + row_pos<16>(slot, lane * 4)) = pk;
                    if (lane == 0) (side == 0 ? t.k8e : t.v8e)[slot] = (signed char)ex;
                }
            }
        }
        if (lane == 0) {
            t.page_tok[((size_t)u * t.P + page) * PAGE + row] = i;
            t.tok_cluster[(size_t)u * t.max_tokens + i] = j;
        }
    }
}

// One warp per cluster: r_j = the final centre, M2_j = sum over members ||k - r_j||^2.
template <typename KV, int HD>
__global__ void __launch_bounds__(256) k_fin_stats(Tables t, int M, const float* __restrict__ C) {
    const int lane = threadIdx.x & 31;
    long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (w >= (long long)t.U * M) return;
    int u = (int)(w / M), j = (int)(w % M);
    size_t cj = (size_t)u * t.max_clusters + j;
    constexpr int EPL = HD / 32;
    float r[EPL];
#pragma unroll
    for (int e = 0; e < EPL; e++) {
        r[e] = C[((size_t)u * M + j) * HD + lane * EPL + e];
        t.cl_r[cj * HD + lane * EPL + e] = r[e];
    }
    int c = t.cl_n[cj];
    const KV* kp = reinterpret_cast<const KV*>(t.kpages);
    float m2 = 0.f;
    int page = t.cl_head[cj];
    for (int s = 0; s < c; s++) {
        int row = s % PAGE;
        if (s > 0 && row == 0) page = t.page_next[(size_t)u * t.P + page];
        if (!DKV_IN(t, SITE_STATS_PAGE, page, 0, t.P)) break;          // uniform in the warp
        const size_t kslot = ((size_t)u * t.P + page) * PAGE + row;
        float kx[EPL];
        load_key<KV, HD, EPL>(t, kslot, lane * EPL, kx);
        float part = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; e++) { float df = kx[e] - r[e]; part = fmaf(df, df, part); }
        m2 += warp_sum(part);
    }
    if (lane == 0) t.cl_M2[cj] = m2;
}

// One block per unit: tau = alpha * mean over live clusters of M2_j / n_j.
__global__ void __launch_bounds__(256) k_fin_tau(Tables t, int M, float alpha) {
    const int u = blockIdx.x;
    __shared__ float red[256];
    float s = 0.f;
    for (int j = threadIdx.x; j < M; j += blockDim.x) {
        size_t cj = (size_t)u * t.max_clusters + j;
        int c = t.cl_n[cj];
        if (c > 0) s += t.cl_M2[cj] / (float)c;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o]; __syncthreads(); }
    if (threadIdx.x == 0) t.u_tau[u] = alpha * red[0] / (float)max(t.u_Mlive[u], 1);
}

// ------------------------------------------------------------------ checkpoint: rows out in token order, partition in

// One block per (cluster, unit): the members' K and V rows go to [U][n][d] arrays at their token ids.
template <typename KV, int HD>
__global__ void __launch_bounds__(128) k_export_rows(Tables t, KV* __restrict__ Kout, KV* __restrict__ Vout, long long n) {
    const int j = blockIdx.x, u = blockIdx.y;
    if (j >= t.u_M[u]) return;
    const size_t cj = (size_t)u * t.max_clusters + j;
    const int c = t.cl_n[cj];
    const KV* kp = reinterpret_cast<const KV*>(t.kpages);
    const KV* vp = reinterpret_cast<const KV*>(t.vpages);
    int page = t.cl_head[cj];
    constexpr int V16 = HD * (int)sizeof(KV) / 16;        // 16-byte pieces per row
    for (int s0 = 0; s0 < c; s0 += PAGE) {
        const int rows = min(PAGE, c - s0);
        if (!DKV_IN(t, SITE_EXPORT_PAGE, page, 0, t.P)) break;           // uniform in the block
        for (int idx = threadIdx.x; idx < rows * V16; idx += blockDim.x) {
            const int r = idx / V16, v = idx % V16;
            const size_t slot = ((size_t)u * t.P + page) * PAGE + r;
            const int tok = t.page_tok[slot];
            if (tok < 0 || tok >= n) continue;
            const int pv = row_pos<1>(slot, v);          // in chunks
            if (t.fp8) {
                // FP8 storage keeps the rows as bytes: eight of them and the row's scale give this 16-byte piece back exactly
                if constexpr (HD == 128 && sizeof(KV) == 2) {
#pragma unroll
                    for (int side = 0; side < 2; side++) {
                        const uint2 by = *reinterpret_cast<const uint2*>((side == 0 ? t.k8 : t.v8) + slot * HD + row_pos<16>(slot, v * 8));
                        const float sc = pow2f((side == 0 ? t.k8e : t.v8e)[slot]);
                        KV* o8 = (side == 0 ? Kout : Vout) + ((size_t)u * n + tok) * HD + v * 8;
                        const unsigned w[2] = {by.x, by.y};
#pragma unroll
                        for (int h = 0; h < 2; h++) {
                            const float2 a = fp8_unpack2((unsigned short)(w[h] & 0xffffu), sc), b = fp8_unpack2((unsigned short)(w[h] >> 16), sc);
                            o8[4 * h] = (KV)a.x; o8[4 * h + 1] = (KV)a.y; o8[4 * h + 2] = (KV)b.x; o8[4 * h + 3] = (KV)b.y;
                        }
                    }
                }
            } else {
                reinterpret_cast<uint4*>(Kout + ((size_t)u * n + tok) * HD)[v] = reinterpret_cast<const uint4*>(kp + slot * HD)[pv];
                reinterpret_cast<uint4*>(Vout + ((size_t)u * n + tok) * HD)[v] = reinterpret_cast<const uint4*>(vp + slot * HD)[pv];
            }
        }
        page = t.page_next[(size_t)u * t.P + page];
    }
}

// A given partition's per-unit bookkeeping after the layout kernels have run with a common id count M: every unit
// gets its own number of ids in use and its threshold back.
__global__ void k_import_units(Tables t, const int* __restrict__ n_ids, const float* __restrict__ tau) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= t.U) return;
    t.u_M[u] = n_ids[u];
    t.u_tau[u] = tau[u];
}

template <typename KV, int HD>
static void export_rows_t(const Tables& t, void* K, void* V, long long n, cudaStream_t s) {
    k_export_rows<KV, HD><<<dim3(t.max_clusters, t.U), 128, 0, s>>>(t, (KV*)K, (KV*)V, n);
}

// ------------------------------------------------------------------ launchers

template <typename KV, int HD>
static void init_centres_t(const Tables& t, const void* K, long long n, int M, unsigned long long seed, int mode,
                           const BuildScratch& b, cudaStream_t s, long long* launches) {
    if (mode == DYNAKV_INIT_KMEANSPP)
        k_init_kmeanspp<KV, HD><<<t.U, 1024, 0, s>>>((const KV*)K, (int)n, M, seed, b.C, b.D2, b.picks);
    else
        k_init_random<KV, HD><<<t.U, 1024, 0, s>>>((const KV*)K, (int)n, M, seed, b.C, b.picks);
    (*launches)++;
}

#define DKV_DISPATCH(FN, ...)                                                             \
    do {                                                                                  \
        if (t.kv_dtype == DYNAKV_F32) {                                                   \
            if (t.d == 64) FN<float, 64>(__VA_ARGS__); else FN<float, 128>(__VA_ARGS__);  \
        } else {                                                                          \
            if (t.d == 64) FN<__nv_bfloat16, 64>(__VA_ARGS__); else FN<__nv_bfloat16, 128>(__VA_ARGS__); \
        }                                                                                 \
    } while (0)

void launch_init_centres(const Tables& t, const void* K, long long n, int M, unsigned long long seed,
                         int init_mode, const BuildScratch& b, cudaStream_t s, long long* launches) {
    DKV_DISPATCH(init_centres_t, t, K, n, M, seed, init_mode, b, s, launches);
}

template <typename KV, int HD>
static void assign_f32_t(const Tables& t, const void* K, long long n, int M, const float* C, int* assign,
                         const int* list, const unsigned* counts, unsigned long long* listed_total,
                         cudaStream_t s, long long* launches) {
    // the opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of the kernel instance
    static bool opted[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !opted[dev]) {
        cudaFuncSetAttribute(k_assign_f32<KV, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AssignSmem<HD>::bytes);
        if (dev >= 0 && dev < 64) opted[dev] = true;
    }
    // list mode: the lists hold well under one tile per unit on every workload seen (their length is known on the device
    // only); two blocks per unit loop over whatever there is instead of n / 128 blocks that mostly find nothing to do
    dim3 grid(list ? 2u : (unsigned)((n + AS_BK - 1) / AS_BK), t.U);
    k_assign_f32<KV, HD><<<grid, AS_THREADS, AssignSmem<HD>::bytes, s>>>((const KV*)K, (int)n, M, C, assign, list, counts,
                                                                       listed_total);
    (*launches)++;
}

void launch_assign_f32(const Tables& t, const void* K, long long n, int M, const float* C, int* assign,
                       cudaStream_t s, long long* launches) {
    const int* list = nullptr; const unsigned* counts = nullptr; unsigned long long* listed_total = nullptr;
    DKV_DISPATCH(assign_f32_t, t, K, n, M, C, assign, list, counts, listed_total, s, launches);
}

void launch_assign_f32_listed(const Tables& t, const void* K, long long n, int M, const float* C, int* assign,
                              const int* list, const unsigned* counts, unsigned long long* listed_total,
                              cudaStream_t s, long long* launches) {
    DKV_DISPATCH(assign_f32_t, t, K, n, M, C, assign, list, counts, listed_total, s, launches);
}

template <typename KV, int HD>
static void update_t(const Tables& t, const void* K, long long n, int M, const int* assign, const BuildScratch& b,
                     cudaStream_t s, long long* launches) {
    long long total = (long long)t.U * n;
    if (!t.det_sums && b.upd_order && b.upd_offset && b.upd_cursor) {
        cudaMemsetAsync(b.counts, 0, sizeof(int) * (size_t)t.U * M, s);
        const unsigned gb = (unsigned)((total + 255) / 256 < 148LL * 16 ? (total + 255) / 256 : 148LL * 16);
        k_upd_hist<<<gb, 256, 0, s>>>(assign, total, (int)n, M, b.counts);
        k_upd_scan<<<t.U, 1024, 0, s>>>(b.counts, M, b.upd_offset, b.upd_cursor);
        k_upd_scatter<<<gb, 256, 0, s>>>(assign, total, (int)n, M, b.upd_cursor, b.upd_order);
        const long long cw = (long long)t.U * M;
        const unsigned rb = (unsigned)((cw + 7) / 8 < 148LL * 16 ? (cw + 7) / 8 : 148LL * 16);
        k_upd_reduce<KV, HD><<<rb, 256, 0, s>>>((const KV*)K, t.U, (int)n, M, b.counts, b.upd_offset, b.upd_order, b.C);
        (*launches) += 4;
        return;
    }
    cudaMemsetAsync(b.sums, 0, sizeof(float) * (size_t)t.U * M * HD * (t.det_sums ? 2 : 1), s);
    cudaMemsetAsync(b.counts, 0, sizeof(int) * (size_t)t.U * M, s);
    long long blocks = (total + 7) / 8;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    long long cd = (long long)t.U * M * HD;
    if (t.det_sums) {
        long long* isums = reinterpret_cast<long long*>(b.sums);
        k_update_sums_det<KV, HD><<<(unsigned)blocks, 256, 0, s>>>((const KV*)K, total, (int)n, M, assign, isums, b.counts, t.status);
        k_centroid_div_det<<<(unsigned)((cd + 255) / 256), 256, 0, s>>>(b.C, isums, b.counts, cd, HD);
        (*launches) += 2;
        return;
    }
    k_update_sums<KV, HD><<<(unsigned)blocks, 256, 0, s>>>((const KV*)K, total, (int)n, M, assign, b.sums, b.counts);
    {
        long long db = (cd / 4 + 255) / 256;
        if (db > 148LL * 16) db = 148LL * 16;
        k_centroid_div<<<(unsigned)db, 256, 0, s>>>(b.C, b.sums, b.counts, cd, HD);
    }
    (*launches) += 2;
}

void launch_update(const Tables& t, const void* K, long long n, int M, const int* assign, const BuildScratch& b,
                   cudaStream_t s, long long* launches) {
    DKV_DISPATCH(update_t, t, K, n, M, assign, b, s, launches);
}

template <typename KV, int HD>
static void finalize_t(const Tables& t, const void* K, const void* V, long long n, int M, const BuildScratch& b,
                       float alpha, const int* order, cudaStream_t s, long long* launches) {
    k_fin_layout<<<t.U, 1024, 0, s>>>(t, (int)n, M, b.counts, b.cursor, order);
    long long total = (long long)t.U * n;
    long long blocks = (total + 7) / 8;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    k_fin_scatter<KV, HD><<<(unsigned)blocks, 256, 0, s>>>(t, (const KV*)K, (const KV*)V, total, (int)n, M, b.assign, b.cursor);
    long long nw = (long long)t.U * M;
    k_fin_stats<KV, HD><<<(unsigned)((nw + 7) / 8), 256, 0, s>>>(t, M, b.C);
    k_fin_tau<<<t.U, 256, 0, s>>>(t, M, alpha);
    (*launches) += 4;
}

void launch_finalize(const Tables& t, const void* K, const void* V, long long n, int M, const BuildScratch& b,
                     float alpha, cudaStream_t s, long long* launches, const int* order) {
    DKV_DISPATCH(finalize_t, t, K, V, n, M, b, alpha, order, s, launches);
}

// ------------------------------------------------------------------ correlation-aware placement (Section 5.1, Eq. 8)

// One block per unit, after a selection: every pair of clusters the query retrieved together is counted once, in both
// directions of the unit's M x M frequency matrix f (the adjacency matrix of retrieval frequencies).
__global__ void __launch_bounds__(256) k_pair_count(Tables t, int M, unsigned int* __restrict__ f) {
    const int u = blockIdx.x;
    const int L = t.sel_n[u];
    const int* sel = t.sel_ids + (size_t)u * t.max_clusters;
    unsigned int* fu = f + (size_t)u * M * M;
    for (int p = threadIdx.x; p < L * L; p += blockDim.x) {
        const int a = sel[p / L], b = sel[p % L];
        if (a != b && a < M && b < M) atomicAdd(&fu[(size_t)a * M + b], 1u);
    }
}

// One block per unit: a placement order from the frequencies.  The co-retrieval probability of Eq. 8 is f divided by
// one constant per unit, so ordering by f is ordering by it.  The order is a greedy chain: it starts at the cluster
// that was co-retrieved most often in all, and every next cluster is the one not yet placed that was co-retrieved
// most often with the one just placed (lowest id among equals; the lowest unplaced id when none ever was).
__global__ void __launch_bounds__(256) k_place_order(int M, const unsigned int* __restrict__ f, int* __restrict__ order) {
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned int* fu = f + (size_t)u * M * M;
    int* ou = order + (size_t)u * M;
    __shared__ unsigned int placed[128];           // one bit per cluster id (ids are below 4096)
    __shared__ unsigned long long best_s[8];
    __shared__ int cur_s;
    for (int i = tid; i < 128; i += 256) placed[i] = 0u;
    // key of a candidate: (frequency, then the lower id) as one 64-bit value to maximise
    auto key = [](unsigned long long freq, int id) -> unsigned long long { return (freq << 32) | (unsigned)(0x7fffffff - id); };
    auto block_max = [&](unsigned long long k) -> unsigned long long {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const unsigned long long y = __shfl_xor_sync(0xffffffffu, k, o); if (y > k) k = y; }
        __syncthreads();
        if (lane == 0) best_s[warp] = k;
        __syncthreads();
        unsigned long long r = best_s[0];
#pragma unroll
        for (int w = 1; w < 8; w++) if (best_s[w] > r) r = best_s[w];
        return r;
    };
    __syncthreads();
    // start: the largest row sum
    unsigned long long k0 = 0;
    for (int j = tid; j < M; j += 256) {
        unsigned long long sum = 0;
        for (int i = 0; i < M; i++) sum += fu[(size_t)j * M + i];
        const unsigned long long kj = key(sum > 0xffffffffull ? 0xffffffffull : sum, j);
        if (kj > k0) k0 = kj;
    }
    int cur = 0x7fffffff - (int)(block_max(k0) & 0xffffffffull);
    for (int p = 0; p < M; p++) {
        if (tid == 0) { ou[p] = cur; placed[cur >> 5] |= 1u << (cur & 31); }
        __syncthreads();
        if (p + 1 == M) break;
        unsigned long long kb = 0;
        for (int j = tid; j < M; j += 256) {
            if ((placed[j >> 5] >> (j & 31)) & 1u) continue;
            const unsigned long long kj = key(fu[(size_t)cur * M + j], j) | (1ull << 63);      // any unplaced id beats "none"
            if (kj > kb) kb = kj;
        }
        cur = 0x7fffffff - (int)(block_max(kb) & 0xffffffffull);
    }
}

void launch_pair_count(const Tables& t, int M, unsigned int* f, cudaStream_t s, long long* launches) {
    k_pair_count<<<t.U, 256, 0, s>>>(t, M, f);
    (*launches)++;
}
void launch_place_order(const Tables& t, int M, const unsigned int* f, int* order, cudaStream_t s, long long* launches) {
    k_place_order<<<t.U, 256, 0, s>>>(M, f, order);
    (*launches)++;
}

void launch_export_rows(const Tables& t, void* K, void* V, long long n, cudaStream_t s, long long* launches) {
    DKV_DISPATCH(export_rows_t, t, K, V, n, s);
    (*launches)++;
}

void launch_import_units(const Tables& t, const int* n_ids, const float* tau, cudaStream_t s, long long* launches) {
    k_import_units<<<(t.U + 255) / 256, 256, 0, s>>>(t, n_ids, tau);
    (*launches)++;
}

}  // namespace dkv
