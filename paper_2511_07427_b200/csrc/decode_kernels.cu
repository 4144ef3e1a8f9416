// Decode-step kernels: centroid scoring + budgeted top-cluster selection, the baseline
// gather-attention over the selected clusters' pages with split-K combine, and the append
// of a new entry to its nearest cluster (arXiv 2511.07427, Section 4.1 retrieval,
// Algorithm 1 lines "Load top-k clusters", "Assign new KV entry", UpdateVar, AddEntry).
#include <float.h>

#include "common.cuh"

namespace dkv {

// ------------------------------------------------------------------ score + select

__device__ __forceinline__ unsigned int ord_f32(float f) {
    unsigned int b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

constexpr int SS_THREADS = 1024;
constexpr int SS_MAXM = 4096;

// One block per unit.  score_j = (sum_g q_g) . r_j / G for live clusters; 64-bit keys
// (orderable score, ~id) are bitonic-sorted descending, which orders by score descending
// then id ascending; the selected prefix is the longest one whose sizes sum to <= budget.
// Emits the ordered ids, the counts, and the flat (page, rows) work list of the selection.
template <int HD>
__global__ void __launch_bounds__(SS_THREADS) k_score_select(Tables t, StepPtr qp, int budget, int* __restrict__ user_ids) {
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int EPL = HD / 32;
    __shared__ unsigned long long keys[SS_MAXM];
    __shared__ int sh[33];
    __shared__ int s_L, s_live, s_tok;
    const float* q = reinterpret_cast<const float*>(qp.get()) + (size_t)u * t.G * HD;
    const int Mcur = t.u_M[u];
    int N = 32;
    while (N < Mcur) N <<= 1;
    float qs[EPL];
#pragma unroll
    for (int e = 0; e < EPL; e++) {
        float s = 0.f;
        for (int g = 0; g < t.G; g++) s += q[g * HD + lane * EPL + e];
        qs[e] = s;
    }
    const float invG = 1.0f / (float)t.G;
    if (tid == 0) { s_L = 0; s_live = 0; s_tok = 0; }
    const float* R = t.cl_r + (size_t)u * t.max_clusters * HD;
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    for (int j = warp; j < N; j += SS_THREADS / 32) {
        unsigned long long key = 0ull;
        if (j < Mcur && CN[j] > 0) {
            float p = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; e++) p = fmaf(qs[e], R[(size_t)j * HD + lane * EPL + e], p);
            p = warp_sum(p) * invG;
            if (lane == 0) t.scores[(size_t)u * t.max_clusters + j] = p;
            key = ((unsigned long long)ord_f32(p) << 32) | (unsigned long long)(0xffffffffu - (unsigned int)j);
        }
        if (lane == 0) keys[j] = key;
    }
    __syncthreads();
    // bitonic sort, descending
    for (int k = 2; k <= N; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < N; i += SS_THREADS) {
                int p = i ^ j;
                if (p > i) {
                    unsigned long long a = keys[i], b = keys[p];
                    bool desc = ((i & k) == 0);
                    if (desc ? (a < b) : (a > b)) { keys[i] = b; keys[p] = a; }
                }
            }
            __syncthreads();
        }
    }
    // cumulative sizes over the sorted order (4 consecutive entries per thread)
    int v[4], loc = 0, nlive = 0;
#pragma unroll
    for (int e = 0; e < 4; e++) {
        int p = tid * 4 + e;
        int sz = 0;
        if (p < N && keys[p] != 0ull) { sz = CN[0xffffffffu - (unsigned int)(keys[p] & 0xffffffffull)]; nlive++; }
        v[e] = sz; loc += sz;
    }
    int tot;
    int base = block_scan_excl(loc, sh, &tot);
    int cnt_ok = 0, tok_ok = 0;
#pragma unroll
    for (int e = 0; e < 4; e++) {
        base += v[e];
        if (v[e] > 0 && base <= budget) { cnt_ok++; tok_ok += v[e]; }
    }
    if (cnt_ok) { atomicAdd(&s_L, cnt_ok); atomicAdd(&s_tok, tok_ok); }
    if (nlive) atomicAdd(&s_live, nlive);
    __syncthreads();
    int L = s_L, tokens = s_tok;
    if (L == 0 && budget > 0 && s_live > 0) {
        L = 1;
        tokens = CN[0xffffffffu - (unsigned int)(keys[0] & 0xffffffffull)];
        if (tid == 0) atomicOr(t.status, DYNAKV_ST_BUDGET_EXCEEDED);
    }
    int* sel = t.sel_ids + (size_t)u * t.max_clusters;
    // page counts of the selected clusters -> work-list offsets
    int2* work = t.work + (size_t)u * t.W;
    int wbase = 0;
    for (int b0 = 0; b0 < L; b0 += SS_THREADS) {
        int p = b0 + tid;
        int id = -1, sz = 0, np = 0;
        if (p < L) {
            id = (int)(0xffffffffu - (unsigned int)(keys[p] & 0xffffffffull));
            sz = CN[id]; np = (sz + PAGE - 1) / PAGE;
            sel[p] = id;
        }
        int wtot;
        int off = wbase + block_scan_excl(np, sh, &wtot);
        if (p < L) {
            int page = t.cl_head[(size_t)u * t.max_clusters + id];
            for (int i = 0; i < np && off + i < t.W; i++) {
                work[off + i] = make_int2(page, (i + 1 < np) ? PAGE : sz - PAGE * (np - 1));
                page = t.page_next[(size_t)u * t.P + page];
            }
        }
        wbase += wtot;
    }
    if (tid == 0) {
        t.sel_n[u] = L;
        t.sel_tokens[u] = tokens;
        t.n_work[u] = min(wbase, t.W);
        atomicAdd(&t.counters[CNT_TOKENS_ATTENDED], (unsigned long long)tokens);
        atomicAdd(&t.counters[CNT_CLUSTERS_SELECTED], (unsigned long long)L);
    }
    if (user_ids) {
        int* uo = user_ids + (size_t)u * t.max_clusters;
        for (int p = tid; p < t.max_clusters; p += SS_THREADS)
            uo[p] = p < L ? (int)(0xffffffffu - (unsigned int)(keys[p] & 0xffffffffull)) : -1;
    }
}

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
        size_t pbase = (((size_t)u * t.P + ent.x) * PAGE) * HD;
        for (int r = 0; r < ent.y; r++) {
            const KV* k = kp + pbase + (size_t)r * HD + lane * EPL;
            const KV* v = vp + pbase + (size_t)r * HD + lane * EPL;
            float kk[EPL], vv[EPL];
#pragma unroll
            for (int e = 0; e < EPL; e++) { kk[e] = to_f(k[e]); vv[e] = to_f(v[e]); }
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

// ------------------------------------------------------------------ append

// One block per unit (8 warps).  Nearest live representative in squared Euclidean
// distance (ties to the lowest id), incremental statistics
//   n <- n+1, delta = k - r, r <- r + delta/n, M2 <- M2 + delta.(k - r_new),
// and the (k, v) row goes to the next slot of the cluster's tail page; a fresh page is
// linked when the tail is full.  No stored entry moves.
template <typename KV, int HD>
__global__ void __launch_bounds__(256) k_append(Tables t, StepPtr kp_, StepPtr vp_) {
    constexpr int EPL = HD / 32;
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const KV* knew = reinterpret_cast<const KV*>(kp_.get()) + (size_t)u * HD;
    const KV* vnew = reinterpret_cast<const KV*>(vp_.get()) + (size_t)u * HD;
    __shared__ float red_d[8];
    __shared__ int red_j[8];
    const int Mcur = t.u_M[u];
    const int N = t.u_N[u];
    if (N >= t.max_tokens) { if (tid == 0) atomicOr(t.status, DYNAKV_ST_MAX_TOKENS); return; }
    float kk[EPL];
#pragma unroll
    for (int e = 0; e < EPL; e++) kk[e] = to_f(knew[lane * EPL + e]);
    const float* R = t.cl_r + (size_t)u * t.max_clusters * HD;
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    float bd = FLT_MAX; int bj = 0x7fffffff;
    for (int j = warp; j < Mcur; j += 8) {
        if (CN[j] <= 0) continue;
        float p = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; e++) { float df = kk[e] - R[(size_t)j * HD + lane * EPL + e]; p = fmaf(df, df, p); }
        p = warp_sum(p);
        if (p < bd) { bd = p; bj = j; }
    }
    if (lane == 0) { red_d[warp] = bd; red_j[warp] = bj; }
    __syncthreads();
    if (warp != 0) return;
    bd = red_d[0]; bj = red_j[0];
#pragma unroll
    for (int w = 1; w < 8; w++) if (red_d[w] < bd || (red_d[w] == bd && red_j[w] < bj)) { bd = red_d[w]; bj = red_j[w]; }
    if (bj == 0x7fffffff) return;    // no live cluster
    const size_t cj = (size_t)u * t.max_clusters + bj;
    const int n_old = CN[bj];
    int page = t.cl_tail[cj];
    const int row = n_old % PAGE;
    if (row == 0) {   // tail is full: link a fresh page
        int np = -1;
        if (lane == 0) {
            int fc = t.u_free_cnt[u];
            if (fc > 0) { np = t.free_stack[(size_t)u * t.P + fc - 1]; t.u_free_cnt[u] = fc - 1; }
            else { int top = t.u_page_top[u]; if (top < t.P) { np = top; t.u_page_top[u] = top + 1; } }
            if (np >= 0) { t.page_next[(size_t)u * t.P + page] = np; t.page_next[(size_t)u * t.P + np] = -1; t.cl_tail[cj] = np; }
            else atomicOr(t.status, DYNAKV_ST_PAGE_POOL);
        }
        np = __shfl_sync(0xffffffffu, np, 0);
        if (np < 0) return;
        page = np;
    }
    // statistics
    const float n_new = (float)(n_old + 1);
    float* r = t.cl_r + cj * HD;
    float add = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; e++) {
        float ro = r[lane * EPL + e];
        float delta = kk[e] - ro;
        float rn = ro + delta / n_new;
        r[lane * EPL + e] = rn;
        add = fmaf(delta, kk[e] - rn, add);
    }
    add = warp_sum(add);
    KV* kpg = reinterpret_cast<KV*>(t.kpages) + (((size_t)u * t.P + page) * PAGE + row) * HD;
    KV* vpg = reinterpret_cast<KV*>(t.vpages) + (((size_t)u * t.P + page) * PAGE + row) * HD;
#pragma unroll
    for (int e = 0; e < EPL; e++) { kpg[lane * EPL + e] = knew[lane * EPL + e]; vpg[lane * EPL + e] = vnew[lane * EPL + e]; }
    if (lane == 0) {
        t.cl_M2[cj] += add;
        t.cl_n[cj] = n_old + 1;
        t.cl_flags[cj] &= ~FLAG_HOLD;
        t.page_tok[((size_t)u * t.P + page) * PAGE + row] = N;
        t.tok_cluster[(size_t)u * t.max_tokens + N] = bj;
        t.u_N[u] = N + 1;
        atomicAdd(&t.counters[CNT_APPENDED], 1ull);
    }
}

__global__ void k_step_inc(int* ctr) { *ctr += 1; }

// ------------------------------------------------------------------ launchers

void launch_score_select(const Tables& t, StepPtr q, int budget, int* user_sel_ids, cudaStream_t s, long long* launches) {
    if (t.d == 64) k_score_select<64><<<t.U, SS_THREADS, 0, s>>>(t, q, budget, user_sel_ids);
    else k_score_select<128><<<t.U, SS_THREADS, 0, s>>>(t, q, budget, user_sel_ids);
    (*launches)++;
}

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

void launch_append(const Tables& t, StepPtr k, StepPtr v, cudaStream_t s, long long* launches) {
    if (t.kv_dtype == DYNAKV_F32) {
        if (t.d == 64) k_append<float, 64><<<t.U, 256, 0, s>>>(t, k, v); else k_append<float, 128><<<t.U, 256, 0, s>>>(t, k, v);
    } else {
        if (t.d == 64) k_append<__nv_bfloat16, 64><<<t.U, 256, 0, s>>>(t, k, v); else k_append<__nv_bfloat16, 128><<<t.U, 256, 0, s>>>(t, k, v);
    }
    (*launches)++;
}

void launch_step_inc(int* ctr, cudaStream_t s, long long* launches) {
    k_step_inc<<<1, 1, 0, s>>>(ctr);
    (*launches)++;
}

}  // namespace dkv
