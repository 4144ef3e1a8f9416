// Front half of a decode step (arXiv 2511.07427, Section 4.1 and Algorithm 1):
//   k_front          one streaming pass over the fp32 representatives that produces both
//                    the query scores ("similarity scores between q and all
//                    representatives") and the new key's squared distances ("assign new KV
//                    entry to its nearest cluster"), so the centroid table is read once;
//   k_select         budgeted top-cluster selection by weighted radix select on the scores,
//                    then the flat (page, rows) work list of the selected clusters;
//   k_append_apply   argmin of the distances, incremental statistics, slot claim.
#include <float.h>

#include "append_block.cuh"
#include "common.cuh"
#include "front_rows.cuh"

namespace dkv {

__device__ __forceinline__ unsigned int ord_key(float f) {
    unsigned int b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ------------------------------------------------------------------ k_front

constexpr int FR_THREADS = 256;
#ifndef DKV_FR_ROWS
#define DKV_FR_ROWS 128
#endif
constexpr int FR_ROWS = DKV_FR_ROWS;      // representatives per block (a multiple of 32)

// Grid (ceil(max_clusters / FR_ROWS), U).  Eight lanes share one representative row (each
// lane reads HD/8 floats as float4s), four rows per warp instruction.  Every global load of a
// thread -- its rows, their cluster sizes, its share of the query heads, the new key -- is issued
// before the first use of any of them, so a block pays one memory latency, not a chain of them.
template <typename KV, int HD>
__global__ void __launch_bounds__(FR_THREADS, 2) k_front(Tables t, StepPtr qp, StepPtr kp, int has_q, int has_k) {
    constexpr int V4 = HD / 32;   // float4 loads per lane per row
    constexpr int NIT = FR_ROWS / ((FR_THREADS / 32) * 4);
    const int u = blockIdx.y;
    const int j0 = blockIdx.x * FR_ROWS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane >> 3, l8 = lane & 7;
    pdl_wait();                          // inside a captured loop the representatives come from the iteration before
    // A unit never has fewer clusters than the build gave it: blocks wholly below that count need not
    // wait for the unit's current count before they issue their row loads.
    int jend = j0 + FR_ROWS;
    if (jend > t.M_floor) {
        const int Mcur = t.u_M[u];
        if (j0 >= Mcur) { pdl_trigger(); return; }
        jend = min(Mcur, jend);
    }
    const float* R = t.cl_r + (size_t)u * t.max_clusters * HD;
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    // rows of dead clusters are read too and masked afterwards, so no load waits for the cluster-size load
    float4 rv[NIT][V4];
    int cn[NIT];
#pragma unroll
    for (int it = 0; it < NIT; it++) {
        const int j = j0 + warp * 4 + sub + it * (FR_THREADS / 32) * 4;
        const bool in = j < jend;
        cn[it] = in ? CN[j] : 0;
#pragma unroll
        for (int i = 0; i < V4; i++)
            rv[it][i] = in ? __ldcs(reinterpret_cast<const float4*>(R + (size_t)j * HD + l8 * 4 + 32 * i)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // the unit's query heads (summed) and the new key, as this lane's share of a row
    float qs[V4][4], kk[V4][4];
#pragma unroll
    for (int i = 0; i < V4; i++)
#pragma unroll
        for (int e = 0; e < 4; e++) { qs[i][e] = 0.f; kk[i][e] = 0.f; }
    if (has_q) front_qsum_load<HD>(reinterpret_cast<const float*>(qp.get()) + (size_t)u * t.G * HD, t.G, lane, qs);
    if (has_k) front_key_load<KV, HD>(reinterpret_cast<const KV*>(kp.get()) + (size_t)u * HD, lane, kk);
    if (has_q) front_qsum_finish<HD>(qs);
    const float invG = 1.0f / (float)t.G;
    float* SC = t.scores + (size_t)u * t.max_clusters;
    float* DS = t.dists + (size_t)u * t.max_clusters;
#pragma unroll
    for (int it = 0; it < NIT; it++) {
        const int j = j0 + warp * 4 + sub + it * (FR_THREADS / 32) * 4;
        const bool in = j < jend;
        const bool live = in && cn[it] > 0;
        float s, dd;
        front_row<HD>(rv[it], qs, kk, s, dd);
        if (in && l8 == 0) {
            if (has_q) SC[j] = live ? s * invG : -INFINITY;
            if (has_k) DS[j] = live ? dd : INFINITY;
        }
    }
    pdl_trigger();
}

// ------------------------------------------------------------------ k_select

constexpr int SL_THREADS = 1024;
constexpr int SL_MAXM = 4096;
constexpr int SL_EPT = SL_MAXM / SL_THREADS;   // entries per thread

// One block per unit.  Finds, in (score descending, id ascending) order, the longest
// prefix of live clusters whose sizes sum to <= budget, by a three-level radix select on
// the orderable score key with the cluster sizes as weights; if not even the best cluster
// fits it is taken alone.  Writes the selection (id order) and its work list (first row, rows) of
// runs inside one page; when
// `user_ids` is given it also writes the selection in score order, -1 padded.  The last block
// to finish also writes the exclusive prefix of the units' work-list lengths.
__global__ void __launch_bounds__(SL_THREADS) k_select(Tables t, int budget, int* __restrict__ user_ids) {
    const int u = blockIdx.x, tid = threadIdx.x;
    __shared__ unsigned int keys[SL_MAXM];
    __shared__ int hist[2048];
    __shared__ int sh[33];
    __shared__ int s_bin, s_rem, s_done, s_eqtake, s_eqcnt, s_L, s_tok;
    __shared__ unsigned long long s_best;
    pdl_wait();                          // the scores come from the kernel before
    const int Mcur = t.u_M[u];
    const float* SC = t.scores + (size_t)u * t.max_clusters;
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    unsigned int key[SL_EPT]; int sz[SL_EPT];
    unsigned long long best = 0ull;
#pragma unroll
    for (int e = 0; e < SL_EPT; e++) {
        const int j = tid + e * SL_THREADS;
        key[e] = 0u; sz[e] = 0;
        if (j < Mcur) { sz[e] = CN[j]; if (sz[e] > 0) key[e] = ord_key(SC[j]); }
        keys[j] = key[e];
        if (sz[e] > 0) {
            unsigned long long kk = ((unsigned long long)key[e] << 32) | (unsigned long long)(0xffffffffu - (unsigned)j);
            best = kk > best ? kk : best;
        }
    }
    if (tid == 0) { s_rem = budget; s_done = 0; s_eqtake = 0; s_eqcnt = 0; s_L = 0; s_tok = 0; s_best = 0ull; }
    __syncthreads();
    // ---- radix select: digits [31:21], [20:10], [9:0]
    unsigned int prefix = 0u, pmask = 0u;
    const int shifts[3] = {21, 10, 0};
    const int nbins[3] = {2048, 2048, 1024};
    for (int lvl = 0; lvl < 3; lvl++) {
        for (int b = tid; b < 2048; b += SL_THREADS) hist[b] = 0;
        __syncthreads();
        if (s_done) break;
#pragma unroll
        for (int e = 0; e < SL_EPT; e++)
            if (sz[e] > 0 && (key[e] & pmask) == prefix) atomicAdd(&hist[(key[e] >> shifts[lvl]) & (nbins[lvl] - 1)], sz[e]);
        __syncthreads();
        // suffix sums over the bins, descending: thread i owns bins (nb-1-2i, nb-2-2i)
        const int nb = nbins[lvl];
        int b_hi = nb - 1 - 2 * tid, b_lo = nb - 2 - 2 * tid;
        int h_hi = b_hi >= 0 ? hist[b_hi] : 0, h_lo = b_lo >= 0 ? hist[b_lo] : 0;
        int tot;
        int before = block_scan_excl(h_hi + h_lo, sh, &tot);   // weight of all bins above b_hi
        const int rem = s_rem;
        __syncthreads();
        if (tid == 0 && tot <= rem) s_done = 1;                 // everything under this prefix fits
        // the boundary bin is the first (from the top) whose inclusive suffix sum exceeds rem
        if (b_hi >= 0 && before <= rem && before + h_hi > rem) { s_bin = b_hi; s_rem = rem - before; }
        else if (b_lo >= 0 && before + h_hi <= rem && before + h_hi + h_lo > rem) { s_bin = b_lo; s_rem = rem - before - h_hi; }
        __syncthreads();
        if (s_done) break;
        prefix |= (unsigned int)s_bin << shifts[lvl];
        pmask |= (unsigned int)(nb - 1) << shifts[lvl];
    }
    __syncthreads();
    // Selected: key above the boundary key; among clusters exactly at the boundary key, the
    // lowest ids while they still fit.  With s_done every key >= the current prefix range is in.
    const bool all_in = s_done != 0;
    const unsigned int kb = prefix;
    if (!all_in) {
        // a single cluster at the boundary key cannot fit (its bin overflowed the remaining budget);
        // only with several equal scores does the id-order walk matter
        int ne = 0;
#pragma unroll
        for (int e = 0; e < SL_EPT; e++) ne += (sz[e] > 0 && key[e] == kb) ? 1 : 0;
        if (ne) atomicAdd(&s_eqcnt, ne);
        __syncthreads();
        if (tid == 0 && s_eqcnt > 1) {
            int rem = s_rem, take = 0;
            for (int j = 0; j < Mcur; j++)
                if (keys[j] == kb && CN[j] > 0) { if (CN[j] <= rem) { rem -= CN[j]; take++; } else break; }
            s_eqtake = take;
        }
    }
    __syncthreads();
    // When all_in, pmask covers the levels already fixed: keys matching the prefix there, or larger, are selected.
    int selc = 0, tokc = 0;
    bool selected[SL_EPT];
#pragma unroll
    for (int e = 0; e < SL_EPT; e++) {
        bool in = false;
        if (sz[e] > 0) {
            if (all_in) in = (key[e] & pmask) >= prefix;
            else in = key[e] > kb;
        }
        selected[e] = in;
    }
    if (!all_in && s_eqtake > 0) {
        // the first s_eqtake clusters (by id) with key == kb are selected too
#pragma unroll
        for (int e = 0; e < SL_EPT; e++) {
            const int j = tid + e * SL_THREADS;
            if (sz[e] > 0 && key[e] == kb) {
                int rank = 0;
                for (int jj = 0; jj < j; jj++) rank += (keys[jj] == kb) ? 1 : 0;
                if (rank < s_eqtake) selected[e] = true;
            }
        }
    }
#pragma unroll
    for (int e = 0; e < SL_EPT; e++) if (selected[e]) { selc++; tokc += sz[e]; }
    if (selc) { atomicAdd(&s_L, selc); atomicAdd(&s_tok, tokc); }
    if (best) atomicMax(&s_best, best);
    __syncthreads();
    int L = s_L;
    if (L == 0 && budget > 0 && s_best != 0ull) {
        // not even the best cluster fits: take it alone
        const int jb = (int)(0xffffffffu - (unsigned)(s_best & 0xffffffffull));
#pragma unroll
        for (int e = 0; e < SL_EPT; e++) if (tid + e * SL_THREADS == jb) selected[e] = true;
        L = 1;
        if (tid == 0) { s_tok = CN[jb]; atomicOr(t.status, DYNAKV_ST_BUDGET_EXCEEDED); }
    }
    __syncthreads();
    // ---- compaction in id order + work list.  Thread-major order (j = tid + e*T) is not id
    // order, so scan one e-slab at a time.
    int* sel = t.sel_ids + (size_t)u * t.max_clusters;
    int2* work = t.work + (size_t)u * t.W;
    int sbase = 0, wbase = 0;
#pragma unroll
    for (int e = 0; e < SL_EPT; e++) {
        if (e * SL_THREADS >= Mcur) break;
        const int j = tid + e * SL_THREADS;
        const int isel = selected[e] ? 1 : 0;
        const int np = isel ? (sz[e] + ENTRY_ROWS - 1) / ENTRY_ROWS : 0;   // work entries: runs of <= ENTRY_ROWS rows inside one page
        int ts, tw;
        const int spos = sbase + block_scan_excl(isel, sh, &ts);
        const int wpos = wbase + block_scan_excl(np, sh, &tw);
        if (isel) {
            sel[spos] = j;
            int page = t.cl_head[(size_t)u * t.max_clusters + j];
            for (int i = 0; i < np && wpos + i < t.W; i++) {
                constexpr int EPP = PAGE / ENTRY_ROWS;       // entries per page
                work[wpos + i] = make_int2(page * PAGE + (i % EPP) * ENTRY_ROWS, min(ENTRY_ROWS, sz[e] - ENTRY_ROWS * i));
                if (i % EPP == EPP - 1) page = t.page_next[(size_t)u * t.P + page];
            }
        }
        sbase += ts; wbase += tw;
    }
    if (tid == 0) {
        t.sel_n[u] = L;
        t.sel_tokens[u] = s_tok;
        t.n_work[u] = min(wbase, t.W);
        atomicAdd(&t.counters[CNT_TOKENS_ATTENDED], (unsigned long long)s_tok);
        atomicAdd(&t.counters[CNT_CLUSTERS_SELECTED], (unsigned long long)L);
    }
    if (user_ids) {
        // score order: rank = number of selected clusters that come first
        __syncthreads();
        int* uo = user_ids + (size_t)u * t.max_clusters;
        for (int a = tid; a < L; a += SL_THREADS) {
            const int j = sel[a];
            const unsigned int kj = keys[j];
            int rank = 0;
            for (int b = 0; b < L; b++) {
                const int jb = sel[b];
                const unsigned int kq = keys[jb];
                rank += (kq > kj || (kq == kj && jb < j)) ? 1 : 0;
            }
            uo[rank] = j;
        }
        for (int p = L + tid; p < t.max_clusters; p += SL_THREADS) uo[p] = -1;
    }
    // ---- the last unit block to finish lays the units' work lists end to end: exclusive prefix of n_work
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int old = atomicAdd(t.plan_counter, 1);
        s_done = (old == t.U - 1) ? 1 : 0;
    }
    __syncthreads();
    if (s_done) {
        __threadfence();
        const int per_t = (t.U + SL_THREADS - 1) / SL_THREADS;
        const int b0 = min(tid * per_t, t.U), b1 = min(b0 + per_t, t.U);
        int sum = 0;
        for (int i = b0; i < b1; i++) sum += __ldcg(&t.n_work[i]);
        int tot;
        int base = block_scan_excl(sum, sh, &tot);
        for (int i = b0; i < b1; i++) { t.work_prefix[i] = base; base += __ldcg(&t.n_work[i]); }
        if (tid == 0) { t.work_prefix[t.U] = tot; *t.plan_counter = 0; }
    }
    pdl_trigger();
}

// ------------------------------------------------------------------ k_append_apply

// One block per unit: see append_block().
template <typename KV, int HD>
__global__ void __launch_bounds__(256) k_append_apply(Tables t, StepPtr kp_, StepPtr vp_) {
    append_block<KV, HD>(t, blockIdx.x, kp_, vp_);
}

// ------------------------------------------------------------------ launchers

void launch_front(const Tables& t, StepPtr q, StepPtr k, int has_q, int has_k, cudaStream_t s, long long* launches) {
    dim3 grid((t.max_clusters + FR_ROWS - 1) / FR_ROWS, t.U);
    if (t.kv_dtype == DYNAKV_F32) {
        if (t.d == 64) launch_pdl(k_front<float, 64>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k);
        else launch_pdl(k_front<float, 128>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k);
    } else {
        if (t.d == 64) launch_pdl(k_front<__nv_bfloat16, 64>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k);
        else launch_pdl(k_front<__nv_bfloat16, 128>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k);
    }
    (*launches)++;
}

void launch_select(const Tables& t, int budget, int* user_sel_ids, cudaStream_t s, long long* launches) {
    launch_pdl(k_select, dim3(t.U), dim3(SL_THREADS), 0, s, t, budget, user_sel_ids);
    (*launches)++;
}

void launch_append_apply(const Tables& t, StepPtr k, StepPtr v, cudaStream_t s, long long* launches) {
    if (t.kv_dtype == DYNAKV_F32) {
        if (t.d == 64) k_append_apply<float, 64><<<t.U, 256, 0, s>>>(t, k, v); else k_append_apply<float, 128><<<t.U, 256, 0, s>>>(t, k, v);
    } else {
        if (t.d == 64) k_append_apply<__nv_bfloat16, 64><<<t.U, 256, 0, s>>>(t, k, v); else k_append_apply<__nv_bfloat16, 128><<<t.U, 256, 0, s>>>(t, k, v);
    }
    (*launches)++;
}

}  // namespace dkv
