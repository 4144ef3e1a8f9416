// Front half of a decode step (arXiv 2511.07427, Section 4.1 and Algorithm 1):
//   k_front          one streaming pass over the fp32 representatives that produces both
//                    the query's score against every representative and the new key's
//                    squared distance to every representative (for its nearest-cluster
//                    assignment), so the centroid table is read once;
//   k_select         budgeted top-cluster selection by weighted radix select on the scores,
//                    then the flat (page, rows) work list of the selected clusters;
//   k_append_apply   argmin of the distances, incremental statistics, slot claim.
#include <float.h>

#include "append_block.cuh"
#include "common.cuh"
#include "front_rows.cuh"
#include "select_unit.cuh"

namespace dkv {

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
__global__ void __launch_bounds__(FR_THREADS, 2) k_front(Tables t, StepPtr qp, StepPtr kp, int has_q, int has_k, LoopBegin lb) {
    constexpr int V4 = HD / 32;   // float4 loads per lane per row
    constexpr int NIT = FR_ROWS / ((FR_THREADS / 32) * 4);
    const int u = blockIdx.y;
    const int j0 = blockIdx.x * FR_ROWS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane >> 3, l8 = lane & 7;
    pdl_wait();                          // inside a captured loop the representatives come from the iteration before
    if (lb.on && blockIdx.x == 0 && threadIdx.x == 0) {
        // opening a captured loop: this pass is step 0's and runs on the caller's arrays directly
        t.front_done[u] = 0; t.tail_queue[2 * u] = 0; t.tail_queue[2 * u + 1] = 0;
        if (u == 0) {
            *lb.step_ctr = 0; *lb.step_lim = lb.n_steps;
            t.plan_counter[1] = 0; t.tail_sync[0] = 0; t.tail_sync[1] = 0; t.tail_sync[2] = 0;
            lb.args[0] = lb.q; lb.args[1] = lb.k; lb.args[2] = lb.v; lb.args[3] = lb.out;
        }
    }
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
    if (has_k) front_key_load<KV, HD>(reinterpret_cast<const KV*>(kp.get()) + (size_t)u * HD, lane, kk, t.fp8);
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

// One block per unit: see select_unit().  Block size: 512 threads when all units fit the GPU in one wave (the
// shortest chain per block), 256 threads when there are more units than that (more blocks resident per SM; a
// block's time is latency, not work).
template <int THREADS, int MAXPER>
__global__ void __launch_bounds__(THREADS) k_select(Tables t, int budget, int* __restrict__ user_ids) {
    extern __shared__ __align__(16) unsigned char sel_dyn[];
    __shared__ int s_last;
    const SelectSmem sm = select_smem_at(sel_dyn, t.max_clusters);
    pdl_wait();                          // the scores come from the kernel before
    select_unit<THREADS, MAXPER>(t, blockIdx.x, budget, user_ids, sm);
    // ---- With more units than the gather-attention CTAs keep in shared memory, the last unit block to finish lays
    // the units' work lists end to end (otherwise every attention CTA does that itself from n_work).
    if (!t.attn_pf_in_smem) {
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            const int old = atomicAdd(t.plan_counter, 1);
            s_last = (old == t.U - 1) ? 1 : 0;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            work_prefix_block<THREADS>(t, sm.sh);
            if (threadIdx.x == 0) *t.plan_counter = 0;
        }
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

void launch_front(const Tables& t, StepPtr q, StepPtr k, int has_q, int has_k, cudaStream_t s, long long* launches,
                  const LoopBegin* lbp) {
    LoopBegin lb = {};
    if (lbp) lb = *lbp;
    dim3 grid((t.max_clusters + FR_ROWS - 1) / FR_ROWS, t.U);
    if (t.kv_dtype == DYNAKV_F32) {
        if (t.d == 64) launch_pdl(k_front<float, 64>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k, lb);
        else launch_pdl(k_front<float, 128>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k, lb);
    } else {
        if (t.d == 64) launch_pdl(k_front<__nv_bfloat16, 64>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k, lb);
        else launch_pdl(k_front<__nv_bfloat16, 128>, grid, dim3(FR_THREADS), 0, s, t, q, k, has_q, has_k, lb);
    }
    (*launches)++;
}

void launch_select(const Tables& t, int budget, int* user_sel_ids, cudaStream_t s, long long* launches) {
    const size_t smem = select_smem_bytes(t.max_clusters);
    // threads x ids per thread >= the unit's id capacity.  One wave of units: the shortest chain per block (512
    // threads, few ids each); more units than that: small blocks with few registers, many per SM.
    const bool one_wave = t.U <= t.n_attn_ctas;
    if (t.max_clusters > 2048 && one_wave) launch_pdl(k_select<512, 8>, dim3(t.U), dim3(512), smem, s, t, budget, user_sel_ids);
    else if (t.max_clusters > 2048) launch_pdl(k_select<256, 16>, dim3(t.U), dim3(256), smem, s, t, budget, user_sel_ids);
    else if (one_wave) launch_pdl(k_select<512, 4>, dim3(t.U), dim3(512), smem, s, t, budget, user_sel_ids);
    else if (t.max_clusters <= 1024) launch_pdl(k_select<256, 4>, dim3(t.U), dim3(256), smem, s, t, budget, user_sel_ids);
    else launch_pdl(k_select<256, 8>, dim3(t.U), dim3(256), smem, s, t, budget, user_sel_ids);
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
