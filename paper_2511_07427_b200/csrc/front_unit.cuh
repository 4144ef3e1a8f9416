// The centroid pass of ONE unit by one block, for the tail of a loop iteration: as soon as a unit's
// append and splits of step t are done, its block scores the unit's representatives against the
// query of step t + 1 and measures the distances of the key of step t + 1, while other units' blocks
// may still be splitting (units are independent, so nothing else has to be waited for).
//
// The unit's representatives are one contiguous array, so the block streams them through a three-stage
// shared-memory ring with bulk-asynchronous copies (TMA, 1-D) of one pass of rows each: thread 0 issues
// the copies, warp 0 waits on the stage's mbarrier with the rest of the block asleep in a barrier behind it,
// the pass is computed out of shared memory with the same row arithmetic as the stand-alone kernel, and the
// same barrier hands the stage back.
#pragma once

#include "bulk_copy.cuh"
#include "common.cuh"
#include "front_rows.cuh"

namespace dkv {

template <int THREADS, int HD> struct FrontUnit {
    static constexpr int ROWS = (THREADS / 32) * 4;          // rows per pass: four per warp
    static constexpr int STAGE_BYTES = ROWS * HD * 4;
};

// The pass comes in two calls so that its first copies are in flight while the block does its append:
// the append changes one row only (the representative of the cluster that took the new key), and that row
// is recomputed afterwards from the values the block itself wrote.
//
// front_unit_begin: called by all THREADS threads at the start of the block (thread 0 has initialised the two
// FR_STAGES mbarriers `bars` with count 1).  stages: 16-byte aligned shared memory of STAGE_BYTES each;
// live_s: shared bytes, one per cluster id of the unit.
template <typename KV, int HD>
__device__ __forceinline__ void front_patch(const Tables& t, int u, const float* __restrict__ q, const KV* __restrict__ k, int ja,
                                            const float* ra, int jb, const float* rb);

constexpr int FR_STAGES = 3;
template <int HD, int THREADS> struct FrontIssue {
    const float* R; int Mcur; unsigned bar[FR_STAGES], dst[FR_STAGES];
    static_assert(FR_STAGES == 3, "the selects below spell the stages out (no run-time indexing of register arrays)");
    __device__ __forceinline__ unsigned bar_of(int st) const { return st == 0 ? bar[0] : (st == 1 ? bar[1] : bar[2]); }
    __device__ __forceinline__ void operator()(int c) const {
        constexpr int ROWS = FrontUnit<THREADS, HD>::ROWS;
        const int rows = min(ROWS, Mcur - c * ROWS);
        const unsigned bytes = (unsigned)rows * HD * 4u;
        const int st = c % FR_STAGES;
        mbar_arrive_expect_tx(bar_of(st), bytes);
        bulk_g2s(st == 0 ? dst[0] : (st == 1 ? dst[1] : dst[2]), R + (size_t)c * ROWS * HD, bytes, bar_of(st));
    }
};
// stages: FR_STAGES pointers; the first two must be free from the start of the block, the third from the call of
// front_unit() on.
template <int HD, int THREADS>
__device__ __forceinline__ FrontIssue<HD, THREADS> front_unit_begin(const Tables& t, int u, unsigned char* const* stages,
                                                                    unsigned long long* bars, unsigned char* live_s) {
    constexpr int ROWS = FrontUnit<THREADS, HD>::ROWS;
    FrontIssue<HD, THREADS> is;
    is.Mcur = t.u_M[u];
    is.R = t.cl_r + (size_t)u * t.max_clusters * HD;
#pragma unroll
    for (int i = 0; i < FR_STAGES; i++) { is.bar[i] = smem_u32(&bars[i]); is.dst[i] = smem_u32(stages[i]); }
    const int nch = (is.Mcur + ROWS - 1) / ROWS;
    if (threadIdx.x == 0) {
        fence_proxy_async();
        if (nch > 0) is(0);
        if (nch > 1) is(1);
    }
    // which clusters are live does not change with an append (its target is live already)
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    for (int j = threadIdx.x; j < is.Mcur; j += THREADS) live_s[j] = CN[j] > 0 ? 1 : 0;
    return is;
}

// front_unit: the passes themselves, called by all THREADS threads after a __syncthreads() that follows
// front_unit_begin (and the block's append).  `appended` is the cluster the block's append went to (-1: none):
// its row is recomputed at the end from global memory.  Returns false (in every thread) when a bounded wait
// ran out; the status word is raised then.
template <typename KV, int HD, int THREADS>
__device__ __forceinline__ bool front_unit(const Tables& t, int u, const float* __restrict__ q, const KV* __restrict__ k,
                                           const FrontIssue<HD, THREADS>& issue, unsigned char* const* stages,
                                           unsigned char* live_s, int appended) {
    constexpr int V4 = HD / 32;
    constexpr int ROWS = FrontUnit<THREADS, HD>::ROWS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane >> 3, l8 = lane & 7;
    const int Mcur = issue.Mcur;
    const int nch = (Mcur + ROWS - 1) / ROWS;
    // the third stage is free now (the caller's barrier is behind every earlier use of that memory)
    if (tid == 0 && nch > 2) { fence_proxy_async(); issue(2); }
    float qs[V4][4], kk[V4][4];
    front_qsum_load<HD>(q, t.G, lane, qs);
    front_key_load<KV, HD>(k, lane, kk, t.fp8);
    front_qsum_finish<HD>(qs);
    const float invG = 1.0f / (float)t.G;
    float* SC = t.scores + (size_t)u * t.max_clusters;
    float* DS = t.dists + (size_t)u * t.max_clusters;
    // Only warp 0 polls the mbarriers; everybody else sleeps in the block barrier behind it, so a block that
    // waits for its data leaves the SM's issue slots to the block it shares the SM with.  One barrier per pass
    // says both "every thread is done with this stage" and "the next stage has landed".
    bool ok = true;
    if (warp == 0 && nch > 0) ok = mbar_wait(issue.bar[0], 0u);
    int failed_at = __syncthreads_or(ok ? 0 : 1) ? 0 : -1;        // also: live_s is complete
    for (int c = 0; c < nch && failed_at < 0; c++) {
        {
            // every lane of a warp goes through the row arithmetic (its shuffles name the full warp);
            // lanes of rows beyond the unit's last one compute on zeros and store nothing
            const int j = c * ROWS + warp * 4 + sub;
            const bool in = j < Mcur;
            const int st = c % FR_STAGES;
            const unsigned char* row = (st == 0 ? stages[0] : (st == 1 ? stages[1] : stages[2])) + (size_t)(warp * 4 + sub) * HD * 4;
            float4 rv[V4];
#pragma unroll
            for (int i = 0; i < V4; i++)
                rv[i] = in ? *reinterpret_cast<const float4*>(row + (l8 * 4 + 32 * i) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
            float s, dd;
            front_row<HD>(rv, qs, kk, s, dd);
            if (in && l8 == 0) {
                const bool live = live_s[j] != 0;
                SC[j] = live ? s * invG : -INFINITY;
                DS[j] = live ? dd : INFINITY;
            }
        }
        ok = true;
        if (warp == 0 && c + 1 < nch) ok = mbar_wait(issue.bar_of((c + 1) % FR_STAGES), (unsigned)((c + 1) / FR_STAGES) & 1u);
        if (__syncthreads_or(ok ? 0 : 1)) { failed_at = c + 1; break; }
        if (tid == 0 && c + FR_STAGES < nch) issue(c + FR_STAGES);
    }
    if (failed_at >= 0) {
        // a bounded wait ran out: report it, and let the copies still in flight (at most FR_STAGES passes from the
        // failed one on) land before the block's shared memory can be handed to another block
        if (tid == 0) {
            atomicOr(t.status, DYNAKV_ST_INTERNAL);
            for (int f = failed_at; f < nch && f < failed_at + FR_STAGES; f++)
                mbar_wait(issue.bar_of(f % FR_STAGES), (unsigned)(f / FR_STAGES) & 1u);
        }
        __syncthreads();
        return false;
    }
    // the appended cluster's row as the append left it (the pass may have seen it before, or half-way through, the update)
    if (appended >= 0 && warp == 0)
        front_patch<KV, HD>(t, u, q, k, appended, t.cl_r + ((size_t)u * t.max_clusters + appended) * HD, -1, nullptr);
    return true;
}

// The same two values for two single rows (the children of a split), by one full warp.  ra / rb point at the
// rows' HD floats (shared or global memory, written before a block barrier); both clusters are live.
template <typename KV, int HD>
__device__ __forceinline__ void front_patch(const Tables& t, int u, const float* __restrict__ q, const KV* __restrict__ k, int ja,
                                            const float* ra, int jb, const float* rb) {
    constexpr int V4 = HD / 32;
    const int lane = threadIdx.x & 31, sub = lane >> 3, l8 = lane & 7;
    float qs[V4][4], kk[V4][4];
    front_qsum_load<HD>(q, t.G, lane, qs);
    front_key_load<KV, HD>(k, lane, kk, t.fp8);
    front_qsum_finish<HD>(qs);
    const int j = sub == 0 ? ja : (sub == 1 ? jb : -1);
    const float* R = sub == 0 ? ra : rb;
    float4 rv[V4];
#pragma unroll
    for (int i = 0; i < V4; i++)
        rv[i] = j >= 0 ? *reinterpret_cast<const float4*>(R + l8 * 4 + 32 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
    float s, dd;
    front_row<HD>(rv, qs, kk, s, dd);
    if (j >= 0 && l8 == 0) {
        t.scores[(size_t)u * t.max_clusters + j] = s * (1.0f / (float)t.G);
        t.dists[(size_t)u * t.max_clusters + j] = dd;
    }
}

}  // namespace dkv
