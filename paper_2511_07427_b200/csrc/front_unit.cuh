// The centroid pass of ONE unit by one block, for the tail of a loop iteration: as soon as a unit's
// append and splits of step t are done, its block scores the unit's representatives against the
// query of step t + 1 and measures the distances of the key of step t + 1, while other units' blocks
// may still be splitting (units are independent, so nothing else has to be waited for).
//
// The unit's representatives are one contiguous array, so the block streams them through a two-stage
// shared-memory ring with bulk-asynchronous copies (TMA, 1-D) of one pass of rows each: thread 0 issues
// the copies, every thread waits on the stage's mbarrier, the pass is computed out of shared memory
// with the same row arithmetic as the stand-alone kernel, and a block barrier hands the stage back.
#pragma once

#include "bulk_copy.cuh"
#include "common.cuh"
#include "front_rows.cuh"

namespace dkv {

template <int THREADS, int HD> struct FrontUnit {
    static constexpr int ROWS = (THREADS / 32) * 4;          // rows per pass: four per warp
    static constexpr int STAGE_BYTES = ROWS * HD * 4;
};

// Called by all THREADS threads of the block, after a __syncthreads() that follows the block's own
// writes to the unit's tables.  stage0 / stage1: 16-byte aligned shared memory of STAGE_BYTES each;
// bars: two mbarriers initialised with count 1; live_s: shared bytes, one per cluster id of the unit.
// Returns false (in every thread) when a bounded wait ran out; the status word is raised then.
template <typename KV, int HD, int THREADS>
__device__ __forceinline__ bool front_unit(const Tables& t, int u, const float* __restrict__ q, const KV* __restrict__ k,
                                           unsigned char* stage0, unsigned char* stage1, unsigned long long* bars, unsigned char* live_s) {
    constexpr int V4 = HD / 32;
    constexpr int ROWS = FrontUnit<THREADS, HD>::ROWS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane >> 3, l8 = lane & 7;
    const int Mcur = t.u_M[u];
    const float* R = t.cl_r + (size_t)u * t.max_clusters * HD;
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    const int nch = (Mcur + ROWS - 1) / ROWS;
    // This block's append and splits wrote representatives with ordinary stores, and the ring's first stage
    // may alias shared memory written the same way: order all of that before the asynchronous proxy.
    __threadfence();
    fence_proxy_async();
    __syncthreads();
    const unsigned bar0 = smem_u32(&bars[0]), bar1 = smem_u32(&bars[1]);
    const unsigned dst0 = smem_u32(stage0), dst1 = smem_u32(stage1);
    auto issue = [&](int c) {
        const int rows = min(ROWS, Mcur - c * ROWS);
        const unsigned bytes = (unsigned)rows * HD * 4u;
        const unsigned bar = (c & 1) ? bar1 : bar0;
        mbar_arrive_expect_tx(bar, bytes);
        bulk_g2s((c & 1) ? dst1 : dst0, R + (size_t)c * ROWS * HD, bytes, bar);
    };
    if (tid == 0) {
        if (nch > 0) issue(0);
        if (nch > 1) issue(1);
    }
    for (int j = tid; j < Mcur; j += THREADS) live_s[j] = CN[j] > 0 ? 1 : 0;
    float qs[V4][4], kk[V4][4];
    front_qsum_load<HD>(q, t.G, lane, qs);
    front_key_load<KV, HD>(k, lane, kk);
    front_qsum_finish<HD>(qs);
    const float invG = 1.0f / (float)t.G;
    float* SC = t.scores + (size_t)u * t.max_clusters;
    float* DS = t.dists + (size_t)u * t.max_clusters;
    __syncthreads();                 // live_s is complete
    int failed_at = -1;
    for (int c = 0; c < nch; c++) {
        // warp-uniform outcome: the row arithmetic below is executed by whole warps or not at all
        const bool ok = __all_sync(0xffffffffu, mbar_wait((c & 1) ? bar1 : bar0, (unsigned)(c >> 1) & 1u) ? 1 : 0) != 0;
        if (ok) {
            // every lane of the warp goes through the row arithmetic (its shuffles name the full warp);
            // lanes of rows beyond the unit's last one compute on zeros and store nothing
            const int j = c * ROWS + warp * 4 + sub;
            const bool in = j < Mcur;
            const unsigned char* row = ((c & 1) ? stage1 : stage0) + (size_t)(warp * 4 + sub) * HD * 4;
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
        if (__syncthreads_or(ok ? 0 : 1)) { failed_at = c; break; }      // also: every thread is done with the stage
        if (tid == 0 && c + 2 < nch) issue(c + 2);
    }
    if (failed_at >= 0) {
        // a bounded wait ran out: report it, and let the copies still in flight land before the block's
        // shared memory can be handed to another block
        if (tid == 0) {
            atomicOr(t.status, DYNAKV_ST_INTERNAL);
            mbar_wait((failed_at & 1) ? bar1 : bar0, (unsigned)(failed_at >> 1) & 1u);
            if (failed_at + 1 < nch) mbar_wait(((failed_at + 1) & 1) ? bar1 : bar0, (unsigned)((failed_at + 1) >> 1) & 1u);
        }
        __syncthreads();
        return false;
    }
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
    front_key_load<KV, HD>(k, lane, kk);
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
