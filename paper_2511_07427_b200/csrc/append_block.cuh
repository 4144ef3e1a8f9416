// The append of one decode step for one unit, as a block-level device function shared by the stand-alone
// append kernel and by the split-check kernel of the fused loop iteration (arXiv 2511.07427, Algorithm 1:
// nearest-cluster assignment of the new entry, UpdateVar, AddEntry, UpdateStats).
#pragma once

#include "common.cuh"
#include "fp8_rows.cuh"

namespace dkv {

// One block per unit: argmin over the distances written by k_front (ties to the lowest id; in the local-update
// mode only over the clusters born during decoding, and a first new entry founds a cluster of its own),
// then n <- n+1, delta = k - r, r <- r + delta/n, M2 <- M2 + delta.(k - r_new), and the
// (k, v) row goes to the next slot of the cluster's tail page (a fresh page is linked when
// the tail is full).  No stored entry moves.
// Called by every thread of a block (any block size that is a multiple of 32, up to 1024); contains one
// __syncthreads().  Global writes are made by warp 0; callers that go on reading them synchronise first.
// What an append did, for a caller that goes on to the split decision without reading the tables back.
struct AppendResult {
    int cluster;      // cluster that took the new entry, -1 when nothing was appended
    int n_new;        // its size after the append
    float M2_new;     // its M2 after the append
    int N_new;        // tokens of the unit after the append
};

// `res` (shared memory, may be null) is written by lane 0 of warp 0; the caller reads it after its own barrier.
template <typename KV, int HD>
__device__ __forceinline__ void append_block(const Tables& t, int u, StepPtr kp_, StepPtr vp_, AppendResult* res = nullptr) {
    constexpr int EPL = HD / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
    __shared__ float red_d[32];
    __shared__ int red_j[32];
    const int Mcur = t.u_M[u];
    const int N = t.u_N[u];
    if (res && tid == 0) { res->cluster = -1; res->n_new = 0; res->M2_new = 0.f; res->N_new = N; }
    if (N >= t.max_tokens) { if (tid == 0) atomicOr(t.status, DYNAKV_ST_MAX_TOKENS); return; }
    const float* DS = t.dists + (size_t)u * t.max_clusters;
    float bd = INFINITY; int bj = 0x7fffffff;
    // local-update mode: the clusters of the build (ids below M_floor) take no new entries
    const int j_first = t.update_mode == DYNAKV_MODE_LOCAL ? t.M_floor : 0;
    for (int j = j_first + tid; j < Mcur; j += blockDim.x) {
        const float dd = DS[j];
        if (dd < bd) { bd = dd; bj = j; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float od = __shfl_xor_sync(0xffffffffu, bd, o); const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
        if (od < bd || (od == bd && oj < bj)) { bd = od; bj = oj; }
    }
    if (lane == 0) { red_d[warp] = bd; red_j[warp] = bj; }
    __syncthreads();
    if (warp != 0) return;
    bd = red_d[0]; bj = red_j[0];
#pragma unroll
    for (int w = 1; w < nwarp; w++) if (red_d[w] < bd || (red_d[w] == bd && red_j[w] < bj)) { bd = red_d[w]; bj = red_j[w]; }
    const KV* knew = reinterpret_cast<const KV*>(kp_.get()) + (size_t)u * HD;
    const KV* vnew = reinterpret_cast<const KV*>(vp_.get()) + (size_t)u * HD;
    bool found = false;              // local-update mode: the entry founds a new cluster
    if (bj == 0x7fffffff && t.update_mode == DYNAKV_MODE_LOCAL) {
        if (Mcur < t.max_clusters) { bj = Mcur; found = true; }
        else {
            // no id left: the nearest cluster of all takes the entry
            if (lane == 0) atomicOr(t.status, DYNAKV_ST_MAX_CLUSTERS);
            for (int j = lane; j < Mcur; j += 32) {
                const float dd = DS[j];
                if (dd < bd || (dd == bd && j < bj)) { bd = dd; bj = j; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float od = __shfl_xor_sync(0xffffffffu, bd, o); const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
                if (od < bd || (od == bd && oj < bj)) { bd = od; bj = oj; }
            }
        }
    }
    if (bj == 0x7fffffff) return;    // no live cluster
    if (!DKV_IN(t, SITE_APPEND_CLUSTER, bj, 0, t.max_clusters)) return;
    const size_t cj = (size_t)u * t.max_clusters + bj;
    const int n_old = found ? 0 : t.cl_n[cj];
    int page = found ? -1 : t.cl_tail[cj];
    const int row = n_old % PAGE;
    if (row == 0) {   // tail is full (or there is no page yet): link a fresh page
        int np = -1;
        if (lane == 0) {
            int fc = t.u_free_cnt[u];
            if (fc > 0) { np = t.free_stack[(size_t)u * t.P + fc - 1]; t.u_free_cnt[u] = fc - 1; }
            else { int top = t.u_page_top[u]; if (top < t.P) { np = top; t.u_page_top[u] = top + 1; } }
            if (np >= 0 && !DKV_IN(t, SITE_APPEND_PAGE, np, 0, t.P)) np = -1;
            if (np >= 0 && page >= 0 && !DKV_IN(t, SITE_APPEND_PAGE, page, 0, t.P)) np = -1;
            if (np >= 0) {
                if (page >= 0) t.page_next[(size_t)u * t.P + page] = np; else t.cl_head[cj] = np;
                t.page_next[(size_t)u * t.P + np] = -1; t.cl_tail[cj] = np;
            } else atomicOr(t.status, DYNAKV_ST_PAGE_POOL);
        }
        np = __shfl_sync(0xffffffffu, np, 0);
        if (np < 0) return;
        page = np;
    }
    if (!DKV_IN(t, SITE_APPEND_PAGE, page, 0, t.P) || !DKV_IN(t, SITE_APPEND_TOKEN, N, 0, t.max_tokens)) return;
    const float n_new = (float)(n_old + 1);
    float* r = t.cl_r + cj * HD;
    float add = 0.f;
    float kk[EPL], vv[EPL];
#pragma unroll
    for (int e = 0; e < EPL; e++) { kk[e] = to_f(knew[lane * EPL + e]); vv[e] = to_f(vnew[lane * EPL + e]); }
    unsigned k8w = 0, v8w = 0;        // FP8 mode: the row's four bytes of this lane, and the rows' scale exponents
    int k8x = 0, v8x = 0;
    if (t.fp8) {
        // the new row enters the library here: round it to the storage grid (a warp holds the whole row)
        if constexpr (EPL == 4) {
            float am = fmaxf(fmaxf(fabsf(kk[0]), fabsf(kk[1])), fmaxf(fabsf(kk[2]), fabsf(kk[3])));
            k8x = fp8_row_exp(group_max(am, 32));
            am = fmaxf(fmaxf(fabsf(vv[0]), fabsf(vv[1])), fmaxf(fabsf(vv[2]), fabsf(vv[3])));
            v8x = fp8_row_exp(group_max(am, 32));
            const float ki = pow2f(-k8x), ks = pow2f(k8x), vi = pow2f(-v8x), vs = pow2f(v8x);
            k8w = (unsigned)fp8_pack2(kk[0], kk[1], ki) | ((unsigned)fp8_pack2(kk[2], kk[3], ki) << 16);
            v8w = (unsigned)fp8_pack2(vv[0], vv[1], vi) | ((unsigned)fp8_pack2(vv[2], vv[3], vi) << 16);
            float2 a = fp8_unpack2((unsigned short)(k8w & 0xffffu), ks), b = fp8_unpack2((unsigned short)(k8w >> 16), ks);
            kk[0] = a.x; kk[1] = a.y; kk[2] = b.x; kk[3] = b.y;
            a = fp8_unpack2((unsigned short)(v8w & 0xffffu), vs); b = fp8_unpack2((unsigned short)(v8w >> 16), vs);
            vv[0] = a.x; vv[1] = a.y; vv[2] = b.x; vv[3] = b.y;
        }
    }
#pragma unroll
    for (int e = 0; e < EPL; e++) {
        const float ro = found ? kk[e] : r[lane * EPL + e];          // a founded cluster starts at r = k, M2 = 0
        const float delta = kk[e] - ro;
        const float rn = ro + delta / n_new;
        r[lane * EPL + e] = rn;
        add = fmaf(delta, kk[e] - rn, add);
    }
    add = warp_sum(add);
    KV* kpg = reinterpret_cast<KV*>(t.kpages) + (((size_t)u * t.P + page) * PAGE + row) * HD;
    KV* vpg = reinterpret_cast<KV*>(t.vpages) + (((size_t)u * t.P + page) * PAGE + row) * HD;
    const size_t aslot = ((size_t)u * t.P + page) * PAGE + row;
    const int apos = row_pos<Epc<KV>::v>(aslot, lane * EPL);
#pragma unroll
    for (int e = 0; e < EPL; e++) if (!t.fp8) { kpg[apos + e] = (KV)kk[e]; vpg[apos + e] = (KV)vv[e]; }
    if (t.fp8) {
        const size_t slot = ((size_t)u * t.P + page) * PAGE + row;
        *reinterpret_cast<unsigned*>(t.k8 + slot * HD + row_pos<16>(slot, lane * 4)) = k8w;
        *reinterpret_cast<unsigned*>(t.v8 + slot * HD + row_pos<16>(slot, lane * 4)) = v8w;
        if (lane == 0) { t.k8e[slot] = (signed char)k8x; t.v8e[slot] = (signed char)v8x; }
    }
    if (lane == 0) {
        const float m2_new = found ? 0.f : t.cl_M2[cj] + add;
        t.cl_M2[cj] = m2_new;
        if (found) { t.u_M[u] = Mcur + 1; t.u_Mlive[u] = t.u_Mlive[u] + 1; }
        if (res) { res->cluster = bj; res->n_new = n_old + 1; res->M2_new = m2_new; res->N_new = N + 1; }
        t.cl_n[cj] = n_old + 1;
        const int fl = found ? 0 : t.cl_flags[cj];
        t.cl_flags[cj] = (unsigned char)(fl & ~FLAG_HOLD);
        if (fl & FLAG_SPLIT) t.cl_buf[cj] = t.cl_buf[cj] + 1;      // delayed-split mode: an entry for a flagged cluster is buffered
        t.page_tok[((size_t)u * t.P + page) * PAGE + row] = N;
        t.tok_cluster[(size_t)u * t.max_tokens + N] = bj;
        t.u_N[u] = N + 1;
        // an append whose split check is still owed, to another cluster: the next check has to scan them all
        const int owed = t.u_last[u];
        if (owed >= 0 && owed != bj) t.u_scan[u] = 1;
        t.u_last[u] = bj;
        atomicAdd(&t.counters[CNT_APPENDED], 1ull);
    }
}


}  // namespace dkv
