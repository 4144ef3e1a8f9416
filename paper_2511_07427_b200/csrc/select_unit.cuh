// Budgeted top-cluster selection of ONE unit by one block (arXiv 2511.07427, Section 4.1: the clusters with
// the highest query scores are retrieved; here up to a token budget).  In (score descending, id ascending)
// order the longest prefix of live clusters whose sizes sum to <= budget is selected, by a three-level
// weighted radix select on an order-preserving integer image of the score; if not even the best cluster
// fits it is taken alone.  The block then writes the selection in id order and the flat work list of the
// selected clusters' rows: entries (first row, rows <= ENTRY_ROWS), each inside one page.
//
// A device function for any block size (a multiple of 32), so that the stand-alone selection kernel and the
// tail kernel of a loop iteration share one implementation.  Per-cluster state lives in shared memory.
#pragma once

#include "common.cuh"

namespace dkv {

constexpr int SL_MAXM = 4096;          // most cluster ids a unit can have (dynakv_create enforces it)

// The block's working set, carved out of shared memory by the caller: `ids` is the unit's id capacity
// (max_clusters), so small configurations leave room for more resident blocks.
struct SelectSmem {
    unsigned int* keys;                // [ids] orderable score of every cluster id (0 = dead / beyond the unit's ids)
    int* sizes;                        // [ids] cluster sizes; the sign bit marks "selected" at the end
    int* hist;                         // [2048]
    int* sh;                           // [33]
    int* sc;                           // [8] scalars: SEL_bin .. SEL_tok below
    unsigned long long* best64;        // [1]
};
#define SEL_bin sm.sc[0]
#define SEL_rem sm.sc[1]
#define SEL_done sm.sc[2]
#define SEL_eqtake sm.sc[3]
#define SEL_eqcnt sm.sc[4]
#define SEL_L sm.sc[5]
#define SEL_tok sm.sc[6]
#define SEL_best (*sm.best64)
__host__ __device__ constexpr size_t select_smem_bytes(int ids) { return (size_t)ids * 8 + 2048 * 4 + 48 * 4 + 8 + 16; }
__device__ __forceinline__ SelectSmem select_smem_at(unsigned char* base, int ids) {      // base: 8-byte aligned
    SelectSmem sm;
    sm.best64 = reinterpret_cast<unsigned long long*>(base);
    sm.keys = reinterpret_cast<unsigned int*>(base + 8);
    sm.sizes = reinterpret_cast<int*>(sm.keys + ids);
    sm.hist = sm.sizes + ids;
    sm.sh = sm.hist + 2048;
    sm.sc = sm.sh + 36;
    return sm;
}

__device__ __forceinline__ unsigned int ord_key(float f) {
    unsigned int b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Called by every thread of the block.  scores: the unit's scores in global memory (written before a barrier or
// by an earlier kernel).  user_ids (may be null): the selection in score order, -1 padded, [max_clusters].
// On return (all global writes issued; no trailing barrier) thread 0 has written sel_n / sel_tokens / n_work.
// buf: which copy of the work lists to write (0 outside a captured loop).
template <int THREADS>
__device__ void select_unit(const Tables& t, int u, int budget, int* __restrict__ user_ids, const SelectSmem& sm, int buf = 0) {
    const int tid = threadIdx.x;
    const float* SC = t.scores + (size_t)u * t.max_clusters;
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    // A unit never has fewer ids than the build gave it, so the first id of every thread below that count is
    // loaded without waiting for the unit's current count.
    const bool early = tid < t.M_floor;
    int sz0 = 0; float sc0 = 0.f;
    if (early) { sz0 = __ldcg(CN + tid); sc0 = __ldcg(SC + tid); }
    const int Mcur = __ldcg(&t.u_M[u]);
    unsigned long long best = 0ull;
    for (int j = tid; j < Mcur; j += THREADS) {
        const int sz = (j == tid && early) ? sz0 : __ldcg(CN + j);
        const unsigned int key = sz > 0 ? ord_key((j == tid && early) ? sc0 : __ldcg(SC + j)) : 0u;
        sm.keys[j] = key; sm.sizes[j] = sz;
        if (sz > 0) {
            const unsigned long long kk = ((unsigned long long)key << 32) | (unsigned long long)(0xffffffffu - (unsigned)j);
            best = kk > best ? kk : best;
        }
    }
    if (tid == 0) { SEL_rem = budget; SEL_done = 0; SEL_eqtake = 0; SEL_eqcnt = 0; SEL_L = 0; SEL_tok = 0; SEL_best = 0ull; }
    __syncthreads();
    // ---- radix select: digits [31:21], [20:10], [9:0]
    unsigned int prefix = 0u, pmask = 0u;
    const int shifts[3] = {21, 10, 0};
    const int nbins[3] = {2048, 2048, 1024};
    for (int lvl = 0; lvl < 3; lvl++) {
        for (int b = tid; b < 2048; b += THREADS) sm.hist[b] = 0;
        __syncthreads();
        if (SEL_done) break;
        const int nb = nbins[lvl];
        for (int j = tid; j < Mcur; j += THREADS) {
            const int sz = sm.sizes[j];
            const unsigned int key = sm.keys[j];
            if (sz > 0 && (key & pmask) == prefix) atomicAdd(&sm.hist[(key >> shifts[lvl]) & (nb - 1)], sz);
        }
        __syncthreads();
        // suffix sums over the bins, descending: thread i owns the BPT bins below nb - i * BPT
        constexpr int BPT = (2048 + THREADS - 1) / THREADS;
        int mine = 0;
#pragma unroll
        for (int k = 0; k < BPT; k++) { const int b = nb - 1 - (tid * BPT + k); mine += b >= 0 ? sm.hist[b] : 0; }
        int tot;
        const int before = block_scan_excl(mine, sm.sh, &tot);   // weight of all bins above this thread's first
        const int rem = SEL_rem;
        __syncthreads();
        if (tid == 0 && tot <= rem) SEL_done = 1;                 // everything under this prefix fits
        // the boundary bin is the first (from the top) whose inclusive suffix sum exceeds rem
        int acc = before;
#pragma unroll
        for (int k = 0; k < BPT; k++) {
            const int b = nb - 1 - (tid * BPT + k);
            const int h = b >= 0 ? sm.hist[b] : 0;
            if (b >= 0 && acc <= rem && acc + h > rem) { SEL_bin = b; SEL_rem = rem - acc; }
            acc += h;
        }
        __syncthreads();
        if (SEL_done) break;
        prefix |= (unsigned int)SEL_bin << shifts[lvl];
        pmask |= (unsigned int)(nb - 1) << shifts[lvl];
    }
    __syncthreads();
    // Selected: key above the boundary key; among clusters exactly at the boundary key, the lowest ids while
    // they still fit.  With `done` every key >= the current prefix range is in.
    const bool all_in = SEL_done != 0;
    const unsigned int kb = prefix;
    if (!all_in) {
        // a single cluster at the boundary key cannot fit (its bin overflowed the remaining budget);
        // only with several equal scores does the id-order walk matter
        int ne = 0;
        for (int j = tid; j < Mcur; j += THREADS) ne += (sm.sizes[j] > 0 && sm.keys[j] == kb) ? 1 : 0;
        if (ne) atomicAdd(&SEL_eqcnt, ne);
        __syncthreads();
        if (tid == 0 && SEL_eqcnt > 1) {
            int rem = SEL_rem, take = 0;
            for (int j = 0; j < Mcur; j++)
                if (sm.keys[j] == kb && sm.sizes[j] > 0) { if (sm.sizes[j] <= rem) { rem -= sm.sizes[j]; take++; } else break; }
            SEL_eqtake = take;
        }
    }
    __syncthreads();
    // When all_in, pmask covers the levels already fixed: keys matching the prefix there, or larger, are selected.
    const int eqtake = SEL_eqtake;
    int selc = 0, tokc = 0;
    for (int j = tid; j < Mcur; j += THREADS) {
        const int sz = sm.sizes[j];
        if (sz <= 0) continue;
        const unsigned int key = sm.keys[j];
        bool in = all_in ? ((key & pmask) >= prefix) : (key > kb);
        if (!in && !all_in && eqtake > 0 && key == kb) {
            // the first eqtake clusters (by id) with key == kb are selected too
            int rank = 0;
            for (int jj = 0; jj < j; jj++) rank += (sm.keys[jj] == kb && sm.sizes[jj] != 0) ? 1 : 0;
            in = rank < eqtake;
        }
        if (in) { selc++; tokc += sz; sm.sizes[j] = sz | (int)0x80000000; }
    }
    if (selc) { atomicAdd(&SEL_L, selc); atomicAdd(&SEL_tok, tokc); }
    if (best) atomicMax(&SEL_best, best);
    __syncthreads();
    int L = SEL_L;
    if (L == 0 && budget > 0 && SEL_best != 0ull) {
        // not even the best cluster fits: take it alone
        const int jb = (int)(0xffffffffu - (unsigned)(SEL_best & 0xffffffffull));
        __syncthreads();
        if (tid == 0) { SEL_tok = sm.sizes[jb]; sm.sizes[jb] |= (int)0x80000000; atomicOr(t.status, DYNAKV_ST_BUDGET_EXCEEDED); }
        L = 1;
    }
    __syncthreads();
    // ---- compaction in id order + work list: every thread owns a run of consecutive ids
    int* sel = t.sel_ids + (size_t)u * t.max_clusters;
    int2* work = t.work + ((size_t)buf * t.U + u) * t.W;
    const int per = (Mcur + THREADS - 1) / THREADS;
    const int j_lo = min(Mcur, tid * per), j_hi = min(Mcur, j_lo + per);
    int my_sel = 0, my_w = 0;
    for (int j = j_lo; j < j_hi; j++) {
        const int sz = sm.sizes[j];
        if (sz < 0) { my_sel++; my_w += ((sz & 0x7fffffff) + ENTRY_ROWS - 1) / ENTRY_ROWS; }
    }
    int ts, tw;
    int spos = block_scan_excl(my_sel, sm.sh, &ts);
    __syncthreads();
    int wpos = block_scan_excl(my_w, sm.sh, &tw);
    for (int j = j_lo; j < j_hi; j++) {
        const int szs = sm.sizes[j];
        if (szs >= 0) continue;
        const int sz = szs & 0x7fffffff;
        const int np = (sz + ENTRY_ROWS - 1) / ENTRY_ROWS;     // work entries: runs of <= ENTRY_ROWS rows inside one page
        sel[spos++] = j;
        int page = __ldcg(&t.cl_head[(size_t)u * t.max_clusters + j]);
        for (int i = 0; i < np && wpos + i < t.W; i++) {
            constexpr int EPP = PAGE / ENTRY_ROWS;       // entries per page
            work[wpos + i] = make_int2(page * PAGE + (i % EPP) * ENTRY_ROWS, min(ENTRY_ROWS, sz - ENTRY_ROWS * i));
            if (i % EPP == EPP - 1) page = __ldcg(&t.page_next[(size_t)u * t.P + page]);
        }
        wpos += np;
    }
    if (tid == 0) {
        t.sel_n[u] = L;
        t.sel_tokens[u] = SEL_tok;
        t.n_work[(size_t)buf * t.U + u] = min(tw, t.W);
        atomicAdd(&t.counters[CNT_TOKENS_ATTENDED], (unsigned long long)SEL_tok);
        atomicAdd(&t.counters[CNT_CLUSTERS_SELECTED], (unsigned long long)L);
    }
    if (user_ids) {
        // score order: rank = number of selected clusters that come first
        __syncthreads();
        int* uo = user_ids + (size_t)u * t.max_clusters;
        for (int a = tid; a < L; a += THREADS) {
            const int j = sel[a];
            const unsigned int kj = sm.keys[j];
            int rank = 0;
            for (int b = 0; b < L; b++) {
                const int jb = sel[b];
                const unsigned int kq = sm.keys[jb];
                rank += (kq > kj || (kq == kj && jb < j)) ? 1 : 0;
            }
            uo[rank] = j;
        }
        for (int p = L + tid; p < t.max_clusters; p += THREADS) uo[p] = -1;
    }
}

#undef SEL_bin
#undef SEL_rem
#undef SEL_done
#undef SEL_eqtake
#undef SEL_eqcnt
#undef SEL_L
#undef SEL_tok
#undef SEL_best

// Exclusive prefix of the units' work-list lengths, by one block (after every unit's n_work is visible).
template <int THREADS>
__device__ void work_prefix_block(const Tables& t, int* sh, int buf = 0) {
    const int tid = threadIdx.x;
    const int* n_work = t.n_work + (size_t)buf * t.U;
    const int per_t = (t.U + THREADS - 1) / THREADS;
    const int b0 = min(tid * per_t, t.U), b1 = min(b0 + per_t, t.U);
    int sum = 0;
    for (int i = b0; i < b1; i++) sum += __ldcg(&n_work[i]);
    int tot;
    int base = block_scan_excl(sum, sh, &tot);
    for (int i = b0; i < b1; i++) { t.work_prefix[i] = base; base += __ldcg(&n_work[i]); }
    if (tid == 0) t.work_prefix[t.U] = tot;
}

}  // namespace dkv
