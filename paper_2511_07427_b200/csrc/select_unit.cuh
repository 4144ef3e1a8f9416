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
    int* cand;                         // [SL_MAXCAND] undecided cluster ids of the short way, then their order
    float* wred;                       // [64] per-warp score minima and maxima
    unsigned long long* wtot;          // [32] per-warp totals of the packed (selected, work entries) scan
};
constexpr int SL_MAXCAND = 64;         // clusters the short way resolves by ranking them against each other
#define SEL_bin sm.sc[0]
#define SEL_rem sm.sc[1]
#define SEL_done sm.sc[2]
#define SEL_eqtake sm.sc[3]
#define SEL_eqcnt sm.sc[4]
#define SEL_L sm.sc[5]
#define SEL_tok sm.sc[6]
#define SEL_best (*sm.best64)
__host__ __device__ constexpr size_t select_smem_bytes(int ids) {
    return (size_t)ids * 8 + 2048 * 4 + 48 * 4 + 8 + 16 + 2 * 64 * 4 + 64 * 4 + 32 * 8 + 16;
}
__device__ __forceinline__ SelectSmem select_smem_at(unsigned char* base, int ids) {      // base: 8-byte aligned
    SelectSmem sm;
    sm.best64 = reinterpret_cast<unsigned long long*>(base);
    sm.keys = reinterpret_cast<unsigned int*>(base + 8);
    sm.sizes = reinterpret_cast<int*>(sm.keys + ids);
    sm.hist = sm.sizes + ids;
    sm.sh = sm.hist + 2048;
    sm.sc = sm.sh + 36;
    sm.cand = sm.sc + 12;
    sm.wred = reinterpret_cast<float*>(sm.cand + 2 * SL_MAXCAND);
    // 8-byte aligned: base + 8 + ids * 8 + 2048 * 4 + (36 + 12 + 128 + 64) * 4
    sm.wtot = reinterpret_cast<unsigned long long*>(sm.wred + 64);
    return sm;
}

__device__ __forceinline__ unsigned int ord_key(float f) {
    unsigned int b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
// the score an orderable key was made from
__device__ __forceinline__ float ord_key_score(unsigned int k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Called by every thread of the block.  scores: the unit's scores in global memory (written before a barrier or
// by an earlier kernel).  user_ids (may be null): the selection in score order, -1 padded, [max_clusters].
// On return (all global writes issued; no trailing barrier) thread 0 has written sel_n / sel_tokens / n_work.
// This is the general version (three histogram levels over the key's bits); select_unit() below tries a shorter way
// first and comes here when its one histogram level leaves too many clusters undecided.
template <int THREADS>
__device__ void select_unit_radix(const Tables& t, int u, int budget, int* __restrict__ user_ids, const SelectSmem& sm) {
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
    int2* work = t.work + (size_t)u * t.W;
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
            if (i % EPP == EPP - 1) {
                if (!DKV_IN(t, SITE_SELECT_PAGE, page, 0, t.P)) break;
                page = __ldcg(&t.page_next[(size_t)u * t.P + page]);
            }
        }
        wpos += np;
    }
    if (tid == 0) {
        t.sel_n[u] = L;
        t.sel_tokens[u] = SEL_tok;
        t.n_work[u] = min(tw, t.W);
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

// Exclusive prefix sum over the block of one 32-bit value per thread with ONE block barrier: a shuffle scan inside
// every warp, the warp totals through `wtot` (32 entries, not reused before the caller's next barrier), and a second
// shuffle scan of those totals by every warp for itself.  *total gets the block sum.
template <int THREADS>
__device__ __forceinline__ unsigned int block_scan_excl_1sync(unsigned int v, unsigned int* wtot, unsigned int* total) {
    constexpr int NW = THREADS / 32;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const unsigned int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
    if (lane == 31) wtot[w] = x;
    __syncthreads();
    unsigned int ws = lane < NW ? wtot[lane] : 0u;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const unsigned int y = __shfl_up_sync(0xffffffffu, ws, o); if (lane >= o) ws += y; }
    *total = __shfl_sync(0xffffffffu, ws, 31);
    const unsigned int before = __shfl_sync(0xffffffffu, ws, (w + 31) & 31);      // inclusive total of warp w - 1
    return (w > 0 ? before : 0u) + x - v;
}

// The selection itself.  Short way: ONE histogram of cluster sizes over 2048 bins that are linear in the score
// between the unit's smallest and largest live score (bin index monotone in the score); a suffix scan from the top
// finds the bin in which the budget runs out; clusters in higher bins are selected, clusters in lower bins are not,
// and the few clusters inside that bin are ranked against each other by (score descending, id ascending) and
// taken while they fit.  If that bin holds more than SL_MAXCAND clusters the general version above decides instead.
// Then the selection is written in id order, with the work list of the selected clusters' rows.
// Nothing here waits for the unit's current id count: ids not yet handed out have size 0, like dead clusters, so
// every load of the per-cluster tables is issued at once over the unit's whole id capacity.
// MAXPER: most consecutive ids a thread owns; the caller picks THREADS * MAXPER >= max_clusters.
template <int THREADS, int MAXPER>
__device__ void select_unit(const Tables& t, int u, int budget, int* __restrict__ user_ids, const SelectSmem& sm) {
    static_assert(2048 % THREADS == 0 && THREADS % 32 == 0 && THREADS <= 1024, "bins are dealt out evenly to the threads");
    constexpr int BPT = 2048 / THREADS;           // histogram bins per thread
    constexpr int NW = THREADS / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // ids to look at: the whole id capacity, so that no load waits for the unit's id count -- unless the capacity is
    // far above what the build handed out (a unit that may grow a lot): then the count is fetched first
    const int Mlim = (t.max_clusters > 2 * t.M_floor + 64) ? min(t.max_clusters, __ldcg(&t.u_M[u])) : t.max_clusters;
    const float* SC = t.scores + (size_t)u * t.max_clusters;
    const int* CN = t.cl_n + (size_t)u * t.max_clusters;
    const int* HEAD = t.cl_head + (size_t)u * t.max_clusters;
    const int* NEXT = t.page_next + (size_t)u * t.P;
    unsigned int* wtot = reinterpret_cast<unsigned int*>(sm.wtot);
    // ---- every thread owns a run of consecutive ids; all its loads are issued together (through L2: other blocks of a
    // running kernel may have written these)
    const int per = (Mlim + THREADS - 1) / THREADS;
    const int j_lo = min(Mlim, tid * per), j_hi = min(Mlim, j_lo + per);
    int szr[MAXPER], head[MAXPER];
    float scr[MAXPER];
#pragma unroll
    for (int i = 0; i < MAXPER; i++) {
        const bool in = j_lo + i < j_hi;
        szr[i] = in ? __ldcg(CN + j_lo + i) : 0;
        scr[i] = in ? __ldcg(SC + j_lo + i) : 0.f;
        head[i] = in ? __ldcg(HEAD + j_lo + i) : -1;
    }
    for (int b = tid; b < 2048; b += THREADS) sm.hist[b] = 0;
    if (tid == 0) { SEL_rem = 0; SEL_done = 1; SEL_bin = -1; SEL_eqcnt = 0; SEL_L = 0; SEL_tok = 0; SEL_eqtake = 0; }
    float smin = INFINITY, smax = -INFINITY;
    int nxt[MAXPER];                              // second page of a cluster of more than one page, fetched ahead
#pragma unroll
    for (int i = 0; i < MAXPER; i++) {
        const int sz = szr[i];
        nxt[i] = (sz > PAGE && head[i] >= 0) ? __ldcg(NEXT + head[i]) : -1;
        if (j_lo + i < j_hi) { sm.keys[j_lo + i] = sz > 0 ? ord_key(scr[i]) : 0u; sm.sizes[j_lo + i] = sz; }
        if (sz > 0) { smin = fminf(smin, scr[i]); smax = fmaxf(smax, scr[i]); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        smin = fminf(smin, __shfl_xor_sync(0xffffffffu, smin, o));
        smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, o));
    }
    if (lane == 0) { sm.wred[warp] = smin; sm.wred[32 + warp] = smax; }
    __syncthreads();                                                        // (1) keys, sizes, zeroed bins, warp extrema
    smin = lane < NW ? sm.wred[lane] : INFINITY; smax = lane < NW ? sm.wred[32 + lane] : -INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        smin = fminf(smin, __shfl_xor_sync(0xffffffffu, smin, o));
        smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, o));
    }
    // bin of a score: monotone non-decreasing in the score (a subtraction of, and a multiplication by, block constants)
    const float bscale = (smax > smin) ? 2047.f / (smax - smin) : 0.f;
    auto bin_of = [&](float sc) -> int { return min(2047, max(0, (int)((sc - smin) * bscale))); };
    int bin[MAXPER];
#pragma unroll
    for (int i = 0; i < MAXPER; i++) {
        bin[i] = bin_of(scr[i]);
        if (szr[i] > 0) atomicAdd(&sm.hist[bin[i]], szr[i]);
    }
    __syncthreads();                                                        // (2) histogram complete
    // ---- suffix sums from the top bin down: thread i owns bins 2047 - i * BPT - k
    int hb[BPT];
    int mine = 0;
#pragma unroll
    for (int k = 0; k < BPT; k++) { hb[k] = sm.hist[2047 - (tid * BPT + k)]; mine += hb[k]; }
    unsigned int tot_all;
    const int above = (int)block_scan_excl_1sync<THREADS>((unsigned int)mine, wtot, &tot_all);        // (3) inside
    {
        int acc = above;
#pragma unroll
        for (int k = 0; k < BPT; k++) {
            // the bin in which the budget runs out: everything above it fits, with it it does not
            if (acc <= budget && acc + hb[k] > budget) { SEL_bin = 2047 - (tid * BPT + k); SEL_rem = budget - acc; SEL_done = 0; SEL_tok = acc; }
            acc += hb[k];
        }
    }
    __syncthreads();                                                        // (4) boundary bin known
    const int bstar = SEL_bin;                  // -1: every live cluster fits
    int selc = 0;
#pragma unroll
    for (int i = 0; i < MAXPER; i++) {
        if (szr[i] <= 0) continue;
        if (bin[i] > bstar) { sm.sizes[j_lo + i] = szr[i] | (int)0x80000000; selc++; }
        else if (bin[i] == bstar) { const int c = atomicAdd(&SEL_eqcnt, 1); if (c < SL_MAXCAND) sm.cand[c] = j_lo + i; }
    }
    if (selc) atomicAdd(&SEL_L, selc);
    __syncthreads();                                                        // (5) undecided clusters listed
    const int ncand = SEL_eqcnt;
    if (ncand > SL_MAXCAND) {
        // too many clusters share the boundary bin (scores bunched against one far outlier): the general way
        __syncthreads();
        select_unit_radix<THREADS>(t, u, budget, user_ids, sm);
        return;
    }
    if (warp == 0 && ncand > 0) {
        // rank the undecided clusters by (score descending, id ascending); lane 0 takes them in that order while
        // they fit.  With nothing selected above and a first cluster larger than the budget, it is taken alone.
        for (int c = lane; c < ncand; c += 32) {
            const int j = sm.cand[c];
            const unsigned int kj = sm.keys[j];
            int rank = 0;
            for (int b = 0; b < ncand; b++) {
                const int jb = sm.cand[b];
                const unsigned int kb = sm.keys[jb];
                rank += (kb > kj || (kb == kj && jb < j)) ? 1 : 0;
            }
            sm.cand[SL_MAXCAND + rank] = j;
        }
        __syncwarp();
        if (lane == 0) {
            int rem = SEL_rem, took = 0, tok = 0;
            for (int r = 0; r < ncand; r++) {
                const int j = sm.cand[SL_MAXCAND + r];
                const int sz = sm.sizes[j];
                if (sz > rem) break;
                rem -= sz; tok += sz; took++;
                sm.sizes[j] = sz | (int)0x80000000;
            }
            if (took == 0 && SEL_L == 0 && budget > 0) {
                const int j = sm.cand[SL_MAXCAND];
                tok = sm.sizes[j]; took = 1;
                sm.sizes[j] |= (int)0x80000000;
                atomicOr(t.status, DYNAKV_ST_BUDGET_EXCEEDED);
            }
            SEL_L += took; SEL_tok += tok;
        }
    } else if (tid == 0 && bstar < 0) {
        SEL_tok = (int)tot_all;
    }
    __syncthreads();                                                        // (6) selection marks final
    const int L = SEL_L;
    // ---- compaction in id order + work list
    int* sel = t.sel_ids + (size_t)u * t.max_clusters;
    int2* work = t.work + (size_t)u * t.W;
    unsigned int my = 0;                          // work entries << 13 | selected clusters (at most 4096 ids, W < 2^19)
    bool on[MAXPER];
#pragma unroll
    for (int i = 0; i < MAXPER; i++) {
        on[i] = (j_lo + i < j_hi) && sm.sizes[j_lo + i] < 0;
        if (on[i]) my += 1u + ((unsigned int)((szr[i] + ENTRY_ROWS - 1) / ENTRY_ROWS) << 13);
    }
    unsigned int tot2;
    const unsigned int pos2 = block_scan_excl_1sync<THREADS>(my, wtot, &tot2);                          // (7) inside
    int spos = (int)(pos2 & 8191u), wpos = (int)(pos2 >> 13);
    const int tw = (int)(tot2 >> 13);
#pragma unroll
    for (int i = 0; i < MAXPER; i++) {
        if (!on[i]) continue;
        const int sz = szr[i];
        const int np = (sz + ENTRY_ROWS - 1) / ENTRY_ROWS;     // work entries: runs of <= ENTRY_ROWS rows inside one page
        sel[spos++] = j_lo + i;
        int page = head[i];
        for (int e = 0; e < np && wpos + e < t.W; e++) {
            constexpr int EPP = PAGE / ENTRY_ROWS;       // entries per page
            work[wpos + e] = make_int2(page * PAGE + (e % EPP) * ENTRY_ROWS, min(ENTRY_ROWS, sz - ENTRY_ROWS * e));
            if (e % EPP == EPP - 1 && e + 1 < np) {
                if (!DKV_IN(t, SITE_SELECT_PAGE, page, 0, t.P)) break;
                page = (e / EPP == 0) ? nxt[i] : __ldcg(NEXT + page);
            }
        }
        wpos += np;
    }
    if (tid == 0) {
        t.sel_n[u] = L;
        t.sel_tokens[u] = SEL_tok;
        t.n_work[u] = min(tw, t.W);
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
__device__ void work_prefix_block(const Tables& t, int* sh) {
    const int tid = threadIdx.x;
    const int* n_work = t.n_work;
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
