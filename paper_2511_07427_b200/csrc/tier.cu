// A second memory tier under the page pool (arXiv 2511.07427, Section 6: fast memory as a cache of clusters over the
// slow one, with a cluster-aligned replacement policy; Section 7, the note on CPU-GPU platforms).  Here the page pool
// lives in pinned, mapped HOST memory; HBM holds a cache of page frames per unit, filled and replaced in whole
// clusters, and the attention kernels read frames only.  Everything that writes rows (build, append, splits) keeps
// writing the pool, through the same pointers as without the tier.
//
// After the selection of a step, k_tier_resolve (one block per unit) looks at every selected cluster:
//   hit      its copy was made of the cluster as it is now (same split version, same first page, same size);
//   grown    same version and first page, but entries were appended since: only the page that was the last one then
//            (if it had room left) and the pages linked after it are copied;
//   missing  no copy, or a copy from before a split of the cluster (dropped): every page is copied.
// Frames for the copies come from the unit's free stack; when it runs short, whole clusters that this step does not
// use are evicted until it suffices (cluster-aligned: never part of a cluster).  The order of eviction follows the
// two principles of Section 6.2: copies made useless by a split go first; then clusters unchanged since they were
// copied, the ones with more pages first (small clusters are the ones worth keeping), the longest unused first among
// equals; clusters that took appends since they were copied go last (recently updated clusters are retained).
// k_tier_fetch then copies the listed pages from host memory into their frames, and the step's gather list has
// been rewritten from pool rows to frame rows.
#include "common.cuh"

namespace dkv {

__global__ void k_tier_init(Tables t, TierState ts) {
    const size_t U = t.U, Mx = t.max_clusters, P = t.P, Fc = ts.Fc;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = i0; i < U * Mx; i += stride) { ts.cl_fr_head[i] = -1; ts.cl_fr_tail[i] = -1; ts.cl_lru[i] = 0u; t.cl_ver[i] = 0; }
    for (size_t i = i0; i < U * P; i += stride) ts.page_frame[i] = -1;
    for (size_t i = i0; i < U * Fc; i += stride) { ts.frame_page[i] = -1; ts.frame_next[i] = -1; ts.fr_free[i] = (int)(Fc - 1 - i % Fc); }
    for (size_t i = i0; i < U; i += stride) { ts.fr_free_cnt[i] = (int)Fc; ts.n_jobs[i] = 0; ts.clock[i] = 0u; }
    for (size_t i = i0; i < TIER_COUNTERS; i += stride) ts.counters[i] = 0ull;
}

constexpr int TIER_GROWN = 1 << 30;       // mark in the miss list: the cluster's copy only lacks appended entries

__global__ void __launch_bounds__(256) k_tier_resolve(Tables t, TierState ts) {
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Mx = t.max_clusters, P = t.P, Fc = ts.Fc;
    const int L = t.sel_n[u];
    const int* sel = t.sel_ids + (size_t)u * Mx;
    const int* cl_n = t.cl_n + (size_t)u * Mx;
    const int* cl_head = t.cl_head + (size_t)u * Mx;
    const int* cl_tail = t.cl_tail + (size_t)u * Mx;
    const int* cl_ver = t.cl_ver + (size_t)u * Mx;
    const int* pnext = t.page_next + (size_t)u * P;
    int* fr_head = ts.cl_fr_head + (size_t)u * Mx;
    int* fr_tail = ts.cl_fr_tail + (size_t)u * Mx;
    int* snap = ts.cl_snap + (size_t)u * Mx * 4;
    unsigned int* lru = ts.cl_lru + (size_t)u * Mx;
    int* page_frame = ts.page_frame + (size_t)u * P;
    int* frame_page = ts.frame_page + (size_t)u * Fc;
    int* frame_next = ts.frame_next + (size_t)u * Fc;
    int* fr_free = ts.fr_free + (size_t)u * Fc;
    int* miss = ts.miss_list + (size_t)u * Mx;
    int2* jobs = ts.jobs + (size_t)u * (Fc + Mx);
    __shared__ int s_nmiss, s_free, s_need, s_fail, s_njobs, s_victim, s_cnt[TIER_COUNTERS];
    __shared__ unsigned long long s_best[8];
    const unsigned int clock = ts.clock[u] + 1u;
    if (tid == 0) { s_nmiss = 0; s_free = ts.fr_free_cnt[u]; s_need = 0; s_fail = 0; s_njobs = 0; }
    if (tid < TIER_COUNTERS) s_cnt[tid] = 0;
    __syncthreads();
    auto pages_of = [](int n) { return (n + PAGE - 1) / PAGE; };
    // ---- every selected cluster: hit, grown or missing
    for (int i = tid; i < L; i += 256) {
        const int j = sel[i];
        const int n = cl_n[j];
        const bool same = fr_head[j] >= 0 && snap[4 * j + 1] == cl_ver[j] && snap[4 * j + 2] == cl_head[j];
        if (same && n == snap[4 * j]) { lru[j] = clock; atomicAdd(&s_cnt[TIER_HITS], 1); }
        else if (same && n > snap[4 * j]) {
            lru[j] = clock;
            atomicAdd(&s_need, pages_of(n) - pages_of(snap[4 * j]));
            miss[atomicAdd(&s_nmiss, 1)] = j | TIER_GROWN;
        } else {
            atomicAdd(&s_need, pages_of(n));
            miss[atomicAdd(&s_nmiss, 1)] = j;
        }
    }
    __syncthreads();
    const int nmiss = s_nmiss;
    // gives the frames of cluster j's copy back (one lane; pushes only, so several warps may do it at once)
    auto drop = [&](int j) {
        int f = fr_head[j];
        for (int guard = 0; f >= 0 && guard < Fc; guard++) {
            const int nx = frame_next[f];
            const int home = frame_page[f];
            if (home >= 0 && home < P && page_frame[home] == f) page_frame[home] = -1;   // unless the page has a newer copy
            frame_page[f] = -1; frame_next[f] = -1;
            const int at = atomicAdd(&s_free, 1);
            if (at >= 0 && at < Fc) fr_free[at] = f; else atomicOr(t.status, DYNAKV_ST_INTERNAL);      // cannot happen: more frames freed than exist
            f = nx;
        }
        fr_head[j] = -1; fr_tail[j] = -1;
    };
    // ---- copies of selected clusters from before a split
    for (int m = warp; m < nmiss; m += 8) {
        const int e = miss[m];
        if (lane == 0 && !(e & TIER_GROWN) && fr_head[e] >= 0) { drop(e); atomicAdd(&s_cnt[TIER_STALE], 1); }
    }
    __syncthreads();
    // ---- cluster-aligned replacement.  A cluster's eviction key does not change while victims are taken (only the
    // victim's own copy goes), so every thread keeps the smallest key of the ids it owns (tid, tid + 256, ...) in a
    // register; an eviction is then one block-wide minimum, the return of the victim's frames by thread 0, and a
    // rescan by the one thread that owned the victim.
    auto key_of = [&](int j) -> unsigned long long {
        if (fr_head[j] < 0 || lru[j] == clock) return ~0ull;           // no copy, or in use by this step
        const int sn = snap[4 * j];
        const unsigned long long cls = (snap[4 * j + 1] != cl_ver[j] || snap[4 * j + 2] != cl_head[j]) ? 0ull : (cl_n[j] == sn ? 1ull : 2ull);
        return (cls << 60) | ((unsigned long long)(0xFFFFF - pages_of(sn)) << 40) |
               ((unsigned long long)(lru[j] & 0xFFFFFFFu) << 12) | (unsigned long long)j;
    };
    unsigned long long mine = ~0ull;
    // Whether another victim is needed is read by every thread at the same point -- right behind a barrier, before
    // anything may change the free count again -- and kept in a register: a thread that is late (the one that rescans)
    // must not find the count already lowered by the hand-out of frames below and go round once more on its own.
    bool more = s_free < s_need;
    if (more) {
        for (int j = tid; j < Mx; j += 256) { const unsigned long long k = key_of(j); if (k < mine) mine = k; }
    }
    while (more) {
        unsigned long long best = mine;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const unsigned long long y = __shfl_xor_sync(0xffffffffu, best, o); if (y < best) best = y; }
        if (lane == 0) s_best[warp] = best;
        __syncthreads();
        if (tid == 0) {
            unsigned long long b = s_best[0];
            for (int w = 1; w < 8; w++) if (s_best[w] < b) b = s_best[w];
            if (b == ~0ull) s_fail = 1;                 // nothing left to evict: the cache cannot hold this step's clusters
            else {
                const int v = (int)(b & 0xFFFull);
                s_victim = v;
                s_cnt[(b >> 60) == 0ull ? TIER_STALE : TIER_EVICTED] += 1;
                drop(v);
            }
        }
        __syncthreads();
        more = s_free < s_need && !s_fail;
        if (more && (s_victim & 255) == tid) {          // the victim was one of this thread's ids
            mine = ~0ull;
            for (int j = tid; j < Mx; j += 256) { const unsigned long long k = key_of(j); if (k < mine) mine = k; }
        }
    }
    __syncthreads();          // nobody hands out frames before every thread has left the loop
    if (!s_fail) {
        // ---- frames and copy jobs (pops only from here on)
        for (int m = warp; m < nmiss; m += 8) {
            if (lane != 0) continue;
            const int e = miss[m], j = e & ~TIER_GROWN;
            const int n = cl_n[j];
            // a job copies rows [row0, row0 + rows) of a page into the same rows of a frame: only rows that hold entries,
            // and of a grown cluster's former last page only the ones added since
            auto job = [&](int pg, int f, int row0, int rows) {
                jobs[atomicAdd(&s_njobs, 1)] = make_int2(pg, f | (row0 << 20) | ((rows - 1) << 25));
                atomicAdd(&s_cnt[TIER_PAGES_FETCHED], 1);
                atomicAdd(&s_cnt[TIER_ROWS], rows);
            };
            int page, prev, todo, pk;          // pk: number of the next page inside the cluster
            if (e & TIER_GROWN) {
                const int sn = snap[4 * j], old_tail = snap[4 * j + 3];
                pk = pages_of(sn);
                if (sn % PAGE != 0 && old_tail >= 0 && old_tail < P) job(old_tail, page_frame[old_tail], sn % PAGE, min(n, pk * PAGE) - sn);
                page = (old_tail >= 0 && old_tail < P) ? pnext[old_tail] : -1; prev = fr_tail[j]; todo = pages_of(n) - pk;
                atomicAdd(&s_cnt[TIER_REFRESHED], 1);
            } else {
                page = cl_head[j]; prev = -1; todo = pages_of(n); pk = 0;
                atomicAdd(&s_cnt[TIER_FETCHED], 1);
            }
            for (int k = 0; k < todo && page >= 0 && page < P; k++) {
                const int at = atomicSub(&s_free, 1) - 1;
                if (at < 0 || at >= Fc) { atomicAdd(&s_free, 1); atomicOr(t.status, DYNAKV_ST_INTERNAL); break; }   // cannot happen: the need was counted
                const int f = fr_free[at];
                if (f < 0 || f >= Fc) { atomicOr(t.status, DYNAKV_ST_INTERNAL); break; }
                frame_next[f] = -1;
                if (prev < 0) fr_head[j] = f; else frame_next[prev] = f;
                prev = f;
                frame_page[f] = page;
                page_frame[page] = f;
                job(page, f, 0, min(PAGE, n - (pk + k) * PAGE));
                page = pnext[page];
            }
            fr_tail[j] = prev;
            snap[4 * j] = n; snap[4 * j + 1] = cl_ver[j]; snap[4 * j + 2] = cl_head[j]; snap[4 * j + 3] = cl_tail[j];
            lru[j] = clock;
        }
    }
    __syncthreads();
    if (tid == 0) {
        ts.clock[u] = clock;
        ts.fr_free_cnt[u] = s_free;
        ts.n_jobs[u] = s_fail ? 0 : s_njobs;
        if (s_fail) atomicOr(t.status, DYNAKV_ST_TIER_CACHE);
    }
    if (tid < TIER_COUNTERS && s_cnt[tid]) atomicAdd(&ts.counters[tid], (unsigned long long)s_cnt[tid]);
    // ---- the gather list, from pool rows to frame rows (a unit whose clusters did not fit reads frame 0: in bounds,
    // meaningless, and the status word says so)
    const int nw = t.n_work[u];
    int2* work = t.work + (size_t)u * t.W;
    const bool fail = s_fail != 0;
    for (int e = tid; e < nw; e += 256) {
        int2 ent = work[e];
        const int pg = ent.x / PAGE;
        const int f = (fail || pg < 0 || pg >= P) ? 0 : page_frame[pg];
        ent.x = (f >= 0 && f < Fc ? f : 0) * PAGE + ent.x % PAGE;
        work[e] = ent;
    }
}

// Copies the listed rows, K and V, from the pool (host memory) into the same rows of their frames; in FP8 mode the
// one-byte rows and the page's 32 scale exponents.
__global__ void __launch_bounds__(256) k_tier_fetch(Tables t, TierState ts, int row_bytes) {
    const int u = blockIdx.y;
    const int nj = ts.n_jobs[u];
    const size_t page_bytes = (size_t)PAGE * row_bytes;
    const char* kpool = t.fp8 ? (const char*)t.k8 : (const char*)t.kpages;
    const char* vpool = t.fp8 ? (const char*)t.v8 : (const char*)t.vpages;
    for (int jb = blockIdx.x; jb < nj; jb += gridDim.x) {
        const int2 job = ts.jobs[(size_t)u * (ts.Fc + t.max_clusters) + jb];
        const int f = job.y & 0xFFFFF, row0 = (job.y >> 20) & 31, rows = ((job.y >> 25) & 31) + 1;
        if (job.x < 0 || job.x >= t.P || f >= ts.Fc || row0 + rows > PAGE) continue;
        const size_t src = (size_t)u * t.P + job.x, dst = (size_t)u * ts.Fc + f;
        const size_t off = (size_t)row0 * row_bytes;
        const int v16 = rows * row_bytes / 16;
        const uint4* ks = reinterpret_cast<const uint4*>(kpool + src * page_bytes + off);
        const uint4* vs = reinterpret_cast<const uint4*>(vpool + src * page_bytes + off);
        uint4* kd = reinterpret_cast<uint4*>((char*)ts.kcache + dst * page_bytes + off);
        uint4* vd = reinterpret_cast<uint4*>((char*)ts.vcache + dst * page_bytes + off);
        for (int i = threadIdx.x; i < v16; i += 256) { kd[i] = ks[i]; vd[i] = vs[i]; }
        if (t.fp8 && threadIdx.x < 2 * (PAGE / 16)) {
            const int i = threadIdx.x % (PAGE / 16);
            if (threadIdx.x < PAGE / 16) reinterpret_cast<uint4*>(ts.kecache + dst * PAGE)[i] = reinterpret_cast<const uint4*>(t.k8e + src * PAGE)[i];
            else reinterpret_cast<uint4*>(ts.vecache + dst * PAGE)[i] = reinterpret_cast<const uint4*>(t.v8e + src * PAGE)[i];
        }
    }
}

void launch_tier_init(const Tables& t, const TierState& ts, cudaStream_t s, long long* launches) {
    k_tier_init<<<256, 256, 0, s>>>(t, ts);
    (*launches)++;
}

void launch_tier_resolve_fetch(const Tables& t, const TierState& ts, cudaStream_t s, long long* launches) {
    // Ordinary launches on purpose.  The kernels of a step are otherwise chained by programmatic dependent launch, and
    // the attention kernel lets its successor -- the kernel that appends -- move in as soon as it has started itself.
    // If these two did the same, the append of the step could run beside k_tier_resolve, which reads the very sizes and
    // page chains the append changes.  As full launches they finish before the attention kernel can start.
    k_tier_resolve<<<t.U, 256, 0, s>>>(t, ts);
    const int row_bytes = t.fp8 ? t.d : t.d * (t.kv_dtype == DYNAKV_F32 ? 4 : 2);
    k_tier_fetch<<<dim3(16, t.U), 256, 0, s>>>(t, ts, row_bytes);
    (*launches) += 2;
}

}  // namespace dkv
