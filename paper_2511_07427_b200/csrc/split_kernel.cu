// Split check: Algorithm 1's split decision and SplitCluster of arXiv 2511.07427
// (Section 4.2: a flagged cluster is re-clustered locally; Section 5.2: one child keeps
// growing where the parent was and the other is written elsewhere).  One block per unit walks the unit's clusters in ascending id; a triggered
// cluster is 2-means-partitioned, the staying child is compacted inside the pages it
// already owns, and the moving child is written to fresh pages under the next free id.
#include <float.h>

#include "append_block.cuh"
#include "common.cuh"
#include "fp8_rows.cuh"
#include "front_unit.cuh"
#include "split_small.cuh"

namespace dkv {

#ifndef DKV_SP_THREADS
#define DKV_SP_THREADS 512
#endif
constexpr int SP_THREADS = DKV_SP_THREADS;    // a multiple of 128 (one thread per (side, dimension) and per staged member)
#ifndef DKV_SP_MINBLOCKS
#define DKV_SP_MINBLOCKS 2          // blocks per SM the register budget is held to (a loop iteration wants all units resident)
#endif
constexpr int SP_HELPERS = 32;                 // extra blocks of a loop iteration's tail kernel that do the splits
constexpr int SP_CACHE_BYTES = 32 * 1024;      // member keys of the cluster being split are staged here when they fit
constexpr int SP_WARPS = SP_THREADS / 32;

// Dynamic shared memory, in order:
//   area 0: chain[maxch], newpg[maxch], trig[max_clusters] (ints), the split code's partial sums
//           wsum[SP_WARPS][2][HD] (floats); at least one ring stage long, because in a unit block of a loop
//           iteration it becomes stage 2 of the fused centroid pass once the trigger list has been handed over;
//   area 1: the staged member keys (SP_CACHE_BYTES; stage 0 of the pass) and their token ids;
//   area 2: the staged member values (SP_CACHE_BYTES; stage 1 of the pass);
//   one live flag per cluster id.
template <int HD, int KVB> struct SplitSmem {
    static constexpr int cache_rows = SP_CACHE_BYTES / (HD * KVB);
    static constexpr int stage_bytes = FrontUnit<SP_THREADS, HD>::STAGE_BYTES;
    static_assert(stage_bytes <= SP_CACHE_BYTES, "stages 0 and 1 of the centroid pass live in the staging areas");
    __host__ __device__ static size_t wsum_off(int maxch, int max_clusters) { return (((size_t)(2 * maxch + max_clusters) * sizeof(int)) + 15) & ~(size_t)15; }
    __host__ __device__ static size_t keys_off(int maxch, int max_clusters) {
        size_t a = wsum_off(maxch, max_clusters) + (size_t)SP_WARPS * 2 * HD * sizeof(float);
        if (a < (size_t)stage_bytes) a = stage_bytes;
        return (a + 127) & ~(size_t)127;
    }
    __host__ __device__ static size_t stage1_off(int maxch, int max_clusters) {
        return (keys_off(maxch, max_clusters) + SP_CACHE_BYTES + (size_t)cache_rows * sizeof(int) + 127) & ~(size_t)127;
    }
    __host__ __device__ static size_t live_off(int maxch, int max_clusters) { return stage1_off(maxch, max_clusters) + SP_CACHE_BYTES; }
    __host__ __device__ static size_t total(int maxch, int max_clusters) { return live_off(maxch, max_clusters) + (size_t)max_clusters + 16; }
};

// FP8 mode: the one-byte copy of a row (128 bytes and the two scale exponents) follows the row from slot src to slot
// dst of unit u's pages; called by a full warp.
__device__ __forceinline__ void fp8_move_row(const Tables& t, int u, size_t src, size_t dst, int lane) {
    const size_t gs = (size_t)u * t.P * PAGE + src, gd = (size_t)u * t.P * PAGE + dst;
    const int ps = row_pos<16>(gs, lane * 4), pd = row_pos<16>(gd, lane * 4);      // each slot's own chunk order
    *reinterpret_cast<unsigned*>(t.k8 + gd * t.d + pd) = *reinterpret_cast<const unsigned*>(t.k8 + gs * t.d + ps);
    *reinterpret_cast<unsigned*>(t.v8 + gd * t.d + pd) = *reinterpret_cast<const unsigned*>(t.v8 + gs * t.d + ps);
    if (lane == 0) { t.k8e[gd] = t.k8e[gs]; t.v8e[gd] = t.v8e[gs]; }
}

// ---- hand-over of triggered units from the unit blocks to the helper blocks of a loop iteration's tail kernel.
// tail_sync[0] = queue slots reserved, [1] = slots claimed by helpers, [2] = unit blocks that have decided.
// A unit block with triggered clusters reserves a slot (two words) and stores a hint, then unit + 1, in it; a
// helper claims slots in order.  The hint spares the helper two trips to memory in the common case of one
// triggered cluster whose size the unit block knows and that has fewer than 2^18 members: (cluster id + 1) | (size << 13), else 0.  Helpers never hold
// more than SP_HELPERS of the GPU's block slots, so the unit blocks they wait for always get to run; all the same
// every wait here is bounded.
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Called by one thread.  Returns the next unit to split, -1 when every unit block has decided and the queue is
// drained, -2 when a bounded wait ran out (the status word is raised).
__device__ int next_queued_unit(const Tables& t, int* hint) {
    unsigned long long t_begin = 0;
    for (int i = 0;; i++) {
        const int pushed = ld_acquire(t.tail_sync + 0);
        const int taken = ld_acquire(t.tail_sync + 1);
        if (taken < pushed) {
            if (atomicCAS(t.tail_sync + 1, taken, taken + 1) != taken) continue;
            for (int k = 0; k < (1 << 20); k++) {                 // the unit id lands right after its slot was reserved
                const int v = ld_acquire(t.tail_queue + 2 * taken + 1);
                if (v != 0) { *hint = t.tail_queue[2 * taken]; t.tail_queue[2 * taken + 1] = 0; return v - 1; }
            }
            atomicOr(t.status, DYNAKV_ST_INTERNAL);
            return -2;
        }
        if (ld_acquire(t.tail_sync + 2) >= t.U && ld_acquire(t.tail_sync + 0) == pushed) return -1;
        __nanosleep(200);
        if ((i & 31) == 31) {
            const unsigned long long now = global_ns();
            if (t_begin == 0) t_begin = now;
            else if (now - t_begin > 500000000ull) { atomicOr(t.status, DYNAKV_ST_INTERNAL); return -2; }
        }
    }
}

// Delayed-split mode (Algorithm 1, its last two blocks): the trigger scan of one unit, by all SP_THREADS threads of its
// block.  A cluster whose trigger fires or whose flag is owed is listed for a split now if the step's query retrieved it
// (sel[0..L), the selection's id list); a firing trigger outside that set raises the flag, and that entry is the first
// buffered one.  Then, if the buffered entries of the clusters left flagged reach buf_max, the one with the most of
// them (lowest id among equals) is listed as well, after the others.  Returns the number of listed clusters (the same
// in every thread).  Kept out of line: it runs in this mode only and must not weigh on the kernel's registers.
__device__ __noinline__ int delayed_scan(const int* cl_n, unsigned char* cl_flags, const float* cl_M2, int* cl_buf, const int* sel, int L,
                                         int M0, int min_size, int var_enabled, float tau, float gamma, int Mlive0, int N,
                                         int buf_max, int* trig, int* sh, float* red_f, int* red_i, int* red_k) {
    __shared__ unsigned int req_bits[128];     // the retrieved clusters of the step, one bit per id (ids are below 4096)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < 128; i += SP_THREADS) req_bits[i] = 0u;
    __syncthreads();
    for (int i = tid; i < L; i += SP_THREADS) { const int j = sel[i]; if (j >= 0 && j < 4096) atomicOr(&req_bits[j >> 5], 1u << (j & 31)); }
    __syncthreads();
    int base = 0, buf_sum = 0, buf_best = 0, buf_id = 0x7fffffff;
    for (int b0 = 0; b0 < M0; b0 += SP_THREADS) {
        const int j = b0 + tid;
        int hit = 0;
        if (j < M0) {
            const int c = cl_n[j];
            const int fl = cl_flags[j];
            if (c > 0 && c >= min_size && !(fl & FLAG_HOLD)) {
                const bool by_var = var_enabled && (cl_M2[j] / (float)c > tau);
                const bool by_size = gamma > 0.f && ((double)c * (double)Mlive0 > (double)gamma * (double)N);
                hit = (by_var || by_size) ? 1 : 0;
            }
            const bool owed_j = c > 0 && (fl & FLAG_SPLIT);
            const bool inreq = j < 4096 && ((req_bits[j >> 5] >> (j & 31)) & 1u);
            int bufj = owed_j ? cl_buf[j] : 0;
            if ((hit || owed_j) && inreq) hit = 1;
            else {
                if (hit && !owed_j) { cl_flags[j] = (unsigned char)(fl | FLAG_SPLIT); cl_buf[j] = 1; bufj = 1; }
                if (hit || owed_j) {
                    buf_sum += bufj;
                    if (bufj > buf_best || (bufj == buf_best && j < buf_id)) { buf_best = bufj; buf_id = j; }
                }
                hit = 0;
            }
        }
        int tot;
        const int pos = base + block_scan_excl(hit, sh, &tot);
        if (hit) trig[pos] = j;
        base += tot;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        buf_sum += __shfl_xor_sync(0xffffffffu, buf_sum, o);
        const int ob = __shfl_xor_sync(0xffffffffu, buf_best, o), oi = __shfl_xor_sync(0xffffffffu, buf_id, o);
        if (ob > buf_best || (ob == buf_best && oi < buf_id)) { buf_best = ob; buf_id = oi; }
    }
    __syncthreads();
    if (lane == 0) { red_f[warp] = __int_as_float(buf_sum); red_i[warp] = buf_best; red_k[warp] = buf_id; }
    __syncthreads();
    int tot = 0, bb = 0, bi = 0x7fffffff;
    for (int w = 0; w < SP_WARPS; w++) {
        tot += __float_as_int(red_f[w]);
        if (red_i[w] > bb || (red_i[w] == bb && red_k[w] < bi)) { bb = red_i[w]; bi = red_k[w]; }
    }
    if (bb > 0 && tot >= buf_max) { if (tid == 0) trig[base] = bi; base++; }
    __syncthreads();
    return base;
}

template <typename KV, int HD>
__global__ void __launch_bounds__(SP_THREADS, DKV_SP_MINBLOCKS) k_split_check(Tables t, float gamma, int var_enabled, int min_size, int iters,
                                                            int do_append, StepPtr app_k, StepPtr app_v, int* step_ctr,
                                                            int do_front, StepPtr next_q, StepPtr next_k, const int* step_lim) {
    constexpr int EPL = HD / 32;
    extern __shared__ __align__(128) int dyn[];
    __shared__ unsigned long long fr_bars[FR_STAGES];
    const int maxch = t.max_tokens / PAGE + 2;
    int* chain = dyn;                 // pages of the cluster being split, in chain order
    int* newpg = dyn + maxch;         // pages allocated for the moving child
    __shared__ __align__(16) float cA[HD], cB[HD];
    __shared__ float red_f[SP_WARPS];
    __shared__ int red_i[SP_WARPS], red_k[SP_WARPS];
    __shared__ int sh[33];
    __shared__ int s_cnt[4];          // changed, nA, nB, misc
    __shared__ int s_a, s_ok;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The next kernel on the stream may be scheduled as soon as every block of this grid has started: its blocks move
    // in as blocks of this grid retire, set themselves up and wait for this grid's completion before they read anything.
    pdl_trigger();
    // In a loop iteration (do_front) the grid is U unit blocks followed by SP_HELPERS helper blocks: a unit block
    // appends, finds its triggered clusters, hands them to the helpers and runs the unit's centroid pass of the
    // next step; the helpers split.  Otherwise block u does the whole job for unit u.
    const bool loop_mode = do_front != 0;
    const bool helper = loop_mode && (int)blockIdx.x >= t.U;
    int u = helper ? 0 : (int)blockIdx.x;
    // the step this iteration belongs to: read once, before the last block of the iteration can advance it
    const int t0 = step_ctr ? *step_ctr : 0;
    const bool fronted = loop_mode && (t0 + 1 < *step_lim);
    __shared__ int s_ntrig, s_nsplit, s_unit, s_flag, s_hint;
    int c_hint = 0;                  // helper: size of the single triggered cluster when the unit block passed it along
    __shared__ AppendResult s_app;
    // the same three arrays in shared memory for a cluster small enough to be staged
    __shared__ unsigned char label_s[SP_CACHE_BYTES / 128];
    __shared__ int rank_s[SP_CACHE_BYTES / 128], holes_s[SP_CACHE_BYTES / 128];

    // ---- triggered clusters, ascending id, evaluated on the state at entry.  A full scan is
    // needed only after a split changed M_live or created clusters (u_scan); otherwise only the
    // cluster that received the last append can have become triggered: for every other cluster
    // n_j and M2_j are unchanged while N only grew.
    int* trig = dyn + 2 * maxch;
    // staged copy of the member keys (and their token ids) when the cluster fits: every pass below then
    // reads shared memory instead of walking the pages again
    using Lay = SplitSmem<HD, (int)sizeof(KV)>;
    constexpr int CACHE_ROWS = Lay::cache_rows;
    unsigned char* dynb = reinterpret_cast<unsigned char*>(dyn);
    float* wsum = reinterpret_cast<float*>(dynb + Lay::wsum_off(maxch, t.max_clusters));   // [SP_WARPS][2][HD]
    auto WS = [&](int w, int side, int x) -> float& { return wsum[((size_t)w * 2 + side) * HD + x]; };
    KV* krows = reinterpret_cast<KV*>(dynb + Lay::keys_off(maxch, t.max_clusters));
    int* tok_s = reinterpret_cast<int*>(krows + (size_t)CACHE_ROWS * HD);
    if (tid == 0) { s_ntrig = 0; s_nsplit = 0; }
    int ntrig = 0;
    if (!helper) {
        // The unit's centroid pass for the NEXT step starts here, ahead of the append: its first copies are in
        // flight while the append runs, and the one row the append changes is recomputed at the end of the pass.
        unsigned char* const fr_stages[FR_STAGES] = {reinterpret_cast<unsigned char*>(krows), dynb + Lay::stage1_off(maxch, t.max_clusters), dynb};
        unsigned char* fr_live = dynb + Lay::live_off(maxch, t.max_clusters);
        FrontIssue<HD, SP_THREADS> fr_issue = {};
        if (fronted) {
            if (tid == 0) {
                for (int i = 0; i < FR_STAGES; i++) mbar_init(smem_u32(&fr_bars[i]), 1);
                asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
            }
            fr_issue = front_unit_begin<HD, SP_THREADS>(t, u, fr_stages, fr_bars, fr_live);
        }
        // what the trigger test needs and the append does not change: loaded ahead of the append's own chain of loads
        const int owed = t.u_last[u];            // an earlier append whose check is still owed (-1 in a loop's steady state)
        int full = t.u_scan[u];
        const bool delayed = t.update_mode == DYNAKV_MODE_DELAYED;
        if (delayed) full = 1;       // every cluster is looked at at every check (flags owed from earlier checks, the buffer limit)
        const int Mlive0 = t.u_Mlive[u];
        const float tau = t.u_tau[u];
        // fused loop iteration: the step's append for this unit comes first (Algorithm 1's order)
        if (do_append) append_block<KV, HD>(t, u, app_k, app_v, &s_app);
        __syncthreads();
        const int last = do_append ? s_app.cluster : owed;
        if (do_append && owed >= 0 && owed != last) full = 1;
        if (!full && do_append) {
            // Only the cluster that took the append can have become triggered (for every other cluster n_j and M2_j
            // are unchanged while N only grew), and the append has just computed its new statistics.
            if (tid == 0 && last >= 0) {
                const int c = s_app.n_new;
                // the append cleared the cluster's hold flag
                if (c >= min_size) {
                    bool hit;
                    if (t.update_mode == DYNAKV_MODE_LOCAL) hit = last >= t.M_floor && c > t.local_max;   // decode-born clusters, by absolute size
                    else if (t.update_mode == DYNAKV_MODE_STATIC) hit = false;
                    else {
                        const bool by_var = var_enabled && (s_app.M2_new / (float)c > tau);
                        const bool by_size = gamma > 0.f && ((double)c * (double)Mlive0 > (double)gamma * (double)s_app.N_new);
                        hit = by_var || by_size;
                    }
                    if (hit) { trig[0] = last; s_ntrig = 1; }
                }
            }
            __syncthreads();
        } else if (delayed) {
            const size_t c0 = (size_t)u * t.max_clusters;
            const int nt = delayed_scan(t.cl_n + c0, t.cl_flags + c0, t.cl_M2 + c0, t.cl_buf + c0, t.sel_ids + c0, t.sel_n[u], t.u_M[u],
                                        min_size, var_enabled, tau, gamma, Mlive0, t.u_N[u], t.buf_max, trig, sh, red_f, red_i, red_k);
            if (tid == 0) s_ntrig = nt;
            __syncthreads();
        } else {
        const int N = t.u_N[u], M0 = t.u_M[u];
        int base = 0;
        const int jlim = full ? M0 : (last >= 0 ? 1 : 0);
        for (int b0 = 0; b0 < jlim; b0 += SP_THREADS) {
            const int j = full ? b0 + tid : (tid == 0 ? last : -1);
            int hit = 0;
            if (j >= 0 && j < M0) {
                const size_t cj = (size_t)u * t.max_clusters + j;
                const int c = t.cl_n[cj];
                if (c > 0 && c >= min_size && !(t.cl_flags[cj] & FLAG_HOLD)) {
                    if (t.update_mode == DYNAKV_MODE_LOCAL) hit = (j >= t.M_floor && c > t.local_max) ? 1 : 0;
                    else if (t.update_mode == DYNAKV_MODE_STATIC) hit = 0;
                    else {
                        const bool by_var = var_enabled && (t.cl_M2[cj] / (float)c > tau);
                        const bool by_size = gamma > 0.f && ((double)c * (double)Mlive0 > (double)gamma * (double)N);
                        hit = (by_var || by_size) ? 1 : 0;
                    }
                }
            }
            int tot;
            const int pos = base + block_scan_excl(hit, sh, &tot);
            if (hit) trig[pos] = j;
            base += tot;
        }
        if (tid == 0) s_ntrig = base;
        __syncthreads();
        }
        ntrig = s_ntrig;
        if (loop_mode) {
            // ---- hand the triggered clusters to a helper block; this block goes on to the centroid pass
            if (tid == 0) { t.u_scan[u] = 0; t.u_last[u] = -1; }
            if (ntrig > 0) {
                int* tl = t.trig_list + (size_t)u * t.max_clusters;
                for (int i = tid; i < ntrig; i += SP_THREADS) tl[i] = trig[i];
                if (tid == 0) t.trig_n[u] = ntrig;
            }
            __threadfence();
            fence_proxy_async();          // area 0 (written above with ordinary stores) becomes a ring stage below
            __syncthreads();
            if (tid == 0) {
                if (ntrig > 0) {
                    const int slot = atomicAdd(t.tail_sync + 0, 1);
                    int hint = 0;
                    if (ntrig == 1 && !full && do_append && s_app.cluster == trig[0] && s_app.n_new < (1 << 18)) hint = (trig[0] + 1) | (s_app.n_new << 13);
                    t.tail_queue[2 * slot] = hint;
                    __threadfence();
                    atomicExch(t.tail_queue + 2 * slot + 1, u + 1);
                }
                __threadfence();
                atomicAdd(t.tail_sync + 2, 1);
            }
            // the rest of the unit's centroid pass for the NEXT step (its query scores and its new key's distances).
            // It needs nothing from the gather-attention kernel that may still be running and nothing from other
            // units; a helper that splits a cluster of this unit patches the two rows it changes once this pass
            // has finished (front_done).
            if (fronted) {
                const float* q1 = reinterpret_cast<const float*>(next_q.at(t0 + 1)) + (size_t)u * t.G * HD;
                const KV* k1 = reinterpret_cast<const KV*>(next_k.at(t0 + 1)) + (size_t)u * HD;
                front_unit<KV, HD, SP_THREADS>(t, u, q1, k1, fr_issue, fr_stages, fr_live, last);
                __threadfence();
                __syncthreads();
                if (tid == 0) atomicExch(t.front_done + u, t0 + 1);
            }
            ntrig = 0;            // nothing is split here
        }
    }
    // ---- splits: of the block's own unit, or (helper) of every unit taken from the queue
    for (;;) {
        if (helper) {
            if (tid == 0) { int h = 0; s_unit = next_queued_unit(t, &h); s_hint = h; }
            __syncthreads();
            u = s_unit;
            if (u < 0) break;
            __threadfence();                 // the unit block's writes (append, trigger list) precede its queue entry
            c_hint = 0;
            if (s_hint != 0) {
                ntrig = 1; c_hint = s_hint >> 13;
                if (tid == 0) { trig[0] = (s_hint & 8191) - 1; s_nsplit = 0; }
            } else {
                ntrig = t.trig_n[u];
                const int* tl = t.trig_list + (size_t)u * t.max_clusters;
                for (int i = tid; i < ntrig; i += SP_THREADS) trig[i] = tl[i];
                if (tid == 0) s_nsplit = 0;
            }
            __syncthreads();
        }
        // Everything before this reads and writes only what the gather-attention kernel ahead never touches (statistics,
        // the new row beyond every listed row, next step's scores); the splits move rows, so they wait for it.
        if (ntrig > 0) pdl_wait();
        KV* kpg = reinterpret_cast<KV*>(t.kpages) + (size_t)u * t.P * PAGE * HD;
        KV* vpg = reinterpret_cast<KV*>(t.vpages) + (size_t)u * t.P * PAGE * HD;
        int* ptok = t.page_tok + (size_t)u * t.P * PAGE;
        int* pnext = t.page_next + (size_t)u * t.P;
        unsigned char* label_g = t.sp_label + (size_t)u * t.max_tokens;
        int* rank_g = t.sp_pos + (size_t)u * 2 * t.max_tokens;      // per position
        int* holes_g = rank_g + t.max_tokens;                       // hole positions, in order
        bool front_seen = false;             // helper: the unit's centroid pass of the next step is known to be complete
        // Next step's scores and distances of the two children of a split, once the unit's own pass (which read the
        // rows as they were before, or half-way through, the split) can no longer overwrite them.  ra / rb: the
        // children's means (written before a block barrier).
        auto patch_children = [&](int ja, const float* ra, int jb, const float* rb) {
            if (!front_seen) {
                if (tid == 0) {
                    int ok = 0;
                    const unsigned long long t_begin = global_ns();
                    for (int i = 0; i < (1 << 24); i++) {
                        if (ld_acquire(t.front_done + u) == t0 + 1) { ok = 1; break; }
                        __nanosleep(200);
                        if ((i & 31) == 31 && global_ns() - t_begin > 500000000ull) break;
                    }
                    if (!ok) atomicOr(t.status, DYNAKV_ST_INTERNAL);
                    s_flag = ok;
                }
                __syncthreads();
                front_seen = true;
            }
            if (s_flag && warp == 0) {
                const float* q1 = reinterpret_cast<const float*>(next_q.at(t0 + 1)) + (size_t)u * t.G * HD;
                const KV* k1 = reinterpret_cast<const KV*>(next_k.at(t0 + 1)) + (size_t)u * HD;
                front_patch<KV, HD>(t, u, q1, k1, ja, ra, jb, rb);
            }
        };
        SplitScratch sc;
        sc.cA = cA; sc.cB = cB; sc.label = label_s; sc.rank = rank_s; sc.holes = holes_s; sc.tok = tok_s; sc.newpg = newpg;
        sc.part = wsum; sc.nsplit = &s_nsplit;
        KV* vrows = reinterpret_cast<KV*>(dynb + Lay::stage1_off(maxch, t.max_clusters));
        for (int li = 0; li < ntrig; li++) {
            const int j = trig[li];
            const size_t cj = (size_t)u * t.max_clusters + j;
            const int c = c_hint > 0 ? c_hint : t.cl_n[cj];
            __syncthreads();    // previous cluster's work is complete
            if (c <= CACHE_ROWS) {
                // the common case: everything out of shared memory
                int stay_side = 0;
                const int nid = split_small<KV, HD, SP_THREADS, CACHE_ROWS>(t, u, j, c, iters, krows, vrows, sc, &stay_side);
                if (nid >= 0 && helper && fronted) patch_children(j, stay_side ? cB : cA, nid, stay_side ? cA : cB);
                continue;
            }
            if (t.u_M[u] >= t.max_clusters) { if (tid == 0) atomicOr(t.status, DYNAKV_ST_MAX_CLUSTERS); continue; }

            const int npg = (c + PAGE - 1) / PAGE;
            if (tid == 0) {
                int p = t.cl_head[cj];
#ifdef DYNAKV_CHECKED
                s_ok = 1;
#endif
                for (int i = 0; i < npg; i++) {
                    if (!DKV_IN(t, SITE_SPLIT_PAGE, p, 0, t.P)) { s_ok = 0; break; }
                    chain[i] = p; p = pnext[p];
                }
            }
            for (int e = tid; e < HD; e += SP_THREADS) cA[e] = t.cl_r[cj * HD + e];
            __syncthreads();
#ifdef DYNAKV_CHECKED
            if (!s_ok) continue;          // a page of the chain was out of range: the cluster is left as it is
#endif
            // general path (the cluster does not fit the staging area): every pass walks the pages.  The labels, ranks
            // and hole list of a cluster of up to GEN_ROWS members live in the two staging areas, which this path does
            // not use otherwise (every member's label is read and written once per 2-means round); beyond that in
            // global memory.
            constexpr int GEN_ROWS = 6144;
            static_assert(8192 + 2 * GEN_ROWS * 4 <= 2 * SP_CACHE_BYTES, "labels, ranks and holes fit the two staging areas");
            unsigned char* area = reinterpret_cast<unsigned char*>(krows);
            const bool on_chip = c <= GEN_ROWS;
            unsigned char* label = on_chip ? area : label_g;
            int* rank_of = on_chip ? reinterpret_cast<int*>(area + 8192) : rank_g;
            int* holes = on_chip ? reinterpret_cast<int*>(area + 8192) + GEN_ROWS : holes_g;
            // key row and token id of member position p
            // (keys are read through load_key: from the row's page, or decoded from its bytes in FP8 storage)
            const size_t gbase = (size_t)u * t.P * PAGE;          // the unit's first slot in the whole pool
            auto gslot_of = [&](int p) -> size_t { return gbase + (size_t)chain[p >> 5] * PAGE + (p & 31); };
            auto tok_of = [&](int p) -> int { return ptok[(size_t)chain[p >> 5] * PAGE + (p & 31)]; };

            // ---- centre A: member farthest from r_j; centre B: member farthest from A (ties: lowest token id)
            for (int round = 0; round < 2; round++) {
                float cen[EPL];
#pragma unroll
                for (int e = 0; e < EPL; e++) cen[e] = cA[lane * EPL + e];
                float bd = -1.f; int bt = 0x7fffffff, bp = -1;
                for (int p = warp; p < c; p += SP_WARPS) {
                    float kx[EPL];
                    load_key<KV, HD, EPL>(t, gslot_of(p), lane * EPL, kx);
                    float part = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; e++) { float df = kx[e] - cen[e]; part = fmaf(df, df, part); }
                    part = warp_sum(part);
                    int tok = tok_of(p);
                    if (part > bd || (part == bd && tok < bt)) { bd = part; bt = tok; bp = p; }
                }
                if (lane == 0) { red_f[warp] = bd; red_i[warp] = bt; red_k[warp] = bp; }
                __syncthreads();
                if (tid == 0) {
                    float d0 = red_f[0]; int t0 = red_i[0], p0 = red_k[0];
                    for (int w = 1; w < SP_WARPS; w++)
                        if (red_f[w] > d0 || (red_f[w] == d0 && red_i[w] < t0)) { d0 = red_f[w]; t0 = red_i[w]; p0 = red_k[w]; }
                    s_a = p0;
                }
                __syncthreads();
                {
                    float* dst = (round == 0) ? cA : cB;
                    __syncthreads();
                    for (int e = tid; e < HD; e += SP_THREADS) { float x1[1]; load_key<KV, HD, 1>(t, gslot_of(s_a), e, x1); dst[e] = x1[0]; }
                    __syncthreads();
                }
            }
            // After round 0, cA = key A and the second round measured distances to cA: correct.

            // ---- 2-means rounds
            for (int p = tid; p < c; p += SP_THREADS) label[p] = 255;
            __syncthreads();
            int nA = 0, nB = 0;
            bool abandoned = false;
            for (int it = 0; it < iters; it++) {
                if (tid < 4) s_cnt[tid] = 0;
                __syncthreads();
                float a_c[EPL], b_c[EPL], sa[EPL], sb[EPL];
#pragma unroll
                for (int e = 0; e < EPL; e++) { a_c[e] = cA[lane * EPL + e]; b_c[e] = cB[lane * EPL + e]; sa[e] = 0.f; sb[e] = 0.f; }
                int chg = 0, ca = 0, cb = 0;
                // two rows of the warp at a time, their loads issued together (the rows live in global memory)
                for (int p0 = warp; p0 < c; p0 += 2 * SP_WARPS) {
                    const int p1 = p0 + SP_WARPS;
                    float k0[EPL], k1[EPL];
                    {
                        load_key<KV, HD, EPL>(t, gslot_of(p0), lane * EPL, k0);
                        load_key<KV, HD, EPL>(t, gslot_of(p1 < c ? p1 : p0), lane * EPL, k1);
                    }
#pragma unroll
                    for (int b2 = 0; b2 < 2; b2++) {
                        const int p = b2 ? p1 : p0;
                        if (p >= c) break;
                        float da = 0.f, db = 0.f;
#pragma unroll
                        for (int e = 0; e < EPL; e++) {
                            const float kv = b2 ? k1[e] : k0[e];
                            float x = kv - a_c[e], y = kv - b_c[e];
                            da = fmaf(x, x, da); db = fmaf(y, y, db);
                        }
                        da = warp_sum(da); db = warp_sum(db);
                        const int l = db < da ? 1 : 0;
                        if (lane == 0) { if (label[p] != l) chg = 1; label[p] = (unsigned char)l; if (l) cb++; else ca++; }
#pragma unroll
                        for (int e = 0; e < EPL; e++) { const float kv = b2 ? k1[e] : k0[e]; if (l) sb[e] += kv; else sa[e] += kv; }
                    }
                }
#pragma unroll
                for (int e = 0; e < EPL; e++) { WS(warp, 0, lane * EPL + e) = sa[e]; WS(warp, 1, lane * EPL + e) = sb[e]; }
                if (lane == 0) { if (chg) atomicOr(&s_cnt[0], 1); atomicAdd(&s_cnt[1], ca); atomicAdd(&s_cnt[2], cb); }
                __syncthreads();
                nA = s_cnt[1]; nB = s_cnt[2];
                const int changed = s_cnt[0];
                if (nA == 0 || nB == 0) { abandoned = true; break; }
                if (!changed) break;
                for (int e = tid; e < 2 * HD; e += SP_THREADS) {
                    int side = e / HD, x = e % HD;
                    float s = 0.f;
                    for (int w = 0; w < SP_WARPS; w++) s += WS(w, side, x);
                    if (side == 0) cA[x] = s / (float)nA; else cB[x] = s / (float)nB;
                }
                __syncthreads();
            }
            if (abandoned) { if (tid == 0) { t.cl_flags[cj] = FLAG_HOLD; t.cl_buf[cj] = 0; } continue; }

            // ---- which side stays: the one holding the smallest token id
            {
                int bt = 0x7fffffff, bl = 0;
                for (int p = tid; p < c; p += SP_THREADS) {
                    int tok = tok_of(p);
                    if (tok < bt) { bt = tok; bl = label[p]; }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    int ot = __shfl_xor_sync(0xffffffffu, bt, o), ol = __shfl_xor_sync(0xffffffffu, bl, o);
                    if (ot < bt) { bt = ot; bl = ol; }
                }
                if (lane == 0) { red_i[warp] = bt; red_k[warp] = bl; }
                __syncthreads();
                if (tid == 0) {
                    int t0 = red_i[0], l0 = red_k[0];
                    for (int w = 1; w < SP_WARPS; w++) if (red_i[w] < t0) { t0 = red_i[w]; l0 = red_k[w]; }
                    s_a = l0;
                }
                __syncthreads();
            }
            const int stay = s_a;
            const int s_n = stay ? nB : nA, m_n = c - s_n;
            const int need = (m_n + PAGE - 1) / PAGE, keep = (s_n + PAGE - 1) / PAGE;

            // ---- pages for the moving child
            if (tid == 0) {
                int fc = t.u_free_cnt[u], top = t.u_page_top[u];
                int ok = (fc + (t.P - top) >= need) ? 1 : 0;
                if (ok) {
                    for (int i = 0; i < need; i++) {
                        int pg;
                        if (fc > 0) pg = t.free_stack[(size_t)u * t.P + --fc]; else pg = top++;
                        newpg[i] = pg;
                        if (!DKV_IN(t, SITE_SPLIT_PAGE, pg, 0, t.P)) ok = 0;
                    }
                    t.u_free_cnt[u] = fc; t.u_page_top[u] = top;
                } else atomicOr(t.status, DYNAKV_ST_PAGE_POOL);
                s_ok = ok;
            }
            __syncthreads();
            if (!s_ok) continue;
            const int new_id = t.u_M[u];

            // ---- ranks: movers in position order; fillers (stayers at positions >= s_n); holes (movers at positions < s_n)
            int base_m = 0, base_f = 0, base_h = 0;
            for (int b0 = 0; b0 < c; b0 += SP_THREADS) {
                const int p = b0 + tid;
                const int mv = (p < c && label[p] != stay) ? 1 : 0;
                const int fl = (p < c && !mv && p >= s_n) ? 1 : 0;
                const int hl = (p < c && mv && p < s_n) ? 1 : 0;
                int tm, tf, th;
                const int rm = base_m + block_scan_excl(mv, sh, &tm);
                const int rf = base_f + block_scan_excl(fl, sh, &tf);
                const int rh = base_h + block_scan_excl(hl, sh, &th);
                if (p < c) rank_of[p] = mv ? rm : (fl ? rf : -1);
                if (hl) holes[rh] = p;
                base_m += tm; base_f += tf; base_h += th;
            }
            __syncthreads();

            // ---- phase 1: movers go to the new pages (one warp per row)
            for (int p = warp; p < c; p += SP_WARPS) {
                if (label[p] == stay) continue;
                const int r = rank_of[p];
                const size_t src = (size_t)chain[p >> 5] * PAGE + (p & 31);
                const size_t dst = (size_t)newpg[r >> 5] * PAGE + (r & 31);
                const int ps = row_pos<Epc<KV>::v>(src, lane * EPL), pd = row_pos<Epc<KV>::v>(dst, lane * EPL);
#pragma unroll
                for (int e = 0; e < EPL; e++) {
                    if (!t.fp8) { kpg[dst * HD + pd + e] = kpg[src * HD + ps + e]; vpg[dst * HD + pd + e] = vpg[src * HD + ps + e]; }
                }
                if (t.fp8) fp8_move_row(t, u, src, dst, lane);
                if (lane == 0) {
                    int tok = ptok[src];
                    ptok[dst] = tok;
                    if (DKV_IN(t, SITE_SPLIT_TOKEN, tok, 0, t.max_tokens)) t.tok_cluster[(size_t)u * t.max_tokens + tok] = new_id;
                }
            }
            __syncthreads();
            // ---- phase 2: stayers beyond position s_n fill the holes
            for (int p = s_n + warp; p < c; p += SP_WARPS) {
                if (label[p] != stay) continue;
                const int h = holes[rank_of[p]];
                const size_t src = (size_t)chain[p >> 5] * PAGE + (p & 31);
                const size_t dst = (size_t)chain[h >> 5] * PAGE + (h & 31);
                const int ps = row_pos<Epc<KV>::v>(src, lane * EPL), pd = row_pos<Epc<KV>::v>(dst, lane * EPL);
#pragma unroll
                for (int e = 0; e < EPL; e++) {
                    if (!t.fp8) { kpg[dst * HD + pd + e] = kpg[src * HD + ps + e]; vpg[dst * HD + pd + e] = vpg[src * HD + ps + e]; }
                }
                if (t.fp8) fp8_move_row(t, u, src, dst, lane);
                if (lane == 0) ptok[dst] = ptok[src];
            }
            __syncthreads();
            // ---- phase 3: chains, ids, allocator
            const size_t cn = (size_t)u * t.max_clusters + new_id;
            if (tid == 0) {
                pnext[chain[keep - 1]] = -1;
                t.cl_tail[cj] = chain[keep - 1];
                int fc = t.u_free_cnt[u];
                for (int i = keep; i < npg; i++) t.free_stack[(size_t)u * t.P + fc++] = chain[i];
                t.u_free_cnt[u] = fc;
                for (int i = 0; i < need; i++) pnext[newpg[i]] = (i + 1 < need) ? newpg[i + 1] : -1;
                t.cl_head[cn] = newpg[0]; t.cl_tail[cn] = newpg[need - 1];
                t.cl_n[cj] = s_n; t.cl_n[cn] = m_n;
                t.cl_flags[cj] = 0; t.cl_flags[cn] = 0; t.cl_buf[cj] = 0; t.cl_buf[cn] = 0;
                if (t.cl_ver) t.cl_ver[cj] = t.cl_ver[cj] + 1;      // two-tier mode: copies of the cluster made before now are void
                t.u_M[u] = new_id + 1; t.u_Mlive[u] = t.u_Mlive[u] + 1;
                atomicAdd(&t.counters[CNT_SPLITS], 1ull);
                s_nsplit = s_nsplit + 1;
            }
            __syncthreads();
            // ---- phase 4: exact statistics of both children (mean, then M2 about the mean)
            for (int child = 0; child < 2; child++) {
                const int cc = child == 0 ? s_n : m_n;
                const int* pages = child == 0 ? chain : newpg;
                const size_t cid = child == 0 ? cj : cn;
                float sa[EPL];
#pragma unroll
                for (int e = 0; e < EPL; e++) sa[e] = 0.f;
                // the child's rows in their new place
                for (int p = warp; p < cc; p += SP_WARPS) {
                    const size_t kslot = (size_t)pages[p >> 5] * PAGE + (p & 31);
                    float kx[EPL];
                    load_key<KV, HD, EPL>(t, (size_t)u * t.P * PAGE + kslot, lane * EPL, kx);
#pragma unroll
                    for (int e = 0; e < EPL; e++) sa[e] += kx[e];
                }
#pragma unroll
                for (int e = 0; e < EPL; e++) WS(warp, 0, lane * EPL + e) = sa[e];
                __syncthreads();
                for (int e = tid; e < HD; e += SP_THREADS) {
                    float s = 0.f;
                    for (int w = 0; w < SP_WARPS; w++) s += WS(w, 0, e);
                    s /= (float)cc;
                    cA[e] = s;
                    t.cl_r[cid * HD + e] = s;
                }
                __syncthreads();
                float mean[EPL], m2 = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; e++) mean[e] = cA[lane * EPL + e];
                for (int p = warp; p < cc; p += SP_WARPS) {
                    const size_t kslot = (size_t)pages[p >> 5] * PAGE + (p & 31);
                    float kx[EPL];
                    load_key<KV, HD, EPL>(t, (size_t)u * t.P * PAGE + kslot, lane * EPL, kx);
                    float part = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; e++) { float df = kx[e] - mean[e]; part = fmaf(df, df, part); }
                    m2 += warp_sum(part);
                }
                if (lane == 0) red_f[warp] = m2;
                __syncthreads();
                if (tid == 0) {
                    float s = 0.f;
                    for (int w = 0; w < SP_WARPS; w++) s += red_f[w];
                    t.cl_M2[cid] = s;
                }
                __syncthreads();
            }
            if (helper && fronted) patch_children(j, t.cl_r + cj * HD, new_id, t.cl_r + ((size_t)u * t.max_clusters + new_id) * HD);
        }
        if (!helper) break;
        __syncthreads();
        if (tid == 0 && s_nsplit > 0) t.u_scan[u] = 1;
    }
    __syncthreads();
    // No block leaves before the kernel ahead has completed: the next kernel on the stream (the next iteration's
    // centroid pass and selection, which rewrite the work lists) is ordered behind THIS kernel only.
    pdl_wait();
    if (tid == 0) {
        if (!loop_mode) { t.u_scan[u] = s_nsplit > 0 ? 1 : 0; t.u_last[u] = -1; }
        if (step_ctr) {
            // the last block of the iteration advances the device-side step index that every kernel of the loop reads,
            // and clears the hand-over words for the next iteration
            __threadfence();
            if (atomicAdd(t.plan_counter + 1, 1) == (int)gridDim.x - 1) {
                t.plan_counter[1] = 0; t.tail_sync[0] = 0; t.tail_sync[1] = 0; t.tail_sync[2] = 0;
                *step_ctr += 1;
            }
        }
    }
}

template <typename KV, int HD>
static void split_t(const Tables& t, float gamma, int var_enabled, int min_size, int iters, int do_append, StepPtr k, StepPtr v,
                    int* step_ctr, const NextFront& nf, cudaStream_t s) {
    const size_t dyn = SplitSmem<HD, (int)sizeof(KV)>::total(t.max_tokens / PAGE + 2, t.max_clusters);
    // the opt-in to more than 48 KB of dynamic shared memory: once per size, device and kernel instance
    static size_t opted[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dyn > 32 * 1024 && (dev < 0 || dev >= 64 || opted[dev] != dyn)) {
        cudaFuncSetAttribute(k_split_check<KV, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
        if (dev >= 0 && dev < 64) opted[dev] = dyn;
    }
    launch_pdl(k_split_check<KV, HD>, dim3(t.U + (nf.on ? SP_HELPERS : 0)), dim3(SP_THREADS), dyn, s, t, gamma, var_enabled, min_size, iters, do_append, k, v, step_ctr,
               nf.on, nf.q, nf.k, nf.step_lim);
}

void launch_split_check(const Tables& t, float gamma, int var_enabled, int min_size, int iters, cudaStream_t s,
                        long long* launches) {
    launch_append_split(t, gamma, var_enabled, min_size, iters, 0, StepPtr{nullptr, 0, nullptr}, StepPtr{nullptr, 0, nullptr}, nullptr,
                        NextFront{0, StepPtr{nullptr, 0, nullptr}, StepPtr{nullptr, 0, nullptr}, nullptr}, s, launches);
}

// The tail of a fused loop iteration in one launch: append (when do_append), the next step's centroid pass (when
// nf.on and the next step exists), split check, and, when step_ctr is given, the increment of the device-side
// step index by the last block to finish.
void launch_append_split(const Tables& t, float gamma, int var_enabled, int min_size, int iters, int do_append, StepPtr k,
                         StepPtr v, int* step_ctr, const NextFront& nf, cudaStream_t s, long long* launches) {
    if (t.kv_dtype == DYNAKV_F32) {
        if (t.d == 64) split_t<float, 64>(t, gamma, var_enabled, min_size, iters, do_append, k, v, step_ctr, nf, s);
        else split_t<float, 128>(t, gamma, var_enabled, min_size, iters, do_append, k, v, step_ctr, nf, s);
    } else {
        if (t.d == 64) split_t<__nv_bfloat16, 64>(t, gamma, var_enabled, min_size, iters, do_append, k, v, step_ctr, nf, s);
        else split_t<__nv_bfloat16, 128>(t, gamma, var_enabled, min_size, iters, do_append, k, v, step_ctr, nf, s);
    }
    (*launches)++;
}

}  // namespace dkv
