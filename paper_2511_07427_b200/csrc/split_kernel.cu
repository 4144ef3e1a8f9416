// Split check: Algorithm 1's split decision and SplitCluster of arXiv 2511.07427
// (Section 4.2 "a local clustering algorithm is executed", Section 5.2 "one of the
// resulting sub-clusters continues to grow from the original head, the other is
// migrated").  One block per unit walks the unit's clusters in ascending id; a triggered
// cluster is 2-means-partitioned, the staying child is compacted inside the pages it
// already owns, and the moving child is written to fresh pages under the next free id.
#include <float.h>

#include "append_block.cuh"
#include "common.cuh"
#include "front_unit.cuh"

namespace dkv {

constexpr int SP_THREADS = 512;
constexpr int SP_CACHE_BYTES = 32 * 1024;      // member keys of the cluster being split are staged here when they fit
constexpr int SP_WARPS = SP_THREADS / 32;

// Dynamic shared memory, in order: chain[maxch], newpg[maxch], trig[max_clusters] (ints); the staged member
// keys (SP_CACHE_BYTES, 16-byte aligned; also stage 0 of the fused centroid pass) and their token ids; stage 1
// of the fused centroid pass; one live flag per cluster id.
template <int HD, int KVB> struct SplitSmem {
    static constexpr int cache_rows = SP_CACHE_BYTES / (HD * KVB);
    static constexpr int stage_bytes = FrontUnit<SP_THREADS, HD>::STAGE_BYTES;
    static_assert(stage_bytes <= SP_CACHE_BYTES, "stage 0 of the centroid pass lives in the staging area");
    __host__ __device__ static size_t keys_off(int maxch, int max_clusters) { return (((size_t)(2 * maxch + max_clusters) * sizeof(int)) + 127) & ~(size_t)127; }
    __host__ __device__ static size_t stage1_off(int maxch, int max_clusters) {
        return (keys_off(maxch, max_clusters) + SP_CACHE_BYTES + (size_t)cache_rows * sizeof(int) + 127) & ~(size_t)127;
    }
    __host__ __device__ static size_t live_off(int maxch, int max_clusters) { return stage1_off(maxch, max_clusters) + stage_bytes; }
    __host__ __device__ static size_t total(int maxch, int max_clusters) { return live_off(maxch, max_clusters) + (size_t)max_clusters + 16; }
};

template <typename KV, int HD>
__global__ void __launch_bounds__(SP_THREADS) k_split_check(Tables t, float gamma, int var_enabled, int min_size, int iters,
                                                            int do_append, StepPtr app_k, StepPtr app_v, int* step_ctr,
                                                            int do_front, StepPtr next_q, StepPtr next_k, const int* step_lim) {
    constexpr int EPL = HD / 32;
    extern __shared__ __align__(128) int dyn[];
    __shared__ unsigned long long fr_bars[2];
    const int maxch = t.max_tokens / PAGE + 2;
    int* chain = dyn;                 // pages of the cluster being split, in chain order
    int* newpg = dyn + maxch;         // pages allocated for the moving child
    __shared__ float cA[HD], cB[HD];
    __shared__ float wsum[SP_WARPS][2][HD];
    __shared__ float red_f[SP_WARPS];
    __shared__ int red_i[SP_WARPS], red_k[SP_WARPS];
    __shared__ int sh[33];
    __shared__ int s_cnt[4];          // changed, nA, nB, misc
    __shared__ int s_a, s_ok;

    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // the step this iteration belongs to: read once, before the last block of the iteration can advance it
    const int t0 = step_ctr ? *step_ctr : 0;
    if (do_front && tid == 0) {
        mbar_init(smem_u32(&fr_bars[0]), 1); mbar_init(smem_u32(&fr_bars[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    // fused loop iteration: the step's append for this unit comes first (Algorithm 1's order)
    if (do_append) { append_block<KV, HD>(t, u, app_k, app_v); __syncthreads(); }
    const int N = t.u_N[u], M0 = t.u_M[u], Mlive0 = t.u_Mlive[u];
    const float tau = t.u_tau[u];
    KV* kpg = reinterpret_cast<KV*>(t.kpages) + (size_t)u * t.P * PAGE * HD;
    KV* vpg = reinterpret_cast<KV*>(t.vpages) + (size_t)u * t.P * PAGE * HD;
    int* ptok = t.page_tok + (size_t)u * t.P * PAGE;
    int* pnext = t.page_next + (size_t)u * t.P;
    unsigned char* label_g = t.sp_label + (size_t)u * t.max_tokens;
    int* rank_g = t.sp_pos + (size_t)u * 2 * t.max_tokens;      // per position
    int* holes_g = rank_g + t.max_tokens;                       // hole positions, in order
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
    KV* krows = reinterpret_cast<KV*>(dynb + Lay::keys_off(maxch, t.max_clusters));
    int* tok_s = reinterpret_cast<int*>(krows + (size_t)CACHE_ROWS * HD);
    __shared__ int s_ntrig, s_nsplit;
    if (tid == 0) { s_ntrig = 0; s_nsplit = 0; }
    __syncthreads();
    {
        const int full = t.u_scan[u];
        const int last = t.u_last[u];
        int base = 0;
        const int jlim = full ? M0 : (last >= 0 ? 1 : 0);
        for (int b0 = 0; b0 < jlim; b0 += SP_THREADS) {
            const int j = full ? b0 + tid : (tid == 0 ? last : -1);
            int hit = 0;
            if (j >= 0 && j < M0) {
                const size_t cj = (size_t)u * t.max_clusters + j;
                const int c = t.cl_n[cj];
                if (c > 0 && c >= min_size && !(t.cl_flags[cj] & FLAG_HOLD)) {
                    const bool by_var = var_enabled && (t.cl_M2[cj] / (float)c > tau);
                    const bool by_size = gamma > 0.f && ((double)c * (double)Mlive0 > (double)gamma * (double)N);
                    hit = (by_var || by_size) ? 1 : 0;
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
    const int ntrig = s_ntrig;
    // ---- fused loop iteration: the unit's centroid pass for the NEXT step (its query scores and its new key's
    // distances) on the state after this step's append.  It needs nothing from the gather-attention kernel that
    // may still be running, and nothing from other units; a split below patches the two rows it changes.
    const bool fronted = do_front && (t0 + 1 < *step_lim);
    const float* q1 = nullptr; const KV* k1 = nullptr;
    if (fronted) {
        q1 = reinterpret_cast<const float*>(next_q.at(t0 + 1)) + (size_t)u * t.G * HD;
        k1 = reinterpret_cast<const KV*>(next_k.at(t0 + 1)) + (size_t)u * HD;
        front_unit<KV, HD, SP_THREADS>(t, u, q1, k1, reinterpret_cast<unsigned char*>(krows), dynb + Lay::stage1_off(maxch, t.max_clusters),
                                       fr_bars, dynb + Lay::live_off(maxch, t.max_clusters));
    }
    // Everything above reads and writes only what the gather-attention kernel before this one never touches
    // (statistics, the new row beyond every listed row, next step's scores); the splits below move rows, so
    // they wait for it.
    if (ntrig > 0) pdl_wait();
    for (int li = 0; li < ntrig; li++) {
        const int j = trig[li];
        const size_t cj = (size_t)u * t.max_clusters + j;
        const int c = t.cl_n[cj];
        if (t.u_M[u] >= t.max_clusters) { if (tid == 0) atomicOr(t.status, DYNAKV_ST_MAX_CLUSTERS); continue; }

        __syncthreads();    // previous cluster's work is complete
        const int npg = (c + PAGE - 1) / PAGE;
        if (tid == 0) {
            int p = t.cl_head[cj];
            for (int i = 0; i < npg; i++) { chain[i] = p; p = pnext[p]; }
        }
        for (int e = tid; e < HD; e += SP_THREADS) cA[e] = t.cl_r[cj * HD + e];
        __syncthreads();
        const bool cached = c <= CACHE_ROWS;
        if (cached) {
            constexpr int V16 = HD * (int)sizeof(KV) / 16;      // 16-byte pieces per row
            for (int idx = tid; idx < c * V16; idx += SP_THREADS) {
                const int p = idx / V16, v = idx % V16;
                const size_t row = (size_t)chain[p >> 5] * PAGE + (p & 31);
                reinterpret_cast<uint4*>(krows + (size_t)p * HD)[v] = reinterpret_cast<const uint4*>(kpg + row * HD)[v];
            }
            for (int p = tid; p < c; p += SP_THREADS) tok_s[p] = ptok[(size_t)chain[p >> 5] * PAGE + (p & 31)];
            __syncthreads();
        }
        unsigned char* label = cached ? label_s : label_g;
        int* rank_of = cached ? rank_s : rank_g;
        int* holes = cached ? holes_s : holes_g;
        // key row and token id of member position p
        auto key_of = [&](int p) -> const KV* {
            return cached ? krows + (size_t)p * HD : kpg + ((size_t)chain[p >> 5] * PAGE + (p & 31)) * HD;
        };
        auto tok_of = [&](int p) -> int { return cached ? tok_s[p] : ptok[(size_t)chain[p >> 5] * PAGE + (p & 31)]; };

        // ---- centre A: member farthest from r_j; centre B: member farthest from A (ties: lowest token id)
        for (int round = 0; round < 2; round++) {
            float cen[EPL];
#pragma unroll
            for (int e = 0; e < EPL; e++) cen[e] = cA[lane * EPL + e];
            float bd = -1.f; int bt = 0x7fffffff, bp = -1;
            for (int p = warp; p < c; p += SP_WARPS) {
                const KV* k = key_of(p) + lane * EPL;
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; e++) { float df = to_f(k[e]) - cen[e]; part = fmaf(df, df, part); }
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
                const KV* src = key_of(s_a);
                float* dst = (round == 0) ? cA : cB;
                __syncthreads();
                for (int e = tid; e < HD; e += SP_THREADS) dst[e] = to_f(src[e]);
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
            for (int p = warp; p < c; p += SP_WARPS) {
                const KV* k = key_of(p) + lane * EPL;
                float kk[EPL], da = 0.f, db = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; e++) {
                    kk[e] = to_f(k[e]);
                    float x = kk[e] - a_c[e], y = kk[e] - b_c[e];
                    da = fmaf(x, x, da); db = fmaf(y, y, db);
                }
                da = warp_sum(da); db = warp_sum(db);
                const int l = db < da ? 1 : 0;
                if (lane == 0) { if (label[p] != l) chg = 1; label[p] = (unsigned char)l; if (l) cb++; else ca++; }
#pragma unroll
                for (int e = 0; e < EPL; e++) { if (l) sb[e] += kk[e]; else sa[e] += kk[e]; }
            }
#pragma unroll
            for (int e = 0; e < EPL; e++) { wsum[warp][0][lane * EPL + e] = sa[e]; wsum[warp][1][lane * EPL + e] = sb[e]; }
            if (lane == 0) { if (chg) atomicOr(&s_cnt[0], 1); atomicAdd(&s_cnt[1], ca); atomicAdd(&s_cnt[2], cb); }
            __syncthreads();
            nA = s_cnt[1]; nB = s_cnt[2];
            const int changed = s_cnt[0];
            if (nA == 0 || nB == 0) { abandoned = true; break; }
            if (!changed) break;
            for (int e = tid; e < 2 * HD; e += SP_THREADS) {
                int side = e / HD, x = e % HD;
                float s = 0.f;
                for (int w = 0; w < SP_WARPS; w++) s += wsum[w][side][x];
                if (side == 0) cA[x] = s / (float)nA; else cB[x] = s / (float)nB;
            }
            __syncthreads();
        }
        if (abandoned) { if (tid == 0) t.cl_flags[cj] |= FLAG_HOLD; continue; }

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
#pragma unroll
            for (int e = 0; e < EPL; e++) {
                kpg[dst * HD + lane * EPL + e] = kpg[src * HD + lane * EPL + e];
                vpg[dst * HD + lane * EPL + e] = vpg[src * HD + lane * EPL + e];
            }
            if (lane == 0) {
                int tok = ptok[src];
                ptok[dst] = tok;
                t.tok_cluster[(size_t)u * t.max_tokens + tok] = new_id;
            }
        }
        __syncthreads();
        // ---- phase 2: stayers beyond position s_n fill the holes
        for (int p = s_n + warp; p < c; p += SP_WARPS) {
            if (label[p] != stay) continue;
            const int h = holes[rank_of[p]];
            const size_t src = (size_t)chain[p >> 5] * PAGE + (p & 31);
            const size_t dst = (size_t)chain[h >> 5] * PAGE + (h & 31);
#pragma unroll
            for (int e = 0; e < EPL; e++) {
                kpg[dst * HD + lane * EPL + e] = kpg[src * HD + lane * EPL + e];
                vpg[dst * HD + lane * EPL + e] = vpg[src * HD + lane * EPL + e];
            }
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
            t.cl_flags[cj] = 0; t.cl_flags[cn] = 0;
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
            // staged members of this child (by label) when the cluster was staged, else its rows in their new place
            const int n_scan = cached ? c : cc;
            for (int p = warp; p < n_scan; p += SP_WARPS) {
                if (cached && ((label[p] == stay) != (child == 0))) continue;
                const KV* k = (cached ? krows + (size_t)p * HD : kpg + ((size_t)pages[p >> 5] * PAGE + (p & 31)) * HD) + lane * EPL;
#pragma unroll
                for (int e = 0; e < EPL; e++) sa[e] += to_f(k[e]);
            }
#pragma unroll
            for (int e = 0; e < EPL; e++) wsum[warp][0][lane * EPL + e] = sa[e];
            __syncthreads();
            for (int e = tid; e < HD; e += SP_THREADS) {
                float s = 0.f;
                for (int w = 0; w < SP_WARPS; w++) s += wsum[w][0][e];
                s /= (float)cc;
                cA[e] = s;
                t.cl_r[cid * HD + e] = s;
            }
            __syncthreads();
            float mean[EPL], m2 = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; e++) mean[e] = cA[lane * EPL + e];
            for (int p = warp; p < n_scan; p += SP_WARPS) {
                if (cached && ((label[p] == stay) != (child == 0))) continue;
                const KV* k = (cached ? krows + (size_t)p * HD : kpg + ((size_t)pages[p >> 5] * PAGE + (p & 31)) * HD) + lane * EPL;
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; e++) { float df = to_f(k[e]) - mean[e]; part = fmaf(df, df, part); }
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
        // next step's scores and distances of the two children
        if (fronted && warp == 0) front_patch<KV, HD>(t, u, q1, k1, j, new_id);
    }
    __syncthreads();
    // No block leaves before the kernel ahead has completed: the next kernel on the stream (the next iteration's
    // centroid pass and selection, which rewrite the work lists) is ordered behind THIS kernel only.
    pdl_wait();
    if (tid == 0) {
        t.u_scan[u] = s_nsplit > 0 ? 1 : 0; t.u_last[u] = -1;
        if (step_ctr) {
            // the last block of the iteration advances the device-side step index that every kernel of the loop reads
            __threadfence();
            if (atomicAdd(t.plan_counter + 1, 1) == (int)gridDim.x - 1) { t.plan_counter[1] = 0; *step_ctr += 1; }
        }
    }
}

template <typename KV, int HD>
static void split_t(const Tables& t, float gamma, int var_enabled, int min_size, int iters, int do_append, StepPtr k, StepPtr v,
                    int* step_ctr, const NextFront& nf, cudaStream_t s) {
    const size_t dyn = SplitSmem<HD, (int)sizeof(KV)>::total(t.max_tokens / PAGE + 2, t.max_clusters);
    if (dyn > 32 * 1024)
        cudaFuncSetAttribute(k_split_check<KV, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    launch_pdl(k_split_check<KV, HD>, dim3(t.U), dim3(SP_THREADS), dyn, s, t, gamma, var_enabled, min_size, iters, do_append, k, v, step_ctr,
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
