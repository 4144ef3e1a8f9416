// SplitCluster (arXiv 2511.07427, Section 4.2 and Algorithm 1) for a cluster small enough to be staged in
// shared memory -- the common case, since a cluster is split soon after it has outgrown its siblings.
//
// A split sits on the critical path of a decode iteration and runs while other blocks saturate the memory
// system, so this version is built around two rules: (1) as few dependent trips to global memory as possible
// -- one for everything that depends only on the cluster id, the walk along its (short) page chain, one to
// stage its K rows, V rows and token ids; after that global memory is only written; (2) few block barriers --
// eight lanes share a row in every distance pass (three shuffle steps per reduction), a block-wide vote
// doubles as the "did any label change" test, and the member sums are taken by one thread per (row slice,
// dimension) for both sides at once.
//
// What is computed is exactly the split rule: centre A = member farthest from the representative, centre B =
// member farthest from A (ties: lowest token id); Lloyd on the two centres for at most `iters` rounds, ties to
// A, stopping when no label changes; a side left empty abandons the split; the child holding the smallest
// token id keeps the id and the pages, compacted in place; the other child moves to fresh pages under the
// next free id; both children get exact statistics (mean, M2 about the mean).
#pragma once

#include "common.cuh"
#include "fp8_rows.cuh"

namespace dkv {

struct SplitScratch {            // shared memory of the calling block
    float* cA; float* cB;        // [HD] each: the two centres; on return the children's means
    unsigned char* label;        // [rows]
    int* rank;                   // [rows]
    int* holes;                  // [rows]
    int* tok;                    // [rows]
    int* newpg;                  // [>= rows / PAGE + 1]
    float* part;                 // [THREADS / HD][2][HD] partial member sums
    int* nsplit;                 // [1] splits done by this block for the current unit
};

// Every thread of the block calls this with the same arguments.  krows / vrows: shared memory for `c` rows of
// K and of V.  Returns the new cluster's id, or -1 when the cluster stays as it is (abandoned, no id or no
// page left); *stay_side tells which of cA (0) / cB (1) is the mean of the child that kept id j.
template <typename KV, int HD, int THREADS, int MAXROWS>
__device__ int split_small(const Tables& t, int u, int j, int c, int iters, KV* krows, KV* vrows, const SplitScratch& sc,
                           int* stay_side) {
    constexpr int V4 = HD / 32;                           // 4-element pieces per lane of a row group
    constexpr int V16 = HD * (int)sizeof(KV) / 16;        // 16-byte pieces per row
    constexpr int MAXPG = MAXROWS / PAGE;                 // pages of a staged cluster
    constexpr int NW = THREADS / 32, NG = THREADS / 8;    // warps, row groups
    static_assert(MAXROWS <= THREADS && 2 * HD <= THREADS && THREADS % HD == 0 && MAXROWS % PAGE == 0, "one thread per member, per (side, dimension)");
    __shared__ float r_d[2][NW];
    __shared__ int r_t[2][NW], r_p[2][NW];
    __shared__ int s_ok;
    constexpr int Q = THREADS / HD;                       // row slices of the member-sum pass
    __shared__ int s_pcnt[Q];
    __shared__ signed char s_kx[MAXROWS], s_vx[MAXROWS];     // FP8 mode: the staged rows' scale exponents
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, sub = lane >> 3, l8 = lane & 7;
    const int grp = warp * 4 + sub;
    const size_t cj = (size_t)u * t.max_clusters + j;
    const int M = t.u_M[u];
    if (M >= t.max_clusters) { if (tid == 0) atomicOr(t.status, DYNAKV_ST_MAX_CLUSTERS); return -1; }
    KV* kpg = reinterpret_cast<KV*>(t.kpages) + (size_t)u * t.P * PAGE * HD;
    KV* vpg = reinterpret_cast<KV*>(t.vpages) + (size_t)u * t.P * PAGE * HD;
    int* ptok = t.page_tok + (size_t)u * t.P * PAGE;
    int* pnext = t.page_next + (size_t)u * t.P;

    // ---- everything that depends only on (u, j); the allocator state is thread 0's business
    const int npg = (c + PAGE - 1) / PAGE;
    int pg[MAXPG];
    pg[0] = t.cl_head[cj];
    int fc = 0, top = 0, mlive = 0;
    if (tid == 0) { fc = t.u_free_cnt[u]; top = t.u_page_top[u]; mlive = t.u_Mlive[u]; }
    for (int e = tid; e < HD; e += THREADS) sc.cA[e] = t.cl_r[cj * HD + e];
    // every thread walks the short chain itself: no broadcast through shared memory, no barrier
#pragma unroll
    for (int i = 1; i < MAXPG; i++) pg[i] = (i < npg && DKV_IN(t, SITE_SPLIT_PAGE, pg[i - 1], 0, t.P)) ? pnext[pg[i - 1]] : -1;
#ifdef DYNAKV_CHECKED
    // every thread has walked the same chain, so all of them leave together
    for (int i = 0; i < MAXPG; i++) if (i < npg && !DKV_IN(t, SITE_SPLIT_PAGE, pg[i], 0, t.P)) return -1;
#endif
    auto page_of = [&](int i) -> int {
        int r = pg[0];
#pragma unroll
        for (int k = 1; k < MAXPG; k++) r = (i == k) ? pg[k] : r;
        return r;
    };
    int fs[MAXPG];                       // top of the free stack, in pop order
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < MAXPG; i++) fs[i] = (fc > i) ? t.free_stack[(size_t)u * t.P + fc - 1 - i] : -1;
    }
    // ---- stage K rows, V rows, token ids
    for (int idx = tid; idx < c * V16; idx += THREADS) {
        const int p = idx / V16, v = idx % V16;
        const size_t row = (size_t)page_of(p >> 5) * PAGE + (p & 31);
        const int pv = row_pos<1>(row, v);       // the staged copies are in logical chunk order
        if (!t.fp8) {
            reinterpret_cast<uint4*>(krows + (size_t)p * HD)[v] = reinterpret_cast<const uint4*>(kpg + row * HD)[pv];
            reinterpret_cast<uint4*>(vrows + (size_t)p * HD)[v] = reinterpret_cast<const uint4*>(vpg + row * HD)[pv];
        } else {
            // FP8 storage keeps the rows as bytes only.  K is staged decoded (exact), eight elements per piece, so that
            // everything below works on the same bf16 rows as in bf16 storage; V's HD bytes are staged as they are.
            if constexpr (sizeof(KV) == 2) {
                const size_t g = (size_t)u * t.P * PAGE + row;
                const uint2 by = *reinterpret_cast<const uint2*>(t.k8 + g * HD + row_pos<16>(g, v * 8));
                const float sck = pow2f(t.k8e[g]);
                KV* o8 = krows + (size_t)p * HD + v * 8;
                const unsigned w2[2] = {by.x, by.y};
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    const float2 a = fp8_unpack2((unsigned short)(w2[h] & 0xffffu), sck), b = fp8_unpack2((unsigned short)(w2[h] >> 16), sck);
                    o8[4 * h] = (KV)a.x; o8[4 * h + 1] = (KV)a.y; o8[4 * h + 2] = (KV)b.x; o8[4 * h + 3] = (KV)b.y;
                }
                if (v < HD / 16)
                    reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(vrows) + (size_t)p * HD)[v] =
                        reinterpret_cast<const uint4*>(t.v8 + g * HD)[row_pos<1>(row, v)];
            }
        }
    }
    if (tid < c) {
        const size_t slot = (size_t)page_of(tid >> 5) * PAGE + (tid & 31);
        sc.tok[tid] = ptok[slot]; sc.label[tid] = 255;
        if (t.fp8) { s_kx[tid] = t.k8e[(size_t)u * t.P * PAGE + slot]; s_vx[tid] = t.v8e[(size_t)u * t.P * PAGE + slot]; }
    }
    __syncthreads();

    // ---- member farthest from a centre (ties: lowest token id).  The centre arrives in registers, as this
    // lane's share of a row; `buf` alternates so that the next call cannot overwrite what slow threads still read.
    auto farthest = [&](const float (&cen)[V4][4], int buf) -> int {
        float bd = -1.f; int bt = 0x7fffffff, bp = -1;
        for (int p0 = 0; p0 < c; p0 += NG) {
            const int p = p0 + grp;
            const bool valid = p < c;
            const KV* row = krows + (size_t)(valid ? p : 0) * HD;
            float d = 0.f;
#pragma unroll
            for (int i = 0; i < V4; i++) {
                const float4 k4 = ld4(row, l8 * 4 + 32 * i);
                const float a = k4.x - cen[i][0], b = k4.y - cen[i][1], e2 = k4.z - cen[i][2], f = k4.w - cen[i][3];
                d = fmaf(a, a, d); d = fmaf(b, b, d); d = fmaf(e2, e2, d); d = fmaf(f, f, d);
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            if (valid) {
                const int tok = sc.tok[p];
                if (d > bd || (d == bd && tok < bt)) { bd = d; bt = tok; bp = p; }
            }
        }
#pragma unroll
        for (int o = 8; o <= 16; o <<= 1) {
            const float od = __shfl_xor_sync(0xffffffffu, bd, o);
            const int ot = __shfl_xor_sync(0xffffffffu, bt, o), op = __shfl_xor_sync(0xffffffffu, bp, o);
            if (od > bd || (od == bd && ot < bt)) { bd = od; bt = ot; bp = op; }
        }
        if (lane == 0) { r_d[buf][warp] = bd; r_t[buf][warp] = bt; r_p[buf][warp] = bp; }
        __syncthreads();
        float d0 = r_d[buf][0]; int t0 = r_t[buf][0], p0 = r_p[buf][0];
#pragma unroll
        for (int w = 1; w < NW; w++)
            if (r_d[buf][w] > d0 || (r_d[buf][w] == d0 && r_t[buf][w] < t0)) { d0 = r_d[buf][w]; t0 = r_t[buf][w]; p0 = r_p[buf][w]; }
        return p0;
    };
    float cen[V4][4];
#pragma unroll
    for (int i = 0; i < V4; i++)
#pragma unroll
        for (int e = 0; e < 4; e++) cen[i][e] = sc.cA[l8 * 4 + 32 * i + e];
    const int pA = farthest(cen, 0);
#pragma unroll
    for (int i = 0; i < V4; i++) {
        const float4 k4 = ld4(krows + (size_t)pA * HD, l8 * 4 + 32 * i);
        cen[i][0] = k4.x; cen[i][1] = k4.y; cen[i][2] = k4.z; cen[i][3] = k4.w;
    }
    const int pB = farthest(cen, 1);
    // every thread is past its reads of the representative (the barrier inside the first call)
    for (int e = tid; e < HD; e += THREADS) { sc.cA[e] = to_f(krows[(size_t)pA * HD + e]); sc.cB[e] = to_f(krows[(size_t)pB * HD + e]); }
    __syncthreads();

    // ---- Lloyd on the two centres
    int nA = 0, nB = 0;
    bool abandoned = false;
    for (int it = 0; it < iters; it++) {
        float ca[V4][4], cb[V4][4];
#pragma unroll
        for (int i = 0; i < V4; i++)
#pragma unroll
            for (int e = 0; e < 4; e++) { ca[i][e] = sc.cA[l8 * 4 + 32 * i + e]; cb[i][e] = sc.cB[l8 * 4 + 32 * i + e]; }
        int chg = 0;
        for (int p0 = 0; p0 < c; p0 += NG) {
            const int p = p0 + grp;
            const bool valid = p < c;
            const KV* row = krows + (size_t)(valid ? p : 0) * HD;
            float da = 0.f, db = 0.f;
#pragma unroll
            for (int i = 0; i < V4; i++) {
                const float4 k4 = ld4(row, l8 * 4 + 32 * i);
                float x = k4.x - ca[i][0], y = k4.x - cb[i][0];
                da = fmaf(x, x, da); db = fmaf(y, y, db);
                x = k4.y - ca[i][1]; y = k4.y - cb[i][1];
                da = fmaf(x, x, da); db = fmaf(y, y, db);
                x = k4.z - ca[i][2]; y = k4.z - cb[i][2];
                da = fmaf(x, x, da); db = fmaf(y, y, db);
                x = k4.w - ca[i][3]; y = k4.w - cb[i][3];
                da = fmaf(x, x, da); db = fmaf(y, y, db);
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) { da += __shfl_xor_sync(0xffffffffu, da, o); db += __shfl_xor_sync(0xffffffffu, db, o); }
            if (valid && l8 == 0) {
                const unsigned char l = db < da ? 1 : 0;
                if (sc.label[p] != l) chg = 1;
                sc.label[p] = l;
            }
        }
        const int changed = __syncthreads_or(chg);        // also: the labels are complete
        // Member sums: thread (slice, dimension) adds up its slice of the rows for both sides at once (a
        // non-member contributes an exact + 0), the slices are combined in order afterwards.
        {
            const int x = tid % HD, qr = tid / HD;
            const int per = (c + Q - 1) / Q, p_lo = min(c, qr * per), p_hi = min(c, p_lo + per);
            float sA = 0.f, sB = 0.f; int nb = 0;
            for (int p = p_lo; p < p_hi; p++) {
                const float v = to_f(krows[(size_t)p * HD + x]);
                const int l = sc.label[p];
                sA += l ? 0.f : v; sB += l ? v : 0.f; nb += l;
            }
            sc.part[(qr * 2 + 0) * HD + x] = sA; sc.part[(qr * 2 + 1) * HD + x] = sB;
            if (x == 0) s_pcnt[qr] = nb;
        }
        __syncthreads();
        nB = 0;
#pragma unroll
        for (int q = 0; q < Q; q++) nB += s_pcnt[q];
        nA = c - nB;
        if (nA == 0 || nB == 0) { abandoned = true; break; }
        if (!changed) break;
        if (tid < 2 * HD) {
            const int side = tid / HD, x = tid % HD;
            float sum = 0.f;
#pragma unroll
            for (int q = 0; q < Q; q++) sum += sc.part[(q * 2 + side) * HD + x];
            (side ? sc.cB : sc.cA)[x] = sum / (float)(side ? nB : nA);
        }
        __syncthreads();
    }
    if (abandoned) { if (tid == 0) { t.cl_flags[cj] = FLAG_HOLD; t.cl_buf[cj] = 0; } return -1; }

    // ---- which side stays: the one holding the smallest token id
    int stay;
    {
        int bt = 0x7fffffff, bl = 0;
        if (tid < c) { bt = sc.tok[tid]; bl = sc.label[tid]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const int ot = __shfl_xor_sync(0xffffffffu, bt, o), ol = __shfl_xor_sync(0xffffffffu, bl, o);
            if (ot < bt) { bt = ot; bl = ol; }
        }
        if (lane == 0) { r_t[0][warp] = bt; r_p[0][warp] = bl; }
        __syncthreads();
        int t0 = r_t[0][0]; stay = r_p[0][0];
#pragma unroll
        for (int w = 1; w < NW; w++) if (r_t[0][w] < t0) { t0 = r_t[0][w]; stay = r_p[0][w]; }
    }
    const int s_n = stay ? nB : nA, m_n = c - s_n;
    const int need = (m_n + PAGE - 1) / PAGE, keep = (s_n + PAGE - 1) / PAGE;
    const int new_id = M;

    // ---- pages for the moving child (thread 0), ranks of every member (its own thread)
    if (tid == 0) {
        int ok = (fc + (t.P - top) >= need) ? 1 : 0;
        if (ok) {
            int used = 0;
            for (int i = 0; i < need; i++) {
                int pgi = -1;
                if (fc > 0) {
#pragma unroll
                    for (int k = 0; k < MAXPG; k++) pgi = (used == k) ? fs[k] : pgi;
                    used++; fc--;
                } else pgi = top++;
                sc.newpg[i] = pgi;
                if (!DKV_IN(t, SITE_SPLIT_PAGE, pgi, 0, t.P)) ok = 0;
            }
        } else atomicOr(t.status, DYNAKV_ST_PAGE_POOL);
        s_ok = ok;
    }
    if (tid < c) {
        // movers keep their order; stayers beyond position s_n fill, in order, the holes movers leave below s_n
        const int p = tid;
        int rm = 0, mb = 0;                     // movers before p; movers before min(p, s_n)
        for (int q = 0; q < p; q++) { const int mv = sc.label[q] != stay ? 1 : 0; rm += mv; mb += (q < s_n) ? mv : 0; }
        const bool mv = sc.label[p] != stay;
        int code = -1;                          // stays where it is
        if (mv) { code = rm; if (p < s_n) sc.holes[rm] = p; }
        else if (p >= s_n) code = -2 - ((p - s_n) - (rm - mb));     // filler number (p - s_n) - movers in [s_n, p)
        sc.rank[p] = code;
    }
    __syncthreads();
    if (!s_ok) return -1;

    // ---- moves, all out of shared memory: movers to the new pages, fillers into the holes
    for (int idx = tid; idx < c * V16; idx += THREADS) {
        const int p = idx / V16, v = idx % V16;
        const int code = sc.rank[p];
        if (code == -1) continue;
        size_t dst;
        if (code >= 0) dst = (size_t)sc.newpg[code >> 5] * PAGE + (code & 31);
        else { const int h = sc.holes[-2 - code]; dst = (size_t)page_of(h >> 5) * PAGE + (h & 31); }
        const int pv = row_pos<1>(dst, v);       // the destination slot's chunk order
        if (!t.fp8) {
            reinterpret_cast<uint4*>(kpg + dst * HD)[pv] = reinterpret_cast<const uint4*>(krows + (size_t)p * HD)[v];
            reinterpret_cast<uint4*>(vpg + dst * HD)[pv] = reinterpret_cast<const uint4*>(vrows + (size_t)p * HD)[v];
        }
        if (t.fp8) {
            if constexpr (sizeof(KV) == 2) {
                const size_t g = (size_t)u * t.P * PAGE + dst;
                // K's one-byte copy follows the row: the staged values are on the grid, so packing them with the row's
                // own scale gives the row's bytes back
                {
                    const KV* src = krows + (size_t)p * HD + v * 8;
                    const float inv = pow2f(-(int)s_kx[p]);
                    uint2 pk;
                    pk.x = (unsigned)fp8_pack2(to_f(src[0]), to_f(src[1]), inv) | ((unsigned)fp8_pack2(to_f(src[2]), to_f(src[3]), inv) << 16);
                    pk.y = (unsigned)fp8_pack2(to_f(src[4]), to_f(src[5]), inv) | ((unsigned)fp8_pack2(to_f(src[6]), to_f(src[7]), inv) << 16);
                    *reinterpret_cast<uint2*>(t.k8 + g * HD + row_pos<16>(g, v * 8)) = pk;
                    if (v == 0) { t.k8e[g] = s_kx[p]; t.v8e[g] = s_vx[p]; }
                }
                // V's bytes go from the staging area to the destination slot as they are
                if (v < HD / 16)
                    reinterpret_cast<uint4*>(t.v8 + g * HD)[row_pos<1>(dst, v)] =
                        reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(vrows) + (size_t)p * HD)[v];
            }
        }
    }
    if (tid < c) {
        const int code = sc.rank[tid], tok = sc.tok[tid];
        if (code >= 0) {
            ptok[(size_t)sc.newpg[code >> 5] * PAGE + (code & 31)] = tok;
            if (DKV_IN(t, SITE_SPLIT_TOKEN, tok, 0, t.max_tokens)) t.tok_cluster[(size_t)u * t.max_tokens + tok] = new_id;
        } else if (code <= -2) {
            const int h = sc.holes[-2 - code];
            ptok[(size_t)page_of(h >> 5) * PAGE + (h & 31)] = tok;
        }
    }
    // ---- chains, ids, allocator
    const size_t cn = (size_t)u * t.max_clusters + new_id;
    if (tid == 0) {
        const int last_kept = page_of(keep - 1);
        pnext[last_kept] = -1;
        t.cl_tail[cj] = last_kept;
        for (int i = keep; i < npg; i++) t.free_stack[(size_t)u * t.P + fc++] = page_of(i);
        t.u_free_cnt[u] = fc; t.u_page_top[u] = top;
        for (int i = 0; i < need; i++) pnext[sc.newpg[i]] = (i + 1 < need) ? sc.newpg[i + 1] : -1;
        t.cl_head[cn] = sc.newpg[0]; t.cl_tail[cn] = sc.newpg[need - 1];
        t.cl_n[cj] = s_n; t.cl_n[cn] = m_n;
        t.cl_flags[cj] = 0; t.cl_flags[cn] = 0; t.cl_buf[cj] = 0; t.cl_buf[cn] = 0;
        if (t.cl_ver) t.cl_ver[cj] = t.cl_ver[cj] + 1;      // two-tier mode: copies of the cluster made before now are void
        t.u_M[u] = new_id + 1; t.u_Mlive[u] = mlive + 1;
        atomicAdd(&t.counters[CNT_SPLITS], 1ull);
        *sc.nsplit = *sc.nsplit + 1;
    }
    // ---- exact statistics: cA / cB already are the means of the final labels; M2 about them
    if (tid < 2 * HD) {
        const int side = tid / HD, x = tid % HD;
        t.cl_r[(side == stay ? cj : cn) * HD + x] = (side ? sc.cB : sc.cA)[x];
    }
    {
        float ca[V4][4], cb[V4][4];
#pragma unroll
        for (int i = 0; i < V4; i++)
#pragma unroll
            for (int e = 0; e < 4; e++) { ca[i][e] = sc.cA[l8 * 4 + 32 * i + e]; cb[i][e] = sc.cB[l8 * 4 + 32 * i + e]; }
        float mA = 0.f, mB = 0.f;
        for (int p0 = 0; p0 < c; p0 += NG) {
            const int p = p0 + grp;
            const bool valid = p < c;
            const KV* row = krows + (size_t)(valid ? p : 0) * HD;
            const int l = valid ? sc.label[p] : 0;
            float d = 0.f;
#pragma unroll
            for (int i = 0; i < V4; i++) {
                const float4 k4 = ld4(row, l8 * 4 + 32 * i);
                const float a = k4.x - (l ? cb[i][0] : ca[i][0]), b = k4.y - (l ? cb[i][1] : ca[i][1]);
                const float e2 = k4.z - (l ? cb[i][2] : ca[i][2]), f = k4.w - (l ? cb[i][3] : ca[i][3]);
                d = fmaf(a, a, d); d = fmaf(b, b, d); d = fmaf(e2, e2, d); d = fmaf(f, f, d);
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            if (valid && l8 == 0) { if (l) mB += d; else mA += d; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { mA += __shfl_xor_sync(0xffffffffu, mA, o); mB += __shfl_xor_sync(0xffffffffu, mB, o); }
        if (lane == 0) { r_d[0][warp] = mA; r_d[1][warp] = mB; }
        __syncthreads();
        if (tid < 2) {
            float s = 0.f;
            for (int w = 0; w < NW; w++) s += r_d[tid][w];
            t.cl_M2[(tid == stay) ? cj : cn] = s;
        }
    }
    __syncthreads();
    *stay_side = stay;
    return new_id;
}

}  // namespace dkv
