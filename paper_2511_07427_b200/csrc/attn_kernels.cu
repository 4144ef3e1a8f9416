// Gather-attention over the selected clusters' pages for bf16 K/V: attention restricted to
// the retrieved entries (arXiv 2511.07427, Section 2.1 / 4.1), G query heads sharing every
// K/V row that is read.
//
// One persistent CTA per half SM.  The step's pages of ALL units form one flat list
// (work_prefix[u] .. work_prefix[u+1] are unit u's entries); CTA b owns the contiguous
// slice [b*per, (b+1)*per).  A producer warp streams the slice's pages -- exactly the
// valid rows of each, K and V, as two bulk-asynchronous copies (TMA, 1-D) -- into a
// shared-memory ring guarded by full/empty mbarriers; three consumer warps take the pages
// round-robin, each keeping an online-softmax state (m, l, acc) for the unit in progress.
//
// Consumer arithmetic: mma.sync m16n8k16 bf16 with fp32 accumulation.  K and V rows go
// from shared memory into operand registers with 128-bit loads: the contraction index of
// Q.K^T is permuted so that the 16 bytes a thread loads from a K row are exactly its B
// fragments of two k-steps, and the output columns of P.V are permuted so that the 16
// bytes a thread loads from each of its four V rows become, after one byte-permute per
// register, its B fragments of eight n-tiles.  Q (pre-scaled by log2(e)/sqrt(d)) and the
// softmax weights P are each split into bf16 hi + lo parts that sit in rows r and r+8 of
// the 16-row MMA tile, which the same thread accumulates, so fp32 queries and weights
// lose nothing that matters (2^-17 relative).
//
// Split-K combine: a unit whose entries lie inside one CTA's slice is normalised and
// written by that CTA.  A unit cut by slice boundaries leaves one unnormalised partial per
// CTA; each such CTA bumps the unit's arrival counter and the last one to arrive merges
// the partials and writes the output, so no CTA ever waits for another.
//
// FP8 storage (F8 = true, d = 128): the producer streams the one-byte copy of the pages -- e4m3 rows of 128 bytes and the
// rows' scale exponents -- so a row costs 258 bytes instead of 512.  The consumers turn the bytes into f16 operands
// (exact: e4m3 has four significant bits) with the paired conversion instruction and use f16 MMAs; Q, divided by a
// power of two per head so that it fits f16 whatever its size, and the softmax weights are split into f16 hi + lo
// parts.  A K row's scale multiplies its logit; a V row's scale 2^e is folded into the softmax: the running maximum is
// kept over (logit + e), the MMA weight is 2^(logit + e - max) <= 1 and the denominator adds that weight times 2^-e,
// so numerator and denominator carry the same factor and every merge below works unchanged.
#include <cuda_fp16.h>
#include <float.h>

#include "bulk_copy.cuh"
#include "common.cuh"
#include "fp8_rows.cuh"

namespace dkv {

__device__ __forceinline__ void mma_bf16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (hi, lo) bf16 split of two floats packed as bf16x2 (first value in the low half).
__device__ __forceinline__ void split2(float x, float y, unsigned& hi, unsigned& lo) {
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(hi) : "f"(y), "f"(x));          // first source operand goes to the upper half
    const float xr = x - __uint_as_float(hi << 16), yr = y - __uint_as_float(hi & 0xffff0000u);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(lo) : "f"(yr), "f"(xr));
}

__device__ __forceinline__ void mma_f16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                        unsigned b0, unsigned b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (hi, lo) f16 split of two floats in [-1, 1], packed as f16x2 (first value in the low half).
__device__ __forceinline__ void split2h(float x, float y, unsigned& hi, unsigned& lo) {
    const __half2 h = __floats2half2_rn(x, y);
    const float2 hf = __half22float2(h);
    const __half2 l = __floats2half2_rn(x - hf.x, y - hf.y);
    hi = *reinterpret_cast<const unsigned*>(&h);
    lo = *reinterpret_cast<const unsigned*>(&l);
}

// Four e4m3 bytes as two f16x2 registers: lo from bytes 0 and 1, hi from bytes 2 and 3.
__device__ __forceinline__ void e4m3x4_to_f16x2(unsigned b, unsigned& lo, unsigned& hi) {
    asm("{\n .reg .b16 l, h;\n mov.b32 {l, h}, %2;\n cvt.rn.f16x2.e4m3x2 %0, l;\n cvt.rn.f16x2.e4m3x2 %1, h;\n}\n"
        : "=r"(lo), "=r"(hi) : "r"(b));
}

__device__ __forceinline__ int lds_s8x2(unsigned addr) {      // two signed bytes: low byte in .x of the result pair
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];\n" : "=h"(v) : "r"(addr));
    return (int)v;
}

// 2^x for x <= 8 or so (flushes tiny results to zero; -inf gives 0): one special-function instruction.
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 lds16(unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

#ifndef DKV_AT_CONSUMERS
#define DKV_AT_CONSUMERS 3
#endif
#ifndef DKV_AT_STAGES
#define DKV_AT_STAGES 6
#endif
constexpr int AT_CONSUMERS = DKV_AT_CONSUMERS;      // consumer warps
constexpr int AT_THREADS = (AT_CONSUMERS + 1) * 32; // + one producer warp
constexpr int AT_STAGES = DKV_AT_STAGES;                      // work entries (runs of <= ENTRY_ROWS rows) in flight per CTA
#ifndef DKV_AT_STAGES_F8
#define DKV_AT_STAGES_F8 9
#endif
constexpr int AT_STAGES_F8 = DKV_AT_STAGES_F8;                // the same for the one-byte rows (stages half the size)
// Item i of a CTA's slice is consumed by warp i % AT_CONSUMERS from ring stage i % stages.  A stage
// must always be consumed by the same warp: a parity wait cannot tell phase p from phase p + 2, so a
// warp must never be able to run two phases ahead of another warp on a shared stage.
static_assert(AT_STAGES <= 32 && AT_STAGES % AT_CONSUMERS == 0, "each ring stage belongs to one consumer warp");
static_assert(AT_STAGES_F8 <= 32 && AT_STAGES_F8 % AT_CONSUMERS == 0, "each ring stage belongs to one consumer warp");

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;\n" ::"n"(AT_CONSUMERS * 32) : "memory"); }

template <int HD, bool F8> struct AttnSmem {
    static constexpr int stages = F8 ? AT_STAGES_F8 : AT_STAGES;
    static constexpr int row_bytes = F8 ? HD : HD * 2;
    // K rows then V rows of one entry; FP8: then the K rows' and the V rows' scale exponents (ENTRY_ROWS bytes each)
    static constexpr int stage_bytes = 2 * ENTRY_ROWS * row_bytes + (F8 ? 128 : 0);
    static constexpr int ring_bytes = stages * stage_bytes;
    static constexpr int merge_row = HD + 2;                              // floats between rows of the merge scratch
    static constexpr int merge_bytes = AT_CONSUMERS * 8 * (merge_row + 2) * 4;   // per warp: acc[8][HD + 2], m[8], l[8]
    static constexpr int fixed_bytes = ring_bytes + merge_bytes + 2 * stages * 8 + stages * 4 + 64;
};

// Smallest u with pf[u+1] > k, starting the search at u0 (pf non-decreasing).
__device__ __forceinline__ int unit_of(const int* pf, int u0, int k) {
    int u = u0;
    while (pf[u + 1] <= k) u++;
    return u;
}

// Same by bisection over all U units.
__device__ __forceinline__ int unit_of_bisect(const int* pf, int U, int k) {
    int a = 0, b = U - 1;            // invariant: the answer lies in [a, b]
    while (a < b) {
        const int mid = (a + b) >> 1;
        if (pf[mid + 1] > k) b = mid; else a = mid + 1;
    }
    return a;
}

template <int HD, bool F8>
__global__ void __launch_bounds__(AT_THREADS, 2) k_gather_attn_tma(Tables t, StepPtr qp, StepPtrW outp) {
    static_assert(!F8 || HD == 128, "the one-byte rows are kept for d = 128");
    using SM = AttnSmem<HD, F8>;
    constexpr int AT_STAGES = SM::stages;
    constexpr int KS = HD / 16;       // k-steps of Q.K^T
    constexpr int KJ = F8 ? KS / 4 : KS / 2;   // 16-byte chunks a thread loads per K row
    constexpr int NT = HD / 8;        // n-tiles of P.V
    constexpr int VI = F8 ? 1 : HD / 64;       // 16-byte chunks a thread loads per V row
    constexpr int ROWB = SM::row_bytes;        // bytes per K or V row
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* ring = smem;
    float* mrg = reinterpret_cast<float*>(smem + SM::ring_bytes);
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + SM::ring_bytes + SM::merge_bytes);
    int* meta = reinterpret_cast<int*>(bars + 2 * AT_STAGES);
    int* s_flag = meta + AT_STAGES;                  // [0] abort, [1] combine-here, [2..] warp totals of the prefix scan
    int* pf_s = s_flag + 16;                         // the units' work-list prefix when it fits
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int U = t.U, G = t.G;
    const int nb = gridDim.x, b = blockIdx.x;

    // ---- prologue: barriers, prefix copy, slice bounds
    if (tid == 0) {
        for (int s = 0; s < AT_STAGES; s++) { mbar_init(smem_u32(&bars[s]), 1); mbar_init(smem_u32(&bars[AT_STAGES + s]), 1); }
        s_flag[0] = 0; s_flag[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    pdl_trigger();       // the append/split kernel may move in as CTAs of this grid retire; it waits before it moves rows
    pdl_wait();          // the work lists and their prefix come from the selection (the kernel before)
    const int* n_work = t.n_work;
    const int2* work = t.work;
    const int* pf = t.work_prefix;
    if (t.attn_pf_in_smem) {
        // Every CTA lays the units' work lists end to end itself: an exclusive prefix of their lengths, each
        // thread taking a run of consecutive units (all its loads in flight together), then a block scan.
        constexpr int MAXPER = 1024 / AT_THREADS;         // attn_pf_in_smem is set for at most 1024 units
        const int per_t = (U + AT_THREADS - 1) / AT_THREADS;
        const int b0 = min(tid * per_t, U);
        int nw[MAXPER];
        int sum = 0;
#pragma unroll
        for (int i = 0; i < MAXPER; i++) { nw[i] = (i < per_t && b0 + i < U) ? n_work[b0 + i] : 0; sum += nw[i]; }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        if (lane == 31) s_flag[2 + warp] = incl;
        __syncthreads();
        int base = incl - sum;
        for (int w = 0; w < warp; w++) base += s_flag[2 + w];
#pragma unroll
        for (int i = 0; i < MAXPER; i++) if (i < per_t && b0 + i < U) { pf_s[b0 + i] = base; base += nw[i]; }
        if (tid == AT_THREADS - 1) pf_s[U] = base;
        pf = pf_s;
    }
    __syncthreads();
    const int Wtot = pf[U];
    const int per = max((Wtot + nb - 1) / nb, 1);
    const int lo = min(b * per, Wtot), hi = min(lo + per, Wtot);
    float* out = reinterpret_cast<float*>(outp.get());
    // units with nothing selected: zeros
    if (warp > 0) {
        for (int u = b; u < U; u += nb)
            if (pf[u + 1] == pf[u])
                for (int i = tid - 32; i < G * HD; i += AT_CONSUMERS * 32) out[(size_t)u * G * HD + i] = 0.f;
    }
    if (lo >= hi) return;
    const int n_items = hi - lo;

    if (warp == 0) {
        // =============================== producer ===============================
        // Lane j owns ring stage j: it fetches the work entries of items j, j + stages, ... and issues their copies as
        // soon as the stage's consumer has released it.  The lanes stay in lockstep: every turn of the loop each lane
        // takes one non-suspending look at its own stage's barrier and the lanes whose stage is free refill it, so a lane
        // whose stage is still in use never holds up one whose stage has just been released.
        const bool mine = lane < AT_STAGES && lane < n_items;
        const int sl = lane < AT_STAGES ? lane : 0;
        const unsigned char* kp = F8 ? t.k8 : reinterpret_cast<const unsigned char*>(t.kpages);
        const unsigned char* vp = F8 ? t.v8 : reinterpret_cast<const unsigned char*>(t.vpages);
        const unsigned full = smem_u32(&bars[sl]), empty = smem_u32(&bars[AT_STAGES + sl]);
        const unsigned dst = smem_u32(ring + (size_t)sl * SM::stage_bytes);
        int it = lane;                     // this lane's next item
        int u = 0;
        int2 ent = make_int2(0, 0);
        if (mine) {
            u = unit_of_bisect(pf, U, lo + lane);
            ent = work[(size_t)u * t.W + (lo + lane - pf[u])];
        }
        bool active = mine, failed = false;
        int last_issued = -1, idle = 0;
        unsigned long long t_idle = 0;
        while (__any_sync(0xffffffffu, active)) {
            const bool ready = active && mbar_test_wait(empty, (((unsigned)(it / AT_STAGES)) & 1u) ^ 1u);
            if (ready) {
                int2 cur = ent;
                const int cu = u;
                // checked build: a bad entry is replaced by one row of the unit's first page, so the stage still fills
                if (!DKV_IN(t, SITE_ATTN_ENTRY, cur.y, 1, ENTRY_ROWS + 1)) cur.y = 1;
                if (!DKV_IN(t, SITE_ATTN_ENTRY, cur.x, 0, (long long)t.P * PAGE - cur.y + 1)) cur.x = 0;
                const int nx = it + AT_STAGES;
                if (nx < n_items) {          // next entry: its load is in flight until the stage comes round again
                    u = unit_of(pf, u, lo + nx);
                    ent = DKV_IN(t, SITE_ATTN_WORK, lo + nx - pf[u], 0, t.W) ? work[(size_t)u * t.W + (lo + nx - pf[u])] : make_int2(0, 1);
                }
                const unsigned bytes = (unsigned)cur.y * ROWB;
                const size_t row0 = (size_t)cu * t.P * PAGE + cur.x;
                const size_t src = row0 * ROWB;
                meta[sl] = cur.y;
                mbar_arrive_expect_tx(full, 2 * bytes + (F8 ? 2 * ENTRY_ROWS : 0));
                bulk_g2s(dst, kp + src, bytes, full);
                bulk_g2s(dst + ENTRY_ROWS * ROWB, vp + src, bytes, full);
                if constexpr (F8) {
                    // the run's scale exponents: first row a multiple of ENTRY_ROWS, so source and size are multiples of 16
                    bulk_g2s(dst + 2 * ENTRY_ROWS * ROWB, t.k8e + row0, ENTRY_ROWS, full);
                    bulk_g2s(dst + 2 * ENTRY_ROWS * ROWB + ENTRY_ROWS, t.v8e + row0, ENTRY_ROWS, full);
                }
                last_issued = it;
                it = nx;
                active = nx < n_items;
            }
            if (__any_sync(0xffffffffu, ready)) { idle = 0; t_idle = 0; continue; }
            // nothing was free this turn: the wait is bounded by turns and by time, and ends when a consumer gave up
            idle++;
            if ((idle & 63) == 0) {
                bool stop = idle >= (1 << 22) || *(volatile int*)&s_flag[0] != 0;
                if (lane == 0) {
                    const unsigned long long now = global_ns();
                    if (t_idle == 0) t_idle = now;
                    else if (now - t_idle > 200000000ull) stop = true;
                }
                if (__any_sync(0xffffffffu, stop)) { failed = true; break; }
            }
        }
        if (failed || *(volatile int*)&s_flag[0]) {
            // a bounded wait ran out: report it, and let every lane's last copy land before the CTA's shared memory can
            // be handed to another CTA
            if (lane == 0) { s_flag[0] = 1; atomicOr(t.status, DYNAKV_ST_INTERNAL); }
            if (mine && last_issued >= 0) mbar_wait(full, (unsigned)(last_issued / AT_STAGES) & 1u);
        }
        return;
    }

    // =============================== consumers ===============================
    const int cw = warp - 1, ctid = tid - 32;
    const int r = lane >> 2, c = lane & 3;
    const float scale = rsqrtf((float)HD) * 1.4426950408889634f;
    const float* qbase = reinterpret_cast<const float*>(qp.get());
    // Merge scratch.  A warp's accumulator fragments go out with lanes (r, c) writing row r at columns 16 or 32 apart:
    // with rows HD floats apart every lane of such a store would hit one of two banks (or one).  Rows are HD + 2
    // floats apart and column x sits at x ^ bit5(x) ^ (bit6(x) << 4), which spreads the 32 lanes of every store over
    // the 32 banks and leaves the merge loop's row-wise reads conflict-free.
    constexpr int MR = SM::merge_row;
    auto mcol = [](int x) -> int { return x ^ ((x >> 5) & 1) ^ (((x >> 6) & 1) << 4); };
    float* mrg_o = mrg;                                   // [AT_CONSUMERS][8][MR]
    float* mrg_m = mrg + AT_CONSUMERS * 8 * MR;           // [AT_CONSUMERS][8]
    float* mrg_l = mrg_m + AT_CONSUMERS * 8;              // [AT_CONSUMERS][8]

    int u = unit_of_bisect(pf, U, lo);
    const int u_first = u;
    int k = lo;
    while (k < hi) {
        u = unit_of(pf, u, k);
        const int seg_end = min(hi, pf[u + 1]);
        // ---- Q fragments of unit u: rows 0..7 = hi part of head r, rows 8..15 = lo part of head r
        const float* q = qbase + (size_t)u * G * HD;
        unsigned qa[KS][4];
        float head_scale = 0.f;          // FP8: what a logit of head r is multiplied by besides the K row's scale
        if constexpr (F8) {
            // k-step ks takes elements 16 (2c + ks / 4) + 4 (ks % 4) .. + 3: the 16 bytes a thread loads from a K row
            // are its B fragments of four k-steps.  Head r is divided by 2^ex, ex the exponent of its largest magnitude.
            float4 qv[KS];
            float amax = 0.f;
#pragma unroll
            for (int ks = 0; ks < KS; ks++) {
                const int base = 16 * (2 * c + (ks >> 2)) + 4 * (ks & 3);
                qv[ks] = r < G ? *reinterpret_cast<const float4*>(q + r * HD + base) : make_float4(0.f, 0.f, 0.f, 0.f);
                amax = fmaxf(fmaxf(amax, fmaxf(fabsf(qv[ks].x), fabsf(qv[ks].y))), fmaxf(fabsf(qv[ks].z), fabsf(qv[ks].w)));
            }
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            int ex = 0;
            if (amax > 0.f && amax < INFINITY) frexpf(amax, &ex);
            ex = max(-100, min(100, ex));
            const float inv = pow2f(-ex);
            head_scale = pow2f(ex) * scale;
#pragma unroll
            for (int ks = 0; ks < KS; ks++) {
                split2h(qv[ks].x * inv, qv[ks].y * inv, qa[ks][0], qa[ks][1]);
                split2h(qv[ks].z * inv, qv[ks].w * inv, qa[ks][2], qa[ks][3]);
            }
        } else {
#pragma unroll
        for (int ks = 0; ks < KS; ks++) {
            const int base = 8 * (2 * c + ((ks >> 1) & 1) + (KJ > 2 ? 8 : 2) * (ks >> 2)) + 4 * (ks & 1);
            float x0 = 0.f, x1 = 0.f, x2 = 0.f, x3 = 0.f;
            if (r < G) {
                const float4 v = *reinterpret_cast<const float4*>(q + r * HD + base);
                x0 = v.x * scale; x1 = v.y * scale; x2 = v.z * scale; x3 = v.w * scale;
            }
            split2(x0, x1, qa[ks][0], qa[ks][1]);
            split2(x2, x3, qa[ks][2], qa[ks][3]);
        }
        }
        float o[NT][4];
#pragma unroll
        for (int x = 0; x < NT; x++) { o[x][0] = 0.f; o[x][1] = 0.f; o[x][2] = 0.f; o[x][3] = 0.f; }
        float m = -INFINITY, l = 0.f;

        // first item of this segment owned by this warp: (kk - lo) % AT_CONSUMERS == cw
        int kk = k + ((cw - ((k - lo) % AT_CONSUMERS)) + AT_CONSUMERS) % AT_CONSUMERS;
        bool dead = false;
        for (; kk < seg_end; kk += AT_CONSUMERS) {
            const int it = kk - lo, stage = it % AT_STAGES;
            const unsigned ph = (unsigned)(it / AT_STAGES) & 1u;
            if (!mbar_wait(smem_u32(&bars[stage]), ph)) { s_flag[0] = 1; dead = true; break; }
            const int rows = meta[stage];
            const unsigned kbase = smem_u32(ring + (size_t)stage * SM::stage_bytes);
            const unsigned vbase = kbase + ENTRY_ROWS * ROWB;
#pragma unroll 1
            for (int sub = 0; sub < ENTRY_ROWS / 16; sub++) {
                const int nvalid = rows - sub * 16;
                if (nvalid <= 0) break;
                const unsigned krow0 = kbase + (unsigned)(sub * 16) * ROWB, vrow0 = vbase + (unsigned)(sub * 16) * ROWB;
                if constexpr (F8) {
                // ---- loads: K rows (tile*8 + r), chunks 2c + j; V rows 2c, 2c+1, 2c+8, 2c+9, chunk r (each at its place in
                // the row's stored chunk order, which keeps the lanes of one load on distinct banks); the scale exponents
                // of this thread's four tokens (tile*8 + 2c, + 1)
                // (rows past the run's end are read from its last row instead: their logits are masked and their weights
                // are zero, so all they must be is finite)
                uint4 kw[2][KJ];
#pragma unroll
                for (int tile = 0; tile < 2; tile++) {
                    const unsigned row = (unsigned)min(tile * 8 + r, nvalid - 1);
#pragma unroll
                    for (int j = 0; j < KJ; j++) kw[tile][j] = lds16(krow0 + row * ROWB + 16u * ((2 * c + j) ^ (row & 7)));
                }
                uint4 vw[4];
#pragma unroll
                for (int rr = 0; rr < 4; rr++) {
                    const unsigned tok = (unsigned)min(2 * c + (rr & 1) + 8 * (rr >> 1), nvalid - 1);
                    vw[rr] = lds16(vrow0 + tok * ROWB + 16u * (r ^ (tok & 7)));
                }
                const unsigned xbase = kbase + 2 * ENTRY_ROWS * ROWB + (unsigned)(sub * 16);
                int kx[4], vx[4];
#pragma unroll
                for (int tile = 0; tile < 2; tile++) {
                    const int kp2 = lds_s8x2(xbase + tile * 8 + 2 * c), vp2 = lds_s8x2(xbase + ENTRY_ROWS + tile * 8 + 2 * c);
                    kx[tile * 2] = (int)(signed char)(kp2 & 0xff); kx[tile * 2 + 1] = (int)(signed char)(kp2 >> 8);
                    vx[tile * 2] = (int)(signed char)(vp2 & 0xff); vx[tile * 2 + 1] = (int)(signed char)(vp2 >> 8);
                }
                // ---- S = Q K^T for the two 8-token tiles: word w of chunk j holds the B fragments of k-step 4j + w
                float sc[2][4];
#pragma unroll
                for (int tile = 0; tile < 2; tile++) {
                    float s2[4] = {0.f, 0.f, 0.f, 0.f};      // two chains of four MMAs instead of one of eight
                    sc[tile][0] = 0.f; sc[tile][1] = 0.f; sc[tile][2] = 0.f; sc[tile][3] = 0.f;
#pragma unroll
                    for (int j = 0; j < KJ; j++) {
                        const unsigned* w4 = reinterpret_cast<const unsigned*>(&kw[tile][j]);
#pragma unroll
                        for (int w = 0; w < 4; w++) {
                            const int ks = 4 * j + w;
                            unsigned b0, b1;
                            e4m3x4_to_f16x2(w4[w], b0, b1);
                            if (w & 1) mma_f16(s2, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                            else mma_f16(sc[tile], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                        }
                    }
#pragma unroll
                    for (int e = 0; e < 4; e++) sc[tile][e] += s2[e];
                }
                // logits of head r (hi row + lo row) times the head's and the K row's scales; for the softmax the V row's
                // exponent is added
                float lg[4];
#pragma unroll
                for (int tile = 0; tile < 2; tile++) {
                    const int tok = tile * 8 + 2 * c;
#pragma unroll
                    for (int h = 0; h < 2; h++) {
                        const int e = tile * 2 + h;
                        const bool ok = tok + h < nvalid;
                        if (!ok) { kx[e] = 0; vx[e] = 0; }
                        lg[e] = ok ? (sc[tile][h] + sc[tile][2 + h]) * head_scale * pow2f(kx[e]) + (float)vx[e] : -INFINITY;
                    }
                }
                float mx = fmaxf(fmaxf(lg[0], lg[1]), fmaxf(lg[2], lg[3]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                // the reference point of the exponentials follows the running maximum lazily: it moves only when the maximum
                // has grown by more than 2^8, so weights stay below 2^8 and the accumulators are rarely rescaled
                const float mn = mx > m + 8.f ? mx : m;        // finite: row 0 of the entry is valid
                const float corr = ex2(m - mn);
                m = mn;
                float p[4];
#pragma unroll
                for (int e = 0; e < 4; e++) p[e] = ex2(lg[e] - mn);
                l = l * corr + (p[0] * pow2f(-vx[0]) + p[1] * pow2f(-vx[1])) + (p[2] * pow2f(-vx[2]) + p[3] * pow2f(-vx[3]));
                unsigned pa[4];
                split2h(p[0], p[1], pa[0], pa[1]);   // a0 = hi(tile 0), a1 = lo(tile 0)
                split2h(p[2], p[3], pa[2], pa[3]);   // a2 = hi(tile 1), a3 = lo(tile 1)
                if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
                    for (int x = 0; x < NT; x++) { o[x][0] *= corr; o[x][1] *= corr; o[x][2] *= corr; o[x][3] *= corr; }
                }
                // ---- O += P V : n-tile e takes byte e of the chunk of the thread's four rows (column 16 r + e)
                const unsigned* a0 = reinterpret_cast<const unsigned*>(&vw[0]);
                const unsigned* a1 = reinterpret_cast<const unsigned*>(&vw[1]);
                const unsigned* a2 = reinterpret_cast<const unsigned*>(&vw[2]);
                const unsigned* a3 = reinterpret_cast<const unsigned*>(&vw[3]);
#pragma unroll
                for (int w = 0; w < 4; w++) {
#pragma unroll
                    for (int h = 0; h < 2; h++) {
                        // bytes (2h, 2h+1) of word w of two rows, interleaved: row A byte, row B byte, row A next, row B next
                        const unsigned sel = h ? 0x7362u : 0x5140u;
                        const unsigned t01 = __byte_perm(a0[w], a1[w], sel), t23 = __byte_perm(a2[w], a3[w], sel);
                        unsigned b0e, b0o, b1e, b1o;      // even / odd byte of the pair
                        e4m3x4_to_f16x2(t01, b0e, b0o);
                        e4m3x4_to_f16x2(t23, b1e, b1o);
                        mma_f16(o[4 * w + 2 * h], pa[0], pa[1], pa[2], pa[3], b0e, b1e);
                        mma_f16(o[4 * w + 2 * h + 1], pa[0], pa[1], pa[2], pa[3], b0o, b1o);
                    }
                }
                } else {
                // ---- loads: K rows (tile*8 + r), chunks 2c, 2c+1, 2c+8, 2c+9; V rows 2c, 2c+1, 2c+8, 2c+9, chunks r + 8i
                // (each at its place in the row's stored chunk order, which keeps the lanes of one load on distinct banks)
                uint4 kw[2][KJ];
#pragma unroll
                // (rows past the run's end are read from its last row instead: their logits are masked and their weights
                // are zero, so all they must be is finite)
                for (int tile = 0; tile < 2; tile++) {
                    const unsigned row = (unsigned)min(tile * 8 + r, nvalid - 1);
#pragma unroll
                    for (int j = 0; j < KJ; j++)
                        kw[tile][j] = lds16(krow0 + row * ROWB + 16u * ((2 * c + (j & 1) + (KJ > 2 ? 8 : 2) * (j >> 1)) ^ (row & 7)));
                }
                uint4 vw[4][VI];
#pragma unroll
                for (int rr = 0; rr < 4; rr++) {
                    const unsigned tok = (unsigned)min(2 * c + (rr & 1) + 8 * (rr >> 1), nvalid - 1);
#pragma unroll
                    for (int i = 0; i < VI; i++) vw[rr][i] = lds16(vrow0 + tok * ROWB + 16u * ((r + 8 * i) ^ (tok & 7)));
                }
                // ---- S = Q K^T for the two 8-token tiles
                float sc[2][4];
#pragma unroll
                for (int tile = 0; tile < 2; tile++) {
                    float s2[4] = {0.f, 0.f, 0.f, 0.f};      // two chains of MMAs instead of one twice as long
                    sc[tile][0] = 0.f; sc[tile][1] = 0.f; sc[tile][2] = 0.f; sc[tile][3] = 0.f;
#pragma unroll
                    for (int j = 0; j < KJ; j++) {
                        mma_bf16(sc[tile], qa[2 * j][0], qa[2 * j][1], qa[2 * j][2], qa[2 * j][3], kw[tile][j].x, kw[tile][j].y);
                        mma_bf16(s2, qa[2 * j + 1][0], qa[2 * j + 1][1], qa[2 * j + 1][2], qa[2 * j + 1][3], kw[tile][j].z, kw[tile][j].w);
                    }
#pragma unroll
                    for (int e = 0; e < 4; e++) sc[tile][e] += s2[e];
                }
                // logits of head r for tokens tile*8 + 2c + {0,1}: hi row + lo row
                float lg[4];
#pragma unroll
                for (int tile = 0; tile < 2; tile++) {
                    const int tok = tile * 8 + 2 * c;
                    lg[tile * 2 + 0] = tok < nvalid ? sc[tile][0] + sc[tile][2] : -INFINITY;
                    lg[tile * 2 + 1] = tok + 1 < nvalid ? sc[tile][1] + sc[tile][3] : -INFINITY;
                }
                float mx = fmaxf(fmaxf(lg[0], lg[1]), fmaxf(lg[2], lg[3]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                // the reference point of the exponentials follows the running maximum lazily: it moves only when the maximum
                // has grown by more than 2^8, so weights stay below 2^8 and the accumulators are rarely rescaled
                const float mn = mx > m + 8.f ? mx : m;        // finite: row 0 of the entry is valid
                const float corr = ex2(m - mn);
                m = mn;
                float p[4];
#pragma unroll
                for (int e = 0; e < 4; e++) p[e] = ex2(lg[e] - mn);
                l = l * corr + (p[0] + p[1]) + (p[2] + p[3]);
                unsigned pa[4];
                split2(p[0], p[1], pa[0], pa[1]);   // a0 = hi(tile 0), a1 = lo(tile 0)
                split2(p[2], p[3], pa[2], pa[3]);   // a2 = hi(tile 1), a3 = lo(tile 1)
                if (__any_sync(0xffffffffu, corr != 1.f)) {      // the running maximum rarely moves after the first entries
#pragma unroll
                    for (int x = 0; x < NT; x++) { o[x][0] *= corr; o[x][1] *= corr; o[x][2] *= corr; o[x][3] *= corr; }
                }
                // ---- O += P V : n-tile (i, e) takes element e of chunk i of the thread's four rows
#pragma unroll
                for (int i = 0; i < VI; i++) {
                    const unsigned* a0 = reinterpret_cast<const unsigned*>(&vw[0][i]);
                    const unsigned* a1 = reinterpret_cast<const unsigned*>(&vw[1][i]);
                    const unsigned* a2 = reinterpret_cast<const unsigned*>(&vw[2][i]);
                    const unsigned* a3 = reinterpret_cast<const unsigned*>(&vw[3][i]);
#pragma unroll
                    for (int e = 0; e < 8; e++) {
                        const unsigned sel = (e & 1) ? 0x7632u : 0x5410u;
                        const unsigned b0 = __byte_perm(a0[e >> 1], a1[e >> 1], sel);
                        const unsigned b1 = __byte_perm(a2[e >> 1], a3[e >> 1], sel);
                        mma_bf16(o[i * 8 + e], pa[0], pa[1], pa[2], pa[3], b0, b1);
                    }
                }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[AT_STAGES + stage]));
        }
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);

        // ---- merge the consumer warps' states for unit u
        if (c == 0) { mrg_m[cw * 8 + r] = m; mrg_l[cw * 8 + r] = l; }
#pragma unroll
        for (int x = 0; x < NT; x++) {
            if constexpr (F8) {           // n-tile x, accumulator columns 2c and 2c+1: output columns 16 (2c) + x and 16 (2c+1) + x
                mrg_o[(cw * 8 + r) * MR + mcol(16 * (2 * c) + x)] = o[x][0] + o[x][2];
                mrg_o[(cw * 8 + r) * MR + mcol(16 * (2 * c + 1) + x)] = o[x][1] + o[x][3];
            } else {
            const int i = x >> 3, e = x & 7;
            mrg_o[(cw * 8 + r) * MR + mcol(8 * (2 * c + 8 * i) + e)] = o[x][0] + o[x][2];
            mrg_o[(cw * 8 + r) * MR + mcol(8 * (2 * c + 1 + 8 * i) + e)] = o[x][1] + o[x][3];
            }
        }
        consumer_sync();
        if (*(volatile int*)&s_flag[0] || dead) {
            if (ctid == 0) atomicOr(t.status, DYNAKV_ST_INTERNAL);
            return;      // all consumer warps see the flag after the barrier and leave together
        }
        const bool whole = pf[u] >= lo && pf[u + 1] <= hi;
        // partial record: acc[G][HD], then m[8], then l[8] (floats; every row 16-byte aligned)
        const size_t rec_floats = (size_t)G * HD + 16;
        float* part = t.part + (size_t)(2 * b + (u == u_first ? 0 : 1)) * rec_floats;
        for (int idx = ctid; idx < G * HD; idx += AT_CONSUMERS * 32) {
            const int g = idx / HD, e = idx % HD;
            float mm = mrg_m[g];
#pragma unroll
            for (int w = 1; w < AT_CONSUMERS; w++) mm = fmaxf(mm, mrg_m[w * 8 + g]);
            float a = 0.f, ll = 0.f;
            if (mm != -INFINITY) {
#pragma unroll
                for (int w = 0; w < AT_CONSUMERS; w++) {
                    const float f = exp2f(mrg_m[w * 8 + g] - mm);
                    a += mrg_o[(w * 8 + g) * MR + mcol(e)] * f; ll += mrg_l[w * 8 + g] * f;
                }
            }
            if (whole) out[(size_t)u * G * HD + idx] = ll > 0.f ? a / ll : 0.f;
            else {
                __stcg(&part[idx], a);
                if (e == 0) { __stcg(&part[G * HD + g], mm); __stcg(&part[G * HD + 8 + g], ll); }
            }
        }
        if (!whole) {
            // ---- arrival: the last CTA holding a piece of unit u merges all pieces
            const int c_lo = pf[u] / per, c_hi = (pf[u + 1] - 1) / per;
            __threadfence();
            consumer_sync();
            if (ctid == 0) {
                const int old = atomicAdd(&t.unit_arrive[u], 1);
                s_flag[1] = (old == c_hi - c_lo) ? 1 : 0;
                if (old == c_hi - c_lo) t.unit_arrive[u] = 0;
            }
            consumer_sync();
            if (s_flag[1]) {
                __threadfence();
                // every thread merges up to three float4 columns (one head each); a unit is rarely cut into more than
                // four pieces, and then ALL loads of the thread -- every column, every piece -- are issued before the first
                // use, so the merge costs one trip to memory
                constexpr int NC = (MAX_G * HD / 4 + AT_CONSUMERS * 32 - 1) / (AT_CONSUMERS * 32);
                const int ncols = G * HD / 4;
                if (c_hi - c_lo < 4) {
                    float mv[NC][4], lv[NC][4]; float4 pv[NC][4];
#pragma unroll
                    for (int x = 0; x < NC; x++) {
                        const int i4 = ctid + x * AT_CONSUMERS * 32;
                        const int g = (i4 * 4) / HD;
#pragma unroll
                        for (int j = 0; j < 4; j++) {
                            const int cc = c_lo + j;
                            mv[x][j] = -INFINITY; lv[x][j] = 0.f; pv[x][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (i4 < ncols && cc <= c_hi) {
                                const int slot = (cc == c_lo && cc * per != pf[u]) ? 1 : 0;
                                const float* ps = t.part + (size_t)(2 * cc + slot) * rec_floats;
                                mv[x][j] = __ldcg(ps + G * HD + g); lv[x][j] = __ldcg(ps + G * HD + 8 + g);
                                pv[x][j] = __ldcg(reinterpret_cast<const float4*>(ps) + i4);
                            }
                        }
                    }
#pragma unroll
                    for (int x = 0; x < NC; x++) {
                        const int i4 = ctid + x * AT_CONSUMERS * 32;
                        if (i4 >= ncols) continue;
                        const float mm = fmaxf(fmaxf(mv[x][0], mv[x][1]), fmaxf(mv[x][2], mv[x][3]));
                        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                        float ll = 0.f;
                        if (mm != -INFINITY) {
#pragma unroll
                            for (int j = 0; j < 4; j++) {
                                const float f = mv[x][j] == -INFINITY ? 0.f : exp2f(mv[x][j] - mm);
                                a.x += pv[x][j].x * f; a.y += pv[x][j].y * f; a.z += pv[x][j].z * f; a.w += pv[x][j].w * f;
                                ll += lv[x][j] * f;
                            }
                        }
                        const float inv = ll > 0.f ? 1.f / ll : 0.f;
                        reinterpret_cast<float4*>(out + (size_t)u * G * HD)[i4] = make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
                    }
                } else
                for (int i4 = ctid; i4 < ncols; i4 += AT_CONSUMERS * 32) {
                    const int g = (i4 * 4) / HD;
                    float mm = -INFINITY, ll = 0.f;
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int cc0 = c_lo; cc0 <= c_hi; cc0 += 4) {
                        float mv[4], lv[4]; float4 pv[4];
#pragma unroll
                        for (int j = 0; j < 4; j++) {
                            const int cc = cc0 + j;
                            mv[j] = -INFINITY; lv[j] = 0.f; pv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (cc <= c_hi) {
                                const int slot = (cc == c_lo && cc * per != pf[u]) ? 1 : 0;
                                const float* ps = t.part + (size_t)(2 * cc + slot) * rec_floats;
                                mv[j] = __ldcg(ps + G * HD + g); lv[j] = __ldcg(ps + G * HD + 8 + g);
                                pv[j] = __ldcg(reinterpret_cast<const float4*>(ps) + i4);
                            }
                        }
                        const float mnew = fmaxf(fmaxf(mm, mv[0]), fmaxf(fmaxf(mv[1], mv[2]), mv[3]));
                        if (mnew != -INFINITY) {
                            const float f0 = mm == -INFINITY ? 0.f : exp2f(mm - mnew);
                            a.x *= f0; a.y *= f0; a.z *= f0; a.w *= f0; ll *= f0;
#pragma unroll
                            for (int j = 0; j < 4; j++) {
                                const float f = mv[j] == -INFINITY ? 0.f : exp2f(mv[j] - mnew);
                                a.x += pv[j].x * f; a.y += pv[j].y * f; a.z += pv[j].z * f; a.w += pv[j].w * f;
                                ll += lv[j] * f;
                            }
                            mm = mnew;
                        }
                    }
                    const float inv = ll > 0.f ? 1.f / ll : 0.f;
                    reinterpret_cast<float4*>(out + (size_t)u * G * HD)[i4] = make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
                }
            }
        }
        consumer_sync();     // merge scratch and s_flag[1] are free again
        k = seg_end;
    }
}

// Self-test of the bounded waits: one thread waits on an mbarrier that nobody ever arrives at, with a limit of a few
// thousand polls.  The wait must give up, the kernel raises the same status bit the production kernels raise on an
// expired wait, and returns normally; nothing faults, traps or spins on.
__global__ void k_selftest_wait_expiry(unsigned int* status, int* gave_up) {
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        const bool ok = mbar_wait(smem_u32(&bar), 0u, 4096);
        if (!ok) { atomicOr(status, DYNAKV_ST_INTERNAL); *gave_up = 1; }
    }
}

void launch_selftest_wait_expiry(const Tables& t, int* gave_up, cudaStream_t s, long long* launches) {
    k_selftest_wait_expiry<<<1, 32, 0, s>>>(t.status, gave_up);
    (*launches)++;
}

size_t attn_tma_smem_bytes(const Tables& t) {
    const size_t fixed = t.fp8 ? AttnSmem<128, true>::fixed_bytes : t.d == 64 ? AttnSmem<64, false>::fixed_bytes : AttnSmem<128, false>::fixed_bytes;
    return fixed + (t.attn_pf_in_smem ? (size_t)(t.U + 1) * 4 : 0) + 64;
}

int attn_tma_prepare(const Tables& t) {
    const int bytes = (int)attn_tma_smem_bytes(t);
    cudaError_t e = t.fp8 ? cudaFuncSetAttribute(k_gather_attn_tma<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)
        : t.d == 64 ? cudaFuncSetAttribute(k_gather_attn_tma<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)
        : cudaFuncSetAttribute(k_gather_attn_tma<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e == cudaSuccess ? 0 : -1;
}

// The same kernel as an ordinary launch (no programmatic dependence on its neighbours): for timing it alone.
void launch_gather_attn_plain(const Tables& t, StepPtr q, StepPtrW out, cudaStream_t s, long long* launches) {
    const size_t bytes = attn_tma_smem_bytes(t);
    if (t.fp8) k_gather_attn_tma<128, true><<<t.n_attn_ctas, AT_THREADS, bytes, s>>>(t, q, out);
    else if (t.d == 64) k_gather_attn_tma<64, false><<<t.n_attn_ctas, AT_THREADS, bytes, s>>>(t, q, out);
    else k_gather_attn_tma<128, false><<<t.n_attn_ctas, AT_THREADS, bytes, s>>>(t, q, out);
    (*launches)++;
}

void launch_gather_attn_tma(const Tables& t, StepPtr q, StepPtrW out, cudaStream_t s, long long* launches) {
    const size_t bytes = attn_tma_smem_bytes(t);
    if (t.fp8) launch_pdl(k_gather_attn_tma<128, true>, dim3(t.n_attn_ctas), dim3(AT_THREADS), bytes, s, t, q, out);
    else if (t.d == 64) launch_pdl(k_gather_attn_tma<64, false>, dim3(t.n_attn_ctas), dim3(AT_THREADS), bytes, s, t, q, out);
    else launch_pdl(k_gather_attn_tma<128, false>, dim3(t.n_attn_ctas), dim3(AT_THREADS), bytes, s, t, q, out);
    (*launches)++;
}

}  // namespace dkv
