// Nearest-centre assignment of the k-means rounds as a tensor-core distance GEMM fused with
// argmin (arXiv 2511.07427, Section 4.1: the k-means partition of Eq. 3; NewCluster of
// Algorithm 1), for bf16 keys with d = 128.
//
//   a_i = argmin_j ||k_i - c_j||^2 = argmin_j ( ||c_j||^2 - 2 k_i . c_j )
//
// Filter + exact re-decision.  The [n x M] matrix of k_i . c_j is a dense contraction: it runs
// on the 5th-generation tensor cores (tcgen05.mma, kind::f16, fp32 accumulators in TMEM) with the
// keys converted to fp16 (exact for |k| in [2^-14, 65504], which a pre-pass checks) and the fp32
// centres rounded to fp16.  Rounding the centres perturbs every value by at most
// E_i = 2 ||k_i|| max_j||c_j|| 2^-11 (plus accumulation and fixed-point slack), so the tensor-core
// result is used as a FILTER: the epilogue keeps, per key, the three smallest values; when the
// second is further than 2 E_i from the first, the first is provably the true argmin.  Otherwise
// the key is re-decided exactly in fp32 with the direct form sum (k - c)^2, the same arithmetic
// as the plain fp32 assignment kernel: between the best two centres when the third value is out
// of reach, over all centres when it is not.  The [n x M] matrix never
// leaves the chip.
//
// Kernel shape.  Persistent CTAs, one per SM, each looping over (unit, 128-key block) items.
// Warp 0 issues TMA tensor loads (128-byte swizzle, every CTA loads for itself) of the key block (kept for
// all centre tiles of the item) and of 256-centre tiles into a two-stage ring; warp 1 issues
// tcgen05.mma (M=128, N=256, K=16, eight per tile) into one of two 256-column TMEM accumulators
// and commits to an mbarrier; warps 2-17 drain the accumulators with tcgen05.ld, one key per
// thread (four groups of four warps: two per accumulator, half of its columns each).  Every wait
// is bounded; on expiry the kernel sets a status bit, frees its TMEM and returns.
#include <cuda.h>
#include <float.h>

#include <cuda_fp16.h>

#include "common.cuh"

namespace dkv {

// ------------------------------------------------------------------ small PTX wrappers

__device__ __forceinline__ unsigned tc_smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void tc_mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
// One poll; the thread is suspended in hardware until the phase completes or about `hint_ns` have passed, so
// a waiting role does not compete for issue slots with the warps that drain the accumulators.
__device__ __forceinline__ bool tc_mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    const unsigned hint_ns = 20000u;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long tc_global_ns() {
    unsigned long long v;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(v));
    return v;
}
// Bounded wait: 2^22 polls or about 0.5 s.
__device__ __forceinline__ bool tc_mbar_wait(unsigned bar, unsigned parity) {
    unsigned long long t0 = 0;
    for (int i = 0; i < (1 << 22); i++) {
        if (tc_mbar_try_wait(bar, parity)) return true;
        if ((i & 63) == 63) {
            const unsigned long long now = tc_global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > 500000000ull) return false;
        }
    }
    return false;
}
// 2-D tiled TMA load (inner coordinate x in elements, outer coordinate y in rows); every CTA loads for itself.
__device__ __forceinline__ void tc_tma_load_2d(unsigned dst, const CUtensorMap* map, int x, int y, unsigned bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
// D[tmem] (+)= A[smem desc] * B[smem desc]; accumulate = 0 overwrites D.
__device__ __forceinline__ void tc_mma_f16(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                           unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrive once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld32(unsigned taddr, unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }

// ------------------------------------------------------------------ tiles, descriptors

constexpr int TC_D = 128;                 // head dimension = contraction length
constexpr int TC_BM = 128;                // keys per item (one TMEM lane each)
#ifndef DKV_TC_BN
#define DKV_TC_BN 256
#endif
constexpr int TC_BN = DKV_TC_BN;          // centres per accumulator: 256 (two accumulators) or 128 (four)
constexpr int TC_NACC = 512 / TC_BN;      // accumulators in the 512 columns of tensor memory
constexpr int TC_NB = (2 * 256) / TC_BN;  // centre-tile stages (128 KB of shared memory in all)
constexpr int TC_A_BYTES = TC_BM * TC_D * 2;          // 32 KB: two [128 rows x 128 B] swizzle panels
constexpr int TC_B_BYTES = TC_BN * TC_D * 2;          // 64 KB or 32 KB: two [TC_BN rows x 128 B] swizzle panels
constexpr int TC_XCHG_BYTES = 2 * 3 * TC_BM * 5 * 4;      // hand-over of (g1, g2, g3, j1, j2) between the drain groups
constexpr int TC_SMEM_BYTES = 2 * TC_A_BYTES + TC_NB * TC_B_BYTES + 1024 /* alignment */ + 256 /* barriers */ + TC_XCHG_BYTES;
#ifndef DKV_TC_GROUPS
#define DKV_TC_GROUPS 4
#endif
constexpr int TC_GROUPS = DKV_TC_GROUPS;  // drain groups of four warps: 2 (one per accumulator) or 4 (two per accumulator, half the columns each)
constexpr int TC_THREADS = 64 + 128 * TC_GROUPS;   // warp 0 loads, warp 1 issues MMAs, the rest drain the accumulators
constexpr unsigned TC_TMEM_COLS = 512;    // TC_NACC fp32 accumulators of TC_BN columns
// mbarriers: key block full / empty (2 each), centre stage full / empty (TC_NB each), accumulator full / empty
constexpr int BAR_AF = 0, BAR_AE = 2, BAR_BF = 4, BAR_BE = 4 + TC_NB, BAR_CF = 4 + 2 * TC_NB, BAR_CE = BAR_CF + TC_NACC,
              BAR_COUNT = BAR_CE + TC_NACC;
static_assert((BAR_COUNT + 2) * 8 <= 256, "barrier block");

// Shared-memory matrix descriptor of a K-major panel with 128-byte rows under the 128-byte swizzle:
// start address / 16, leading offset unused (1), 1024 B between 8-row groups, descriptor version 1,
// layout type 2 (128-byte swizzle).
__device__ __forceinline__ unsigned long long tc_panel_desc(unsigned smem_addr) {
    return (unsigned long long)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((unsigned long long)(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulate, fp16 A and B, both K-major, M = 128, N = 256.
constexpr unsigned TC_IDESC = (1u << 4) | ((unsigned)(TC_BN >> 3) << 17) | ((unsigned)(TC_BM >> 4) << 24);

// ------------------------------------------------------------------ pre-passes

// Keys bf16 -> fp16 (exact unless |k| > 65504, which raises *bad; values below 2^-24 lose bits, which
// the margin covers) and ||k_i|| in fp32.  One warp per key.
__global__ void __launch_bounds__(256) k_tc_prep_keys(const __nv_bfloat16* __restrict__ K, long long rows, int n,
                                                      __half* __restrict__ A16, float* __restrict__ knorm,
                                                      unsigned* __restrict__ knmax_bits, int* __restrict__ bad) {
    const int lane = threadIdx.x & 31;
    const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nw = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long per = (rows + nw - 1) / nw;          // a contiguous run of keys per warp: few unit changes
    long long cur_u = -1;
    float cur_max = 0.f;
    for (long long w = wid * per; w < min(rows, (wid + 1) * per); w++) {
        const float4 v = ld4(K + (size_t)w * TC_D, lane * 4);
        const float m = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
        if (!(m <= 65504.f)) atomicOr(bad, 1);
        __half2 h0 = __floats2half2_rn(v.x, v.y), h1 = __floats2half2_rn(v.z, v.w);
        uint2 pk;
        pk.x = *reinterpret_cast<unsigned*>(&h0); pk.y = *reinterpret_cast<unsigned*>(&h1);
        *reinterpret_cast<uint2*>(A16 + (size_t)w * TC_D + lane * 4) = pk;
        float s = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        s = warp_sum(s);
        const float kn = sqrtf(s);
        if (lane == 0) knorm[w] = kn;
        const long long uu = w / n;
        if (uu != cur_u) {
            if (lane == 0 && cur_u >= 0) atomicMax(&knmax_bits[cur_u], __float_as_uint(cur_max));
            cur_u = uu; cur_max = 0.f;
        }
        cur_max = fmaxf(cur_max, kn);
    }
    if (lane == 0 && cur_u >= 0) atomicMax(&knmax_bits[cur_u], __float_as_uint(cur_max));   // largest key norm of the unit
}

// Centres fp32 -> fp16 into a copy padded to Mpad rows per unit (padding rows are zero, so their dot products
// are exactly zero), bias_j = ||c_j||^2 in fp32 of the unrounded centre, cmax[u] = max_j ||c_j||.
// One warp per (unit, padded centre index).
__global__ void __launch_bounds__(256) k_tc_prep_centres(const float* __restrict__ C, int U, int M, int Mpad,
                                                         __half* __restrict__ B16, float* __restrict__ bias,
                                                         unsigned* __restrict__ cmax_bits, int* __restrict__ bad) {
    const int lane = threadIdx.x & 31;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    // a grid that loops over the rows: a warp per row would be a quarter of a million warps of a dozen instructions
    for (long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < (long long)U * Mpad; w += nwarps) {
    const int u = (int)(w / Mpad), j = (int)(w % Mpad);
    if (j >= M) {
        *reinterpret_cast<uint2*>(B16 + (size_t)w * TC_D + lane * 4) = make_uint2(0u, 0u);
        if (lane == 0) bias[w] = 0.f;
        continue;
    }
    const size_t row = (size_t)u * M + j;
    const float4 v = *reinterpret_cast<const float4*>(C + row * TC_D + lane * 4);
    const float m = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
    if (!(m <= 65504.f)) atomicOr(bad, 1);
    __half2 h0 = __floats2half2_rn(v.x, v.y), h1 = __floats2half2_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<unsigned*>(&h0); pk.y = *reinterpret_cast<unsigned*>(&h1);
    *reinterpret_cast<uint2*>(B16 + (size_t)w * TC_D + lane * 4) = pk;
    float s = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    s = warp_sum(s);
    if (lane == 0) {
        bias[w] = s;
        atomicMax(&cmax_bits[u], __float_as_uint(sqrtf(s)));     // non-negative floats order like their bit patterns
    }
    }
}

// Fixed-point form of the filter values.  With S_u a power of two such that |x| S_u <= 2^29 for every value
// x = ||c_j||^2 - 2 k.c_j of the unit, the single fma  v = acc * (-2 S_u) + B_j,  B_j = 1.5 * 2^31 + bias_j S_u,
// lands in [2^31, 2^32), where floats are 256 apart: the 23 mantissa bits of v ARE the value on a grid of
// g_u = 256 / S_u (offset 2^22), already rounded, and one integer multiply-add  bits(v) * 256 + column  (the
// exponent falls off the top) makes a word whose low 8 bits are free for the column and which still orders like
// the value when compared as a positive float.  Padding columns get the largest mantissa in use.
// scale[u] = (S_u, g_u); one thread per (unit, padded column).
constexpr float TC_MAGIC = 3221225472.f;                 // 1.5 * 2^31
constexpr unsigned TC_PAD_MANT = 0x700000u;              // above 2^22 + 2^21, below the NaN patterns after the shift
__global__ void __launch_bounds__(256) k_tc_fixed_bias(const float* __restrict__ bias, const unsigned* __restrict__ cmax_bits,
                                                       const unsigned* __restrict__ knmax_bits, int U, int M, int Mpad,
                                                       float* __restrict__ Bfix, float2* __restrict__ scale) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)U * Mpad) return;
    const int u = (int)(idx / Mpad), j = (int)(idx % Mpad);
    const float cm = __uint_as_float(cmax_bits[u]), kn = __uint_as_float(knmax_bits[u]);
    const float xmax = fmaxf(cm * cm + 2.f * kn * cm, 1e-30f);
    int e = (int)floorf(log2f(536870912.f / xmax));      // 2^29 / xmax
    e = max(-100, min(100, e));
    const float S = exp2f((float)e);
    if (j == 0) scale[u] = make_float2(S, 256.f / S);
    Bfix[idx] = j < M ? TC_MAGIC + bias[idx] * S : __uint_as_float(0x4F000000u | TC_PAD_MANT);   // 2^31 * (1 + mant / 2^23)
}

// ------------------------------------------------------------------ the distance GEMM + top-3 filter

__device__ __forceinline__ float tc_min3(float a, float b, float c) {
    float r;
    asm("min.f32 %0, %1, %2, %3;\n" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// Fixed-point filter word: bits(v) * 256 + column tag (see k_tc_fixed_bias), as a positive float for min/max.  The
// multiply-add is written in PTX, with the factor 256 in a register the compiler knows nothing about (a kernel
// argument) and the tag as a compile-time constant, so that it stays ONE integer multiply-add on the FMA pipe:
// a known power of two turns it into shift-and-add on the ALU pipe, which the min/max chains keep busy.
__device__ __forceinline__ float tc_pack(float v, unsigned mul256, int tag) {
    unsigned r;
    asm("mad.lo.u32 %0, %1, %2, %3;\n" : "=r"(r) : "r"(__float_as_uint(v)), "r"(mul256), "r"((unsigned)tag));
    return __uint_as_float(r);
}
// (t1 <= t2 <= t3) <- the three smallest of {t1, t2, t3, x, y}.
__device__ __forceinline__ void tc_top3_pair(float& t1, float& t2, float& t3, float x, float y) {
    const float lo = fminf(x, y), hi = fmaxf(x, y);
    t3 = tc_min3(t3, fmaxf(t2, lo), fmaxf(t1, hi));
    t2 = tc_min3(fmaxf(t1, lo), t2, hi);
    t1 = fminf(t1, lo);
}
// a <- the three smallest of the sorted triples a and c.
__device__ __forceinline__ void tc_merge3(float (&a)[3], const float (&c)[3]) {
    const float t1 = fminf(a[0], c[0]);
    const float t2 = tc_min3(fmaxf(a[0], c[0]), a[1], c[1]);
    const float t3 = fminf(tc_min3(a[2], c[2], fmaxf(a[1], c[0])), fmaxf(a[0], c[1]));
    a[0] = t1; a[1] = t2; a[2] = t3;
}
// Insert (v, j) into the sorted best two (with indices) and third value.
__device__ __forceinline__ void tc_insert(float& g1, int& j1, float& g2, int& j2, float& g3, float v, int j) {
    if (v < g1) { g3 = g2; g2 = g1; j2 = j1; g1 = v; j1 = j; }
    else if (v < g2) { g3 = g2; g2 = v; j2 = j; }
    else if (v < g3) g3 = v;
}

struct TcArgs {
    int U, n, M, Mpad, KB;               // KB = 128-key blocks per unit
    unsigned tag_mul;                    // 256, handed over as data: see tc_pack
    const float* Bfix;                   // [U][Mpad] fixed-point bias 1.5 * 2^31 + ||c_j||^2 S_u
    const float2* scale;                 // [U] (S_u, g_u = 256 / S_u)
    const float* knorm;                  // [U * n]
    const unsigned* cmax_bits;           // [U]
    int* assign;                         // [U * n]
    int* recheck_list;                   // [U][n] key indices (inside the unit) to re-decide exactly
    unsigned* recheck_count;             // [U]
    int2* pair_list;                     // [U * n] (global key row, j1 | j2 << 16): decide exactly between two centres
    unsigned long long* pair_count;      // [1]
    unsigned int* status;
};

__global__ void __launch_bounds__(TC_THREADS, 1) k_tc_assign(const __grid_constant__ CUtensorMap mapA,
                                                             const __grid_constant__ CUtensorMap mapB, TcArgs p) {
    extern __shared__ unsigned char tc_smem_raw[];
    const unsigned raw = tc_smem_u32(tc_smem_raw);
    const unsigned base = (raw + 1023u) & ~1023u;                    // swizzle panels need 1024-byte alignment
    unsigned char* gen = tc_smem_raw + (base - raw);
    const unsigned sA = base, sB = base + 2 * TC_A_BYTES;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(gen + 2 * TC_A_BYTES + TC_NB * TC_B_BYTES);
    auto bar = [&](int i) { return tc_smem_u32(&bars[i]); };
    volatile unsigned* s_tmem = reinterpret_cast<volatile unsigned*>(&bars[BAR_COUNT]);
    volatile int* s_abort = reinterpret_cast<volatile int*>(&bars[BAR_COUNT + 1]);
    float* xchg = reinterpret_cast<float*>(gen + 2 * TC_A_BYTES + TC_NB * TC_B_BYTES + 256);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NT = p.Mpad / TC_BN;
    const long long n_items = (long long)p.U * p.KB;

    if (tid == 0) {
        for (int i = 0; i < BAR_CE; i++) tc_mbar_init(bar(i), 1);
        for (int i = 0; i < TC_NACC; i++) tc_mbar_init(bar(BAR_CE + i), 2 * TC_GROUPS);   // one arrival per draining warp of the accumulator
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                     ::"r"(tc_smem_u32((const void*)s_tmem)), "r"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = *s_tmem;

    if (warp == 0) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            long long ia = 0, tb = 0;
            long long lastA[2] = {-1, -1}, lastB[TC_NB];
            for (int i = 0; i < TC_NB; i++) lastB[i] = -1;
            for (long long it = blockIdx.x; it < n_items && !*s_abort; it += gridDim.x, ia++) {
                const int u = (int)(it / p.KB), kb = (int)(it % p.KB);
                const int ab = (int)(ia & 1);
                if (!tc_mbar_wait(bar(BAR_AE + ab), (unsigned)((ia >> 1) & 1) ^ 1u)) { *s_abort = 1; break; }
                tc_mbar_expect_tx(bar(BAR_AF + ab), TC_A_BYTES);
                const int rowA = u * p.n + kb * TC_BM;
                tc_tma_load_2d(sA + ab * TC_A_BYTES, &mapA, 0, rowA, bar(BAR_AF + ab));
                tc_tma_load_2d(sA + ab * TC_A_BYTES + TC_A_BYTES / 2, &mapA, 64, rowA, bar(BAR_AF + ab));
                lastA[ab] = ia;
                for (int nt = 0; nt < NT; nt++, tb++) {
                    const int st = (int)(tb % TC_NB);
                    if (!tc_mbar_wait(bar(BAR_BE + st), (unsigned)((tb / TC_NB) & 1) ^ 1u)) { *s_abort = 1; break; }
                    tc_mbar_expect_tx(bar(BAR_BF + st), TC_B_BYTES);
                    const int rowB = u * p.Mpad + nt * TC_BN;
                    tc_tma_load_2d(sB + st * TC_B_BYTES, &mapB, 0, rowB, bar(BAR_BF + st));
                    tc_tma_load_2d(sB + st * TC_B_BYTES + TC_B_BYTES / 2, &mapB, 64, rowB, bar(BAR_BF + st));
                    lastB[st] = tb;
                }
            }
            if (*s_abort) {
                // let the copies already issued land before the shared memory can be reused
                for (int i = 0; i < 2; i++)
                    if (lastA[i] >= 0) tc_mbar_wait(bar(BAR_AF + i), (unsigned)((lastA[i] >> 1) & 1));
                for (int i = 0; i < TC_NB; i++)
                    if (lastB[i] >= 0) tc_mbar_wait(bar(BAR_BF + i), (unsigned)((lastB[i] / TC_NB) & 1));
            }
        }
    } else if (warp == 1) {
        // =============================== MMA issuer ===============================
        if (lane == 0) {
            long long ia = 0, tb = 0;
            for (long long it = blockIdx.x; it < n_items && !*s_abort; it += gridDim.x, ia++) {
                const int ab = (int)(ia & 1);
                if (!tc_mbar_wait(bar(BAR_AF + ab), (unsigned)((ia >> 1) & 1))) { *s_abort = 1; break; }
                for (int nt = 0; nt < NT; nt++, tb++) {
                    const int st = (int)(tb % TC_NB), ac = (int)(tb % TC_NACC);
                    if (!tc_mbar_wait(bar(BAR_BF + st), (unsigned)((tb / TC_NB) & 1)) ||
                        !tc_mbar_wait(bar(BAR_CE + ac), (unsigned)((tb / TC_NACC) & 1) ^ 1u)) { *s_abort = 1; break; }
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < TC_D / 16; k++) {
                        const unsigned a_addr = sA + ab * TC_A_BYTES + (k >> 2) * (TC_A_BYTES / 2) + (k & 3) * 32;
                        const unsigned b_addr = sB + st * TC_B_BYTES + (k >> 2) * (TC_B_BYTES / 2) + (k & 3) * 32;
                        tc_mma_f16(tmem + ac * TC_BN, tc_panel_desc(a_addr), tc_panel_desc(b_addr), TC_IDESC, k > 0 ? 1u : 0u);
                    }
                    tc_commit(bar(BAR_BE + st));  // centre tile may be overwritten
                    tc_commit(bar(BAR_CF + ac));  // accumulator is complete
                }
                if (*s_abort) break;
                tc_commit(bar(BAR_AE + ab));      // key block may be overwritten
            }
        }
    } else {
        // =============================== accumulator drain (warps 2 and up) ===============================
        // Groups of four warps (one warp per TMEM lane quarter).  Group g drains accumulator g mod 2, i.e. the
        // tiles whose running number is g mod 2, and of those the column range g / 2, so both accumulators are
        // drained at the same time while the next MMAs run.  One key per thread and group.  Per tile the thread
        // keeps the three smallest fixed-point words (low 8 bits = column) in four independent chains and merges
        // them into its best two (with indices) and third value; at the end of an item the other groups hand
        // their triples to group 0 through shared memory, and group 0 decides.
        const int grp = (warp - 2) >> 2;              // drain group
        const int team = grp & 1;                     // tiles of this parity are this group's (accumulators team, team + 2, ...)
        constexpr int CPG = (TC_BN / 32) / (TC_GROUPS / 2);   // 32-column chunks per group and tile
        const int c_first = (grp >> 1) * CPG;         // first chunk of this group's column range
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;                // key of this thread inside the item
        long long tb = 0, item_no = 0;
        for (long long it = blockIdx.x; it < n_items; it += gridDim.x, item_no++) {
            const int u = (int)(it / p.KB), kb = (int)(it % p.KB);
            const int i = kb * TC_BM + row;
            float g1 = INFINITY, g2 = INFINITY, g3 = INFINITY;
            int j1 = 0, j2 = 0;
            bool dead = false;
            const float2 sc = p.scale[u];
            const float m2S = -2.f * sc.x;
            const unsigned mul256 = p.tag_mul;
            for (int nt = 0; nt < NT; nt++, tb++) {
                if ((int)(tb & 1) != team) continue;
                const int st = (int)(tb % TC_NACC);
                if (*s_abort || !tc_mbar_wait(bar(BAR_CF + st), (unsigned)((tb / TC_NACC) & 1))) { *s_abort = 1; dead = true; break; }
                tc_fence_after();
                float ch[4][3];                                        // four independent chains of three smallest
#pragma unroll
                for (int x = 0; x < 4; x++) { ch[x][0] = INFINITY; ch[x][1] = INFINITY; ch[x][2] = INFINITY; }
                const float4* bias4 = reinterpret_cast<const float4*>(p.Bfix + (size_t)u * p.Mpad + (size_t)nt * TC_BN);
                const unsigned tbase = tmem + st * TC_BN + ((unsigned)(q * 32) << 16);
                unsigned acc[2][32];
                float bs[2][32];
                auto load_bias = [&](int c, float (&dst)[32]) {
#pragma unroll
                    for (int e = 0; e < 8; e++) {
                        const float4 v = __ldg(bias4 + c * 8 + e);
                        dst[4 * e] = v.x; dst[4 * e + 1] = v.y; dst[4 * e + 2] = v.z; dst[4 * e + 3] = v.w;
                    }
                };
                tc_ld32(tbase + c_first * 32, acc[0]);
                load_bias(c_first, bs[0]);
#pragma unroll
                for (int cc = 0; cc < CPG; cc++) {
                    const int c = c_first + cc;
                    tc_ld_wait();                                           // chunk c has arrived
                    if (cc + 1 < CPG) {                                     // chunk c + 1 and its bias in flight
                        tc_ld32(tbase + (c + 1) * 32, acc[(cc + 1) & 1]);
                        load_bias(c + 1, bs[(cc + 1) & 1]);
                    }
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
#pragma unroll
                        for (int x = 0; x < 4; x++) {
                            const int e0 = e + 2 * x;
                            // the tag is the column inside this group's range: a compile-time constant per element
                            const float x0 = tc_pack(fmaf(__uint_as_float(acc[cc & 1][e0]), m2S, bs[cc & 1][e0]), mul256, cc * 32 + e0);
                            const float x1 = tc_pack(fmaf(__uint_as_float(acc[cc & 1][e0 + 1]), m2S, bs[cc & 1][e0 + 1]), mul256, cc * 32 + e0 + 1);
                            tc_top3_pair(ch[x][0], ch[x][1], ch[x][2], x0, x1);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) tc_mbar_arrive(bar(BAR_CE + st));      // accumulator may be overwritten
                // the tile's three smallest out of the four chains
                tc_merge3(ch[0], ch[1]);
                tc_merge3(ch[2], ch[3]);
                tc_merge3(ch[0], ch[2]);
                const float t1 = ch[0][0], t2 = ch[0][1], t3 = ch[0][2];
                const int col0 = nt * TC_BN + c_first * 32;
                tc_insert(g1, j1, g2, j2, g3, t1, col0 + (int)(__float_as_uint(t1) & 0xFFu));
                tc_insert(g1, j1, g2, j2, g3, t2, col0 + (int)(__float_as_uint(t2) & 0xFFu));
                tc_insert(g1, j1, g2, j2, g3, t3, col0 + (int)(__float_as_uint(t3) & 0xFFu));
            }
            // ---- hand-over: group 1 -> group 0 (slot alternates per item; the barrier orders write, read and reuse)
            float* slots = xchg + (size_t)(item_no & 1) * 3 * TC_BM * 5 + row * 5;     // [3 groups][128 keys][5]
            if (grp > 0) {
                float* slot = slots + (size_t)(grp - 1) * TC_BM * 5;
                slot[0] = g1; slot[1] = g2; slot[2] = g3; slot[3] = __int_as_float(j1); slot[4] = __int_as_float(j2);
            }
            asm volatile("bar.sync 2, %0;\n" ::"n"(128 * TC_GROUPS) : "memory");
            if (dead || *s_abort) break;
            if (grp == 0) {
#pragma unroll
                for (int g = 0; g < TC_GROUPS - 1; g++) {
                    const float* slot = slots + (size_t)g * TC_BM * 5;
                    tc_insert(g1, j1, g2, j2, g3, slot[0], __float_as_int(slot[3]));
                    tc_insert(g1, j1, g2, j2, g3, slot[1], __float_as_int(slot[4]));
                    tc_insert(g1, j1, g2, j2, g3, slot[2], 0);
                }
            }
            if (grp == 0 && i < p.n) {
                const size_t gi = (size_t)u * p.n + i;
                if (j1 >= p.M) j1 = 0;
                p.assign[gi] = j1;
                const float kn = p.knorm[gi], cm = __uint_as_float(p.cmax_bits[u]);
                // Bound on |filter value - true value|, term by term:
                //   fp16 rounding of the centres: 2 |k.(c - c16)| <= 2 kn cm 2^-11 = kn cm 2^-10;
                //   fp32 accumulation of 128 exact products in the tensor core, doubled by the factor -2: below
                //   kn cm 2^-15, covered with margin by the 10 % slack on the first term;
                //   sub-normal fp16 elements of keys and centres (absolute error 2^-25 each, 128 of them): (kn + cm) 1e-6;
                //   fp32 rounding of ||c||^2: cm^2 5e-7;  the two roundings to the fixed-point grid: 2 g.
                const float E = kn * cm * (1.10f / 1024.f) + 2.f * sc.y + (kn + cm) * 1e-6f + cm * cm * 5e-7f;
                // gaps in value units: mantissa differences times the grid
                const unsigned m1 = __float_as_uint(g1) >> 8, m2 = __float_as_uint(g2) >> 8, m3 = __float_as_uint(g3) >> 8;
                const float gap2 = (float)(m2 - m1) * sc.y, gap3 = (float)(m3 - m1) * sc.y;
                if (!(gap2 > 2.f * E)) {
                    if (gap3 > 2.f * E && j2 < p.M) {
                        // only the best two can be the true argmin: decide between them exactly
                        const unsigned long long pos = atomicAdd(p.pair_count, 1ull);
                        p.pair_list[pos] = make_int2((int)gi, j1 | (j2 << 16));
                    } else {
                        const unsigned pos = atomicAdd(&p.recheck_count[u], 1u);
                        p.recheck_list[(size_t)u * p.n + pos] = i;
                    }
                }
            }
        }
    }
    // ---- everyone meets here, on every path; then the allocating warp frees the tensor memory
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(TC_TMEM_COLS) : "memory");
    }
    if (tid == 0 && *s_abort) atomicOr(p.status, DYNAKV_ST_INTERNAL);
}

// Exact decision between two centres for the keys whose third-best filter value is out of reach: squared
// distances by the direct form, summed in index order in fp32 like the plain assignment kernel; ties to the
// lower id.  One thread per listed key.
__global__ void __launch_bounds__(256) k_tc_pair_decide(const __nv_bfloat16* __restrict__ K, const float* __restrict__ C, int n, int M,
                                                        const int2* __restrict__ list, const unsigned long long* __restrict__ count,
                                                        int* __restrict__ assign, unsigned long long* __restrict__ rechecked_total) {
    const unsigned long long idx = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long cnt = *count;
    if (idx == 0 && cnt) atomicAdd(rechecked_total, cnt);
    if (idx >= cnt) return;
    const int2 ent = list[idx];
    const int j1 = ent.y & 0xFFFF, j2 = (ent.y >> 16) & 0xFFFF;
    const int u = ent.x / n;
    const __nv_bfloat16* k = K + (size_t)ent.x * TC_D;
    const float* ca = C + ((size_t)u * M + j1) * TC_D;
    const float* cb = C + ((size_t)u * M + j2) * TC_D;
    float d1 = 0.f, d2 = 0.f;
#pragma unroll 4
    for (int e = 0; e < TC_D; e += 4) {
        const float4 kk = ld4(k, e);
        const float4 a = *reinterpret_cast<const float4*>(ca + e);
        const float4 b = *reinterpret_cast<const float4*>(cb + e);
        float df;
        df = kk.x - a.x; d1 = fmaf(df, df, d1); df = kk.y - a.y; d1 = fmaf(df, df, d1);
        df = kk.z - a.z; d1 = fmaf(df, df, d1); df = kk.w - a.w; d1 = fmaf(df, df, d1);
        df = kk.x - b.x; d2 = fmaf(df, df, d2); df = kk.y - b.y; d2 = fmaf(df, df, d2);
        df = kk.z - b.z; d2 = fmaf(df, df, d2); df = kk.w - b.w; d2 = fmaf(df, df, d2);
    }
    assign[ent.x] = (d2 < d1 || (d2 == d1 && j2 < j1)) ? j2 : j1;
}

// ------------------------------------------------------------------ host side

static size_t tc_align(size_t x) { return (x + 255) & ~(size_t)255; }

struct TcLayout {
    size_t a16, knorm, b16, bias, bfix, scale, cmax, knmax, bad, list, count, pairs, pair_count, total;
    int Mpad;
};
static TcLayout tc_layout(const Tables& t, long long n, int M) {
    TcLayout L;
    const size_t U = t.U;
    L.Mpad = (M + TC_BN - 1) / TC_BN * TC_BN;
    size_t off = 0;
    L.a16 = off; off += tc_align(U * (size_t)n * TC_D * 2);
    L.knorm = off; off += tc_align(U * (size_t)n * 4);
    L.b16 = off; off += tc_align(U * (size_t)L.Mpad * TC_D * 2);
    L.bias = off; off += tc_align(U * (size_t)L.Mpad * 4);
    L.bfix = off; off += tc_align(U * (size_t)L.Mpad * 4);
    L.scale = off; off += tc_align(U * 8);
    L.cmax = off; off += tc_align(U * 4);
    L.knmax = off; off += tc_align(U * 4);
    L.bad = off; off += 256;
    L.list = off; off += tc_align(U * (size_t)n * 4);
    L.count = off; off += tc_align(U * 4);
    L.pairs = off; off += tc_align(U * (size_t)n * 8);
    L.pair_count = off; off += 256;
    L.total = off;
    return L;
}

bool tc_assign_supported(const Tables& t, long long n, int M) {
    return t.kv_dtype == DYNAKV_BF16 && t.d == TC_D && M >= 1 && n >= 1 && (long long)t.U * n < (1ll << 31) &&
           (long long)t.U * (M + TC_BN) < (1ll << 31);
}

size_t tc_assign_scratch_bytes(const Tables& t, long long n, int M) { return tc_layout(t, n, M).total; }

// Once per build: fp16 copy of the keys and their norms.  Synchronises the stream to read the range flag;
// returns false (use the fp32 kernel) when a key does not fit fp16 or a CUDA call failed.
bool tc_assign_begin(const Tables& t, const void* K, long long n, int M, void* scratch, cudaStream_t s, long long* launches) {
    const TcLayout L = tc_layout(t, n, M);
    char* base = reinterpret_cast<char*>(scratch);
    int* bad = reinterpret_cast<int*>(base + L.bad);
    if (cudaMemsetAsync(bad, 0, 256, s) != cudaSuccess) return false;
    const long long rows = (long long)t.U * n;
    long long blocks = (rows + 7) / 8;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    if (cudaMemsetAsync(base + L.knmax, 0, (size_t)t.U * 4, s) != cudaSuccess) return false;
    k_tc_prep_keys<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(K), rows, (int)n,
                                                   reinterpret_cast<__half*>(base + L.a16),
                                                   reinterpret_cast<float*>(base + L.knorm),
                                                   reinterpret_cast<unsigned*>(base + L.knmax), bad);
    (*launches)++;
    int h_bad = 1;
    if (cudaMemcpyAsync(&h_bad, bad, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return false;
    if (cudaStreamSynchronize(s) != cudaSuccess) return false;
    if (h_bad) return false;
    // the opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of the kernel
    static bool opted[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
    if (dev < 0 || dev >= 64 || !opted[dev]) {
        if (cudaFuncSetAttribute(k_tc_assign, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        if (dev >= 0 && dev < 64) opted[dev] = true;
    }
    return true;
}

// cuTensorMapEncodeTiled is looked up through the runtime, so the library carries no link-time dependency on
// the driver library and still loads on a machine without a GPU.
typedef CUresult (*tc_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static tc_encode_fn tc_encode_entry() {
    static tc_encode_fn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<tc_encode_fn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

static bool tc_make_map(CUtensorMap* map, void* ptr, unsigned long long rows, unsigned box_rows) {
    tc_encode_fn enc = tc_encode_entry();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)TC_D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)TC_D * 2};
    cuuint32_t box[2] = {64u, box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// One Lloyd round's assignment: centre pre-pass, distance GEMM + filter, exact re-decision of the listed keys.
void launch_assign_tc(const Tables& t, const void* K, long long n, int M, const float* C, int* assign, void* scratch,
                      cudaStream_t s, long long* launches) {
    const TcLayout L = tc_layout(t, n, M);
    char* base = reinterpret_cast<char*>(scratch);
    __half* A16 = reinterpret_cast<__half*>(base + L.a16);
    __half* B16 = reinterpret_cast<__half*>(base + L.b16);
    float* bias = reinterpret_cast<float*>(base + L.bias);
    unsigned* cmax = reinterpret_cast<unsigned*>(base + L.cmax);
    int* bad = reinterpret_cast<int*>(base + L.bad);
    int* list = reinterpret_cast<int*>(base + L.list);
    unsigned* count = reinterpret_cast<unsigned*>(base + L.count);
    cudaMemsetAsync(cmax, 0, (size_t)t.U * 4, s);
    cudaMemsetAsync(count, 0, (size_t)t.U * 4, s);
    int2* pairs = reinterpret_cast<int2*>(base + L.pairs);
    unsigned long long* pair_count = reinterpret_cast<unsigned long long*>(base + L.pair_count);
    cudaMemsetAsync(pair_count, 0, 8, s);
    const long long cw = (long long)t.U * L.Mpad;
    {
        long long pb = (cw + 7) / 8;
        if (pb > 148LL * 16) pb = 148LL * 16;
        k_tc_prep_centres<<<(unsigned)pb, 256, 0, s>>>(C, t.U, M, L.Mpad, B16, bias, cmax, bad);
    }
    float* Bfix = reinterpret_cast<float*>(base + L.bfix);
    float2* scale = reinterpret_cast<float2*>(base + L.scale);
    k_tc_fixed_bias<<<(unsigned)((cw + 255) / 256), 256, 0, s>>>(bias, cmax, reinterpret_cast<const unsigned*>(base + L.knmax), t.U, M,
                                                                 L.Mpad, Bfix, scale);
    CUtensorMap mapA, mapB;
    if (!tc_make_map(&mapA, A16, (unsigned long long)t.U * n, TC_BM) || !tc_make_map(&mapB, B16, (unsigned long long)t.U * L.Mpad, TC_BN)) {
        // cannot describe the operands to the TMA unit: do the whole round exactly
        launch_assign_f32(t, K, n, M, C, assign, s, launches);
        return;
    }
    TcArgs a;
    a.U = t.U; a.n = (int)n; a.M = M; a.Mpad = L.Mpad; a.KB = (int)((n + TC_BM - 1) / TC_BM);
    a.tag_mul = 256u;
    a.Bfix = Bfix; a.scale = scale; a.knorm = reinterpret_cast<const float*>(base + L.knorm); a.cmax_bits = cmax;
    a.assign = assign; a.recheck_list = list; a.recheck_count = count; a.status = t.status;
    a.pair_list = pairs; a.pair_count = pair_count;
    const int grid = t.n_attn_ctas / 2;        // one persistent CTA per SM
    k_tc_assign<<<grid, TC_THREADS, TC_SMEM_BYTES, s>>>(mapA, mapB, a);
    const unsigned long long rows = (unsigned long long)t.U * n;
    k_tc_pair_decide<<<(unsigned)((rows + 255) / 256), 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(K), C, (int)n, M, pairs,
                                                                    pair_count, assign, &t.counters[CNT_RECHECKED]);
    (*launches) += 4;
    launch_assign_f32_listed(t, K, n, M, C, assign, list, count, &t.counters[CNT_RECHECKED], s, launches);
}

}  // namespace dkv
