// Shared declarations of libdynakv's kernels: the table of device arrays that holds one
// context's index and KV store, small device helpers, and the host launchers each .cu
// file exports to api.cu.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dynakv.h"

namespace dkv {

constexpr int PAGE = 32;            // tokens per page
#ifndef DKV_ENTRY_ROWS
#define DKV_ENTRY_ROWS 32
#endif
// Storage order inside a page row.  The row in slot s (its index in the unit's page pool) keeps its 16-byte chunks
// permuted: logical chunk q sits at position q ^ (s & 7).  A run of rows that a bulk copy drops into shared memory
// unchanged can then be read by the attention kernel's fragment loads -- several rows at one logical chunk, or one
// row at several -- without two lanes of a load hitting the same banks.  Every reader and writer of the pages goes
// through row_pos(); a row has at least eight chunks for every supported (type, d).
//   row_pos<EPC>(s, e): position, in elements, of logical element e; EPC = elements per 16-byte chunk
template <int EPC> __device__ __forceinline__ int row_pos(size_t slot, int e) { return e ^ (((int)slot & 7) * EPC); }
template <typename KV> struct Epc { static constexpr int v = 16 / (int)sizeof(KV); };
constexpr int ENTRY_ROWS = DKV_ENTRY_ROWS;   // rows per gather work entry (16 or 32: a run inside one page)
constexpr int MAX_G = 8;
constexpr int FLAG_HOLD = 1;        // split abandoned; not retried until the next append
constexpr int FLAG_SPLIT = 2;       // delayed-split mode: a split is owed (Algorithm 1's f_j)

// Device-resident state of a context.  All arrays are unit-major.
//   KV store: kpages/vpages [U][P][PAGE][d] in kv dtype; every cluster owns a chain of
//   pages (cl_head -> page_next -> ... -> cl_tail) in which all pages but the tail are
//   full, so cluster members are contiguous page by page (intra-cluster placement).
struct Tables {
    int U, G, d, kv_dtype, max_tokens, max_clusters, P, n_splits_attn;
    int update_mode, local_max;      // DYNAKV_MODE_*; LOCAL: size above which a decode-born cluster splits
    int det_sums;                    // 1: centroid sums of the build in 64-bit fixed point (order-independent)
    int buf_max;                     // delayed-split mode: buffered entries per unit that force a split
    int* cl_buf;                     // [U][Mmax] delayed-split mode: entries buffered for a flagged cluster
    int* cl_ver;                     // [U][Mmax] two-tier mode (else null): splits the cluster id has been through
    // FP8 mode (fp8 != 0): kv_dtype is DYNAKV_BF16 for every kernel, all rows lie on the e4m3-times-power-of-two grid,
    // and a one-byte copy of the pages is kept for the gather-attention kernel
    int fp8;
    unsigned char* k8; unsigned char* v8;          // [U][P][PAGE][d] e4m3 bytes
    signed char* k8e; signed char* v8e;            // [U][P][PAGE] exponent of the row's power-of-two scale
    int W;                           // work-list capacity per unit (entries)
    int M_floor;                     // clusters every unit has had since the build (ids never go away); 0 before it
    void* kpages; void* vpages;
    int* page_tok;                   // [U][P][PAGE] token id per slot
    int* page_next;                  // [U][P]
    int* free_stack;                 // [U][P]
    float* cl_r;                     // [U][Mmax][d] representatives (fp32)
    float* cl_M2;                    // [U][Mmax]
    int* cl_n;                       // [U][Mmax]   0 = dead / unused
    int* cl_head; int* cl_tail;      // [U][Mmax]
    unsigned char* cl_flags;         // [U][Mmax]
    int* u_N; int* u_M; int* u_Mlive; float* u_tau; int* u_page_top; int* u_free_cnt;   // [U]
    int* u_scan; int* u_last;        // [U] split check: full scan needed; cluster of the last append (-1 none)
    int* tok_cluster;                // [U][max_tokens]
    // decode scratch
    float* scores;                   // [U][Mmax]
    float* dists;                    // [U][Mmax] squared distance of the step's new key to every representative
    int* sel_ids;                    // [U][Mmax]
    int* sel_n; int* sel_tokens;     // [U]
    int2* work;                      // [U][W] (first row = page * PAGE + offset, rows <= ENTRY_ROWS)
    int* n_work;                     // [U]
    float* part;                     // partial (acc, m, l) records of [G][d + 2] floats: [U][S] (plain kernel) or [2 * n_attn_ctas]
    int* work_prefix;                // [U + 1] exclusive prefix of n_work over the units (written by the last select block)
    int* unit_arrive;                // [U] arrival counters of the split-K combine (zero between steps)
    int* plan_counter;               // [2] blocks finished in this step: [0] of the selection, [1] of the append/split kernel
    // hand-over of triggered units from the unit blocks to the helper blocks of a loop iteration's tail kernel
    int* tail_sync;                  // [4] queue slots reserved, slots claimed, unit blocks that have decided
    int* tail_queue;                 // [U][2] per reserved slot: hint, unit + 1 (0 = not yet written / consumed)
    int* front_done;                 // [U] step + 1 of the last fused centroid pass the unit's block completed
    int* trig_n; int* trig_list;     // [U], [U][Mmax] triggered cluster ids of a unit, ascending
    int n_attn_ctas;                 // persistent gather-attention CTAs (2 per SM)
    int attn_pf_in_smem;             // 1: every attention CTA keeps a copy of work_prefix in shared memory
    // split scratch
    unsigned char* sp_label;         // [U][max_tokens]
    int* sp_pos;                     // [U][2 * max_tokens]: rank per position, then hole list
    // status / counters
    unsigned int* status;            // [1]
    unsigned long long* counters;    // [8]: see CNT_*; 4..6 are scratch of get_status
    int* check_rec;                  // [2] checked build: site of the first index test that failed (0: none), spare
};

// ---- checked build ------------------------------------------------------------------------------------------------
// Compiled with -DDYNAKV_CHECKED, every index that a kernel takes out of a table and turns into an address is tested
// against the array it indexes.  A failing test records its site once (Tables::check_rec), sets DYNAKV_ST_BOUNDS and
// yields false; the caller then skips the access or substitutes an in-range value, so that the kernel's protocol
// (barrier counts, bytes of copies in flight) stays whole.  Without the flag the tests compile to nothing.
enum { SITE_ATTN_ENTRY = 1, SITE_ATTN_WORK = 2, SITE_PLAIN_ENTRY = 3, SITE_SELECT_PAGE = 4, SITE_APPEND_CLUSTER = 5,
       SITE_APPEND_PAGE = 6, SITE_APPEND_TOKEN = 7, SITE_SPLIT_PAGE = 8, SITE_SPLIT_ID = 9, SITE_LAYOUT_PAGE = 10,
       SITE_SPLIT_TOKEN = 11, SITE_STATS_PAGE = 12, SITE_EXPORT_PAGE = 13 };
#ifdef DYNAKV_CHECKED
__device__ __noinline__ static bool dkv_bounds_fail(const Tables& t, int site) {
    atomicOr(t.status, DYNAKV_ST_BOUNDS);
    atomicCAS(&t.check_rec[0], 0, site);
    return false;
}
#define DKV_IN(t, site, v, lo, hi) \
    ((((long long)(v) >= (long long)(lo)) && ((long long)(v) < (long long)(hi))) || dkv::dkv_bounds_fail((t), (site)))
#else
#define DKV_IN(t, site, v, lo, hi) true
#endif

enum { CNT_APPENDED = 0, CNT_SPLITS = 1, CNT_RECHECKED = 2, CNT_TOKENS_ATTENDED = 3, CNT_CLUSTERS_SELECTED = 7 };

// A per-step operand: base pointer plus a stride applied with the device-side step index,
// so the same kernel serves a direct call (ctr == nullptr) and a captured graph replay.  With
// `ind` set the base pointer itself is read from device memory (written at the start of a loop),
// so one captured graph serves every call of the loop whatever arrays the caller passes.
struct StepPtr {
    const void* base;
    long long stride_bytes;
    const int* ctr;
    const void* const* ind;
    __device__ __forceinline__ const char* origin() const { return ind ? (const char*)(*ind) : (const char*)base; }
    __device__ __forceinline__ const void* get() const {
        long long t = ctr ? (long long)(*ctr) : 0;
        return origin() + t * stride_bytes;
    }
    // the operand of step `step`, whatever the step index says
    __device__ __forceinline__ const void* at(long long step) const { return origin() + step * stride_bytes; }
};
struct StepPtrW {
    void* base;
    long long stride_bytes;
    const int* ctr;
    void* const* ind;
    __device__ __forceinline__ void* get() const {
        long long t = ctr ? (long long)(*ctr) : 0;
        return (ind ? (char*)(*ind) : (char*)base) + t * stride_bytes;
    }
};

// ---- element load helpers -------------------------------------------------------------
__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }

// Load 4 consecutive elements starting at element index e (e % 4 == 0) as floats.
__device__ __forceinline__ float4 ld4(const float* p, int e) {
    return *reinterpret_cast<const float4*>(p + e);
}
__device__ __forceinline__ float4 ld4(const __nv_bfloat16* p, int e) {
    uint2 r = *reinterpret_cast<const uint2*>(p + e);
    float4 o;
    o.x = __uint_as_float(r.x << 16); o.y = __uint_as_float(r.x & 0xffff0000u);
    o.z = __uint_as_float(r.y << 16); o.w = __uint_as_float(r.y & 0xffff0000u);
    return o;
}
__device__ __forceinline__ void st4(float* p, int e, float4 v) { *reinterpret_cast<float4*>(p + e) = v; }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Exclusive prefix sum of one int per thread over the block; *total gets the block sum.
// `sh` must hold 33 ints.  Contains __syncthreads; every thread of the block must call it.
__device__ __forceinline__ int block_scan_excl(int v, int* sh, int* total) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
    __syncthreads();
    if (lane == 31) sh[w] = x;
    __syncthreads();
    if (w == 0) {
        int s = lane < nw ? sh[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(0xffffffffu, s, o); if (lane >= o) s += y; }
        sh[lane] = s;
        if (lane == 31) sh[32] = s;
    }
    __syncthreads();
    int base = w > 0 ? sh[w - 1] : 0;
    *total = sh[32];
    return base + x - v;
}

// Counter-based uniform with 23 random bits, u = (bits + 1/2) / 2^23: the 64-bit counter
// built from (seed, unit, round, i) goes through the splitmix64 finaliser.
__device__ __forceinline__ unsigned int hash23(unsigned long long seed, int unit, int round, long long i) {
    unsigned long long x = seed ^ ((unsigned long long)(unit + 1) * 0x9E3779B97F4A7C15ULL);
    x += (unsigned long long)round * 0xBF58476D1CE4E5B9ULL + (unsigned long long)i * 0x94D049BB133111EBULL;
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ULL;
    x ^= x >> 27; x *= 0x94D049BB133111EBULL;
    x ^= x >> 31;
    return (unsigned int)(x >> 41);
}

// ---- programmatic dependent launch: a kernel launched with launch_pdl may start while its predecessor on the
// stream is still finishing; it must call pdl_wait() before it touches anything the predecessor writes (or
// writes anything the predecessor reads).  pdl_trigger() in the predecessor lets the dependents start early;
// without it they start when the predecessor's blocks have exited.  Both are no-ops in an ordinary launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Kernel classes for the optional per-kernel event timing.
enum { KC_INIT = 0, KC_ASSIGN = 1, KC_UPDATE = 2, KC_FINALIZE = 3, KC_SELECT = 4, KC_ATTN = 5, KC_COMBINE = 6,
       KC_APPEND = 7, KC_SPLIT = 8, KC_FRONT = 9, KC_TIER = 10, KC_COUNT = 11 };

// ---- host launchers (defined in the kernel files) ---------------------------------------
struct BuildScratch {
    float* C;            // [U][M][d] current centres
    float* sums;         // [U][M][d]
    int* counts;         // [U][M]
    int* assign;         // [U][n] (or a slice of the trace)
    float* D2;           // [U][n] k-means++ distances
    int* picks;          // [U][M]
    int* cursor;         // [U][M]
    // centroid update by member lists (optional: all three or none)
    int* upd_offset;     // [U][M] first position of the cluster's members in upd_order
    int* upd_cursor;     // [U][M] next free position while the lists are filled
    int* upd_order;      // [U][n] key indices (inside the unit), cluster by cluster
};

void launch_init_centres(const Tables& t, const void* K, long long n, int M, unsigned long long seed,
                         int init_mode, const BuildScratch& b, cudaStream_t s, long long* launches);
void launch_assign_f32(const Tables& t, const void* K, long long n, int M, const float* C, int* assign,
                       cudaStream_t s, long long* launches);
void launch_assign_f32_listed(const Tables& t, const void* K, long long n, int M, const float* C, int* assign,
                              const int* list, const unsigned* counts, unsigned long long* listed_total,
                              cudaStream_t s, long long* launches);
void launch_update(const Tables& t, const void* K, long long n, int M, const int* assign, const BuildScratch& b,
                   cudaStream_t s, long long* launches);
void launch_finalize(const Tables& t, const void* K, const void* V, long long n, int M, const BuildScratch& b,
                     float alpha, cudaStream_t s, long long* launches, const int* order = nullptr);
void launch_pair_count(const Tables& t, int M, unsigned int* f, cudaStream_t s, long long* launches);
void launch_place_order(const Tables& t, int M, const unsigned int* f, int* order, cudaStream_t s, long long* launches);
// What the stand-alone centroid pass does in addition when it opens a captured loop: it resets the device-side
// step index and the hand-over words of the loop's tail kernel, and stores the caller's arrays where the
// captured kernels look them up.
struct LoopBegin {
    int on;                   // 0: an ordinary pass
    int* step_ctr; int* step_lim; int n_steps;
    const void** args;        // device: [4] q, k, v, out of the loop in flight
    const void* q; const void* k; const void* v; void* out;
};
void launch_fp8_round_rows(const void* X, void* Y, long long rows, cudaStream_t s, long long* launches);
void launch_export_rows(const Tables& t, void* K, void* V, long long n, cudaStream_t s, long long* launches);
void launch_import_units(const Tables& t, const int* n_ids, const float* tau, cudaStream_t s, long long* launches);
void launch_front(const Tables& t, StepPtr q, StepPtr k, int has_q, int has_k, cudaStream_t s, long long* launches,
                  const LoopBegin* lb = nullptr);
void launch_select(const Tables& t, int budget, int* user_sel_ids, cudaStream_t s, long long* launches);
void launch_append_apply(const Tables& t, StepPtr k, StepPtr v, cudaStream_t s, long long* launches);
void launch_gather_attn_tma(const Tables& t, StepPtr q, StepPtrW out, cudaStream_t s, long long* launches);
void launch_gather_attn_plain(const Tables& t, StepPtr q, StepPtrW out, cudaStream_t s, long long* launches);
int attn_tma_prepare(const Tables& t);
void launch_selftest_wait_expiry(const Tables& t, int* gave_up, cudaStream_t s, long long* launches);
void launch_gather_attn_v1(const Tables& t, StepPtr q, cudaStream_t s, long long* launches);
void launch_attn_combine(const Tables& t, StepPtrW out, cudaStream_t s, long long* launches);
void launch_split_check(const Tables& t, float gamma, int var_enabled, int min_size, int iters, cudaStream_t s,
                        long long* launches);
// Operands of the next step's centroid pass when it is fused into the tail of a loop iteration.
struct NextFront {
    int on;                  // 0: no fused pass
    StepPtr q, k;            // per-step query and key arrays (indexed with step + 1)
    const int* step_lim;     // device: number of steps of the loop; the pass is skipped when step + 1 reaches it
};
void launch_append_split(const Tables& t, float gamma, int var_enabled, int min_size, int iters, int do_append, StepPtr k,
                         StepPtr v, int* step_ctr, const NextFront& nf, cudaStream_t s, long long* launches);

// Two-tier mode: the page pool (Tables::kpages / vpages) is pinned host memory and this is the HBM cache of page
// frames over it, per unit, filled and replaced in whole clusters.
enum { TIER_PAGES_FETCHED = 0, TIER_HITS = 1, TIER_FETCHED = 2, TIER_REFRESHED = 3, TIER_EVICTED = 4, TIER_STALE = 5, TIER_ROWS = 6,
       TIER_COUNTERS = 8 };
struct TierState {
    int Fc;                          // frames per unit
    void* kcache; void* vcache;      // [U][Fc][PAGE][d] rows in the pool's storage type (one byte per element in FP8 mode)
    signed char* kecache; signed char* vecache;   // [U][Fc][PAGE] FP8 mode: the rows' scale exponents
    int* cl_fr_head; int* cl_fr_tail;   // [U][Mmax] first / last frame of the cluster's copy (-1: no copy)
    int* cl_snap;                    // [U][Mmax][4] the cluster when it was copied: n, version, first page, last page
    unsigned int* cl_lru;            // [U][Mmax] resolve turn that last used the copy
    int* page_frame;                 // [U][P] frame holding a copy of the page (-1: none)
    int* frame_page; int* frame_next;   // [U][Fc] page the frame copies; next frame of the same cluster's copy
    int* fr_free; int* fr_free_cnt;  // [U][Fc] stack of free frames, [U] its height
    int* miss_list;                  // [U][Mmax] selected clusters that need frames this turn
    int2* jobs; int* n_jobs;         // [U][Fc + Mmax] copies of this turn: (page, frame | first row << 20 | rows - 1 << 25), [U] how many
    unsigned int* clock;             // [U] resolve turns so far
    unsigned long long* counters;    // [TIER_COUNTERS]
};
void launch_tier_init(const Tables& t, const TierState& ts, cudaStream_t s, long long* launches);
void launch_tier_resolve_fetch(const Tables& t, const TierState& ts, cudaStream_t s, long long* launches);

}  // namespace dkv
