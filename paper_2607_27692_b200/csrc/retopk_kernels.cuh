// Device code of the ReTopK decode step (sm_100a).
//
// Three kernels per step, all reading caller-owned bf16 q / K / V:
//   recall_kernel  one CTA per (sequence, query head): normalise the query, cosine
//                  similarity to the cached queries (Eq. 6), Top-r recall and rho_max
//                  (Eq. 7), path decision (Eq. 13), insert of the normalised query.  A head
//                  on the exact path flags its KV group.
//   scan_kernel    persistent CTAs over the flagged KV groups: full-history scores
//                  e_i = q.k_i/sqrt(d) (Eq. 4); every key row streams once through the
//                  tensor cores for all G query heads of its group; also the maximum of
//                  every 16-row tile.  Leaves at once when no group is flagged.
//   finish_kernel  one CTA per (sequence, query head) - or a thread-block cluster of 2-8 CTAs
//                  when there are few heads, or 512-thread CTAs two to an SM when there are
//                  more heads than SMs - with heads of both paths side by side.
//                  Reuse path: candidate union (Eq. 8-9) in a shared-memory bitmap, fp32 scores
//                  of the gathered key rows (Eq. 10), Top-K by one histogram (Eq. 11).
//                  Exact path: global Top-K (Eq. 1) of the scanned scores (tile maxima give a
//                  lower bound for the K-th score, only the tiles that reach it are read back).
//                  Both: softmax.V (Eq. 12) and the support insert.
//                  Exact Top-K attention is scan + finish with every head on the exact path.
// All three are programmatic dependent launches; ingest_kernel serves the host-buffer entry point.
//
// (One launch per reuse head - recall stage and reuse path in one kernel, the exact heads
// finished from a list behind the scan - was built and measured: the two launches that are
// then empty on a reuse-only step cost as much as the recall launch saves, and a step with a
// few exact heads pays reuse time PLUS scan PLUS exact finish instead of their maximum.)
//
// Code size matters here: behind a full-history scan the per-head kernels start with cold
// instruction caches, and the fetch cost grows with the size of a kernel's code whether that
// code runs or not.  So: softmax.V and the listed Top-K exist once, out of line, for both paths;
// one general selection; no automatic unrolling of loops that run once; rare cases out of line
// (taking scalars, never the argument block by reference: that would force a copy of it into
// local memory at kernel entry).
#pragma once
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

// Measurement aid: with -DRETOPK_PHASE_CLOCKS thread 0 of every CTA stamps the SM clock at
// phase boundaries into a global table (read back through retopk_debug_read_phases; the
// benchmark's --phases flag builds such a variant of the library and prints the table).
#ifdef RETOPK_PHASE_CLOCKS
#define RETOPK_PHASE_SLOTS 24
__device__ long long g_phase_clk[3][1024][RETOPK_PHASE_SLOTS];
#define RETOPK_PHASE(kernel, n)                                                            \
    do {                                                                                   \
        if (threadIdx.x == 0 && blockIdx.x < 1024) g_phase_clk[kernel][blockIdx.x][n] = clock64(); \
    } while (0)
#else
#define RETOPK_PHASE(kernel, n) do { } while (0)
#endif

namespace retopk {

constexpr int PATH_REUSE = 0, PATH_FALLBACK = 1, PATH_REFRESH = 2;
constexpr int MODE_RETOPK = 0, MODE_EXACT = 1;

constexpr int FINISH_THREADS = 1024;
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_TILE_ROWS = 256;  // key rows per scan work item
constexpr int MAX_GROUPS = 4096;     // B * H_kv limit (shared list in scan_kernel)
constexpr int SEL_BINS = 2048;       // histogram bins of the threshold search
constexpr int SEL_LIST = 256;        // members of the boundary bin ranked exhaustively
constexpr int SCRATCH_WORDS = SEL_BINS + 2 * SEL_LIST + 160;  // bins | boundary list (key, position) | totals, coarse bins, results
constexpr int WS_WORDS = 64;         // scratch of the block-wide prefix sums
constexpr int TILE_ROWS = 16;        // rows per score tile whose maximum the scan records

struct StepArgs {
    int B, Hq, Hkv, G, d, M, r, W, K, cap;
    long long max_seq_len;   // rows per KV head in k / v
    long long score_stride;  // elements per head in ws_scores (multiple of 4)
    int L;                   // seq_len of this step
    float tau, scale;
    int fill;                // cached entries = min(n_inserted, M)
    int slot;                // ring slot written by this step = n_inserted % M
    int refresh;             // 1 when Eq. 13's first case holds (known on the host)
    int mode;                // MODE_RETOPK or MODE_EXACT
    int prefill;             // 1: cache seeding (every head exact, nothing counted)
    int recall_recent;       // 1: recall the newest entries instead of the most similar (Recent-R ablation)
    int NS;                  // entries in the exact path's shared collection lists
    int tile_cap;            // entries in the exact path's list of hit tiles
    int g_shift;             // log2(G) when G is a power of two, else -1
    int step_id;             // call serial number; a KV group is flagged by storing it
    int stage_depth;         // rows in flight per row slot in the reuse path's landing zone
    int exact_stage_depth;   // same for the exact path
    const uint16_t* q;
    const uint16_t* k;
    const uint16_t* v;
    uint16_t* out;
    float* qbar_cache;       // [B*Hq][M][d]
    uint16_t* qbar16;        // same, kept as bf16 (storage variant); null: qbar_cache is in use
    int32_t* sup_cache;      // [B*Hq][M][K]
    uint8_t* ws_path;        // [B*Hq]
    float* ws_rho;           // [B*Hq]
    int32_t* ws_ncand;       // [B*Hq]
    int32_t* ws_sel;         // [B*Hq][r] recalled cache slots, -1 padded
    int32_t* ws_gflag;       // [B*Hkv + 1] == step_id when the group needs a full scan; last word: any group
    int32_t* dbg_cand;       // [B*Hq][cap] test hook: candidate list of the last reuse step, or null
    float* ws_scores;        // [B*Hq][score_stride]
    float* ws_tmax;          // [B*Hq][tmax_stride] largest score of every 16-row key tile
    long long tmax_stride;   // multiple of 4
    unsigned long long* counters;   // [B*Hq][4] reuse, fallback, refresh, cand_sum
    unsigned int* status;
    unsigned long long* slow_select;
    unsigned long long* scan_groups;
    unsigned int* scan_counter;  // pool cursor of scan_kernel; finish_kernel resets it
    int32_t* idx_out;        // MODE_EXACT only, may be null
    int cl_shift;            // finish_kernel runs 2^cl_shift CTAs (one thread-block cluster) per head
    // Fusion-ladder levels below the production one (see retopk_ladder.cuh): the reuse path runs
    // as separate kernels that hand their intermediates on through these global buffers, and
    // finish_kernel then leaves heads on the reuse path alone.
    int skip_reuse;
    float* lw_rho;           // [B*Hq][M] similarities
    float* lw_qbar;          // [B*Hq][d] normalised query
    int32_t* lw_cand;        // [B*Hq][cap] candidate indices
    uint32_t* lw_key;        // [B*Hq][cap] candidate score keys
    uint16_t* lw_rows;       // [B*Hq][cap][d] packed candidate key rows (level 1 only)
    int32_t* lw_sup_idx;     // [B*Hq][K] selected indices
    uint32_t* lw_sup_key;    // [B*Hq][K] their score keys
    int32_t* lw_meta;        // [B*Hq][4] ns, kmax, -, -
};

// ------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------

// fp32 score -> unsigned key with the same order (-0.0 folded onto +0.0 first).
__device__ __forceinline__ uint32_t score_key(float s) {
    s += 0.0f;
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute
// may start while its predecessor still runs; it must call pdl_wait() before touching
// anything the predecessor writes.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// 16-byte asynchronous global -> shared copy (L2 only), and its completion wait.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// L2 residency hints for the scan: key rows are read once (first to go), scores and tile
// maxima are read again by the finish kernel (last to go).
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint4 ldg_stream_hint(const void* p, uint64_t policy) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p), "l"(policy));
    return r;
}
__device__ __forceinline__ void stg_hint(float* p, float v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" :: "l"(p), "f"(v), "l"(policy) : "memory");
}

// One tensor-core step of the scan's dot products: 16 rows x 16 bf16 values against 16 x 8 (fp32 accumulate).
__device__ __forceinline__ void mma_bf16_16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void unpack8(const uint4& x, float* f) {
    f[0] = bf16_lo(x.x); f[1] = bf16_hi(x.x); f[2] = bf16_lo(x.y); f[3] = bf16_hi(x.y);
    f[4] = bf16_lo(x.z); f[5] = bf16_hi(x.z); f[6] = bf16_lo(x.w); f[7] = bf16_hi(x.w);
}

// The cached normalised queries live in fp32 or, as a storage variant, in bf16 (rounded once,
// to nearest even, when stored).  Four consecutive elements of a cache row / one element.
__device__ __forceinline__ float4 load_qbar4(const StepArgs& a, size_t row_off, int lane) {
    if (a.qbar16) {
        const uint2 raw = reinterpret_cast<const uint2*>(a.qbar16 + row_off)[lane];
        return make_float4(bf16_lo(raw.x), bf16_hi(raw.x), bf16_lo(raw.y), bf16_hi(raw.y));
    }
    return reinterpret_cast<const float4*>(a.qbar_cache + row_off)[lane];
}
__device__ __forceinline__ void store_qbar(const StepArgs& a, size_t off, float v) {
    if (a.qbar16) a.qbar16[off] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
    else a.qbar_cache[off] = v;
}

// A head may get a whole thread-block cluster: cluster number and rank of this CTA.
__device__ __forceinline__ int cluster_slot(const StepArgs& a) { return (int)(blockIdx.x >> a.cl_shift); }
__device__ __forceinline__ int cluster_rank(const StepArgs& a) { return (int)(blockIdx.x & ((1u << a.cl_shift) - 1u)); }

// (sequence, KV head) index of query head bh: bh / G without a division when G is 2^k.
__device__ __forceinline__ int kv_group_of(int bh, const StepArgs& a) {
    return a.g_shift >= 0 ? bh >> a.g_shift : bh / a.G;
}

// Exclusive prefix sum of v over the block in thread order; `total` gets the block sum.
// s_ws: NT/32 ints of shared scratch.  Every thread of the block must call.
template <int NT>
__device__ __noinline__ int block_excl_scan(int v, int* s_ws, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) s_ws[warp] = inc;
    __syncthreads();
    int wsum = (lane < NT / 32) ? s_ws[lane] : 0;
    int winc = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
    }
    int wexcl = __shfl_sync(0xffffffffu, winc - wsum, warp);
    total = __shfl_sync(0xffffffffu, winc, NT / 32 - 1);
    __syncthreads();
    return wexcl + inc - v;
}

// Same for two counters at once: .x and .y are scanned side by side (totals may pass 2^16).
// s_ws: 2 * NT/32 ints.
template <int NT>
__device__ __noinline__ int2 block_excl_scan2(int2 v, int* s_ws, int2& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int2 inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int tx = __shfl_up_sync(0xffffffffu, inc.x, o), ty = __shfl_up_sync(0xffffffffu, inc.y, o);
        if (lane >= o) { inc.x += tx; inc.y += ty; }
    }
    if (lane == 31) { s_ws[warp] = inc.x; s_ws[NT / 32 + warp] = inc.y; }
    __syncthreads();
    const int wx = (lane < NT / 32) ? s_ws[lane] : 0, wy = (lane < NT / 32) ? s_ws[NT / 32 + lane] : 0;
    int ix = wx, iy = wy;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int tx = __shfl_up_sync(0xffffffffu, ix, o), ty = __shfl_up_sync(0xffffffffu, iy, o);
        if (lane >= o) { ix += tx; iy += ty; }
    }
    const int ex = __shfl_sync(0xffffffffu, ix - wx, warp), ey = __shfl_sync(0xffffffffu, iy - wy, warp);
    total.x = __shfl_sync(0xffffffffu, ix, NT / 32 - 1);
    total.y = __shfl_sync(0xffffffffu, iy, NT / 32 - 1);
    __syncthreads();
    return make_int2(ex + inc.x - v.x, ey + inc.y - v.y);
}

// ------------------------------------------------------------------------------------
// selection primitives
// ------------------------------------------------------------------------------------
// Where the general (rarely taken) selection code reads its keys: a list in shared memory
// (key, idx) or, with key == nullptr, the score array of a head in global memory (entry i is
// row i).  One type, so there is one copy of that code: the size of a kernel's code costs time
// on every launch that follows a long scan, whether the code runs or not.
struct KeySrc {
    const uint32_t* key;
    const int32_t* idx;
    const float* sc;
    __device__ __forceinline__ uint32_t k(int i) const { return key ? key[i] : score_key(sc[i]); }
    __device__ __forceinline__ int x(int i) const { return key ? idx[i] : i; }
};

// Threshold by radix bisection.  Finds v, a multiple of 2^low_bit, with at least K of
// the keys of src[0..n) >= v (n >= K >= 1), five key bits per round, starting at the first bit in
// which the keys differ at all.  Each round histograms the next digit of the keys that
// still match the prefix into 32 bins x 32 lane columns (a lane only ever adds to its own
// column, so clustered keys do not serialise), sums the columns, and descends into the
// digit that holds the K-th largest key.
//   count == K : exactly K keys are >= v (the search stopped as soon as that held);
//   count  > K : v is the largest multiple with >= K keys at or above it; for low_bit 0 it
//                is the K-th largest key itself and `need` of the keys equal to it belong
//                to the top K.
// s_h: SCRATCH_WORDS ints.  Every thread returns the same result; kmax = largest key.
struct Threshold {
    uint32_t v;
    int count;
    int need;
    uint32_t kmax;
};

template <int NT>
__device__ __noinline__ Threshold count_threshold(const KeySrc src, int n, int K, int low_bit, int* s_h) {
    static_assert(NT % 32 == 0 && NT >= 256, "32 digits are shared out over NT / 32 warps");
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // scratch: two histograms of 32 x 32 words used alternately, then 96 words of totals
    int* s_tot = s_h + 2048;
    // common leading bits of all keys
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    for (int i = tid; i < n; i += NT) { const uint32_t k = src.k(i); kmin = min(kmin, k); kmax = max(kmax, k); }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) { s_tot[warp] = (int)kmin; s_tot[32 + warp] = (int)kmax; }
#pragma unroll
    for (int i = tid; i < 2048; i += NT) s_h[i] = 0;
    __syncthreads();
    kmin = __reduce_min_sync(0xffffffffu, lane < NW ? (uint32_t)s_tot[lane] : 0xffffffffu);
    kmax = __reduce_max_sync(0xffffffffu, lane < NW ? (uint32_t)s_tot[32 + lane] : 0u);
    Threshold res;
    res.kmax = kmax;
    res.count = n;
    int hi = 32 - __clz(kmin ^ kmax);                 // bits [hi-1:0] may differ
    uint32_t prefix = hi >= 32 ? 0u : (kmax >> hi) << hi;
    int kk = K;                                       // rank wanted among the keys matching prefix
    int* hist = s_h;
    while (hi > low_bit && res.count != K) {
        const int width = hi - low_bit < 5 ? hi - low_bit : 5;
        const int shift = hi - width;
        const uint32_t himask = hi >= 32 ? 0u : 0xffffffffu << hi;
        for (int i = tid; i < n; i += NT) {
            const uint32_t k = src.k(i);
            if ((k & himask) == prefix) atomicAdd(&hist[(((k >> shift) & ((1u << width) - 1u)) << 5) + lane], 1);
        }
        __syncthreads();
#pragma unroll
        for (int dgt = warp; dgt < 32; dgt += NW) {   // a warp sums the lane columns of its digit(s)
            const int tot = __reduce_add_sync(0xffffffffu, hist[(dgt << 5) + lane]);
            hist[(dgt << 5) + lane] = 0;              // ready for the round after next
            if (lane == 0) s_tot[64 + dgt] = tot;
        }
        __syncthreads();
        const int c = s_tot[64 + 31 - lane];          // lane l looks at digit 31 - l: descending
        int inc = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        const int above = inc - c;
        const unsigned bal = __ballot_sync(0xffffffffu, above < kk && kk <= above + c);
        const int sel = __ffs(bal) - 1;
        const int above_sel = __shfl_sync(0xffffffffu, above, sel);
        const int c_sel = __shfl_sync(0xffffffffu, c, sel);
        prefix |= (uint32_t)(31 - sel) << shift;
        kk -= above_sel;
        res.count = (K - kk) + c_sel;                 // keys >= the new prefix
        hi = shift;
        hist = (hist == s_h) ? s_h + 1024 : s_h;
    }
    __syncthreads();
    res.v = prefix;
    res.need = kk;
    return res;
}

// Per-warp counts cnt (one per warp, written by lane 0 into s_cnt[warp]) -> the number of
// items in the warps before this one, and the block total.  Call after a barrier.
template <int NT>
__device__ __forceinline__ int warp_base(const int* s_cnt, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int v = lane < NT / 32 ? s_cnt[lane] : 0;
    total = __reduce_add_sync(0xffffffffu, v);
    return __reduce_add_sync(0xffffffffu, lane < warp ? v : 0);
}

// Write, in source order, every element with key > v and the first need_eq elements with
// key == v into s_sup_idx / s_sup_key.  Source order is ascending index, so the output is
// the support in ascending index order with ties resolved to the lower index.  Every thread
// takes one contiguous run of the source, so a single prefix sum places them all.  The general
// form (any number of ties at v); s_ws: WS_WORDS ints.
template <int NT>
__device__ __noinline__ void ordered_emit(const KeySrc src, int n, uint32_t vstar, int need_eq, int32_t* s_sup_idx,
                             uint32_t* s_sup_key, int* s_ws) {
    const int tid = threadIdx.x;
    const int ipt = (n + NT - 1) / NT;                 // NT is a power of two: a shift
    const int lo = min(n, tid * ipt), hi = min(n, lo + ipt);
    int2 cnt = make_int2(0, 0);
    for (int i = lo; i < hi; ++i) {
        const uint32_t key = src.k(i);
        cnt.x += (int)(key > vstar);
        cnt.y += (int)(key == vstar);
    }
    int2 total;
    const int2 excl = block_excl_scan2<NT>(cnt, s_ws, total);
    int g_before = excl.x, e_before = excl.y;
    if (cnt.x | cnt.y) {
        for (int i = lo; i < hi; ++i) {
            const uint32_t key = src.k(i);
            if (key > vstar) {
                const int pos = g_before + (e_before < need_eq ? e_before : need_eq);
                s_sup_idx[pos] = src.x(i);
                s_sup_key[pos] = key;
                ++g_before;
            } else if (key == vstar) {
                if (e_before < need_eq) {
                    const int pos = g_before + e_before;
                    s_sup_idx[pos] = src.x(i);
                    s_sup_key[pos] = key;
                }
                ++e_before;
            }
        }
    }
}

// ------------------------------------------------------------------------------------
// Threshold by ONE histogram over the span of the scores, for lists of at most R * NT keys,
// written without loops: every thread keeps its (at most R) keys and bins in registers and all
// accesses are predicated.  Key i falls into bin floor((score_i - min) / (max - min) *
// (SEL_BINS - 1)): a monotone map, so every key in a bin above the bin b* that holds the K-th
// largest key belongs to the top K, and only b*'s members (a handful when the scores are
// spread) need ranking.  A coarse histogram (one bin per 32 fine ones) beside the fine one lets
// a warp find b* with two 32-lane prefix sums.  On this hardware a taken branch to code that was not just executed costs about
// a hundred cycles, a barrier about eighty, a straight-line instruction a few: the block-wide
// phases of a decode step are short, so their cost is the number of branches and barriers on
// the path, and this form has five barriers and next to no branches.
//   EXACT = true : Top-K of (s_key, s_idx)[0..n) into s_sup_idx / s_sup_key in ascending index
//                  order; returns 1, or 0 (nothing written) when the list needs the general
//                  code: all keys equal, or a boundary bin with too many members.
//   EXACT = false: returns 1 with *v_out = the smallest key of the bins from the boundary bin
//                  up (at least K keys are >= it), or 0 when all keys are equal.
// n > K >= 1 (EXACT) or n >= K (bound).  s_h: SCRATCH_WORDS ints.  *kmax_out = largest key.
// ------------------------------------------------------------------------------------
template <int NT, int R, bool EXACT>
__device__ __forceinline__ int select_small(const uint32_t* s_key, const int32_t* s_idx, int n, int K,
                                            int32_t* s_sup_idx, uint32_t* s_sup_key, int* s_h,
                                            uint32_t* kmax_out, uint32_t* v_out) {
    constexpr int NW = NT / 32, NC = SEL_BINS / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int* s_bl = s_h + SEL_BINS;                      // boundary list: key[SEL_LIST] position[SEL_LIST]
    int* s_tot = s_h + SEL_BINS + 2 * SEL_LIST;      // [0,32) minima [32,64) maxima [64,128) coarse bins [128,136) results
    int* s_res = s_tot + 128;
    uint32_t k[R];
    bool in[R];
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    if (EXACT) RETOPK_PHASE(0, 8);
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int i = r * NT + tid;
        in[r] = i < n;
        k[r] = in[r] ? s_key[i] : 0u;
        kmin = min(kmin, in[r] ? k[r] : 0xffffffffu);
        kmax = max(kmax, k[r]);
    }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) { s_tot[warp] = (int)kmin; s_tot[32 + warp] = (int)kmax; }
#pragma unroll
    for (int j = 0; j < SEL_BINS / NT; ++j) s_h[j * NT + tid] = 0;
    if (tid < NC) s_tot[64 + tid] = 0;
    if (tid < 8) s_res[tid] = tid == 4 ? (int)0xffffffffu : 0;
    __syncthreads();
    if (EXACT) RETOPK_PHASE(0, 9);
    kmin = __reduce_min_sync(0xffffffffu, lane < NW ? (uint32_t)s_tot[lane] : 0xffffffffu);
    kmax = __reduce_max_sync(0xffffffffu, lane < NW ? (uint32_t)s_tot[32 + lane] : 0u);
    *kmax_out = kmax;
    if (__builtin_expect(kmin == kmax, 0)) return 0;
    const float smin = key_score(kmin);
    const float scale = (float)(SEL_BINS - 1) / (key_score(kmax) - smin);
    int b[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int raw = __float2int_rd((key_score(k[r]) - smin) * scale);
        b[r] = min(max(raw, 0), SEL_BINS - 1);          // also tames non-finite scores
        if (in[r]) {
            atomicAdd(&s_h[b[r]], 1);
            atomicAdd(&s_tot[64 + (b[r] >> 5)], 1);
        }
    }
    __syncthreads();
    if (EXACT) RETOPK_PHASE(0, 10);
    // Every warp finds the boundary bin for itself (a lone warp runs several times slower than
    // 32 in step, and this way no barrier is needed to spread the result): coarse bins from the
    // top, two per lane, then the 32 fine bins of the coarse bin found.
    int bstar, above, m;
    {
        const int c0 = s_tot[64 + NC - 1 - 2 * lane], c1 = s_tot[64 + NC - 2 - 2 * lane];
        int inc = c0 + c1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, inc, o); inc += lane >= o ? t : 0; }
        int ab = inc - c0 - c1;
        const unsigned hit = __ballot_sync(0xffffffffu, ab < K && K <= inc);
        const int src = __ffs(hit) - 1;
        const bool first = ab < K && K <= ab + c0;            // the upper of the lane's two coarse bins
        int cb = NC - 1 - 2 * lane - (first ? 0 : 1);
        ab += first ? 0 : c0;
        cb = __shfl_sync(0xffffffffu, cb, src);
        ab = __shfl_sync(0xffffffffu, ab, src);
        const int f = s_h[cb * 32 + 31 - lane];               // fine bins of cb, from the top
        int finc = f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, finc, o); finc += lane >= o ? t : 0; }
        const int fabove = ab + finc - f;
        const unsigned fhit = __ballot_sync(0xffffffffu, fabove < K && K <= fabove + f);
        const int fsrc = __ffs(fhit) - 1;
        bstar = cb * 32 + 31 - fsrc;
        above = __shfl_sync(0xffffffffu, fabove, fsrc);
        m = __shfl_sync(0xffffffffu, f, fsrc);
    }
    if (EXACT) RETOPK_PHASE(0, 11);
    if (!EXACT) {
        uint32_t lo = 0xffffffffu;
#pragma unroll
        for (int r = 0; r < R; ++r) lo = min(lo, in[r] && b[r] == bstar ? k[r] : 0xffffffffu);
        lo = __reduce_min_sync(0xffffffffu, lo);
        if (lane == 0 && lo != 0xffffffffu) atomicMin(reinterpret_cast<unsigned int*>(&s_res[4]), lo);
        __syncthreads();
        *v_out = (uint32_t)s_res[4];
        return 1;
    }
    if (__builtin_expect(m > SEL_LIST - 8, 0)) return 0;
    const int need = K - above;                       // 1..m of the boundary bin's members belong to the top K
    bool member = false;
#pragma unroll
    for (int r = 0; r < R; ++r)
        if (in[r] && b[r] == bstar) {
            member = true;
            const int p = atomicAdd(&s_res[3], 1);
            s_bl[p] = (int)k[r];
            s_bl[SEL_LIST + p] = r * NT + tid;
        }
    __syncthreads();
    if (EXACT) RETOPK_PHASE(0, 12);
    // each owner ranks its own member(s) among the boundary bin's members by (key desc, position
    // asc) and keeps those of rank < need; keys in the bins above are all taken
    bool take[R];
#pragma unroll
    for (int r = 0; r < R; ++r) take[r] = in[r] && b[r] > bstar;
    if (member) {
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (in[r] && b[r] == bstar) {
                const int pos = r * NT + tid;
                int rank = 0;
#pragma unroll 4
                for (int j = 0; j < m; ++j) {
                    const uint32_t o = (uint32_t)s_bl[j];
                    rank += (int)(o > k[r]) | ((int)(o == k[r]) & (int)(s_bl[SEL_LIST + j] < pos));
                }
                take[r] = rank < need;
            }
    }
    if (EXACT) RETOPK_PHASE(0, 13);
    // places from ballots and a small table of per-(round, warp) counts
    int* s_tab = s_h;                                 // (the fine bins are dead: every warp passed the barrier above)
    unsigned bal[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        bal[r] = __ballot_sync(0xffffffffu, take[r]);
        if (lane == 0) s_tab[r * NW + warp] = __popc(bal[r]);
    }
    __syncthreads();
    if (EXACT) RETOPK_PHASE(0, 14);
    int run = 0;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int c = lane < NW ? s_tab[r * NW + lane] : 0;
        const int total = __reduce_add_sync(0xffffffffu, c);
        const int base = run + __reduce_add_sync(0xffffffffu, lane < warp ? c : 0);
        if (take[r]) {
            const int pos = base + __popc(bal[r] & ((1u << lane) - 1u));
            s_sup_idx[pos] = s_idx[r * NT + tid];
            s_sup_key[pos] = k[r];
        }
        run += total;
    }
    return 1;
}

// Top-K of src[0..n) (n > K) by radix bisection and the general emit, for any number of ties:
// ascending index order out, ties to the lower index.  Returns the largest key.
template <int NT>
__device__ __forceinline__ uint32_t select_general(const KeySrc src, int n, int K, int32_t* s_sup_idx,
                                                   uint32_t* s_sup_key, uint32_t* s_hist, int* s_ws) {
    const Threshold t = count_threshold<NT>(src, n, K, 0, reinterpret_cast<int*>(s_hist));
    uint32_t vstar;
    int need_eq;
    if (t.count == K) { vstar = t.v - 1u; need_eq = 0; }            // exactly K keys are >= v
    else { vstar = t.v; need_eq = t.need; }                          // v = K-th largest key
    ordered_emit<NT>(src, n, vstar, need_eq, s_sup_idx, s_sup_key, s_ws);
    return t.kmax;
}

// Top-K of the n listed entries (ascending index order in, ascending index order out).
// *kmax_out: the largest listed key.
// Short lists (at most 3 * NT keys, the usual case) take the loop-free form; longer ones, or
// a list it hands back (all keys equal, a boundary bin with hundreds of members), the radix
// bisection and the general emit.  s_hist: SCRATCH_WORDS words; s_ws: WS_WORDS ints.
// One copy serves both paths of finish_kernel.
template <int NT>
__device__ __noinline__ int select_listed(const uint32_t* s_key, const int32_t* s_idx, int n, int K,
                                          int32_t* s_sup_idx, uint32_t* s_sup_key, uint32_t* s_hist, int* s_ws,
                                          uint32_t* kmax_out) {
    int ns;
    uint32_t kmax = 0u;
    if (n <= K) {
#pragma unroll 1
        for (int i = threadIdx.x; i < n; i += NT) { s_sup_idx[i] = s_idx[i]; s_sup_key[i] = s_key[i]; kmax = max(kmax, s_key[i]); }
        ns = n;
        // (the largest key of a short list: one more reduction, it is rare)
        kmax = __reduce_max_sync(0xffffffffu, kmax);
        if ((threadIdx.x & 31) == 0) s_ws[threadIdx.x >> 5] = (int)kmax;
        __syncthreads();
        kmax = __reduce_max_sync(0xffffffffu, (threadIdx.x & 31) < NT / 32 ? (uint32_t)s_ws[threadIdx.x & 31] : 0u);
    } else if (n <= 3 * NT && select_small<NT, 3, true>(s_key, s_idx, n, K, s_sup_idx, s_sup_key,
                                                           reinterpret_cast<int*>(s_hist), &kmax, nullptr)) {
        ns = K;
    } else {
        __syncthreads();                               // (the short form may have left the scratch in use)
        kmax = select_general<NT>(KeySrc{s_key, s_idx, nullptr}, n, K, s_sup_idx, s_sup_key, s_hist, s_ws);
        ns = K;
    }
    __syncthreads();
    *kmax_out = kmax;
    return ns;
}

// Largest key of s_key[0..n) (the rare callers that select without learning it).  Ends with a barrier.
template <int NT>
__device__ __noinline__ uint32_t block_max_key(const uint32_t* s_key, int n, int* s_ws) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t kmax = 0u;
#pragma unroll 1
    for (int i = tid; i < n; i += NT) kmax = max(kmax, s_key[i]);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) s_ws[warp] = (int)kmax;
    __syncthreads();
    kmax = __reduce_max_sync(0xffffffffu, lane < NT / 32 ? (uint32_t)s_ws[lane] : 0u);
    __syncthreads();
    return kmax;
}

// ------------------------------------------------------------------------------------
// Pieces of the recall stage (one block per head).
// ------------------------------------------------------------------------------------

// Four per-lane partials a[0..3] (one per cache row) summed over the 32 lanes of a warp with
// 6 shuffles instead of 20: lanes trade values as the tree narrows.  Returns the total of row
// (lane >> 3) & 3 ... precisely: row = ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1), on every lane.
__device__ __forceinline__ float reduce4_across32(const float* a, int lane, int& row) {
    const bool h16 = lane & 16, h8 = lane & 8;
    float b[2];
#pragma unroll
    for (int j = 0; j < 2; ++j)
        b[j] = (h16 ? a[j + 2] : a[j]) + __shfl_xor_sync(0xffffffffu, h16 ? a[j] : a[j + 2], 16);
    float c = (h8 ? b[1] : b[0]) + __shfl_xor_sync(0xffffffffu, h8 ? b[0] : b[1], 8);
    c += __shfl_xor_sync(0xffffffffu, c, 4);
    c += __shfl_xor_sync(0xffffffffu, c, 2);
    c += __shfl_xor_sync(0xffffffffu, c, 1);
    row = (h16 ? 2 : 0) + (h8 ? 1 : 0);
    return c;
}

// Eq. 6: rho_c = (qbar_c . q) / |q| for every cached entry c < fill into s_rho[c], and the
// normalised query into s_q[0..D).  Every warp reads the query itself (four elements per
// lane) next to its cache rows, so one memory latency covers both.  No barrier at the end.
template <int D, int NT>
__device__ __forceinline__ void cache_similarities(const StepArgs& a, int bh, float* s_q, float* s_rho) {
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int M = a.M, fill = a.fill;
    float q4[4] = {0.f, 0.f, 0.f, 0.f};
    if (lane < D / 4) {
        const uint2 raw = *reinterpret_cast<const uint2*>(a.q + (size_t)bh * D + 4 * lane);
        q4[0] = bf16_lo(raw.x); q4[1] = bf16_hi(raw.x); q4[2] = bf16_lo(raw.y); q4[3] = bf16_hi(raw.y);
    }
    float inv_nrm = 0.f;
    constexpr int U = NT >= 1024 ? 4 : 8;            // cache rows per warp and trip, all requested before any is used
#pragma unroll 1
    for (int c0 = warp; c0 < fill || c0 == warp; c0 += NW * U) {
        float4 x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + NW * u;
            x[u] = (c < fill && lane < D / 4) ? load_qbar4(a, ((size_t)bh * M + c) * D, lane)
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (c0 == warp) {
            // first trip: the query norm while the loads fly
            float n2 = q4[0] * q4[0];
            n2 = fmaf(q4[1], q4[1], n2); n2 = fmaf(q4[2], q4[2], n2); n2 = fmaf(q4[3], q4[3], n2);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
            const float nrm = sqrtf(n2);
            inv_nrm = nrm > 0.f ? 1.f / nrm : 0.f;
            if (warp == 0 && lane < D / 4) {
#pragma unroll
                for (int e = 0; e < 4; ++e) s_q[4 * lane + e] = nrm > 0.f ? q4[e] / nrm : 0.f;
            }
        }
        if (c0 >= fill) continue;                      // (warp-uniform) nothing cached for this warp
#pragma unroll
        for (int u0 = 0; u0 < U; u0 += 4) {
            float part[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float acc = x[u0 + u].x * q4[0];
                acc = fmaf(x[u0 + u].y, q4[1], acc);
                acc = fmaf(x[u0 + u].z, q4[2], acc);
                acc = fmaf(x[u0 + u].w, q4[3], acc);
                part[u] = acc;
            }
            int row;
            const float tot = reduce4_across32(part, lane, row);
            const int c = c0 + NW * (u0 + row);
            if ((lane & 7) == 0 && c < fill) s_rho[c] = tot * inv_nrm;
        }
    }
}

// Eq. 7: rho_max and the min(r, fill) most similar slots into s_sel (places beyond that keep
// the -1 the caller put there; s_misc[0] must hold -inf): larger rho first, ties -> lower slot.
// Up to 256 cached entries and r <= 8 (the common case) are ranked in registers, eight entries
// per lane, one argmax round per recalled slot; larger caches by one warp per 256 entries and
// a merge of their short lists by warp 0.  The first eight recalled slots also come back in
// sel8 (-1 beyond min(r, fill)), the same on every thread.  s_rho must be complete (barrier
// before the call); s_sel is complete at the block's next barrier.  s_ws: WS_WORDS ints.
__device__ __forceinline__ void warp_top_slots(const float* s_rho, int lo, int hi, int n_take, int lane,
                                               uint32_t* out_key, int* out_slot) {
    // entry lo + v*32 + lane in value v; taken entries drop out by key 0 / slot INT_MAX
    uint32_t key[8];
#pragma unroll
    for (int v = 0; v < 8; ++v) {
        const int c = lo + v * 32 + lane;
        key[v] = c < hi ? score_key(s_rho[c]) : 0u;            // a live key is 0 only for one NaN pattern
    }
#pragma unroll 1
    for (int j = 0; j < n_take; ++j) {
        uint32_t best = 0u;
        int best_c = 0x7fffffff;
#pragma unroll
        for (int v = 0; v < 8; ++v)
            if (key[v] > best) { best = key[v]; best_c = lo + v * 32 + lane; }      // ascending c: the first maximum is the lowest slot
        const uint32_t top = __reduce_max_sync(0xffffffffu, best);
        const int c_star = __reduce_min_sync(0xffffffffu, best == top && top != 0u ? best_c : 0x7fffffff);
#pragma unroll
        for (int v = 0; v < 8; ++v)
            if (lo + v * 32 + lane == c_star) key[v] = 0u;
        if (lane == 0) { out_key[j] = top; out_slot[j] = c_star == 0x7fffffff ? -1 : c_star; }
    }
}

// The cases beside the common one (Recent-R, more than eight recalled slots, more than 256
// cached entries), kept out of line so the common path stays short.  Ends without a barrier.
template <int NT>
__device__ __noinline__ void recall_slots_general(bool recent, int r, int M, int fill, int slot, const float* s_rho,
                                                  int* s_sel, float* s_misc, int* s_ws) {
    // (scalars, not the argument block: a reference to it would force a copy in local memory)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_sel = r < fill ? r : fill;
    if (recent) {
        // Recent-R ablation: the newest n_sel entries (newest first), rho_max over those only
        if (tid < 32) {
            float best = -CUDART_INF_F;
#pragma unroll 1
            for (int j = lane; j < n_sel; j += 32) {
                const int c = ((slot - 1 - j) % M + M) % M;
                s_sel[j] = c;
                best = fmaxf(best, s_rho[c]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
            if (lane == 0) s_misc[0] = best;
        }
    } else if (n_sel > 8) {
        // many recalled slots: every cached entry ranks itself against the others.  P threads
        // share an entry (P a power of two <= 32): each counts the better entries in its slice
        // of the cache, a shuffle tree adds the slices.
        int lp = 5;
        while (lp > 0 && (fill << lp) > NT) --lp;
        const int P = 1 << lp, part = tid & (P - 1);
#pragma unroll 1
        for (int me = tid >> lp; me < ((fill + (NT >> lp) - 1) / (NT >> lp)) * (NT >> lp); me += NT >> lp) {
            const bool live = me < fill;
            const float mine = live ? s_rho[me] : 0.f;
            int rank = 0;
#pragma unroll 2
            for (int c = part; c < fill; c += P) {
                const float o = s_rho[c];
                rank += (int)(o > mine) | ((int)(o == mine) & (int)(c < me));
            }
            for (int o = P >> 1; o > 0; o >>= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
            if (live && part == 0) {
                if (rank < n_sel) s_sel[rank] = me;
                if (rank == 0) s_misc[0] = mine;
            }
        }
    } else if (fill > 256) {
        // one warp per 256 entries leaves its n_sel best in s_ws (keys in [g*16, g*16+8), slots behind them);
        // at most four such warps (M <= 1024)
        const int groups = (fill + 255) >> 8;
        if (warp < groups)
            warp_top_slots(s_rho, warp << 8, min(fill, (warp + 1) << 8), n_sel, lane,
                           reinterpret_cast<uint32_t*>(s_ws) + warp * 16, s_ws + warp * 16 + 8);
        __syncthreads();
        if (warp == 0) {
            // lane l holds candidate (group l >> 3, place l & 7); groups' lists are in rank order already
            const int g = lane >> 3, j = lane & 7;
            uint32_t key = (g < groups && j < n_sel) ? reinterpret_cast<uint32_t*>(s_ws)[g * 16 + j] : 0u;
            int slot = (g < groups && j < n_sel) ? s_ws[g * 16 + 8 + j] : 0x7fffffff;
            if (slot < 0) { slot = 0x7fffffff; key = 0u; }
#pragma unroll 1
            for (int t = 0; t < n_sel; ++t) {
                const uint32_t top = __reduce_max_sync(0xffffffffu, key);
                const int c_star = __reduce_min_sync(0xffffffffu, key == top && top != 0u ? slot : 0x7fffffff);
                if (slot == c_star) key = 0u;
                if (lane == 0 && c_star != 0x7fffffff) { s_sel[t] = c_star; if (t == 0) s_misc[0] = s_rho[c_star]; }
            }
        }
    }
}

template <int NT>
__device__ __forceinline__ float recall_slots(const StepArgs& a, const float* s_rho, int* s_sel, float* s_misc, int* s_ws,
                                              int* sel8) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int fill = a.fill;
    const int n_sel = a.r < fill ? a.r : fill;
    if (__builtin_expect(!a.recall_recent && n_sel <= 8 && fill <= 256 && fill > 0, 1)) {
        // The common case: one warp, up to eight entries per lane, one argmax round per recalled
        // slot (two warp reductions each).  (Having every warp do it for itself was tried: it
        // saves the barrier but costs several times more issue slots than it saves.)
        if (warp == 0) {
            uint32_t* k_out = reinterpret_cast<uint32_t*>(s_ws);
            warp_top_slots(s_rho, 0, fill, n_sel, lane, k_out, s_sel);
            __syncwarp();
            if (lane == 0 && s_sel[0] >= 0) s_misc[0] = s_rho[s_sel[0]];
        }
    } else {
        recall_slots_general<NT>(a.recall_recent != 0, a.r, a.M, fill, a.slot, s_rho, s_sel, s_misc, s_ws);
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 8; ++j) sel8[j] = j < a.r ? s_sel[j] : -1;
    return s_misc[0];
}

// Eq. 13
__device__ __forceinline__ int decide_path(const StepArgs& a, float rho_max) {
    if (a.refresh) return PATH_REFRESH;
    return rho_max < a.tau ? PATH_FALLBACK : PATH_REUSE;
}

// Leave the decision of one head where the later kernels (and the caller) find it; a head
// on the exact path flags its KV group for the scan.
__device__ __forceinline__ void record_decision(const StepArgs& a, int bh, int bkv, const int* s_sel, int path,
                                                float rho_max) {
    const int tid = threadIdx.x;
    if (tid < a.r) a.ws_sel[(size_t)bh * a.r + tid] = s_sel[tid];
    if (tid == 0) {
        a.ws_path[bh] = (uint8_t)path;
        a.ws_rho[bh] = rho_max;
        if (path != PATH_REUSE) {
            a.ws_gflag[bkv] = a.step_id;       // same value from every head of the group
            a.ws_gflag[a.B * a.Hkv] = a.step_id;   // "some group needs a scan in this step"
            a.ws_ncand[bh] = a.L;
            if (!a.prefill) atomicAdd(a.counters + (size_t)bh * 4 + path, 1ull);   // no return value: not waited for
        }
    }
}

// ------------------------------------------------------------------------------------
// Pieces of the reuse path (one block per head).
// ------------------------------------------------------------------------------------

// ------------------------------------------------------------------------------------
// recall_kernel: Eq. 6, Eq. 7, Eq. 13 and the insert of the normalised query, per head.
// Leaves the recalled slots, rho_max and the path in global memory and flags the KV group
// of every head that takes the exact path.  Layout (words): q[D] rho[M+] ws[WS_WORDS] sel[r+] misc[4].
// ------------------------------------------------------------------------------------
constexpr int RECALL_THREADS = 1024;
template <int D>
__global__ void __launch_bounds__(RECALL_THREADS, 1) recall_kernel(const StepArgs a) {
    constexpr int NT = RECALL_THREADS;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* s_q = reinterpret_cast<float*>(smem_raw);
    float* s_rho = s_q + D;
    int* s_ws = reinterpret_cast<int*>(s_rho + ((a.M + 3) & ~3));
    int* s_sel = s_ws + WS_WORDS;
    float* s_misc = reinterpret_cast<float*>(s_sel + ((a.r + 3) & ~3));

    const int tid = threadIdx.x;
    const int bh = blockIdx.x;
    const int bkv = kv_group_of(bh, a);
    if (tid < a.r) s_sel[tid] = -1;
    if (tid == 0) s_misc[0] = -CUDART_INF_F;
    pdl_wait();        // the caches were written by the step before; q by whatever ran before this call
    RETOPK_PHASE(1, 0);
    cache_similarities<D, NT>(a, bh, s_q, s_rho);
    __syncthreads();
    RETOPK_PHASE(1, 1);
    int sel8[8];
    const float rho_max = recall_slots<NT>(a, s_rho, s_sel, s_misc, s_ws, sel8);
    RETOPK_PHASE(1, 3);
    const int path = decide_path(a, rho_max);
    // insert the normalised query now: every similarity of this step has been taken
    if (tid < D) store_qbar(a, ((size_t)bh * a.M + a.slot) * D + tid, s_q[tid]);
    record_decision(a, bh, bkv, s_sel, path, rho_max);
    RETOPK_PHASE(1, 2);
}

// ------------------------------------------------------------------------------------
// Pieces of the reuse path (one block per head).
// ------------------------------------------------------------------------------------

// Eight bf16 values (16 bytes of a key row) against eight query values.
__device__ __forceinline__ float dot8(const uint4& x, const float* qf) {
    float a = bf16_lo(x.x) * qf[0];
    a = fmaf(bf16_hi(x.x), qf[1], a);
    a = fmaf(bf16_lo(x.y), qf[2], a);
    a = fmaf(bf16_hi(x.y), qf[3], a);
    a = fmaf(bf16_lo(x.z), qf[4], a);
    a = fmaf(bf16_hi(x.z), qf[5], a);
    a = fmaf(bf16_lo(x.w), qf[6], a);
    a = fmaf(bf16_hi(x.w), qf[7], a);
    return a;
}

// Sum each of eight per-lane partials a[0..7] over the LPR lanes of a row group, trading
// values between lanes as the tree narrows (7-8 shuffles instead of 8 * log2(LPR)).
// Returns the total of row `row`; for LPR = 16 both lanes of a pair hold the same row.
template <int LPR>
__device__ __forceinline__ float reduce8_across(const float* a, int sub, int& row) {
    float b[4], c[2], d;
    if (LPR == 16) {
        const bool h8 = sub & 8, h4 = sub & 4, h2 = sub & 2;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            b[j] = (h8 ? a[j + 4] : a[j]) + __shfl_xor_sync(0xffffffffu, h8 ? a[j] : a[j + 4], 8);
#pragma unroll
        for (int j = 0; j < 2; ++j)
            c[j] = (h4 ? b[j + 2] : b[j]) + __shfl_xor_sync(0xffffffffu, h4 ? b[j] : b[j + 2], 4);
        d = (h2 ? c[1] : c[0]) + __shfl_xor_sync(0xffffffffu, h2 ? c[0] : c[1], 2);
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        row = sub >> 1;
    } else {
        const bool h4 = sub & 4, h2 = sub & 2, h1 = sub & 1;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            b[j] = (h4 ? a[j + 4] : a[j]) + __shfl_xor_sync(0xffffffffu, h4 ? a[j] : a[j + 4], 4);
#pragma unroll
        for (int j = 0; j < 2; ++j)
            c[j] = (h2 ? b[j + 2] : b[j]) + __shfl_xor_sync(0xffffffffu, h2 ? b[j] : b[j + 2], 2);
        d = (h1 ? c[1] : c[0]) + __shfl_xor_sync(0xffffffffu, h1 ? c[0] : c[1], 1);
        row = sub;
    }
    return d;
}

// Eq. 8-9: the sorted unique candidate list of head bh into s_idx; returns its length.
// Recalled indices below the window go through a bitmap over key positions (ordered
// extraction = sorted and deduplicated for free); the window itself is a contiguous run
// appended behind them, whatever the supports held there.  The bitmap must be clear and
// s_sel loaded (barrier before the call); no barrier at the end.
template <int NT>
__device__ __forceinline__ int candidate_union(const StepArgs& a, int bh, const int* s_sel, int n_sel,
                                               uint32_t* s_bm, int32_t* s_idx, int* s_ws) {
    const int tid = threadIdx.x;
    const int M = a.M, L = a.L, K = a.K;
    const int w_lo = L - a.W > 0 ? L - a.W : 0;
    {
        bool bad = false;
        for (int s0 = 0; s0 < n_sel; s0 += 4)
#pragma unroll 1
            for (int i = tid; i < K; i += NT) {
                int idx[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = s0 + u < n_sel ? s_sel[s0 + u] : -1;
                    idx[u] = c >= 0 ? a.sup_cache[((size_t)bh * M + c) * K + i] : -1;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (idx[u] >= 0) {
                        if (idx[u] < w_lo) atomicOr(&s_bm[idx[u] >> 5], 1u << (idx[u] & 31));
                        else if (idx[u] >= L) bad = true;
                    }
            }
        if (bad) atomicOr(a.status, 1u);
    }
    __syncthreads();
    RETOPK_PHASE(0, 2);
    const int nw_lo = (w_lo + 31) >> 5;               // words that can hold bits below the window
    const int wpt = (nw_lo + NT - 1) / NT;
    const int w0 = tid * wpt;
    const int w1 = (w0 + wpt < nw_lo) ? w0 + wpt : nw_lo;
    int cnt = 0;
#pragma unroll 4
    for (int w = w0; w < w1; ++w) cnt += __popc(s_bm[w]);
    int n_low;
    int pos = block_excl_scan<NT>(cnt, s_ws, n_low);
#pragma unroll 1
    for (int w = w0; w < w1; ++w) {
        uint32_t bits = s_bm[w];
        while (bits) {
            const int bit = __ffs(bits) - 1;
            s_idx[pos++] = w * 32 + bit;
            bits &= bits - 1;
        }
    }
#pragma unroll 1
    for (int i = w_lo + tid; i < L; i += NT) s_idx[n_low + (i - w_lo)] = i;
    return n_low + (L - w_lo);
}

// Eq. 10: exact current-query scores of n key rows as order-preserving keys into key_out.
// Row i is kbase[row_of[i]] (INDEXED) or kbase[i] (rows already packed).  Every lane copies
// its 16 bytes of each row asynchronously into its own landing zone and reads them back
// itself, so a whole wave of rows is in flight with no registers held and no barrier.
// s_qraw: the raw query as D floats; s_stage: depth * NT uint4.  No barrier at the end.
template <int D, int NT, bool INDEXED>
__device__ __forceinline__ void score_candidates(const uint16_t* kbase, const int32_t* row_of, int n,
                                                 const float* s_qraw, uint4* s_stage, int depth, float scale,
                                                 uint32_t* key_out) {
    constexpr int LPR = D / 8, RPW = 32 / LPR, SLOTS = (NT / 32) * RPW;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, myslot = warp * RPW + lane / LPR;
    const char* ksrc = reinterpret_cast<const char*>(kbase) + sub * 16;
    float qf[8];
    *reinterpret_cast<float4*>(qf) = *reinterpret_cast<const float4*>(s_qraw + sub * 8);
    *reinterpret_cast<float4*>(qf + 4) = *reinterpret_cast<const float4*>(s_qraw + sub * 8 + 4);
    uint4* my_stage = s_stage + tid;
    // each wave goes out as two groups of copies, so that the dot products of the first
    // half run while the second half is still arriving
    const int half = (depth + 1) / 2;
    for (int base = 0; base < n; base += SLOTS * depth) {
#pragma unroll 4
        for (int u = 0; u < depth; ++u) {
            const int i = base + u * SLOTS + myslot;
            if (i < n) cp_async16(my_stage + u * NT, ksrc + (size_t)(INDEXED ? row_of[i] : i) * (D * 2));
            if (u == half - 1) cp_async_commit();
        }
        cp_async_commit();
        if (base == 0) RETOPK_PHASE(0, 21);
        for (int g2 = 0; g2 < 2; ++g2) {
            if (g2 == 0) cp_async_wait_but_one();
            else cp_async_wait_all();
            if (base == 0) { if (g2 == 0) RETOPK_PHASE(0, 22); else RETOPK_PHASE(0, 7); }
            const int u_begin = g2 == 0 ? 0 : half, u_end = g2 == 0 ? half : depth;
            for (int u0 = u_begin; u0 < u_end; u0 += 8) {
                float part[8];
#pragma unroll
                for (int uu = 0; uu < 8; ++uu) {
                    const int i = base + (u0 + uu) * SLOTS + myslot;
                    part[uu] = (u0 + uu < u_end && i < n) ? dot8(my_stage[(u0 + uu) * NT], qf) : 0.f;
                }
                int row;
                const float tot = reduce8_across<LPR>(part, sub, row);
                const int i = base + (u0 + row) * SLOTS + myslot;
                if ((LPR == 8 || (sub & 1) == 0) && u0 + row < u_end && i < n) key_out[i] = score_key(tot * scale);
            }
            if (base == 0 && g2 == 0) RETOPK_PHASE(0, 23);
        }
    }
}

// ------------------------------------------------------------------------------------
// Eq. 12: out = sum_i softmax(e)_i v_i over the ns selected rows.
// The value rows are fetched with 16-byte asynchronous copies into a per-thread landing
// zone (depth rows per row slot in flight at once); the softmax weights are computed while
// the first wave is in the air.  s_w: ns floats; s_red: (NT/32) * D + NT floats; s_ws:
// WS_WORDS words; s_stage: depth * NT uint4.
// With a cluster of cl_size CTAs per head (every CTA holding the same support), CTA cl_rank
// fetches and weighs its contiguous share of the rows; the partial sums meet in rank 0
// through distributed shared memory and are added there in rank order.
// ------------------------------------------------------------------------------------
template <int D, int NT>
__device__ __noinline__ void attend(const uint16_t* vbase, int ns, const int32_t* s_sup_idx, const uint32_t* s_sup_key,
                                    float* s_w, float* s_red, int* s_ws, uint4* s_stage, int depth, uint32_t kmax,
                                    uint16_t* out_row, int cl_rank = 0, int cl_size = 1, int ptab = 1) {
    constexpr int LPR = D / 8;                  // lanes per bf16 row (16 bytes each)
    constexpr int RPW = 32 / LPR;               // rows per warp load
    constexpr int SLOTS = (NT / 32) * RPW;      // row slots per block
    constexpr int NW = NT / 32;
    constexpr int PARTS = NT / D;               // second-stage partial sums
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, myslot = warp * RPW + lane / LPR;
    const char* vsrc = reinterpret_cast<const char*>(vbase) + sub * 16;
    uint4* my_stage = s_stage + tid;
    // this CTA's share of the support: [i_lo, i_hi)
    const int share = (ns + cl_size - 1) / cl_size;
    const int i_lo = min(ns, cl_rank * share), i_hi = min(ns, i_lo + share);
    float denom = 0.f;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    RETOPK_PHASE(ptab, 16);
    for (int base = i_lo;;) {
        // (code kept compact on purpose: loops, not unrolled copies)
#pragma unroll 4
        for (int u = 0; u < depth; ++u) {
            const int i = base + u * SLOTS + myslot;
            if (i < i_hi) cp_async16(my_stage + u * NT, vsrc + (size_t)s_sup_idx[i] * (D * 2));
        }
        cp_async_commit();
        if (base == i_lo) {
            // the softmax weights (all ns of them: the denominator is the whole sum) while the
            // first wave of rows is in the air
            RETOPK_PHASE(ptab, 17);
            const float smax = key_score(kmax);
            float wsum = 0.f;
#pragma unroll 1
            for (int i = tid; i < ns; i += NT) {
                const float w = expf(key_score(s_sup_key[i]) - smax);
                s_w[i] = w;
                wsum += w;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
            float* s_wsf = reinterpret_cast<float*>(s_ws);
            if (lane == 0) s_wsf[warp] = wsum;
            __syncthreads();
            denom = lane < NW ? s_wsf[lane] : 0.f;         // fixed tree: the same sum on every lane and run
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, o);
            RETOPK_PHASE(ptab, 18);
        }
        cp_async_wait_all();
        if (base == i_lo) RETOPK_PHASE(ptab, 19);
#pragma unroll 4
        for (int u = 0; u < depth; ++u) {
            const int i = base + u * SLOTS + myslot;
            if (i < i_hi) {
                const float w = s_w[i];
                float f[8];
                unpack8(my_stage[u * NT], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(w, f[e], acc[e]);
            }
        }
        base += SLOTS * depth;
        if (base >= i_hi) break;
    }
    RETOPK_PHASE(ptab, 20);
    // fixed-order reduction: row slots of a warp, then warps in groups, then groups
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    if (lane < LPR) {
#pragma unroll
        for (int e = 0; e < 8; ++e) s_red[warp * D + sub * 8 + e] = acc[e];
    }
    __syncthreads();
    {
        const int j = tid % D, part = tid / D;
        constexpr int WPP = NW / PARTS;          // warps per part
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < WPP; ++w) sum += s_red[(part * WPP + w) * D + j];
        s_red[NW * D + part * D + j] = sum;
    }
    __syncthreads();
    float sum = 0.f;
    if (tid < D) {
#pragma unroll
        for (int p = 0; p < PARTS; ++p) sum += s_red[NW * D + p * D + tid];
    }
    if (cl_size > 1) {
        // s_red[0..D) is free again (its readers passed the barrier above)
        namespace cg = cooperative_groups;
        cg::cluster_group cluster = cg::this_cluster();
        if (tid < D) s_red[tid] = sum;
        cluster.sync();
        if (cl_rank == 0 && tid < D) {
            sum = 0.f;
#pragma unroll 1
            for (int r = 0; r < cl_size; ++r) sum += *cluster.map_shared_rank(s_red + tid, r);
        }
        cluster.sync();           // nobody leaves while its shared memory may still be read
        if (cl_rank != 0) return;
    }
    if (tid < D) {
        const float o = ns > 0 ? sum / denom : 0.f;
        out_row[tid] = __bfloat16_as_ushort(__float2bfloat16_rn(o));
    }
}

// ------------------------------------------------------------------------------------
// reuse path of finish_kernel: candidate union (Eq. 8-9), candidate scores (Eq. 10), Top-K
// (Eq. 11), softmax.V (Eq. 12) and the support insert for one head, all in shared memory.
// (Also built and measured against this form: candidate scores on the tensor cores from
// 16-row staging tiles, and the window's rows requested ahead of the recalled lists.  Phase
// clocks showed them level or ahead, the timed pipeline 3 us per step behind: dropped.)
// ------------------------------------------------------------------------------------
// What either path reads first from global memory, requested at kernel entry together with the
// head's path so that one memory latency covers both: the recalled slot and the two query
// elements this thread will stage (reuse path), eight tile maxima (exact path; a reuse head
// drops them unused, 32 KB of L2 reads per head).
struct FirstLoads {
    int sel;
    uint32_t qraw;
    float4 m4[2];
};
template <int D, int NT>
__device__ __forceinline__ FirstLoads first_loads(const StepArgs& a, int bh, bool want_reuse) {
    const int tid = threadIdx.x;
    FirstLoads f;
    f.sel = (want_reuse && tid < a.r) ? a.ws_sel[(size_t)bh * a.r + tid] : -1;
    f.qraw = (want_reuse && tid >= 32 && tid < 32 + D / 2) ? reinterpret_cast<const uint32_t*>(a.q + (size_t)bh * D)[tid - 32] : 0u;
    const int ntile = (a.L + TILE_ROWS - 1) / TILE_ROWS;
    const float* tm = a.ws_tmax + (size_t)bh * a.tmax_stride;
#pragma unroll
    for (int u = 0; u < 2; ++u)
        f.m4[u] = tid * 8 + 4 * u < ntile ? *reinterpret_cast<const float4*>(tm + tid * 8 + 4 * u)
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
    return f;
}

template <int D, int NT>
__device__ __forceinline__ void reuse_path(const StepArgs& a, unsigned char* smem_raw, const FirstLoads& first) {
    constexpr int NW = NT / 32;
    // layout (words): qraw[D] sel[r] ws[WS_WORDS] hist[SCRATCH_WORDS] sup_idx[K] sup_key[K] w[K]
    //                 | big: idx[cap] key[cap], aliased later by red[NW*D+NT] | bitmap | stage[depth*NT*4]
    float* s_qraw = reinterpret_cast<float*>(smem_raw);
    int* s_sel = reinterpret_cast<int*>(s_qraw + D);
    int* s_ws = s_sel + a.r;
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_ws + WS_WORDS);
    int32_t* s_sup_idx = reinterpret_cast<int32_t*>(s_hist + SCRATCH_WORDS);
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);
    float* s_w = reinterpret_cast<float*>(s_sup_key + a.K);
    const int head_words = (D + a.r + WS_WORDS + SCRATCH_WORDS + 3 * a.K + 3) & ~3;
    int32_t* s_idx = reinterpret_cast<int32_t*>(smem_raw) + head_words;
    uint32_t* s_key = reinterpret_cast<uint32_t*>(s_idx + a.cap);
    float* s_red = reinterpret_cast<float*>(s_idx);
    const int big_words = (max(2 * a.cap, NW * D + NT) + 3) & ~3;
    uint32_t* s_bm = reinterpret_cast<uint32_t*>(s_idx) + big_words;
    uint4* s_stage = reinterpret_cast<uint4*>(s_bm + ((((int)a.max_seq_len + 31) / 32 + 3) & ~3));

    const int tid = threadIdx.x;
    const int bh = cluster_slot(a);
    const int cl_rank = cluster_rank(a), cl_size = 1 << a.cl_shift;
    const int bkv = kv_group_of(bh, a);
    const int M = a.M, fill = a.fill, L = a.L, K = a.K;
    const int n_sel = a.r < fill ? a.r : fill;
    RETOPK_PHASE(0, 0);
    // peers write into this CTA's shared memory later on: all of them must be running by then
    if (cl_size > 1) cooperative_groups::this_cluster().sync();

    // recalled slots and the raw query (requested at kernel entry); clear the bitmap meanwhile
    if (tid < a.r) s_sel[tid] = first.sel;
    if (tid >= 32 && tid < 32 + D / 2) {
        s_qraw[2 * (tid - 32)] = bf16_lo(first.qraw);
        s_qraw[2 * (tid - 32) + 1] = bf16_hi(first.qraw);
    }
    {
        const int nwords = (L + 31) >> 5;
        uint4* bm4 = reinterpret_cast<uint4*>(s_bm);
#pragma unroll 1
        for (int w = tid; w < (nwords + 3) >> 2; w += NT) bm4[w] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    RETOPK_PHASE(0, 1);

    // Eq. 8-9
    const int n = candidate_union<NT>(a, bh, s_sel, n_sel, s_bm, s_idx, s_ws);
    __syncthreads();
    RETOPK_PHASE(0, 3);

    if (a.dbg_cand && cl_rank == 0)
#pragma unroll 1
        for (int i = tid; i < n; i += NT) a.dbg_cand[(size_t)bh * a.cap + i] = s_idx[i];

    // Eq. 10.  In a cluster every CTA built the same list; each scores a contiguous share of
    // it and hands the keys to the others through distributed shared memory.
    {
        const int share = (n + cl_size - 1) / cl_size;
        const int lo = min(n, cl_rank * share), hi = min(n, lo + share);
        score_candidates<D, NT, true>(a.k + (size_t)bkv * a.max_seq_len * D, s_idx + lo, hi - lo, s_qraw, s_stage,
                                      a.stage_depth, a.scale, s_key + lo);
        __syncthreads();
        if (cl_size > 1) {
            namespace cg = cooperative_groups;
            cg::cluster_group cluster = cg::this_cluster();
#pragma unroll 1
            for (int r = 1; r < cl_size; ++r) {
                uint32_t* peer = cluster.map_shared_rank(s_key, (cl_rank + r) & (cl_size - 1));
#pragma unroll 1
                for (int i = lo + tid; i < hi; i += NT) peer[i] = s_key[i];
            }
            cluster.sync();
        }
    }
    RETOPK_PHASE(0, 4);

    // Eq. 11: Top-K of the candidates; insert the support
    uint32_t kmax;
    const int ns = select_listed<NT>(s_key, s_idx, n, K, s_sup_idx, s_sup_key, s_hist, s_ws, &kmax);
    RETOPK_PHASE(0, 5);
    if (cl_rank == 0) {
        int32_t* sup_out = a.sup_cache + ((size_t)bh * M + a.slot) * K;
#pragma unroll 1
        for (int i = tid; i < K; i += NT) sup_out[i] = i < ns ? s_sup_idx[i] : -1;
    }

    // Eq. 12 (s_red aliases the candidate lists, which are dead now)
    attend<D, NT>(a.v + (size_t)bkv * a.max_seq_len * D, ns, s_sup_idx, s_sup_key, s_w, s_red, s_ws, s_stage,
                  a.stage_depth, kmax, a.out + (size_t)bh * D, cl_rank, cl_size, 0);
    if (tid == 0 && cl_rank == 0) {      // the step record is written last: nothing in this kernel waits for it
        a.ws_ncand[bh] = n;
        atomicAdd(a.counters + (size_t)bh * 4 + PATH_REUSE, 1ull);
        atomicAdd(a.counters + (size_t)bh * 4 + 3, (unsigned long long)n);
    }
    RETOPK_PHASE(0, 6);
}

// ------------------------------------------------------------------------------------
// scan_kernel: full-history scores on the tensor cores (mma.sync m16n8k16, bf16 -> fp32)
//
// A 16-row key tile is the A operand, the group's query heads (zero padded to 8) the B
// operand.  A dot product does not care in which order its terms are paired, so each
// thread loads 16 contiguous bytes of a key row straight into its A-fragment registers
// and the query fragment is permuted to match: no shared memory, no transposes.
// CTAs are persistent: the flagged groups' rows are cut into 256-row work items and every
// CTA takes one contiguous share of them.
// ------------------------------------------------------------------------------------

template <int D, int NTILE>   // NTILE = ceil(G / 8) head tiles
__device__ __forceinline__ void scan_body(const StepArgs& a) {
    constexpr int NJ = D / 32;   // 64-byte column groups per row
    __shared__ unsigned short s_list[MAX_GROUPS];
    __shared__ int s_ws[SCAN_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = a.G, L = a.L;
    const int n_groups = a.B * a.Hkv;

    // nothing flagged in this step: leave at once (the common case on the reuse path).  (Reading
    // the flags straight away instead saves a memory latency in front of a short scan, 0.3 us on
    // a mixed step, and costs 0.5 us on every step that scans nothing: measured, not kept.)
    if (a.mode != MODE_EXACT && a.ws_gflag[n_groups] != a.step_id) return;

    // the groups to scan, in ascending order (all of them for Exact Top-K attention)
    int n_act = 0;
    if (a.mode == MODE_EXACT) n_act = n_groups;
    else
        for (int base = 0; base < n_groups; base += SCAN_THREADS) {
            const int i = base + tid;
            const int f = (i < n_groups) && a.ws_gflag[i] == a.step_id;
            int total;
            const int pos = n_act + block_excl_scan<SCAN_THREADS>(f, s_ws, total);
            if (f) s_list[pos] = (unsigned short)i;
            n_act += total;
        }
    if (n_act == 0) return;
    __syncthreads();
    if (blockIdx.x == 0 && tid == 0 && !a.prefill) atomicAdd(a.scan_groups, (unsigned long long)n_act);

    // Work items of 256 rows.  Seven eighths of them are handed out as one contiguous share
    // per CTA (locality, no traffic on the counter); the rest sit in a pool that the CTAs
    // drain one item at a time as they finish, so that the kernel ends on all SMs together
    // (with fixed shares alone the last CTA finished 13 us after the first).
    const int tpg = (L + SCAN_TILE_ROWS - 1) / SCAN_TILE_ROWS;     // work items per group
    const int total_items = n_act * tpg;                            // < 2^31: checked on the host
    const int per = (int)(((long long)total_items * 7 / 8) / (int)gridDim.x);
    const int pool0 = per * (int)gridDim.x;                         // first item of the pool
    __shared__ int s_next;

    const uint64_t pol_first = l2_policy_evict_first(), pol_last = l2_policy_evict_last();
    uint32_t bq[NTILE][NJ][2][2];
    unsigned need = 0;
    int cur = -1, head0 = 0;
    const uint16_t* kbase = nullptr;
    const float scale = a.scale;

    int item = (int)blockIdx.x * per;
    int left = per;                      // items left in the fixed share
    int grabbed = 0;                     // thread 0: pool item requested ahead of time
    if (left == 0) {
        if (tid == 0) s_next = pool0 + (int)atomicAdd(a.scan_counter, 1u);
        __syncthreads();
        item = s_next;
        __syncthreads();
    }
    while (item < total_items) {
        // ask for the next pool item now; the answer is only needed after this item
        const bool last_fixed = left == 1, in_pool = left == 0;
        if ((last_fixed || in_pool) && tid == 0) grabbed = pool0 + (int)atomicAdd(a.scan_counter, 1u);
        const int gi = item / tpg, rb = item - gi * tpg;

        const int bkv = (a.mode == MODE_EXACT) ? gi : s_list[gi];
        if (bkv != cur) {
            cur = bkv;
            head0 = bkv * G;                 // first query head of the group
            kbase = a.k + (size_t)bkv * a.max_seq_len * D;
            need = 0;
            if (a.mode == MODE_EXACT) need = (1u << G) - 1u;
            else
                for (int j = 0; j < G; ++j)
                    if (a.ws_path[head0 + j] != PATH_REUSE) need |= 1u << j;
            // query fragments (B operand), permuted like the key loads below
#pragma unroll
            for (int nt = 0; nt < NTILE; ++nt) {
                const int head = nt * 8 + g;
                const uint32_t* qrow = reinterpret_cast<const uint32_t*>(a.q + (size_t)(head0 + head) * D);
#pragma unroll
                for (int j = 0; j < NJ; ++j)
#pragma unroll
                    for (int p = 0; p < 2; ++p) {
                        const int w = j * 16 + t * 4 + 2 * p;
                        bq[nt][j][p][0] = head < G ? qrow[w] : 0u;
                        bq[nt][j][p][1] = head < G ? qrow[w + 1] : 0u;
                    }
            }
        }
        // this warp's two 16-row tiles of the 256-row item; all loads first
        const int rbase = rb * SCAN_TILE_ROWS + warp * 16;
        uint4 x[2][NJ], y[2][NJ];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const int r0 = rbase + s * 128 + g, r1 = r0 + 8;
            const int c0 = r0 < L ? r0 : L - 1, c1 = r1 < L ? r1 : L - 1;   // never read past L
            const uint16_t* p0 = kbase + (size_t)c0 * D + t * 8;
            const uint16_t* p1 = kbase + (size_t)c1 * D + t * 8;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                x[s][j] = ldg_stream_hint(p0 + j * 32, pol_first);
                y[s][j] = ldg_stream_hint(p1 + j * 32, pol_first);
            }
        }
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const int r0 = rbase + s * 128 + g, r1 = r0 + 8;
#pragma unroll
            for (int nt = 0; nt < NTILE; ++nt) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < NJ; ++j) {
                    mma_bf16_16816(c, x[s][j].x, y[s][j].x, x[s][j].y, y[s][j].y, bq[nt][j][0][0], bq[nt][j][0][1]);
                    mma_bf16_16816(c, x[s][j].z, y[s][j].z, x[s][j].w, y[s][j].w, bq[nt][j][1][0], bq[nt][j][1][1]);
                }
                // c0,c1: row r0, heads 2t, 2t+1 of this tile; c2,c3: row r1
                const int tile_row = rbase + s * 128;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int head = nt * 8 + 2 * t + e;
                    // tile maximum over the 16 rows (rows past L repeat row L-1: harmless)
                    float m = fmaxf(c[e], c[2 + e]);
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
                    if (head < G && ((need >> head) & 1u)) {
                        float* srow = a.ws_scores + (size_t)(head0 + head) * a.score_stride;
                        if (r0 < L) stg_hint(srow + r0, c[e] * scale, pol_last);
                        if (r1 < L) stg_hint(srow + r1, c[2 + e] * scale, pol_last);
                        if (g == 0 && tile_row < L)
                            stg_hint(a.ws_tmax + (size_t)(head0 + head) * a.tmax_stride + (tile_row >> 4), m * scale, pol_last);
                    }
                }
            }
        }
        if (left > 1) { ++item; --left; }
        else {
            if (left == 1) left = 0;
            if (tid == 0) s_next = grabbed;
            __syncthreads();
            item = s_next;
            __syncthreads();
        }
    }
}

// scan_kernel: the launch around scan_body, a dependent launch behind recall_kernel (or, for
// Exact Top-K, behind whatever ran before).  (Letting it come up beside a per-head kernel and
// wait for the decisions only was tried: its CTAs then share SMs whose shared memory is carved
// up for the per-head CTAs, and with that little L1 the scan streams 1.6x slower.)
template <int D, int NTILE>
__global__ void __launch_bounds__(SCAN_THREADS) scan_kernel(const StepArgs a) {
    pdl_wait();        // group flags and paths come from recall_kernel
    scan_body<D, NTILE>(a);
}

// ------------------------------------------------------------------------------------
// exact path of finish_kernel
//
// Global Top-K without reading all L scores again.  The scan left the maximum of every
// 16-row tile.  If v is the K-th largest of (groups of) tile maxima, at least K different
// tiles hold a score >= v, so the K-th largest score is >= v: every member of the exact
// support lies in a tile whose maximum reaches v.  Only those tiles (about K of them) are
// read back, their scores >= v are listed in index order, and the exact Top-K with the
// lower-index tie rule is taken from that list.
// ------------------------------------------------------------------------------------
template <int D, int NT>
__device__ __forceinline__ void exact_path(const StepArgs& a, unsigned char* smem_raw, const FirstLoads& first) {
    // In a cluster every CTA of a head selects the same support on its own (the lists are short
    // and come from L2); only the value rows are shared out, and rank 0 writes the results.
    const int bh = cluster_slot(a);
    const int cl_rank = cluster_rank(a), cl_size = 1 << a.cl_shift;
    // layout (words): sup_idx[K] sup_key[K] w[K] cnt[SCRATCH_WORDS] ws[WS_WORDS] (8 spare)
    //                 | lists: key[NS] idx[NS] tile[tile_cap]; dead once the support is emitted and
    //                   then reused by attend: red[NW*D+NT], stage[depth*NT*4] (may run past the lists)
    constexpr int NW = NT / 32;
    int32_t* s_sup_idx = reinterpret_cast<int32_t*>(smem_raw);
    uint32_t* s_sup_key = reinterpret_cast<uint32_t*>(s_sup_idx + a.K);
    float* s_w = reinterpret_cast<float*>(s_sup_key + a.K);
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_w + a.K);
    int* s_ws = reinterpret_cast<int*>(s_hist + SCRATCH_WORDS);
    uint32_t* s_key = reinterpret_cast<uint32_t*>(smem_raw) + ((3 * a.K + SCRATCH_WORDS + WS_WORDS + 8 + 3) & ~3);
    int32_t* s_idx = reinterpret_cast<int32_t*>(s_key + a.NS);
    int32_t* s_tile = s_idx + a.NS;
    float* s_red = reinterpret_cast<float*>(s_key);
    uint4* s_stage = reinterpret_cast<uint4*>(s_key + ((NW * D + NT + 3) & ~3));

    const int tid = threadIdx.x;
    const int bkv = kv_group_of(bh, a);
    const int K = a.K, L = a.L, NS = a.NS;
    const float* sc = a.ws_scores + (size_t)bh * a.score_stride;
    const float* tm = a.ws_tmax + (size_t)bh * a.tmax_stride;

    int ns = -1;      // selected entries in s_sup_*; -1 = not selected yet
    int n = 0;        // listed entries in s_key / s_idx
    bool slow = false;
    RETOPK_PHASE(2, 0);

    if (L <= K) {
#pragma unroll 1
        for (int i = tid; i < L; i += NT) { s_sup_idx[i] = i; s_sup_key[i] = score_key(sc[i]); }
        ns = L;
        __syncthreads();
    } else {
        const int ntile = (L + TILE_ROWS - 1) / TILE_ROWS;
        const int tcap = a.tile_cap;
        // 1. lower bound v for the K-th score from the tile maxima (grouped so the list is short)
        uint32_t thr_key = 0;
        int sh = 0;                                  // groups of g2 = 2^sh tiles
        while (((ntile + (1 << sh) - 1) >> sh) > 1024 && (ntile >> (sh + 1)) >= 2 * K) ++sh;
        while (((ntile + (1 << sh) - 1) >> sh) > NS) ++sh;
        const int g2 = 1 << sh;
        const int n2 = (ntile + g2 - 1) >> sh;
        // the usual shape: eight tile maxima per thread, kept in registers for step 2
        const bool regs8 = sh == 3 && n2 <= NT;
        float mv[8];
        if (regs8) {
            const int t0 = tid * 8;                 // (the maxima first_loads() asked for)
            const float raw[8] = {first.m4[0].x, first.m4[0].y, first.m4[0].z, first.m4[0].w,
                                  first.m4[1].x, first.m4[1].y, first.m4[1].z, first.m4[1].w};
            float m = -CUDART_INF_F;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                mv[e] = t0 + e < ntile ? raw[e] : -CUDART_INF_F;
                m = fmaxf(m, mv[e]);
            }
            if (tid < n2) s_key[tid] = score_key(m);
            __syncthreads();
        } else if (n2 >= K) {
#pragma unroll 1
            for (int i2 = tid; i2 < n2; i2 += NT) {
                const int t0 = i2 << sh;
                float m;
                if (g2 >= 4) {
                    // g2 is a power of two: whole float4 chunks, all requested before any is used
                    m = -CUDART_INF_F;
                    for (int c0 = 0; c0 < g2; c0 += 16) {
                        float4 x[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            x[u] = (c0 + 4 * u < g2 && t0 + c0 + 4 * u < ntile)
                                ? *reinterpret_cast<const float4*>(tm + t0 + c0 + 4 * u)
                                : make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int tt = t0 + c0 + 4 * u;
                            m = fmaxf(m, x[u].x);
                            if (tt + 1 < ntile) m = fmaxf(m, x[u].y);
                            if (tt + 2 < ntile) m = fmaxf(m, x[u].z);
                            if (tt + 3 < ntile) m = fmaxf(m, x[u].w);
                        }
                    }
                } else {
                    m = tm[t0];
                    if (g2 == 2 && t0 + 1 < ntile) m = fmaxf(m, tm[t0 + 1]);
                }
                s_key[i2] = score_key(m);
            }
            __syncthreads();
        }
        if (n2 >= K) {
            // one histogram over the span of the maxima when they fit the loop-free form (the
            // bound it gives is a key of the list, tighter than a truncated one), else bisection
            uint32_t unused;
            const int done = n2 <= NT
                ? select_small<NT, 1, false>(s_key, nullptr, n2, K, nullptr, nullptr, reinterpret_cast<int*>(s_hist), &unused, &thr_key)
                : 0;
            if (!done) {
                __syncthreads();
                thr_key = count_threshold<NT>(KeySrc{s_key, nullptr, nullptr}, n2, K, 16, reinterpret_cast<int*>(s_hist)).v;
            }
        }
        RETOPK_PHASE(2, 1);
        // 2. the tiles whose maximum reaches v, in ascending order: eight consecutive tile
        //    maxima per thread and one prefix sum per 8 * NT tiles
        int nhit = 0;
#pragma unroll 1
        for (int base = 0; base < ntile; base += NT * 8) {
            const int t0 = base + tid * 8;
            if (!regs8) {
                float4 m4[2];
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    m4[u] = t0 + 4 * u < ntile ? *reinterpret_cast<const float4*>(tm + t0 + 4 * u)
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
                mv[0] = m4[0].x; mv[1] = m4[0].y; mv[2] = m4[0].z; mv[3] = m4[0].w;
                mv[4] = m4[1].x; mv[5] = m4[1].y; mv[6] = m4[1].z; mv[7] = m4[1].w;
            }
            unsigned hits = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (t0 + e < ntile && score_key(mv[e]) >= thr_key) hits |= 1u << e;
            int total;
            int pos = nhit + block_excl_scan<NT>(__popc(hits), s_ws, total);
#pragma unroll
            for (int e = 0; e < 8; ++e) {               // predicated, no loop: a few hits per thread at most
                const bool hit = (hits >> e) & 1u;
                if (hit && pos < tcap) s_tile[pos] = t0 + e;
                pos += hit ? 1 : 0;
            }
            nhit += total;
        }
        __syncthreads();
        RETOPK_PHASE(2, 2);
        if (nhit > tcap) slow = true;
        else {
            // 3. one thread per hit tile: its 16 scores, those >= v listed in index order
#pragma unroll 1
            for (int base = 0; base < nhit; base += NT) {
                const int it = base + tid;
                float4 x[4];
                int row0 = 0;
                unsigned fl = 0;
                if (it < nhit) {
                    row0 = s_tile[it] * TILE_ROWS;
#pragma unroll
                    for (int u = 0; u < 4; ++u) x[u] = *reinterpret_cast<const float4*>(sc + row0 + 4 * u);
                } else {
#pragma unroll
                    for (int u = 0; u < 4; ++u) x[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                const float v16[16] = {x[0].x, x[0].y, x[0].z, x[0].w, x[1].x, x[1].y, x[1].z, x[1].w,
                                       x[2].x, x[2].y, x[2].z, x[2].w, x[3].x, x[3].y, x[3].z, x[3].w};
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    if (it < nhit && row0 + e < L && score_key(v16[e]) >= thr_key) fl |= 1u << e;
                int total;
                int pos = n + block_excl_scan<NT>(__popc(fl), s_ws, total);
#pragma unroll
                for (int e = 0; e < 16; ++e) {          // from the registers, predicated
                    const bool hit = (fl >> e) & 1u;
                    if (hit && pos < NS) { s_key[pos] = score_key(v16[e]); s_idx[pos] = row0 + e; }
                    pos += hit ? 1 : 0;
                }
                n += total;
            }
            __syncthreads();
            if (n > NS) slow = true;
        }
    }
    RETOPK_PHASE(2, 3);
    uint32_t kmax;
    if (slow) {
        // straight from the score array (heavy ties, odd distributions)
        kmax = select_general<NT>(KeySrc{nullptr, nullptr, sc}, L, K, s_sup_idx, s_sup_key, s_hist, s_ws);
        ns = K;
        if (tid == 0 && cl_rank == 0) atomicAdd(a.slow_select, 1ull);
        __syncthreads();
    } else if (ns < 0) {
        ns = select_listed<NT>(s_key, s_idx, n, K, s_sup_idx, s_sup_key, s_hist, s_ws, &kmax);
    } else {
        kmax = block_max_key<NT>(s_sup_key, ns, s_ws);      // L <= K: everything is selected
    }
    RETOPK_PHASE(2, 4);

    // record the support (cache insert / caller's index output)
    int32_t* sup_out = nullptr;
    if (a.mode == MODE_RETOPK) sup_out = a.sup_cache + ((size_t)bh * a.M + a.slot) * K;
    else if (a.idx_out) sup_out = a.idx_out + (size_t)bh * K;
    if (sup_out && cl_rank == 0)
#pragma unroll 1
        for (int i = tid; i < K; i += NT) sup_out[i] = i < ns ? s_sup_idx[i] : -1;

    attend<D, NT>(a.v + (size_t)bkv * a.max_seq_len * D, ns, s_sup_idx, s_sup_key, s_w, s_red, s_ws, s_stage,
                  a.exact_stage_depth, kmax, a.out + (size_t)bh * D, cl_rank, cl_size, 2);
    RETOPK_PHASE(2, 5);
}

// ------------------------------------------------------------------------------------
// finish_kernel: one CTA (or cluster) per (sequence, query head), launched behind the scan.
// A head on the reuse path never needed the scan's results, a head on the exact path selects
// from them; both end with softmax.V and the support insert.  Heads of one step run side by
// side, so a step with a few exact heads costs the longer of the two paths, not their sum.
// ------------------------------------------------------------------------------------
// WITH_REUSE = false leaves the reuse path out: the kernel of the Exact Top-K entry points
// (the size of a kernel's code costs time at every launch behind a long scan).
template <int D, int NT, bool WITH_REUSE = true>
__global__ void __launch_bounds__(NT, 1024 / NT) finish_kernel(const StepArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_wait();        // scores and tile maxima come from the scan, recalled slots and paths from recall_kernel
    if (blockIdx.x == 0 && threadIdx.x == 0) *a.scan_counter = 0u;      // the scan before this kernel is complete
    const int bh = cluster_slot(a);
    const bool retopk = WITH_REUSE && a.mode == MODE_RETOPK;
    const int path = retopk ? (int)a.ws_path[bh] : (int)PATH_FALLBACK;
    const FirstLoads first = first_loads<D, NT>(a, bh, retopk);
    if (path == PATH_REUSE) {
        if (!a.skip_reuse) reuse_path<D, NT>(a, smem_raw, first);
    } else {
        exact_path<D, NT>(a, smem_raw, first);
    }
}

// Host-buffer entry point, when the caller's buffers are pinned and mapped: one launch reads
// the step's query block and the new key / value row of every (sequence, KV head) straight
// from host memory, 16 bytes per thread, into the staging copy of q and into row `pos` of the
// caches.  q_vecs = B*H_q*d/8; rows: [B*H_kv][d] each.
__global__ void ingest_kernel(const uint4* q_src, uint4* q_dst, int q_vecs, const uint4* k_src, const uint4* v_src,
                              uint16_t* k_cache, uint16_t* v_cache, int groups, int d, long long max_seq_len,
                              long long pos) {
    const int lpr = d / 8;                              // 16-byte pieces per row
    const int row_vecs = groups * lpr;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < q_vecs) {
        q_dst[i] = q_src[i];
    } else if (i < q_vecs + 2 * row_vecs) {
        const int j = i - q_vecs;
        const bool is_v = j >= row_vecs;
        const int jj = is_v ? j - row_vecs : j;
        const int g = jj / lpr, sub = jj - g * lpr;
        uint16_t* cache = is_v ? v_cache : k_cache;
        uint4* dst = reinterpret_cast<uint4*>(cache + ((size_t)g * max_seq_len + pos) * d) + sub;
        *dst = (is_v ? v_src : k_src)[jj];
    }
}

// Conversions between the bf16 cache and the fp32 layout of export / import.
__global__ void widen_kernel(const uint16_t* src, float* dst, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = __uint_as_float((uint32_t)src[i] << 16);
}
__global__ void narrow_kernel(const float* src, uint16_t* dst, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = __bfloat16_as_ushort(__float2bfloat16_rn(src[i]));
}

// Clear the caches (supports to -1, queries and counters to 0).
__global__ void reset_kernel(float* qbar, size_t n_q, int32_t* sup, size_t n_sup, unsigned long long* counters,
                             size_t n_cnt, int32_t* gflag, size_t n_flag, unsigned int* status,
                             unsigned long long* slow, unsigned long long* groups, unsigned int* scan_counter) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t t0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (size_t i = t0; i < n_q; i += stride) qbar[i] = 0.f;
    for (size_t i = t0; i < n_sup; i += stride) sup[i] = -1;
    for (size_t i = t0; i < n_cnt; i += stride) counters[i] = 0;
    for (size_t i = t0; i < n_flag; i += stride) gflag[i] = -1;
    if (t0 == 0) { *status = 0u; *slow = 0ull; *groups = 0ull; *scan_counter = 0u; }
}

}  // namespace retopk
