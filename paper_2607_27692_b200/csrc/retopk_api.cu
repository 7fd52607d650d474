// Host side of the ReTopK library: context, argument checks, launch sequence, C interface.
#include "retopk_kernels.cuh"
#include "retopk_ladder.cuh"

#include <math.h>
#include <mutex>
#include <new>
#include <stdio.h>
#include <string.h>

#include "../../include/retopk.h"

using namespace retopk;

struct retopk_ctx {
    int device;
    int B, Hq, Hkv, G, d, M, r, W, K, R, cap;
    float tau;
    long long max_seq_len, score_stride, tmax_stride;
    long long n_ins, t_dec;
    int NS, tile_cap, stage_depth, exact_stage_depth;      // of the block shape in use
    int finish_threads;          // threads per CTA of the per-head kernels: that of the block shape in use
    int shape_id;                // block shape in use (index into shape[])
    // block shapes of finish_kernel: (threads, CTAs per SM) = (1024,1) (512,2) (512,1)
    struct FinishShape { int nt, per_sm, ok, stage_depth, exact_stage_depth, NS, tile_cap; size_t smem_reuse, smem_exact, smem_finish; } shape[3];
    int num_sms, scan_grid;
    int call_serial;
    int recall_recent;
    int broken;                  // a launch failed in the middle of a step: the caches are inconsistent until reset
    mutable int fail_launch;     // test hook: the next launch of kernel 1 (step), 2 (scan) or 3 (finish) reports a failure
    size_t smem_recall, smem_reuse, smem_exact, smem_finish;
    // device state
    float* qbar_cache;
    uint16_t* qbar16;            // bf16 copy of the layout, allocated when that format is chosen
    int qbar_bf16;
    int32_t* sup_cache;
    uint8_t* ws_path;
    float* ws_rho;
    int32_t* ws_ncand;
    int32_t* ws_sel;
    int32_t* ws_gflag;
    int32_t* dbg_cand;           // candidate lists of the last reuse step (test hook), or null
    float* ws_scores;
    float* ws_tmax;
    unsigned long long* counters;
    unsigned int* status;
    unsigned long long* slow_select;
    unsigned long long* scan_groups;
    unsigned int* scan_counter;
    // per-kernel event timing (measurement hook)
    cudaEvent_t* prof_events;
    int prof_max, prof_calls;
    unsigned char* prof_kind;   // per call: 0 = retopk step, 1 = exact_topk_decode
    // staging for the host-buffer entry point
    uint16_t* stage_q;
    uint16_t* stage_out;
    uint16_t* stage_kv;   // [2][B*Hkv*d]
    int last_launches;
    // fusion ladder (measurement): level 1..5, dependent launches on or off, and the buffers
    // the unfused levels hand their intermediates through
    int cluster;                 // CTAs per head in finish_kernel (1, 2, 4 or 8)
    int fusion_level, dependent_launches;
    cudaMemPool_t pool;          // levels 1-3 draw the buffers from here in every step
    void* lw_persist[8];         // level 4 keeps them
    size_t lw_bytes[8];
    size_t sm_sim, sm_topr, sm_union, sm_discover, sm_score, sm_select, sm_attend, sm_fused;
};

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

template <class T>
bool dev_alloc(T** p, size_t count) {
    return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T) > 0 ? count * sizeof(T) : 16) == cudaSuccess;
}

void free_all(retopk_ctx* c) {
    cudaFree(c->qbar_cache); cudaFree(c->sup_cache); cudaFree(c->ws_path); cudaFree(c->ws_rho);
    cudaFree(c->ws_ncand); cudaFree(c->ws_sel); cudaFree(c->ws_gflag); cudaFree(c->ws_scores); cudaFree(c->ws_tmax); cudaFree(c->counters);
    cudaFree(c->status); cudaFree(c->slow_select); cudaFree(c->scan_groups); cudaFree(c->scan_counter); cudaFree(c->stage_q); cudaFree(c->stage_out);
    cudaFree(c->stage_kv);
    cudaFree(c->qbar16);
    cudaFree(c->dbg_cand);
    for (int i = 0; i < 8; ++i) cudaFree(c->lw_persist[i]);
    if (c->pool) cudaMemPoolDestroy(c->pool);
}

StepArgs make_args(const retopk_ctx* c, const void* q, const void* k, const void* v, long long L,
                   void* out, int mode) {
    StepArgs a;
    memset(&a, 0, sizeof a);
    a.B = c->B; a.Hq = c->Hq; a.Hkv = c->Hkv; a.G = c->G; a.d = c->d; a.M = c->M; a.r = c->r;
    a.W = c->W; a.K = c->K; a.cap = c->cap;
    a.max_seq_len = c->max_seq_len; a.score_stride = c->score_stride;
    a.L = (int)L;
    a.tau = c->tau;
    a.scale = 1.0f / sqrtf((float)c->d);
    a.fill = (int)(c->n_ins < c->M ? c->n_ins : c->M);
    a.slot = (int)(c->n_ins % c->M);
    a.refresh = (c->R > 0 && c->t_dec > 0 && c->t_dec % c->R == 0) ? 1 : 0;
    a.mode = mode;
    a.recall_recent = c->recall_recent;
    a.NS = c->NS;
    a.tile_cap = c->tile_cap;
    a.step_id = c->call_serial;
    a.g_shift = (c->G & (c->G - 1)) == 0 ? __builtin_ctz((unsigned)c->G) : -1;
    a.stage_depth = c->stage_depth;
    a.exact_stage_depth = c->exact_stage_depth;
    a.dbg_cand = c->dbg_cand;
    a.q = static_cast<const uint16_t*>(q);
    a.k = static_cast<const uint16_t*>(k);
    a.v = static_cast<const uint16_t*>(v);
    a.out = static_cast<uint16_t*>(out);
    a.qbar_cache = c->qbar_cache; a.sup_cache = c->sup_cache;
    a.qbar16 = c->qbar_bf16 ? c->qbar16 : nullptr;
    a.ws_path = c->ws_path; a.ws_rho = c->ws_rho; a.ws_ncand = c->ws_ncand; a.ws_sel = c->ws_sel; a.ws_gflag = c->ws_gflag;
    a.ws_scores = c->ws_scores; a.ws_tmax = c->ws_tmax; a.tmax_stride = c->tmax_stride; a.counters = c->counters; a.status = c->status;
    a.slow_select = c->slow_select;
    a.scan_groups = c->scan_groups;
    a.scan_counter = c->scan_counter;
    a.idx_out = nullptr;
    a.cl_shift = __builtin_ctz((unsigned)(c->cluster > 0 ? c->cluster : 1));
    return a;
}

// CTAs per head in finish_kernel: with few heads, as many (a power of two up to 8, one SM each)
// as still fit one wave.
int auto_cluster(long long heads, int num_sms) {
    int cl = 1;
    while (cl < 8 && heads * cl * 2 <= num_sms) cl *= 2;
    return cl;
}

// More heads than SMs: two narrower CTAs per SM, so that one head's selection overlaps
// another's row copies.
int auto_shape(const retopk_ctx* c) {
    return (long long)c->B * c->Hq > c->num_sms && c->shape[1].ok ? 1 : 0;
}

void use_finish_shape(retopk_ctx* c, int id) {
    const retopk_ctx::FinishShape& sh = c->shape[id];
    c->shape_id = id;
    c->finish_threads = sh.nt;
    c->stage_depth = sh.stage_depth;
    c->exact_stage_depth = sh.exact_stage_depth;
    c->NS = sh.NS;
    c->tile_cap = sh.tile_cap;
    c->smem_reuse = sh.smem_reuse;
    c->smem_exact = sh.smem_exact;
    c->smem_finish = sh.smem_finish;
}

// Launch with programmatic stream serialisation: the kernel may be set up while its
// predecessor in the stream still runs; it waits (pdl_wait) before reading its inputs.
template <class Kernel>
int launch_dependent(Kernel kernel, unsigned grid, unsigned block, size_t smem, cudaStream_t s,
                     const StepArgs& a, int allowed = 1, int cluster = 1) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = allowed;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cluster > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, kernel, a) == cudaSuccess ? RETOPK_OK : RETOPK_ECUDA;
}

// Test hook (host side only): pretend that the launch of kernel `which` failed.
bool injected_failure(const retopk_ctx* c, int which) {
    if (c->fail_launch != which) return false;
    c->fail_launch = 0;
    return true;
}

int launch_recall(const retopk_ctx* c, const StepArgs& a, cudaStream_t s) {
    if (injected_failure(c, 1)) return RETOPK_ECUDA;
    const unsigned grid = (unsigned)(c->B * c->Hq);
    if (c->d == 128) return launch_dependent(recall_kernel<128>, grid, RECALL_THREADS, c->smem_recall, s, a, c->dependent_launches);
    return launch_dependent(recall_kernel<64>, grid, RECALL_THREADS, c->smem_recall, s, a, c->dependent_launches);
}

int launch_scan(const retopk_ctx* c, const StepArgs& a, cudaStream_t s) {
    if (injected_failure(c, 2)) return RETOPK_ECUDA;
    // persistent CTAs; no more of them than there are 256-row work items
    const long long items = (long long)c->B * c->Hkv * ((a.L + SCAN_TILE_ROWS - 1) / SCAN_TILE_ROWS);
    const unsigned grid = (unsigned)(items < c->scan_grid ? items : c->scan_grid);
    const int ntile = (c->G + 7) / 8;
    // A dependent launch behind recall_kernel (or behind the previous call's last kernel for
    // Exact Top-K).  Behind a kernel that takes ALL of an SM's shared memory the scan ran 1.6x
    // slower: its CTAs then land on SMs still carved up for that kernel, and it needs about
    // 100 KB of L1 per SM to keep its loads in flight.  recall_kernel uses a few KB, so the SMs
    // are back in the default split by the time the scan's CTAs start.
    if (c->d == 128 && ntile == 1) return launch_dependent(scan_kernel<128, 1>, grid, SCAN_THREADS, 0, s, a, c->dependent_launches);
    if (c->d == 128) return launch_dependent(scan_kernel<128, 2>, grid, SCAN_THREADS, 0, s, a, c->dependent_launches);
    if (ntile == 1) return launch_dependent(scan_kernel<64, 1>, grid, SCAN_THREADS, 0, s, a, c->dependent_launches);
    return launch_dependent(scan_kernel<64, 2>, grid, SCAN_THREADS, 0, s, a, c->dependent_launches);
}

int launch_finish(const retopk_ctx* c, const StepArgs& a, cudaStream_t s) {
    if (injected_failure(c, 3)) return RETOPK_ECUDA;
    const unsigned grid = (unsigned)(c->B * c->Hq * c->cluster);      // one cluster of CTAs per head
    const unsigned nt = (unsigned)c->finish_threads;
    const int dep = c->dependent_launches, cl = c->cluster;
    const size_t smem = a.mode == MODE_EXACT ? c->smem_exact : c->smem_finish;
    if (a.mode == MODE_EXACT) {      // the variant without the reuse path's code
        if (c->d == 128) {
            if (nt == 1024) return launch_dependent(finish_kernel<128, 1024, false>, grid, nt, smem, s, a, dep, cl);
            return launch_dependent(finish_kernel<128, 512, false>, grid, nt, smem, s, a, dep, cl);
        }
        if (nt == 1024) return launch_dependent(finish_kernel<64, 1024, false>, grid, nt, smem, s, a, dep, cl);
        return launch_dependent(finish_kernel<64, 512, false>, grid, nt, smem, s, a, dep, cl);
    }
    if (c->d == 128) {
        if (nt == 1024) return launch_dependent(finish_kernel<128, 1024>, grid, nt, smem, s, a, dep, cl);
        return launch_dependent(finish_kernel<128, 512>, grid, nt, smem, s, a, dep, cl);
    }
    if (nt == 1024) return launch_dependent(finish_kernel<64, 1024>, grid, nt, smem, s, a, dep, cl);
    return launch_dependent(finish_kernel<64, 512>, grid, nt, smem, s, a, dep, cl);
}

// Measurement hook: event number `which` (0..3) of the current call, if recording.
void prof_mark(retopk_ctx* c, int which, cudaStream_t s) {
    if (c->prof_events && c->prof_calls < c->prof_max)
        cudaEventRecord(c->prof_events[(size_t)c->prof_calls * 4 + which], s);
}
void prof_done(retopk_ctx* c, int kind) {
    if (c->prof_events && c->prof_calls < c->prof_max) c->prof_kind[c->prof_calls++] = (unsigned char)kind;
}

// Sizes of the exact path's shared lists.  The landing zone of the value rows reuses their
// space, so they cost nothing up to the size of that zone.  16384 entries hold the maximum of
// every 16-row tile of a history of up to 256 Ki keys (longer ones are bounded through groups
// of tiles); the narrow shape (two CTAs per SM, half an SM's shared memory each) takes 8192.
void exact_list_sizes(int K, bool narrow, int* NS, int* tile_cap) {
    if (narrow && K <= 512) { *NS = 8192; *tile_cap = 4096; }
    else { *NS = 16384; *tile_cap = 8192; }
}

// Shared memory of the exact path for a block of nt threads within `budget` bytes (mirrors the
// carve-up at the top of exact_path): the live arrays, then the lists, whose space the
// reduction scratch and the value-row landing zone take over once the support is emitted.
// Returns 0 if not even `min_waves` rows per row slot fit; else the bytes, and the depth.
size_t exact_smem(int K, int NS, int tile_cap, int d, int nt, size_t budget, int min_waves, int* depth) {
    const size_t live = ((size_t)3 * K + SCRATCH_WORDS + WS_WORDS + 8 + 3) & ~(size_t)3;
    const size_t lists = (size_t)2 * NS + tile_cap;
    const size_t red = ((size_t)(nt / 32) * d + nt + 3) & ~(size_t)3;
    const size_t wave = (size_t)nt * 16;
    if (budget < (live + lists) * 4 || budget < (live + red) * 4 + (size_t)min_waves * wave) return 0;
    const int slots = nt / (d / 8);
    long long fit = (long long)((budget - (live + red) * 4) / wave);
    long long want = (K + slots - 1) / slots;
    long long dep = fit < want ? fit : want;
    *depth = (int)(dep < 1 ? 1 : (dep > 16 ? 16 : dep));
    const size_t tail = red + (size_t)*depth * wave / 4;
    return (live + (lists > tail ? lists : tail)) * 4;
}

// The context's buffers live on the device that was current at create: work enqueued with
// another device current would run there with these pointers.
bool on_ctx_device(const retopk_ctx* c) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == c->device;
}

int check_step_args(const retopk_ctx* c, const void* q, const void* k, const void* v, long long L,
                    const void* out) {
    if (!c || !q || !k || !v || !out) return RETOPK_EINVAL;
    if (L < 1 || L > c->max_seq_len) return RETOPK_EINVAL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return RETOPK_EINVAL;
    if (!on_ctx_device(c)) return RETOPK_EINVAL;
    return RETOPK_OK;
}

// ---------------------------------------------------------------------------------------
// Fusion ladder (levels 1-4): the reuse path as separate kernels.
// ---------------------------------------------------------------------------------------
enum { LW_RHO, LW_QBAR, LW_CAND, LW_KEY, LW_ROWS, LW_SUP_IDX, LW_SUP_KEY, LW_META };

// Which buffers a level needs.
bool ladder_needs(int level, int which) {
    switch (which) {
        case LW_RHO: case LW_QBAR: case LW_ROWS: return level == 1;
        case LW_SUP_IDX: case LW_SUP_KEY: case LW_META: return level <= 2;
        default: return true;     // candidates and their keys: every unfused level
    }
}

template <class Kernel>
bool opt_in(Kernel kernel, size_t smem) {
    return smem <= 48 * 1024 ||
           cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess;
}

// Shared-memory footprints of the ladder kernels (mirror the carve-ups at their tops).
int ladder_prepare(retopk_ctx* c) {
    const size_t d = c->d, K = c->K, cap = c->cap, r = c->r;
    const size_t Mp = (c->M + 3) & ~3, capp = (cap + 3) & ~(size_t)3;
    const size_t bm_words = (((size_t)c->max_seq_len + 31) / 32 + 3) & ~(size_t)3;
    const size_t red_words = (size_t)(LADDER_THREADS / 32) * d + LADDER_THREADS;
    const size_t wave = (size_t)LADDER_THREADS * 16 * c->stage_depth;
    const size_t union_words = ((r + 3) & ~(size_t)3) + WS_WORDS + capp + bm_words;
    c->sm_sim = (d + Mp) * 4;
    c->sm_topr = (Mp + WS_WORDS + r + 4) * 4;
    c->sm_union = union_words * 4;
    c->sm_discover = (d + Mp + 4 + union_words) * 4;
    c->sm_score = (d + capp) * 4 + wave;
    c->sm_select = (WS_WORDS + SCRATCH_WORDS + 2 * K + 2 * cap) * 4;
    c->sm_attend = (WS_WORDS + ((3 * K + 3) & ~(size_t)3) + red_words) * 4 + wave;
    const size_t head_words = (WS_WORDS + SCRATCH_WORDS + 3 * K + 3) & ~(size_t)3;
    const size_t big_words = ((2 * cap > red_words ? 2 * cap : red_words) + 3) & ~(size_t)3;
    c->sm_fused = (head_words + big_words) * 4 + wave;
    int max_smem = 0;
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device);
    const size_t all[] = {c->sm_sim, c->sm_topr, c->sm_union, c->sm_discover, c->sm_score, c->sm_select,
                          c->sm_attend, c->sm_fused};
    for (size_t v : all)
        if (v > (size_t)max_smem) return RETOPK_EUNSUPPORTED;
    bool ok = opt_in(ladder_topr_kernel, c->sm_topr) && opt_in(ladder_union_kernel, c->sm_union) &&
              opt_in(ladder_select_kernel, c->sm_select);
    if (c->d == 128)
        ok = ok && opt_in(ladder_similarity_kernel<128>, c->sm_sim) && opt_in(ladder_discover_kernel<128>, c->sm_discover) &&
             opt_in(ladder_score_kernel<128, true>, c->sm_score) && opt_in(ladder_score_kernel<128, false>, c->sm_score) &&
             opt_in(ladder_attend_kernel<128>, c->sm_attend) &&
             opt_in(ladder_select_attend_insert_kernel<128>, c->sm_fused);
    else
        ok = ok && opt_in(ladder_similarity_kernel<64>, c->sm_sim) && opt_in(ladder_discover_kernel<64>, c->sm_discover) &&
             opt_in(ladder_score_kernel<64, true>, c->sm_score) && opt_in(ladder_score_kernel<64, false>, c->sm_score) &&
             opt_in(ladder_attend_kernel<64>, c->sm_attend) &&
             opt_in(ladder_select_attend_insert_kernel<64>, c->sm_fused);
    if (!ok) { cudaGetLastError(); return RETOPK_ECUDA; }
    const size_t nh = (size_t)c->B * c->Hq;
    c->lw_bytes[LW_RHO] = nh * c->M * 4;
    c->lw_bytes[LW_QBAR] = nh * d * 4;
    c->lw_bytes[LW_CAND] = nh * cap * 4;
    c->lw_bytes[LW_KEY] = nh * cap * 4;
    c->lw_bytes[LW_ROWS] = nh * cap * d * 2;
    c->lw_bytes[LW_SUP_IDX] = nh * K * 4;
    c->lw_bytes[LW_SUP_KEY] = nh * K * 4;
    c->lw_bytes[LW_META] = nh * 4 * 4;
    return RETOPK_OK;
}

void ladder_bind(StepArgs& a, void* const* buf) {
    a.lw_rho = static_cast<float*>(buf[LW_RHO]);
    a.lw_qbar = static_cast<float*>(buf[LW_QBAR]);
    a.lw_cand = static_cast<int32_t*>(buf[LW_CAND]);
    a.lw_key = static_cast<uint32_t*>(buf[LW_KEY]);
    a.lw_rows = static_cast<uint16_t*>(buf[LW_ROWS]);
    a.lw_sup_idx = static_cast<int32_t*>(buf[LW_SUP_IDX]);
    a.lw_sup_key = static_cast<uint32_t*>(buf[LW_SUP_KEY]);
    a.lw_meta = static_cast<int32_t*>(buf[LW_META]);
}

#define LADDER_LAUNCH(kernel, smem, ...)                                    \
    do {                                                                    \
        kernel<<<grid, LADDER_THREADS, smem, s>>>(__VA_ARGS__);             \
        if (cudaGetLastError() != cudaSuccess) return RETOPK_ECUDA;         \
        ++launches;                                                         \
    } while (0)

// The launches of one decode step at fusion level 1..4.  Order: decision kernels, scan (exact
// heads), the reuse path's kernels, finish_kernel (exact heads only).
int ladder_launches(retopk_ctx* c, const StepArgs& a, cudaStream_t s, int* n_launches) {
    const int level = c->fusion_level;
    const unsigned grid = (unsigned)(c->B * c->Hq);
    int launches = 0, rc;
    const bool d128 = c->d == 128;

    prof_mark(c, 0, s);
    if (level == 1) {
        if (d128) LADDER_LAUNCH(ladder_similarity_kernel<128>, c->sm_sim, a);
        else LADDER_LAUNCH(ladder_similarity_kernel<64>, c->sm_sim, a);
        LADDER_LAUNCH(ladder_topr_kernel, c->sm_topr, a);
    } else {
        if (d128) LADDER_LAUNCH(ladder_discover_kernel<128>, c->sm_discover, a);
        else LADDER_LAUNCH(ladder_discover_kernel<64>, c->sm_discover, a);
    }
    prof_mark(c, 1, s);
    if ((rc = launch_scan(c, a, s)) != RETOPK_OK) return rc;
    ++launches;
    prof_mark(c, 2, s);
    if (level == 1) {
        LADDER_LAUNCH(ladder_union_kernel, c->sm_union, a);
        if (d128) {
            LADDER_LAUNCH(ladder_pack_rows_kernel<128>, 0, a);
            LADDER_LAUNCH((ladder_score_kernel<128, false>), c->sm_score, a);
        } else {
            LADDER_LAUNCH(ladder_pack_rows_kernel<64>, 0, a);
            LADDER_LAUNCH((ladder_score_kernel<64, false>), c->sm_score, a);
        }
    } else {
        if (d128) LADDER_LAUNCH((ladder_score_kernel<128, true>), c->sm_score, a);
        else LADDER_LAUNCH((ladder_score_kernel<64, true>), c->sm_score, a);
    }
    if (level <= 2) {
        LADDER_LAUNCH(ladder_select_kernel, c->sm_select, a);
        if (d128) LADDER_LAUNCH(ladder_attend_kernel<128>, c->sm_attend, a);
        else LADDER_LAUNCH(ladder_attend_kernel<64>, c->sm_attend, a);
        LADDER_LAUNCH(ladder_insert_kernel, 0, a, level == 1 ? 1 : 0);
    } else {
        if (d128) LADDER_LAUNCH(ladder_select_attend_insert_kernel<128>, c->sm_fused, a);
        else LADDER_LAUNCH(ladder_select_attend_insert_kernel<64>, c->sm_fused, a);
    }
    if ((rc = launch_finish(c, a, s)) != RETOPK_OK) return rc;
    ++launches;
    prof_mark(c, 3, s);
    prof_done(c, 0);
    *n_launches = launches;
    return RETOPK_OK;
}

// One decode step at fusion level 1..4: the buffers (kept by the context at level 4, from the
// pool otherwise) around the launches.
int ladder_step(retopk_ctx* c, StepArgs a, cudaStream_t s) {
    const int level = c->fusion_level;
    void* buf[8] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    int rc = RETOPK_OK;
    if (level == 4) {
        for (int i = 0; i < 8; ++i) buf[i] = c->lw_persist[i];
    } else {
        for (int i = 0; i < 8 && rc == RETOPK_OK; ++i)
            if (ladder_needs(level, i) &&
                cudaMallocFromPoolAsync(&buf[i], c->lw_bytes[i] ? c->lw_bytes[i] : 16, c->pool, s) != cudaSuccess) {
                cudaGetLastError();
                buf[i] = nullptr;
                rc = RETOPK_ENOMEM;
            }
    }
    int launches = 0;
    if (rc == RETOPK_OK) {
        ladder_bind(a, buf);
        a.skip_reuse = 1;
        rc = ladder_launches(c, a, s, &launches);
    }
    if (level != 4)
        for (int i = 0; i < 8; ++i)
            if (buf[i] && cudaFreeAsync(buf[i], s) != cudaSuccess && rc == RETOPK_OK) rc = RETOPK_ECUDA;
    if (rc == RETOPK_OK) c->last_launches = launches;
    return rc;
}
#undef LADDER_LAUNCH

// Can a cluster of `cl` CTAs of `kernel` with this much shared memory be scheduled at all?
template <class Kernel>
bool cluster_fits(Kernel kernel, int threads, size_t smem, int cl) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)cl);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return false; }
    return n > 0;
}

}  // namespace

extern "C" {

int retopk_create_batched(retopk_ctx** out, int B, int H_q, int H_kv, int d, int M, int r, int W,
                          int K, float tau, int R, int64_t max_seq_len) {
    if (!out) return RETOPK_EINVAL;
    *out = nullptr;
    if (B < 1 || H_q < 1 || H_kv < 1 || H_q % H_kv != 0 || M < 1 || r < 1 || r > M || W < 0 || K < 1 ||
        R < 0 || max_seq_len < 1 || d < 1)
        return RETOPK_EINVAL;
    if ((d != 64 && d != 128) || H_q / H_kv > 16 || M > 1024 || K > 4096 || max_seq_len > 1048576 ||
        (long long)B * H_kv > MAX_GROUPS)
        return RETOPK_EUNSUPPORTED;
    if (tau != tau) return RETOPK_EINVAL;
    retopk_ctx* c = new (std::nothrow) retopk_ctx;
    if (!c) return RETOPK_ENOMEM;
    memset(c, 0, sizeof *c);
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return RETOPK_ECUDA; }
    c->B = B; c->Hq = H_q; c->Hkv = H_kv; c->G = H_q / H_kv; c->d = d; c->M = M; c->r = r; c->W = W;
    c->K = K; c->R = R; c->tau = tau; c->max_seq_len = max_seq_len;
    c->cap = r * K + W;
    c->fusion_level = 5;
    c->dependent_launches = 1;
    c->score_stride = (max_seq_len + TILE_ROWS - 1) / TILE_ROWS * TILE_ROWS;   // whole 16-row tiles
    c->tmax_stride = ((max_seq_len + TILE_ROWS - 1) / TILE_ROWS + 3) / 4 * 4;
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    c->num_sms = sms > 0 ? sms : 148;

    // shared-memory footprints (must mirror the carve-up at the top of each kernel)
    c->smem_recall = ((size_t)d + ((M + 3) & ~3) + WS_WORDS + ((r + 3) & ~3) + 4) * 4;
    int max_smem = 0, sm_smem = 0;
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device);
    cudaDeviceGetAttribute(&sm_smem, cudaDevAttrMaxSharedMemoryPerMultiprocessor, c->device);
    static const int kShapeThreads[3] = {1024, 512, 512}, kShapePerSm[3] = {1, 2, 1};
    for (int v = 0; v < 3; ++v) {
        // a CTA that shares its SM gets half of the SM's shared memory (1 KB per CTA is the system's)
        const int nt = kShapeThreads[v];
        const bool narrow = kShapePerSm[v] == 2;
        const size_t budget = narrow ? (size_t)(sm_smem / 2 - 1024) : (size_t)max_smem;
        retopk_ctx::FinishShape& sh = c->shape[v];
        sh.nt = nt;
        sh.per_sm = kShapePerSm[v];
        const size_t red_words = (size_t)(nt / 32) * d + nt;
        const size_t head_words = ((size_t)d + r + WS_WORDS + SCRATCH_WORDS + 3 * (size_t)K + 3) & ~(size_t)3;
        const size_t big_words = (((size_t)2 * c->cap > red_words ? (size_t)2 * c->cap : red_words) + 3) & ~(size_t)3;
        const size_t bm_words = (((size_t)max_seq_len + 31) / 32 + 3) & ~(size_t)3;
        const size_t fixed = (head_words + big_words + bm_words) * 4;
        // exact path: shared lists for the tile maxima (then for the scores that reach the bound,
        // about 1.1-1.4 K of them) and for the tiles that hold them
        exact_list_sizes(K, narrow, &sh.NS, &sh.tile_cap);
        sh.smem_exact = exact_smem(K, sh.NS, sh.tile_cap, d, nt, budget, narrow ? 3 : 1, &sh.exact_stage_depth);
        // the rest of shared memory is the landing zone of the asynchronous row copies: one
        // 16-byte piece per thread per row kept in flight per row slot
        const size_t wave = (size_t)nt * 16;
        // the narrow shape only pays with a few waves of rows in flight on either path
        const size_t min_waves = narrow ? 3 : 1;
        sh.ok = budget >= fixed + min_waves * wave && sh.smem_exact > 0;
        if (!sh.ok) continue;
        const int slots = nt / (d / 8);
        const long long fit = (long long)((budget - fixed) / wave);
        auto waves_for = [&](int rows) { return (long long)((rows + slots - 1) / slots); };
        // enough for one wave of candidates (typically K and a bit) and for the K value rows
        long long want = waves_for(K + K / 4 > c->cap ? c->cap : K + K / 4);
        if (waves_for(K) > want) want = waves_for(K);
        long long dep = fit < want ? fit : want;
        sh.stage_depth = (int)(dep < 1 ? 1 : (dep > 16 ? 16 : dep));
        sh.smem_reuse = fixed + (size_t)sh.stage_depth * wave;
        sh.smem_finish = sh.smem_reuse > sh.smem_exact ? sh.smem_reuse : sh.smem_exact;
    }
    if (!c->shape[0].ok) { delete c; return RETOPK_EUNSUPPORTED; }
    // opt in to the device maximum once; contexts of different sizes then coexist
    bool attr_ok = true;
    auto opt = [&](auto kernel) {
        attr_ok = attr_ok && cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) == cudaSuccess;
    };
    int occ = 0;
    const int ntile = (c->G + 7) / 8;
    if (d == 128) {
        opt(finish_kernel<128, 1024>); opt(finish_kernel<128, 512>);
        opt(finish_kernel<128, 1024, false>); opt(finish_kernel<128, 512, false>);
        if (ntile == 1) cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, scan_kernel<128, 1>, SCAN_THREADS, 0);
        else cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, scan_kernel<128, 2>, SCAN_THREADS, 0);
    } else {
        opt(finish_kernel<64, 1024>); opt(finish_kernel<64, 512>);
        opt(finish_kernel<64, 1024, false>); opt(finish_kernel<64, 512, false>);
        if (ntile == 1) cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, scan_kernel<64, 1>, SCAN_THREADS, 0);
        else cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, scan_kernel<64, 2>, SCAN_THREADS, 0);
    }
    if (!attr_ok) { cudaGetLastError(); delete c; return RETOPK_ECUDA; }
    c->scan_grid = c->num_sms * (occ > 0 ? occ : 2);
    // with few heads, a cluster of CTAs (one SM each) per head, as many as fit one wave
    c->cluster = auto_cluster((long long)B * H_q, c->num_sms);
    use_finish_shape(c, auto_shape(c));


    const size_t nh = (size_t)B * H_q;
    bool ok = dev_alloc(&c->qbar_cache, nh * M * d) && dev_alloc(&c->sup_cache, nh * M * K) &&
              dev_alloc(&c->ws_path, nh) && dev_alloc(&c->ws_rho, nh) && dev_alloc(&c->ws_ncand, nh) &&
              dev_alloc(&c->ws_sel, nh * r) && dev_alloc(&c->ws_gflag, (size_t)B * H_kv + 1) &&
              dev_alloc(&c->ws_scores, nh * (size_t)c->score_stride) &&
              dev_alloc(&c->ws_tmax, nh * (size_t)c->tmax_stride) &&
              dev_alloc(&c->counters, nh * 4) && dev_alloc(&c->status, 1) &&
              dev_alloc(&c->slow_select, 1) && dev_alloc(&c->scan_groups, 1) && dev_alloc(&c->scan_counter, 1) && dev_alloc(&c->stage_q, nh * d) &&
              dev_alloc(&c->stage_out, nh * d) && dev_alloc(&c->stage_kv, (size_t)2 * B * H_kv * d);
    if (!ok) { cudaGetLastError(); free_all(c); delete c; return RETOPK_ENOMEM; }
    *out = c;
    int rc = retopk_reset(c, nullptr);
    if (rc == RETOPK_OK && cudaStreamSynchronize(nullptr) != cudaSuccess) rc = RETOPK_ECUDA;
    if (rc != RETOPK_OK) { free_all(c); delete c; *out = nullptr; }
    return rc;
}

int retopk_create(retopk_ctx** ctx, int H_q, int H_kv, int d, int M, int r, int W, int K, float tau,
                  int R) {
    return retopk_create_batched(ctx, 1, H_q, H_kv, d, M, r, W, K, tau, R, RETOPK_DEFAULT_MAX_SEQ_LEN);
}

int retopk_set_recall_mode(retopk_ctx* c, int mode) {
    if (!c || (mode != RETOPK_RECALL_SIMILAR && mode != RETOPK_RECALL_RECENT)) return RETOPK_EINVAL;
    c->recall_recent = mode == RETOPK_RECALL_RECENT;
    return RETOPK_OK;
}

int retopk_set_qbar_format(retopk_ctx* c, int format) {
    if (!c || (format != RETOPK_QBAR_FP32 && format != RETOPK_QBAR_BF16) || c->n_ins != 0) return RETOPK_EINVAL;
    DeviceGuard g(c->device);
    if (format == RETOPK_QBAR_BF16 && !c->qbar16) {
        const size_t n = (size_t)c->B * c->Hq * c->M * c->d;
        if (cudaMalloc(reinterpret_cast<void**>(&c->qbar16), n * 2) != cudaSuccess) { cudaGetLastError(); c->qbar16 = nullptr; return RETOPK_ENOMEM; }
        if (cudaMemset(c->qbar16, 0, n * 2) != cudaSuccess) return RETOPK_ECUDA;
    }
    c->qbar_bf16 = format == RETOPK_QBAR_BF16;
    return RETOPK_OK;
}

int retopk_set_cluster_size(retopk_ctx* c, int ctas_per_head) {
    if (!c || (ctas_per_head != 1 && ctas_per_head != 2 && ctas_per_head != 4 && ctas_per_head != 8)) return RETOPK_EINVAL;
    if (ctas_per_head > 1) {
        // checked here, so that a size the device cannot schedule fails now and not in the middle of a step
        DeviceGuard g(c->device);
        const int nt = c->finish_threads;
        bool ok;
        if (c->d == 128)
            ok = nt == 1024 ? cluster_fits(finish_kernel<128, 1024>, nt, c->smem_finish, ctas_per_head)
                            : cluster_fits(finish_kernel<128, 512>, nt, c->smem_finish, ctas_per_head);
        else
            ok = nt == 1024 ? cluster_fits(finish_kernel<64, 1024>, nt, c->smem_finish, ctas_per_head)
                            : cluster_fits(finish_kernel<64, 512>, nt, c->smem_finish, ctas_per_head);
        if (!ok) return RETOPK_EUNSUPPORTED;
    }
    c->cluster = ctas_per_head;
    return RETOPK_OK;
}

int retopk_debug_fail_next_launch(retopk_ctx* c, int which) {
    if (!c || which < 0 || which > 3) return RETOPK_EINVAL;
    c->fail_launch = which;
    return RETOPK_OK;
}

int retopk_set_block_shape(retopk_ctx* c, int threads, int ctas_per_sm) {
    if (!c) return RETOPK_EINVAL;
    int id = -1;
    for (int v = 0; v < 3; ++v)
        if (c->shape[v].nt == threads && c->shape[v].per_sm == ctas_per_sm) id = v;
    if (id < 0) return RETOPK_EINVAL;
    if (!c->shape[id].ok) return RETOPK_EUNSUPPORTED;
    if (id != 0 && c->fusion_level < 5) return RETOPK_EINVAL;
    use_finish_shape(c, id);
    return RETOPK_OK;
}

int retopk_set_finish_threads(retopk_ctx* c, int threads) {
    if (!c || (threads != 1024 && threads != 512)) return RETOPK_EINVAL;
    return retopk_set_block_shape(c, threads, threads == 512 ? 2 : 1);
}

int retopk_set_fusion_level(retopk_ctx* c, int level, int dependent_launches) {
    if (!c || level < 1 || level > 5 || (dependent_launches != 0 && dependent_launches != 1)) return RETOPK_EINVAL;
    if (dependent_launches && level != 5) return RETOPK_EINVAL;   // the unfused kernels are plain launches
    DeviceGuard g(c->device);
    // the unfused kernels are sized for the wide finish shape; level 5 goes back to the default
    use_finish_shape(c, level < 5 ? 0 : auto_shape(c));
    if (level < 5) {
        int rc = ladder_prepare(c);
        if (rc != RETOPK_OK) return rc;
        if (cudaDeviceSynchronize() != cudaSuccess) return RETOPK_ECUDA;
        if (level == 4) {
            for (int i = 0; i < 8; ++i)
                if (ladder_needs(4, i) && !c->lw_persist[i] &&
                    cudaMalloc(&c->lw_persist[i], c->lw_bytes[i] ? c->lw_bytes[i] : 16) != cudaSuccess) {
                    cudaGetLastError();
                    return RETOPK_ENOMEM;
                }
        } else if (!c->pool) {
            cudaMemPoolProps props;
            memset(&props, 0, sizeof props);
            props.allocType = cudaMemAllocationTypePinned;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = c->device;
            if (cudaMemPoolCreate(&c->pool, &props) != cudaSuccess) { cudaGetLastError(); c->pool = nullptr; return RETOPK_ECUDA; }
            unsigned long long keep = ~0ull;     // freed blocks stay with the pool for the next step
            cudaMemPoolSetAttribute(c->pool, cudaMemPoolAttrReleaseThreshold, &keep);
        }
    }
    c->fusion_level = level;
    c->dependent_launches = dependent_launches;
    return RETOPK_OK;
}

int retopk_destroy(retopk_ctx* c) {
    if (!c) return RETOPK_EINVAL;
    DeviceGuard g(c->device);
    cudaDeviceSynchronize();
    free_all(c);
    delete c;
    return RETOPK_OK;
}

int retopk_reset(retopk_ctx* c, void* stream) {
    if (!c || !on_ctx_device(c)) return RETOPK_EINVAL;
    const size_t nh = (size_t)c->B * c->Hq;
    reset_kernel<<<c->num_sms * 4, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        c->qbar_cache, nh * c->M * c->d, c->sup_cache, nh * c->M * c->K, c->counters, nh * 4, c->ws_gflag,
        (size_t)c->B * c->Hkv + 1, c->status, c->slow_select, c->scan_groups, c->scan_counter);
    c->n_ins = 0;
    c->t_dec = 0;
    c->broken = 0;
    if (cudaGetLastError() != cudaSuccess) return RETOPK_ECUDA;
    if (c->qbar16 && cudaMemsetAsync(c->qbar16, 0, nh * c->M * c->d * 2, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return RETOPK_ECUDA;
    return RETOPK_OK;
}

int retopk_decode_step(retopk_ctx* c, const void* q, const void* k_cache, const void* v_cache,
                       int64_t seq_len, void* out, void* stream) {
    int rc = check_step_args(c, q, k_cache, v_cache, seq_len, out);
    if (rc != RETOPK_OK) return rc;
    if (c->broken) return RETOPK_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    StepArgs a = make_args(c, q, k_cache, v_cache, seq_len, out, MODE_RETOPK);
    c->call_serial = (c->call_serial + 1) & 0x3fffffff;
    a.step_id = c->call_serial;
    if (c->fusion_level < 5) {
        // a failure inside may have left some of the step's kernels enqueued
        if ((rc = ladder_step(c, a, s)) != RETOPK_OK) { c->broken = 1; return rc; }
        c->n_ins += 1;
        c->t_dec += 1;
        return RETOPK_OK;
    }
    prof_mark(c, 0, s);
    if ((rc = launch_recall(c, a, s)) != RETOPK_OK) return rc;    // nothing of this step is enqueued yet
    prof_mark(c, 1, s);
    // From here on the step's first kernel is in the stream (normalised queries inserted): a
    // failed launch leaves the caches half advanced, so the context refuses further steps until
    // retopk_reset.
    if ((rc = launch_scan(c, a, s)) != RETOPK_OK) { c->broken = 1; return rc; }
    prof_mark(c, 2, s);
    if ((rc = launch_finish(c, a, s)) != RETOPK_OK) { c->broken = 1; return rc; }
    prof_mark(c, 3, s);
    prof_done(c, 0);
    c->last_launches = 3;
    c->n_ins += 1;
    c->t_dec += 1;
    return RETOPK_OK;
}

int retopk_prefill(retopk_ctx* c, const void* q_tail, const void* k_cache, const void* v_cache,
                   int64_t prompt_len, int n_tail, void* stream) {
    if (!c || !q_tail || !k_cache || !v_cache) return RETOPK_EINVAL;
    if (n_tail < 1 || n_tail > c->M || n_tail > prompt_len || prompt_len > c->max_seq_len) return RETOPK_EINVAL;
    if (!aligned16(q_tail) || !aligned16(k_cache) || !aligned16(v_cache)) return RETOPK_EINVAL;
    if (!on_ctx_device(c)) return RETOPK_EINVAL;
    if (c->broken) return RETOPK_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t slab = (size_t)c->B * c->Hq * c->d;          // elements per prompt position
    for (int j = 0; j < n_tail; ++j) {
        // position p = prompt_len - n_tail + j sees keys 0..p: the exact path with L = p + 1
        StepArgs a = make_args(c, static_cast<const uint16_t*>(q_tail) + (size_t)j * slab, k_cache, v_cache,
                               prompt_len - n_tail + j + 1, c->stage_out, MODE_RETOPK);
        a.refresh = 1;                 // every head takes the exact path
        a.prefill = 1;                 // and nothing is counted
        c->call_serial = (c->call_serial + 1) & 0x3fffffff;
        a.step_id = c->call_serial;
        int rc;
        if ((rc = launch_recall(c, a, s)) != RETOPK_OK) return rc;
        if ((rc = launch_scan(c, a, s)) != RETOPK_OK) { c->broken = 1; return rc; }
        if ((rc = launch_finish(c, a, s)) != RETOPK_OK) { c->broken = 1; return rc; }
        c->n_ins += 1;
    }
    c->last_launches = 3 * n_tail;
    return RETOPK_OK;
}

int exact_topk_decode(retopk_ctx* c, const void* q, const void* k_cache, const void* v_cache,
                      int64_t seq_len, void* out, int32_t* idx_out, void* stream) {
    int rc = check_step_args(c, q, k_cache, v_cache, seq_len, out);
    if (rc != RETOPK_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    StepArgs a = make_args(c, q, k_cache, v_cache, seq_len, out, MODE_EXACT);
    a.idx_out = idx_out;
    prof_mark(c, 0, s);
    prof_mark(c, 1, s);
    if ((rc = launch_scan(c, a, s)) != RETOPK_OK) return rc;
    prof_mark(c, 2, s);
    if ((rc = launch_finish(c, a, s)) != RETOPK_OK) {
        // the scan is enqueued and nothing will put its work counter back: do it here
        cudaMemsetAsync(c->scan_counter, 0, sizeof(unsigned int), s);
        return rc;
    }
    prof_mark(c, 3, s);
    prof_done(c, 1);
    c->last_launches = 2;
    return RETOPK_OK;
}

// Device-side alias of a host pointer the GPU can address directly (pinned and mapped), or null.
static void* device_alias(const void* host) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (at.type != cudaMemoryTypeHost) return nullptr;
    return at.devicePointer;
}

int retopk_decode_step_host(retopk_ctx* c, const void* q_host, const void* k_new_host,
                            const void* v_new_host, void* k_cache, void* v_cache, int64_t seq_len,
                            void* out_host, void* stream) {
    if (!c || !q_host || !k_new_host || !v_new_host || !k_cache || !v_cache || !out_host)
        return RETOPK_EINVAL;
    if (seq_len < 1 || seq_len > c->max_seq_len) return RETOPK_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t row = (size_t)c->d * 2;
    const size_t nq = (size_t)c->B * c->Hq * row, nkv = (size_t)c->B * c->Hkv;
    // Pinned, mapped host buffers are read and written by the kernels themselves: one small
    // launch brings q and the new rows across, finish_kernel stores the output rows to the
    // host.  Anything else goes through staged copies.
    void* q_dev = device_alias(q_host);
    void* k_dev = device_alias(k_new_host);
    void* v_dev = device_alias(v_new_host);
    void* out_dev = device_alias(out_host);
    const bool direct = q_dev && k_dev && v_dev && out_dev && aligned16(q_dev) && aligned16(k_dev) &&
                        aligned16(v_dev) && aligned16(k_cache) && aligned16(v_cache);
    if (direct) {
        const int q_vecs = (int)(nq / 16), row_vecs = (int)(nkv * row / 16);
        const int total = q_vecs + 2 * row_vecs;
        ingest_kernel<<<(total + 255) / 256, 256, 0, s>>>(
            static_cast<const uint4*>(q_dev), reinterpret_cast<uint4*>(c->stage_q), q_vecs,
            static_cast<const uint4*>(k_dev), static_cast<const uint4*>(v_dev), static_cast<uint16_t*>(k_cache),
            static_cast<uint16_t*>(v_cache), (int)nkv, c->d, c->max_seq_len, seq_len - 1);
        if (cudaGetLastError() != cudaSuccess) return RETOPK_ECUDA;
        int rc = retopk_decode_step(c, c->stage_q, k_cache, v_cache, seq_len, out_dev, stream);
        if (rc != RETOPK_OK) return rc;
        c->last_launches += 1;
        return cudaStreamSynchronize(s) == cudaSuccess ? RETOPK_OK : RETOPK_ECUDA;
    }
    if (cudaMemcpyAsync(c->stage_q, q_host, nq, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return RETOPK_ECUDA;
    // append the current token's key / value row of every (sequence, KV head)
    const size_t pitch = (size_t)c->max_seq_len * row;
    char* kdst = static_cast<char*>(k_cache) + (size_t)(seq_len - 1) * row;
    char* vdst = static_cast<char*>(v_cache) + (size_t)(seq_len - 1) * row;
    if (cudaMemcpy2DAsync(kdst, pitch, k_new_host, row, row, nkv, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpy2DAsync(vdst, pitch, v_new_host, row, row, nkv, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return RETOPK_ECUDA;
    int rc = retopk_decode_step(c, c->stage_q, k_cache, v_cache, seq_len, c->stage_out, stream);
    if (rc != RETOPK_OK) return rc;
    if (cudaMemcpyAsync(out_host, c->stage_out, nq, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return RETOPK_ECUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_stats(retopk_ctx* c, retopk_stats_t* st) {
    if (!c || !st) return RETOPK_EINVAL;
    DeviceGuard g(c->device);
    const size_t nh = (size_t)c->B * c->Hq;
    unsigned long long* host = new (std::nothrow) unsigned long long[nh * 4];
    if (!host) return RETOPK_ENOMEM;
    unsigned int status = 0;
    unsigned long long slow = 0, groups = 0;
    bool ok = cudaDeviceSynchronize() == cudaSuccess &&
              cudaMemcpy(&groups, c->scan_groups, sizeof groups, cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemcpy(host, c->counters, nh * 4 * sizeof(unsigned long long), cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemcpy(&status, c->status, sizeof status, cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemcpy(&slow, c->slow_select, sizeof slow, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (ok) {
        memset(st, 0, sizeof *st);
        for (size_t i = 0; i < nh; ++i) {
            st->reuse += (int64_t)host[i * 4 + 0];
            st->fallback += (int64_t)host[i * 4 + 1];
            st->refresh += (int64_t)host[i * 4 + 2];
            st->cand_sum += (int64_t)host[i * 4 + 3];
        }
        st->steps = st->reuse + st->fallback + st->refresh;
        st->slow_select = (int64_t)slow;
        st->scan_groups = (int64_t)groups;
        st->status = status;
    }
    delete[] host;
    return ok ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_last_step(retopk_ctx* c, int32_t* support, uint8_t* path, float* rho_max, int32_t* n_cand,
                     void* stream) {
    if (!c || !on_ctx_device(c)) return RETOPK_EINVAL;
    if (c->n_ins < 1) return RETOPK_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t nh = (size_t)c->B * c->Hq;
    bool ok = true;
    if (support) {
        const int slot = (int)((c->n_ins - 1) % c->M);
        const size_t width = (size_t)c->K * 4;
        ok = ok && cudaMemcpy2DAsync(support, width, c->sup_cache + (size_t)slot * c->K,
                                     (size_t)c->M * width, width, nh, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    }
    if (path) ok = ok && cudaMemcpyAsync(path, c->ws_path, nh, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    if (rho_max) ok = ok && cudaMemcpyAsync(rho_max, c->ws_rho, nh * 4, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    if (n_cand) ok = ok && cudaMemcpyAsync(n_cand, c->ws_ncand, nh * 4, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    return ok ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_last_recall(retopk_ctx* c, int32_t* sel, void* stream) {
    if (!c || !sel || c->n_ins < 1 || !on_ctx_device(c)) return RETOPK_EINVAL;
    const size_t bytes = (size_t)c->B * c->Hq * c->r * 4;
    return cudaMemcpyAsync(sel, c->ws_sel, bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_debug_candidates(retopk_ctx* c, int enable) {
    if (!c || (enable != 0 && enable != 1)) return RETOPK_EINVAL;
    DeviceGuard g(c->device);
    if (cudaDeviceSynchronize() != cudaSuccess) return RETOPK_ECUDA;
    if (enable && !c->dbg_cand) {
        const size_t n = (size_t)c->B * c->Hq * c->cap;
        if (cudaMalloc(reinterpret_cast<void**>(&c->dbg_cand), n * 4 > 0 ? n * 4 : 16) != cudaSuccess) {
            cudaGetLastError();
            c->dbg_cand = nullptr;
            return RETOPK_ENOMEM;
        }
    } else if (!enable && c->dbg_cand) {
        cudaFree(c->dbg_cand);
        c->dbg_cand = nullptr;
    }
    return RETOPK_OK;
}

int retopk_last_candidates(retopk_ctx* c, int32_t* cand, void* stream) {
    if (!c || !cand || !c->dbg_cand || c->n_ins < 1 || !on_ctx_device(c)) return RETOPK_EINVAL;
    const size_t bytes = (size_t)c->B * c->Hq * c->cap * 4;
    return cudaMemcpyAsync(cand, c->dbg_cand, bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_export_state(retopk_ctx* c, float* qbar, int32_t* supports, int64_t* n_inserted,
                        int64_t* t_dec, void* stream) {
    if (!c || !on_ctx_device(c)) return RETOPK_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t nh = (size_t)c->B * c->Hq;
    bool ok = true;
    if (qbar && c->qbar_bf16) {
        widen_kernel<<<c->num_sms * 4, 256, 0, s>>>(c->qbar16, qbar, nh * c->M * c->d);
        ok = ok && cudaGetLastError() == cudaSuccess;
    } else if (qbar) {
        ok = ok && cudaMemcpyAsync(qbar, c->qbar_cache, nh * c->M * c->d * 4, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    }
    if (supports) ok = ok && cudaMemcpyAsync(supports, c->sup_cache, nh * c->M * c->K * 4, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    if (n_inserted) *n_inserted = c->n_ins;
    if (t_dec) *t_dec = c->t_dec;
    return ok ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_import_state(retopk_ctx* c, const float* qbar, const int32_t* supports, int64_t n_inserted,
                        int64_t t_dec, void* stream) {
    if (!c || !qbar || !supports || n_inserted < 0 || t_dec < 0 || !on_ctx_device(c)) return RETOPK_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t nh = (size_t)c->B * c->Hq;
    bool ok;
    if (c->qbar_bf16) {
        narrow_kernel<<<c->num_sms * 4, 256, 0, s>>>(qbar, c->qbar16, nh * c->M * c->d);
        ok = cudaGetLastError() == cudaSuccess;
    } else {
        ok = cudaMemcpyAsync(c->qbar_cache, qbar, nh * c->M * c->d * 4, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    }
    ok = ok &&
              cudaMemcpyAsync(c->sup_cache, supports, nh * c->M * c->K * 4, cudaMemcpyDeviceToDevice, s) == cudaSuccess;
    c->n_ins = n_inserted;
    c->t_dec = t_dec;
    return ok ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_profile_begin(retopk_ctx* c, int max_calls) {
    if (!c || max_calls < 1 || c->prof_events) return RETOPK_EINVAL;
    DeviceGuard g(c->device);
    cudaEvent_t* ev = new (std::nothrow) cudaEvent_t[(size_t)max_calls * 4];
    unsigned char* kind = new (std::nothrow) unsigned char[max_calls];
    int made = 0, rc = (ev && kind) ? RETOPK_OK : RETOPK_ENOMEM;
    for (; rc == RETOPK_OK && made < max_calls * 4; ++made)
        if (cudaEventCreate(&ev[made]) != cudaSuccess) { cudaGetLastError(); rc = RETOPK_ECUDA; break; }
    if (rc != RETOPK_OK) {         // nothing is kept of a half-made set
        for (int i = 0; i < made; ++i) cudaEventDestroy(ev[i]);
        delete[] ev;
        delete[] kind;
        return rc;
    }
    c->prof_events = ev;
    c->prof_kind = kind;
    c->prof_max = max_calls;
    c->prof_calls = 0;
    return RETOPK_OK;
}

int retopk_profile_end(retopk_ctx* c, double ms_host[3], int64_t launches_host[3]) {
    if (!c || !c->prof_events || !ms_host || !launches_host) return RETOPK_EINVAL;
    DeviceGuard g(c->device);
    bool ok = cudaDeviceSynchronize() == cudaSuccess;
    for (int j = 0; j < 3; ++j) { ms_host[j] = 0.0; launches_host[j] = 0; }
    for (int i = 0; ok && i < c->prof_calls; ++i) {
        cudaEvent_t* e = c->prof_events + (size_t)i * 4;
        for (int j = (c->prof_kind[i] == 1 ? 1 : 0); j < 3; ++j) {
            float ms = 0.f;
            ok = ok && cudaEventElapsedTime(&ms, e[j], e[j + 1]) == cudaSuccess;
            ms_host[j] += ms;
            launches_host[j] += 1;
        }
    }
    for (int i = 0; i < c->prof_max * 4; ++i) cudaEventDestroy(c->prof_events[i]);
    delete[] c->prof_events;
    delete[] c->prof_kind;
    c->prof_events = nullptr;
    c->prof_kind = nullptr;
    c->prof_max = c->prof_calls = 0;
    return ok ? RETOPK_OK : RETOPK_ECUDA;
}

int retopk_last_launch_count(const retopk_ctx* c) { return c ? c->last_launches : 0; }

// ---------------------------------------------------------------------------------------
// Exact Top-K attention for callers that may not allocate.
//
// The score workspace lives in this fixed array instead of cudaMalloc'ed memory.  In host
// code the name `g_static_scratch` is only a handle for the runtime, not a device address:
// the address every kernel gets is looked up once per device with cudaGetSymbolAddress
// while that device is current.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[RETOPK_STATIC_SCRATCH_BYTES];

namespace {
constexpr int STATIC_MAX_DEVICES = 64;
struct StaticSetup {
    bool ready;
    unsigned char* scratch;      // device address of g_static_scratch on this device
    int num_sms, max_smem;
    int occ[2][2];               // scan CTAs per SM for d in {64,128} x head tiles in {1,2}
};
StaticSetup g_static_setup[STATIC_MAX_DEVICES];
std::mutex g_static_mutex;       // host threads may race for the first call on a device

// First use on the current device: resolve the array's address, opt in to large shared memory.
int static_setup(int dev, StaticSetup** out) {
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return RETOPK_EUNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup* st = &g_static_setup[dev];
    if (!st->ready) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return RETOPK_ECUDA; }
        st->scratch = static_cast<unsigned char*>(p);
        if (cudaDeviceGetAttribute(&st->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&st->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return RETOPK_ECUDA;
        if (cudaFuncSetAttribute(finish_kernel<128, 1024, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, st->max_smem) != cudaSuccess ||
            cudaFuncSetAttribute(finish_kernel<64, 1024, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, st->max_smem) != cudaSuccess)
            return RETOPK_ECUDA;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&st->occ[0][0], scan_kernel<64, 1>, SCAN_THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&st->occ[0][1], scan_kernel<64, 2>, SCAN_THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&st->occ[1][0], scan_kernel<128, 1>, SCAN_THREADS, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&st->occ[1][1], scan_kernel<128, 2>, SCAN_THREADS, 0);
        st->ready = true;
    }
    *out = st;
    return RETOPK_OK;
}
}  // namespace

int exact_topk_decode_static(int B, int H_q, int H_kv, int d, int K, int64_t max_seq_len, const void* q,
                             const void* k_cache, const void* v_cache, int64_t seq_len, void* out,
                             int32_t* idx_out, void* stream) {
    if (!q || !k_cache || !v_cache || !out) return RETOPK_EINVAL;
    if (B < 1 || H_q < 1 || H_kv < 1 || H_q % H_kv != 0 || K < 1 || max_seq_len < 1 || seq_len < 1 ||
        seq_len > max_seq_len)
        return RETOPK_EINVAL;
    if ((d != 64 && d != 128) || H_q / H_kv > 16 || K > 4096 || max_seq_len > 1048576 ||
        (long long)B * H_kv > MAX_GROUPS)
        return RETOPK_EUNSUPPORTED;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache)) return RETOPK_EINVAL;

    // does the shape fit the fixed array?  (256 bytes of counters, then scores, then tile maxima)
    const long long nh = (long long)B * H_q;
    const long long score_stride = (max_seq_len + TILE_ROWS - 1) / TILE_ROWS * TILE_ROWS;
    const long long tmax_stride = ((max_seq_len + TILE_ROWS - 1) / TILE_ROWS + 3) / 4 * 4;
    const long long need = 256 + nh * (score_stride + tmax_stride) * 4;
    if (need > (long long)RETOPK_STATIC_SCRATCH_BYTES) return RETOPK_ETOOLARGE;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return RETOPK_ECUDA;
    StaticSetup* st = nullptr;
    int rc = static_setup(dev, &st);
    if (rc != RETOPK_OK) return rc;

    int NS = 0, tile_cap = 0;
    exact_list_sizes(K, false, &NS, &tile_cap);
    int depth = 1;
    const size_t smem = exact_smem(K, NS, tile_cap, d, FINISH_THREADS, (size_t)st->max_smem, 1, &depth);
    if (smem == 0) return RETOPK_EUNSUPPORTED;

    StepArgs a;
    memset(&a, 0, sizeof a);
    a.B = B; a.Hq = H_q; a.Hkv = H_kv; a.G = H_q / H_kv; a.d = d; a.M = 1; a.r = 1; a.W = 0; a.K = K; a.cap = K;
    a.max_seq_len = max_seq_len;
    a.score_stride = score_stride;
    a.tmax_stride = tmax_stride;
    a.L = (int)seq_len;
    a.scale = 1.0f / sqrtf((float)d);
    a.mode = MODE_EXACT;
    a.NS = NS;
    a.tile_cap = tile_cap;
    a.g_shift = (a.G & (a.G - 1)) == 0 ? __builtin_ctz((unsigned)a.G) : -1;
    a.exact_stage_depth = (int)depth;
    a.q = static_cast<const uint16_t*>(q);
    a.k = static_cast<const uint16_t*>(k_cache);
    a.v = static_cast<const uint16_t*>(v_cache);
    a.out = static_cast<uint16_t*>(out);
    a.idx_out = idx_out;
    // the two diagnostic counters the kernels add to are sinks here; they need no clearing
    a.slow_select = reinterpret_cast<unsigned long long*>(st->scratch);
    a.scan_groups = reinterpret_cast<unsigned long long*>(st->scratch + 8);
    a.scan_counter = reinterpret_cast<unsigned int*>(st->scratch + 16);
    a.ws_scores = reinterpret_cast<float*>(st->scratch + 256);
    a.ws_tmax = a.ws_scores + nh * score_stride;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The scan's work counter is the one word of the array that must start at zero.  It is
    // cleared here in every call (a stream-ordered fill of four bytes: no allocation, no
    // synchronisation), so a call never depends on how an earlier one ended.
    if (cudaMemsetAsync(a.scan_counter, 0, sizeof(unsigned int), s) != cudaSuccess) return RETOPK_ECUDA;
    const int ntile = (a.G + 7) / 8;
    const int occ = st->occ[d == 128][ntile - 1];
    const long long items = (long long)B * H_kv * ((a.L + SCAN_TILE_ROWS - 1) / SCAN_TILE_ROWS);
    const long long cap_grid = (long long)st->num_sms * (occ > 0 ? occ : 2);
    const unsigned grid = (unsigned)(items < cap_grid ? items : cap_grid);
    if (d == 128 && ntile == 1) scan_kernel<128, 1><<<grid, SCAN_THREADS, 0, s>>>(a);
    else if (d == 128) scan_kernel<128, 2><<<grid, SCAN_THREADS, 0, s>>>(a);
    else if (ntile == 1) scan_kernel<64, 1><<<grid, SCAN_THREADS, 0, s>>>(a);
    else scan_kernel<64, 2><<<grid, SCAN_THREADS, 0, s>>>(a);
    if (cudaGetLastError() != cudaSuccess) return RETOPK_ECUDA;
    const int cluster = auto_cluster(nh, st->num_sms);
    a.cl_shift = __builtin_ctz((unsigned)cluster);
    if (d == 128) return launch_dependent(finish_kernel<128, 1024, false>, (unsigned)(nh * cluster), FINISH_THREADS, smem, s, a, 0, cluster);
    return launch_dependent(finish_kernel<64, 1024, false>, (unsigned)(nh * cluster), FINISH_THREADS, smem, s, a, 0, cluster);
}

#ifdef RETOPK_PHASE_CLOCKS
// Measurement aid, only in a library built with -DRETOPK_PHASE_CLOCKS (the benchmark's --phases
// flag builds one): copy the phase clock table [3][1024][RETOPK_PHASE_SLOTS] to the host.
int retopk_debug_read_phases(long long* host) {
    cudaDeviceSynchronize();
    return cudaMemcpyFromSymbol(host, g_phase_clk, sizeof(long long) * 3 * 1024 * RETOPK_PHASE_SLOTS) == cudaSuccess ? 0 : -4;
}
#endif

const char* retopk_strerror(int code) {
    switch (code) {
        case RETOPK_OK: return "ok";
        case RETOPK_EINVAL: return "invalid argument";
        case RETOPK_EUNSUPPORTED: return "configuration not supported by this build";
        case RETOPK_ENOMEM: return "device memory allocation failed";
        case RETOPK_ECUDA: return "CUDA runtime call or kernel launch failed";
        case RETOPK_ETOOLARGE: return "shape exceeds the fixed scratch array of exact_topk_decode_static";
        default: return "unknown error";
    }
}

}  // extern "C"
