/*
 * retopk.h - C interface of the ReTopK decode-step library (CUDA, sm_100a).
 *
 * One call of retopk_decode_step() is one attention layer's decode step for a batch of
 * B independent sequences: per query head it recalls the supports of the most similar
 * cached queries, reranks the compact candidate set with exact current-query scores,
 * attends over the K winners, falls back to full-history Exact Top-K when similarity is
 * low or a refresh is due, and inserts the new (query, support) pair into its cache
 * (Sec. 3.3 "Recall-Before-Rerank Selection", Sec. 3.4 "Reliable Reuse via Fallback and
 * Refresh").  exact_topk_decode() is the paper's Exact Top-K attention (Sec. 3.2, Eq. 4,
 * Eq. 1, Eq. 12), the comparator and the fallback path.
 *
 * Names: M = cache capacity (the paper's C), r = recalled entries (the paper's R),
 * W = recent window, K = support size, tau = similarity threshold, R = refresh period in
 * decode steps (the paper's T_r; 0 disables refresh).
 *
 * Conventions shared by every call
 *   - All tensor pointers are DEVICE pointers on the device that was current at
 *     retopk_create time, unless the argument name ends in _host.  Calls that enqueue work
 *     return RETOPK_EINVAL when another device is current.
 *   - bf16 tensors are raw 16-bit patterns, innermost dimension d contiguous:
 *       q, out           [B, H_q, d]
 *       k_cache, v_cache [B, H_kv, max_seq_len, d]
 *     Query head h reads KV head h / (H_q / H_kv).  Key indices are 0-based int32.
 *   - seq_len counts the keys available INCLUDING the current token: the caller appends
 *     k_t, v_t at position seq_len - 1 before the call.  The library never writes the
 *     KV cache (except retopk_decode_step_host, which performs that append itself).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work; none synchronises except where stated.  A context must be driven from
 *     one stream at a time.
 *   - The caller owns q / k_cache / v_cache / out; the context owns its cache state and
 *     workspaces, allocated once in create and released in destroy.  decode calls allocate
 *     nothing (the measurement-only fusion levels 1-3 of retopk_set_fusion_level excepted).
 *   - Return value: 0 on success, a negative RETOPK_E* code otherwise.  Inputs containing
 *     NaN or Inf give unspecified (but memory-safe) results.  The kernels never trap.
 */
#ifndef RETOPK_H
#define RETOPK_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct retopk_ctx retopk_ctx;

enum {
    RETOPK_OK = 0,
    RETOPK_EINVAL = -1,      /* bad argument (null pointer, size out of range) */
    RETOPK_EUNSUPPORTED = -2,/* legal but not built (d not 64/128, H_q/H_kv > 16, ...) */
    RETOPK_ENOMEM = -3,      /* device allocation failed in create */
    RETOPK_ECUDA = -4,       /* a CUDA runtime call or launch failed */
    RETOPK_ETOOLARGE = -5    /* the shape does not fit the fixed scratch of exact_topk_decode_static */
};

enum { RETOPK_PATH_REUSE = 0, RETOPK_PATH_FALLBACK = 1, RETOPK_PATH_REFRESH = 2 };

/* Bits of retopk_stats_t.status (sticky until retopk_reset). */
enum {
    RETOPK_STATUS_BAD_INDEX = 1u  /* a stored support held an index >= seq_len; it was skipped */
};

/* Counters since create/reset, summed over every (sequence, query head). */
typedef struct {
    int64_t steps;       /* head-steps taken = reuse + fallback + refresh */
    int64_t reuse;       /* Eq. 13 "otherwise" branch */
    int64_t fallback;    /* rho_max < tau (includes the empty cache) */
    int64_t refresh;     /* scheduled refresh (counted as refresh even if rho_max < tau) */
    int64_t cand_sum;    /* sum of candidate-set sizes |A_t| over reuse head-steps (Eq. 9) */
    int64_t slow_select; /* exact-path selections that needed the multi-pass fallback */
    int64_t scan_groups; /* (sequence, KV head) groups whose keys were scanned in full, summed over steps */
    uint32_t status;     /* RETOPK_STATUS_* bits */
    uint32_t reserved;
} retopk_stats_t;

#define RETOPK_DEFAULT_MAX_SEQ_LEN 139264  /* 128K context + 8K decode steps */

/*
 * Create a context for one sequence (B = 1) with the default max_seq_len.  The nine
 * parameters are the method's: head counts and head dim (Sec. 3.2), cache capacity M,
 * recall count r, window W, support size K (Sec. 3.3), threshold tau and refresh period
 * R (Sec. 3.4, Eq. 13).  The cache starts empty, so the first step takes the exact path.
 * Constraints: H_q % H_kv == 0, H_q / H_kv <= 16, d in {64, 128}, 1 <= r <= M <= 1024,
 * W >= 0, 1 <= K <= 4096, R >= 0; tau may be any float (<= -1 never falls back on
 * similarity, > 1 always does).
 */
int retopk_create(retopk_ctx** ctx, int H_q, int H_kv, int d, int M, int r, int W, int K,
                  float tau, int R);

/* Same, for B independent sequences sharing seq_len, and an explicit KV-cache row count
 * (max_seq_len fixes the k_cache / v_cache strides and the workspace sizes;
 * 1 <= max_seq_len <= 1048576). */
int retopk_create_batched(retopk_ctx** ctx, int B, int H_q, int H_kv, int d, int M, int r, int W,
                          int K, float tau, int R, int64_t max_seq_len);

/*
 * Recall rule.  RETOPK_RECALL_SIMILAR (default) is the method's Eq. 7: the r most similar
 * cached queries.  RETOPK_RECALL_RECENT is the component study's "Recent-R" row (Table 3):
 * the min(r, filled) most recently inserted entries are recalled instead and rho_max is the
 * largest similarity among those (the paper prints no formula for this row).
 */
enum { RETOPK_RECALL_SIMILAR = 0, RETOPK_RECALL_RECENT = 1 };
int retopk_set_recall_mode(retopk_ctx* ctx, int mode);

/*
 * Storage format of the cached normalised queries.  RETOPK_QBAR_FP32 (default) keeps them as
 * computed; RETOPK_QBAR_BF16 rounds every element once, to nearest even, to bf16 when it is
 * stored and halves the bytes the similarity search (Eq. 6) reads.  The paper runs in BF16
 * and does not say how its cached queries are kept; the similarity of a later step is the
 * dot product of that step's unrounded normalised query with the stored rounded entry.
 * Only while the cache is empty (after create or reset), else EINVAL; allocates the bf16
 * cache on first use (ENOMEM).  retopk_export_state / retopk_import_state keep their fp32
 * layout in both formats (values are widened / rounded on the way).
 */
enum { RETOPK_QBAR_FP32 = 0, RETOPK_QBAR_BF16 = 1 };
int retopk_set_qbar_format(retopk_ctx* ctx, int format);

/*
 * CTAs per (sequence, query head) in the finish kernel: 1, 2, 4 or 8.  With more than one, the
 * CTAs of a head form a thread-block cluster on as many SMs: each scores a share of the
 * candidate rows (Eq. 10) and fetches a share of the selected value rows (Eq. 12); keys and
 * partial sums cross through distributed shared memory.  The paper has no counterpart; it is
 * how a small batch uses the SMs that one CTA per head would leave idle.  retopk_create*
 * picks the largest size with B*H_q*size <= the SM count (1 from B*H_q = 75 up on B200).
 * Supports and decisions do not depend on the size; outputs differ in the last bits of the
 * fp32 sum order.  EINVAL for any other size; EUNSUPPORTED when the device cannot schedule a
 * cluster of that size for this context's kernels (checked here, not in the middle of a step).
 */
int retopk_set_cluster_size(retopk_ctx* ctx, int ctas_per_head);

/*
 * Block shape of the finish kernel: 1024 threads (one CTA per SM) or 512 (two CTAs per SM,
 * each with half of the SM's shared memory, so that the selection of one head overlaps the
 * row copies of another).  retopk_create* picks 512 when there are more heads than SMs and
 * the shape fits.  Results do not depend on the number of CTAs per SM; outputs differ between
 * the two shapes in the fp32 sum order only.  EUNSUPPORTED when the narrow shape does not fit
 * (large K or r*K+W, or a long max_seq_len), EINVAL for other values or below fusion level 5.
 */
int retopk_set_finish_threads(retopk_ctx* ctx, int threads);

/*
 * The same choice in full: (threads, CTAs per SM) is one of (1024, 1), (512, 2), (512, 1).
 * With one CTA per SM the CTA takes all of the SM's shared memory whatever its thread count;
 * fewer threads per head mean fewer issue slots spent on block-wide bookkeeping and more
 * work per thread.  retopk_set_finish_threads(512) is (512, 2).
 * EINVAL for other pairs or below fusion level 5, EUNSUPPORTED when the shape does not fit.
 */
int retopk_set_block_shape(retopk_ctx* ctx, int threads, int ctas_per_sm);

/*
 * Fusion level of the reuse path, for measuring what kernel fusion buys (the paper's kernel
 * efficiency analysis, Table 4, reports five cumulative stages for its own kernels; the cut
 * points here follow its description of them and are this library's own).  Results do not
 * depend on the level: supports and outputs are bit-identical.
 *   1  separate kernels: similarity | top-r and path | candidate union | pack candidate key
 *      rows | score packed rows | top-K | softmax.V | cache insert
 *   2  one kernel for cache search + support union; candidate rows scored through their indices
 *   3  top-K, softmax.V and the support insert in one kernel
 *   4  as 3, the intermediate buffers owned by the context; levels 1-3 take them from a
 *      stream-ordered memory pool (created on first use, blocks kept between steps) and give
 *      them back in every step
 *   5  candidate union through output in one kernel (the default)
 * dependent_launches = 1 (default, only valid with level 5) launches the step's kernels with
 * programmatic stream serialisation, 0 as plain stream-ordered launches.  Heads on the exact
 * path run scan + finish at every level.  Levels below 5 allocate device memory: level 4 in
 * this call (about B*H_q*(2*(r*K+W)) words), levels 1-3 from the pool inside
 * retopk_decode_step, which then must not run under stream capture.  This call
 * synchronises the device.  Errors: EINVAL (bad level / flag), EUNSUPPORTED (a kernel of the
 * level does not fit shared memory), ENOMEM, ECUDA.
 */
int retopk_set_fusion_level(retopk_ctx* ctx, int level, int dependent_launches);

/* Release the context and its device memory (synchronises the device). */
int retopk_destroy(retopk_ctx* ctx);

/* Empty every cache, set the decode offset t_dec to 0 and clear the counters. */
int retopk_reset(retopk_ctx* ctx, void* stream);

/*
 * One ReTopK decode step (Sec. 3.3-3.4: Eq. 6-13 and the cache insert) for all B * H_q
 * heads.  q, k_cache, v_cache are read, out is written; 1 <= seq_len <= max_seq_len.
 * The path of each head is decided on the device; no host synchronisation happens.
 * Advances t_dec and the insert count by one.  Three launches: the recall kernel (similarity
 * search, decision, insert of the normalised query), the full-history scan of the flagged KV
 * groups (leaves at once when no head fell back), and the finish kernel with heads of both
 * paths side by side.  If a launch fails after the first kernel of the step was enqueued, the
 * caches are half advanced: the call returns RETOPK_ECUDA and so does every later step of
 * this context until retopk_reset.
 */
int retopk_decode_step(retopk_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                       int64_t seq_len, void* out, void* stream);

/*
 * Seed the caches from the end of the prompt (Sec. 3.3, cache paragraph: the cache starts
 * from the last C prompt tokens).  q_tail [n_tail,B,H_q,d] (device) holds the queries
 * of prompt positions prompt_len - n_tail .. prompt_len - 1, oldest first; k_cache / v_cache
 * hold the prompt's keys and values.  Entry j gets the normalised query of its position p and
 * the CAUSAL Exact Top-K support over keys 0..p (Eq. 1 with L = p + 1; the paper leaves the
 * supports of prompt tokens undefined).  1 <= n_tail <= min(M, prompt_len).  The insert count
 * advances by n_tail, the decode offset t_dec and the counters do not change.  Costs n_tail
 * full-history scans: a one-off at the end of prefill.
 */
int retopk_prefill(retopk_ctx* ctx, const void* q_tail, const void* k_cache, const void* v_cache,
                   int64_t prompt_len, int n_tail, void* stream);

/*
 * The same step for a caller whose per-token tensors live in HOST memory: copies q_host
 * [B,H_q,d] to the device, appends k_new_host / v_new_host [B,H_kv,d] at position
 * seq_len - 1 of the device-resident k_cache / v_cache, runs the step, copies the result
 * to out_host [B,H_q,d] and synchronises `stream`.  When all four host buffers are pinned
 * and mapped (cudaHostAlloc / cudaHostRegister memory, 16-byte aligned) no copy is enqueued:
 * one small kernel reads q and the new rows straight from host memory and the last kernel
 * stores the output rows to out_host.  Otherwise the tensors go through staged copies
 * (pageable buffers work but serialise).
 */
int retopk_decode_step_host(retopk_ctx* ctx, const void* q_host, const void* k_new_host,
                            const void* v_new_host, void* k_cache, void* v_cache,
                            int64_t seq_len, void* out_host, void* stream);

/*
 * Exact Top-K attention (Eq. 4: score every key; Eq. 1: global Top-K, ties to the lower
 * index; Eq. 12: softmax . V over the support) for all B * H_q heads.  Stateless with
 * respect to the caches (uses the context only for shapes and workspaces).
 * idx_out: device int32 [B,H_q,K], ascending, -1 padded when seq_len < K; may be NULL.
 */
int exact_topk_decode(retopk_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                      int64_t seq_len, void* out, int32_t* idx_out, void* stream);

/* Copy the counters to host memory.  Synchronises the device. */
int retopk_stats(retopk_ctx* ctx, retopk_stats_t* stats_host);

/*
 * What the most recent retopk_decode_step did, per head (device pointers, any may be
 * NULL): support [B,H_q,K] int32 ascending (-1 padded), path [B,H_q] uint8
 * (RETOPK_PATH_*), rho_max [B,H_q] float (-inf for an empty cache), n_cand [B,H_q] int32
 * (|A_t| on reuse steps, seq_len otherwise).  Enqueued on `stream`.
 */
int retopk_last_step(retopk_ctx* ctx, int32_t* support, uint8_t* path, float* rho_max,
                     int32_t* n_cand, void* stream);

/*
 * The cache slots recalled by the most recent retopk_decode_step (Eq. 7), most similar
 * first: sel [B,H_q,r] int32 (device pointer), -1 where fewer than r entries were cached.
 * Written for every head, whatever path it then took.  Enqueued on `stream`.
 */
int retopk_last_recall(retopk_ctx* ctx, int32_t* sel, void* stream);

/*
 * Test hook (no counterpart in the paper): keep the candidate list A_t (Eq. 9) of every head
 * that reuses, so that a test can compare it element by element.  enable = 1 allocates a
 * buffer of B*H_q*(r*K+W) int32 (ENOMEM), enable = 0 frees it; both synchronise the device.
 * While it is off (the default) the finish kernel writes nothing extra.
 * retopk_last_candidates copies the buffer to cand [B,H_q,r*K+W] (device pointer): for a head
 * on the reuse path in the most recent step, its first n_cand entries (retopk_last_step) are
 * the list in ascending order; other rows are stale.  EINVAL while the hook is off.
 */
int retopk_debug_candidates(retopk_ctx* ctx, int enable);
int retopk_last_candidates(retopk_ctx* ctx, int32_t* cand, void* stream);

/*
 * Test hook (host side only; nothing on the device fails): the next launch of kernel `which`
 * (1: recall, 2: scan, 3: finish; 0 clears the request) is skipped and reported as a failed
 * launch, so that the error handling of retopk_decode_step can be exercised.
 */
int retopk_debug_fail_next_launch(retopk_ctx* ctx, int which);

/*
 * Cache state out / in (device pointers): qbar [B,H_q,M,d] float32 normalised queries,
 * supports [B,H_q,M,K] int32 (ascending, -1 padded); the entry inserted n-th sits in slot
 * n % M.  n_inserted and t_dec are host scalars.  Import replaces the whole state (this
 * is how a test re-seeds the caches from a reference each step); it does not touch the
 * counters.  Enqueued on `stream`.
 */
int retopk_export_state(retopk_ctx* ctx, float* qbar, int32_t* supports, int64_t* n_inserted,
                        int64_t* t_dec, void* stream);
int retopk_import_state(retopk_ctx* ctx, const float* qbar, const int32_t* supports,
                        int64_t n_inserted, int64_t t_dec, void* stream);

/*
 * Exact Top-K attention without a context and without any allocation (the paper has no
 * counterpart: this entry point exists for callers that must not allocate device memory).
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a region whose memory
 * is fully owned by another allocator (an inference server's arena, a framework's caching
 * allocator that forbids raw allocations), or in a plug-in that is only handed input and
 * output buffers.  retopk_create allocates the
 * score workspace with cudaMalloc; this call instead keeps its workspace in a fixed array
 * that is part of the library image (RETOPK_STATIC_SCRATCH_BYTES of device memory on every
 * GPU that loads the library, held until the process exits).
 *
 * Same computation and same results as exact_topk_decode (Eq. 4, Eq. 1, Eq. 12) for
 * q [B,H_q,d], k_cache / v_cache [B,H_kv,max_seq_len,d] -> out [B,H_q,d], idx_out [B,H_q,K]
 * or NULL; all device pointers, caller-owned.  Constraints as for retopk_create_batched.
 * The workspace holds B * H_q rows of max_seq_len scores plus their tile maxima, so
 *     B * H_q * (ceil16(max_seq_len) + ceil4(ceil(max_seq_len / 16))) * 4 + 256
 * must not exceed RETOPK_STATIC_SCRATCH_BYTES; larger shapes return RETOPK_ETOOLARGE and
 * nothing is launched.
 *
 * The first call on a device looks up the array's device address and opts the kernels in to
 * large shared memory; make that first call before any stream capture begins.  That set-up is
 * guarded by a lock, so host threads may race for it.  No call allocates, frees or
 * synchronises.  All calls on a device share the one array, which keeps the last call's
 * contents: scores and tile maxima are rewritten by every call before they are read, and the
 * one word that must start at zero (the scan's work counter) is cleared on the stream at the
 * start of every call, so a call does not depend on how an earlier one ended.  Two calls that
 * overlap on the GPU (different streams, no dependency) race on the array.
 */
#define RETOPK_STATIC_SCRATCH_BYTES (32u << 20)
int exact_topk_decode_static(int B, int H_q, int H_kv, int d, int K, int64_t max_seq_len, const void* q,
                             const void* k_cache, const void* v_cache, int64_t seq_len, void* out,
                             int32_t* idx_out, void* stream);

/*
 * Measurement hooks (no counterpart in the paper).  Between begin and end, every decode
 * call of this context brackets each of its kernels with CUDA events on the call's stream
 * (up to max_calls calls; later calls run unrecorded).  retopk_profile_end synchronises
 * the device and returns, per kernel slot {0: recall, 1: scan, 2: finish}, the summed
 * device time in milliseconds and the number of launches.  Not for use
 * inside a timed region: the events themselves cost a little, and an event between two
 * kernels keeps the second from starting early.  A failed begin keeps nothing allocated.
 */
int retopk_profile_begin(retopk_ctx* ctx, int max_calls);
int retopk_profile_end(retopk_ctx* ctx, double ms_host[3], int64_t launches_host[3]);

/* Number of kernels the last decode call of this context launched (host-side count). */
int retopk_last_launch_count(const retopk_ctx* ctx);

/* Static description of an error code. */
const char* retopk_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* RETOPK_H */
