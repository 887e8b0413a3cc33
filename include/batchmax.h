/*
 * batchmax.h -- C ABI of libbatchmax: attention with KV-cache eviction during
 * prefilling and decoding (Batch-Max, arXiv 2412.05693) on one NVIDIA B200.
 *
 * Notation (Sec. 3 of the paper unless noted):
 *   b        batch size (samples processed in parallel)
 *   Hq, Hkv  query heads / KV heads, g = Hq / Hkv (g = 1 is plain multi-head)
 *   d        head dimension
 *   K        kv_max: size every (sample, kv-head) cache is cut back to by an
 *            eviction.  Algorithm 1's limit \overline{|kv|} is K + p, its
 *            eviction amount p is the growth allowed above K.
 *   I        number of inputs (queries) in one forward pass; I = 1 in decoding
 *   n        current number of KV pairs in a cache; n <= cap = K + growth
 *   kv_ids, sum_weights, curr_id   as in Sec. 3.2
 *
 * General rules
 *   - Every pointer argument is labelled HOST or DEVICE.  DEVICE pointers must
 *     belong to cfg.device, be 16-byte aligned, and are only borrowed for the
 *     stream-ordered duration of the call.  The library never allocates or
 *     frees device memory: the cache lives in a caller-owned arena, per-call
 *     scratch in a caller-owned workspace.
 *   - Calls validate on the host, enqueue kernels on `cuda_stream`
 *     (a cudaStream_t passed as void*, NULL = the legacy default stream) and
 *     return without synchronising, except where stated.
 *   - Every function returns a bm_status_t; nothing throws, aborts or traps.
 *     Every check of the arguments and of the cache state runs before the first launch: on any non-BM_OK return
 *     other than BM_ERR_CUDA nothing was enqueued and the cache is unchanged.  BM_ERR_CUDA (a launch or copy was
 *     refused by the runtime) can come after part of the call was enqueued: the state of the call's sample range is
 *     then undefined (see bm_last_cuda_error).
 *   - A handle is not thread-safe; distinct handles are independent.  One host thread may keep calls on disjoint
 *     sample ranges of one handle in flight on different streams at the same time (the caches of different samples
 *     are independent, and a range's scratch has its own place in the workspace) as long as max_call_samples
 *     covers the batch (0 does) and the calls are not the *_static or *_host variants; calls that touch the same
 *     sample must be ordered by the caller (same stream, or events).
 *   - All (sample, kv-head) caches of one (layer, sample) hold the same n, and
 *     n after a call is a function of n before, I and evict_to only, so the
 *     library mirrors n and curr_id on the host and never reads them back.
 */
#ifndef BATCHMAX_H_
#define BATCHMAX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bm_cache bm_cache_t; /* opaque, owned by the library */

typedef enum {
  BM_OK = 0,
  BM_ERR_INVALID = 1,  /* null / negative / misaligned argument, unsupported shape        */
  BM_ERR_OOM = 2,      /* arena, workspace or budget too small                            */
  BM_ERR_CAPACITY = 3, /* the call would make n exceed cap, or too many candidates        */
  BM_ERR_STATE = 4,    /* pos0 does not follow curr_id, or the sample range has unequal n */
  BM_ERR_CUDA = 5,     /* a CUDA runtime or driver call failed                            */
  BM_ERR_TIMEOUT = 6,  /* a bounded device-side wait expired (see bm_cache_status)        */
  BM_ERR_BOUNDS = 7    /* checked build only: a kernel met a row index outside its cache  */
} bm_status_t;

typedef enum { BM_F32 = 0, BM_BF16 = 1 } bm_dtype_t;

/* Eviction rule.  BM_RULE_AVERAGE is the method's own (Sec. 3.2).  The other two are the rules Sec. 2 ascribes to
 * earlier methods, as far as that section describes them, run on the same kernels:
 *   BM_RULE_SUM_RECENT    (H2O): the cache is split evenly between a window of the most recent pairs and the pairs
 *                         with the largest sum of past attention weights -- the floor(target / 2) most recent
 *                         candidates always stay, the others are ranked by their raw sum_weights;
 *   BM_RULE_CURRENT_QUERY (TOVA): pairs are ranked by the attention weights of the current query alone --
 *                         sum_weights is overwritten (not accumulated) with the weights of the block's last
 *                         query, or of the decode step's query, summed over the group's heads.
 *   BM_RULE_WINDOW_POOLED (SnapKV): a window of recent pairs stays -- the min(window, target) most recent candidates --
 *                         and the others are ranked by the attention weights summed over the last `window` queries:
 *                         sum_weights is overwritten by every pass with the column sums over its last min(window, I)
 *                         inputs (a decode step: its one query), and at an eviction every score is replaced by the
 *                         maximum over the `pool` neighbouring candidates centred on it (cache order, the window left
 *                         out), so that kept positions come in runs.  Pooling by maximum and both widths are this
 *                         library's parameters: the paper names the pooling layer without describing it.
 *   BM_RULE_AVERAGE_STD   (RoCo; also Sec. 3.2, last paragraph): the kept pairs are split between the
 *                         floor(target * std_share_permille / 1000) pairs whose attention weights have the largest
 *                         standard deviation, sqrt(E[w^2] - E[w]^2) over the g * (curr_id + 1 - kv_ids) weights a pair
 *                         has received, and the largest ave_weights among the rest.  The cache keeps one more fp32
 *                         per row (the sum of squared weights: 4 more bytes per row in the memory model).  Not
 *                         available with left padding or through bm_prefill_block_static.
 * Ties keep the lower position under every rule.  The last two rank by the rows' position order and need
 * BM_COMPACT_STABLE. */
typedef enum { BM_RULE_AVERAGE = 0, BM_RULE_SUM_RECENT = 1, BM_RULE_CURRENT_QUERY = 2, BM_RULE_WINDOW_POOLED = 3,
               BM_RULE_AVERAGE_STD = 4 } bm_rule_t;

/* What the removal step of Algorithm 1 does to the rows of a cache.  Attention, the scores and the kept sets do not
 * depend on the order of a cache's rows; only the work of removing does.
 *   BM_COMPACT_STABLE: rows stay in ascending kv_ids order; the rows behind a pair that leaves move up.
 *   BM_COMPACT_FILL:   rows are an unordered set: a pair that stays never moves, the pairs that arrive (the block's
 *                      kept pairs, the decode step's pair) take the rows that were freed.  Kept sets, sum_weights and
 *                      outputs are the same as under BM_COMPACT_STABLE (ties still keep the lower position, decided
 *                      on kv_ids; the recent window of BM_RULE_SUM_RECENT and bm_keep_most_recent rank by kv_ids);
 *                      bm_cache_export returns the rows in storage order. */
typedef enum { BM_COMPACT_STABLE = 0, BM_COMPACT_FILL = 1 } bm_compaction_t;

/* Problem statement: Algorithm 1's inputs (\overline{|kv|}, p) generalised as (K, growth), plus the
 * attention shape.  All sizes in elements. */
typedef struct {
  int32_t batch;            /* b                                                              */
  int32_t n_layers;         /* L independent attention layers sharing the handle              */
  int32_t n_q_heads;        /* Hq                                                             */
  int32_t n_kv_heads;       /* Hkv, must divide Hq; g = Hq / Hkv <= 8                         */
  int32_t head_dim;         /* d: 64 or 128                                                   */
  int32_t kv_max;           /* K >= 1                                                         */
  int32_t block_max;        /* largest I any bm_prefill_block call will pass, >= 1            */
  int32_t growth;           /* G >= 1: rows above K a cache may hold between evictions        */
  int32_t dtype;            /* bm_dtype_t of q/k/v/out and of the cached rows                 */
  float softmax_scale;      /* 0 selects 1/sqrt(d)                                            */
  int32_t device;           /* CUDA device ordinal                                            */
  int32_t max_call_samples; /* largest nsamples of any call (sizes the workspace); 0 -> batch */
  int32_t rule;             /* bm_rule_t: what pairs are ranked by at an eviction; 0 = the paper's  */
  int32_t compaction;       /* bm_compaction_t: 0 = rows stay in position order                     */
  int32_t window;           /* BM_RULE_WINDOW_POOLED: queries observed = recent pairs kept, >= 1     */
  int32_t pool;             /* BM_RULE_WINDOW_POOLED: width of the max-pooling, odd, 1 .. 255 (1 = none) */
  int32_t std_share_permille; /* BM_RULE_AVERAGE_STD: share of the kept pairs chosen by deviation, 0 .. 1000 */
} bm_config_t;

/* ---- cache layout, allocator and memory model (Sec. 1: batch size under a fixed memory budget) ----
 * Per sample the arena holds, for every layer and kv-head, cap = K + growth rows of:
 * key (d elements), value (d elements), sum_weights (fp32) and kv_ids (int32):
 *     bytes_per_sample = L * Hkv * cap * (2 * d * elem_size + 8)      (+ 4 per row under BM_RULE_AVERAGE_STD).
 * The arena adds a fixed 1024-byte header (status word, alignment of the four slabs). */
bm_status_t bm_cache_bytes_per_sample(const bm_config_t* cfg /*HOST*/, size_t* bytes /*HOST out*/);
/* Arena size for cfg->batch samples. */
bm_status_t bm_arena_bytes(const bm_config_t* cfg /*HOST*/, size_t* bytes /*HOST out*/);
/* Largest batch whose arena fits in hbm_budget_bytes (cfg->batch is ignored); 0 if none fits. */
bm_status_t bm_max_batch(const bm_config_t* cfg /*HOST*/, size_t hbm_budget_bytes, int32_t* b /*HOST out*/);
/* Scratch of a handle: per call, the log-sum-exp of every query row and the new pairs' column sums, for calls of
 * up to max_call_samples samples and block_max inputs; plus one padding count per sample (bm_cache_set_left_pad). */
bm_status_t bm_workspace_bytes(const bm_config_t* cfg /*HOST*/, size_t* bytes /*HOST out*/);

/* Carve `arena` (DEVICE, 256-byte aligned, >= bm_arena_bytes) into the slabs
 * K,V: [L][b][Hkv][cap][d], sum_weights: fp32 [L][b][Hkv][cap], kv_ids: int32 [L][b][Hkv][cap],
 * zero it on `cuda_stream`, and return a handle with every cache empty (n = 0, curr_id = -1).
 * `workspace` (DEVICE, 256-byte aligned, >= bm_workspace_bytes) is used by every later call; calls that touch the
 * same samples must be stream-ordered with respect to each other (calls on disjoint sample ranges may overlap
 * under the conditions of the general rules above: each range has its own place in the workspace).
 * Both buffers stay owned by the caller and must outlive the handle.
 * Errors: BM_ERR_INVALID (bad config / null / misaligned), BM_ERR_OOM (a buffer is too small). */
bm_status_t bm_cache_create(const bm_config_t* cfg /*HOST*/, void* arena /*DEVICE*/, size_t arena_bytes,
                            void* workspace /*DEVICE*/, size_t workspace_bytes, void* cuda_stream,
                            bm_cache_t** out /*HOST out*/);
bm_status_t bm_cache_destroy(bm_cache_t* cache); /* frees the host handle only */

/* ---- the forward pass with a block of I inputs (Sec. 3.2; the block-processing step of Algorithm 1) ----
 * For samples sample0 .. sample0+nsamples-1 of `layer`: the I queries at positions pos0 .. pos0+I-1
 * attend to all n cached pairs and to the block's own pairs at positions <= their own (causal);
 *   out = softmax(scale * q k^T) v,      sum_weights += sum_i attn_weights[i]
 * (summed over the g query heads of each KV head; new pairs start from 0), the block's pairs join the
 * cache with kv_ids = their positions, curr_id becomes pos0+I-1.  Then, if evict_to >= 0 and
 * n + I > evict_to, the caches are cut back to evict_to pairs exactly as bm_evict does.
 *   q   DEVICE [nsamples][I][Hq][d]     k, v  DEVICE [nsamples][I][Hkv][d]    (contiguous, cfg.dtype)
 *   out DEVICE [nsamples][I][Hq][d]     (cfg.dtype)
 * The block's K/V are read from the caller's buffers (they are not staged in the cache first), so the
 * call needs min(n + I, evict_to if evicting) <= cap, not n + I <= cap.
 * Errors: BM_ERR_INVALID (range, I < 1, I > block_max, null, misaligned), BM_ERR_STATE (pos0 !=
 * curr_id + 1, or the samples of the range hold different n), BM_ERR_CAPACITY (the row limit above, more
 * than 12288 candidates per cache, or more than 65535 caches -- nsamples * Hkv -- in one call: split the
 * batch into sample ranges). */
bm_status_t bm_prefill_block(bm_cache_t* cache, int32_t layer, int32_t sample0, int32_t nsamples,
                             const void* q, const void* k, const void* v, int32_t I, int32_t pos0,
                             void* out, int32_t evict_to, void* cuda_stream);

/* ---- one decoding step (the generation step of Algorithm 1; Sec. 3.2: a block of one input) ----
 * Same as bm_prefill_block with I = 1 and pos0 = curr_id + 1, in one bandwidth-bound pass.
 *   q, out DEVICE [nsamples][Hq][d]     k, v DEVICE [nsamples][Hkv][d]
 * Needs n + 1 <= cap (the new pair is appended before an optional eviction). */
bm_status_t bm_decode_step(bm_cache_t* cache, int32_t layer, int32_t sample0, int32_t nsamples,
                           const void* q, const void* k, const void* v, void* out, int32_t evict_to,
                           void* cuda_stream);

/* ---- eviction (the removal step of Algorithm 1; Sec. 3.2 average-attention rule) ----
 * For every (sample, kv-head) of the range independently:
 *   ave_weights = sum_weights / (g * (curr_id + 1 - kv_ids));
 * keep the `target` pairs that rank first under (ave_weights descending, kv_ids ascending), move them
 * to the front of the cache in ascending kv_ids order together with their sum_weights and kv_ids,
 * n becomes target.  No-op when n <= target.  Errors: BM_ERR_INVALID (target < 0, range), BM_ERR_STATE. */
bm_status_t bm_evict(bm_cache_t* cache, int32_t layer, int32_t sample0, int32_t nsamples, int32_t target,
                     void* cuda_stream);

/* ---- the rule of the extreme decoding-only comparison (Algorithm 3: only the newest pair survives a cut) ----
 * Keep the `keep` most recent pairs of every cache of the range, moved to the front with their
 * sum_weights and kv_ids; n becomes keep.  No-op when n <= keep.  It exists so that the comparison arm
 * of the paper's experiments (Sec. 4, ED) runs on the same kernels and memory model as the method itself.
 * Errors as bm_evict. */
bm_status_t bm_keep_most_recent(bm_cache_t* cache, int32_t layer, int32_t sample0, int32_t nsamples,
                                int32_t keep, void* cuda_stream);

/* ---- bm_prefill_block for callers that cannot provide scratch (the paper has no counterpart) ----
 * Identical to bm_prefill_block in arguments, result and errors, but the per-call scratch (log-sum-exp of
 * the query rows, column sums of the new pairs) is taken from a fixed 5 MiB array that is part of the
 * library image on every GPU that loads it, instead of the workspace given to bm_cache_create.  It is
 * meant for callers that must not allocate device memory themselves: a serving loop whose memory plan is
 * frozen after start-up, a plug-in under a framework whose caching allocator owns the whole device, or a
 * thread that may not issue allocating CUDA calls.  The call itself calls no allocating routine.
 *   Limits: nsamples * Hq * I <= 1,048,576 and nsamples * Hkv * I <= 262,144, else BM_ERR_CAPACITY
 *   (nothing is enqueued); the limits of bm_prefill_block apply as well (nsamples <= max_call_samples,
 *   I <= block_max, at most 65535 caches per call).  cfg.device must be below 64.
 *   First call on a device: resolves the array's device address (cudaGetSymbolAddress with that device
 *   current).  Under the runtime's lazy module loading that first call is also what places the library's
 *   device code and with it the 5 MiB array in that GPU's memory -- an allocation in all but name -- so make
 *   it during start-up, and before starting any stream capture.  The table of resolved addresses is shared by
 *   all handles and threads of the process (concurrent first calls store the same value).
 *   Sharing: all handles and all calls on a device use the same array, and it keeps the previous call's
 *   contents.  Nothing in it has to start from zero (every entry a call reads is written by that call
 *   first), but two calls that overlap on the GPU -- different streams, or different handles without
 *   stream ordering -- race on it and corrupt each other's scores. */
bm_status_t bm_prefill_block_static(bm_cache_t* cache, int32_t layer, int32_t sample0, int32_t nsamples,
                                    const void* q, const void* k, const void* v, int32_t I, int32_t pos0,
                                    void* out, int32_t evict_to, void* cuda_stream);

/* ---- the same two passes fed from HOST memory (end-to-end use without device-side producers) ----
 * q/k/v/out are HOST pointers (pinned memory makes the copies asynchronous); `staging` is a DEVICE
 * buffer of at least bm_staging_bytes(cfg, nsamples, I) bytes.  The call copies q, k, v to the device,
 * runs the pass and copies out back to `out`; it does not synchronise.  The three stages run on streams
 * owned by the handle, so that the input copy, the pass and the output copy of consecutive calls overlap;
 * cuda_stream is made to wait for the call's output copy (synchronising cuda_stream makes `out` valid,
 * and later work on cuda_stream sees the updated cache).  The pipeline is ordered after cuda_stream's
 * position only where it has to be: at the first host-fed call and after any device-fed call on this
 * handle.  The input copies start at call time, so q/k/v must hold their final contents when the call
 * is made and until cuda_stream has passed the call.  Passing up to four staging buffers in turn keeps as
 * many calls in flight; a staging buffer is reused only after the earlier call that used it has finished
 * (tracked by the handle).  While cuda_stream is being captured into a CUDA graph everything stays on
 * cuda_stream. */
bm_status_t bm_staging_bytes(const bm_config_t* cfg /*HOST*/, int32_t nsamples, int32_t I, size_t* bytes);
bm_status_t bm_prefill_block_host(bm_cache_t* cache, int32_t layer, int32_t sample0, int32_t nsamples,
                                  const void* q /*HOST*/, const void* k /*HOST*/, const void* v /*HOST*/,
                                  int32_t I, int32_t pos0, void* out /*HOST*/, int32_t evict_to,
                                  void* staging /*DEVICE*/, size_t staging_bytes, void* cuda_stream);
bm_status_t bm_decode_step_host(bm_cache_t* cache, int32_t layer, int32_t sample0, int32_t nsamples,
                                const void* q /*HOST*/, const void* k /*HOST*/, const void* v /*HOST*/,
                                void* out /*HOST*/, int32_t evict_to, void* staging /*DEVICE*/,
                                size_t staging_bytes, void* cuda_stream);

/* ---- left-padded samples (Sec. 3: prompts of unequal length are padded on the left) ----
 * pads[s] = number of padding positions at the start of sample s (HOST array of cfg.batch entries; NULL or
 * all zeros switches padding off).  From then on, for sample s: a pair whose position id is below pads[s] is
 * masked for every real query, so its sum_weights stays 0, and it ranks below every real pair at an eviction
 * (padding leaves first, highest position first); a query at a padding position produces an all-zero output
 * row and adds nothing to sum_weights.  Padding pairs occupy cache rows like any other pair until they are
 * evicted, so n stays equal over the samples of a call.  The paper does not say how padding meets eviction;
 * this is the build's reading.  Must be called while every cache of the handle is empty, else BM_ERR_STATE;
 * negative entries give BM_ERR_INVALID.  The copy to the device is ordered on cuda_stream, like the calls
 * that use it. */
bm_status_t bm_cache_set_left_pad(bm_cache_t* cache, const int32_t* pads /*HOST*/, void* cuda_stream);

/* ---- state access ---- */
/* Host mirror of n and curr_id (-1 when empty) of one (layer, sample); no synchronisation. */
bm_status_t bm_cache_len(const bm_cache_t* cache, int32_t layer, int32_t sample, int32_t* n /*HOST out*/,
                         int32_t* curr_id /*HOST out, may be NULL*/);
/* Copy one (layer, sample, kv-head) cache to HOST arrays: kv_ids[n], sum_weights[n] and, when not
 * NULL, k_rows / v_rows [n][d] in cfg.dtype.  Synchronises cuda_stream before returning. */
bm_status_t bm_cache_export(bm_cache_t* cache, int32_t layer, int32_t sample, int32_t kv_head,
                            int32_t* kv_ids /*HOST out*/, float* sum_weights /*HOST out*/,
                            void* k_rows /*HOST out*/, void* v_rows /*HOST out*/, int32_t* n /*HOST out*/,
                            void* cuda_stream);
/* Inverse of bm_cache_export for checkpoint / resume: overwrite the first n rows of one
 * (layer, sample, kv-head) cache; n must equal the mirrored n of that sample (set it first with
 * bm_cache_set_len).  Synchronises cuda_stream before returning. */
bm_status_t bm_cache_import(bm_cache_t* cache, int32_t layer, int32_t sample, int32_t kv_head,
                            const int32_t* kv_ids /*HOST*/, const float* sum_weights /*HOST*/,
                            const void* k_rows /*HOST*/, const void* v_rows /*HOST*/, int32_t n,
                            void* cuda_stream);
/* The same for the sums of squared weights a cache keeps under BM_RULE_AVERAGE_STD (n entries, n = the sample's
 * mirrored length); BM_ERR_INVALID under any other rule.  Both synchronise cuda_stream. */
bm_status_t bm_cache_export_sum_sq(bm_cache_t* cache, int32_t layer, int32_t sample, int32_t kv_head,
                                   float* sum_sq /*HOST out*/, void* cuda_stream);
bm_status_t bm_cache_import_sum_sq(bm_cache_t* cache, int32_t layer, int32_t sample, int32_t kv_head,
                                   const float* sum_sq /*HOST*/, void* cuda_stream);
/* Set the mirrored n (0 <= n <= cap) and curr_id of one (layer, sample) when restoring a checkpoint. */
bm_status_t bm_cache_set_len(bm_cache_t* cache, int32_t layer, int32_t sample, int32_t n, int32_t curr_id);
/* Synchronise cuda_stream and read the device status word: BM_OK, or BM_ERR_TIMEOUT if a kernel gave
 * up a bounded wait (its results are then undefined; the context stays usable). */
bm_status_t bm_cache_status(bm_cache_t* cache, int32_t* device_status /*HOST out*/, void* cuda_stream);

/* Reset the device status word to BM_OK (stream-ordered). */
bm_status_t bm_cache_clear_status(bm_cache_t* cache, void* cuda_stream);
/* Failure-detection self-test (the paper has no counterpart): enqueue a one-warp kernel whose bounded wait can
 * never be satisfied.  It gives up after its poll limit, writes BM_ERR_TIMEOUT to the status word and ends
 * normally; bm_cache_status then reports BM_ERR_TIMEOUT and the context stays usable.  Nothing else is touched. */
bm_status_t bm_selftest_wait_timeout(bm_cache_t* cache, void* cuda_stream);

/* ---- the checked build (the paper has no counterpart) ----
 * libbatchmax_debug.so is the same library compiled with -DBM_DEBUG (python -m paper_2412_05693_b200.build --debug).
 * Its kernels test every cache row index they are about to write with plain stores against the cache's capacity; a
 * bad index is recorded as BM_ERR_BOUNDS in the device status word (bm_cache_status) and the access is skipped --
 * nothing traps, the context stays usable.  Its arena has a 256-byte guard behind every slab (the header grows to
 * 4096 bytes, so bm_arena_bytes / bm_max_batch differ from the ordinary build's); bm_cache_check_canaries counts the
 * guards that no longer hold their pattern (synchronises cuda_stream).  In the ordinary build bm_debug_build returns
 * 0 and there are no guards to damage. */
int32_t bm_debug_build(void);
/* Self-test of the row test: enqueue a one-thread kernel that asks it about the first row index past a cache (no
 * memory is touched).  In the checked build bm_cache_status then reports BM_ERR_BOUNDS (clear it with
 * bm_cache_clear_status); in the ordinary build the status word stays BM_OK. */
bm_status_t bm_selftest_row_check(bm_cache_t* cache, void* cuda_stream);
bm_status_t bm_cache_check_canaries(bm_cache_t* cache, int32_t* damaged /*HOST out*/, void* cuda_stream);

/* ---- rows moved by compactions (measurement aid: the compaction term of the decode step's memory traffic) ----
 * While switched on for a handle, every eviction adds the number of cache rows it moves (each row = one key and one
 * value row read and written) to counters in the arena's status block: the rows behind the first removed pair for
 * the stable compaction of bm_prefill_block / bm_evict, the rows behind the hole for the one-row shift of an
 * evicting decode step.  bm_cache_moved_rows returns the total so far (and clears it when reset != 0); it
 * synchronises cuda_stream. */
bm_status_t bm_cache_count_moved_rows(bm_cache_t* cache, int32_t on);
bm_status_t bm_cache_moved_rows(bm_cache_t* cache, uint64_t* rows /*HOST out*/, int32_t reset, void* cuda_stream);

/* ---- per-kernel timing (measurement aid; the paper has no counterpart) ----
 * While enabled, every kernel launch of this library is bracketed by two CUDA events on its stream.
 * bm_profile_read waits for the recorded launches of one kernel class, returns their summed duration in
 * milliseconds and their count, and forgets them.  Not thread-safe; leave disabled in production. */
enum { BM_KERNEL_ATTN_FWD = 0, BM_KERNEL_SCORE = 1, BM_KERNEL_EVICT = 2, BM_KERNEL_DECODE = 3 };
bm_status_t bm_profile_enable(int32_t on);
bm_status_t bm_profile_read(int32_t kernel_class, float* total_ms /*HOST out*/, int32_t* launches /*HOST out*/);

/* Number of kernels this library has launched in the calling process (monotone counter). */
uint64_t bm_kernel_launch_count(void);
/* Which attention implementation the last bm_prefill_block used: 0 = fp32 SIMT, 1 = tcgen05 bf16 (forward kernel,
 * then the score pass), 2 = tcgen05 bf16 with forward pass and column sums in one kernel (a block of at most 128
 * query rows, I * g, against at most four tiles of 128 keys, cached and new counted apart; no padding; not the
 * current-query rule). */
int32_t bm_last_prefill_path(void);
const char* bm_status_string(bm_status_t s);
/* Text of the CUDA error behind the calling thread's most recent BM_ERR_CUDA from a kernel launch ("no error" if
 * none).  After BM_ERR_CUDA the state of the call's sample range is undefined: some of the call's kernels may have
 * been enqueued; restore the range with bm_cache_import / bm_cache_set_len, or drop the handle. */
const char* bm_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* BATCHMAX_H_ */
