/*
 * kvfold.h - C ABI of the B200 (sm_100a) KV-Fold fold-step library.
 *
 * One `kvf_cache` is the accumulated K/V of ONE attention layer of ONE sequence:
 * the accumulator of the paper's left fold (Section 2, "A recurrent view":
 * (K,V)^(t) = F((K,V)^(t-1), x_t), started from the empty pair).  One call of
 * kvf_fold_step is the attention part of one application of F at that layer.
 *
 * Conventions that hold for every entry point
 *   - Device memory is never allocated or freed here.  The caller owns the cache
 *     storage, the workspace, q/k/v/out and the stream; the library owns only the
 *     host-side handle (and the TMA descriptors inside it).
 *   - "device pointer" below means memory of the CUDA device that was current when
 *     kvf_cache_create was called; the same device must be current at every later call.
 *   - Calls are stream-ordered and asynchronous: they enqueue work on `cuda_stream`
 *     (a cudaStream_t passed as void*, NULL = the default stream) and return.
 *   - Errors are return codes.  A call that returns an error has enqueued nothing and has
 *     changed neither the cache contents nor its length.  Nothing aborts or traps.  The one
 *     exception is KVF_ERR_CUDA from a fold step: the launch of one of the step's kernels was
 *     refused by the runtime after an earlier kernel of the same step (and, for the host and the
 *     static entry points, its copies or its memset) had been enqueued, so rows [len, len+n) of
 *     the planes may have been written; the length is unchanged, and repeating the step rewrites
 *     those rows.
 *   - A handle is not thread-safe; distinct handles are independent.  Several caches may
 *     share one workspace if all of their calls go to the same stream.
 *   - Results are deterministic: the same inputs, config and chunking give the same bits.
 */
#ifndef KVFOLD_H_
#define KVFOLD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvf_cache kvf_cache; /* opaque host-side handle */

typedef enum {
    KVF_OK = 0,
    KVF_ERR_INVALID_ARG = 1, /* null / misaligned pointer, n_tokens < 1 or > max_chunk, bad config */
    KVF_ERR_CAPACITY = 2,    /* len + n_tokens > capacity, or a buffer smaller than required     */
    KVF_ERR_UNSUPPORTED = 3, /* head_dim / head ratio / dtype outside what the kernels cover     */
    KVF_ERR_CUDA = 4,        /* a CUDA runtime or driver call failed (see kvf_last_cuda_error)   */
    KVF_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (read via kvf_cache_status)   */
    KVF_ERR_POS = 6,         /* KVF_STRICT_POS set and pos0 != current length                    */
    KVF_ERR_RANGE = 7        /* an fp32 cache on the tensor-core path met a rotated key, query or
                                value above 65 504 in magnitude (read via kvf_cache_status)      */
} kvf_status;

typedef enum { KVF_BF16 = 0, KVF_F32 = 1 } kvf_dtype;

enum {
    KVF_ROPE_INTERLEAVED = 1u, /* rotate pairs (2j,2j+1) instead of (j, j+d/2)                   */
    KVF_STRICT_POS = 2u,       /* reject pos0 != len (positions must continue across chunks)     */
    KVF_OUT_F32 = 4u,          /* `out` is fp32 even when dtype is bf16                          */
    KVF_FORCE_SIMT = 8u,       /* use the CUDA-core attention kernel even where a tensor-core
                                  kernel applies (bisecting aid, and the path for fp32 caches whose
                                  values leave fp16's range; same results within tolerance)      */
    KVF_HOST_UPLOAD_AHEAD = 32u, /* kvf_fold_step_host copies a step's q/k/v to the device on a stream of the
                                  library's own, into one of two staging sets, so that the upload of step
                                  t+1 runs while step t computes (the call's stream waits for the upload;
                                  results and errors are as without the flag).  Needs a workspace that no
                                  other cache's host steps use at the same time */
    KVF_HOST_DOWNLOAD_BEHIND = 128u, /* kvf_fold_step_host copies a step's results (out, lse) back on a stream of
                                  the library's own, behind the step, from one of two result staging sets, so
                                  that the copy of step t runs while step t+1 computes instead of standing in
                                  front of it on the caller's stream.  The contract on the results relaxes:
                                  those of call t are in host memory once the caller's stream has passed the
                                  end of call t+1, or of a kvf_cache_host_flush made after call t - not
                                  already at the end of call t.  Can be combined with KVF_HOST_UPLOAD_AHEAD;
                                  needs a workspace that no other cache's host steps use at the same time */
    KVF_COMBINE_BEHIND = 256u, /* kvf_fold_step and kvf_fold_step_host launch the kernel that merges the key
                                  ranges' partial results (the last kernel of a step whose plan has three)
                                  on a stream of the library's own, behind the attention kernel, and keep two
                                  sets of partial results, so that the merge of step t runs beside the rotate
                                  + append and the attention kernel of step t+1 instead of in front of them.
                                  The contract on the results relaxes: `out` and `lse` of call t are complete
                                  on the caller's stream once that stream has passed the end of call t+1 on
                                  this cache, or of a kvf_cache_flush made after call t - not already at the
                                  end of call t - and until then they belong to the library (call t+1 must
                                  be given other result buffers).  Same values as without the flag.  A
                                  stream capture has to hold whole chains: a step or a flush that meets a
                                  merge left open outside its own capture returns KVF_ERR_INVALID_ARG and
                                  enqueues nothing - flush before a capture begins and before it ends.  The
                                  stream and its events are made by kvf_cache_create /
                                  kvf_paged_cache_create, and kvf_workspace_bytes grows by the second set.
                                  Needs a workspace that no other cache's steps use while a merge is open
                                  (the merge reads its partial results there behind the caller's stream);
                                  batches and kvf_fold_step_static ignore the flag */
    KVF_CACHE_INT8 = 16u,      /* store the cache as int8 codes with one fp32 scale per row (one token of
                                  one KV head): d + 4 bytes per row instead of 2 d (kvf_cache_storage_bytes
                                  pads each head's scales to a multiple of 16 bytes).  The paper's Discussion
                                  perturbs the stored K/V by a round trip bf16 -> intN -> bf16 and leaves
                                  the scheme open; here a row is quantised once, when it is appended:
                                  scale = max|x| / 127, code = clamp(rint(x * (127 / max|x|)), +-127) in
                                  fp32 (keys: on the rotated row before any rounding to bf16), and the
                                  attention sees bf16(code * scale).  dtype KVF_BF16 and head_dim 128
                                  only (KVF_ERR_UNSUPPORTED otherwise, and for kvf_fold_step_static);
                                  the attention kernel expands code tiles to bf16 tiles in shared
                                  memory - or, for steps of at most 16 query rows (n_tokens * H/Hkv) on
                                  a cache (or a batch of caches) without a window, straight into the
                                  register fragments of its MMAs - so a step reads d + 4 bytes per
                                  cached row.  Paged caches and
                                  batches of them take the flag too (see kvf_paged_cache_create) */
    KVF_CACHE_INT4 = 64u       /* the same with 4-bit codes (the other width the paper reports): scale =
                                  max|x| / 7, codes within +-7, stored two to a byte as code + 8 (element
                                  2i in the low nibble of byte i): d / 2 + 4 bytes per row.  Not together
                                  with KVF_CACHE_INT8 (KVF_ERR_INVALID_ARG) */
};

/*
 * Shape and numerics of one cache.
 *   n_q_heads (H), n_kv_heads (Hkv): grouped-query attention, query head h reads KV head
 *       h / (H/Hkv); H % Hkv == 0 and H/Hkv <= 64 (the models of the paper's experiments have
 *       groups of 4 (Llama-3.1-8B: 32/8), 7 (Qwen2.5-7B: 28/4), 6 (Qwen2.5-1.5B: 12/2) and 1
 *       (OLMoE: 16/16)).  The tensor-core kernels lay a group that is no power of two out as
 *       the next power of two, so 1/8 (groups of 7) or 1/4 (groups of 6) of their tensor-core
 *       work is spent on padding rows.
 *   head_dim (d): 64 or 128.
 *   dtype: element type of q, k_new, v_new, of the cache planes and (unless KVF_OUT_F32) of out.
 *       KVF_BF16: rotation, scores, softmax state and the output sum are fp32, probabilities
 *       and the rotated q/k are rounded once to bf16.  KVF_F32: fp32 throughout.  With head_dim
 *       128 the fp32 attention runs on the tensor cores: each operand is split into two fp16
 *       halves (22 significant bits; elements below 2^-3 to an absolute 2^-25) and each product
 *       is three MMAs, with the output summed in round-to-nearest fp32 registers; magnitudes
 *       must stay within fp16's 65 504 (else KVF_ERR_RANGE in the status word and non-finite
 *       outputs).  With head_dim 64, or under KVF_FORCE_SIMT, it runs on the CUDA cores in plain
 *       fp32 with no such limits.
 *   capacity: most tokens the cache will ever hold.
 *   max_chunk: largest n_tokens of any later kvf_fold_step (sizes the workspace).
 *   rope_base: theta = pos * rope_base^(-2j/d) (RoPE at the tokens' absolute positions, which
 *       run on across chunk boundaries: Section 2, the paragraph that defines the one-step update).
 *   softmax_scale: 0 means 1/sqrt(d).
 *   inv_freq: optional HOST pointer to d/2 doubles replacing rope_base^(-2j/d)
 *       (frequency-scaled RoPE variants); copied at create, may be freed afterwards.
 */
typedef struct kvf_config {
    int32_t n_q_heads;
    int32_t n_kv_heads;
    int32_t head_dim;
    int32_t dtype; /* kvf_dtype */
    int64_t capacity;
    int32_t max_chunk;
    uint32_t flags;
    double rope_base;
    double softmax_scale;
    const double *inv_freq;
} kvf_config;

/* Bytes of device storage one cache needs: K plane then V plane, each
 * [n_kv_heads][capacity][head_dim] of dtype (head-major, one row = one token of one head;
 * Section 5 gives the same count: KV heads x head_dim x (K,V) x bytes, per token).
 * Returns 0 for an invalid config. */
size_t kvf_cache_storage_bytes(const kvf_config *cfg);

/* Bytes of device workspace: a status word, the rotated queries of one chunk, staging for
 * kvf_fold_step_host, and the split partial results.  Returns 0 for an invalid config. */
size_t kvf_workspace_bytes(const kvf_config *cfg);

/*
 * Create the empty accumulator (the (empty, empty) start of the fold, Section 2).
 *   dev_storage   device pointer, 256-byte aligned, >= kvf_cache_storage_bytes(cfg); need not be
 *                 initialised; the library writes only rows it appends (plus zeroed value rows up
 *                 to the next multiple of 128 rows, which are not cache content).
 *   dev_workspace device pointer, 256-byte aligned, >= kvf_workspace_bytes(cfg).
 *   *out          receives the handle.
 * Builds the TMA descriptors for the planes (driver entry point looked up at run time) and
 * clears the device status word on the default stream.  Returns KVF_ERR_UNSUPPORTED for shapes
 * outside the documented set, KVF_ERR_CAPACITY for short buffers, KVF_ERR_CUDA if no device.
 */
kvf_status kvf_cache_create(const kvf_config *cfg, void *dev_storage, size_t storage_bytes,
                            void *dev_workspace, size_t workspace_bytes, kvf_cache **out);

/*
 * Paged variant of the accumulator (the paper's cache grows by appending; serving systems it
 * cites manage such caches in fixed-size pages - Related work, "Chunked serving infrastructure").  bf16 caches
 * with head_dim 128 only (KVF_ERR_UNSUPPORTED otherwise), stored as bf16 or, under KVF_CACHE_INT8 /
 * KVF_CACHE_INT4, as codes and row scales.
 *   A page holds 128 consecutive tokens of every KV head: [K|V][n_kv_heads][128][head_dim]; quantised:
 *   [K codes|V codes][n_kv_heads][128][head_dim or head_dim / 2 bytes], then [K scales|V scales]
 *   [n_kv_heads][128] fp32 (kvf_paged_pool_bytes counts both; the scale accessors return NULL).
 *   dev_pool        device, 256-byte aligned, n_pool_pages pages (kvf_paged_pool_bytes); pages may be
 *                   shared by many caches of the same shape
 *   dev_page_table  device int32 array, entry i = pool page of tokens [128 i, 128 i + 128); needs
 *                   ceil(capacity / 128) entries.  The caller owns it and may fill entries at any time
 *                   before the step that first touches their tokens is enqueued (stream order).
 * Everything else - workspace, steps, length, status - is as for kvf_cache_create; the plane
 * accessors return NULL.  A step zeroes the value rows between the new end and the end of its
 * page, so a page must not be shared between two live caches.
 */
size_t kvf_paged_pool_bytes(const kvf_config *cfg, int32_t n_pages);
kvf_status kvf_paged_cache_create(const kvf_config *cfg, void *dev_pool, size_t pool_bytes, int32_t n_pool_pages,
                                  const int32_t *dev_page_table, void *dev_workspace, size_t workspace_bytes,
                                  kvf_cache **out);

/*
 * One fold step at this layer (Section 2: queries from the new tokens, keys/values
 * [K_0;...;K_t], positions continued from the chunk's absolute start; Figure "KV-Fold":
 * the chunk's K/V are appended, the prefix is passed on unchanged).
 *   q      device, [n_tokens][H][d]   dtype, contiguous, 16-byte aligned, before rotation
 *   k_new  device, [n_tokens][Hkv][d] dtype, before rotation
 *   v_new  device, [n_tokens][Hkv][d] dtype
 *   pos0   absolute position of the chunk's first token (the fold passes pos0 = len); used
 *          only for the rotation - visibility is by cache row
 *   out    device, [n_tokens][H][d], dtype (or fp32 with KVF_OUT_F32): row i is the attention
 *          output of token i over cache rows 0 .. len+i (all earlier chunks, then causal)
 *   lse    device, [n_tokens][H] fp32 natural-log softmax denominators, or NULL
 * Effects, in stream order: rotate q into the workspace; write rotated k and v as rows
 * [len, len+n_tokens); attention; then the host-side length becomes len + n_tokens.
 * Errors: INVALID_ARG, CAPACITY (cache full), POS, CUDA (launch failure; length unchanged).
 * A step is two or three kernels on cuda_stream.  Short steps launch them with programmatic stream
 * serialisation (a kernel's set-up overlaps the tail of the one before); steps with long
 * tensor-bound attention kernels launch them plainly, which on a power-capped board is the faster
 * of the two.  KVF_DEPENDENT_LAUNCH=always or =never in the environment (read once) overrides the
 * choice; results do not depend on it.
 */
kvf_status kvf_fold_step(kvf_cache *c, const void *q, const void *k_new, const void *v_new,
                         int32_t n_tokens, int64_t pos0, void *out, float *lse, void *cuda_stream);

/*
 * The same step with HOST buffers (pinned memory recommended): copies q/k/v to the workspace
 * staging area, runs the step, copies `out` (and lse if not NULL) back, all on `cuda_stream`
 * (with KVF_HOST_UPLOAD_AHEAD the three uploads run on an internal stream that `cuda_stream` then
 * waits for; with KVF_HOST_DOWNLOAD_BEHIND the results are copied back on an internal stream, see
 * that flag for when they are there).  The host buffers must stay valid until the stream reaches
 * the end of the call (result buffers under KVF_HOST_DOWNLOAD_BEHIND: until the results are there).
 */
/*
 * Queries only: the n_tokens query rows are rotated at positions pos0, pos0+1, ... and attend to ALL
 * rows the cache holds (no causal limit: none of them is a row of this chunk); nothing is appended
 * and kvf_cache_len does not change.  out and lse as in kvf_fold_step; pass lse whenever the result
 * is to be merged with others.  (Section 2: a chunk's queries attend to the concatenation of the
 * rows of all chunks so far; when those rows are spread over several caches - one sequence split
 * by row range over GPUs, Section 5's single-GPU memory limit being what such a split lifts - the
 * cache that takes the chunk runs kvf_fold_step and every other one kvf_attend, and
 * kvf_merge_partials puts the results together.)  KVF_ERR_INVALID_ARG on an empty cache (there is
 * nothing to attend to: leave that part out of the merge, or give it lse = -inf),
 * KVF_ERR_UNSUPPORTED under a sink + window mask.  Same stream semantics, workspace use and error
 * contract as kvf_fold_step.
 */
kvf_status kvf_attend(kvf_cache *c, const void *q, int32_t n_tokens, int64_t pos0, void *out, float *lse,
                      void *cuda_stream);

/*
 * Merges n_parts attention results over disjoint sets of rows into the result over their union:
 *     lse = log sum_r exp(lse_r),   out = sum_r exp(lse_r - lse) * out_r     (parts in index order).
 * parts_out: device, [n_parts][n_rows][head_dim], elements of `dtype` (KVF_BF16 or KVF_F32: what the
 * steps wrote - fp32 under KVF_OUT_F32, which keeps the merged result free of a second rounding);
 * parts_lse: device, [n_parts][n_rows] fp32 natural-log values as kvf_fold_step / kvf_attend return
 * them (-inf: that part saw no row and is skipped); n_rows = tokens * query heads; out: device,
 * [n_rows][head_dim] of `dtype`; lse: device [n_rows] or null.  This layout is what an all-gather of
 * every rank's (out, lse) produces.  head_dim 64 or 128; pointers 16-byte (lse: 4-byte) aligned.
 * Stateless: needs no cache handle and no workspace; one kernel on cuda_stream.  (The paper runs on one
 * GPU and has no counterpart; the identity is the softmax over a union of key sets, Section 2.)
 */
kvf_status kvf_merge_partials(int32_t n_parts, int64_t n_rows, int32_t head_dim, kvf_dtype dtype, const void *parts_out,
                              const float *parts_lse, void *out, float *lse_or_null, void *cuda_stream);

kvf_status kvf_fold_step_host(kvf_cache *c, const void *q_host, const void *k_host,
                              const void *v_host, int32_t n_tokens, int64_t pos0, void *out_host,
                              float *lse_host, void *cuda_stream);

/* Makes `cuda_stream` wait for whatever part of the steps enqueued so far runs on a stream of the
 * library's own: the merge of the last step under KVF_COMBINE_BEHIND, the result copies of the host
 * steps under KVF_HOST_DOWNLOAD_BEHIND (synchronising that stream afterwards means "all results are
 * there").  Without those flags, or with nothing outstanding, it does nothing.  Enqueues waits only;
 * returns at once.  No counterpart in the paper: it closes the two relaxed contracts above.
 * KVF_ERR_INVALID_ARG for a null handle, or when the open merge belongs to another stream capture
 * than `cuda_stream` (or to none while `cuda_stream` is being captured). */
kvf_status kvf_cache_flush(kvf_cache *c, void *cuda_stream);
/* The same call under its earlier name. */
kvf_status kvf_cache_host_flush(kvf_cache *c, void *cuda_stream);

/* Tokens appended by all steps enqueued so far: the size of the accumulator (K,V)^(t) of Section
 * 2's left fold after t steps, which holds the rows of chunks 0..t (host counter; after t steps
 * of C tokens it is t*C without any synchronisation).  -1 for a null handle. */
int64_t kvf_cache_len(const kvf_cache *c);

/* Back to the empty accumulator the fold starts from (Section 2: the fold's initial value is the
 * pair of empty K and V; also the start of every chunk under the paper's ISOLATED condition,
 * Section 2, "Three reference conditions").  len = 0; storage is not cleared. */
kvf_status kvf_cache_reset(kvf_cache *c);

/* Sets the number of rows the accumulator holds, 0 <= len <= capacity (else KVF_ERR_CAPACITY);
 * host counter only, nothing is enqueued and no row is touched.
 * Section 2 states that the cache IS the whole state of the fold, so a fold can be taken back to
 * an earlier accumulator (K,V)^(t') by forgetting the rows behind it.  The paper's multi-needle
 * protocol ("Multi-needle retrieval", in the section on scaling) asks K questions about ONE folded
 * haystack, each queried separately: fold the haystack once, then per key a question chunk and the
 * decoded tokens, then kvf_cache_set_len(c, haystack_len) - instead of folding 128 K tokens K times.
 * len <= kvf_cache_len: rows [len, old len) are forgotten; the next step appends at row len (and
 *   rotates at the pos0 the caller passes).  Steps enqueued before the call are not affected.
 * len >  kvf_cache_len: resuming from restored storage.  The caller vouches that the planes hold what a
 *   cache of at least len rows held (a byte copy of the storage of a live cache, taken when its
 *   length was >= len, is that); rows the library never wrote may hold non-finite bits, which a
 *   masked key tile would turn into NaN outputs.
 * With KVF_COMBINE_BEHIND / KVF_HOST_DOWNLOAD_BEHIND the results of the last step are still on their
 * way as after any step; this call does not wait for them. */
kvf_status kvf_cache_set_len(kvf_cache *c, int64_t len);

/* Reads the device status word (synchronises the default stream with a blocking copy): KVF_OK,
 * KVF_ERR_TIMEOUT if a bounded wait inside a kernel gave up, or KVF_ERR_RANGE (see kvf_status).  Call after synchronising the
 * streams that carried the steps.  (The paper has no counterpart: this reports on the kernels'
 * own waits, not on anything the method computes.) */
kvf_status kvf_cache_status(kvf_cache *c);

/* The raw device status word behind kvf_cache_status (same synchronisation): 0, or for the first
 * bounded wait that gave up 5 + 256 * (index of the barrier in the kernel's control block)
 * + 65536 * (waiting warp) + 2^24 * (awaited parity) - what a bug report should quote.
 * -1 for a null handle or a failed copy. */
int32_t kvf_cache_status_word(kvf_cache *c);

/* The SM clock the attention kernels ran at, measured by the kernels themselves.  (The paper has
 * no counterpart: a measurement aid.)  One CTA of every tensor-core attention launch (the last row block of the first key range) adds the
 * SM cycles and the nanoseconds (device timer) it was running to two sums kept beside the status
 * word; cycles_ns[0] / cycles_ns[1] receive the sums since the cache was created, so the difference
 * of two readings gives cycles * 1000 / ns = MHz over the launches in between.  Blocking copy, as
 * kvf_cache_status; the CUDA-core kernel does not count.  Caches that share a workspace share the sums. */
kvf_status kvf_cache_sm_clock(kvf_cache *c, uint64_t cycles_ns[2]);

/* Device pointers of the planes, [n_kv_heads][capacity][head_dim] of dtype (int8 codes under
 * KVF_CACHE_INT8), and of the rows' fp32 scales (NULL without that flag): [n_kv_heads][stride] with
 * stride = capacity rounded up to a multiple of 4, so that every head's scales start 16-byte aligned. */
void *kvf_cache_k_plane(const kvf_cache *c);
void *kvf_cache_v_plane(const kvf_cache *c);
float *kvf_cache_k_scales(const kvf_cache *c);
float *kvf_cache_v_scales(const kvf_cache *c);

/*
 * What a step of n_tokens on a prefix of prefix_len would launch:
 *   plan[0] 1 = a tensor-core (tcgen05) attention kernel (bf16, or fp32 with head_dim 128), 0 = CUDA-core kernel
 *   plan[1] parts the key range of one KV head is cut into (1 = none).  CUDA-core kernel: equal
 *           splits.  Tensor-core kernel: the (KV head, key tile) pairs are cut into plan[2] /
 *           (row blocks: 256-row pairs in bf16, 128-row blocks in fp32) contiguous ranges that
 *           need not end at KV-head boundaries; this is their number per KV head, rounded up
 *   plan[2] CTAs of the attention kernel
 *   plan[3] kernels launched by the step (3 = a combine kernel merges partial results; chunks of
 *           at most 128 / (H / Hkv) tokens always take that route on the tensor-core path)
 */
kvf_status kvf_cache_plan(const kvf_cache *c, int32_t n_tokens, int64_t prefix_len, int32_t plan[4]);

/* Force the number of splits (0 = automatic).  Values the workspace cannot hold are clamped. */
kvf_status kvf_cache_set_splits(kvf_cache *c, int32_t splits);

/*
 * Sink + window variant of the attention mask (Section 6 of the paper, the comparison with
 * StreamingLLM at 4 sink tokens plus a window of 1020 recent ones; the rows that stay keep the
 * positions they were appended at, no RoPE re-anchoring).  From the next step on, a chunk that starts at row P sees,
 * of the rows before it, only rows r < n_sink and rows r >= P - window - what a cache evicted to
 * "sinks + the last `window` rows" after every chunk would still hold - and its own rows causally.
 * window = 0 (with n_sink = 0) restores the full prefix.  n_sink <= 64.
 * Rows are still appended at their place and nothing is deleted: the mask alone changes, and key
 * tiles without a visible row are never read.  With a paged cache the caller may therefore hand
 * the pages of such tiles to another use (every page below row P - window except page 0 when
 * n_sink > 0): their table entries are not looked at again.
 */
kvf_status kvf_cache_set_window(kvf_cache *c, int32_t n_sink, int64_t window);

/* Kernels launched through this handle since creation. */
uint64_t kvf_cache_launch_count(const kvf_cache *c);

/*
 * Per-kernel timing.  With enable != 0 every step records CUDA events around each of its
 * kernels on the step's stream.  kvf_cache_profile_read synchronises, then ADDS the elapsed
 * milliseconds and launch counts since the last read to
 *   ms[0]/launches[0] rotate+append, [1] attention, [2] split combine
 * and forgets the recorded events.  At most 65536 launches are kept between reads.
 */
kvf_status kvf_cache_profile(kvf_cache *c, int32_t enable);
kvf_status kvf_cache_profile_read(kvf_cache *c, double ms[3], uint64_t launches[3]);

/* Frees the host handle (and its events); device memory stays with the caller. */
void kvf_cache_destroy(kvf_cache *c);

/*
 * One launch over many caches.  The paper's fold runs once per layer (and per sequence) for every
 * chunk, each layer with its own accumulated K/V (Section 2: the per-layer caches of chunk t are
 * what chunk t+1 attends to); a 32-layer model folding 4 sequences has 128 caches that all stand
 * at the same length.  A batch folds one chunk into every member with ONE launch of each kernel
 * instead of one per cache: the members' CTAs fill the GPU together, which matters while the
 * prefix is short or the chunk is small.
 *
 * Members: caches made by kvf_paged_cache_create over the SAME pool with the same configuration
 * (they share the pool's tensor maps; each keeps its own page table), no cache twice; otherwise
 * KVF_ERR_UNSUPPORTED (not paged) or KVF_ERR_INVALID_ARG.  The handles stay owned by the caller,
 * stay usable on their own between batch steps, and must outlive the batch.
 * dev_workspace: caller-owned, 256-byte aligned, kvf_batch_workspace_bytes(cfg, n_caches) bytes
 * (0 = invalid arguments; n_caches 1..65535): the rotated chunks of all members, their partial
 * results and one status word.  Creation copies the members' table pointers into it (blocking).
 */
typedef struct kvf_batch kvf_batch;
size_t kvf_batch_workspace_bytes(const kvf_config *cfg, int32_t n_caches);
kvf_status kvf_batch_create(kvf_cache *const *caches, int32_t n_caches, void *dev_workspace,
                            size_t workspace_bytes, kvf_batch **out);

/*
 * kvf_fold_step for every member at once.  q, out: [n_caches][n_tokens][n_q_heads][head_dim];
 * k_new, v_new: [n_caches][n_tokens][n_kv_heads][head_dim]; lse_or_null: [n_caches][n_tokens]
 * [n_q_heads]; all device pointers, contiguous, member i's block at index i in the order given
 * to kvf_batch_create.  n_tokens and pos0 are common to the members.  All members must hold the
 * same number of rows (KVF_ERR_INVALID_ARG otherwise); each one's length advances by n_tokens.
 * Per member the result is what kvf_fold_step gives: the same cache bits, the output within
 * rounding of it (the key range may be cut differently, which reorders the sums).  Asynchronous
 * on cuda_stream; errors and their effect as for kvf_fold_step.
 */
kvf_status kvf_batch_fold_step(kvf_batch *b, const void *q, const void *k_new, const void *v_new,
                               int32_t n_tokens, int64_t pos0, void *out, float *lse_or_null,
                               void *cuda_stream);

/*
 * The same step for members that hold DIFFERENT numbers of rows (sequences of different length
 * decoded together).  n_tokens is still common.  pos0_or_null: host array [n_caches] of the chunks'
 * first positions, or null = each member's own length.  One more small launch per 64 members hands
 * the members' row counts to the kernels; the key range is cut as the longest member needs.  Not
 * available under a sink + window mask (KVF_ERR_UNSUPPORTED).
 */
kvf_status kvf_batch_fold_step_ragged(kvf_batch *b, const void *q, const void *k_new, const void *v_new,
                                      int32_t n_tokens, const int64_t *pos0_or_null, void *out,
                                      float *lse_or_null, void *cuda_stream);

/*
 * The ragged step for members whose CHUNKS differ in length as well (the paper's trials end with a
 * question chunk and up to 30 decoded tokens each - Section 4, the needle protocol - so sequences
 * that are served together take steps of different length, and finish at different times).
 *   n_tokens    host array [n_caches]: member i folds n_tokens[i] tokens, 0 <= n_tokens[i] <= max_tokens;
 *               0 = the member sits this step out (its cache, length and block of `out` are untouched)
 *   max_tokens  1 .. max_chunk: the stride of the members' blocks - q, out: [n_caches][max_tokens][n_q_heads]
 *               [head_dim], k_new, v_new: [n_caches][max_tokens][n_kv_heads][head_dim], lse_or_null:
 *               [n_caches][max_tokens][n_q_heads]; member i uses the first n_tokens[i] rows of its blocks
 * Everything else as kvf_batch_fold_step_ragged; at least one member must take part.
 */
kvf_status kvf_batch_fold_step_varlen(kvf_batch *b, const void *q, const void *k_new, const void *v_new,
                                      const int32_t *n_tokens, int32_t max_tokens, const int64_t *pos0_or_null,
                                      void *out, float *lse_or_null, void *cuda_stream);

/* kvf_cache_plan for a batch step; plan[2] counts the CTAs of all members. */
kvf_status kvf_batch_plan(const kvf_batch *b, int32_t n_tokens, int64_t prefix_len, int32_t plan[4]);

/* The batch's own device status word, encoded as kvf_cache_status_word (0 = no wait gave up). */
int32_t kvf_batch_status_word(kvf_batch *b);

/* Kernels launched through this batch since creation. */
uint64_t kvf_batch_launch_count(const kvf_batch *b);

/* Frees the host handle; the members and all device memory stay with the caller. */
void kvf_batch_destroy(kvf_batch *b);

/*
 * The fold step for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for the sake of such callers only.)
 *
 * Who they are: a server that has already handed every byte of device memory to its own pool
 * (KV pages sized to fill the GPU) and has nothing left to give for a workspace; a latency-bound
 * loop that must stay out of the allocator because an allocation can stall the whole device for
 * an unbounded time; a plug-in that runs under a policy forbidding allocation calls.  For them
 * the step's scratch (status word, rotated queries, split partial results) lives in a fixed
 * array inside the library, KVF_STATIC_SCRATCH_BYTES (about 20 MiB), which every GPU that loads
 * the library holds from load until the process exits.  The call, and everything it calls,
 * allocates and frees nothing on the device.
 *
 * There is no handle: the caller owns the planes and the length.
 *   cfg           as for kvf_cache_create (max_chunk sizes the rotated-query area)
 *   dev_storage   device, 256-byte aligned, >= kvf_cache_storage_bytes(cfg): K plane then V plane,
 *                 holding `len` tokens appended by earlier calls (of this or of kvf_fold_step)
 *   len           tokens already in the planes; after KVF_OK the caller's length is len + n_tokens
 *   q, k_new, v_new, n_tokens, pos0, out, lse, cuda_stream: as for kvf_fold_step
 * Limits (KVF_ERR_CAPACITY beyond them, nothing enqueued; kvf_last_cuda_error names the limit):
 *   max_chunk * n_q_heads * head_dim * sizeof(dtype) <= 4 MiB   (32 heads x 128, bf16: 512 tokens)
 *   n_tokens * n_q_heads * head_dim * 4 <= 16 MiB; the key range is split at most as many ways as
 *   16 MiB of fp32 partial results hold (32 heads x 128: splits * n_tokens <= 1024), so a step
 *   may run with fewer splits than kvf_fold_step would use - same result within tolerance.
 * First call on a device: looks up the array's device address (cudaGetSymbolAddress, with that
 * device current) and keeps it; make this first call before any stream capture begins.
 * Sharing: all calls on one device use the one array, which keeps whatever the last call left
 * (the call clears the status word it needs at zero; everything else is written before it is
 * read).  Two calls whose kernels may overlap on the GPU - different streams, or different
 * threads - race on it: keep all calls on a device in one stream order.  A bounded device-side
 * wait that gives up cannot be reported here (there is no handle to ask); results are then
 * undefined, as with kvf_fold_step before kvf_cache_status is read.
 */
#define KVF_STATIC_SCRATCH_BYTES 21234688
kvf_status kvf_fold_step_static(const kvf_config *cfg, void *dev_storage, size_t storage_bytes, int64_t len,
                                const void *q, const void *k_new, const void *v_new, int32_t n_tokens,
                                int64_t pos0, void *out, float *lse, void *cuda_stream);

const char *kvf_status_str(kvf_status s);

/* Text of the last CUDA error seen by this thread's calls into the library ("" if none). */
const char *kvf_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* KVFOLD_H_ */
