/*
 * streaming_thinker.h -- C ABI of the B200 (sm_100a) streaming dual-KV-cache attention library.
 *
 * The library implements the inference hot path of "streaming thinking" (Section 3.3 and
 * Algorithm 1 of the StreamingThinker paper): attention over two decoupled KV caches.
 *   - source cache    : input tokens, appended unit by unit (Algorithm 1, prefill loop);
 *   - reasoning cache : reasoning tokens, appended one by one or span by span (decode loop).
 * A source token attends causally to the source cache only (the ordinary causal mask that
 * Eq. 2 keeps for input rows). A reasoning token attends to a visible PREFIX of the source
 * cache plus the reasoning cache up to and including itself (Eq. 1, Eq. 2, and the
 * N_EOS == N_EOT + 1 rule of Algorithm 1). Position ids follow the streaming position
 * encoding of Section 3.2: each cache counts its own tokens from zero.
 *
 * Conventions
 *   - All functions return ST_OK (0) or a negative ST_ERR_* code; st_last_error_string()
 *     describes the last failure of a context. No C++ exception crosses this boundary.
 *   - "device" pointers are CUDA device memory of the context's device; "host" pointers are
 *     ordinary host memory. q/k/v are bf16, un-rotated, packed token-major
 *     [tokens][heads][128]; out is fp32 [tokens][n_q_heads][128]. The caller owns them.
 *   - Calls are asynchronous on the cudaStream_t passed as `stream` (NULL = legacy default
 *     stream). Every argument is validated on the host before anything is launched; a call
 *     that fails changes no state. That holds for a CUDA runtime failure in the middle of a call
 *     (ST_ERR_CUDA) too: pages the call had taken return to the free list and its step is no longer
 *     pending, so the same call can be issued again; work it had already queued on the stream is not
 *     recalled (it only rewrites page-table entries and cache slots that the repeated call writes again).
 *   - One context is driven from one host thread. All source-side calls
 *     (st_append_source_chunk) must be stream-ordered among themselves, and so must all
 *     reasoning-side calls (st_reason_decode, st_reason_extend); the two sides may use two
 *     different streams and then run concurrently (Algorithm 1's two parallel loops): a
 *     reasoning-side call waits, on the device, for exactly the source appends it reads.
 *   - Multi-layer contexts: a step is issued for layer 0, 1, ..., n_layers-1 in order with
 *     identical sequence lists and token counts; lengths and unit counters advance when the
 *     last layer has been issued.
 */
#ifndef STREAMING_THINKER_H_
#define STREAMING_THINKER_H_

#include <stdint.h>

#if defined(__GNUC__)
#define ST_API __attribute__((visibility("default")))
#else
#define ST_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define ST_OK                  0
#define ST_ERR_INVALID_ARG    -1   /* bad pointer, size, id or flag                                     */
#define ST_ERR_OOM_PAGES      -2   /* a page pool (or a per-sequence page table) is exhausted            */
#define ST_ERR_NOT_READY      -3   /* the requested source unit has not been appended (Alg. 1: "wait")   */
#define ST_ERR_STATE          -4   /* layer out of order, or step arguments differ between layers        */
#define ST_ERR_CUDA           -5   /* a CUDA runtime call failed                                          */
#define ST_ERR_DEVICE_TIMEOUT -6   /* a bounded device-side wait expired (reported by st_device_status)  */
#define ST_ERR_DEVICE_CHECK   -7   /* a device-side bounds check failed: a page id read from a page table
                                      lies outside its pool. The access was skipped, nothing faulted; rows
                                      of the call are undefined (reported by st_device_status)            */

/* st_config.flags */
#define ST_CFG_HOST_ONLY       1u  /* plan only: no device memory, no launches (host logic and its tests) */
#define ST_CFG_DEBUG_CHECKS    2u  /* debug context: free pages (at st_create, and again when st_reset releases
                                      them) hold a large finite sentinel (bf16 9.95e29) instead of zeros, so
                                      that a key or value read from beyond the visible ranges -- which the
                                      kernels would otherwise multiply by a weight of zero without a trace --
                                      shows up in the rows. The kernels' page-id checks are always on.     */
#define ST_CFG_PRECISE_P       4u  /* chunk prefill and reasoning spans carry the softmax weights into the
                                      weights-times-values product as two bf16 terms (16 significant bits)
                                      instead of one (8 bits). One term bounds a row's error by about 2^-9
                                      times the largest |v| the row mixes: within 1e-2 for values of order 1,
                                      not for values of a few tens (outlier channels). The second term costs
                                      one more tensor-core product per key tile. Decode steps always use two
                                      terms (free there).                                                   */
/* per-call flags */
#define ST_END_OF_UNIT         1u  /* source side: this chunk completes a source unit (N_EOS += 1);
                                      reasoning side: the unit's boundary token was produced (N_EOT += 1) */
#define ST_REFERENCE_KERNELS   2u  /* run the slow, simple attention kernels instead of the tuned ones    */
#define ST_IO_HOST             4u  /* q/k/v/out are HOST pointers (page-locked memory recommended). A large
                                      call copies them to and from internal device staging on `stream`; a
                                      st_reason_decode call whose q + k + v stay below 1 MiB and whose buffers
                                      are all page-locked is served in place: its kernels read q/k/v and
                                      write the rows directly in host memory. Either way the buffers belong
                                      to the call until the work queued on `stream` has completed            */

/* st_config.position_mode */
#define ST_POS_STREAMING       0   /* Section 3.2, streaming position encoding: the reasoning cache counts its
                                      tokens from zero on a counter of its own (the method's encoding)      */
#define ST_POS_CONCATENATED    1   /* the original RoPE ids Section 3.2 starts from: reasoning token t gets
                                      T + t, T = tokens in the source cache when the sequence's first
                                      reasoning token is appended (the whole input in the batch setting, where
                                      the paper compares the two encodings)                                  */
#define ST_POS_UNIT_ALIGNED    2   /* variant of this library, not the paper's: the i-th token of reasoning
                                      unit u gets P_{u-1} + i (the unit restarts where its source unit starts);
                                      tokens decoded with ST_VIS_ALL (final depth) get S + i, S = source
                                      tokens at the first such call                                          */

/* visible_units values */
#define ST_VIS_DEFAULT        -1   /* Algorithm 1: unit N_EOT + 1                                         */
#define ST_VIS_ALL            -2   /* everything appended so far (final-depth reasoning, Eq. 1 last term) */

typedef struct st_ctx st_ctx;      /* opaque; owns page tables, unit boundaries, counters, events, scratch */

typedef struct st_config {
  int32_t  n_layers;               /* >= 1                                                                */
  int32_t  n_q_heads;              /* multiple of n_kv_heads; n_q_heads / n_kv_heads <= 8                 */
  int32_t  n_kv_heads;
  int32_t  head_dim;               /* must be 128                                                         */
  int32_t  max_batch;              /* number of sequence slots; ids are 0 .. max_batch-1                  */
  int32_t  page_size;              /* must be 64 tokens                                                   */
  int64_t  n_pages_source;         /* pages per layer in the source pool                                  */
  int64_t  n_pages_reason;         /* pages per layer in the reasoning pool                               */
  int32_t  max_source_len;         /* tokens per sequence (bounds the page table); 0 = whole pool         */
  int32_t  max_reason_len;         /* same for the reasoning cache                                        */
  int32_t  max_tokens_per_call;    /* bound on the packed token count of one call (sizes the scratch)     */
  int32_t  device;                 /* CUDA device ordinal                                                 */
  void    *pool_base;              /* device memory of st_pool_bytes() bytes, 1024-byte aligned, or NULL:
                                      the library then allocates (and frees) the pools itself             */
  uint64_t pool_bytes;             /* size of pool_base when it is given                                  */
  double   rope_theta;             /* RoPE base, e.g. 1e6                                                 */
  float    softmax_scale;          /* 0 = 1/sqrt(head_dim)                                                */
  uint32_t flags;                  /* ST_CFG_*                                                            */
  int32_t  position_mode;          /* ST_POS_*: position ids of reasoning tokens (source tokens always count
                                      from zero)                                                          */
  int32_t  reserved;               /* must be 0                                                           */
  const float *q_norm_weight;      /* HOST arrays [n_layers][128], or both NULL: per-head RMS normalisation of */
  const float *k_norm_weight;      /* q and k over the head dimension before the rotation, x / sqrt(mean(x^2)
                                      + qk_norm_eps) * weight, as the Qwen3 backbones of Section 4.1 apply it
                                      (not part of the paper's method; fused into the kernels that rotate:
                                      one rounding to bf16, after the rotation). Copied at st_create.        */
  float    qk_norm_eps;            /* e.g. 1e-6                                                             */
  int32_t  reserved2;              /* must be 0                                                             */
} st_config;

/* Bytes of device memory the two page pools need: n_layers * (n_pages_source + n_pages_reason) *
 * n_kv_heads * 32 KiB (one page holds, per kv head, 64 rotated keys and 64 values in bf16).
 * Pure host function. Returns 0 for an invalid configuration. */
ST_API uint64_t st_pool_bytes(const st_config *cfg);

/* Create a context (Algorithm 1, line 1: initialise the caches). Allocates page tables, scratch
 * and, if cfg->pool_base is NULL, the pools; zero-fills the pools. `*out` is set on success.
 * Scratch besides the pools: the split-K records of the decode kernel (a few MB), two rotation tables, per side a
 * rotated-query buffer of max_tokens_per_call rows and 19.5 MB in which the attention kernel's key-split halves meet
 * (two CTAs share a long work item when the last wave of a launch would leave SMs idle); host-I/O staging buffers
 * are allocated by the first call that needs them. */
ST_API int st_create(const st_config *cfg, st_ctx **out);

/* Wait for the device, then free everything the context owns (never cfg->pool_base). */
ST_API int st_destroy(st_ctx *ctx);

/* Forget the listed sequences (host array of n_seq ids; n_seq == 0: all): both caches are emptied,
 * pages return to the free lists, N_EOS = N_EOT = 0. Waits for the device first, because kernels in
 * flight may still read the pages. */
ST_API int st_reset(st_ctx *ctx, const int32_t *seq_ids, int32_t n_seq);

/* Prefill loop of Algorithm 1: append one chunk of source tokens per listed sequence and compute
 * the chunk's attention rows. For sequence seq_ids[b] the chunk is rows cu_tokens[b] .. cu_tokens[b+1]
 * of q/k/v (cu_tokens: host, n_seq+1 non-decreasing ints starting at 0). Token i of the chunk gets
 * position p+i (p = tokens already in that source cache); its key is rotated at that position
 * (streaming position encoding) and stored with its value; its query, rotated the same way, attends
 * to source positions 0 .. p+i (causal, Eq. 2's unmodified part) and never to a reasoning token.
 * out (may be NULL: cache only) receives softmax(q k^T * scale) v per q head in fp32.
 * flags: ST_END_OF_UNIT closes the current source unit of every listed sequence. */
ST_API int st_append_source_chunk(st_ctx *ctx, int32_t layer,
                           const int32_t *seq_ids, const int32_t *cu_tokens, int32_t n_seq,
                           const void *q, const void *k, const void *v, void *out,
                           uint32_t flags, void *stream);

/* Decode loop of Algorithm 1: one new reasoning token per listed sequence. The token gets position
 * r (= tokens already in that reasoning cache), is rotated and appended there, and attends to the
 * source prefix [0, vis) plus reasoning positions 0 .. r. vis comes from visible_units[b] (host array,
 * or NULL = ST_VIS_DEFAULT for all): k >= 0 selects the end of source unit k (k = 0: nothing);
 * ST_VIS_DEFAULT selects unit N_EOT + 1, the slice Algorithm 1 keeps; ST_VIS_ALL the whole source.
 * A unit that has not been closed yet yields ST_ERR_NOT_READY (the caller decides to wait).
 * q/k/v: [n_seq][heads][128]; out: [n_seq][n_q_heads][128] fp32.
 * flags: ST_END_OF_UNIT counts one finished reasoning unit for every listed sequence. */
ST_API int st_reason_decode(st_ctx *ctx, int32_t layer,
                     const int32_t *seq_ids, int32_t n_seq, const int32_t *visible_units,
                     const void *q, const void *k, const void *v, void *out,
                     uint32_t flags, void *stream);

/* A span of m_b >= 0 reasoning tokens per listed sequence at once (teacher-forced reasoning, or the
 * injected text that sets the final reasoning depth, Algorithm 1 last step). Token i of the span gets
 * position r+i, sees the source prefix [0, vis) (one vis for the whole span, as in st_reason_decode)
 * and reasoning positions 0 .. r+i. Packing as in st_append_source_chunk. A span of length 0 only
 * carries the flags. */
ST_API int st_reason_extend(st_ctx *ctx, int32_t layer,
                     const int32_t *seq_ids, const int32_t *cu_tokens, int32_t n_seq,
                     const int32_t *visible_units,
                     const void *q, const void *k, const void *v, void *out,
                     uint32_t flags, void *stream);

/* One pass over the training layout of Section 3.2 (the layout Eq. 2's mask is written on): for every listed
 * sequence the packed rows are [all source tokens ; all reasoning tokens], sequence after sequence in q/k/v/out
 * (device, as in the other calls; the total row count is bounded by max_tokens_per_call). The schedule comes as in
 * st_schedule_build, for n_seq sequences: n_units[b] units per sequence, their source and reasoning lengths
 * concatenated over the sequences in src_unit_len / rsn_unit_len (host arrays of sum(n_units) ints), final_len[b]
 * final-depth tokens, lag_units as in st_schedule_build. Every source row attends causally to the source tokens
 * (Eq. 2's unmodified part); every reasoning row of unit u attends to the source prefix of unit min(u + lag, U)
 * (Eq. 1 / the streaming mask region) and causally to the reasoning tokens; final-depth rows see the whole source.
 * Position ids follow the context's position_mode (streaming or concatenated; the unit-aligned variant is not
 * supported here). Forward only. The listed sequences must be empty; afterwards both caches hold the whole
 * sequence with N_EOS = N_EOT = n_units[b], exactly as if the units had been streamed in, so decoding can go on from
 * there. Multi-layer contexts: one call per layer, in order, with identical arguments. flags: ST_REFERENCE_KERNELS,
 * ST_IO_HOST. out may be NULL (caches only). */
ST_API int st_forward_packed(st_ctx *ctx, int32_t layer, const int32_t *seq_ids, int32_t n_seq, const int32_t *n_units,
                             const int32_t *src_unit_len, const int32_t *rsn_unit_len, const int32_t *final_len,
                             int32_t lag_units, const void *q, const void *k, const void *v, void *out, uint32_t flags,
                             void *stream);

/* Schedule generator (pure host, no context): turns a streaming-unit schedule -- n_units source-unit
 * lengths, the reasoning-unit length that follows each, and final_len final-depth tokens -- into the
 * paper's position ids and visibility. With S = sum(src_unit_len), R = sum(rsn_unit_len) + final_len:
 *   pos_ids[S+R] : source token j -> j; reasoning token r -> r (both counters start at zero);
 *   vis_len[R]   : visible source prefix of reasoning token r = end of unit min(u + lag_units, n_units)
 *                  for a token of unit u (1-based), S for final-depth tokens.
 * Either output may be NULL; *S_out / *R_out (may be NULL) receive S and R. */
ST_API int st_schedule_build(const int32_t *src_unit_len, const int32_t *rsn_unit_len, int32_t n_units,
                      int32_t final_len, int32_t lag_units,
                      int32_t *pos_ids, int32_t *vis_len, int64_t *S_out, int64_t *R_out);

/* Dense (S+R) x (S+R) streaming mask of the same schedule over the layout [source ; reasoning],
 * row-major, 1 = may attend (Eq. 2 applied to the causal mask, unit-level). Pure host. */
ST_API int st_schedule_dense_mask(const int32_t *src_unit_len, const int32_t *rsn_unit_len, int32_t n_units,
                           int32_t final_len, int32_t lag_units, uint8_t *mask);

/* Per-sequence state (host): any output pointer may be NULL. */
ST_API int st_seq_state(const st_ctx *ctx, int32_t seq_id, int32_t *source_len, int32_t *reason_len,
                 int32_t *n_eos, int32_t *n_eot);

/* Free pages left in each pool. */
ST_API int st_pages_free(const st_ctx *ctx, int64_t *source_pages, int64_t *reason_pages);

/* Test surface: what the kernels of the most recent attention call were given. For each packed
 * token of that call (up to cap): its position id, its visible source length (for a source token:
 * its own position + 1) and its visible reasoning length (0 for source tokens). Returns the token
 * count of that call in *n_tokens. */
ST_API int st_debug_last_call_meta(const st_ctx *ctx, int32_t *pos_ids, int32_t *vis_source, int32_t *vis_reason,
                            int32_t cap, int32_t *n_tokens);

/* Test surface: read back cache contents in plain layout. which = 0 source, 1 reasoning. Copies tokens
 * [tok0, tok0 + ntok) of sequence seq_id, layer `layer`, to HOST buffers k_out / v_out, each
 * [ntok][n_kv_heads][128] bf16 (k_out holds the rotated, rounded keys). Synchronises the device. */
ST_API int st_debug_read_cache(st_ctx *ctx, int32_t layer, int32_t seq_id, int32_t which,
                        int32_t tok0, int32_t ntok, void *k_out, void *v_out);

/* Test surface: the page ids of one sequence in one cache (which = 0 source, 1 reasoning), in token
 * order (entry i holds tokens 64 i .. 64 i + 63). Copies up to cap ids to the HOST array `pages` (may be
 * NULL) and returns the count in *n_pages. */
ST_API int st_debug_page_table(const st_ctx *ctx, int32_t seq_id, int32_t which, int32_t *pages, int32_t cap,
                               int32_t *n_pages);

/* Test surface for the bounded device-side waits (every wait inside the kernels gives up after 2 s, records the
 * status word and lets the kernel return, so that a stalled pipeline becomes an error code instead of a hang):
 * launches, on `stream`, a one-warp kernel whose only work is such a wait on a barrier that nothing ever arrives at,
 * with a limit of limit_ms milliseconds (1..2000, else ST_ERR_INVALID_ARG). After it st_device_status returns
 * ST_ERR_DEVICE_TIMEOUT once and the context is usable as before. Nothing faults, traps or spins without bound. */
ST_API int st_debug_wait_expiry(st_ctx *ctx, int32_t limit_ms, void *stream);

/* Device-side status word: ST_OK, ST_ERR_DEVICE_TIMEOUT if a kernel gave up a bounded wait, or
 * ST_ERR_DEVICE_CHECK if a kernel met a page id outside its pool, since the last call of this function
 * (which clears it). Synchronises the device. */
ST_API int st_device_status(st_ctx *ctx);

/* Test surface for the failure path of the attention calls: the n_steps-th device step issued from now on
 * (stream wait, page-table update, staging copy, append launch, attention launch; counted across calls)
 * fails on the host with ST_ERR_CUDA before it does anything, as a failing CUDA runtime call would.
 * n_steps = 0 disarms. Works on host-only contexts too. */
ST_API int st_debug_fail_after(st_ctx *ctx, int32_t n_steps);

/* Test surface for the kernels' page-id check: overwrites entry `index` of the device page table of
 * sequence seq_id (which = 0 source, 1 reasoning) with `page`, which may lie outside the pool. The next
 * kernel that reads the entry records ST_ERR_DEVICE_CHECK and skips the access. The host-side table is
 * not changed; st_reset followed by new appends rewrites the entry. Synchronises `stream`. */
ST_API int st_debug_corrupt_page_table(st_ctx *ctx, int32_t seq_id, int32_t which, int32_t index, int32_t page,
                                       void *stream);

/* Kernel timing for benchmarks. While enabled (every > 0), launches of the two dominant kernels are
 * bracketed by CUDA events on the stream they are launched on: every `every`-th launch of the dual-cache
 * decode kernel (which = 0; its launches within a run are alike, so a sample gives their average),
 * starting with the first after the call, and every launch of the tensor-core attention kernel of chunk
 * prefill and reasoning spans (which = 1; its launches differ, their sum is wanted). every = 1 brackets
 * all launches, every = 0 switches timing off, a negative value is ST_ERR_INVALID_ARG. A bracketed launch
 * is fully serialised against its neighbours in the stream (the events sit between them); the others
 * overlap their prologue with the tail of the kernel in front. st_kernel_timing_read waits for the
 * device, returns the number of bracketed launches and the sum of their durations in milliseconds since
 * the last read, and clears both. */
ST_API int st_kernel_timing_enable(st_ctx *ctx, int32_t every);
ST_API int st_kernel_timing_read(st_ctx *ctx, int32_t which, int64_t *launches, double *total_ms);

/* Number of kernel launches this context has issued so far. */
ST_API int64_t st_launch_count(const st_ctx *ctx);

/* Text of the last error of this context ("" if none); valid until the next call on the context.
 * With ctx == NULL: the last error of a failed st_create on this thread. */
ST_API const char *st_last_error_string(const st_ctx *ctx);

/* Dual-cache decode attention without any allocation. The paper has no counterpart of this call: it
 * exists for hosts that may not allocate device memory -- a serving process whose own memory manager has
 * claimed the whole GPU, so that a cudaMalloc issued from inside a library fails or takes memory the
 * manager counts as its own; or a latency-bound loop that cannot afford the device-wide synchronisation
 * cudaMalloc and cudaFree imply. It needs no st_ctx. It runs the same split-K decode and merge kernels as
 * st_reason_decode, but their workspace is a fixed array built into the library image (3.4 MB, resident on
 * every GPU that loads the library until the process ends), and it calls no allocating routine.
 *
 * For each of n_seq sequences it computes, per q head, attention of one rotated query over
 *   source keys [0, source_len[b])  and  reasoning keys [0, reason_len[b])   (reason_len counts the new token,
 * which must already be in the reasoning cache), exactly the row st_reason_decode produces.
 *
 * Inputs (device unless stated): pool_source / pool_reason = first byte of the layer's page blocks in each
 * pool (block of page p, kv head h at ((p * n_kv_heads) + h) * 32768; see "Pool layout" below), holding
 * n_pages_source / n_pages_reason pages; page_table_* = int32 [slot][table_stride_*] page ids;
 * slots / source_len / reason_len = HOST arrays of n_seq ints (page-table row, visible source tokens,
 * reasoning tokens); q_rotated = bf16 [n_seq][n_q_heads][128], already rotated at position
 * reason_len[b] - 1; out = fp32 [n_seq][n_q_heads][128]. softmax_scale 0 means 1/sqrt(128).
 * err / err_cap: optional HOST buffer that receives a message on failure.
 *
 * The page tables are the caller's, so the kernel checks every page id it reads against n_pages_* before it
 * builds an address from it: an id outside the pool is never dereferenced; the kernel stops, and
 * st_decode_static_status reports ST_ERR_DEVICE_CHECK (rows of that call are undefined, rows that only the
 * merge kernel would have written stay untouched). The same word reports a bounded wait that ran out
 * (ST_ERR_DEVICE_TIMEOUT). The call itself returns before the kernels have run and cannot report either.
 *
 * Limits: n_seq <= 112 and n_seq * n_kv_heads <= 512 per call; larger calls are rejected with
 * ST_ERR_INVALID_ARG and a message. The first call on a device looks up the address of the built-in array and
 * sets kernel attributes for that device, so make that first call outside any stream capture. All calls on a
 * GPU share the one array, which keeps the previous call's contents (the call clears the only word that must
 * start at zero): calls that overlap in time on the same GPU -- from different streams or threads -- race and
 * give wrong results; order them on one stream or with events. The call makes `device` current while it
 * runs and restores the caller's current device before it returns.
 *
 * Pool layout (also what cfg->pool_base holds): the source pool, then the reasoning pool; each pool is
 * [layer][page][kv head] blocks of 32768 bytes. */
ST_API int st_decode_attention_static(int32_t device, const void *pool_source, int64_t n_pages_source,
                                      const void *pool_reason, int64_t n_pages_reason,
                                      const int32_t *page_table_source, int32_t table_stride_source,
                                      const int32_t *page_table_reason, int32_t table_stride_reason,
                                      const int32_t *slots, const int32_t *source_len, const int32_t *reason_len,
                                      int32_t n_seq, const void *q_rotated, void *out, int32_t n_q_heads,
                                      int32_t n_kv_heads, float softmax_scale, void *stream, char *err,
                                      int32_t err_cap);

/* Status of the most recent st_decode_attention_static call on `device` (every such call clears the word when
 * its work starts on the stream, so read it before queueing the next call if each call is to be checked):
 * waits for `stream` (the stream the call was queued on) and reads the status word of the built-in workspace.
 * Returns ST_OK,
 * ST_ERR_DEVICE_CHECK (a page id outside its pool was met; the access was skipped), ST_ERR_DEVICE_TIMEOUT (a
 * bounded wait inside the kernels ran out), ST_ERR_INVALID_ARG (no such call has been made on the device) or
 * ST_ERR_CUDA. Like the call it reports on, it allocates nothing; the paper has no counterpart. */
ST_API int st_decode_static_status(int32_t device, void *stream);

/* Projection y = x W^T on the tensor cores: the Q, K, V and output projections of the attention block around the
 * path (the Qwen3 backbones of Section 4.1; the paper's method starts behind them, so there is no passage to cite).
 * x: device bf16 [m, k] row-major with leading dimension ldx (elements); w: device bf16 [n, k] row-major, one row per
 * output feature (leading dimension ldw); y: device [m, n] row-major (leading dimension ldy), bf16 or, with
 * out_fp32 != 0, fp32; fp32 accumulation. k and n must be multiples of 8, all three base pointers 16-byte aligned
 * and every leading dimension a multiple of 16 bytes. The caller owns all buffers; the call is asynchronous on
 * `stream`. Needs no st_ctx. The first call on a device allocates a 4-byte status word and sets kernel attributes
 * (make it outside stream capture). err / err_cap: optional HOST buffer for a message. The call makes `device`
 * current while it runs and restores the caller's device. */
ST_API int st_linear(int32_t device, const void *x, int64_t m, int64_t k, int64_t ldx, const void *w, int64_t n, int64_t ldw,
                     void *y, int64_t ldy, int32_t out_fp32, void *stream, char *err, int32_t err_cap);

/* Waits for `stream` and returns ST_OK, or ST_ERR_DEVICE_TIMEOUT if a bounded wait inside an st_linear kernel ran out
 * since the last call of this function (which clears the word); ST_ERR_INVALID_ARG before the first st_linear on the
 * device. */
ST_API int st_linear_status(int32_t device, void *stream);

/* fp32 -> bf16 (round to nearest even) of n contiguous values (n a multiple of 8, both pointers 16-byte aligned,
 * device memory): turns attention rows into the operand of the output projection. Asynchronous on `stream`. */
ST_API int st_cast_to_bf16(int32_t device, const void *src, void *dst, int64_t n, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* STREAMING_THINKER_H_ */
