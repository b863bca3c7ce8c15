/*
 * innerq.h - C ABI of libinnerq: decode-step attention over a KV cache quantised
 * group-wise along the inner dimension of each vector-matrix product (InnerQ),
 * for NVIDIA B200 (sm_100a).
 *
 * Conventions (all entry points)
 *   - Every tensor pointer is a DEVICE pointer unless the parameter is documented as
 *     host memory.  Tensors are contiguous, row-major, fp16 (IEEE binary16) unless
 *     stated otherwise.  The caller owns every device byte: the library never calls
 *     cudaMalloc/cudaFree and never synchronises the device; it enqueues work on the
 *     caller's stream (`cuda_stream` is a cudaStream_t passed as void*) and returns.
 *   - Every call returns an int status: INNERQ_OK (0) or a negative INNERQ_ERR_* code.
 *     Arguments are validated on the host before anything is launched; a failed call
 *     leaves the cache unchanged.  Nothing aborts, throws or traps.
 *   - The token count N of a cache lives in the host handle; which tokens are in the
 *     fp16 windows and which are quantised is a function of N alone.
 *   - (batch b, KV head h) is called a "unit" u = b * n_kv_heads + h.  Query head j
 *     reads KV head j / (n_q_heads / n_kv_heads).
 *   - Supported shapes: head_dim == 128; group in {32, 64, 128}; bits in {2, 3, 4};
 *     n_q_heads a multiple of n_kv_heads.
 */
#ifndef INNERQ_H_
#define INNERQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  INNERQ_OK = 0,
  INNERQ_ERR_INVALID_ARG = -1,      /* null pointer, negative size, inconsistent config          */
  INNERQ_ERR_UNSUPPORTED = -2,      /* bits / group / head_dim combination not implemented       */
  INNERQ_ERR_CAPACITY = -3,         /* token count would exceed max_tokens                        */
  INNERQ_ERR_BUFFER_TOO_SMALL = -4, /* caller's cache or workspace buffer smaller than required   */
  INNERQ_ERR_CUDA = -5              /* a CUDA runtime call or launch failed                       */
};

enum { INNERQ_MODE_SYM = 0, INNERQ_MODE_ASYM = 1, INNERQ_MODE_HYBRID = 2 };
enum { INNERQ_SYM_FULLRANGE = 0, INNERQ_SYM_PAPER_LITERAL = 1 };
enum { INNERQ_GROUPING_INNER = 0, INNERQ_GROUPING_OUTER = 1, INNERQ_GROUPING_FP16 = 2 };

/* Hyper-parameters of a cache (Section "Quantization Scheme": b-bit group-wise quantisation with
 * group size G; Section "High-precision Window": w_sink, w_recent). */
typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim;
  int32_t max_tokens;   /* capacity: N never exceeds this                                        */
  int32_t group;        /* G                                                                     */
  int32_t k_bits, v_bits;
  int32_t k_mode, v_mode;   /* INNERQ_MODE_*; per-group choice when HYBRID (Section "Hybrid Quantization") */
  int32_t sym_variant;  /* INNERQ_SYM_*: FULLRANGE  S = max|G|/(2^(b-1)-1), codes in [-(2^(b-1)-1), 2^(b-1)-1];
                           PAPER_LITERAL  S = max|G|/(2^b-1) as printed, codes clipped to [-2^(b-1), 2^(b-1)-1] */
  int32_t w_sink, w_recent;
  int32_t grouping;     /* INNER: K grouped along head_dim inside a token, V along tokens inside a channel
                           (Section "InnerQ"); OUTER: the reverse, asymmetric, no key normalisation (the
                           outer-grouped method the paper compares against); FP16: unquantised cache     */
  int32_t k_normalize;  /* 1: per-channel key normalisation (Section "Per-channel Normalization of K")  */
  float sm_scale;       /* softmax scale; 0 selects 1/sqrt(head_dim)                                     */
} innerq_config_t;

typedef struct innerq_cache innerq_cache_t;   /* opaque host handle: layout, views, host copy of N */

/* Canonical (unpacked) view of a cache, for inspection, tests and checkpoints.  All pointers are
 * DEVICE buffers provided by the caller, or NULL to skip that array.  Shapes use the capacity
 * cap = max_tokens; tokens are oldest first; only the first n_* entries are written.
 *   k_code, v_code    uint8  [units][cap][head_dim]     unsigned codes (offset-binary for symmetric groups)
 *   k_scale, k_zero   uint16 [units][cap][head_dim/G]   (INNER)  or [units][cap/G + 1][head_dim] (OUTER)
 *   v_scale, v_zero   uint16 [units][cap/G + 1][head_dim] (INNER) or [units][cap][head_dim/G]    (OUTER)
 *                     fp16 bit patterns; bit 15 of a scale is the hybrid mask M; zero is 0 when M = 0
 *   norm              float  [units][head_dim]
 *   k_sink, v_sink    fp16   [units][w_sink][head_dim]
 *   k_recent,v_recent fp16   [units][w_recent + G][head_dim]
 * The counts are filled in by innerq_cache_export (host fields). */
typedef struct {
  uint8_t *k_code, *v_code;
  uint16_t *k_scale, *k_zero, *v_scale, *v_zero;
  float *norm;
  uint16_t *k_sink, *v_sink, *k_recent, *v_recent;
  int32_t n_tokens, n_sink, n_qk, n_qv, n_k_recent, n_v_recent;
} innerq_export_t;

/* Size query.  Writes the number of device bytes the caller must provide for the packed cache
 * (codes, fp16 scale/zero pairs with the mask in the scale's sign bit, fp16 window ring buffers,
 * key norms) and for the scratch workspace (split partials of the decode kernel, reduction
 * scratch of the prefill).  Host pointers.  Errors: INVALID_ARG, UNSUPPORTED. */
int innerq_cache_bytes(const innerq_config_t* cfg, size_t* cache_bytes, size_t* workspace_bytes);

/* Size of the packed, per-token payload only: bytes of codes + scales + zero-points that one
 * quantised token of one unit occupies for K (`k_bytes`) and V (`v_bytes`), as double so that the
 * per-group metadata of V is amortised over its G tokens.  Used to check the effective bit-widths
 * of Table "bits".  Host pointers. */
int innerq_token_payload_bytes(const innerq_config_t* cfg, double* k_bytes, double* v_bytes);

/* Create a handle over caller-provided device buffers (256-byte aligned, sizes from
 * innerq_cache_bytes).  The cache starts empty (N = 0, norm = 1).  The buffers must stay valid
 * until innerq_cache_destroy.  `*out` receives the handle.  Enqueues a clear of the buffers on
 * `cuda_stream`.  Errors: INVALID_ARG, UNSUPPORTED, BUFFER_TOO_SMALL, CUDA. */
int innerq_cache_create(const innerq_config_t* cfg, void* dev_cache, size_t cache_bytes,
                        void* dev_workspace, size_t workspace_bytes, void* cuda_stream,
                        innerq_cache_t** out);

/* Frees the host handle only. */
int innerq_cache_destroy(innerq_cache_t* cache);

/* ---- Paged caches -------------------------------------------------------------------------------------
 * The packed part of a cache (codes and scale / zero-point words of the quantised middle, which is what grows
 * with the context; Section "High-precision Window" keeps the rest in two fixed-size fp16 windows) can live in
 * pages of `page_tokens` tokens drawn from a pool that many caches share, instead of inside the cache buffer.
 * page_tokens is a power of two, at least 128 (so a page holds whole groups for every G); a page holds those tokens of all
 * batch * n_kv_heads units of the cache.  The cache buffer then holds only the norms, the fp16 windows and a page
 * table; the pool is one caller-owned device buffer of pool_pages * page_bytes bytes, 256-byte aligned, and a page
 * is named by its index in it.  The caller decides which page goes to which cache (free list, eviction, reuse);
 * the library checks indices against pool_pages and against the cache's own pages, not across caches.
 * Kernels, results and every other entry point are the same as for a contiguous cache; batched calls need caches
 * on one pool.  Not available for grouping FP16 (UNSUPPORTED). */

/* Sizes for a paged cache: bytes of the cache buffer and the workspace, bytes of one page, and the most page slots
 * a cache can use (max_tokens tokens).  Host pointers.  Errors: INVALID_ARG (page_tokens), UNSUPPORTED. */
int innerq_paged_cache_bytes(const innerq_config_t* cfg, int32_t page_tokens, size_t* cache_bytes,
                             size_t* workspace_bytes, size_t* page_bytes, int32_t* max_pages);

/* As innerq_cache_create, over the page pool `dev_pool` of `pool_pages` pages.  The cache starts with no pages. */
int innerq_cache_create_paged(const innerq_config_t* cfg, int32_t page_tokens, void* dev_cache, size_t cache_bytes,
                              void* dev_workspace, size_t workspace_bytes, void* dev_pool, int32_t pool_pages,
                              void* cuda_stream, innerq_cache_t** out);

/* Page slots that the cache needs to hold n_tokens tokens (0 for a contiguous cache), or a negative error code.
 * A prefill to n tokens or an append that makes N = n returns INNERQ_ERR_CAPACITY unless at least this many
 * pages are assigned. */
int innerq_cache_pages_for(const innerq_cache_t* cache, int32_t n_tokens);

/* Pages assigned so far, or a negative error code. */
int innerq_cache_pages_assigned(const innerq_cache_t* cache);

/* Gives the cache `n` more pages: page slots [assigned, assigned + n) map to pool pages pages_host[0..n) (HOST
 * array; read before the call returns).  Enqueues the copy of the new table entries on `cuda_stream` (the
 * stream of the cache's other calls); the pages' old contents are dead from then on.  Pages may be assigned any
 * time before the call that needs them; assigning them a few steps early keeps the copy out of the step that
 * crosses the page boundary.  Errors: INVALID_ARG (contiguous cache, index out of range or already in this
 * cache), CAPACITY (more than max_pages), CUDA. */
int innerq_cache_assign_pages(innerq_cache_t* cache, const int32_t* pages_host, int32_t n, void* cuda_stream);

/* Empties the cache (N = 0) and hands its pages back: writes their pool indices to pages_host[0..count) (HOST
 * array of `capacity` entries) and returns count, or a negative error code (BUFFER_TOO_SMALL leaves the cache as
 * it was).  Host-side only: kernels already enqueued for this cache still read the pages, so the caller may give
 * them to another cache only on the same stream (or after synchronising). */
int innerq_cache_release_pages(innerq_cache_t* cache, int32_t* pages_host, int32_t capacity);

/* Number of tokens currently cached (host value), or a negative error code. */
int innerq_cache_n_tokens(const innerq_cache_t* cache);

/* Prefill quantisation (Section "High-precision Window", window-split equation; Section
 * "Per-channel Normalization of K").  Resets the cache to exactly n_tokens tokens taken from
 * k, v: fp16 [batch][n_kv_heads][n_tokens][head_dim].  Computes norm[c] = sqrt(max_t |K[t,c]|)
 * per unit over all n_tokens (when k_normalize), keeps the first w_sink and the last w_recent
 * tokens in fp16, and quantises the middle: per group statistics, symmetric / asymmetric
 * candidates, the hybrid choice, bit-packing.  Tokens grouped G at a time (V under INNER) that do
 * not fill a group stay fp16 in front of the recent window.  0 <= n_tokens <= max_tokens.
 * Errors: INVALID_ARG, CAPACITY, CUDA. */
int innerq_quantize_prefill(innerq_cache_t* cache, const void* k, const void* v, int32_t n_tokens,
                            void* cuda_stream);

/* Append the decode step's own token (Section "High-precision Window", last paragraph; Section
 * "Latency": one key token is quantised every step, G value tokens every G steps; the reverse
 * under OUTER).  k_new, v_new: fp16 [batch][n_kv_heads][head_dim].  The token enters the sink
 * window while it is not full, else the recent window; tokens leaving the recent window are
 * normalised with the norm fixed at prefill (keys) and quantised into the packed cache.
 * Stream order as for innerq_decode_attention: when the cache's previous call was a decode, this kernel reads
 * k_new, v_new and writes the cache while that decode is still running (the decode lets it start once it has
 * read everything an append writes: the fp16 windows and the newest packed rows; the packed range it goes on
 * streaming is never written again), so k_new and v_new must be complete before the call under the same rule as `q`.
 * Errors: INVALID_ARG, CAPACITY, CUDA. */
int innerq_append_token(innerq_cache_t* cache, const void* k_new, const void* v_new, void* cuda_stream);

/* Decode attention (attention equations S = QK^T, P = softmax(S / sqrt(d_h)), O = PV with
 * N_Q = 1, over K = [K_sink; dequant(K^); K_recent] and the same for V; hybrid dequantisation
 * S*K^ + M*Z; Section "InnerQ").  q: fp16 [batch][n_q_heads][head_dim]; out: fp16, same shape,
 * fully overwritten.  Attends over all N cached tokens (append the step's token first); N >= 1.
 * Scores of quantised key rows use q' = q * norm; dequantisation happens in registers, scale and
 * zero-point are applied once per group.  Uses the workspace; two decodes on the same cache must
 * not overlap.
 * Stream order: the kernels of append and decode are launched as programmatic dependents of the kernel before
 * them in the stream, and the decode streams the part of the cache that no earlier call can still be writing
 * (what was packed when the cache's previous decode was launched) and reads `q` BEFORE it waits for that kernel.
 * All calls on one cache must therefore be enqueued in order on one stream (or be ordered by events), and `q`
 * must not come from a kernel that signals programmatic launch completion before it has written `q`; ordinary
 * kernels and copies earlier in the stream are always complete by then.
 * Errors: INVALID_ARG (N == 0 included), CUDA. */
int innerq_decode_attention(innerq_cache_t* cache, const void* q, void* out, void* cuda_stream);

/* One decode step from HOST buffers (the sequence the paper's Section "Latency" times per generated token:
 * quantise-on-evict of the step's own token, then attention over the cache): enqueues on `cuda_stream`
 *   host -> device copies of k_new, v_new ([batch][n_kv_heads][head_dim] fp16) and q ([batch][n_q_heads][head_dim]),
 *   innerq_append_token, innerq_decode_attention, device -> host copy of out ([batch][n_q_heads][head_dim] fp16).
 * `dev_staging` is caller-owned device memory of at least innerq_step_staging_bytes(cfg) bytes, 256-byte aligned,
 * used for the device copies of the four tensors; it must stay untouched until the stream has passed this step.
 * If all four host buffers are pinned (page-locked and mapped, e.g. cudaHostAlloc / cudaHostRegister), the kernels
 * read the inputs and write the result in place over the bus and no copy is enqueued; otherwise the tensors are
 * staged through `dev_staging` with one copy each (pageable memory makes those copies block the caller).
 * `out_host` holds the result once `cuda_stream` has been synchronised.  The call itself does not synchronise
 * and allocates nothing.  INVALID_ARG and CAPACITY are detected before anything is enqueued; after a CUDA error
 * the step may be partly enqueued.
 * Errors: INVALID_ARG, CAPACITY, UNSUPPORTED, CUDA. */
int innerq_decode_step_host(innerq_cache_t* cache, const void* k_new_host, const void* v_new_host, const void* q_host,
                            void* out_host, void* dev_staging, void* cuda_stream);

/* Bytes of device staging innerq_decode_step_host needs for this configuration.  Errors: INVALID_ARG. */
int innerq_step_staging_bytes(const innerq_config_t* cfg, size_t* bytes);

/* Decode attention for n_q consecutive query tokens per sequence in one call (the verification step of
 * speculative decoding, or a short chunked prefill).  The paper decodes one token per step (Section
 * "Preliminaries"); this is that definition applied to n_q queries against one cache state, with a causal mask:
 * the cache already holds the n_q tokens' own keys and values as its newest tokens (append them first), and
 * query token i (0 <= i < n_q) attends to tokens 0 .. N - n_q + i.
 *   q, out        : device, fp16 [batch, n_q, n_q_heads, head_dim]; n_q = 1 is innerq_decode_attention.
 *   dev_scratch   : device, 256-byte aligned, at least innerq_multi_query_scratch_bytes(cfg) bytes; owned by the
 *                   caller, used only during the call (split partials of up to four query rows per KV head).
 * The rows of a KV head (its n_q * r query heads) are processed four per pass over the packed cache: with one
 * query head per KV head four query tokens share one pass, with four or more each token takes its own.
 * Limits: the fused kernel only (packed inner- or outer-grouped cache in a format it supports; decode variant
 * 0 or 2); the n_q - 1 newest tokens must all lie outside the token range in which keys AND values are packed
 * (always true for n_q - 1 <= w_recent once the windows are full).  Otherwise UNSUPPORTED, nothing launched.
 * Errors: INVALID_ARG (n_q < 1 or n_q > N included), BUFFER_TOO_SMALL, UNSUPPORTED, CUDA. */
int innerq_decode_attention_multi(innerq_cache_t* cache, const void* q, void* out, int32_t n_q, void* dev_scratch,
                                  size_t scratch_bytes, void* cuda_stream);

/* Bytes of device scratch innerq_decode_attention_multi needs (independent of n_q).  Errors: INVALID_ARG. */
int innerq_multi_query_scratch_bytes(const innerq_config_t* cfg, size_t* bytes);

/* Append and decode for several caches in one call each: sequences of different lengths that are decoded together
 * (continuous batching).  The paper's kernels take one cache of one length; here every sequence has its own cache
 * object (typically created with batch = 1), its own token count and its own eviction schedule, and one launch
 * serves them all: block x of the grid is (cache i, unit u), and every cache brings its own token counts.
 *   caches : host array of n handles (1 <= n <= 4096; one launch per 32 of them), all created from the SAME
 *            configuration (max_tokens included) and all different; each with its own workspace.
 *   k_new, v_new : device, fp16 [n][batch, n_kv_heads, head_dim]  (cache i's rows at index i)
 *   q, out       : device, fp16 [n][batch, n_q_heads, head_dim]
 * innerq_append_token_batched appends one token to every listed cache (a cache that should not advance is left
 * out of the list); innerq_decode_attention_batched attends for every listed cache over its own tokens.
 * The decode needs the fused kernel (packed inner- or outer-grouped cache in a format it supports, decode variant
 * 0 or 2 on the first cache): otherwise UNSUPPORTED.  Split counts follow the first cache's decode options.
 * Errors: INVALID_ARG (different configurations, a cache listed twice, an empty cache in the decode), CAPACITY (a
 * listed cache is full; nothing is appended to any), UNSUPPORTED, CUDA. */
int innerq_append_token_batched(innerq_cache_t* const* caches, int32_t n, const void* k_new, const void* v_new,
                                void* cuda_stream);
int innerq_decode_attention_batched(innerq_cache_t* const* caches, int32_t n, const void* q, void* out,
                                    void* cuda_stream);

/* Same computation and arguments as innerq_decode_attention, for callers that cannot give the decode
 * step any scratch memory of their own.  (The paper has no counterpart; this is an integration aid.)
 * Typical cases: the workspace passed to innerq_cache_create was only lent for the prefill and has gone
 * back to a pool; or the decode runs in a part of a program (a serving loop with a frozen memory plan,
 * a plug-in without access to the host's allocator) where device memory cannot be allocated, so no
 * workspace can be produced on demand.  Here the kernel's scratch (per-split partial results, merge
 * tickets, error word) lives in a 4 MiB array that is part of the library image on every GPU that loads
 * the library, until the process exits.  The call allocates nothing and frees nothing.
 *   - Limit: the configuration's workspace size (innerq_cache_bytes) must not exceed 4 MiB; otherwise
 *     the call returns INNERQ_ERR_BUFFER_TOO_SMALL and launches nothing.
 *   - The first call on each device looks up the array's device address (one runtime query, made with
 *     that device current).  Make that first call outside any stream capture.
 *   - All caches and all calls on a device share the one array, which keeps the contents of the previous
 *     call; the parts that must start at zero are cleared on `cuda_stream` before the launch.  Two such
 *     calls must not overlap on the GPU (different streams without ordering): they would race on the array.
 *   - The array that is used belongs to the CURRENT device: the cache must live on it (INVALID_ARG if not).
 *   - The caller's workspace is not touched.  The error word of this call is in the array as well;
 *     innerq_read_device_error (called with the same device current) reports it together with the
 *     workspace's own word.  It tells about the last such call only: the next one clears it.
 * Errors: INVALID_ARG (N == 0 included), BUFFER_TOO_SMALL, UNSUPPORTED, CUDA. */
int innerq_decode_attention_static(innerq_cache_t* cache, const void* q, void* out, void* cuda_stream);

/* Unpack the cache into canonical arrays (see innerq_export_t).  `ex` is a host struct holding
 * device pointers; counts are written to it before the call returns, array contents when the
 * stream reaches the enqueued kernels.  Errors: INVALID_ARG, CUDA. */
int innerq_cache_export(innerq_cache_t* cache, innerq_export_t* ex, void* cuda_stream);

/* The inverse of innerq_cache_export (checkpoint / resume, moving a sequence between caches or processes): fills the
 * cache for `n_tokens` tokens from canonical arrays of the SAME configuration, in the shapes and order that the
 * export writes (innerq_export_t; its count fields are ignored: the partition of n_tokens into sink, packed and recent
 * tokens is a function of n_tokens and the configuration).  Replaces the cache's contents like a prefill; a cache
 * restored this way continues (append, decode) exactly like the one that was exported.  The arrays are read when the
 * stream reaches the enqueued kernels and must stay valid until then.  Codes are taken as given (values above 2^b - 1
 * would corrupt neighbouring fields: the caller's responsibility).  The paper has no counterpart.
 * Errors: INVALID_ARG (a needed array is NULL), CAPACITY (n_tokens > max_tokens, or a paged cache without the pages
 * for n_tokens), CUDA. */
int innerq_cache_import(innerq_cache_t* cache, const innerq_export_t* ex, int32_t n_tokens, void* cuda_stream);

/* Tuning knobs for experiments; both default to 0 = automatic.
 *   n_splits : number of token ranges each unit is split into by the decode kernel.  0 = automatic: one wave of two
 *              CTAs per SM, the lowest latency for a launch that runs alone.  148 / (batch * n_kv_heads), i.e. one
 *              CTA per SM and launch, lets consecutive launches share the GPU and hide each other's start and end:
 *              10-15 % more steps per second in a loop of back-to-back calls, 10-25 % slower for a launch alone.
 *   variant  : 0 automatic, 1 plain SIMT kernel, 2 warp-MMA kernel (where supported; UNSUPPORTED otherwise),
 *              3 / 4 warp-MMA kernel with one / two 32-token chunks per loop iteration (sets a process-wide knob).
 *              6 / 7 TIMING ONLY, the output is wrong on purpose: the warp-MMA kernel with the unpack + MMA work of
 *              its key side (6) or value side (7) left out of the streaming loop, the bytes still streamed; what
 *              a side costs is the difference to the full kernel (process-wide knob; any other variant clears it;
 *              contiguous caches with 2-bit keys and values or 4-bit keys and values, the 3-bit / 3-bit and
 *              3-bit / 2-bit formats of the latency study (both sides with zero-points, both without, and 3 / 2 with
 *              scale-only keys and full values) and the outer-grouped cache: UNSUPPORTED elsewhere).
 * Errors: INVALID_ARG. */
int innerq_set_decode_options(innerq_cache_t* cache, int32_t n_splits, int32_t variant);

/* The decode kernel waits for its asynchronous copies with a bounded number of polls; if a wait ever
 * runs out it records that in a device-side error word, contributes nothing for the affected token
 * range and returns normally.  This call copies the word to the host and SYNCHRONISES `cuda_stream`
 * (the only entry point that does).  Returns 0 (no error), 1 (a wait ran out since the cache was
 * created, or in the last innerq_decode_attention_static call of this cache's configuration on the
 * current device) or a negative error code. */
int innerq_read_device_error(innerq_cache_t* cache, void* cuda_stream);

/* Test support for the call above: enqueues a one-warp kernel that waits, with the decode kernels' own bounded
 * wait (256 polls), on a barrier on which nothing ever arrives, gives up, and records that in the cache's device
 * error word exactly as a decode warp would; the kernel returns normally and the context stays usable.  After it
 * innerq_read_device_error returns 1 for this cache for good (the word is never cleared), so use a cache made for
 * the test.  Does not synchronise.  Errors: INVALID_ARG, CUDA. */
int innerq_selftest_wait_expiry(innerq_cache_t* cache, void* cuda_stream);

/* Number of kernels the last call of each kind launched (for launch accounting):
 * which = 0 prefill, 1 append, 2 decode.  Returns the count or a negative error code. */
int innerq_last_launch_count(const innerq_cache_t* cache, int32_t which);

/* Static string for a status code; never NULL. */
const char* innerq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* INNERQ_H_ */
