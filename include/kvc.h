/*
 * kvc -- budgeted KV cache for block-wise ("compress as you prefill") multimodal prefill on B200.
 *
 * C ABI.  No exception crosses it; every function returns an int status (0 = KVC_OK) unless noted.
 * All tensor arguments are raw pointers; whether a pointer is HOST or DEVICE memory is stated per
 * argument.  The caller owns every device buffer (cache blobs, workspace, q/k/v/out); the context
 * owns only host-side state (configuration and the current cache length of every layer).
 *
 * The library implements the per-block body of the paper's Alg. 1 ("Block-wise Prefill with KV
 * Eviction"): the caller loops over blocks (and layers) and calls kvc_prefill_chunk once per
 * (block, layer).  Notation: L layers, Hq query heads, Hkv kv-heads, G = Hq/Hkv, d = head_dim,
 * B = budget (the paper's M), n = tokens in this block (the paper's b), n_c = cache length before
 * the call, tot = n_c + n, w = observer window, cap = B + max_chunk rounded up to 128.
 *
 * One call does, on the caller's stream, for every kv-head independently:
 *   a0  append   C <- C u (K_i, V_i)                                          (Alg. 1)
 *   a1  attend   out = softmax(q k^T / sqrt(d)) v over cache u block, causal
 *                inside the block                                             (Eq. 1)
 *   a2  score    if tot > B: importance of every cached key = attention probability it receives
 *                from the observer queries (the block's last w rows), summed over those rows and
 *                over the G query heads sharing the kv-head                   (Eq. 4)
 *   a3  select   evict the tot - B lowest-scoring entries; ties keep the older entry; the
 *                observers' own w keys are never evicted                      (Alg. 1, Evict)
 *   a4  compact  retained entries are moved into rows [0, B); length becomes B (Sec. 3.1)
 */
#ifndef KVC_H_
#define KVC_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvc_ctx kvc_ctx; /* opaque, host memory, created/destroyed by the library */

/* status codes */
#define KVC_OK        0
#define KVC_EINVAL   -1  /* bad configuration or argument (null/misaligned pointer, n out of range, ...) */
#define KVC_ESTATE   -2  /* call order violated (layer not reset, destroyed context, ...)              */
#define KVC_ECUDA    -3  /* a CUDA call or launch failed; text in kvc_last_error                       */
#define KVC_ETIMEOUT -4  /* a bounded device-side wait ran out (reported by kvc_status)                */

typedef enum { KVC_F32 = 0, KVC_BF16 = 1 } kvc_dtype;
typedef enum {
  KVC_SCORE_ATTN = 0,    /* query-aware score, Eq. 4 */
  KVC_SCORE_KEYDIFF = 1  /* query-agnostic score, Sec. 3.2: anchor = mean of the cached keys after the append,
                            score = 1 - cosine(key, anchor); the least similar keys are kept */
} kvc_policy;

/* flags */
#define KVC_FLAG_CUDA_CORES 1u /* bf16 only: run attention/score on the CUDA-core kernels used for
                                  fp32 instead of the tcgen05 tensor-core kernels (diagnostic) */
#define KVC_FLAG_NO_KEY_SPLIT 4u /* attention: never split the key range over a thread-block cluster */
#define KVC_FLAG_NO_PDL 8u     /* launch the kernels in plain stream order instead of letting each start
                                  while its predecessor drains (programmatic dependent launch) */

#define KVC_FLAG_ASYNC_COMPRESS 16u /* bf16 tensor-core path, kvc_prefill_chunk / _proxy only: score, select and
                                  compact (Alg. 1's eviction step) of a layer are enqueued on a stream the context
                                  owns, ordered after the layer's attention, so that they run beside whatever the
                                  caller enqueues next on its own stream (in a decoder stack the next layer needs
                                  this layer's output, not its compacted cache).  The layer then uses workspace
                                  slot `layer` (kvc_workspace_view / kvc_move_counts take that slot).  Contract:
                                  the call's q must stay unchanged, and the layer's cache must not be read by the
                                  caller, until the next kvc call on that layer, kvc_reset of it, kvc_status or
                                  kvc_join has been enqueued on the stream that does so; every kvc call orders
                                  itself after the pending work of the layers it touches.  Inside a stream
                                  capture, call kvc_join before ending the capture.  All calls of one context must
                                  come from one host thread. */

typedef struct {
  int n_layers;        /* L >= 1                                                                 */
  int n_q_heads;       /* Hq, multiple of n_kv_heads; consecutive query heads share a kv-head     */
  int n_kv_heads;      /* Hkv                                                                     */
  int head_dim;        /* d in {64, 128}                                                          */
  int dtype;           /* kvc_dtype of q/k/v/out and of the cached keys/values                    */
  int budget;          /* B: entries kept per (layer, kv-head) = memory budget M of Alg. 1        */
  int max_chunk;       /* largest n ever passed = block size b of Alg. 1                          */
  int obs_window;      /* w; 0 -> 32.  The window used by a call is min(w, n); needs w <= B       */
  int policy;          /* kvc_policy                                                              */
  float softmax_scale; /* 0 -> 1/sqrt(head_dim) as in Eq. 1 and Eq. 4                             */
  int device;          /* CUDA device ordinal the context is bound to                             */
  unsigned flags;      /* KVC_FLAG_*                                                              */
} kvc_config;

/* Borrowed view of one layer's cache (pointers into the caller's cache blob, nothing is copied).
 * Rows [len, cap) are unspecified.  The order of entries is unspecified; pos identifies them. */
typedef struct {
  void* k;              /* DEVICE  [Hkv][cap][d], dtype                      */
  void* v;              /* DEVICE  [Hkv][cap][d], dtype                      */
  int* pos;             /* DEVICE  [Hkv][cap] int32, absolute token position */
  int len;              /* valid entries per kv-head (same for every head)   */
  int cap;              /* row capacity per kv-head                          */
  int n_kv_heads, head_dim, dtype;
} kvc_view;

/* Sec. 3, Alg. 1 inputs (block size b, budget M) plus the attention shape.  Validates the
 * configuration (Hq % Hkv == 0, d in {64,128}, 1 <= w <= B, max_chunk >= 1, G <= 128) and creates
 * the host context.  *out is set to NULL on failure.  Allocates no device memory. */
int kvc_create(const kvc_config* cfg, kvc_ctx** out);

/* Frees the host context.  Device buffers stay with the caller. */
int kvc_destroy(kvc_ctx* ctx);

/* Sizes the caller must allocate (device memory, 256-byte aligned): per_layer = bytes of one
 * layer's cache blob (K, V, pos; this is the physical bound of Eq. 2 with sequence length cap);
 * workspace = bytes of the scratch area shared by all layers (log-sum-exp of the last block,
 * scores, move lists, status word).  Either pointer may be NULL. */
int kvc_cache_nbytes(const kvc_ctx* ctx, size_t* per_layer, size_t* workspace);

/* Clears the workspace header (status word).  Call once after allocating a workspace, before the
 * first kvc_prefill_chunk that uses it.  Asynchronous on `stream`. */
int kvc_workspace_init(kvc_ctx* ctx, void* workspace, void* stream);

/* Alg. 1 "C <- empty" for `n_layers` consecutive layers starting at `layer`: zero-fills the blobs
 * (asynchronously on `stream`) and sets their length to 0.  Must precede the first
 * kvc_prefill_chunk of a layer.  cache: DEVICE, blob of layer `layer`; blobs of consecutive
 * layers are cache_layer_stride bytes apart (ignored when n_layers == 1). */
int kvc_reset(kvc_ctx* ctx, int layer, int n_layers, void* cache, size_t cache_layer_stride,
              void* stream);

/* The body of Alg. 1's loop for one block and one layer (steps a0..a4 above; Eq. 1, Eq. 4).
 *   q   DEVICE [n][Hq ][d]  queries of the block (already position-encoded), dtype
 *   k,v DEVICE [n][Hkv][d]  keys / values of the block, dtype
 *   n   1 <= n <= max_chunk; pos0 = absolute position of the block's first token.  One exception, the
 *       hybrid schedule the paper uses by default (Sec. 5, Budgeting: the first M tokens go through in a
 *       single forward): a layer whose cache is EMPTY accepts up to B tokens in one call (nothing is evicted)
 *   cache      DEVICE this layer's blob (kvc_cache_nbytes per_layer bytes); read and written
 *   workspace  DEVICE scratch (kvc_cache_nbytes workspace bytes); calls sharing a workspace must
 *              be ordered on one stream
 *   out DEVICE [n][Hq][d]   attention output, dtype
 *   stream     cudaStream_t; the call only enqueues work and returns
 * All pointers must be 16-byte aligned.  Returns KVC_EINVAL / KVC_ESTATE / KVC_ECUDA without
 * enqueuing anything on failure of the host checks. */
int kvc_prefill_chunk(kvc_ctx* ctx, int layer, const void* q, const void* k, const void* v, int n,
                      long long pos0, void* cache, void* workspace, void* out, void* stream);

/* The query-aware policy with the text prompt known up front (Sec. 3.2, Query-Aware Eviction: the observers
 * are proxy query tokens taken from the text prompt and attend over the cached keys): the last n_proxy of the
 * n rows of q/k/v are proxy query tokens.  They are processed like the other tokens of the block (they
 * attend causally to the cache, the block and the proxies before them, and `out` has their rows too),
 * they are the observers of Eq. 4 -- with the softmax normaliser of everything they attend to -- but
 * their keys and values do not stay in the cache, and no entry is protected: all n_c + n - n_proxy
 * entries compete and the B best stay.  1 <= n_proxy < n <= max_chunk; pos0 is the position of the
 * block's first real token.  Cache rows beyond the new length are scratch.  Otherwise as
 * kvc_prefill_chunk. */
int kvc_prefill_chunk_proxy(kvc_ctx* ctx, int layer, const void* q, const void* k, const void* v, int n,
                            int n_proxy, long long pos0, void* cache, void* workspace, void* out,
                            void* stream);

/* Same as kvc_prefill_chunk for `n_layers` consecutive layers in one set of launches (the layer
 * index becomes a grid dimension).  Only meaningful when every layer's q/k/v exist up front
 * (synthetic inputs, or layers of independent models); a real decoder stack cannot use it because
 * layer l+1's input depends on layer l's output.  Layer i's tensors are at q + i*q_layer_stride
 * (strides in ELEMENTS for q/k/v/out, in BYTES for the cache).  All layers must hold the same
 * cache length. */
int kvc_prefill_chunk_layers(kvc_ctx* ctx, int layer0, int n_layers, const void* q,
                             long long q_layer_stride, const void* k, const void* v,
                             long long kv_layer_stride, int n, long long pos0, void* cache,
                             size_t cache_layer_stride, void* workspace, void* out,
                             long long out_layer_stride, void* stream);

/* Bytes of the DEVICE staging buffer kvc_prefill_chunk_host needs (two halves, each with room for q, k, v
 * and out of a block of max(max_chunk, B) tokens). */
int kvc_staging_nbytes(const kvc_ctx* ctx, size_t* nbytes);

/* kvc_prefill_chunk with HOST q/k/v/out (pinned memory recommended): copies the block's q, k, v
 * into `staging` (DEVICE, kvc_staging_nbytes bytes, 256-byte aligned), runs the block, copies `out`
 * back to the host.  Nothing blocks the host.  Consecutive calls alternate between the two halves of
 * `staging`; the copies in either direction run on two streams the context owns: the host-to-device copies of a
 * call start as soon as the block that last used its half is done and `stream` waits for them before the kernels,
 * the device-to-host copy of `out` follows the kernels, and `stream` waits for it only behind the NEXT call's
 * kernels.  So the inbound copies, the kernels and the outbound copy of three consecutive calls overlap.
 * The host inputs of a call may be reused once `stream` has completed the call.  out_host of a call is complete
 * once `stream` has completed the next kvc_prefill_chunk_host call of the context, or a kvc_host_flush after the
 * call.  (Pass the same `staging` to every call of a context; a run-time error before the kernels leaves the call
 * without effect on the cache.) */
int kvc_prefill_chunk_host(kvc_ctx* ctx, int layer, const void* q_host, const void* k_host,
                           const void* v_host, int n, long long pos0, void* cache, void* workspace,
                           void* staging, void* out_host, void* stream);

/* Makes `stream` wait for the device-to-host copies of all kvc_prefill_chunk_host calls made so far (no host wait;
 * nothing is enqueued when there was none): once `stream` has completed, every out_host is filled. */
int kvc_host_flush(kvc_ctx* ctx, void* stream);

/* (No counterpart in the paper: an integration convenience.)
 * kvc_prefill_chunk for callers that have no way to obtain scratch memory: code running where
 * cudaMalloc is off limits -- inside a memory pool that owns the whole device, in a plugin that
 * may only touch the buffers it is handed, or in a latency-critical loop where an allocation would
 * synchronise the device.  The caller passes only the tensors it already owns (q, k, v, the layer's
 * cache blob, out); the scratch that kvc_prefill_chunk takes as `workspace` (log-sum-exp, scores,
 * move lists, status word) lives in a fixed array of KVC_STATIC_WS_BYTES bytes compiled into the
 * library, which every GPU that loads the library holds until the process exits.
 *   - The configuration must need no more than KVC_STATIC_WS_BYTES of single-layer scratch
 *     (lse 4*Hq*max(max_chunk, B) + scores 4*Hkv*cap + move lists 8*Hkv*max_chunk + ~1.5 KB); otherwise
 *     the call returns KVC_EINVAL and kvc_last_error names both sizes.  Nothing is enqueued then.
 *   - The first call on a device looks up the device address of the array (once per device, with
 *     that device current); make that first call outside any stream capture.
 *   - The array is shared by every context and every call on the device and keeps what the last
 *     call left there; a call that passes its argument checks clears the status word before its
 *     kernels run, so kvc_status_static reports on the most recent accepted call only (read it
 *     before the next call if an earlier call's status matters).  Two calls whose GPU work
 *     overlaps (different streams, or different threads without ordering) race on it: keep all
 *     users of this entry point on one stream, or order them with events.
 *   - Calls cudaMalloc/cudaFree never, and returns KVC_ESTATE while kvc_profile_enable is on
 *     (profiling creates events).
 * Arguments and results are otherwise exactly those of kvc_prefill_chunk.  kvc_status_static reads
 * the status word of the current device's array after synchronising `stream`. */
#define KVC_STATIC_WS_BYTES (1u << 20)
int kvc_prefill_chunk_static(kvc_ctx* ctx, int layer, const void* q, const void* k, const void* v,
                             int n, long long pos0, void* cache, void* out, void* stream);
int kvc_status_static(kvc_ctx* ctx, void* stream);

/* Output of Alg. 1: the compressed cache of one layer, as borrowed pointers. */
int kvc_cache_view(const kvc_ctx* ctx, int layer, void* cache, kvc_view* view);

/* Pointers into the workspace for inspection after a call (DEVICE, borrowed):
 *   lse    [n][Hq] fp32   natural-log log-sum-exp of every row's scaled scores (Eq. 1 normaliser)
 *   score  [Hkv][cap] fp32 importance of entry j before compaction (Eq. 4), valid for j < tot - w
 * of the most recent call for layer slot `slot` (0 for single-layer calls, i for layer layer0+i of
 * a batched call). */
int kvc_workspace_view(const kvc_ctx* ctx, void* workspace, int slot, float** lse, float** score);

/* DEVICE pointer (borrowed) to the int32 [Hkv] array holding, for layer slot `slot`, how many
 * entries the most recent eviction moved per kv-head during compaction. */
int kvc_move_counts(const kvc_ctx* ctx, void* workspace, int slot, int** counts);

/* Orders `stream` after every compress kernel that KVC_FLAG_ASYNC_COMPRESS left on the context's own stream
 * (no host wait; a no-op when nothing is pending).  After it, work enqueued on `stream` sees the compacted
 * caches, and a stream capture that the calls were part of may end. */
int kvc_join(kvc_ctx* ctx, void* stream);

/* Joins as kvc_join does, synchronises `stream` and returns the device status word kept in the workspace: KVC_OK, or
 * KVC_ETIMEOUT if a bounded wait inside a kernel gave up (the kernel then left early; results of
 * that call are invalid but the context and the device stay usable). */
int kvc_status(kvc_ctx* ctx, void* workspace, void* stream);

/* (No counterpart in the paper: robustness of the implementation.)  Every wait inside the kernels (on a TMA
 * load, a tensor-core commit, another warp) is bounded; a wait that runs out makes its kernel drain and exit and
 * leaves KVC_ETIMEOUT in the status word.  kvc_set_wait_limit sets that bound for the context's later calls, in
 * clock cycles (default about 2e9, one second; accepted range [1024, 2^40], rounded down to a multiple of 1024).
 * kvc_selftest_wait_timeout enqueues a one-CTA kernel whose only wait has no producer, bounded by the smaller of
 * the context's limit and 2^21 cycles: afterwards kvc_status(workspace) returns KVC_ETIMEOUT, and the context, the
 * device and the workspace (after kvc_workspace_init) stay usable.  workspace: DEVICE. */
int kvc_set_wait_limit(kvc_ctx* ctx, long long cycles);
int kvc_selftest_wait_timeout(kvc_ctx* ctx, void* workspace, void* stream);

/* KV bytes after Eq. 2 (2 x layers x heads x dim_head x precision x sequence length):
 * logical uses sequence length B, physical uses cap (what the blobs really hold, pos excluded),
 * uncompressed uses seq_len. */
int kvc_kv_bytes(const kvc_ctx* ctx, long long seq_len, size_t* logical, size_t* physical,
                 size_t* uncompressed);

/* Per-kernel timing for measurement runs.  kvc_profile_enable(ctx, 1) makes every later call
 * bracket each of its kernels with a pair of CUDA events on the caller's stream (host objects, no
 * device memory).  kvc_profile_read synchronises those events and ADDS, per kernel index
 * (0 append, 1 attention, 2 score when it runs as a kernel of its own, 3 compress = select + compact,
 * with the score inside when it is fused, 4 unused), the elapsed milliseconds into ms[5] and
 * the number of launches into launches[5] (both HOST arrays), then forgets the events.
 * Profiling perturbs end-to-end timing; leave it off in timed regions. */
int kvc_profile_enable(kvc_ctx* ctx, int on);
int kvc_profile_read(kvc_ctx* ctx, double* ms, long long* launches);

/* Per-kernel timing without events, for launches of a few microseconds (an event pair costs as much and keeps
 * consecutive launches from overlapping).  After kvc_profile_device(ctx, records, capacity, stream) -- records:
 * DEVICE, capacity x 16 bytes, 16-byte aligned, cleared by the call on `stream` -- every kernel of the context's later
 * calls stamps the nanosecond global timer when a CTA begins its work (past the wait for the preceding kernel) and
 * when it ends, and the launch's record keeps the earliest begin and the latest end; launches beyond `capacity` are
 * not recorded.  records = NULL switches it off.  kvc_profile_device_read takes a HOST copy of the records (made by
 * the caller after synchronising) and ADDS, per kernel index as in kvc_profile_read, the durations in milliseconds
 * and the launch counts; *span_ms (may be NULL) receives the time from the first begin to the last end. */
int kvc_profile_device(kvc_ctx* ctx, void* records, long long capacity, void* stream);
int kvc_profile_device_read(kvc_ctx* ctx, const void* records_host, double* ms, long long* launches, double* span_ms);

/* Number of kernel launches the library has enqueued through this context so far. */
long long kvc_launch_count(const kvc_ctx* ctx);

/* Text of the most recent error of this context (never NULL; valid until the next call). */
const char* kvc_last_error(const kvc_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* KVC_H_ */
