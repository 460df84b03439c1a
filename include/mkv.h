/*
 * mkv.h -- C ABI of the MorphKV decode + update hot path for NVIDIA B200 (sm_100a).
 *
 * MorphKV ("Dialogue Without Limits: Constant-Sized KV Caches for Extended Responses in
 * LLMs", arXiv 2503.00979) keeps, for every layer and KV head, a cache of C selected
 * distant tokens plus the R most recent tokens.  One *unit* is a (layer, batch row, KV head)
 * triple serving G = n_q_heads / n_kv_heads grouped query heads; units share nothing
 * ("Handling Multiple Heads").  Each decode step does, per unit:
 *
 *   attend   Eq. 1: soft-max attention of the new query over the cached tokens and itself;
 *   score    Eq. 4-6 + Algorithm 1: every cached token outside the recent window gets
 *            F[k] = sum_r or max_r of S_r[k], S_r[k] = sum over the GQA group of the weight
 *            window token r assigned to k when r was generated;
 *   select   Algorithm 1 / Eq. 7: keep the C largest F (ties: the lower position is kept);
 *   update   Eq. 7 + the "lightweight KV cache extension" of the Implementation paragraph:
 *            the evicted slot receives the new token's K/V, and the new query with its
 *            soft-max statistics replaces the oldest row of the recent-query ring.
 *
 * Conventions
 *   - Every `const void*` / `void*` tensor argument is a DEVICE pointer unless the name of
 *     the function ends in `_host`.  Tensors are contiguous, row-major, in the context's
 *     dtype (bf16 or f32).  The library applies no positional encoding: q and k are used
 *     as given.
 *   - `stream` is a `cudaStream_t` passed as `void*` (NULL = the default stream).  Calls
 *     enqueue work on it and return without synchronising unless stated otherwise.
 *   - No call throws or aborts across this boundary.  Every call returns an `mkv_status`;
 *     `mkv_last_error` gives the text of the last failure of a context.
 *   - There is no CPU fallback: without a CUDA device every compute call returns MKV_CUDA.
 *   - Input buffers are borrowed until the enqueued work has completed.
 */
#ifndef MKV_H
#define MKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum mkv_status {
    MKV_OK = 0,
    MKV_INVALID_ARG = 1,    /* a parameter or pointer is out of range / NULL               */
    MKV_BAD_STATE = 2,      /* call order violated (e.g. decode before prefill)            */
    MKV_OOM = 3,            /* workspace too small or device allocation failed             */
    MKV_CUDA = 4,           /* a CUDA runtime call failed (text in mkv_last_error)         */
    MKV_UNSUPPORTED = 5,    /* valid request this build has no kernel for                  */
    MKV_DEVICE_TIMEOUT = 6  /* a bounded device-side wait gave up; state is undefined      */
} mkv_status;

typedef enum mkv_fusion { MKV_FUSION_SUM = 0, MKV_FUSION_MAX = 1 } mkv_fusion;   /* Eq. 5, Eq. 6 */
typedef enum mkv_dtype { MKV_DTYPE_BF16 = 0, MKV_DTYPE_F32 = 1 } mkv_dtype;
/* How a window row's attention weights enter the fused score (Eq. 4).  FROZEN: with the values they had when the
 * row's token was generated.  CURRENT: renormalised over the tokens that are
 * still cached when the scores are taken (a row never saw tokens newer than itself); not with evict_interval > 1. */
typedef enum mkv_norm { MKV_NORM_FROZEN = 0, MKV_NORM_CURRENT = 1 } mkv_norm;
/* where the window tokens' attention profiles come from when the fused scores are taken (Eq. 4-6):
 * RECOMPUTE (default): from the stored window queries and their frozen soft-max normalisers, inside the decode
 *   kernel (same numbers, no table);
 * STORED: from a table of the weights themselves, kept beside the KV cache as the paper's implementation keeps
 *   them (Implementation paragraph): R * (C + R) more floats per unit, read once per policy step.  Trades bytes
 *   for arithmetic; it pays for wide windows.  bf16 / head_dim 128 on the tensor-core kernel only, with per-step
 *   eviction and MKV_NORM_FROZEN; not with mkv_prefill_ragged. */
typedef enum mkv_profile { MKV_PROFILE_RECOMPUTE = 0, MKV_PROFILE_STORED = 1 } mkv_profile;
/* which decode kernel to use: AUTO picks the tensor-core kernel when the shape allows it (bf16, head_dim 128, a
 * window of at most 2048 ring rows R * G', G' the GQA ratio rounded up to a power of two; any window with
 * MKV_PROFILE_STORED), the CUDA-core kernel otherwise */
typedef enum mkv_kernel { MKV_KERNEL_AUTO = 0, MKV_KERNEL_SIMT = 1, MKV_KERNEL_TC = 2 } mkv_kernel;

typedef struct mkv_ctx mkv_ctx;

typedef struct mkv_params {
    int layers, batch, n_q_heads, n_kv_heads, head_dim;
    int C;                  /* distant tokens retained per unit (Eq. 3)                    */
    int R;                  /* recent window (H1)                                           */
    mkv_fusion fusion;
    mkv_dtype dtype;
    int evict_interval;     /* T: run the policy every T-th decode step only (coarse-grained
                               eviction appendix); 0 or 1 = every step.  With T > 1 the cache
                               grows by one token per step and every T-th step keeps the top C
                               older tokens again (a second, small launch compacts the slots);
                               evicted_pos is then always -1.  At most 64.               */
    mkv_kernel kernel;
    int splits;             /* CTAs cooperating on one unit's cache; 0 = choose            */
    void *workspace;        /* device memory owned by the caller, 256-byte aligned, or NULL
                               to let the library allocate it with cudaMalloc              */
    size_t workspace_bytes;
    mkv_norm norm_mode;     /* MKV_NORM_FROZEN (default) or MKV_NORM_CURRENT                                 */
    int full_layers;        /* layer-aware variant (the appendix on selective layer retention): MorphKV is
                               switched off for the first full_layers layers, which keep every token; the
                               other layers run MorphKV as usual.  0 = none.                           */
    int max_tokens;         /* with full_layers > 0: the cache of those layers holds this many tokens (prompt
                               plus generated; > R).  While the sequence stays within it nothing is evicted
                               there; beyond it those layers fall back to MorphKV with that capacity.    */
    mkv_profile profile_mode;
                            /* MKV_PROFILE_RECOMPUTE (default) or MKV_PROFILE_STORED                         */
    unsigned long long wait_limit_cycles;
                            /* how long a device-side wait (on a copy, on the tensor cores, on another
                               warp) may spin before the kernel gives up, in GPU clock ticks; 0 = the
                               default of about two seconds.  A wait that runs out makes the kernel
                               return early and mkv_sync report MKV_DEVICE_TIMEOUT.  Only tests have a
                               reason to lower it.                                                   */
} mkv_params;

/* What one layer of the cache looks like.  Slot order inside a unit is unspecified: the
 * retained set of unit (b, h) is { pos[b][h][i] : i < count }. */
typedef struct mkv_view {
    void *K, *V;            /* [batch][n_kv_heads][capacity][head_dim], context dtype      */
    int32_t *pos;           /* [batch][n_kv_heads][capacity] absolute position, -1 = free  */
    float *F;               /* [batch][n_kv_heads][capacity] fused score of each slot at the
                               last selection (-1 for slots inside the recent window)      */
    int32_t *evicted_pos;   /* [batch][n_kv_heads] position evicted by the last step, -1 = none */
    void *ring_q;           /* [batch][n_kv_heads][R][group_stride][head_dim] recent queries; the
                               query of position p sits in ring row p % R                  */
    float *ring_c;          /* [batch][n_kv_heads][R][group_stride] log2-domain soft-max normaliser of a
                               ring row: weight(k) = exp2(q.k * log2(e)/sqrt(d) - ring_c);
                               +inf marks an empty row                                     */
    int32_t count;          /* tokens cached per unit of this layer (the same for every unit of it) */
    int32_t capacity;       /* slots per unit: C + R, plus evict_interval if that is > 1; max_tokens
                               for a layer that keeps every token                          */
    int64_t next_pos;       /* absolute position of the next token to decode               */
    int32_t group_stride;   /* heads per ring slot as laid out in ring_q / ring_c: G, or G rounded up
                               to a power of two (padding heads: zero query, ring_c = +inf) */
} mkv_view;

/* Fills *p with defaults: bf16, every-step eviction, automatic kernel and split choice,
 * library-owned workspace.  The caller then sets the shape fields. */
void mkv_default_params(mkv_params *p);

/* Bytes of device workspace a context with these parameters needs (0 if they are invalid). */
size_t mkv_workspace_bytes(const mkv_params *p);

/* Problem statement of the paper (Eq. 2-3): a cache of C + R entries per KV head.
 * bf16, every-step eviction, library-owned workspace.  Validates: all sizes >= 1,
 * n_q_heads % n_kv_heads == 0 with a group of at most 16, head_dim in {64, 128}.
 * No kernel is launched. */
mkv_status mkv_create(mkv_ctx **out, int layers, int batch, int n_q_heads, int n_kv_heads,
                      int head_dim, int C, int R, mkv_fusion fusion);

/* Same with every option spelled out.  If p->workspace is non-NULL the context lives in
 * that caller-owned memory (at least mkv_workspace_bytes(p) bytes) and never allocates
 * device memory for its state. */
mkv_status mkv_create_ex(mkv_ctx **out, const mkv_params *p);

/* Releases the context, the prompt-phase scratch it holds, and its workspace if the library
 * allocated it.  NULL is allowed. */
void mkv_destroy(mkv_ctx *ctx);

/* Prompt phase (the paper gives no procedure; this applies Algorithm 1 once with the whole
 * prompt as G_i): k, v [layers][batch][n_kv_heads][prompt_len][head_dim]; q_window
 * [layers][batch][n_q_heads][min(R, prompt_len)][head_dim] = the queries of the last prompt
 * positions, oldest first.  If prompt_len <= C + R everything is kept; otherwise the window
 * rows are scored causally over all prompt keys and the top C older tokens are kept.
 * Allocates device scratch on its first call (up to 1 GiB, for the logits of the window rows);
 * the context keeps it until mkv_destroy.  Synchronises the stream before returning. */
mkv_status mkv_prefill(mkv_ctx *ctx, const void *k, const void *v, const void *q_window,
                       int prompt_len, void *stream);

/* Forgets the sequence a context holds, so that mkv_prefill can load the next one into the same context (and the
 * same workspace and scratch).  Work already enqueued for the old sequence must have completed.  The paper has no
 * counterpart: this is context life-cycle. */
mkv_status mkv_reset(mkv_ctx *ctx);

/* mkv_prefill for callers that must not allocate (the paper has no counterpart: this is an
 * integration aid, not part of the method).  Some hosts of this library cannot let it call
 * cudaMalloc: a serving engine that has already handed all of HBM to its own pool, where a
 * further allocation fails or fragments; and latency-critical threads, for which the
 * device-wide synchronisation inside cudaMalloc/cudaFree stalls every other stream.  Give
 * the context a caller-owned workspace (mkv_create_ex) and use this call instead of
 * mkv_prefill: same arguments, same result, but the temporary table of window-row logits
 * lives in a fixed 16 MiB device array that is part of the library image (every GPU that
 * loads the library holds those 16 MiB until the process exits).
 *   - Limit: (min(R, prompt_len) * G + 1) * prompt_len <= 4 Mi floats for one unit;
 *     beyond that it returns MKV_UNSUPPORTED with an explanatory mkv_last_error and does
 *     nothing.  Units are pushed through the array a few at a time.
 *   - It calls no cudaMalloc, cudaFree or other allocating routine.
 *   - The first call on each device looks up the array's device address (once per device,
 *     with that device current); make that first call outside any stream capture.
 *   - All contexts and calls share the one array.  Nothing in it has to start at zero (every
 *     element is written before it is read within a call), but two calls whose kernels
 *     overlap on the GPU (different streams or threads) race on it: serialise them.
 * Synchronises the stream before returning, like mkv_prefill. */
mkv_status mkv_prefill_static(mkv_ctx *ctx, const void *k, const void *v, const void *q_window,
                              int prompt_len, void *stream);

/* Prompt phase of a batch whose rows have prompts of different lengths (the paper's runs use one length per
 * batch; a serving batch does not).  Tensors are padded to padded_len tokens: k, v
 * [layers][batch][n_kv_heads][padded_len][head_dim], of which row b's first prompt_len[b] tokens are read;
 * q_window [layers][batch][n_q_heads][min(R, padded_len)][head_dim], of which row b's first
 * min(R, prompt_len[b]) entries are the queries of its last prompt positions, oldest first.  prompt_len is a HOST
 * array of `batch` lengths, each in [1, padded_len].  Every row ends up exactly as mkv_prefill with its own length
 * would leave it (Algorithm 1 once over the row's prompt), and every later decode step appends one token to every
 * row: row b's token of step s has position prompt_len[b] + s, its window, eviction decisions and cache fill are
 * its own.  mkv_view.count is then the largest fill among the rows and mkv_view.next_pos the longest row's
 * position; mkv_row_state reports each row.  Rows are processed one by one with the CUDA-core scoring kernels
 * (set-up speed, not tuned).  Not available (MKV_UNSUPPORTED) together with evict_interval > 1 or with a window
 * of more than 256 ring rows on the tensor-core kernel.  Synchronises the stream before returning. */
mkv_status mkv_prefill_ragged(mkv_ctx *ctx, const void *k, const void *v, const void *q_window,
                              const int32_t *prompt_len, int padded_len, void *stream);

/* Cached tokens (count[b]) and position of the next token (next_pos[b]) of every batch row as `layer` holds them
 * now; HOST arrays of `batch` entries, either may be NULL.  Reads the host mirror only (call mkv_sync first if
 * steps were replayed from a CUDA graph).  All rows are equal unless the context was loaded by mkv_prefill_ragged. */
mkv_status mkv_row_state(mkv_ctx *ctx, int layer, int32_t *count, int64_t *next_pos);

/* One decode step for every unit (Eq. 1, Eq. 4-7, Algorithm 1): q, out
 * [layers][batch][n_q_heads][head_dim]; k_new, v_new [layers][batch][n_kv_heads][head_dim].
 * Asynchronous; launches a fixed kernel sequence with no host-side dependence on the step
 * index, so a sequence of calls can be recorded into a CUDA graph. */
mkv_status mkv_decode_step(mkv_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                           void *out, void *stream);

/* One layer of a decode step, for a model that runs its layers one after the other (the paper's implementation
 * hooks MorphKV into each layer's attention call; "Implementation" paragraph): q, out
 * [batch][n_q_heads][head_dim]; k_new, v_new [batch][n_kv_heads][head_dim] of layer `layer`.  The layers of a step
 * must be called in order 0, 1, ..., layers - 1 (MKV_BAD_STATE otherwise); the step is complete after the last one.
 * The results equal those of mkv_decode_step on the stacked tensors; a step may not mix the two calls.
 * Asynchronous on `stream`. */
mkv_status mkv_decode_step_layer(mkv_ctx *ctx, int layer, const void *q, const void *k_new,
                                 const void *v_new, void *out, void *stream);

/* n_steps consecutive decode steps; every tensor has a leading [n_steps] dimension. */
mkv_status mkv_decode_steps(mkv_ctx *ctx, const void *q, const void *k_new, const void *v_new,
                            void *out, int n_steps, void *stream);

/* One decode step with HOST buffers, in stream order on `stream`; does not synchronise.  If all four
 * buffers are pinned (page-locked, hence mapped into the device's address space) and the context runs the
 * tensor-core kernel, the kernel reads q, k_new, v_new and writes `out` directly in host memory; otherwise
 * q, k_new, v_new are copied to the device, the step runs, and `out` is copied back.  Either way the
 * inputs must stay unchanged, and `out` is complete, once the work enqueued on `stream` has finished. */
mkv_status mkv_decode_step_host(mkv_ctx *ctx, const void *q_host, const void *k_new_host,
                                const void *v_new_host, void *out_host, void *stream);

/* Device pointers into one layer of the cache.  Valid until the context is destroyed;
 * contents change with every decode step.  Reading them needs a stream synchronisation. */
mkv_status mkv_cache_view(mkv_ctx *ctx, int layer, mkv_view *view);

/* Waits for `stream` and reports device-side errors (MKV_DEVICE_TIMEOUT) recorded so far. */
mkv_status mkv_sync(mkv_ctx *ctx, void *stream);

/* Text of the last failure on this context ("" if none).  Never NULL. */
const char *mkv_last_error(const mkv_ctx *ctx);

/* Counters for reporting: kernels launched by this context so far, and the name of the
 * decode kernel in use ("simt" or "tc"). */
uint64_t mkv_launch_count(const mkv_ctx *ctx);
const char *mkv_kernel_name(const mkv_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* MKV_H */
