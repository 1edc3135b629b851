/*
 * d2o.h -- C ABI of the B200 (sm_100a) implementation of the D2O KV-cache compression
 * hot path (Dynamic Discriminative Operations, arXiv 2406.13035).
 *
 * The calls follow the paper's own statement of the problem:
 *   (1) after prompt encoding, from every layer's prompt queries and keys, the attention
 *       density F_v^l (Eq. 4) and the per-layer cache size S_l (Eq. 5, Appendix A.2);
 *   (2) per layer, token eviction (Eq. 6-8) and dynamic token merging (Eq. 9-12) of the
 *       prompt cache into a cache of S_l tokens;
 *   (3) per generated token, attention over the compressed cache (Eq. 2-3), score
 *       accumulation (Eq. 6), eviction of one token, and its merge-or-discard under the
 *       EMA threshold (Eq. 9-12).
 *
 * Conventions
 *   - Every pointer is marked HOST or DEVICE.  Device tensors are contiguous, row-major,
 *     16-byte aligned, in the element type `dtype` of the config unless a C type is given.
 *   - The library never allocates or frees device memory.  The caller owns `state` (lives
 *     as long as the context) and `scratch` (only used while a call's work is in flight)
 *     and sizes them with d2o_workspace_size().  Inputs are borrowed until the
 *     stream-ordered work of the call has finished and are never written.
 *   - All device work is enqueued on the given stream (a cudaStream_t passed as void*).
 *     Calls return without synchronising, except d2o_layer_budgets and the *_host
 *     variants, which say so.
 *   - Every call returns a d2o_status.  Invalid arguments are rejected before anything is
 *     launched.  Device-side anomalies (a wait that ran out, an empty candidate set) set
 *     an error word inside `state`, reported by d2o_get_stats(); nothing aborts or traps.
 *   - A context is not thread-safe; distinct contexts are independent.
 */
#ifndef D2O_H_
#define D2O_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  D2O_OK = 0,
  D2O_ERR_INVALID_ARG = 1,
  D2O_ERR_UNSUPPORTED = 2,
  D2O_ERR_WORKSPACE = 3,   /* state or scratch too small / misaligned */
  D2O_ERR_STATE = 4,       /* call out of order (e.g. compress before budgets) */
  D2O_ERR_CUDA = 5,        /* a CUDA runtime call failed; see d2o_last_cuda_error() */
  D2O_ERR_TIMEOUT = 6,
  D2O_ERR_TOO_LARGE = 7    /* problem exceeds the fixed capacity of an allocation-free entry point */
} d2o_status;

typedef enum { D2O_F32 = 0, D2O_F16 = 1, D2O_BF16 = 2 } d2o_dtype;

/* Hyper-parameters and shapes.  Paper symbols in brackets. */
typedef struct {
  int32_t n_layers;        /* [L]                                                          */
  int32_t batch;           /* independent sequences; budgets, tau and caches are per sequence */
  int32_t n_q_heads;       /* query heads per layer                                         */
  int32_t n_kv_heads;      /* KV heads per layer; n_q_heads % n_kv_heads == 0               */
  int32_t d_head;          /* 64 or 128; softmax scale is 1/sqrt(d_head)                    */
  int32_t dtype;           /* d2o_dtype of Q/K/V, the cache and the outputs                 */
  int32_t prompt_len;      /* [L_prompt] = [S] of Eq. 5                                     */
  int32_t max_new_tokens;  /* upper bound on decode steps                                   */
  float   rho;             /* [rho] global cache ratio; sum_l S_l = round(rho*L*L_prompt)   */
  int32_t n_sink;          /* [T] attention-sink tokens always kept                         */
  int32_t window;          /* [M] recent window; <= 0: derive per layer from nm_ratio       */
  float   nm_ratio;        /* [N:M], 3.0 in the paper (Section 5.1)                         */
  float   beta;            /* [beta] weight of the current Max(U_t) in Eq. 10               */
  float   tau_override;    /* NaN: Eq. 10; +inf: pure eviction; -inf: merge everything      */
  float   density_temp;    /* gamma in exp(-F/gamma); 1.0 is Eq. 5 as printed               */
  int32_t min_budget;      /* lower clamp of S_l (>= n_sink + 1)                            */
  int32_t max_budget;      /* upper clamp of S_l; <= 0 means L_prompt                       */
  int32_t head_reduce;     /* layer weight w_l from the per-head densities: 0: sum_h exp(-F_lh/gamma)
                            * (Appendix A.5); 1: exp(-mean_h F_lh/gamma); reciprocal-of-variance allocation of
                            * the ablation (Section 5.4, setting 2): 2: sum_h 1/F_lh; 3: 1/mean_h F_lh          */
  int32_t budget_rule;     /* 0: one size per layer, Eq. 5 with the weights of head_reduce;
                            * 1: one size per (layer, KV head), S_l^h = alpha_l^h * S_total of Appendix A.5, the
                            *    weight of a KV head being the sum of exp(-F/gamma) over its query heads and
                            *    S_total = round(rho * L * Hkv * L_prompt) (head_reduce is ignored);
                            * 2: "exponential decay allocation" of the ablation (Section 5.4, setting 3):
                            *    S_l = round(mean_h exp(-F_lh/gamma) * L_prompt), clamped; the total is not fixed,
                            *    rho is ignored and the cache pool is sized for n_layers * max_budget rows    */
  int32_t sim_feature;     /* rows the similarity of Eq. 9 is computed on: 0: keys (the method); 1: values (the
                            * ablation's "Feature choice" row V)                                                  */
  int32_t merge_policy;    /* 0: similarity-weighted merge (Eq. 11-12); 1: average merge (ablation "Merge policy"):
                            * a kept token and the tokens merged into it weigh the same                           */
} d2o_config;

typedef struct d2o_ctx d2o_ctx;

/* Device pointers into `state` for inspection / checkpointing.  Per-layer fields refer to the
 * layer passed to d2o_get_view().  The cache rows of slice (b, layer, h) are
 * [row_off[b, layer, h], ... + len).  With the per-layer budget rules all KV heads of a layer have the
 * same size.  All DEVICE. */
typedef struct {
  const float*   colsum;     /* [B, Hq, P]   column sums of the prompt attention (Eq. 4)      */
  const double*  density;    /* [B, L, Hq]   F_v per sequence, layer, query head (all layers) */
  const int32_t* budgets;    /* [B, L, Hkv]  cache size of every slice (all layers)            */
  const int32_t* windows;    /* [B, L, Hkv]  recent window M of every slice (all layers)       */
  const int64_t* row_off;    /* [B, L, Hkv]  first cache row of every slice, a multiple of 8   */
  void*          k_cache;    /* base of the K pool, rows of d_head elements (all layers)      */
  void*          v_cache;    /* base of the V pool                                             */
  int32_t*       pos;        /* [rows]       original position of each cache row (pool-wide)  */
  float*         score;      /* [rows]       accumulated attention score (Eq. 6)              */
  float*         rnorm;      /* [rows]       1/|k| of the stored key (0 for a zero key)       */
  int32_t*       len;        /* [L, B, Hkv]  tokens currently held (all layers)               */
  float*         tau;        /* [L, B, Hkv]  EMA threshold (Eq. 10) (all layers)              */
  const int32_t* evict_idx;  /* [B, Hkv, P]  scratch: evicted prompt positions of the last compressed layer */
  const float*   evict_mx;   /* [B, Hkv, P]  scratch: Max(U[i,:])                              */
  const int32_t* evict_nn;   /* [B, Hkv, P]  scratch: Argmax slot (relative to the slice)      */
  int64_t        pool_rows;  /* total cache rows in the pool                                   */
} d2o_view;

typedef struct {
  uint64_t decode_steps;     /* slices x steps processed                                       */
  uint64_t evictions;        /* tokens evicted during decode                                   */
  uint64_t merges;           /* ... of which merged (Max(U) >= tau_t)                          */
  uint64_t discards;         /* ... of which discarded                                         */
  uint64_t prefill_evicted;  /* tokens evicted at prompt stage                                 */
  uint64_t prefill_merged;   /* ... of which merged                                            */
  uint32_t error_word;       /* 0 = none; else first device-side anomaly (d2o_status)         */
  uint32_t error_detail;
  uint64_t decode_launches;  /* decode kernels launched so far (a step over all layers may take two)  */
  uint64_t guess_misses;     /* evictions whose victim was not among the rows guessed before the step (the keys
                              * of that slice were then read a second time)                                   */
} d2o_stats;

const char* d2o_status_string(d2o_status s);
/* Text of the last CUDA runtime error seen by this thread's calls (HOST string). */
const char* d2o_last_cuda_error(void);

/* Sizes in bytes of the caller-owned DEVICE buffers for this config. */
d2o_status d2o_workspace_size(const d2o_config* cfg, size_t* state_bytes, size_t* scratch_bytes);

/* Creates a context over caller-owned DEVICE buffers (256-byte aligned).  Zeroes the
 * bookkeeping part of `state` on `stream`.  The host object is freed by d2o_destroy(). */
d2o_status d2o_create(const d2o_config* cfg, void* state, size_t state_bytes,
                      void* scratch, size_t scratch_bytes, void* stream, d2o_ctx** out);
void d2o_destroy(d2o_ctx* ctx);

/* Ragged batches: lens HOST int32 [B], the prompt length of every sequence (1 .. prompt_len).  The prompt
 * tensors keep their layout for prompt_len positions per sequence; the positions beyond a sequence's length are
 * padding and are never used.  Every sequence gets Eq. 4-5 over its own prompt (its own S_l with
 * sum_l S_l = round(rho * L * its length)), and its generated tokens continue at its own length.  Call before
 * the first d2o_layer_stats of a prompt; returns D2O_ERR_STATE afterwards, D2O_ERR_INVALID_ARG if a length
 * does not satisfy the conditions d2o_create checks for prompt_len.  Synchronises `stream`. */
d2o_status d2o_set_prompt_lens(d2o_ctx* ctx, const int32_t* lens, void* stream);

/* (1) Eq. 4 for one layer.  Q DEVICE [B, Hq, P, d], K DEVICE [B, Hkv, P, d].
 * Computes s = column sums of the causal prompt attention Softmax(Q K^T / sqrt(d)) per query
 * head and F_v = Var(s).  `lse` (DEVICE float [B, Hq, P], natural-log row normalisers of that
 * attention) may be NULL, in which case it is computed here. */
d2o_status d2o_layer_stats(d2o_ctx* ctx, int32_t layer, const void* Q, const void* K,
                           const float* lse, void* stream);

/* The same for layers [l0, l1) in one call (Eq. 4 acts per layer; a caller that holds several
 * layers' Q and K can hand them over together).  Q, K: HOST arrays of l1-l0 DEVICE pointers;
 * lse: NULL, or a HOST array of l1-l0 DEVICE pointers (entries may be NULL).  Two layers are
 * worked on side by side on streams of the library's own (as d2o_prefill_compress_layers does,
 * same fork / join on `stream`, same first-call creation of streams and events), each with its
 * own row-normaliser scratch, so that one layer's last CTAs share the GPU with the next layer's
 * first.  Results are those of l1-l0 calls of d2o_layer_stats, bit for bit. */
d2o_status d2o_layer_stats_layers(d2o_ctx* ctx, int32_t l0, int32_t l1, const void* const* Q,
                                  const void* const* K, const float* const* lse, void* stream);

/* (1') Eq. 5 / Appendix A.2 once every layer has been fed: the cache size of every slice.
 * Writes budgets_host (HOST int32 [B, L, Hkv], may be NULL).  Synchronises `stream`: the host
 * needs the sizes to lay out the cache and to plan the decode launches.  */
d2o_status d2o_layer_budgets(d2o_ctx* ctx, int32_t* budgets_host, void* stream);

/* Eq. 5 as a pure function: density DEVICE double [B, L, H] -> budgets DEVICE int32 [B, L, Hkv]
 * (and, if not NULL, windows DEVICE int32 [B, L, Hkv], row offsets DEVICE int64 [B, L, Hkv]).
 * budget_rule and head_reduce as in d2o_config.  No context; asynchronous. */
d2o_status d2o_budgets_from_density(const double* density, int32_t batch, int32_t n_layers,
                                    int32_t n_heads, int32_t n_kv_heads, int32_t prompt_len,
                                    float rho, int32_t min_budget, int32_t max_budget,
                                    float density_temp, int32_t head_reduce, int32_t budget_rule,
                                    int32_t n_sink, int32_t window, float nm_ratio, int32_t* budgets,
                                    int32_t* windows, int64_t* row_off, int32_t* status_word,
                                    void* stream);

/* (2) Eq. 6-12 for one layer's prompt cache.  K, V DEVICE [B, Hkv, P, d].
 * Keeps T sinks, the Top-N accumulated scores and the last M tokens, matches every evicted
 * key to its most similar kept key, sets tau_0, merges the tokens at or above it, and
 * leaves the compressed cache of the layer in `state`. */
d2o_status d2o_prefill_compress(d2o_ctx* ctx, int32_t layer, const void* K, const void* V,
                                void* stream);

/* The same for layers [l0, l1) in one call (Eq. 5 needs every layer's density before any layer
 * can be compressed, so at this point the caller holds all layers' K and V anyway).
 * K, V: HOST arrays of l1-l0 DEVICE pointers, each [B, Hkv, P, d].  The layers are independent
 * (Eq. 6-12 act per layer and head); the library works on up to four of them side by side, each
 * on a stream of its own with its own part of `scratch`, so that the per-layer kernels of a small
 * batch (B * Hkv CTAs each) fill the GPU together.  The internal streams start behind everything
 * `stream` holds at the call, and `stream` continues behind all of them; the first call creates
 * them (streams and events only, no device memory).  Results are those of l1-l0 calls of
 * d2o_prefill_compress, bit for bit; the inspection arrays of d2o_get_view (evicted positions,
 * Max(U), Argmax) then show one of the layers, not necessarily the last. */
d2o_status d2o_prefill_compress_layers(d2o_ctx* ctx, int32_t l0, int32_t l1, const void* const* K,
                                       const void* const* V, void* stream);

/* (3) One generated token for layers [l0, l1).  DEVICE tensors:
 * q [l1-l0, B, Hq, d], k and v [l1-l0, B, Hkv, d], out [l1-l0, B, Hq, d].
 * Every call advances the token position of those layers by one; all layers must be
 * stepped equally often. */
d2o_status d2o_decode_step(d2o_ctx* ctx, int32_t l0, int32_t l1, const void* q, const void* k,
                           const void* v, void* out, void* stream);

/* n_steps consecutive generated tokens for layers [l0, l1) whose inputs are all resident
 * (Section 4.2, one eviction per generated token; Eq. 2-3, 6-12 per step as in
 * d2o_decode_step).  DEVICE tensors: q [n_steps, l1-l0, B, Hq, d], k and v
 * [n_steps, l1-l0, B, Hkv, d], out [n_steps, l1-l0, B, Hq, d]; every entry must be complete
 * (stream-ordered) before the call, so a step's inputs cannot depend on an earlier step's
 * output.  The results are those of n_steps calls of d2o_decode_step, bit for bit.  What
 * differs is the launch: from the second step on a step's grids are launched with
 * programmatic stream serialisation and start while the previous step's last CTAs still
 * run; every CTA then waits (with the limit of every other wait in the kernel) for a
 * per-slice step counter that the slice's previous CTA publishes as its last act, not for
 * the whole previous grid.  Whatever follows on `stream` is ordered behind all n_steps.
 * Errors: as d2o_decode_step; D2O_ERR_STATE if fewer than n_steps tokens remain of
 * max_new_tokens (nothing is launched then). */
d2o_status d2o_decode_steps(d2o_ctx* ctx, int32_t l0, int32_t l1, int32_t n_steps, const void* q,
                            const void* k, const void* v, void* out, void* stream);

/* Same with HOST buffers (pinned memory recommended): copies q, k, v to the device, runs the
 * step, copies `out` back and synchronises `stream`.  If q, k and v lie back to back in host
 * memory in this order they travel in one transfer. */
d2o_status d2o_decode_step_host(d2o_ctx* ctx, int32_t l0, int32_t l1, const void* q_host,
                                const void* k_host, const void* v_host, void* out_host,
                                void* stream);

/* n_steps consecutive tokens with HOST buffers (pinned memory, or the copies do not overlap
 * anything): q_host [n_steps, l1-l0, B, Hq, d], k_host and v_host [n_steps, l1-l0, B, Hkv, d],
 * out_host [n_steps, l1-l0, B, Hq, d].  Per step the same work as d2o_decode_step_host, but
 * pipelined over three streams (the caller's for the kernels, two of the library's own for the
 * copies, created with the first call; no device memory), in blocks of four steps: while a
 * block computes, the inputs of the next block travel to the device and the outputs of the
 * previous one travel back, through two blocks of staging sets in `scratch`; the steps of a
 * block are chained as in d2o_decode_steps.  As with d2o_decode_steps a step's inputs cannot depend on an earlier
 * step's output.  Returns after everything, the last copy back included, has completed. */
d2o_status d2o_decode_steps_host(d2o_ctx* ctx, int32_t l0, int32_t l1, int32_t n_steps,
                                 const void* q_host, const void* k_host, const void* v_host,
                                 void* out_host, void* stream);

/* Uncompressed decode attention (Eq. 2-3), the comparison kernel: appends k, v at row `len`
 * of k_cache/v_cache DEVICE [n_slices, capacity, d] (n_slices = B*Hkv) and attends over
 * len+1 rows.  q, out DEVICE [n_slices, group, d]; k, v DEVICE [n_slices, d].
 * No context, no state; asynchronous. */
d2o_status d2o_full_decode_step(int32_t dtype, int32_t d_head, int32_t n_slices, int32_t group,
                                int32_t capacity, int32_t len, void* k_cache, void* v_cache,
                                const void* q, const void* k, const void* v, void* out,
                                void* stream);

/* Allocation-free variant of d2o_layer_stats (the paper has no counterpart: this entry point
 * exists for callers that cannot allocate device memory).
 *
 * Who needs it: code that runs where cudaMalloc is off limits, for example inside a serving
 * process whose memory pool has already claimed the whole device, in a plugin that is handed
 * tensors but no allocator, or between the steps of a latency-critical loop where an allocation
 * would synchronise the device.  d2o_layer_stats needs a scratch buffer for the softmax row
 * normalisers of the prompt attention; here that buffer is a fixed array of
 * D2O_STATIC_LSE_FLOATS floats (4 MiB) that is part of the library image, so every GPU that
 * loads the library carries it until the process exits.  No context, no workspace: the caller
 * passes the inputs and the outputs only.
 *
 *   Q DEVICE [B, Hq, P, d], K DEVICE [B, Hkv, P, d] in `dtype`;
 *   colsum DEVICE float [B, Hq, P] (out: column sums of the causal prompt attention, Eq. 4);
 *   density DEVICE double [B, Hq] (out: F_v = Var(colsum) per query head).
 *
 * It always runs the generic kernels (fp32 arithmetic on CUDA cores, any dtype, any prompt
 * length).  d2o_layer_stats runs the same kernels, and then returns bit-identical results, for
 * fp32 inputs, for a prompt length that is not a multiple of 4, or with stats_path = 1; for
 * 16-bit inputs it otherwise takes its tensor-core kernels, which are several times faster and
 * agree with this entry point to rounding (column sums within 2e-4 relative).
 *
 * Limit: batch * n_q_heads * prompt_len <= D2O_STATIC_LSE_FLOATS and batch * n_q_heads <= 65535,
 * else D2O_ERR_TOO_LARGE and nothing is launched.  The call neither allocates nor frees device
 * memory.
 * The first call on each device looks up the device address of the array (one runtime query,
 * made with that device current) and keeps it for the life of the process; make that first call
 * outside of any stream capture.  After cudaDeviceReset() the kept address is stale: a process
 * that resets a device must not call this entry point on it again.
 * All calls share the one array: it is fully rewritten by each call before it is read, so
 * nothing needs clearing, but two calls whose work overlaps on the GPU (different streams)
 * race on it.  Asynchronous on `stream` like the other calls. */
#define D2O_STATIC_LSE_FLOATS (1u << 20)
d2o_status d2o_layer_stats_static(int32_t dtype, int32_t d_head, int32_t batch, int32_t n_q_heads,
                                  int32_t n_kv_heads, int32_t prompt_len, const void* Q, const void* K,
                                  float* colsum, double* density, void* stream);

d2o_status d2o_get_view(d2o_ctx* ctx, int32_t layer, d2o_view* out);
/* Copies the counters to HOST memory; synchronises `stream`. */
d2o_status d2o_get_stats(d2o_ctx* ctx, d2o_stats* out_host, void* stream);

/* Knobs of the decode kernel for measurements: stages of its shared-memory ring (0 = automatic,
 * else 2..12, 16 KB each; a depth that does not fit in shared memory makes the next
 * d2o_decode_step return D2O_ERR_UNSUPPORTED) and whether its copies carry L2 eviction hints
 * (1 = yes, the default; 0 = no); similarity_path 0 = tensor-core kernel for fp16/bf16 keys at the
 * prompt stage (default), 1 = the FFMA kernel for every dtype; stats_path likewise for the column
 * sums of d2o_layer_stats; decode_warps = consumer warps per CTA of the decode kernel (0 = automatic,
 * 4 or 8 with one or two query heads per KV head, 8 or 16 with four or eight); decode_smem_rows =
 * rows of a slice whose logits the decode kernel keeps in shared memory, the rest going through an
 * L2-resident array of the scratch buffer (0 = automatic, else >= 8); decode_long_pairs = how many
 * of the (layer, sequence) pairs with the largest budgets a decode step over all layers runs in a
 * launch of their own with sixteen-warp CTAs, ahead of and overlapping the launch of the rest
 * (0 = automatic, negative = never, positive = that many). */
d2o_status d2o_set_tuning(d2o_ctx* ctx, int32_t decode_stages, int32_t decode_l2_hints,
                          int32_t similarity_path, int32_t stats_path, int32_t decode_warps,
                          int32_t decode_smem_rows, int32_t decode_long_pairs);

/* For failure-detection tests (Section 4.2's decode step has no counterpart; this exercises the library's own
 * promise that no device-side wait is unbounded).  wait_limit_us: how long the decode kernel waits for a stage
 * of cache rows before it gives up (0 = the default of one second).  producer_stop_stage: the kernel's copy
 * engine issues no copy from this stage of a slice on (-1 = never), so that the wait for it runs out.  A wait
 * that runs out sets the error word to D2O_ERR_TIMEOUT (see d2o_get_stats); the kernel returns, the slices
 * whose wait ran out during the key pass are left untouched, and every later decode step on this context does
 * nothing.  Nothing traps and the CUDA context stays usable. */
d2o_status d2o_set_fault_injection(d2o_ctx* ctx, int32_t wait_limit_us, int32_t producer_stop_stage);

#ifdef __cplusplus
}
#endif
#endif /* D2O_H_ */
