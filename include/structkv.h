/*
 * structkv.h -- C ABI of the B200 (sm_100a) StructKV prefill-time KV-compression hot path.
 *
 * The library scores the observation-window queries of one layer against all prompt keys,
 * accumulates the per-token in-degree across depth into the Global In-Degree Centrality,
 * produces the per-layer attention statistics that drive Dynamic Pivot Detection, selects
 * token budgets (top-k union window) and compacts K/V, hidden states and position ids.
 *
 * Conventions
 *   - Every pointer marked "device" is a CUDA device pointer owned by the caller; "host"
 *     pointers are ordinary host memory.  The library allocates no device memory: the
 *     caller passes one workspace at context creation (structkv_workspace_bytes()).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All
 *     calls enqueue work on it and return without synchronising, except structkv_pivot and
 *     structkv_poll_device_status, which synchronise that stream.
 *   - Every call returns a status; invalid arguments are rejected on the host before any
 *     launch.  There is no CPU fallback: an unsupported shape returns
 *     STRUCTKV_ERR_UNSUPPORTED.  Device-side waits are bounded; if one expires the kernel
 *     records STRUCTKV_ERR_TIMEOUT in a device status word read by
 *     structkv_poll_device_status().
 *   - A context serialises its calls through its workspace: calls on one context must be
 *     issued on one stream (or be ordered by the caller).  Distinct contexts are independent.
 *   - Results are deterministic: the same inputs give the same bits.
 *
 * Index conventions: N = n_keys prompt tokens, w = window (the last w positions are the
 * observation-window queries, row i sits at position t = N-w+i and attends to keys j <= t),
 * H query heads, H_kv KV heads, G = H / H_kv, head h reads KV head h / G, d = head_dim.
 */
#ifndef STRUCTKV_H_
#define STRUCTKV_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  STRUCTKV_OK = 0,
  STRUCTKV_ERR_INVALID_ARG = 1, /* null pointer, size out of range, misaligned pointer or stride */
  STRUCTKV_ERR_UNSUPPORTED = 2, /* shape or dtype outside the supported set */
  STRUCTKV_ERR_WORKSPACE = 3,   /* workspace missing or too small */
  STRUCTKV_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed */
  STRUCTKV_ERR_TIMEOUT = 5      /* a bounded device-side wait expired */
} structkv_status;

typedef enum { STRUCTKV_BF16 = 0, STRUCTKV_FP32 = 1 } structkv_dtype;

/* Flags of structkv_score_layer. */
#define STRUCTKV_FLAG_NO_HEAD_STATS 1u /* skip Eq. 5-6: metrics_out[1..2] are written as NaN */
#define STRUCTKV_FLAG_FORCE_SIMT 2u    /* use the CUDA-core scorer even where the tensor-core one applies */
/* The caller vouches that q_window and k are complete and visible to the device before the call
 * is enqueued: no kernel still in flight on `stream` writes them (they were written before an
 * earlier synchronisation, or on another stream joined through an event).  The first scorer
 * pass then starts reading them while the kernels enqueued before it (the previous layer's
 * column reduction) are still draining; results are identical.  Without the flag the pass
 * waits for everything enqueued before it, as any kernel on a stream does. */
#define STRUCTKV_FLAG_INPUTS_READY 4u

typedef struct {
  int n_q_heads;        /* H, a multiple of n_kv_heads */
  int n_kv_heads;       /* H_kv */
  int head_dim;         /* d: 64 or 128 */
  int window;           /* w: 1..256 */
  int max_seq;          /* largest n_keys any call will pass */
  structkv_dtype dtype; /* storage type of q_window and k */
} structkv_config;

typedef struct structkv_ctx structkv_ctx; /* opaque, host-side */

/* Library version (major*10000 + minor*100 + patch). */
int structkv_version(void);

/* Static, human-readable name of a status code. */
const char* structkv_status_string(structkv_status s);

/* Bytes of device workspace a context for `cfg` needs (0 if cfg is invalid). */
size_t structkv_workspace_bytes(const structkv_config* cfg);

/* Creates a context on the current CUDA device.  `workspace_dev` (device, 256-byte aligned,
 * at least structkv_workspace_bytes(cfg) bytes) stays owned by the caller and must outlive
 * the context.  The call zeroes the device status word on the default stream and synchronises.
 * Errors: INVALID_ARG (null pointers, bad config), UNSUPPORTED (head_dim, window),
 * WORKSPACE (too small / misaligned), CUDA. */
structkv_status structkv_create(structkv_ctx** ctx_out, const structkv_config* cfg,
                                void* workspace_dev, size_t workspace_bytes);

/* Frees the host-side context (never touches the workspace). NULL is allowed. */
void structkv_destroy(structkv_ctx* ctx);

/*
 * One layer of observation-window scoring.
 *
 * Paper: Section 3.2, Eq. 1 (window attention weights a_{t,j} = softmax over keys of
 * q_t.k_j * scale, causal), Eq. 2 (local saliency S_j = (1/w) sum over window rows and over
 * all query heads of a_{t,j}), Eq. 3 / Algorithm 1 line 6 (C <- lambda*C + S), and Section
 * 3.3, Eq. 4 (attention entropy, natural log, mean over heads and window rows), Eq. 5
 * (sparsity: mean over heads of the mass of the floor(0.1 N) largest entries of the
 * window-pooled per-head attention) and Eq. 6 (variance: mean over heads of the population
 * variance over keys of that pooled vector).
 *
 *   q_window      device, [H, w, d] contiguous, dtype of the config; positional encoding
 *                 already applied.  16-byte aligned.
 *   k             device, element (g, j, c) at k + g*k_stride_head + j*k_stride_token + c
 *                 (strides in elements; d contiguous).  Base 16-byte aligned, strides
 *                 multiples of 16 bytes.  Read-only; V is never read.
 *   n_keys        N, window <= N <= max_seq.
 *   scale         logit scale (1/sqrt(d), times any temperature the caller folds in).
 *   lambda        decay of Eq. 3; used only if c_inout != NULL.
 *   s_out         device, [N] fp32, required: S^(l).
 *   c_inout       device, [N] fp32 or NULL: updated in place, C <- lambda*C + S.
 *   head_cols_out device, [H, N] fp32 or NULL: pooled per-head attention
 *                 abar^(h)_j = (1/w) sum_i a_{i,j} (each row sums to 1).
 *   metrics_out   device, [3] fp32, required: {entropy, sparsity, variance}.
 *   flags         STRUCTKV_FLAG_*.
 *
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_score_layer(structkv_ctx* ctx, const void* q_window, const void* k,
                                     long long k_stride_head, long long k_stride_token, int n_keys,
                                     float scale, float lambda, float* s_out, float* c_inout,
                                     float* head_cols_out, float* metrics_out, unsigned flags,
                                     void* stream);

/*
 * One layer of observation-window scoring for a BATCH of prompts of different lengths
 * (Section 4.1, implementation details: batches whose prompts reach their pivots at different
 * layers are served with a padded addressing mask; every prompt is an independent problem with
 * its own length, statistics, pivot and index sets).  The prompts' keys are packed back to back
 * along the token axis; one launch per scorer pass covers all prompts, each prompt receiving a
 * share of the grid in proportion to its length.  Per prompt the results equal those of
 * structkv_score_layer on that prompt alone (same equations: Eq. 1, 2, 3, 4, 5, 6).
 *
 *   q_window      device, [batch, H, w, d] contiguous bf16.
 *   k             device, packed keys: element (g, t, c) at k + g*k_stride_head + t*k_stride_token + c,
 *                 prompt b owning tokens cu_seqlens[b] .. cu_seqlens[b+1]-1.
 *   cu_seqlens    HOST, [batch + 1] ints, cu_seqlens[0] = 0, every length in [w, max_seq].
 *   batch         1 .. 32.
 *   s_out         device, [total] fp32 (total = cu_seqlens[batch]): S^(l) of every prompt, packed.
 *   c_inout       device, [total] fp32 or NULL: C <- lambda*C + S, packed.
 *   head_cols_out device, [H, total] fp32 or NULL.
 *   metrics_out   device, [batch, 3] fp32: {entropy, sparsity, variance} of every prompt.
 *   flags         STRUCTKV_FLAG_NO_HEAD_STATS, STRUCTKV_FLAG_INPUTS_READY or 0.
 *   batch_workspace  device, 256-byte aligned, at least
 *                 structkv_batch_workspace_bytes(cfg, batch, total) bytes, caller-owned; calls that
 *                 share it must be ordered by the caller.
 * Served by the tensor-core scorer only (bf16, window 32 / 64 / 128): other configurations
 * return UNSUPPORTED.  Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.  Asynchronous on `stream`.
 */
size_t structkv_batch_workspace_bytes(const structkv_config* cfg, int max_batch, long long max_total_tokens);
structkv_status structkv_score_layer_batch(structkv_ctx* ctx, const void* q_window, const void* k,
                                           long long k_stride_head, long long k_stride_token,
                                           const int* cu_seqlens, int batch, float scale, float lambda,
                                           float* s_out, float* c_inout, float* head_cols_out,
                                           float* metrics_out, unsigned flags, void* batch_workspace,
                                           size_t batch_workspace_bytes, void* stream);

/*
 * Eq. 10 / Eq. 13 for a batch of prompts of different lengths: prompt b selects budgets[b] tokens
 * (window included) from its own scores scores[cu_seqlens[b] .. cu_seqlens[b+1]) and writes them,
 * as positions inside that prompt, ascending, to idx_out + b*idx_stride; the remaining entries of
 * the row are -1 (the padded addressing of a batch: padding is never a token).
 *   cu_seqlens, budgets   HOST arrays, [batch + 1] and [batch]; window <= budgets[b] <= length of b.
 *   idx_out               device, [batch, idx_stride] int32, idx_stride >= max budget.
 * Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_select_batch(structkv_ctx* ctx, const float* scores, const int* cu_seqlens,
                                      const int* budgets, int batch, int window, int* idx_out,
                                      long long idx_stride, void* stream);

/*
 * Algorithm 1 lines 3-6 (Eq. 1-4) for SEVERAL layers whose window queries and keys are all
 * resident (a prompt whose KV cache already exists, or a prefill that ran ahead of the scoring).
 * Per layer the results are the very bits structkv_score_layer gives with
 * STRUCTKV_FLAG_NO_HEAD_STATS: S^(l), the pooled per-head attention, the layer's entropy; C is
 * carried through all layers (C <- lambda*C + S^(l), l ascending).  What differs is the order of
 * the work: the first scorer pass of layer l+1 is enqueued between the two passes of layer l, and
 * the second pass of layer l waits for a completion counter of its own first pass instead of for
 * the kernel enqueued before it, so no SM idles while the slowest CTA of a pass finishes; the
 * sums over heads of all layers are taken by one launch at the end.
 *
 *   q_windows, ks  HOST arrays [n_layers] of device pointers, laid out as for structkv_score_layer
 *                 (one stride pair serves all layers); every tensor must be complete and visible
 *                 before the call is enqueued (as with STRUCTKV_FLAG_INPUTS_READY).
 *   scales        HOST array [n_layers].
 *   s_out         device, fp32: S^(l) at s_out + l*s_layer_stride, s_layer_stride >= n_keys.
 *   c_inout       device, [n_keys] fp32 or NULL.
 *   head_cols_out device, fp32, required: layer l's [H, n_keys] slab at
 *                 head_cols_out + l*head_cols_layer_stride (feed it to structkv_head_stats).
 *   metrics_out   device, [n_layers, 3] fp32: [l][0] = entropy, [l][1..2] = NaN.
 *   layers_workspace  device, 256-byte aligned, at least structkv_layers_workspace_bytes(cfg, n_layers)
 *                 bytes, caller-owned.
 * Shapes the tensor-core scorer does not take are scored layer after layer (same results).
 * Errors: INVALID_ARG, WORKSPACE, CUDA.  Asynchronous on `stream`.
 */
size_t structkv_layers_workspace_bytes(const structkv_config* cfg, int max_layers);
structkv_status structkv_score_layers(structkv_ctx* ctx, int n_layers, const void* const* q_windows,
                                      const void* const* ks, long long k_stride_head,
                                      long long k_stride_token, int n_keys, const float* scales, float lambda,
                                      float* s_out, long long s_layer_stride, float* c_inout,
                                      float* head_cols_out, long long head_cols_layer_stride,
                                      float* metrics_out, void* layers_workspace,
                                      size_t layers_workspace_bytes, void* stream);

/*
 * Eq. 5 and Eq. 6 (Section 3.3) for several layers at once, from the pooled per-head attention
 * that structkv_score_layer wrote to head_cols_out.  A caller that scores many layers passes
 * STRUCTKV_FLAG_NO_HEAD_STATS and a distinct head_cols_out slab per layer, then makes ONE call
 * here before the pivot: the per-head selections of all layers run side by side instead of as
 * a chain of short dependent launches after every layer.
 *
 *   head_cols     device, fp32: entry (l, h, j) at head_cols + l*layer_stride + h*col_stride + j,
 *                 each (l, h) vector non-negative and summing to 1 (Eq. 2's per-head pooling).
 *   n_layers      1 .. 128.
 *   n             N, the number of keys of every vector; col_stride >= n.
 *   metrics       device, [n_layers, 3] fp32: entries [l][1] (sparsity) and [l][2] (variance) are
 *                 written, [l][0] (entropy) is left untouched.
 * Results equal those of structkv_score_layer without the flag.  Uses the context's workspace
 * (calls on one context are ordered by the caller).  Errors: INVALID_ARG, CUDA.  Asynchronous.
 */
structkv_status structkv_head_stats(structkv_ctx* ctx, const float* head_cols, long long layer_stride,
                                    long long col_stride, int n_layers, int n, float* metrics,
                                    void* stream);

/*
 * structkv_score_layer without a context and without a caller workspace.  The paper has no
 * counterpart: this entry point exists for integration only.
 *
 * Some hosts of this library cannot allocate device memory at the point where they score a
 * layer: a serving engine that hands all free HBM to its paged KV-cache pool at start-up has
 * nothing left for cudaMalloc to give, and a step that runs inside a latency budget cannot
 * afford the device-wide synchronisation an allocation or a free implies.  For them the
 * scratch the scorer needs (per-segment row statistics, row log-sum-exp, pooled per-head
 * columns, the status word) lives in one array of STRUCTKV_STATIC_SCRATCH_BYTES that is part
 * of the library image: every GPU that loads the library holds those bytes until the process
 * exits, whether this function is called or not.  The call itself performs no cudaMalloc,
 * cudaFree or other allocating routine; inputs and outputs are still the caller's.
 *
 * Limit: the configuration must satisfy
 *     0 < structkv_workspace_bytes(cfg) <= STRUCTKV_STATIC_SCRATCH_BYTES
 * (a Llama-3-8B shape, 32 query heads, window 64, fits up to max_seq = 16384).  A larger
 * configuration is refused with STRUCTKV_ERR_WORKSPACE before anything is launched.
 *
 * Set-up: the first call on each device (with that device current) resolves the device
 * address of the array and looks up the tensor-map encoder; it synchronises nothing but
 * should happen before any stream capture begins.  Later calls on that device only enqueue.
 *
 * Sharing: all calls on one device use the same array, and it keeps whatever the previous
 * call left.  The function re-initialises on `stream` what has to start from zero, so calls
 * issued one after another on one stream are independent; two calls that can overlap on the
 * GPU (different streams without an ordering between them, or different host threads) race
 * on the scratch and give undefined results.  A device-side bounded wait that expires during
 * this call cannot be polled through this entry point; use a context for that.
 *
 * Arguments: `cfg` host pointer; everything else exactly as structkv_score_layer, with
 * cfg->max_seq >= n_keys.  Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.
 */
#define STRUCTKV_STATIC_SCRATCH_BYTES (8u << 20)
structkv_status structkv_score_layer_static(const structkv_config* cfg, const void* q_window,
                                            const void* k, long long k_stride_head,
                                            long long k_stride_token, int n_keys, float scale,
                                            float lambda, float* s_out, float* c_inout,
                                            float* head_cols_out, float* metrics_out,
                                            unsigned flags, void* stream);

/*
 * Dynamic Pivot Detection.  Paper: Section 3.3, Eq. 7 (first differences of each metric over
 * layers l = 1..L-1, min-max normalised to [0,1]; a metric with zero range contributes 0),
 * Eq. 8 (T_l = w1*grad(-entropy) + w2*grad(sparsity) + w3*grad(variance)), Eq. 9 with
 * Algorithm 1 line 8: the pivot is the layer l in [1, L-1] with the largest T_l (first maximum
 * wins), capped at l_limit.  NaN sparsity/variance columns (head statistics disabled) count
 * as constant.  Evaluated in double precision on the host.
 *
 *   metrics_dev device, [n_layers, 3] fp32 rows as written by structkv_score_layer.
 *   weights     host, {w1, w2, w3}.
 *   l_limit     cap on the pivot, or -1 for none.
 *   pivot_out   host, receives L* (0 if n_layers < 2).
 *   t_out       host, [n_layers] or NULL: receives T_l (T_0 = 0).
 *
 * Synchronises `stream`.  Errors: INVALID_ARG, CUDA.
 */
structkv_status structkv_pivot(structkv_ctx* ctx, const float* metrics_dev, int n_layers,
                               const float* weights, int l_limit, int* pivot_out, float* t_out,
                               void* stream);

/*
 * Global In-Degree Centrality at a known pivot.  Paper: Eq. 3,
 * c_out[j] = sum_{l=0..pivot} lambda^(pivot-l) * s_hist[l*row_stride + j], evaluated as the
 * recursion of Algorithm 1 line 6.
 *
 *   s_hist device, fp32 rows of length >= n, row_stride in elements;  c_out device, [n] fp32.
 * Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_accumulate(structkv_ctx* ctx, const float* s_hist, long long row_stride,
                                    int pivot, int n, float lambda, float* c_out, void* stream);

/*
 * Budgeted token selection.  Paper: Eq. 10 (I_struct = top-k(C) union I_win) and Eq. 13
 * (I_KV = top-k(S^(l)) union I_win), Algorithm 1 lines 10 and 16.  For each of `batch` score
 * vectors: the (budget - window) highest-scoring tokens of the prefix [0, n - window), ties
 * to the lower index, written in ascending position order, followed by the window positions
 * n-window .. n-1.  Scores must not be NaN.
 *
 *   scores  device, fp32, vector b starts at scores + b*row_stride (elements).
 *   idx_out device, [batch, budget] int32.
 *   window <= budget <= n.
 * Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_select(structkv_ctx* ctx, const float* scores, long long row_stride,
                                int batch, int n, int budget, int window, int* idx_out,
                                void* stream);

/*
 * Row gather / compaction.  Paper: Algorithm 1 line 17 (cache K, V at I_KV), line 13 and
 * Eq. 11-12 (hidden states and position ids at I_struct).  For every slab s and output row r:
 * dst[s, r, 0:row_bytes] = src[s*slab_stride_bytes + idx[r]*row_stride_bytes + 0:row_bytes],
 * a byte-exact copy.
 *
 *   src   device; dst device, [n_slabs, n_idx, row_bytes] contiguous; they must not overlap.
 *   idx   device, [n_idx] int32, each in [0, n_rows_src); an out-of-range index copies
 *         nothing for that row and records STRUCTKV_ERR_INVALID_ARG in the device status word.
 *   row_bytes > 0.  When src, dst, both strides and row_bytes are multiples of 16 the copy
 *   uses 16-byte accesses; otherwise 4-byte or single-byte accesses.
 * Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_compact(structkv_ctx* ctx, const void* src, long long slab_stride_bytes,
                                 long long row_stride_bytes, int row_bytes, int n_slabs,
                                 int n_rows_src, const int* idx, int n_idx, void* dst,
                                 void* stream);

/*
 * structkv_compact (Algorithm 1 line 17) for several layers in ONE launch: layer l gathers rows of
 * its own source srcs[l] at its own index list idx + l*idx_layer_stride into
 * dst + l*dst_layer_stride_bytes, laid out [n_slabs, n_idx, row_bytes].  With small budgets a
 * gather per layer is a chain of launches of a few microseconds each; one launch removes it.
 *   srcs      HOST array of n_layers device pointers (1 .. 128 layers), all sources sharing
 *             slab_stride_bytes, row_stride_bytes, row_bytes, n_slabs and n_rows_src.
 *   idx       device, int32, n_idx entries per layer, idx_layer_stride >= n_idx.
 * An out-of-range index copies nothing and records STRUCTKV_ERR_INVALID_ARG in the device status
 * word.  Bit exact.  Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_compact_layers(structkv_ctx* ctx, const void* const* srcs, int n_layers,
                                        long long slab_stride_bytes, long long row_stride_bytes, int row_bytes,
                                        int n_slabs, int n_rows_src, const int* idx, long long idx_layer_stride,
                                        int n_idx, void* dst, long long dst_layer_stride_bytes, void* stream);

/*
 * Per-KV-group saliency and per-slab gathers: the per-head variant of the cache selection.
 * Paper: Section 3.2, the sentence before Eq. 2 (attention is aggregated over the query heads
 * that share a KV head); Eq. 13 applied per KV head instead of per layer; and Section 4.1, the
 * masked state transition for batches whose sequences carry different index sets.
 *
 * structkv_group_saliency: group_out[g, j] = sum over the G = H / H_kv query heads h of KV group
 * g of head_cols[h, j], where head_cols is the pooled per-head attention written by
 * structkv_score_layer (head_cols_out).  Summing group_out over g gives S^(l).
 *   head_cols device, [H, n] fp32 rows col_stride apart (elements);  group_out device, [H_kv, n].
 *
 * structkv_compact_per_slab: structkv_compact with one index list per slab,
 * dst[s, r, :] = src[s, idx[s*idx_slab_stride + r], :]  (idx_slab_stride >= n_idx, in elements):
 * one list per KV head (lists from structkv_select over group_out), or one list per sequence
 * of a batch.  All other arguments, the out-of-range rule and the byte exactness are those of
 * structkv_compact.
 * Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_group_saliency(structkv_ctx* ctx, const float* head_cols, long long col_stride,
                                        int n, float* group_out, void* stream);
structkv_status structkv_compact_per_slab(structkv_ctx* ctx, const void* src, long long slab_stride_bytes,
                                          long long row_stride_bytes, int row_bytes, int n_slabs,
                                          int n_rows_src, const int* idx, long long idx_slab_stride,
                                          int n_idx, void* dst, void* stream);

/*
 * Block-Level Aggregation for block-based KV memory managers.  Paper: Section 4.1,
 * implementation details: the importance of physical block k is the sum of the token scores
 * (the Global In-Degree Centrality) inside it, S_block_k = sum_{t in block_k} C[t]; blocks with
 * the lowest scores are evicted.  Block k covers tokens [k*block_size, min(n, (k+1)*block_size));
 * the last block may be ragged.  Block-granular selection and gathering then go through
 * structkv_select (scores = block scores, budget and window counted in blocks) and
 * structkv_compact (row = one block of one KV head, when n is a multiple of block_size).
 *
 *   scores           device, fp32, vector b starts at scores + b*row_stride (elements).
 *   block_scores_out device, [batch, ceil(n / block_size)] fp32.
 * Sums run in token order in fp32.  Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_block_scores(structkv_ctx* ctx, const float* scores, long long row_stride,
                                      int batch, int n, int block_size, float* block_scores_out,
                                      void* stream);

/*
 * Attention-mass recovery of a retained token set.  Paper: Section 4.4, "Fidelity of Hidden
 * States": the share of the original attention weights covered by the retained tokens, per
 * layer.  With the window attention of Eq. 1-2 every row sums to 1, so for layer l the share is
 * sum_{j in idx} S^(l)_j / sum_j S^(l)_j.
 *
 *   scores       device, fp32, one saliency vector per layer, vector b at scores + b*row_stride.
 *   idx          device, [n_idx] int32 retained positions in [0, n); an out-of-range index adds
 *                nothing and records STRUCTKV_ERR_INVALID_ARG in the device status word.
 *   recovery_out device, [batch] fp32.
 * Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_mass_recovery(structkv_ctx* ctx, const float* scores, long long row_stride,
                                       int batch, int n, const int* idx, int n_idx, float* recovery_out,
                                       void* stream);

/*
 * Self-test of the error path every device-side wait shares (the paper has no counterpart; the
 * conventions at the top of this header define it): launches one thread that waits, with the
 * scorer's bounded-wait helper and a bound of `limit_cycles` SM clock cycles (1 .. 4e9), on a
 * barrier nothing arrives on.  No copy or tensor-core work is in flight; when the bound runs out
 * the kernel records STRUCTKV_ERR_TIMEOUT in the device status word and returns, so the next
 * structkv_poll_device_status() reports TIMEOUT once and OK afterwards.
 * Errors: INVALID_ARG, CUDA.  Asynchronous on `stream`.
 */
structkv_status structkv_selftest_wait_expiry(structkv_ctx* ctx, unsigned long long limit_cycles,
                                              void* stream);

/* Reads and clears the device status word (bounded-wait expiry, bad gather index).
 * Synchronises `stream`.  Returns STRUCTKV_OK if nothing was recorded. */
structkv_status structkv_poll_device_status(structkv_ctx* ctx, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* STRUCTKV_H_ */
