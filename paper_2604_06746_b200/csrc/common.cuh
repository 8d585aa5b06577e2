// Internal declarations shared by the translation units of libstructkv (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "structkv.h"

namespace skv {

constexpr int kKeyTile = 128;        // keys per tile in every scorer
constexpr int kMaxParts = 160;       // upper bound on key segments per score row
constexpr int kRowBlock = 256;       // score rows (head, window row) per tensor-core row block
constexpr int kMaxBatch = 32;        // sequences one batched scoring call may hold
constexpr int kMaxStatLayers = 128;   // layers one batched head-statistics call may cover
constexpr int kMaxGatherLayers = 128; // layers one multi-layer gather may cover (their pointers are a kernel argument)
constexpr int kQueueUnits = 256;      // (KV group, row block) units of one sequence the scorer's work queue can hold
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Device status word values are structkv_status codes; 0 = nothing recorded.
struct Workspace {
  int* status;          // [64] ints, word 0 is the status
  float4* row_part;     // [kMaxParts][rows_pad] (m2, Z, U, unused) partial softmax statistics
  float* row_lse2;      // [rows_pad] log2-domain log-sum-exp of each score row
  float* row_ent;       // [rows_pad] entropy of each score row (nats)
  float* cols;          // [H][n_pad] pooled per-head attention when the caller passes none
  float* head_part;     // [kMaxStatLayers][H][4] per-(layer, head) {sum of squared deviations from 1/n, top-k mass}
  // [kMaxBatch][kQueueUnits] ticket counters of the tensor-core scorer's second pass, one per
  // (sequence slot of a call, KV group, row block); zero when the context is created.  A launch
  // draws exactly T = tiles + CTAs-of-the-unit tickets from a unit's counter and reads a ticket
  // modulo T, so launches of one shape follow each other with no reset and no per-launch host
  // state (a captured launch can be replayed); the host zeroes a slot only when its T changes
  // (queue_period in Ctx)
  unsigned long long* queue;
  size_t bytes;
};

struct Ctx {
  structkv_config cfg;
  Workspace ws;
  int device;
  int sm_count;
  int rows;             // H * w
  int rows_pad;         // rows per KV group padded to kRowBlock, times H_kv
  int n_pad;            // max_seq rounded up to kKeyTile
  void* tc;             // tensor-core scorer state (tensor maps), owned by score_tc.cu
  // tickets per launch (T) the counters of a sequence slot were last used with: [0] for the units
  // on full row blocks, [1] for the units on a KV group's last row block; 0 = counters are zero
  unsigned int queue_period[kMaxBatch][2] = {};
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Carves the workspace; with base == nullptr only the size is computed.
Workspace carve_workspace(const structkv_config& cfg, void* base);

// ---- launchers (each returns cudaGetLastError() of its launches) -------------------------
struct ScoreArgs {
  const void* q;            // [H, w, d]
  const void* k;
  long long k_stride_head, k_stride_token;   // elements
  int n_keys;               // keys of the sequence (a plain call), unused for a batch
  int batch;                // sequences in the call (1 for a plain call)
  int total_keys;           // rows of K along the token axis: n_keys, or cu_seqlens[batch]
  const int* cu_seqlens;    // host, [batch + 1] first key of every sequence in the packed K; NULL = plain call
  float scale;
  bool inputs_ready = false; // q and k are complete and visible: nothing in flight on the stream writes them
  // completion counter of pass 1 (device, or NULL) and how many pass-1 launches, this one included,
  // have used it since it was zeroed: pass 2 of the same layer waits for done_round * grid
  unsigned int* done = nullptr;
  int done_round = 0;
  // ticket counters for this launch alone ([kQueueUnits], zero), or NULL for the context's shared ones
  unsigned long long* queue = nullptr;
  float* cols;              // [H][col_stride] pooled per-head attention (output of pass 2)
  long long col_stride;
};

// CUDA-core two-pass scorer (fp32 or bf16 storage).  parts_out = key segments per row.
cudaError_t launch_score_simt(const Ctx& ctx, const ScoreArgs& a, int* parts_out, int pass,
                              cudaStream_t st);

// Tensor-core (tcgen05) two-pass scorer for bf16 storage.
bool tc_supported(const Ctx& ctx, const ScoreArgs& a);
structkv_status tc_create(Ctx& ctx);
void tc_destroy(Ctx& ctx);
cudaError_t launch_score_tc(Ctx& ctx, const ScoreArgs& a, int* parts_out, int pass, cudaStream_t st);

// One thread waits (bounded by limit_cycles) on a barrier nobody arrives on, then records
// STRUCTKV_ERR_TIMEOUT in *status.
cudaError_t launch_wait_probe(unsigned long long limit_cycles, int* status, cudaStream_t st);

// Merges the per-segment softmax statistics of every row into row_lse2 / row_ent (used by the
// CUDA-core scorer; the tensor-core scorer does this at the start of its second pass).
cudaError_t launch_finalize_rows(const Ctx& ctx, int parts, cudaStream_t st);

// S_j = sum_h cols[h][j]; optional C <- lambda C + S; then the layer's metrics: metrics[0] from
// row_ent (Eq. 4); metrics[1..2] from the pooled per-head attention (Eq. 5-6, computed here when
// with_head_stats), or NaN.
cudaError_t launch_reduce_finish(const Ctx& ctx, const float* cols, long long col_stride, int n, float lambda,
                                 float* s_out, float* c_inout, bool with_head_stats, float* metrics,
                                 cudaStream_t st);
// The same for n_layers layers in one launch: S^(l) rows s_stride apart, C carried from layer to
// layer, entropies from row_ent[l][rows_pad]; metrics [n_layers][3] with NaN for sparsity / variance.
cudaError_t launch_reduce_layers(const Ctx& ctx, const float* cols, long long layer_stride, long long col_stride,
                                 int n, int n_layers, float lambda, float* s_out, long long s_stride,
                                 float* c_inout, const float* row_ent, float* metrics, cudaStream_t st);

// Eq. 5-6 for n_layers layers at once from their pooled per-head attention: writes metrics[l][1..2].
cudaError_t launch_head_stats_batch(const Ctx& ctx, const float* cols, long long layer_stride, long long col_stride,
                                    int n_layers, int n, float* metrics, cudaStream_t st);

cudaError_t launch_accumulate(const float* s_hist, long long row_stride, int pivot, int n,
                              float lambda, float* c_out, cudaStream_t st);

cudaError_t launch_select(const float* scores, long long row_stride, int batch, int n, int budget,
                          int window, int* idx_out, cudaStream_t st);

cudaError_t launch_block_scores(const float* scores, long long row_stride, int batch, int n, int block_size,
                                float* out, cudaStream_t st);
cudaError_t launch_mass_recovery(const float* scores, long long row_stride, int batch, int n, const int* idx,
                                 int n_idx, float* out, int* status, cudaStream_t st);

cudaError_t launch_compact(const void* src, long long slab_stride, long long row_stride,
                           int row_bytes, int n_slabs, int n_rows_src, const int* idx,
                           long long idx_slab_stride, int n_idx, void* dst, int* status, int sm_count,
                           cudaStream_t st);
cudaError_t launch_compact_layers(const void* const* srcs, int n_layers, long long slab_stride, long long row_stride,
                                  int row_bytes, int n_slabs, int n_rows_src, const int* idx,
                                  long long idx_layer_stride, int n_idx, void* dst, long long dst_layer_stride,
                                  int* status, int sm_count, cudaStream_t st);
cudaError_t launch_group_saliency(const float* head_cols, long long col_stride, int n_heads, int group, int n,
                                  float* out, cudaStream_t st);

// Programmatic dependent launch: a kernel launched with launch_pdl() may begin (block scheduling,
// its own set-up) while the kernel before it in the stream is still draining.  pdl_trigger() lets
// the next kernel begin; pdl_wait() returns once the previous kernel has completed and its
// writes are visible, and must precede the first access to anything that kernel wrote or read.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// 2^x on the special-function unit (relative error about 2^-22; denormal results flush to 0).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Called by all threads of a 1024-thread block after a histogram pass over `nb` = 2048 bins.
// Walks the bins from the top and finds the bin holding the `remaining`-th largest candidate;
// writes that bin and the rank still wanted inside it.  `scratch` holds 33 words.
__device__ __forceinline__ void block_pick_from_top(const unsigned* hist, unsigned remaining,
                                                    unsigned* scratch, unsigned* sel_bin, unsigned* sel_rem) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b_hi = 2047 - 2 * tid, b_lo = b_hi - 1;        // this thread's two bins, higher first
  const unsigned c_hi = hist[b_hi], c_lo = hist[b_lo];
  const unsigned mine = c_hi + c_lo;
  unsigned incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  unsigned before = incl - mine;
  for (int w = 0; w < warp; ++w) before += scratch[w];
  if (before < remaining && remaining <= before + mine) {
    if (before + c_hi >= remaining) { *sel_bin = (unsigned)b_hi; *sel_rem = remaining - before; }
    else { *sel_bin = (unsigned)b_lo; *sel_rem = remaining - before - c_hi; }
  }
  __syncthreads();
}

}  // namespace skv
