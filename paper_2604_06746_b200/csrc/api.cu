// C ABI of libstructkv: argument validation, context and workspace bookkeeping, dispatch to
// the kernels, and the host-side pivot rule (Eq. 7-9).
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "common.cuh"

struct structkv_ctx {
  skv::Ctx c;
};

namespace skv {

static bool config_ok(const structkv_config& cfg) {
  if (cfg.n_q_heads <= 0 || cfg.n_kv_heads <= 0 || cfg.n_q_heads % cfg.n_kv_heads != 0) return false;
  if (cfg.n_q_heads > 1024) return false;
  if (cfg.window < 1 || cfg.max_seq < cfg.window) return false;
  if (cfg.dtype != STRUCTKV_BF16 && cfg.dtype != STRUCTKV_FP32) return false;
  if (cfg.head_dim <= 0) return false;
  return true;
}
static bool config_supported(const structkv_config& cfg) {
  return (cfg.head_dim == 64 || cfg.head_dim == 128) && cfg.window <= 256;
}

static int rows_pad_of(const structkv_config& cfg) {
  const int rows_pg = (cfg.n_q_heads / cfg.n_kv_heads) * cfg.window;
  return cfg.n_kv_heads * (int)align_up((size_t)rows_pg, kRowBlock);
}

Workspace carve_workspace(const structkv_config& cfg, void* base) {
  Workspace w{};
  char* p = (char*)base;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* r = p ? (void*)(p + off) : nullptr;
    off += align_up(bytes, 256);
    return r;
  };
  const size_t rows_pad = (size_t)rows_pad_of(cfg);
  const size_t n_pad = align_up((size_t)cfg.max_seq, kKeyTile);
  w.status = (int*)take(256);
  w.row_part = (float4*)take((size_t)kMaxParts * rows_pad * sizeof(float4));
  w.row_lse2 = (float*)take(rows_pad * sizeof(float));
  w.row_ent = (float*)take(rows_pad * sizeof(float));
  w.cols = (float*)take((size_t)cfg.n_q_heads * n_pad * sizeof(float));
  w.head_part = (float*)take((size_t)kMaxStatLayers * cfg.n_q_heads * 4 * sizeof(float));
  w.queue = (unsigned long long*)take((size_t)kMaxBatch * kQueueUnits * sizeof(unsigned long long));
  w.bytes = off;
  return w;
}

}  // namespace skv

using namespace skv;

extern "C" {

int structkv_version(void) { return 100; }

const char* structkv_status_string(structkv_status s) {
  switch (s) {
    case STRUCTKV_OK: return "ok";
    case STRUCTKV_ERR_INVALID_ARG: return "invalid argument";
    case STRUCTKV_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case STRUCTKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case STRUCTKV_ERR_CUDA: return "CUDA call failed";
    case STRUCTKV_ERR_TIMEOUT: return "bounded device wait expired";
  }
  return "unknown status";
}

size_t structkv_workspace_bytes(const structkv_config* cfg) {
  if (!cfg || !config_ok(*cfg) || !config_supported(*cfg)) return 0;
  return carve_workspace(*cfg, nullptr).bytes;
}

structkv_status structkv_create(structkv_ctx** ctx_out, const structkv_config* cfg,
                                void* workspace_dev, size_t workspace_bytes) {
  if (!ctx_out || !cfg) return STRUCTKV_ERR_INVALID_ARG;
  *ctx_out = nullptr;
  if (!config_ok(*cfg)) return STRUCTKV_ERR_INVALID_ARG;
  if (!config_supported(*cfg)) return STRUCTKV_ERR_UNSUPPORTED;
  const size_t need = carve_workspace(*cfg, nullptr).bytes;
  if (!workspace_dev || workspace_bytes < need || ((uintptr_t)workspace_dev % 256) != 0)
    return STRUCTKV_ERR_WORKSPACE;
  structkv_ctx* ctx = new (std::nothrow) structkv_ctx();
  if (!ctx) return STRUCTKV_ERR_INVALID_ARG;
  Ctx& c = ctx->c;
  c.cfg = *cfg;
  c.ws = carve_workspace(*cfg, workspace_dev);
  c.rows = cfg->n_q_heads * cfg->window;
  c.rows_pad = rows_pad_of(*cfg);
  c.n_pad = (int)align_up((size_t)cfg->max_seq, kKeyTile);
  c.tc = nullptr;
  if (cudaGetDevice(&c.device) != cudaSuccess ||
      cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, c.device) != cudaSuccess ||
      cudaMemset(c.ws.status, 0, 256) != cudaSuccess ||
      cudaMemset(c.ws.queue, 0, (size_t)kMaxBatch * kQueueUnits * sizeof(unsigned long long)) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess) {
    delete ctx;
    return STRUCTKV_ERR_CUDA;
  }
  if (cfg->dtype == STRUCTKV_BF16) {
    const structkv_status s = tc_create(c);
    if (s != STRUCTKV_OK) { delete ctx; return s; }
  }
  *ctx_out = ctx;
  return STRUCTKV_OK;
}

void structkv_destroy(structkv_ctx* ctx) {
  if (!ctx) return;
  tc_destroy(ctx->c);
  delete ctx;
}

structkv_status structkv_score_layer(structkv_ctx* ctx, const void* q_window, const void* k,
                                     long long k_stride_head, long long k_stride_token, int n_keys,
                                     float scale, float lambda, float* s_out, float* c_inout,
                                     float* head_cols_out, float* metrics_out, unsigned flags,
                                     void* stream) {
  if (!ctx || !q_window || !k || !s_out || !metrics_out) return STRUCTKV_ERR_INVALID_ARG;
  Ctx& c = ctx->c;
  const structkv_config& cfg = c.cfg;
  const int esz = cfg.dtype == STRUCTKV_BF16 ? 2 : 4;
  if (n_keys < cfg.window || n_keys > cfg.max_seq) return STRUCTKV_ERR_INVALID_ARG;
  if (!std::isfinite(scale) || !std::isfinite(lambda)) return STRUCTKV_ERR_INVALID_ARG;
  if (((uintptr_t)q_window % 16) || ((uintptr_t)k % 16)) return STRUCTKV_ERR_INVALID_ARG;
  if (k_stride_token < cfg.head_dim || k_stride_head < 0) return STRUCTKV_ERR_INVALID_ARG;
  if ((k_stride_token * esz) % 16 || (k_stride_head * esz) % 16) return STRUCTKV_ERR_INVALID_ARG;
  if (((uintptr_t)s_out % 4) || ((uintptr_t)metrics_out % 4) || ((uintptr_t)c_inout % 4) ||
      ((uintptr_t)head_cols_out % 4))
    return STRUCTKV_ERR_INVALID_ARG;
  if (flags & ~(STRUCTKV_FLAG_NO_HEAD_STATS | STRUCTKV_FLAG_FORCE_SIMT | STRUCTKV_FLAG_INPUTS_READY))
    return STRUCTKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;

  ScoreArgs a;
  a.q = q_window; a.k = k;
  a.k_stride_head = k_stride_head; a.k_stride_token = k_stride_token;
  a.n_keys = n_keys; a.scale = scale;
  a.batch = 1; a.total_keys = n_keys; a.cu_seqlens = nullptr;
  a.inputs_ready = (flags & STRUCTKV_FLAG_INPUTS_READY) != 0;
  a.cols = head_cols_out ? head_cols_out : c.ws.cols;
  a.col_stride = head_cols_out ? (long long)n_keys : (long long)c.n_pad;

  const bool use_tc = cfg.dtype == STRUCTKV_BF16 && !(flags & STRUCTKV_FLAG_FORCE_SIMT) &&
                      tc_supported(c, a);
  int parts = 0;
  cudaError_t e;
  e = use_tc ? launch_score_tc(c, a, &parts, 1, st) : launch_score_simt(c, a, &parts, 1, st);
  if (e != cudaSuccess) return STRUCTKV_ERR_CUDA;
  if (!use_tc) {
    e = launch_finalize_rows(c, parts, st);
    if (e != cudaSuccess) return STRUCTKV_ERR_CUDA;
  }
  e = use_tc ? launch_score_tc(c, a, &parts, 2, st) : launch_score_simt(c, a, &parts, 2, st);
  if (e != cudaSuccess) return STRUCTKV_ERR_CUDA;
  e = launch_reduce_finish(c, a.cols, a.col_stride, n_keys, lambda, s_out, c_inout,
                           !(flags & STRUCTKV_FLAG_NO_HEAD_STATS), metrics_out, st);
  return e == cudaSuccess ? STRUCTKV_OK : STRUCTKV_ERR_CUDA;
}

// ---- batches of prompts of different lengths (packed along the token axis) ------------------
namespace skv {
struct BatchWs { float4* row_part; float* row_ent; float* cols; float* head_part; size_t bytes; };
static BatchWs carve_batch(const structkv_config& cfg, int max_batch, long long max_total, void* base) {
  BatchWs w{};
  char* p = (char*)base;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* r = p ? (void*)(p + off) : nullptr;
    off += align_up(bytes, 256);
    return r;
  };
  const size_t rows_all = (size_t)max_batch * rows_pad_of(cfg);
  const size_t t_pad = align_up((size_t)max_total, kKeyTile);
  w.row_part = (float4*)take((size_t)kMaxParts * rows_all * sizeof(float4));
  w.row_ent = (float*)take(rows_all * sizeof(float));
  w.cols = (float*)take((size_t)cfg.n_q_heads * t_pad * sizeof(float));
  w.head_part = (float*)take((size_t)max_batch * cfg.n_q_heads * 4 * sizeof(float));
  w.bytes = off;
  return w;
}
}  // namespace skv

size_t structkv_batch_workspace_bytes(const structkv_config* cfg, int max_batch, long long max_total_tokens) {
  if (!cfg || !config_ok(*cfg) || !config_supported(*cfg)) return 0;
  if (max_batch < 1 || max_batch > kMaxBatch || max_total_tokens < cfg->window || max_total_tokens > 0x7fffff00ll)
    return 0;
  return carve_batch(*cfg, max_batch, max_total_tokens, nullptr).bytes;
}

structkv_status structkv_score_layer_batch(structkv_ctx* ctx, const void* q_window, const void* k,
                                           long long k_stride_head, long long k_stride_token,
                                           const int* cu_seqlens, int batch, float scale, float lambda,
                                           float* s_out, float* c_inout, float* head_cols_out,
                                           float* metrics_out, unsigned flags, void* batch_workspace,
                                           size_t batch_workspace_bytes, void* stream) {
  if (!ctx || !q_window || !k || !cu_seqlens || !s_out || !metrics_out) return STRUCTKV_ERR_INVALID_ARG;
  if (batch < 1 || batch > kMaxBatch) return STRUCTKV_ERR_INVALID_ARG;
  Ctx& c = ctx->c;
  const structkv_config& cfg = c.cfg;
  if (cu_seqlens[0] != 0) return STRUCTKV_ERR_INVALID_ARG;
  for (int b = 0; b < batch; ++b) {
    const long long n_b = (long long)cu_seqlens[b + 1] - cu_seqlens[b];
    if (n_b < cfg.window || n_b > cfg.max_seq) return STRUCTKV_ERR_INVALID_ARG;
  }
  const int total = cu_seqlens[batch];
  if (!std::isfinite(scale) || !std::isfinite(lambda)) return STRUCTKV_ERR_INVALID_ARG;
  if (((uintptr_t)q_window % 16) || ((uintptr_t)k % 16)) return STRUCTKV_ERR_INVALID_ARG;
  if (k_stride_token < cfg.head_dim || k_stride_head < 0) return STRUCTKV_ERR_INVALID_ARG;
  if ((k_stride_token * 2) % 16 || (k_stride_head * 2) % 16) return STRUCTKV_ERR_INVALID_ARG;
  if (flags & ~(STRUCTKV_FLAG_NO_HEAD_STATS | STRUCTKV_FLAG_INPUTS_READY)) return STRUCTKV_ERR_INVALID_ARG;
  const size_t need = carve_batch(cfg, batch, total, nullptr).bytes;
  if (!batch_workspace || batch_workspace_bytes < need || ((uintptr_t)batch_workspace % 256) != 0)
    return STRUCTKV_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const BatchWs bw = carve_batch(cfg, batch, total, batch_workspace);

  Ctx view = c;                       // same device, tensor-map encoder and status word; batch-sized scratch
  view.ws.row_part = bw.row_part;
  view.ws.row_ent = bw.row_ent;
  view.ws.cols = bw.cols;
  view.ws.head_part = bw.head_part;
  // the ticket counters stay the context's own (its workspace is known to be initialised)
  ScoreArgs a;
  a.q = q_window; a.k = k;
  a.k_stride_head = k_stride_head; a.k_stride_token = k_stride_token;
  a.n_keys = 0; a.batch = batch; a.total_keys = total; a.cu_seqlens = cu_seqlens;
  a.scale = scale;
  a.inputs_ready = (flags & STRUCTKV_FLAG_INPUTS_READY) != 0;
  a.cols = head_cols_out ? head_cols_out : bw.cols;
  a.col_stride = head_cols_out ? (long long)total : (long long)align_up((size_t)total, kKeyTile);
  // only the tensor-core scorer handles packed batches
  if (cfg.dtype != STRUCTKV_BF16 || !tc_supported(view, a)) return STRUCTKV_ERR_UNSUPPORTED;
  int parts = 0;
  if (launch_score_tc(view, a, &parts, 1, st) != cudaSuccess) return STRUCTKV_ERR_CUDA;
  if (launch_score_tc(view, a, &parts, 2, st) != cudaSuccess) return STRUCTKV_ERR_CUDA;
  std::memcpy(c.queue_period, view.queue_period, sizeof(c.queue_period));   // the launches updated the view's copy
  // per sequence: S = sum over heads, C <- lambda C + S, and the sequence's metric triple
  for (int b = 0; b < batch; ++b) {
    const int key0 = cu_seqlens[b], n_b = cu_seqlens[b + 1] - key0;
    Ctx one = view;
    one.ws.row_ent = bw.row_ent + (size_t)b * c.rows_pad;
    one.ws.head_part = bw.head_part + (size_t)b * cfg.n_q_heads * 4;
    if (launch_reduce_finish(one, a.cols + key0, a.col_stride, n_b, lambda, s_out + key0,
                             c_inout ? c_inout + key0 : nullptr, !(flags & STRUCTKV_FLAG_NO_HEAD_STATS),
                             metrics_out + 3 * b, st) != cudaSuccess)
      return STRUCTKV_ERR_CUDA;
  }
  return STRUCTKV_OK;
}

// ---- several resident layers in one call, the passes of neighbouring layers interleaved ---------
namespace skv {
struct LayersWs { float4* row_part[2]; float* row_ent; unsigned int* done; unsigned long long* queue; size_t bytes; };
static LayersWs carve_layers(const structkv_config& cfg, int max_layers, void* base) {
  LayersWs w{};
  char* p = (char*)base;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* r = p ? (void*)(p + off) : nullptr;
    off += align_up(bytes, 256);
    return r;
  };
  const size_t rows_pad = (size_t)rows_pad_of(cfg);
  w.done = (unsigned int*)take(256);
  w.queue = (unsigned long long*)take((size_t)max_layers * kQueueUnits * sizeof(unsigned long long));   // follows `done`: one memset
  for (int i = 0; i < 2; ++i) w.row_part[i] = (float4*)take((size_t)kMaxParts * rows_pad * sizeof(float4));
  w.row_ent = (float*)take((size_t)max_layers * rows_pad * sizeof(float));
  w.bytes = off;
  return w;
}
}  // namespace skv

size_t structkv_layers_workspace_bytes(const structkv_config* cfg, int max_layers) {
  if (!cfg || !config_ok(*cfg) || !config_supported(*cfg) || max_layers < 1 || max_layers > 65536) return 0;
  return carve_layers(*cfg, max_layers, nullptr).bytes;
}

structkv_status structkv_score_layers(structkv_ctx* ctx, int n_layers, const void* const* q_windows,
                                      const void* const* ks, long long k_stride_head,
                                      long long k_stride_token, int n_keys, const float* scales, float lambda,
                                      float* s_out, long long s_layer_stride, float* c_inout,
                                      float* head_cols_out, long long head_cols_layer_stride,
                                      float* metrics_out, void* layers_workspace,
                                      size_t layers_workspace_bytes, void* stream) {
  if (!ctx || !q_windows || !ks || !scales || !s_out || !head_cols_out || !metrics_out)
    return STRUCTKV_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > 65536) return STRUCTKV_ERR_INVALID_ARG;
  Ctx& c = ctx->c;
  const structkv_config& cfg = c.cfg;
  const int esz = cfg.dtype == STRUCTKV_BF16 ? 2 : 4;
  if (n_keys < cfg.window || n_keys > cfg.max_seq || !std::isfinite(lambda)) return STRUCTKV_ERR_INVALID_ARG;
  if (k_stride_token < cfg.head_dim || k_stride_head < 0) return STRUCTKV_ERR_INVALID_ARG;
  if ((k_stride_token * esz) % 16 || (k_stride_head * esz) % 16) return STRUCTKV_ERR_INVALID_ARG;
  if (s_layer_stride < n_keys || head_cols_layer_stride < (long long)cfg.n_q_heads * n_keys)
    return STRUCTKV_ERR_INVALID_ARG;
  if (((uintptr_t)s_out % 4) || ((uintptr_t)metrics_out % 4) || ((uintptr_t)c_inout % 4) ||
      ((uintptr_t)head_cols_out % 4))
    return STRUCTKV_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!q_windows[l] || !ks[l] || ((uintptr_t)q_windows[l] % 16) || ((uintptr_t)ks[l] % 16) ||
        !std::isfinite(scales[l]))
      return STRUCTKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;

  auto args_of = [&](int l) {
    ScoreArgs a;
    a.q = q_windows[l]; a.k = ks[l];
    a.k_stride_head = k_stride_head; a.k_stride_token = k_stride_token;
    a.n_keys = n_keys; a.scale = scales[l];
    a.batch = 1; a.total_keys = n_keys; a.cu_seqlens = nullptr;
    a.cols = head_cols_out + (size_t)l * head_cols_layer_stride;
    a.col_stride = n_keys;
    return a;
  };
  ScoreArgs probe = args_of(0);
  if (cfg.dtype != STRUCTKV_BF16 || !tc_supported(c, probe)) {
    // the CUDA-core scorer has no interleaved form: one layer after the other, same results
    for (int l = 0; l < n_layers; ++l) {
      const structkv_status s = structkv_score_layer(
          ctx, q_windows[l], ks[l], k_stride_head, k_stride_token, n_keys, scales[l], lambda,
          s_out + (size_t)l * s_layer_stride, c_inout, head_cols_out + (size_t)l * head_cols_layer_stride,
          metrics_out + 3 * l, STRUCTKV_FLAG_NO_HEAD_STATS, stream);
      if (s != STRUCTKV_OK) return s;
    }
    return STRUCTKV_OK;
  }
  const size_t need = carve_layers(cfg, n_layers, nullptr).bytes;
  if (!layers_workspace || layers_workspace_bytes < need || ((uintptr_t)layers_workspace % 256) != 0)
    return STRUCTKV_ERR_WORKSPACE;
  const LayersWs lw = carve_layers(cfg, n_layers, layers_workspace);
  // completion counters and every layer's own ticket counters start from zero
  if (cudaMemsetAsync(lw.done, 0, 256 + (size_t)n_layers * kQueueUnits * sizeof(unsigned long long), st) != cudaSuccess)
    return STRUCTKV_ERR_CUDA;

  // Stream order: P1(0), then for every layer l: P1(l + 1), P2(l).  P2(l) waits for the completion
  // counter of P1(l), which finished while P1(l + 1) ran, instead of for the whole kernel before it;
  // P1(l + 2) overwrites the row statistics P2(l) reads only after P2(l), the kernel before it in
  // the stream, has completed.  Two statistics buffers and two counters alternate.
  Ctx view = c;
  auto launch = [&](int l, int pass) {
    view.ws.row_part = lw.row_part[l & 1];
    view.ws.row_ent = lw.row_ent + (size_t)l * c.rows_pad;
    ScoreArgs a = args_of(l);
    a.inputs_ready = true;
    a.done = lw.done + (l & 1);
    a.done_round = l / 2 + 1;
    a.queue = lw.queue + (size_t)l * kQueueUnits;
    int parts = 0;
    return launch_score_tc(view, a, &parts, pass, st) == cudaSuccess;
  };
  bool ok = launch(0, 1);
  for (int l = 0; ok && l < n_layers; ++l) {
    if (l + 1 < n_layers) ok = launch(l + 1, 1);
    ok = ok && launch(l, 2);
  }
  if (!ok) return STRUCTKV_ERR_CUDA;
  return launch_reduce_layers(c, head_cols_out, head_cols_layer_stride, n_keys, n_keys, n_layers, lambda, s_out,
                              s_layer_stride, c_inout, lw.row_ent, metrics_out, st) == cudaSuccess
             ? STRUCTKV_OK
             : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_select_batch(structkv_ctx* ctx, const float* scores, const int* cu_seqlens,
                                      const int* budgets, int batch, int window, int* idx_out,
                                      long long idx_stride, void* stream) {
  if (!ctx || !scores || !cu_seqlens || !budgets || !idx_out) return STRUCTKV_ERR_INVALID_ARG;
  if (batch < 1 || batch > kMaxBatch || window < 0) return STRUCTKV_ERR_INVALID_ARG;
  for (int b = 0; b < batch; ++b) {
    const long long n_b = (long long)cu_seqlens[b + 1] - cu_seqlens[b];
    if (n_b < 1 || budgets[b] < window || budgets[b] > n_b || budgets[b] > idx_stride)
      return STRUCTKV_ERR_INVALID_ARG;
  }
  cudaStream_t st = (cudaStream_t)stream;
  // padding entries read -1: no prompt ever addresses a batch-mate's tokens
  if (cudaMemsetAsync(idx_out, 0xff, (size_t)batch * idx_stride * sizeof(int), st) != cudaSuccess)
    return STRUCTKV_ERR_CUDA;
  for (int b = 0; b < batch; ++b) {
    const int key0 = cu_seqlens[b], n_b = cu_seqlens[b + 1] - key0;
    if (launch_select(scores + key0, 0, 1, n_b, budgets[b], window, idx_out + (size_t)b * idx_stride, st) !=
        cudaSuccess)
      return STRUCTKV_ERR_CUDA;
  }
  return STRUCTKV_OK;
}

structkv_status structkv_head_stats(structkv_ctx* ctx, const float* head_cols, long long layer_stride,
                                    long long col_stride, int n_layers, int n, float* metrics,
                                    void* stream) {
  if (!ctx || !head_cols || !metrics) return STRUCTKV_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > kMaxStatLayers || n < 1 || col_stride < n) return STRUCTKV_ERR_INVALID_ARG;
  if (n_layers > 1 && layer_stride < (long long)ctx->c.cfg.n_q_heads * col_stride) return STRUCTKV_ERR_INVALID_ARG;
  return launch_head_stats_batch(ctx->c, head_cols, layer_stride, col_stride, n_layers, n, metrics,
                                 (cudaStream_t)stream) == cudaSuccess ? STRUCTKV_OK : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_pivot(structkv_ctx* ctx, const float* metrics_dev, int n_layers,
                               const float* weights, int l_limit, int* pivot_out, float* t_out,
                               void* stream) {
  if (!ctx || !metrics_dev || !weights || !pivot_out || n_layers < 1 || n_layers > 65536)
    return STRUCTKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  std::vector<float> m((size_t)n_layers * 3);
  if (cudaMemcpyAsync(m.data(), metrics_dev, m.size() * sizeof(float), cudaMemcpyDeviceToHost, st) !=
          cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return STRUCTKV_ERR_CUDA;
  std::vector<double> T((size_t)n_layers, 0.0);
  const double sign[3] = {-1.0, 1.0, 1.0};       // Eq. 8 takes the gradient of -entropy
  for (int col = 0; col < 3 && n_layers >= 2; ++col) {
    bool nan_col = false;
    for (int l = 0; l < n_layers; ++l) nan_col |= std::isnan(m[(size_t)l * 3 + col]);
    if (nan_col) continue;
    double lo = INFINITY, hi = -INFINITY;
    for (int l = 1; l < n_layers; ++l) {
      const double d = sign[col] * ((double)m[(size_t)l * 3 + col] - (double)m[(size_t)(l - 1) * 3 + col]);
      lo = d < lo ? d : lo;
      hi = d > hi ? d : hi;
    }
    if (!(hi > lo)) continue;
    for (int l = 1; l < n_layers; ++l) {
      const double d = sign[col] * ((double)m[(size_t)l * 3 + col] - (double)m[(size_t)(l - 1) * 3 + col]);
      T[l] += (double)weights[col] * (d - lo) / (hi - lo);
    }
  }
  int best = 0;
  if (n_layers >= 2) {
    best = 1;
    for (int l = 2; l < n_layers; ++l)
      if (T[l] > T[best]) best = l;
    if (l_limit >= 0 && best > l_limit) best = l_limit;
  }
  *pivot_out = best;
  if (t_out)
    for (int l = 0; l < n_layers; ++l) t_out[l] = (float)T[l];
  return STRUCTKV_OK;
}

structkv_status structkv_accumulate(structkv_ctx* ctx, const float* s_hist, long long row_stride,
                                    int pivot, int n, float lambda, float* c_out, void* stream) {
  if (!ctx || !s_hist || !c_out || pivot < 0 || n < 1 || row_stride < n || !std::isfinite(lambda))
    return STRUCTKV_ERR_INVALID_ARG;
  return launch_accumulate(s_hist, row_stride, pivot, n, lambda, c_out, (cudaStream_t)stream) == cudaSuccess
             ? STRUCTKV_OK
             : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_select(structkv_ctx* ctx, const float* scores, long long row_stride,
                                int batch, int n, int budget, int window, int* idx_out,
                                void* stream) {
  if (!ctx || !scores || !idx_out) return STRUCTKV_ERR_INVALID_ARG;
  if (batch < 1 || n < 1 || window < 0 || window > budget || budget > n) return STRUCTKV_ERR_INVALID_ARG;
  if (batch > 1 && row_stride < n) return STRUCTKV_ERR_INVALID_ARG;
  return launch_select(scores, row_stride, batch, n, budget, window, idx_out, (cudaStream_t)stream) ==
                 cudaSuccess
             ? STRUCTKV_OK
             : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_compact(structkv_ctx* ctx, const void* src, long long slab_stride_bytes,
                                 long long row_stride_bytes, int row_bytes, int n_slabs,
                                 int n_rows_src, const int* idx, int n_idx, void* dst,
                                 void* stream) {
  if (!ctx || !src || !dst || !idx) return STRUCTKV_ERR_INVALID_ARG;
  if (row_bytes < 1 || n_slabs < 0 || n_rows_src < 1 || n_idx < 0) return STRUCTKV_ERR_INVALID_ARG;
  if (row_stride_bytes < row_bytes || slab_stride_bytes < 0) return STRUCTKV_ERR_INVALID_ARG;
  const Ctx& c = ctx->c;
  return launch_compact(src, slab_stride_bytes, row_stride_bytes, row_bytes, n_slabs, n_rows_src, idx, 0,
                        n_idx, dst, c.ws.status, c.sm_count, (cudaStream_t)stream) == cudaSuccess
             ? STRUCTKV_OK
             : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_compact_layers(structkv_ctx* ctx, const void* const* srcs, int n_layers,
                                        long long slab_stride_bytes, long long row_stride_bytes, int row_bytes,
                                        int n_slabs, int n_rows_src, const int* idx, long long idx_layer_stride,
                                        int n_idx, void* dst, long long dst_layer_stride_bytes, void* stream) {
  if (!ctx || !srcs || !dst || !idx) return STRUCTKV_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > kMaxGatherLayers) return STRUCTKV_ERR_INVALID_ARG;
  if (row_bytes < 1 || n_slabs < 0 || n_rows_src < 1 || n_idx < 0) return STRUCTKV_ERR_INVALID_ARG;
  if (row_stride_bytes < row_bytes || slab_stride_bytes < 0 || idx_layer_stride < n_idx) return STRUCTKV_ERR_INVALID_ARG;
  if (dst_layer_stride_bytes < (long long)n_slabs * n_idx * row_bytes) return STRUCTKV_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!srcs[l]) return STRUCTKV_ERR_INVALID_ARG;
  const Ctx& c = ctx->c;
  return launch_compact_layers(srcs, n_layers, slab_stride_bytes, row_stride_bytes, row_bytes, n_slabs, n_rows_src,
                               idx, idx_layer_stride, n_idx, dst, dst_layer_stride_bytes, c.ws.status, c.sm_count,
                               (cudaStream_t)stream) == cudaSuccess ? STRUCTKV_OK : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_compact_per_slab(structkv_ctx* ctx, const void* src, long long slab_stride_bytes,
                                          long long row_stride_bytes, int row_bytes, int n_slabs,
                                          int n_rows_src, const int* idx, long long idx_slab_stride,
                                          int n_idx, void* dst, void* stream) {
  if (!ctx || !src || !dst || !idx) return STRUCTKV_ERR_INVALID_ARG;
  if (row_bytes < 1 || n_slabs < 0 || n_rows_src < 1 || n_idx < 0) return STRUCTKV_ERR_INVALID_ARG;
  if (row_stride_bytes < row_bytes || slab_stride_bytes < 0 || idx_slab_stride < n_idx)
    return STRUCTKV_ERR_INVALID_ARG;
  const Ctx& c = ctx->c;
  return launch_compact(src, slab_stride_bytes, row_stride_bytes, row_bytes, n_slabs, n_rows_src, idx,
                        idx_slab_stride, n_idx, dst, c.ws.status, c.sm_count,
                        (cudaStream_t)stream) == cudaSuccess ? STRUCTKV_OK : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_group_saliency(structkv_ctx* ctx, const float* head_cols, long long col_stride,
                                        int n, float* group_out, void* stream) {
  if (!ctx || !head_cols || !group_out || n < 1 || col_stride < n) return STRUCTKV_ERR_INVALID_ARG;
  const structkv_config& cfg = ctx->c.cfg;
  return launch_group_saliency(head_cols, col_stride, cfg.n_q_heads, cfg.n_q_heads / cfg.n_kv_heads, n,
                               group_out, (cudaStream_t)stream) == cudaSuccess ? STRUCTKV_OK : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_block_scores(structkv_ctx* ctx, const float* scores, long long row_stride,
                                      int batch, int n, int block_size, float* block_scores_out,
                                      void* stream) {
  if (!ctx || !scores || !block_scores_out) return STRUCTKV_ERR_INVALID_ARG;
  if (batch < 1 || batch > 65535 || n < 1 || block_size < 1) return STRUCTKV_ERR_INVALID_ARG;
  if (batch > 1 && row_stride < n) return STRUCTKV_ERR_INVALID_ARG;
  return launch_block_scores(scores, row_stride, batch, n, block_size, block_scores_out,
                             (cudaStream_t)stream) == cudaSuccess ? STRUCTKV_OK : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_mass_recovery(structkv_ctx* ctx, const float* scores, long long row_stride,
                                       int batch, int n, const int* idx, int n_idx, float* recovery_out,
                                       void* stream) {
  if (!ctx || !scores || !idx || !recovery_out) return STRUCTKV_ERR_INVALID_ARG;
  if (batch < 1 || n < 1 || n_idx < 0) return STRUCTKV_ERR_INVALID_ARG;
  if (batch > 1 && row_stride < n) return STRUCTKV_ERR_INVALID_ARG;
  return launch_mass_recovery(scores, row_stride, batch, n, idx, n_idx, recovery_out, ctx->c.ws.status,
                              (cudaStream_t)stream) == cudaSuccess ? STRUCTKV_OK : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_selftest_wait_expiry(structkv_ctx* ctx, unsigned long long limit_cycles,
                                              void* stream) {
  if (!ctx || limit_cycles == 0 || limit_cycles > 4000000000ull) return STRUCTKV_ERR_INVALID_ARG;
  return launch_wait_probe(limit_cycles, ctx->c.ws.status, (cudaStream_t)stream) == cudaSuccess
             ? STRUCTKV_OK
             : STRUCTKV_ERR_CUDA;
}

structkv_status structkv_poll_device_status(structkv_ctx* ctx, void* stream) {
  if (!ctx) return STRUCTKV_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int word = 0;
  if (cudaMemcpyAsync(&word, ctx->c.ws.status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return STRUCTKV_ERR_CUDA;
  if (word != 0) {
    // a scorer launch that gave up may have left its ticket counters short of what the host
    // expects: start them over together with the status word
    if (cudaMemsetAsync(ctx->c.ws.status, 0, sizeof(int), st) != cudaSuccess ||
        cudaMemsetAsync(ctx->c.ws.queue, 0, (size_t)kMaxBatch * kQueueUnits * sizeof(unsigned long long), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
      return STRUCTKV_ERR_CUDA;
    std::memset(ctx->c.queue_period, 0, sizeof(ctx->c.queue_period));
  }
  if (word < 0 || word > (int)STRUCTKV_ERR_TIMEOUT) return STRUCTKV_ERR_CUDA;
  return (structkv_status)word;
}

}  // extern "C"

// ---- context-free scoring on scratch that is part of the library image --------------------
// In host code `g_static_scratch` is only a handle for the runtime's symbol table, never a
// device address: the address is resolved once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[STRUCTKV_STATIC_SCRATCH_BYTES];

namespace skv {
namespace {
constexpr int kMaxDevices = 64;
struct StaticSlot {
  bool ready = false;
  void* scratch = nullptr;   // device address of g_static_scratch on this device
  int sm_count = 0;
  void* tc = nullptr;        // tensor-map encoder state, kept for the life of the process
};
StaticSlot g_static_slots[kMaxDevices];
std::mutex g_static_mutex;

structkv_status static_slot_for_current_device(int* device_out, StaticSlot** slot_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return STRUCTKV_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return STRUCTKV_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticSlot& s = g_static_slots[dev];
  if (!s.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return STRUCTKV_ERR_CUDA;
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return STRUCTKV_ERR_CUDA;
    Ctx probe{};
    const structkv_status st = tc_create(probe);      // host-side only: a driver entry point lookup
    if (st != STRUCTKV_OK) return st;
    s.tc = probe.tc;
    s.scratch = ptr;
    s.ready = true;
  }
  *device_out = dev;
  *slot_out = &s;
  return STRUCTKV_OK;
}
}  // namespace
}  // namespace skv

extern "C" structkv_status structkv_score_layer_static(
    const structkv_config* cfg, const void* q_window, const void* k, long long k_stride_head,
    long long k_stride_token, int n_keys, float scale, float lambda, float* s_out, float* c_inout,
    float* head_cols_out, float* metrics_out, unsigned flags, void* stream) {
  if (!cfg) return STRUCTKV_ERR_INVALID_ARG;
  if (!config_ok(*cfg)) return STRUCTKV_ERR_INVALID_ARG;
  if (!config_supported(*cfg)) return STRUCTKV_ERR_UNSUPPORTED;
  const size_t need = carve_workspace(*cfg, nullptr).bytes;
  if (need == 0 || need > (size_t)STRUCTKV_STATIC_SCRATCH_BYTES) return STRUCTKV_ERR_WORKSPACE;
  int dev = -1;
  StaticSlot* slot = nullptr;
  const structkv_status st = static_slot_for_current_device(&dev, &slot);
  if (st != STRUCTKV_OK) return st;

  // A context that lives for this call only, laid over the static scratch.
  structkv_ctx tmp;
  Ctx& c = tmp.c;
  c.cfg = *cfg;
  c.ws = carve_workspace(*cfg, slot->scratch);
  c.device = dev;
  c.sm_count = slot->sm_count;
  c.rows = cfg->n_q_heads * cfg->window;
  c.rows_pad = rows_pad_of(*cfg);
  c.n_pad = (int)align_up((size_t)cfg->max_seq, kKeyTile);
  c.tc = cfg->dtype == STRUCTKV_BF16 ? slot->tc : nullptr;
  // The scratch keeps the previous call's contents; the status word must start from zero.
  if (cudaMemsetAsync(c.ws.status, 0, 256, (cudaStream_t)stream) != cudaSuccess) return STRUCTKV_ERR_CUDA;
  // the per-call context starts its ticket counters from zero as well
  if (cudaMemsetAsync(c.ws.queue, 0, (size_t)kMaxBatch * kQueueUnits * sizeof(unsigned long long), (cudaStream_t)stream) !=
      cudaSuccess)
    return STRUCTKV_ERR_CUDA;
  return structkv_score_layer(&tmp, q_window, k, k_stride_head, k_stride_token, n_keys, scale, lambda,
                              s_out, c_inout, head_cols_out, metrics_out, flags, stream);
}
