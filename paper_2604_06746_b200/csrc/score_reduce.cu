// Small deterministic reductions around the scorers: row finalisation (log-sum-exp, entropy),
// column reduction over heads with the centrality update, per-head sparsity / variance, and
// the closed-form centrality re-accumulation.
#include "common.cuh"

namespace skv {
namespace {

constexpr int kFinalThreads = 1024;

__device__ __forceinline__ float block_sum_1024(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float x = (lane < (int)(blockDim.x >> 5)) ? red[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    if (lane == 0) red[32] = x;
  }
  __syncthreads();
  return red[32];
}

// One block.  Row r of group g is valid iff its index inside the group is < rows_pg.
// Each of the `parts` key segments left (ref, Z, U) for the row: Z = sum 2^(x - ref),
// U = sum 2^(x - ref) (x - ref), x = logit * log2(e); ref is any reference the segment chose.
// With l_p = ref_p + log2 Z_p (the segment's log-sum-exp) and M = max_p l_p:
//   lse2 = M + log2 sum_p 2^(l_p - M)
//   mean of (x - M) under the row's softmax = sum_p 2^(l_p - M) (ref_p - M + U_p / Z_p) / sum_p 2^(l_p - M)
//   entropy = ln2 * (lse2 - M - that mean)                                   (Eq. 4, one row)
// The mean entropy over the valid rows goes to metrics[0].
__global__ void __launch_bounds__(kFinalThreads)
finalize_rows(const float4* __restrict__ row_part, int parts, int rows_pad, int rows_pg_pad,
              int rows_pg, int n_valid, float* __restrict__ row_lse2,
              float* __restrict__ row_ent, float* __restrict__ metrics) {
  __shared__ float red[33];
  float ent_sum = 0.f;
  for (int r = threadIdx.x; r < rows_pad; r += kFinalThreads) {
    const bool valid = (r % rows_pg_pad) < rows_pg;
    float lse2 = INFINITY, ent = 0.f;        // padded rows: 2^(x - inf) = 0 in pass 2
    if (valid) {
      float M = -INFINITY;
      for (int p = 0; p < parts; ++p) {
        const float4 v = row_part[(size_t)p * rows_pad + r];
        if (v.y > 0.f) M = fmaxf(M, v.x + log2f(v.y));
      }
      if (M != -INFINITY) {
        float Zt = 0.f, Xt = 0.f;
        for (int p = 0; p < parts; ++p) {
          const float4 v = row_part[(size_t)p * rows_pad + r];
          if (v.y > 0.f) {
            const float wgt = fast_exp2(v.x + log2f(v.y) - M);
            Zt += wgt;
            Xt = fmaf(wgt, (v.x - M) + v.z / v.y, Xt);
          }
        }
        const float lz = log2f(Zt);
        lse2 = M + lz;
        ent = kLn2 * (lz - Xt / Zt);
      }
    }
    row_lse2[r] = lse2;
    row_ent[r] = ent;
    ent_sum += ent;
  }
  const float tot = block_sum_1024(ent_sum, red);
  if (threadIdx.x == 0) metrics[0] = tot / (float)n_valid;
}

// S_j = sum over heads (fixed order) of cols[h][j];  C_j <- lambda C_j + S_j  (Eq. 2, Eq. 3).
__global__ void reduce_columns(const float* __restrict__ cols, long long col_stride, int H, int n,
                               float lambda, float* __restrict__ s_out,
                               float* __restrict__ c_inout) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  float s = 0.f;
  for (int h = 0; h < H; ++h) s += cols[(size_t)h * col_stride + j];
  s_out[j] = s;
  if (c_inout) c_inout[j] = fmaf(lambda, c_inout[j], s);
}

// Per head: sum of squares (Eq. 6) and the mass of the k_rho largest entries (Eq. 5), by a
// three-level radix select on the fp32 bit patterns (all entries are >= 0, so the unsigned
// order of the bits is the order of the values).  One block per head; deterministic.
constexpr int kHsThreads = 1024;
constexpr int kHsBins = 2048;

__global__ void __launch_bounds__(kHsThreads)
head_stats(const float* __restrict__ cols, long long col_stride, int n, int k_rho,
           float* __restrict__ head_part) {
  __shared__ unsigned hist[kHsBins];
  __shared__ float red[33];
  __shared__ unsigned sel_bin, sel_rem;
  const float* a = cols + (size_t)blockIdx.x * col_stride;
  const int tid = threadIdx.x;
  unsigned prefix = 0, prefix_mask = 0, remaining = (unsigned)k_rho;
  const int shifts[3] = {21, 10, 0};
  const int widths[3] = {11, 11, 10};
  float sq = 0.f;
  for (int pass = 0; pass < 3; ++pass) {
    for (int b = tid; b < kHsBins; b += kHsThreads) hist[b] = 0;
    __syncthreads();
    const unsigned bmask = (1u << widths[pass]) - 1u;
    for (int base = 0; base < n; base += kHsThreads) {      // warp-uniform trip count
      const int j = base + tid;
      const float v = (j < n) ? a[j] : 0.f;
      if (pass == 0) sq = fmaf(v, v, sq);
      const unsigned u = __float_as_uint(v);
      const bool cand = (j < n) && ((u & prefix_mask) == prefix);
      hist_add(hist, (u >> shifts[pass]) & bmask, cand);
    }
    __syncthreads();
    if (tid < 32) radix_pick_from_top(hist, 1 << widths[pass], remaining, &sel_bin, &sel_rem);
    __syncthreads();
    prefix |= sel_bin << shifts[pass];
    prefix_mask |= bmask << shifts[pass];
    remaining = sel_rem;
    __syncthreads();
  }
  // prefix is the bit pattern of the k_rho-th largest value; `remaining` copies of it are taken.
  const float thr = __uint_as_float(prefix);
  float mass = 0.f;
  for (int j = tid; j < n; j += kHsThreads) {
    const float v = a[j];
    if (__float_as_uint(v) > prefix) mass += v;
  }
  const float tot_mass = block_sum_1024(mass, red);
  const float tot_sq = block_sum_1024(sq, red);
  if (tid == 0) {
    head_part[blockIdx.x * 4 + 0] = tot_sq;
    head_part[blockIdx.x * 4 + 1] = fmaf((float)remaining, thr, tot_mass);
  }
}

// metrics[1] = mean_h top-mass;  metrics[2] = mean_h (sum_sq / n - 1 / n^2)   (rows sum to 1).
__global__ void head_stats_final(const float* __restrict__ head_part, int H, int n,
                                 float* __restrict__ metrics) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  float rho = 0.f, var = 0.f;
  const float inv_n = 1.f / (float)n;
  for (int h = 0; h < H; ++h) {
    rho += head_part[h * 4 + 1];
    var += head_part[h * 4 + 0] * inv_n - inv_n * inv_n;
  }
  metrics[1] = rho / (float)H;
  metrics[2] = var / (float)H;
}

__global__ void fill_nan_stats(float* metrics) {
  metrics[1] = __int_as_float(0x7fc00000);
  metrics[2] = __int_as_float(0x7fc00000);
}

// c_out[j] = sum_{l <= pivot} lambda^(pivot - l) s_hist[l][j], as the recursion c = lambda c + s.
__global__ void accumulate(const float* __restrict__ s_hist, long long row_stride, int pivot, int n,
                           float lambda, float* __restrict__ c_out) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  float c = 0.f;
  for (int l = 0; l <= pivot; ++l) c = fmaf(lambda, c, s_hist[(size_t)l * row_stride + j]);
  c_out[j] = c;
}

}  // namespace

cudaError_t launch_finalize_rows(const Ctx& ctx, int parts, float* metrics, cudaStream_t st) {
  const int rows_pg_pad = ctx.rows_pad / ctx.cfg.n_kv_heads;
  const int rows_pg = (ctx.cfg.n_q_heads / ctx.cfg.n_kv_heads) * ctx.cfg.window;
  finalize_rows<<<1, kFinalThreads, 0, st>>>(ctx.ws.row_part, parts, ctx.rows_pad, rows_pg_pad,
                                            rows_pg, ctx.rows, ctx.ws.row_lse2, ctx.ws.row_ent,
                                            metrics);
  return cudaGetLastError();
}

cudaError_t launch_reduce_columns(const Ctx& ctx, const float* cols, long long col_stride, int n,
                                  float lambda, float* s_out, float* c_inout, cudaStream_t st) {
  reduce_columns<<<(n + 255) / 256, 256, 0, st>>>(cols, col_stride, ctx.cfg.n_q_heads, n, lambda,
                                                  s_out, c_inout);
  return cudaGetLastError();
}

cudaError_t launch_head_stats(const Ctx& ctx, const float* cols, long long col_stride, int n,
                              float* metrics, cudaStream_t st) {
  int k_rho = n / 10;
  if (k_rho < 1) k_rho = 1;
  head_stats<<<ctx.cfg.n_q_heads, kHsThreads, 0, st>>>(cols, col_stride, n, k_rho,
                                                       ctx.ws.head_part);
  head_stats_final<<<1, 32, 0, st>>>(ctx.ws.head_part, ctx.cfg.n_q_heads, n, metrics);
  return cudaGetLastError();
}

cudaError_t launch_fill_nan_stats(float* metrics, cudaStream_t st) {
  fill_nan_stats<<<1, 1, 0, st>>>(metrics);
  return cudaGetLastError();
}

cudaError_t launch_accumulate(const float* s_hist, long long row_stride, int pivot, int n,
                              float lambda, float* c_out, cudaStream_t st) {
  accumulate<<<(n + 255) / 256, 256, 0, st>>>(s_hist, row_stride, pivot, n, lambda, c_out);
  return cudaGetLastError();
}

}  // namespace skv
