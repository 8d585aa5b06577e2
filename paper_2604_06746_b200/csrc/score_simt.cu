// CUDA-core two-pass scorer: window logits, row softmax statistics (pass 1) and pooled
// per-head attention columns (pass 2).  Serves fp32 storage and any shape the tensor-core
// scorer does not take.  Everything is fp32 arithmetic in the log2 domain.
//
// Row numbering (shared with the tensor-core scorer and the finalize kernel): score row
// (h, i) of KV group g = h / G lives at  g * rows_per_group_pad + (h % G) * w + i.
#include "common.cuh"

namespace skv {
namespace {

constexpr int kP1Keys = 64;      // keys per pass-1 chunk
constexpr int kP1Threads = 256;
constexpr int kP2Threads = 128;  // one key per thread in pass 2

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Pass 1.  grid = (parts, H).  Each block sweeps its key segment in chunks of kP1Keys keys;
// a warp owns window rows i = warp, warp + 8, ... and its lanes own the keys of the chunk.
// Per row it keeps (m2, Z, U): running max of x = logit*log2e, Z = sum 2^(x-m2),
// U = sum 2^(x-m2) (x-m2).
template <typename T, int D>
__global__ void __launch_bounds__(kP1Threads)
simt_pass1(const T* __restrict__ q, const T* __restrict__ k, long long sh, long long st, int N,
           int w, int G, float c2, int parts, int rows_pg_pad, int rows_pad,
           float4* __restrict__ row_part) {
  extern __shared__ float smem[];
  float* qs = smem;                         // [w][D]
  float* ks = qs + (size_t)w * D;           // [kP1Keys][D + 1]
  float* sm = ks + kP1Keys * (D + 1);       // [w] m2
  float* sz = sm + w;                       // [w] Z
  float* su = sz + w;                       // [w] U
  const int h = blockIdx.y, g = h / G, part = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int x = tid; x < w * D; x += kP1Threads) qs[x] = to_f32<T>(q[(size_t)h * w * D + x]);
  for (int x = tid; x < w; x += kP1Threads) { sm[x] = -INFINITY; sz[x] = 0.f; su[x] = 0.f; }

  const int n_chunks = (N + kP1Keys - 1) / kP1Keys;
  const int c_lo = (int)((long long)part * n_chunks / parts);
  const int c_hi = (int)((long long)(part + 1) * n_chunks / parts);
  const T* kg = k + (size_t)g * sh;

  for (int c = c_lo; c < c_hi; ++c) {
    const int j0 = c * kP1Keys;
    __syncthreads();
    for (int x = tid; x < kP1Keys * D; x += kP1Threads) {
      const int key = x / D, col = x - key * D, j = j0 + key;
      ks[key * (D + 1) + col] = (j < N) ? to_f32<T>(kg[(size_t)j * st + col]) : 0.f;
    }
    __syncthreads();
    for (int i = warp; i < w; i += kP1Threads / 32) {
      const int t = N - w + i;
      const float* qi = qs + (size_t)i * D;
      float xs[kP1Keys / 32];
      float mx = -INFINITY;
#pragma unroll
      for (int kk = 0; kk < kP1Keys / 32; ++kk) {
        const int key = lane + 32 * kk;
        const float* kr = ks + key * (D + 1);
        float s = 0.f;
#pragma unroll 8
        for (int col = 0; col < D; ++col) s = fmaf(qi[col], kr[col], s);
        xs[kk] = (j0 + key <= t) ? s * c2 : -INFINITY;
        mx = fmaxf(mx, xs[kk]);
      }
      mx = warp_max(mx);
      if (mx == -INFINITY) continue;        // the whole chunk is masked for this row
      const float m_old = sm[i];
      const float m_new = fmaxf(m_old, mx);
      float zs = 0.f, us = 0.f;
#pragma unroll
      for (int kk = 0; kk < kP1Keys / 32; ++kk) {
        if (xs[kk] != -INFINITY) {
          const float dx = xs[kk] - m_new;
          const float p = fast_exp2(dx);
          zs += p;
          us = fmaf(p, dx, us);
        }
      }
      zs = warp_sum(zs);
      us = warp_sum(us);
      if (lane == 0) {
        float Z = sz[i], U = su[i];
        if (m_old != -INFINITY) {
          const float dm = m_old - m_new, f = fast_exp2(dm);
          U = f * fmaf(dm, Z, U);
          Z = f * Z;
        }
        sm[i] = m_new; sz[i] = Z + zs; su[i] = U + us;
      }
      __syncwarp();
    }
  }
  __syncthreads();
  for (int i = tid; i < w; i += kP1Threads) {
    const int r = g * rows_pg_pad + (h % G) * w + i;
    row_part[(size_t)part * rows_pad + r] = make_float4(sm[i], sz[i], su[i], 0.f);
  }
}

// Pass 2.  grid = (ceil(N / 128), H); thread = key.  cols[h][j] = (1/w) sum_i 2^(x_ij - lse2_i).
template <typename T, int D>
__global__ void __launch_bounds__(kP2Threads)
simt_pass2(const T* __restrict__ q, const T* __restrict__ k, long long sh, long long st, int N,
           int w, int G, float c2, int rows_pg_pad, const float* __restrict__ row_lse2,
           float* __restrict__ cols, long long col_stride) {
  extern __shared__ float smem[];
  float* qs = smem;                         // [w][D]
  float* ls = qs + (size_t)w * D;           // [w]
  const int h = blockIdx.y, g = h / G, tid = threadIdx.x;
  for (int x = tid; x < w * D; x += kP2Threads) qs[x] = to_f32<T>(q[(size_t)h * w * D + x]);
  for (int x = tid; x < w; x += kP2Threads) ls[x] = row_lse2[g * rows_pg_pad + (h % G) * w + x];
  __syncthreads();
  const int j = blockIdx.x * kP2Threads + tid;
  if (j >= N) return;
  float kr[D];
  const T* kp = k + (size_t)g * sh + (size_t)j * st;
#pragma unroll
  for (int col = 0; col < D; ++col) kr[col] = to_f32<T>(kp[col]);
  float acc = 0.f;
  const int i_first = max(0, j - (N - w));   // rows i < i_first do not see key j
  for (int i = i_first; i < w; ++i) {
    const float4* qi = reinterpret_cast<const float4*>(qs + (size_t)i * D);
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int c4 = 0; c4 < D / 4; c4 += 2) {
      const float4 a = qi[c4], b = qi[c4 + 1];
      s0 = fmaf(a.x, kr[4 * c4 + 0], s0); s0 = fmaf(a.y, kr[4 * c4 + 1], s0);
      s0 = fmaf(a.z, kr[4 * c4 + 2], s0); s0 = fmaf(a.w, kr[4 * c4 + 3], s0);
      s1 = fmaf(b.x, kr[4 * c4 + 4], s1); s1 = fmaf(b.y, kr[4 * c4 + 5], s1);
      s1 = fmaf(b.z, kr[4 * c4 + 6], s1); s1 = fmaf(b.w, kr[4 * c4 + 7], s1);
    }
    acc += fast_exp2(fmaf(s0 + s1, c2, -ls[i]));
  }
  cols[(size_t)h * col_stride + j] = acc / (float)w;
}

template <typename T, int D>
cudaError_t launch_typed(const Ctx& ctx, const ScoreArgs& a, int* parts_out, int pass,
                         cudaStream_t st) {
  const int H = ctx.cfg.n_q_heads, G = H / ctx.cfg.n_kv_heads, w = ctx.cfg.window;
  const int N = a.n_keys;
  const int rows_pg_pad = ctx.rows_pad / ctx.cfg.n_kv_heads;
  const float c2 = a.scale * kLog2e;
  if (pass == 1) {
    const int n_chunks = (N + kP1Keys - 1) / kP1Keys;
    int parts = n_chunks < 64 ? n_chunks : 64;
    *parts_out = parts;
    const size_t smem = ((size_t)w * D + kP1Keys * (D + 1) + 3 * (size_t)w) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(simt_pass1<T, D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    simt_pass1<T, D><<<dim3(parts, H), kP1Threads, smem, st>>>(
        (const T*)a.q, (const T*)a.k, a.k_stride_head, a.k_stride_token, N, w, G, c2, parts,
        rows_pg_pad, ctx.rows_pad, ctx.ws.row_part);
  } else {
    const size_t smem = ((size_t)w * D + (size_t)w) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(simt_pass2<T, D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    simt_pass2<T, D><<<dim3((N + kP2Threads - 1) / kP2Threads, H), kP2Threads, smem, st>>>(
        (const T*)a.q, (const T*)a.k, a.k_stride_head, a.k_stride_token, N, w, G, c2,
        rows_pg_pad, ctx.ws.row_lse2, a.cols, a.col_stride);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_simt(const Ctx& ctx, const ScoreArgs& a, int* parts_out, int pass,
                              cudaStream_t st) {
  const bool f32 = ctx.cfg.dtype == STRUCTKV_FP32;
  const int d = ctx.cfg.head_dim;
  if (f32 && d == 64) return launch_typed<float, 64>(ctx, a, parts_out, pass, st);
  if (f32 && d == 128) return launch_typed<float, 128>(ctx, a, parts_out, pass, st);
  if (!f32 && d == 64) return launch_typed<__nv_bfloat16, 64>(ctx, a, parts_out, pass, st);
  if (!f32 && d == 128) return launch_typed<__nv_bfloat16, 128>(ctx, a, parts_out, pass, st);
  return cudaErrorInvalidValue;
}

}  // namespace skv
