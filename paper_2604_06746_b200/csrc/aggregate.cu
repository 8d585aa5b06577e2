// Block-level aggregation of token scores for block-based KV memory managers, and the
// attention-mass recovery diagnostic.  Both are fixed-order fp32 reductions (deterministic).
#include "common.cuh"

namespace skv {
namespace {

// One thread per block of `block_size` consecutive tokens: S_block_k = sum_{t in block k} score[t].
// The last block of a vector may be ragged.
__global__ void block_scores(const float* __restrict__ scores, long long row_stride, int n,
                             int block_size, int n_blocks, int vec4, float* __restrict__ out) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n_blocks) return;
  const float* s = scores + (size_t)blockIdx.y * row_stride;
  const int lo = k * block_size, hi = min(n, lo + block_size);
  float acc = 0.f;
  if (vec4 && hi - lo == block_size) {                   // whole block, 16-byte loads, same token order
    const float4* s4 = reinterpret_cast<const float4*>(s + lo);
#pragma unroll 4
    for (int q = 0; q < block_size / 4; ++q) {
      const float4 v = s4[q];
      acc += v.x; acc += v.y; acc += v.z; acc += v.w;
    }
  } else {
    for (int t = lo; t < hi; ++t) acc += s[t];
  }
  out[(size_t)blockIdx.y * n_blocks + k] = acc;
}

// out[g][j] = sum of the pooled attention of the `group` query heads that share KV head g, heads
// in ascending order.
__global__ void group_saliency(const float* __restrict__ head_cols, long long col_stride, int group, int n,
                               float* __restrict__ out) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const int g = blockIdx.y;
  float acc = 0.f;
  for (int q = 0; q < group; ++q) acc += head_cols[(size_t)(g * group + q) * col_stride + j];
  out[(size_t)g * n + j] = acc;
}

constexpr int kMrThreads = 1024;

__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float x = red[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    if (lane == 0) red[32] = x;
  }
  __syncthreads();
  return red[32];
}

// One block per score vector: out = (sum of the scores at idx) / (sum of all scores).
// An index outside [0, n) contributes nothing and is recorded in the status word.
__global__ void __launch_bounds__(kMrThreads)
mass_recovery(const float* __restrict__ scores, long long row_stride, int n, const int* __restrict__ idx,
              int n_idx, float* __restrict__ out, int* __restrict__ status) {
  __shared__ float red[33];
  const float* s = scores + (size_t)blockIdx.x * row_stride;
  float kept = 0.f, total = 0.f;
  for (int r = threadIdx.x; r < n_idx; r += kMrThreads) {
    const int j = idx[r];
    if (j >= 0 && j < n) kept += s[j];
    else atomicCAS(status, 0, (int)STRUCTKV_ERR_INVALID_ARG);
  }
  for (int j = threadIdx.x; j < n; j += kMrThreads) total += s[j];
  const float k = block_sum(kept, red);
  const float t = block_sum(total, red);
  if (threadIdx.x == 0) out[blockIdx.x] = k / t;
}

}  // namespace

cudaError_t launch_block_scores(const float* scores, long long row_stride, int batch, int n, int block_size,
                                float* out, cudaStream_t st) {
  const int n_blocks = (n + block_size - 1) / block_size;
  const int vec4 = (block_size % 4 == 0) && ((uintptr_t)scores % 16 == 0) && (batch == 1 || row_stride % 4 == 0);
  block_scores<<<dim3((n_blocks + 127) / 128, batch), 128, 0, st>>>(scores, row_stride, n, block_size, n_blocks,
                                                                    vec4, out);
  return cudaGetLastError();
}

cudaError_t launch_group_saliency(const float* head_cols, long long col_stride, int n_heads, int group, int n,
                                  float* out, cudaStream_t st) {
  group_saliency<<<dim3((n + 255) / 256, n_heads / group), 256, 0, st>>>(head_cols, col_stride, group, n, out);
  return cudaGetLastError();
}

cudaError_t launch_mass_recovery(const float* scores, long long row_stride, int batch, int n, const int* idx,
                                 int n_idx, float* out, int* status, cudaStream_t st) {
  mass_recovery<<<batch, kMrThreads, 0, st>>>(scores, row_stride, n, idx, n_idx, out, status);
  return cudaGetLastError();
}

}  // namespace skv
