// Row gather / compaction: dst[s, r, :] = src[s, idx[r], :], byte exact.  Rows are split into
// 16-byte (or 4-byte / 1-byte) units; consecutive threads take consecutive units of a row, so
// writes are fully coalesced and reads are coalesced within each gathered row.
#include "common.cuh"

namespace skv {
namespace {

constexpr int kCpThreads = 256;
constexpr int kCpUnroll = 4;

template <typename V>
__global__ void __launch_bounds__(kCpThreads)
gather_rows(const char* __restrict__ src, long long slab_stride, long long row_stride,
            int units_per_row, int n_slabs, int n_rows_src, const int* __restrict__ idx, int n_idx,
            char* __restrict__ dst, int* __restrict__ status) {
  const long long total = (long long)n_slabs * n_idx * units_per_row;
  const long long stride = (long long)gridDim.x * kCpThreads;
  for (long long u0 = (long long)blockIdx.x * kCpThreads + threadIdx.x; u0 < total;
       u0 += stride * kCpUnroll) {
    V val[kCpUnroll];
    bool ok[kCpUnroll];
#pragma unroll
    for (int e = 0; e < kCpUnroll; ++e) {
      const long long u = u0 + e * stride;
      ok[e] = false;
      if (u < total) {
        const long long row = u / units_per_row;           // s * n_idx + r
        const int c = (int)(u - row * units_per_row);
        const int s = (int)(row / n_idx), r = (int)(row - (long long)s * n_idx);
        const int j = __ldg(idx + r);
        if (j >= 0 && j < n_rows_src) {
          val[e] = *reinterpret_cast<const V*>(src + s * slab_stride + j * row_stride +
                                               (long long)c * sizeof(V));
          ok[e] = true;
        } else if (c == 0) {
          atomicCAS(status, 0, (int)STRUCTKV_ERR_INVALID_ARG);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < kCpUnroll; ++e) {
      const long long u = u0 + e * stride;
      if (ok[e]) *reinterpret_cast<V*>(dst + u * (long long)sizeof(V)) = val[e];
    }
  }
}

}  // namespace

cudaError_t launch_compact(const void* src, long long slab_stride, long long row_stride,
                           int row_bytes, int n_slabs, int n_rows_src, const int* idx, int n_idx,
                           void* dst, int* status, int sm_count, cudaStream_t st) {
  if (n_idx == 0 || n_slabs == 0) return cudaSuccess;
  const bool a16 = ((uintptr_t)src % 16 == 0) && ((uintptr_t)dst % 16 == 0) && slab_stride % 16 == 0 &&
                   row_stride % 16 == 0 && row_bytes % 16 == 0;
  const bool a4 = ((uintptr_t)src % 4 == 0) && ((uintptr_t)dst % 4 == 0) && slab_stride % 4 == 0 &&
                  row_stride % 4 == 0 && row_bytes % 4 == 0;
  const int unit = a16 ? 16 : (a4 ? 4 : 1);
  const int upr = row_bytes / unit;
  const long long total = (long long)n_slabs * n_idx * upr;
  long long blocks = (total + (long long)kCpThreads * kCpUnroll - 1) / ((long long)kCpThreads * kCpUnroll);
  const long long cap = (long long)sm_count * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const char* s = (const char*)src;
  char* d = (char*)dst;
  if (unit == 16)
    gather_rows<uint4><<<(int)blocks, kCpThreads, 0, st>>>(s, slab_stride, row_stride, upr, n_slabs,
                                                          n_rows_src, idx, n_idx, d, status);
  else if (unit == 4)
    gather_rows<unsigned><<<(int)blocks, kCpThreads, 0, st>>>(s, slab_stride, row_stride, upr, n_slabs,
                                                             n_rows_src, idx, n_idx, d, status);
  else
    gather_rows<unsigned char><<<(int)blocks, kCpThreads, 0, st>>>(s, slab_stride, row_stride, upr,
                                                                  n_slabs, n_rows_src, idx, n_idx, d, status);
  return cudaGetLastError();
}

}  // namespace skv
