// Row gather / compaction: dst[s, r, :] = src[s, idx[r], :], byte exact.  Rows are split into
// 16-byte (or 4-byte / 1-byte) units; consecutive threads take consecutive units of a row, so
// writes are fully coalesced and reads are coalesced within each gathered row.  Two loads in
// flight per thread and up to 64 resident blocks per SM measured best on B200 (more unrolling
// or fewer, fatter blocks lose 10-25 % of the copy bandwidth).
#include "common.cuh"

namespace skv {
namespace {

#ifndef SKV_CP_THREADS
#define SKV_CP_THREADS 256
#endif
#ifndef SKV_CP_UNROLL
#define SKV_CP_UNROLL 2
#endif
#ifndef SKV_CP_BLOCKS_PER_SM
#define SKV_CP_BLOCKS_PER_SM 64
#endif
constexpr int kCpThreads = SKV_CP_THREADS;
constexpr int kCpUnroll = SKV_CP_UNROLL;

// Rows are read once and written once: loads bypass L1 allocation, stores are streaming.
template <typename V> __device__ __forceinline__ V ld_stream(const V* p) { return *p; }
template <typename V> __device__ __forceinline__ void st_stream(V* p, const V& v) { *p = v; }
#ifndef SKV_CP_PLAIN
template <> __device__ __forceinline__ uint4 ld_stream<uint4>(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
template <> __device__ __forceinline__ void st_stream<uint4>(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
#endif

template <typename V>
__global__ void __launch_bounds__(kCpThreads)
gather_rows(const char* __restrict__ src, long long slab_stride, long long row_stride,
            int units_per_row, int n_slabs, int n_rows_src, const int* __restrict__ idx,
            long long idx_slab_stride, int n_idx,
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
        const int j = __ldg(idx + s * idx_slab_stride + r);   // stride 0: one list for every slab
        if (j >= 0 && j < n_rows_src) {
          val[e] = ld_stream(reinterpret_cast<const V*>(src + s * slab_stride + j * row_stride +
                                                        (long long)c * sizeof(V)));
          ok[e] = true;
        } else if (c == 0) {
          atomicCAS(status, 0, (int)STRUCTKV_ERR_INVALID_ARG);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < kCpUnroll; ++e) {
      const long long u = u0 + e * stride;
      if (ok[e]) st_stream(reinterpret_cast<V*>(dst + u * (long long)sizeof(V)), val[e]);
    }
  }
}

// The same gather for several layers in one launch: layer blockIdx.y reads its own source (the
// pointers travel as a kernel argument), its own index list and writes its own slab of dst.
struct LayerPtrs { const char* src[kMaxGatherLayers]; };

template <typename V>
__global__ void __launch_bounds__(kCpThreads)
gather_rows_layers(const __grid_constant__ LayerPtrs srcs, long long slab_stride, long long row_stride,
                   int units_per_row, int n_slabs, int n_rows_src, const int* __restrict__ idx,
                   long long idx_layer_stride, int n_idx, char* __restrict__ dst, long long dst_layer_stride,
                   int* __restrict__ status) {
  const int layer = blockIdx.y;
  const char* __restrict__ src = srcs.src[layer];
  const int* __restrict__ my_idx = idx + (long long)layer * idx_layer_stride;
  char* __restrict__ my_dst = dst + (long long)layer * dst_layer_stride;
  const long long total = (long long)n_slabs * n_idx * units_per_row;
  const long long stride = (long long)gridDim.x * kCpThreads;
  for (long long u0 = (long long)blockIdx.x * kCpThreads + threadIdx.x; u0 < total; u0 += stride * kCpUnroll) {
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
        const int j = __ldg(my_idx + r);
        if (j >= 0 && j < n_rows_src) {
          val[e] = ld_stream(reinterpret_cast<const V*>(src + s * slab_stride + j * row_stride +
                                                        (long long)c * sizeof(V)));
          ok[e] = true;
        } else if (c == 0) {
          atomicCAS(status, 0, (int)STRUCTKV_ERR_INVALID_ARG);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < kCpUnroll; ++e) {
      const long long u = u0 + e * stride;
      if (ok[e]) st_stream(reinterpret_cast<V*>(my_dst + u * (long long)sizeof(V)), val[e]);
    }
  }
}

}  // namespace

cudaError_t launch_compact_layers(const void* const* srcs, int n_layers, long long slab_stride, long long row_stride,
                                  int row_bytes, int n_slabs, int n_rows_src, const int* idx,
                                  long long idx_layer_stride, int n_idx, void* dst, long long dst_layer_stride,
                                  int* status, int sm_count, cudaStream_t st) {
  if (n_idx == 0 || n_slabs == 0 || n_layers == 0) return cudaSuccess;
  LayerPtrs lp;
  bool a16 = ((uintptr_t)dst % 16 == 0) && slab_stride % 16 == 0 && row_stride % 16 == 0 && row_bytes % 16 == 0 &&
             dst_layer_stride % 16 == 0;
  bool a4 = ((uintptr_t)dst % 4 == 0) && slab_stride % 4 == 0 && row_stride % 4 == 0 && row_bytes % 4 == 0 &&
            dst_layer_stride % 4 == 0;
  for (int l = 0; l < n_layers; ++l) {
    lp.src[l] = (const char*)srcs[l];
    a16 = a16 && ((uintptr_t)srcs[l] % 16 == 0);
    a4 = a4 && ((uintptr_t)srcs[l] % 4 == 0);
  }
  const int unit = a16 ? 16 : (a4 ? 4 : 1);
  const int upr = row_bytes / unit;
  const long long total = (long long)n_slabs * n_idx * upr;
  long long blocks = (total + (long long)kCpThreads * kCpUnroll - 1) / ((long long)kCpThreads * kCpUnroll);
  const long long cap = ((long long)sm_count * SKV_CP_BLOCKS_PER_SM + n_layers - 1) / n_layers;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const dim3 grid((unsigned)blocks, (unsigned)n_layers);
  char* d = (char*)dst;
  if (unit == 16)
    gather_rows_layers<uint4><<<grid, kCpThreads, 0, st>>>(lp, slab_stride, row_stride, upr, n_slabs, n_rows_src, idx,
                                                          idx_layer_stride, n_idx, d, dst_layer_stride, status);
  else if (unit == 4)
    gather_rows_layers<unsigned><<<grid, kCpThreads, 0, st>>>(lp, slab_stride, row_stride, upr, n_slabs, n_rows_src,
                                                             idx, idx_layer_stride, n_idx, d, dst_layer_stride, status);
  else
    gather_rows_layers<unsigned char><<<grid, kCpThreads, 0, st>>>(lp, slab_stride, row_stride, upr, n_slabs,
                                                                  n_rows_src, idx, idx_layer_stride, n_idx, d,
                                                                  dst_layer_stride, status);
  return cudaGetLastError();
}

cudaError_t launch_compact(const void* src, long long slab_stride, long long row_stride,
                           int row_bytes, int n_slabs, int n_rows_src, const int* idx,
                           long long idx_slab_stride, int n_idx, void* dst, int* status, int sm_count,
                           cudaStream_t st) {
  if (n_idx == 0 || n_slabs == 0) return cudaSuccess;
  const bool a16 = ((uintptr_t)src % 16 == 0) && ((uintptr_t)dst % 16 == 0) && slab_stride % 16 == 0 &&
                   row_stride % 16 == 0 && row_bytes % 16 == 0;
  const bool a4 = ((uintptr_t)src % 4 == 0) && ((uintptr_t)dst % 4 == 0) && slab_stride % 4 == 0 &&
                  row_stride % 4 == 0 && row_bytes % 4 == 0;
  const int unit = a16 ? 16 : (a4 ? 4 : 1);
  const int upr = row_bytes / unit;
  const long long total = (long long)n_slabs * n_idx * upr;
  long long blocks = (total + (long long)kCpThreads * kCpUnroll - 1) / ((long long)kCpThreads * kCpUnroll);
  const long long cap = (long long)sm_count * SKV_CP_BLOCKS_PER_SM;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const char* s = (const char*)src;
  char* d = (char*)dst;
  if (unit == 16)
    gather_rows<uint4><<<(int)blocks, kCpThreads, 0, st>>>(s, slab_stride, row_stride, upr, n_slabs,
                                                          n_rows_src, idx, idx_slab_stride, n_idx, d, status);
  else if (unit == 4)
    gather_rows<unsigned><<<(int)blocks, kCpThreads, 0, st>>>(s, slab_stride, row_stride, upr, n_slabs,
                                                             n_rows_src, idx, idx_slab_stride, n_idx, d, status);
  else
    gather_rows<unsigned char><<<(int)blocks, kCpThreads, 0, st>>>(s, slab_stride, row_stride, upr,
                                                                  n_slabs, n_rows_src, idx, idx_slab_stride, n_idx, d, status);
  return cudaGetLastError();
}

}  // namespace skv
