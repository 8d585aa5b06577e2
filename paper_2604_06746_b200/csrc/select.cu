// Budgeted token selection (top-k of the prefix, ties to the lower index, output in position
// order, window appended): a three-level radix select over order-preserving 32-bit keys in
// shared-memory histograms, then one ordered compaction sweep.  One block per score vector.
#include "common.cuh"

namespace skv {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelBins = 2048;
constexpr int kSelItems = 4;     // consecutive elements per thread in the output sweep

// Larger float -> larger unsigned; -0 is folded onto +0.
__device__ __forceinline__ unsigned order_key(float v) {
  const unsigned b = __float_as_uint(v + 0.0f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(kSelThreads)
select_topk(const float* __restrict__ scores, long long row_stride, int n, int budget, int window,
            int* __restrict__ idx_out) {
  __shared__ unsigned hist[kSelBins];
  __shared__ unsigned warp_tot[32];
  __shared__ unsigned sel_bin, sel_rem;
  const float* s = scores + (size_t)blockIdx.x * row_stride;
  int* out = idx_out + (size_t)blockIdx.x * budget;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int prefix_len = n - window;
  const int k = budget - window;

  for (int i = tid; i < window; i += kSelThreads) out[k + i] = prefix_len + i;
  if (k <= 0) return;

  unsigned thr = 0, need_eq = 0;           // threshold key; how many keys equal to it are taken
  if (k < prefix_len) {
    unsigned prefix = 0, prefix_mask = 0, remaining = (unsigned)k;
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
    for (int pass = 0; pass < 3; ++pass) {
      for (int b = tid; b < kSelBins; b += kSelThreads) hist[b] = 0;
      __syncthreads();
      const unsigned bmask = (1u << widths[pass]) - 1u;
      for (int base = 0; base < prefix_len; base += kSelThreads) {
        const int j = base + tid;
        const unsigned u = (j < prefix_len) ? order_key(s[j]) : 0u;
        const bool cand = (j < prefix_len) && ((u & prefix_mask) == prefix);
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
    thr = prefix;
    need_eq = remaining;
  } else {
    thr = 0; need_eq = 0xffffffffu;        // k == prefix_len: every prefix token is kept
  }

  // Ordered sweep.  Position of token j in the output =
  //   (#keys > thr before j) + min(#keys == thr before j, need_eq).
  unsigned gt_run = 0, eq_run = 0;
  const int chunk = kSelThreads * kSelItems;
  for (int base = 0; base < prefix_len; base += chunk) {
    const int j0 = base + tid * kSelItems;
    unsigned key[kSelItems];
    unsigned packed = 0;                   // (#gt << 16) | #eq among this thread's items
#pragma unroll
    for (int e = 0; e < kSelItems; ++e) {
      const int j = j0 + e;
      const bool in = j < prefix_len;
      key[e] = in ? order_key(s[j]) : 0u;
      if (in) packed += (key[e] > thr) ? 0x10000u : ((key[e] == thr) ? 1u : 0u);
    }
    if (k >= prefix_len) {                 // keep-all: treat everything as greater
      packed = 0;
#pragma unroll
      for (int e = 0; e < kSelItems; ++e) if (j0 + e < prefix_len) packed += 0x10000u;
    }
    unsigned incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    __syncthreads();                       // warp_tot reuse across chunks
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    unsigned warp_before = 0, chunk_tot = 0;
    for (int wv = 0; wv < kSelThreads / 32; ++wv) {
      const unsigned t = warp_tot[wv];
      if (wv < warp) warp_before += t;
      chunk_tot += t;
    }
    unsigned excl = warp_before + incl - packed;
    unsigned gt_before = gt_run + (excl >> 16), eq_before = eq_run + (excl & 0xffffu);
#pragma unroll
    for (int e = 0; e < kSelItems; ++e) {
      const int j = j0 + e;
      if (j < prefix_len) {
        const bool gt = (k >= prefix_len) || key[e] > thr;
        const bool eq = !gt && key[e] == thr;
        if (gt || (eq && eq_before < need_eq)) {
          const unsigned pos = gt_before + (eq_before < need_eq ? eq_before : need_eq);
          out[pos] = j;
        }
        gt_before += gt ? 1u : 0u;
        eq_before += eq ? 1u : 0u;
      }
    }
    gt_run += chunk_tot >> 16;
    eq_run += chunk_tot & 0xffffu;
  }
}

}  // namespace

cudaError_t launch_select(const float* scores, long long row_stride, int batch, int n, int budget,
                          int window, int* idx_out, cudaStream_t st) {
  select_topk<<<batch, kSelThreads, 0, st>>>(scores, row_stride, n, budget, window, idx_out);
  return cudaGetLastError();
}

}  // namespace skv
