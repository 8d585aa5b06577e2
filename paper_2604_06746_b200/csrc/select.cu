// Budgeted token selection (top-k of the prefix, ties to the lower index, output in position
// order, window appended).  A cluster of kSelCluster CTAs shares one score vector, each CTA
// owning a contiguous slice of the prefix.  Three counting sweeps over order-preserving 32-bit
// keys (11 + 11 + 10 bits) find the k-th largest key exactly: every CTA counts its slice in
// shared memory (each bin kept kSelCopies times so that a warp's hits on one bin spread), the
// counts are merged in CTA 0 through distributed shared memory with integer atomics, and every
// CTA reads the merged counts.  One counting sweep then gives each CTA its output offset and
// one ordered sweep writes the indices.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace skv {
namespace {

constexpr int kSelCluster = 8;
constexpr int kSelThreads = 1024;
constexpr int kSelBins = 2048;
constexpr int kSelCopies = 8;
constexpr int kSelItems = 4;     // consecutive elements per thread in the output sweep
constexpr int kSelBatch = 8;     // loads in flight per thread in the counting sweeps

// Larger float -> larger unsigned; -0 is folded onto +0.
__device__ __forceinline__ unsigned order_key(float v) {
  const unsigned b = __float_as_uint(v + 0.0f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Shared memory (dynamic): hist[kSelBins][kSelCopies] | merged[3][kSelBins] (one per level).
__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads)
select_topk(const float* __restrict__ scores, long long row_stride, int n, int budget, int window,
            int* __restrict__ idx_out) {
  extern __shared__ unsigned sel_smem[];
  unsigned* hist = sel_smem;
  unsigned* merged = sel_smem + kSelBins * kSelCopies;
  __shared__ unsigned warp_tot[33];
  __shared__ unsigned cta_gt[kSelCluster], cta_eq[kSelCluster];
  __shared__ unsigned sel_bin, sel_rem;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int vec = blockIdx.x / kSelCluster;
  const float* s = scores + (size_t)vec * row_stride;
  int* out = idx_out + (size_t)vec * budget;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, copy = tid & (kSelCopies - 1);
  const int prefix_len = n - window;
  const int k = budget - window;

  if (rank == 0)
    for (int i = tid; i < window; i += kSelThreads) out[k + i] = prefix_len + i;
  if (k <= 0) return;                                // the same decision in every CTA of the cluster

  const int per = (prefix_len + kSelCluster - 1) / kSelCluster;
  const int lo = min(prefix_len, rank * per), hi = min(prefix_len, lo + per);
  unsigned* merged0 = cluster.map_shared_rank(merged, 0);
  cluster.sync();                                    // all CTAs of the cluster run before any remote access

  unsigned thr = 0, need_eq = 0xffffffffu;           // threshold key; how many keys equal to it are taken
  const bool keep_all = k >= prefix_len;             // every prefix token is kept
  if (!keep_all) {
    unsigned prefix = 0, prefix_mask = 0, remaining = (unsigned)k;
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
    for (int b = tid; b < 3 * kSelBins; b += kSelThreads) merged[b] = 0;
    cluster.sync();                                  // every merged[] is zero before anyone pushes
    for (int pass = 0; pass < 3; ++pass) {
      for (int b = tid; b < kSelBins * kSelCopies; b += kSelThreads) hist[b] = 0;
      __syncthreads();
      const unsigned bmask = (1u << widths[pass]) - 1u;
      for (int j0 = lo + tid; j0 < hi; j0 += kSelThreads * kSelBatch) {
        float val[kSelBatch];
#pragma unroll
        for (int e = 0; e < kSelBatch; ++e) {
          const int j = j0 + e * kSelThreads;
          val[e] = j < hi ? s[j] : 0.f;
        }
#pragma unroll
        for (int e = 0; e < kSelBatch; ++e) {
          const unsigned u = order_key(val[e]);
          if (j0 + e * kSelThreads < hi && (u & prefix_mask) == prefix)
            atomicAdd(&hist[((u >> shifts[pass]) & bmask) * kSelCopies + copy], 1u);
        }
      }
      __syncthreads();
      unsigned* mlevel = merged + pass * kSelBins;   // bins above 2^width stay zero at the last level
      for (int b = tid; b < kSelBins; b += kSelThreads) {
        unsigned c = 0;
#pragma unroll
        for (int q = 0; q < kSelCopies; ++q) c += hist[b * kSelCopies + q];
        if (c) atomicAdd(&merged0[pass * kSelBins + b], c);
      }
      cluster.sync();
      // copy the cluster-wide counts into this CTA (remote reads in parallel), then pick locally
      if (rank != 0)
        for (int b = tid; b < kSelBins; b += kSelThreads) mlevel[b] = merged0[pass * kSelBins + b];
      __syncthreads();
      block_pick_from_top(mlevel, remaining, warp_tot, &sel_bin, &sel_rem);
      prefix |= sel_bin << shifts[pass];
      prefix_mask |= bmask << shifts[pass];
      remaining = sel_rem;
    }
    thr = prefix;
    need_eq = remaining;
  }

  // keys greater than / equal to the threshold in this CTA's slice -> offsets of the slice
  unsigned my_gt = 0, my_eq = 0;
  for (int j0 = lo + tid; j0 < hi; j0 += kSelThreads * kSelBatch) {
    float val[kSelBatch];
#pragma unroll
    for (int e = 0; e < kSelBatch; ++e) {
      const int j = j0 + e * kSelThreads;
      val[e] = j < hi ? s[j] : 0.f;
    }
#pragma unroll
    for (int e = 0; e < kSelBatch; ++e) {
      const unsigned u = order_key(val[e]);
      const bool in = j0 + e * kSelThreads < hi;
      my_gt += (in && (keep_all || u > thr)) ? 1u : 0u;
      my_eq += (in && !keep_all && u == thr) ? 1u : 0u;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    my_gt += __shfl_xor_sync(0xffffffffu, my_gt, o);
    my_eq += __shfl_xor_sync(0xffffffffu, my_eq, o);
  }
  if (lane == 0) warp_tot[warp] = my_gt;
  __syncthreads();
  unsigned blk_gt = 0;
  for (int wv = 0; wv < kSelThreads / 32; ++wv) blk_gt += warp_tot[wv];
  __syncthreads();
  if (lane == 0) warp_tot[warp] = my_eq;
  __syncthreads();
  unsigned blk_eq = 0;
  for (int wv = 0; wv < kSelThreads / 32; ++wv) blk_eq += warp_tot[wv];
  if (tid == 0) {
    for (int r = 0; r < kSelCluster; ++r) {          // every CTA gets every CTA's totals
      cluster.map_shared_rank(cta_gt, r)[rank] = blk_gt;
      cluster.map_shared_rank(cta_eq, r)[rank] = blk_eq;
    }
  }
  cluster.sync();
  unsigned gt_run = 0, eq_run = 0;
  for (int r = 0; r < rank; ++r) { gt_run += cta_gt[r]; eq_run += cta_eq[r]; }

  // Ordered sweep.  Position of token j in the output =
  //   (#keys > thr before j) + min(#keys == thr before j, need_eq).
  const int chunk = kSelThreads * kSelItems;
  for (int base = lo; base < hi; base += chunk) {
    const int j0 = base + tid * kSelItems;
    unsigned key[kSelItems];
    unsigned packed = 0;                   // (#gt << 16) | #eq among this thread's items
#pragma unroll
    for (int e = 0; e < kSelItems; ++e) {
      const int j = j0 + e;
      const bool in = j < hi;
      key[e] = in ? order_key(s[j]) : 0u;
      if (in) packed += (keep_all || key[e] > thr) ? 0x10000u : ((key[e] == thr) ? 1u : 0u);
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
    const unsigned excl = warp_before + incl - packed;
    unsigned gt_before = gt_run + (excl >> 16), eq_before = eq_run + (excl & 0xffffu);
#pragma unroll
    for (int e = 0; e < kSelItems; ++e) {
      const int j = j0 + e;
      if (j < hi) {
        const bool gt = keep_all || key[e] > thr;
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
  const int smem = (kSelBins * kSelCopies + 3 * kSelBins) * (int)sizeof(unsigned);
  cudaError_t e = cudaFuncSetAttribute(select_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  select_topk<<<batch * kSelCluster, kSelThreads, smem, st>>>(scores, row_stride, n, budget, window,
                                                             idx_out);
  return cudaGetLastError();
}

}  // namespace skv
