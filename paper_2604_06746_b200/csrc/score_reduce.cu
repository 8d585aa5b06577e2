// Small deterministic reductions around the scorers: row finalisation (log-sum-exp, entropy),
// column reduction over heads with the centrality update, per-head sparsity / variance, and
// the closed-form centrality re-accumulation.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace skv {
namespace {

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

// One thread per score row.  Row r of group g is valid iff its index inside the group is
// < rows_pg.  Each of the `parts` key segments left (ref, Z, U) for the row: Z = sum 2^(x - ref),
// U = sum 2^(x - ref) (x - ref), x = logit * log2(e); ref is any reference the segment chose.
// With l_p = ref_p + log2 Z_p (the segment's log-sum-exp) and M = max_p l_p:
//   lse2 = M + log2 sum_p 2^(l_p - M)
//   mean of (x - M) under the row's softmax = sum_p 2^(l_p - M) (ref_p - M + U_p / Z_p) / sum_p 2^(l_p - M)
//   entropy = ln2 * (lse2 - M - that mean)                                   (Eq. 4, one row)
__global__ void __launch_bounds__(256)
finalize_rows(const float4* __restrict__ row_part, int parts, int rows_pad, int rows_pg_pad,
              int rows_pg, float* __restrict__ row_lse2, float* __restrict__ row_ent) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows_pad) return;
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
}

// S_j = sum over heads (fixed order) of cols[h][j];  C_j <- lambda C_j + S_j  (Eq. 2, Eq. 3).
// Four keys per thread where the layout allows 16-byte accesses.  NOTE: the order in which heads
// are added differs between the two instantiations (grouped vs. sequential).  Block 0 also finishes the
// layer's metrics: metrics[0] = mean entropy of the valid score rows (Eq. 4); metrics[1] = mean
// over heads of the top-mass (Eq. 5), metrics[2] = mean over heads of (sum of squared deviations
// from 1/n) / n (Eq. 6), both from head_part, or NaN when head statistics are not computed here.
// Fixed summation order throughout.
constexpr int kRcThreads = 256;
template <int VEC>
__global__ void __launch_bounds__(kRcThreads)
reduce_finish(const float* __restrict__ cols, long long col_stride, int H, int n, float lambda,
              float* __restrict__ s_out, float* __restrict__ c_inout, const float* __restrict__ row_ent,
              int rows_pad, int rows_pg_pad, int rows_pg, int n_valid, const float* __restrict__ head_part,
              int with_head_stats, float* __restrict__ metrics) {
  __shared__ float red[33];
  pdl_trigger();
  pdl_wait();
  if (VEC == 4) {
    // 64 threads along the keys (four keys each) x 4 groups of heads: four times the loads in
    // flight; the groups' partial sums are added in group order (fixed order, deterministic)
    __shared__ float4 part[3][64];
    const int lane_j = threadIdx.x & 63, grp = threadIdx.x >> 6;
    const int j4 = (blockIdx.x * 64 + lane_j) * 4;
    const int h_per = (H + 3) / 4, h_lo = grp * h_per, h_hi = min(H, h_lo + h_per);
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j4 < n) {                                  // n is a multiple of 4 in this instantiation
#pragma unroll 4
      for (int h = h_lo; h < h_hi; ++h) {
        const float4 v = *reinterpret_cast<const float4*>(cols + (size_t)h * col_stride + j4);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      }
    }
    if (grp > 0) part[grp - 1][lane_j] = s;
    __syncthreads();
    if (grp == 0 && j4 < n) {
#pragma unroll
      for (int k = 0; k < 3; ++k) {
        const float4 o = part[k][lane_j];
        s.x += o.x; s.y += o.y; s.z += o.z; s.w += o.w;
      }
      *reinterpret_cast<float4*>(s_out + j4) = s;
      if (c_inout) {
        float4 c = *reinterpret_cast<const float4*>(c_inout + j4);
        c.x = fmaf(lambda, c.x, s.x); c.y = fmaf(lambda, c.y, s.y);
        c.z = fmaf(lambda, c.z, s.z); c.w = fmaf(lambda, c.w, s.w);
        *reinterpret_cast<float4*>(c_inout + j4) = c;
      }
    }
  } else if (blockIdx.x * kRcThreads + threadIdx.x < n) {
    const int j = blockIdx.x * kRcThreads + threadIdx.x;
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += cols[(size_t)h * col_stride + j];
    s_out[j] = s;
    if (c_inout) c_inout[j] = fmaf(lambda, c_inout[j], s);
  }
  if (blockIdx.x != 0) return;
  float ent = 0.f;
  for (int r = threadIdx.x; r < rows_pad; r += kRcThreads)
    if ((r % rows_pg_pad) < rows_pg) ent += row_ent[r];
  const float tot = block_sum_1024(ent, red);
  if (threadIdx.x != 0) return;
  metrics[0] = tot / (float)n_valid;
  if (!with_head_stats) {
    metrics[1] = __int_as_float(0x7fc00000);
    metrics[2] = __int_as_float(0x7fc00000);
    return;
  }
  float rho = 0.f, var = 0.f;
  const float inv_n = 1.f / (float)n;
  for (int h = 0; h < H; ++h) {
    rho += head_part[h * 4 + 1];
    var += head_part[h * 4 + 0] * inv_n;
  }
  metrics[1] = rho / (float)H;
  metrics[2] = var / (float)H;
}

// reduce_finish for several layers at once (the layers' scorer passes have all run): per layer l
// S^(l) = sum over heads, in reduce_finish's order, C <- lambda C + S^(l) carried in registers from
// layer to layer, and, in block l, the layer's entropy; sparsity and variance are left as NaN
// (they come from head_stats).  Every bit equals what a chain of reduce_finish launches gives.
template <int VEC>
__global__ void __launch_bounds__(kRcThreads)
reduce_layers(const float* __restrict__ cols, long long layer_stride, long long col_stride, int H, int n,
              int n_layers, float lambda, float* __restrict__ s_out, long long s_stride,
              float* __restrict__ c_inout, const float* __restrict__ row_ent, int rows_pad, int rows_pg_pad,
              int rows_pg, int n_valid, float* __restrict__ metrics) {
  __shared__ float red[33];
  pdl_trigger();
  pdl_wait();
  if (VEC == 4) {
    __shared__ float4 part[3][64];
    const int lane_j = threadIdx.x & 63, grp = threadIdx.x >> 6;
    const int j4 = (blockIdx.x * 64 + lane_j) * 4;
    const int h_per = (H + 3) / 4, h_lo = grp * h_per, h_hi = min(H, h_lo + h_per);
    float4 c = make_float4(0.f, 0.f, 0.f, 0.f);
    if (grp == 0 && j4 < n && c_inout) c = *reinterpret_cast<const float4*>(c_inout + j4);
    for (int l = 0; l < n_layers; ++l) {
      const float* cl = cols + (size_t)l * layer_stride;
      float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
      if (j4 < n) {
#pragma unroll 4
        for (int h = h_lo; h < h_hi; ++h) {
          const float4 v = *reinterpret_cast<const float4*>(cl + (size_t)h * col_stride + j4);
          s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
      }
      if (grp > 0) part[grp - 1][lane_j] = s;
      __syncthreads();
      if (grp == 0 && j4 < n) {
#pragma unroll
        for (int k = 0; k < 3; ++k) {
          const float4 o = part[k][lane_j];
          s.x += o.x; s.y += o.y; s.z += o.z; s.w += o.w;
        }
        *reinterpret_cast<float4*>(s_out + (size_t)l * s_stride + j4) = s;
        c.x = fmaf(lambda, c.x, s.x); c.y = fmaf(lambda, c.y, s.y);
        c.z = fmaf(lambda, c.z, s.z); c.w = fmaf(lambda, c.w, s.w);
      }
      __syncthreads();                               // part[] is reused by the next layer
    }
    if (grp == 0 && j4 < n && c_inout) *reinterpret_cast<float4*>(c_inout + j4) = c;
  } else if (blockIdx.x * kRcThreads + threadIdx.x < n) {
    const int j = blockIdx.x * kRcThreads + threadIdx.x;
    float c = c_inout ? c_inout[j] : 0.f;
    for (int l = 0; l < n_layers; ++l) {
      const float* cl = cols + (size_t)l * layer_stride;
      float s = 0.f;
      for (int h = 0; h < H; ++h) s += cl[(size_t)h * col_stride + j];
      s_out[(size_t)l * s_stride + j] = s;
      c = fmaf(lambda, c, s);
    }
    if (c_inout) c_inout[j] = c;
  }
  // blocks walk over the layers for the entropies (there may be fewer blocks than layers)
  for (int l = blockIdx.x; l < n_layers; l += gridDim.x) {
    float ent = 0.f;
    for (int r = threadIdx.x; r < rows_pad; r += kRcThreads)
      if ((r % rows_pg_pad) < rows_pg) ent += row_ent[(size_t)l * rows_pad + r];
    const float tot = block_sum_1024(ent, red);
    if (threadIdx.x == 0) {
      metrics[l * 3 + 0] = tot / (float)n_valid;
      metrics[l * 3 + 1] = __int_as_float(0x7fc00000);
      metrics[l * 3 + 2] = __int_as_float(0x7fc00000);
    }
    __syncthreads();
  }
}

// Per head: sum of squared deviations from 1/n (Eq. 6: the pooled vector sums to 1, so 1/n is its
// mean; summing deviations instead of squares keeps near-uniform attention from cancelling) and
// the mass of the k_rho largest entries (Eq. 5) of the pooled attention vector.  A cluster of
// CL CTAs shares one head; each CTA owns a slice of the keys.  All entries are >= 0, so the
// unsigned order of the fp32 bit patterns is the order of the values.  Two counting sweeps locate the k_rho-th largest value to 22 bits
// (histograms are merged in CTA 0 of the cluster through distributed shared memory with
// integer atomics, so the result does not depend on arrival order):
//   sweep 1: histogram of bits 30..20 (exponent + 3 mantissa bits); sum of squared deviations
//   sweep 2: exact sum of the entries above the threshold bin (fixed order) and a histogram of
//            bits 19..9 of the entries inside it
// The entries inside the threshold bin are then summed as count x bin midpoint: bins of the
// second level are 2^-14 wide relative to their value, far inside the metric's tolerance.
constexpr int kHsCluster = 8;      // CTAs per (layer, head) when few vectors are in flight (one layer at a time)
constexpr int kHsThreads = 1024;
constexpr int kHsBins = 2048;
// each bin is kept several times (lane & (copies - 1)) so that a warp's hits on one bin spread: 8 copies
// where a cluster shares a vector (two CTAs per SM), 16 where one CTA sweeps a whole vector (a lane
// then shares its banks with one other lane only)
__host__ __device__ constexpr int hs_copies(int cl) { return cl == 1 ? 16 : 8; }
constexpr int kHsItems = 16;      // entries per thread kept in registers between the sweeps

// Applies f to a[lo .. hi) once each, kHsThreads threads together: 16-byte loads, four of them in
// flight per thread, scalar accesses only for the unaligned ends.  The order in which a thread
// meets its entries is fixed.
template <class F>
__device__ __forceinline__ void sweep_from_memory(const float* __restrict__ a, int lo, int hi, int tid, F f) {
  const int mis = (int)((reinterpret_cast<uintptr_t>(a + lo) >> 2) & 3u);
  const int n_head = min(hi - lo, (4 - mis) & 3);
  if (tid < n_head) f(a[lo + tid]);
  const int b0 = lo + n_head;
  const int n4 = (hi - b0) >> 2;
  const float4* a4 = reinterpret_cast<const float4*>(a + b0);
  int i = tid;
  for (; i + 3 * kHsThreads < n4; i += 4 * kHsThreads) {
    const float4 v0 = a4[i], v1 = a4[i + kHsThreads], v2 = a4[i + 2 * kHsThreads], v3 = a4[i + 3 * kHsThreads];
    f(v0.x); f(v0.y); f(v0.z); f(v0.w);
    f(v1.x); f(v1.y); f(v1.z); f(v1.w);
    f(v2.x); f(v2.y); f(v2.z); f(v2.w);
    f(v3.x); f(v3.y); f(v3.z); f(v3.w);
  }
  for (; i < n4; i += kHsThreads) {
    const float4 v = a4[i];
    f(v.x); f(v.y); f(v.z); f(v.w);
  }
  const int t0 = b0 + 4 * n4;
  if (t0 + tid < hi) f(a[t0 + tid]);
}

// Shared memory of head_stats: hist[kHsBins][copies] | merged[2][kHsBins] (dynamic, 80 or 144 KB).
template <int CL>     // CTAs that share one (layer, head) vector: kHsCluster, or 1 when a batch of layers fills the GPU
__global__ void __launch_bounds__(kHsThreads)
head_stats(const float* __restrict__ cols, long long layer_stride, long long col_stride, int H, int n,
           int k_rho, float* __restrict__ head_part) {
  extern __shared__ unsigned hs_smem[];
  constexpr int kHsCopies = hs_copies(CL);
  unsigned* hist = hs_smem;                          // this CTA's counts, kHsCopies per bin
  unsigned* merged = hs_smem + kHsBins * kHsCopies;  // cluster-wide counts of the two levels (CTA 0's copy counts)
  __shared__ float red[33];
  __shared__ unsigned scan_tmp[33];
  __shared__ float slots[2 * kHsCluster];            // CTA 0: per-CTA {sum of squared deviations, mass above}
  __shared__ unsigned sel_bin, sel_rem;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.x / CL;                  // (layer, head) pair: one cluster each
  const float* a = cols + (size_t)(head / H) * layer_stride + (size_t)(head % H) * col_stride;
  const int tid = threadIdx.x, copy = tid & (kHsCopies - 1);
  const int per = (n + CL - 1) / CL;
  const int lo = rank * per, hi = min(n, lo + per);
  const bool in_regs = per <= kHsItems * kHsThreads;  // otherwise the second sweep reads memory again
  unsigned* merged0 = cluster.map_shared_rank(merged, 0);

  auto clear_local = [&]() {
    for (int b = tid; b < kHsBins * kHsCopies; b += kHsThreads) hist[b] = 0;
  };
  auto push = [&](int level) {                       // this CTA's counts into CTA 0's merged[level]
    for (int b = tid; b < kHsBins; b += kHsThreads) {
      unsigned c = 0;
#pragma unroll
      for (int k = 0; k < kHsCopies; ++k) c += hist[b * kHsCopies + ((k + tid) & (kHsCopies - 1))];   // rotated: no bank conflicts
      if (c) atomicAdd(&merged0[level * kHsBins + b], c);
    }
  };

  pdl_trigger();
  clear_local();
  for (int b = tid; b < 2 * kHsBins; b += kHsThreads) merged[b] = 0;
  pdl_wait();                                        // the pooled columns come from the kernels before
  float reg[kHsItems];
#pragma unroll
  for (int e = 0; e < kHsItems; ++e) {
    const int j = lo + e * kHsThreads + tid;
    reg[e] = (in_regs && j < hi) ? a[j] : -1.f;      // -1 marks "no entry" (real entries are >= 0)
  }
  cluster.sync();                                    // every merged[] is zero before anyone pushes
  float sq = 0.f;
  const float mean = 1.f / (float)n;
  if (in_regs) {
#pragma unroll
    for (int e = 0; e < kHsItems; ++e)
      if (reg[e] >= 0.f) {
        const float dv = reg[e] - mean;
        sq = fmaf(dv, dv, sq);
        atomicAdd(&hist[((__float_as_uint(reg[e]) >> 20) & 0x7ffu) * kHsCopies + copy], 1u);
      }
  } else {
    sweep_from_memory(a, lo, hi, tid, [&](float v) {
      const float dv = v - mean;
      sq = fmaf(dv, dv, sq);
      atomicAdd(&hist[((__float_as_uint(v) >> 20) & 0x7ffu) * kHsCopies + copy], 1u);
    });
  }
  __syncthreads();
  push(0);
  cluster.sync();
  // level-1 counts of the whole head: copy them here (remote reads in parallel), pick the bin
  if (rank != 0)
    for (int b = tid; b < kHsBins; b += kHsThreads) merged[b] = merged0[b];
  clear_local();
  __syncthreads();
  block_pick_from_top(merged, (unsigned)k_rho, scan_tmp, &sel_bin, &sel_rem);
  const unsigned b1 = sel_bin, rem1 = sel_rem;
  float mass = 0.f;
  auto second = [&](float v) {
    const unsigned u = __float_as_uint(v), top = (u >> 20) & 0x7ffu;
    if (top > b1) mass += v;
    else if (top == b1) atomicAdd(&hist[((u >> 9) & 0x7ffu) * kHsCopies + copy], 1u);
  };
  if (in_regs) {
#pragma unroll
    for (int e = 0; e < kHsItems; ++e)
      if (reg[e] >= 0.f) second(reg[e]);
  } else {
    sweep_from_memory(a, lo, hi, tid, second);
  }
  __syncthreads();
  push(1);
  const float tot_sq = block_sum_1024(sq, red);
  const float tot_mass = block_sum_1024(mass, red);
  if (tid == 0) {
    float* slots0 = cluster.map_shared_rank(slots, 0);
    slots0[2 * rank] = tot_sq;
    slots0[2 * rank + 1] = tot_mass;
  }
  cluster.sync();
  if (rank == 0) {
    const unsigned* m2 = merged + kHsBins;
    block_pick_from_top(m2, rem1, scan_tmp, &sel_bin, &sel_rem);
    const unsigned b2 = sel_bin, rem2 = sel_rem;
    // entries of the threshold bin above sub-bin b2, and rem2 entries of sub-bin b2 itself
    float in_bin = 0.f;
    for (int b = tid; b < kHsBins; b += kHsThreads) {
      const float mid = __uint_as_float((b1 << 20) | ((unsigned)b << 9) | 0x100u);
      const unsigned cnt = (unsigned)b > b2 ? m2[b] : ((unsigned)b == b2 ? rem2 : 0u);
      in_bin = fmaf((float)cnt, mid, in_bin);
    }
    const float tot_in_bin = block_sum_1024(in_bin, red);
    if (tid == 0) {
      float s2 = 0.f, m = 0.f;
      for (int r = 0; r < CL; ++r) { s2 += slots[2 * r]; m += slots[2 * r + 1]; }
      head_part[head * 4 + 0] = s2;
      head_part[head * 4 + 1] = m + tot_in_bin;
    }
  }
}

// Eq. 5-6 of a batch of layers from their per-head parts: one thread per layer.
__global__ void head_metrics(const float* __restrict__ head_part, int n_layers, int H, int n,
                             float* __restrict__ metrics) {
  pdl_trigger();
  pdl_wait();
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= n_layers) return;
  float rho = 0.f, var = 0.f;
  const float inv_n = 1.f / (float)n;
  for (int h = 0; h < H; ++h) {
    rho += head_part[((size_t)l * H + h) * 4 + 1];
    var += head_part[((size_t)l * H + h) * 4 + 0] * inv_n;
  }
  metrics[l * 3 + 1] = rho / (float)H;
  metrics[l * 3 + 2] = var / (float)H;
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

cudaError_t launch_finalize_rows(const Ctx& ctx, int parts, cudaStream_t st) {
  const int rows_pg_pad = ctx.rows_pad / ctx.cfg.n_kv_heads;
  const int rows_pg = (ctx.cfg.n_q_heads / ctx.cfg.n_kv_heads) * ctx.cfg.window;
  finalize_rows<<<(ctx.rows_pad + 255) / 256, 256, 0, st>>>(ctx.ws.row_part, parts, ctx.rows_pad,
                                                           rows_pg_pad, rows_pg, ctx.ws.row_lse2,
                                                           ctx.ws.row_ent);
  return cudaGetLastError();
}

template <int CL>
static cudaError_t launch_head_stats_cl(const float* cols, long long layer_stride, long long col_stride,
                                        int n_layers, int H, int n, int k_rho, float* head_part, cudaStream_t st) {
  const int smem = (kHsBins * hs_copies(CL) + 2 * kHsBins) * (int)sizeof(unsigned);
  cudaError_t e = cudaFuncSetAttribute(head_stats<CL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_layers * H * CL);
  cfg.blockDim = dim3(kHsThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = CL;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, head_stats<CL>, cols, layer_stride, col_stride, H, n, k_rho, head_part);
}

// One layer at a time the vectors are few and the kernel is a chain of latencies: a cluster of
// CTAs per vector shortens it.  A batch of layers brings enough vectors to fill the GPU with one
// CTA each, which avoids the cluster barriers and remote merges altogether.
static cudaError_t launch_head_stats(const float* cols, long long layer_stride, long long col_stride, int n_layers,
                                     int H, int n, float* head_part, int sm_count, cudaStream_t st) {
  int k_rho = n / 10;
  if (k_rho < 1) k_rho = 1;
  if ((long long)n_layers * H >= 2ll * sm_count)
    return launch_head_stats_cl<1>(cols, layer_stride, col_stride, n_layers, H, n, k_rho, head_part, st);
  return launch_head_stats_cl<kHsCluster>(cols, layer_stride, col_stride, n_layers, H, n, k_rho, head_part, st);
}

cudaError_t launch_reduce_layers(const Ctx& ctx, const float* cols, long long layer_stride, long long col_stride,
                                 int n, int n_layers, float lambda, float* s_out, long long s_stride,
                                 float* c_inout, const float* row_ent, float* metrics, cudaStream_t st) {
  const int H = ctx.cfg.n_q_heads;
  const int rows_pg_pad = ctx.rows_pad / ctx.cfg.n_kv_heads;
  const int rows_pg = (H / ctx.cfg.n_kv_heads) * ctx.cfg.window;
  const bool vec = n % 4 == 0 && col_stride % 4 == 0 && layer_stride % 4 == 0 && s_stride % 4 == 0 &&
                   ((uintptr_t)cols % 16) == 0 && ((uintptr_t)s_out % 16) == 0 && ((uintptr_t)c_inout % 16) == 0;
  if (vec)
    return launch_pdl(reduce_layers<4>, dim3((n / 4 + 63) / 64), dim3(kRcThreads), 0, st, cols, layer_stride,
                      col_stride, H, n, n_layers, lambda, s_out, s_stride, c_inout, row_ent, ctx.rows_pad,
                      rows_pg_pad, rows_pg, ctx.rows, metrics);
  return launch_pdl(reduce_layers<1>, dim3((n + kRcThreads - 1) / kRcThreads), dim3(kRcThreads), 0, st, cols,
                    layer_stride, col_stride, H, n, n_layers, lambda, s_out, s_stride, c_inout, row_ent,
                    ctx.rows_pad, rows_pg_pad, rows_pg, ctx.rows, metrics);
}

cudaError_t launch_reduce_finish(const Ctx& ctx, const float* cols, long long col_stride, int n, float lambda,
                                 float* s_out, float* c_inout, bool with_head_stats, float* metrics,
                                 cudaStream_t st) {
  const int H = ctx.cfg.n_q_heads;
  if (with_head_stats) {
    const cudaError_t e = launch_head_stats(cols, 0, col_stride, 1, H, n, ctx.ws.head_part, ctx.sm_count, st);
    if (e != cudaSuccess) return e;
  }
  const int rows_pg_pad = ctx.rows_pad / ctx.cfg.n_kv_heads;
  const int rows_pg = (H / ctx.cfg.n_kv_heads) * ctx.cfg.window;
  const bool vec = n % 4 == 0 && col_stride % 4 == 0 && ((uintptr_t)cols % 16) == 0 &&
                   ((uintptr_t)s_out % 16) == 0 && ((uintptr_t)c_inout % 16) == 0;
  if (vec)
    return launch_pdl(reduce_finish<4>, dim3((n / 4 + 63) / 64), dim3(kRcThreads), 0, st, cols,
                      col_stride, H, n, lambda, s_out, c_inout, (const float*)ctx.ws.row_ent, ctx.rows_pad,
                      rows_pg_pad, rows_pg, ctx.rows, (const float*)ctx.ws.head_part, with_head_stats ? 1 : 0,
                      metrics);
  return launch_pdl(reduce_finish<1>, dim3((n + kRcThreads - 1) / kRcThreads), dim3(kRcThreads), 0, st, cols,
                    col_stride, H, n, lambda, s_out, c_inout, (const float*)ctx.ws.row_ent, ctx.rows_pad,
                    rows_pg_pad, rows_pg, ctx.rows, (const float*)ctx.ws.head_part, with_head_stats ? 1 : 0,
                    metrics);
}

cudaError_t launch_head_stats_batch(const Ctx& ctx, const float* cols, long long layer_stride, long long col_stride,
                                    int n_layers, int n, float* metrics, cudaStream_t st) {
  const int H = ctx.cfg.n_q_heads;
  cudaError_t e = launch_head_stats(cols, layer_stride, col_stride, n_layers, H, n, ctx.ws.head_part, ctx.sm_count, st);
  if (e != cudaSuccess) return e;
  return launch_pdl(head_metrics, dim3((n_layers + 63) / 64), dim3(64), 0, st, (const float*)ctx.ws.head_part,
                    n_layers, H, n, metrics);
}

cudaError_t launch_accumulate(const float* s_hist, long long row_stride, int pivot, int n,
                              float lambda, float* c_out, cudaStream_t st) {
  accumulate<<<(n + 255) / 256, 256, 0, st>>>(s_hist, row_stride, pivot, n, lambda, c_out);
  return cudaGetLastError();
}

}  // namespace skv
