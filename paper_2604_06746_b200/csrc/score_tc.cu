// Tensor-core scorer for bf16 storage on sm_100a: TMA-staged K tiles, tcgen05.mma with fp32
// accumulators in tensor memory, softmax statistics / column sums computed straight out of
// tensor memory.  Two kernels share one skeleton:
//
//   pass 1  D[rows, keys] = Q K^T     lane = score row  -> per-row (ref, Z, U) over a key segment
//   pass 2  D[keys, rows] = K Q^T     lane = key        -> per-head column sums for every key
//
// so both reductions are loops inside one thread (no shuffles).  A work unit is (KV group g,
// row block rb of up to 256 score rows); the key range of a unit is split into `segs` equal
// segments, one CTA each.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns the
// tensor-memory allocation), warps 2..9 = compute.  Every wait is bounded; on expiry the CTA
// records STRUCTKV_ERR_TIMEOUT, stops, drains its own copies and frees tensor memory.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "common.cuh"

namespace skv {
namespace {

constexpr int kStages = 4;             // K tile ring
constexpr int kAccStages = 2;          // accumulator ring in tensor memory (256 columns each)
constexpr int kTcThreads = 320;        // 10 warps
constexpr int kComputeThreads = 256;
constexpr unsigned long long kWaitCycles = 1000000000ull;   // about 0.5 s at the maximum SM clock
constexpr float kMasked = -1.0e30f;    // stands for -inf: 2^x flushes to 0 and 0 * x stays finite

struct TcParams {
  int n_keys, window, group, rows_pg, rows_pg_pad, rows_pad, n_rb, segs, n_tiles;
  float c2;                            // scale * log2(e)
  float4* row_part;                    // pass 1 out
  const float* row_lse2;               // pass 2 in
  float* cols;                         // pass 2 out [H][col_stride]
  long long col_stride;
  int* status;
};

struct TcState {
  PFN_cuTensorMapEncodeTiled_v12000 encode;
};

// ---- PTX wrappers ----------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the barrier did not flip in time or the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((unsigned long long)(clock64() - t0) > kWaitCycles) { *abort_flag = 1; return false; }
  }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread l of the warp receives row (lane base + l).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, 8-row
// groups 1024 bytes apart (the layout TMA writes with CU_TENSOR_MAP_SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3fffu);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                          // leading-dimension byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                          // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, tile M x N.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---- shared memory layout ----------------------------------------------------------------
template <int D>
struct Smem {
  static constexpr int kSub = D / 64;                      // 64-column (128-byte) sub-tiles per operand
  static constexpr int kQBytes = kRowBlock * 128 * kSub;   // Q block: 256 rows
  static constexpr int kKBytes = kKeyTile * 128 * kSub;    // one K tile: 128 keys
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kQBytes;
  static constexpr int kLseOff = kKOff + kStages * kKBytes;          // 256 floats
  static constexpr int kBarOff = kLseOff + kRowBlock * 4;
  static constexpr int kBytes = kBarOff + 256;
  static constexpr int kAlloc = kBytes + 1024;             // slack to align the base to 1024 bytes
};

// Barrier slots (8 bytes each) inside the barrier area.
enum { kBarFull = 0, kBarEmpty = kStages, kBarQ = 2 * kStages, kBarAccFull = 2 * kStages + 1,
       kBarAccEmpty = kBarAccFull + kAccStages, kBarDrain = kBarAccEmpty + kAccStages,
       kBarCount = kBarDrain + 1 };

template <int D, int PASS, int W>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_score(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
         const TcParams p) {
  using L = Smem<D>;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  const uint32_t bars = base + L::kBarOff;
  float* lse_s = reinterpret_cast<float*>(sm + L::kLseOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + L::kBarOff + 8 * kBarCount);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + L::kBarOff + 8 * kBarCount + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int unit = blockIdx.x / p.segs, seg = blockIdx.x - unit * p.segs;
  const int g = unit / p.n_rb, rb = unit - g * p.n_rb;
  const int t_lo = (int)((long long)seg * p.n_tiles / p.segs);
  const int t_hi = (int)((long long)(seg + 1) * p.n_tiles / p.segs);
  const int n_my = t_hi - t_lo;
  const int rows_here = min(kRowBlock, p.rows_pg - rb * kRowBlock);     // valid score rows in this block
  const int n_half = (rows_here + 127) / 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bars + 8 * (kBarFull + s), 1); mbar_init(bars + 8 * (kBarEmpty + s), 1); }
    mbar_init(bars + 8 * kBarQ, 1);
    for (int a = 0; a < kAccStages; ++a) {
      mbar_init(bars + 8 * (kBarAccFull + a), 1);
      mbar_init(bars + 8 * (kBarAccEmpty + a), kComputeThreads);
    }
    mbar_init(bars + 8 * kBarDrain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (PASS == 2) {
    // log-sum-exp of the block's rows; padded rows hold +inf so they contribute 2^(-inf) = 0
    for (int r = threadIdx.x; r < kRowBlock; r += kTcThreads)
      lse_s[r] = (r < rows_here) ? p.row_lse2[g * p.rows_pg_pad + rb * kRowBlock + r] : INFINITY;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0 && n_my > 0) {
      mbar_expect_tx(bars + 8 * kBarQ, L::kQBytes);
      const int q_row0 = g * p.rows_pg + rb * kRowBlock;
      for (int s = 0; s < L::kSub; ++s)
        tma_load_2d(base + L::kQOff + s * (L::kQBytes / L::kSub), &map_q, bars + 8 * kBarQ, s * 64, q_row0);
      int issued = 0;
      for (int t = 0; t < n_my; ++t) {
        const int s = t % kStages;
        const uint32_t ph = (uint32_t)(t / kStages) & 1u;
        if (!mbar_wait(bars + 8 * (kBarEmpty + s), ph ^ 1u, abort_flag)) break;
        mbar_expect_tx(bars + 8 * (kBarFull + s), L::kKBytes);
        for (int c = 0; c < L::kSub; ++c)
          tma_load_3d(base + L::kKOff + s * L::kKBytes + c * (L::kKBytes / L::kSub), &map_k,
                      bars + 8 * (kBarFull + s), c * 64, (t_lo + t) * kKeyTile, g);
        ++issued;
      }
      // drain: every copy this thread issued must have landed before the CTA may exit
      mbar_wait(bars + 8 * kBarQ, 0, abort_flag);
      for (int t = max(0, issued - kStages); t < issued; ++t)
        mbar_wait(bars + 8 * (kBarFull + t % kStages), (uint32_t)(t / kStages) & 1u, abort_flag);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && n_my > 0) {
      constexpr uint32_t idesc = (PASS == 1) ? instr_desc(128, 128) : instr_desc(128, 256);
      bool ok = mbar_wait(bars + 8 * kBarQ, 0, abort_flag);
      int t = 0;
      for (; ok && t < n_my; ++t) {
        const int s = t % kStages, a = t % kAccStages;
        if (!mbar_wait(bars + 8 * (kBarFull + s), (uint32_t)(t / kStages) & 1u, abort_flag)) break;
        if (!mbar_wait(bars + 8 * (kBarAccEmpty + a), ((uint32_t)(t / kAccStages) & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t k_tile = base + L::kKOff + s * L::kKBytes;
        const uint32_t q_tile = base + L::kQOff;
        if (PASS == 1) {
          for (int hf = 0; hf < n_half; ++hf) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t qa = q_tile + (kk / 4) * (L::kQBytes / L::kSub) + hf * (128 * 128) + (kk % 4) * 32;
              const uint32_t kb = k_tile + (kk / 4) * (L::kKBytes / L::kSub) + (kk % 4) * 32;
              tc_mma_bf16(tmem + a * 256 + hf * 128, smem_desc(qa), smem_desc(kb), idesc, kk > 0);
            }
          }
        } else {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t ka = k_tile + (kk / 4) * (L::kKBytes / L::kSub) + (kk % 4) * 32;
            const uint32_t qb = q_tile + (kk / 4) * (L::kQBytes / L::kSub) + (kk % 4) * 32;
            tc_mma_bf16(tmem + a * 256, smem_desc(ka), smem_desc(qb), idesc, kk > 0);
          }
        }
        tc_commit(bars + 8 * (kBarEmpty + s));       // K stage reusable once these MMAs have read it
        tc_commit(bars + 8 * (kBarAccFull + a));     // accumulator ready for the compute warps
      }
      // drain: all issued MMAs must retire before tensor memory is freed
      tc_commit(bars + 8 * kBarDrain);
      mbar_wait(bars + 8 * kBarDrain, 0, abort_flag);
    }
  } else {
    // ---------------- compute warps ----------------
    const int cw = warp - 2;                 // 0..7
    const int quarter = warp & 3;            // tensor-memory lane quarter this warp may read
    const int half = cw >> 2;                // pass 1: row half; pass 2: column half
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    // a tile is "plain" when all of its keys are visible to every window row (j0 + 127 <= N - w);
    // the first (N - w + 1) / 128 tiles are
    const int first_tail_tile = (p.n_keys - p.window + 1) / kKeyTile;

    if (PASS == 1) {
      const int row_in_block = half * 128 + quarter * 32 + lane;
      const bool row_valid = row_in_block < rows_here;
      const bool warp_active = (half * 128 + quarter * 32) < rows_here;
      const int i_win = (rb * kRowBlock + row_in_block) % p.window;      // window row index of this score row
      const int t_pos = p.n_keys - p.window + i_win;                     // its position: sees keys <= t_pos
      float ref = -INFINITY, Z = 0.f, U = 0.f;
      for (int t = 0; t < n_my; ++t) {
        const int a = t % kAccStages;
        if (!mbar_wait(bars + 8 * (kBarAccFull + a), (uint32_t)(t / kAccStages) & 1u, abort_flag)) break;
        tc_fence_after();
        if (warp_active) {
          const uint32_t taddr = tmem + lane_base + a * 256 + half * 128;
          const int j0 = (t_lo + t) * kKeyTile;
          const bool plain = (t_lo + t) < first_tail_tile && t > 0;
          // Every tensor-memory load below is executed by the whole warp (the instruction is
          // warp-collective); only the arithmetic on the loaded values is per-thread.
          bool redo = !plain;
          const float Z0 = Z, U0 = U;
          if (plain) {
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              float v[32];
              tmem_ld32(taddr + c * 32, v);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const float x = fmaf(v[e], p.c2, -ref);
                const float pr = fast_exp2(x);
                Z += pr;
                U = fmaf(pr, x, U);
              }
            }
            // a logit far above the reference overflowed 2^x: the whole warp re-references the tile
            const bool ovf = !(Z < 3.0e38f) || !(fabsf(U) < 3.0e38f);
            redo = __any_sync(0xffffffffu, ovf);
            if (redo) { Z = Z0; U = U0; }
          }
          if (redo) {
            // masked / first / overflowed tile: find the tile maximum, move the reference, accumulate
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              float v[32];
              tmem_ld32(taddr + c * 32, v);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (j0 + c * 32 + e <= t_pos) mx = fmaxf(mx, v[e] * p.c2);
            }
            if (mx > ref) {
              if (ref != -INFINITY) {
                const float dm = ref - mx, f = fast_exp2(dm);
                U = f * fmaf(dm, Z, U);
                Z = f * Z;
              }
              ref = mx;
            }
            const float ref_use = (ref == -INFINITY) ? 0.f : ref;    // row has seen no key yet: all masked
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              float v[32];
              tmem_ld32(taddr + c * 32, v);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const float x = (j0 + c * 32 + e <= t_pos) ? fmaf(v[e], p.c2, -ref_use) : kMasked;
                const float pr = fast_exp2(x);
                Z += pr;
                U = fmaf(pr, x, U);
              }
            }
          }
        }
        tc_fence_before();
        mbar_arrive(bars + 8 * (kBarAccEmpty + a));
      }
      if (row_valid && n_my > 0)
        p.row_part[(size_t)seg * p.rows_pad + g * p.rows_pg_pad + rb * kRowBlock + row_in_block] =
            make_float4(ref, Z, U, 0.f);
      else if (row_valid)
        p.row_part[(size_t)seg * p.rows_pad + g * p.rows_pg_pad + rb * kRowBlock + row_in_block] =
            make_float4(-INFINITY, 0.f, 0.f, 0.f);
    } else {
      // pass 2: this thread owns key (tile * 128 + quarter * 32 + lane) and the block's score rows
      // [half * 128, half * 128 + 128); those rows belong to 128 / W heads (or half of one head).
      constexpr int kHeads = (W <= 128) ? 128 / W : 1;     // heads per column half
      constexpr int kChunksPerHead = 4 / kHeads;           // 32-column chunks per head
      const float inv_w = 1.0f / (float)p.window;
      const int row0 = rb * kRowBlock + half * 128;        // first local score row of this half
      const bool half_active = half * 128 < rows_here;
      for (int t = 0; t < n_my; ++t) {
        const int a = t % kAccStages;
        if (!mbar_wait(bars + 8 * (kBarAccFull + a), (uint32_t)(t / kAccStages) & 1u, abort_flag)) break;
        tc_fence_after();
        const int j = (t_lo + t) * kKeyTile + quarter * 32 + lane;
        float acc[kHeads];
#pragma unroll
        for (int hh = 0; hh < kHeads; ++hh) acc[hh] = 0.f;
        if (half_active) {
          const uint32_t taddr = tmem + lane_base + a * 256 + half * 128;
          const bool plain = (t_lo + t) < first_tail_tile;
          const int i_min = j - (p.n_keys - p.window);      // window rows i < i_min do not see key j
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            float v[32];
            tmem_ld32(taddr + c * 32, v);
            tmem_ld_wait();
            const float4* l4 = reinterpret_cast<const float4*>(lse_s + half * 128 + c * 32);
            float s = 0.f;
            if (plain) {
#pragma unroll
              for (int e4 = 0; e4 < 8; ++e4) {
                const float4 l = l4[e4];
                s += fast_exp2(fmaf(v[4 * e4 + 0], p.c2, -l.x));
                s += fast_exp2(fmaf(v[4 * e4 + 1], p.c2, -l.y));
                s += fast_exp2(fmaf(v[4 * e4 + 2], p.c2, -l.z));
                s += fast_exp2(fmaf(v[4 * e4 + 3], p.c2, -l.w));
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const int i = (row0 + c * 32 + e) % p.window;
                const float x = fmaf(v[e], p.c2, -lse_s[half * 128 + c * 32 + e]);
                s += (i >= i_min) ? fast_exp2(x) : 0.f;
              }
            }
            acc[c / kChunksPerHead] += s;
          }
        }
        tc_fence_before();
        mbar_arrive(bars + 8 * (kBarAccEmpty + a));
        if (half_active && j < p.n_keys) {
#pragma unroll
          for (int hh = 0; hh < kHeads; ++hh) {
            const int lr = row0 + hh * (128 / kHeads);       // first local row of this head slice
            if (lr < p.rows_pg) {
              const int h = g * p.group + lr / p.window;
              p.cols[(size_t)h * p.col_stride + j] = acc[hh] * inv_w;
            }
          }
        }
      }
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) atomicCAS(p.status, 0, (int)STRUCTKV_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

template <int D, int PASS, int W>
cudaError_t launch_one(const CUtensorMap& mq, const CUtensorMap& mk, const TcParams& p, int grid,
                       cudaStream_t st) {
  auto kern = tc_score<D, PASS, W>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::kAlloc);
  if (e != cudaSuccess) return e;
  kern<<<grid, kTcThreads, Smem<D>::kAlloc, st>>>(mq, mk, p);
  return cudaGetLastError();
}

template <int D, int PASS>
cudaError_t launch_w(int w, const CUtensorMap& mq, const CUtensorMap& mk, const TcParams& p, int grid,
                     cudaStream_t st) {
  switch (w) {
    case 32: return launch_one<D, PASS, 32>(mq, mk, p, grid, st);
    case 64: return launch_one<D, PASS, 64>(mq, mk, p, grid, st);
    case 128: return launch_one<D, PASS, 128>(mq, mk, p, grid, st);
  }
  return cudaErrorInvalidValue;
}

bool encode_maps(const Ctx& ctx, const ScoreArgs& a, CUtensorMap* mq, CUtensorMap* mk) {
  TcState* s = (TcState*)ctx.tc;
  const int d = ctx.cfg.head_dim;
  {
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)ctx.cfg.n_q_heads * ctx.cfg.window};
    cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kRowBlock};
    cuuint32_t estr[2] = {1, 1};
    if (s->encode(mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(a.q), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  {
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)a.n_keys, (cuuint64_t)ctx.cfg.n_kv_heads};
    cuuint64_t strides[2] = {(cuuint64_t)a.k_stride_token * 2, (cuuint64_t)a.k_stride_head * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)kKeyTile, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (ctx.cfg.n_kv_heads == 1) strides[1] = strides[0] * (cuuint64_t)a.n_keys;
    if (s->encode(mk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(a.k), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

}  // namespace

bool tc_supported(const Ctx& ctx, const ScoreArgs& a) {
  if (!ctx.tc || ctx.cfg.dtype != STRUCTKV_BF16) return false;
  const int w = ctx.cfg.window;
  if (w != 32 && w != 64 && w != 128) return false;
  if (ctx.cfg.head_dim != 64 && ctx.cfg.head_dim != 128) return false;
  // tensor-map limits: strides below 2^40 bytes, multiples of 16 bytes (checked by the caller)
  if (a.k_stride_token * 2 >= (1ll << 40) || a.k_stride_head * 2 >= (1ll << 40)) return false;
  if (ctx.cfg.n_kv_heads > 1 && a.k_stride_head == 0) return false;
  return true;
}

structkv_status tc_create(Ctx& ctx) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn)
    return STRUCTKV_ERR_CUDA;
  TcState* s = new TcState();
  s->encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  ctx.tc = s;
  return STRUCTKV_OK;
}

void tc_destroy(Ctx& ctx) {
  delete (TcState*)ctx.tc;
  ctx.tc = nullptr;
}

cudaError_t launch_score_tc(Ctx& ctx, const ScoreArgs& a, int* parts_out, int pass, cudaStream_t st) {
  CUtensorMap mq, mk;
  if (!encode_maps(ctx, a, &mq, &mk)) return cudaErrorInvalidValue;
  TcParams p;
  p.n_keys = a.n_keys;
  p.window = ctx.cfg.window;
  p.group = ctx.cfg.n_q_heads / ctx.cfg.n_kv_heads;
  p.rows_pg = p.group * p.window;
  p.rows_pg_pad = ctx.rows_pad / ctx.cfg.n_kv_heads;
  p.rows_pad = ctx.rows_pad;
  p.n_rb = (p.rows_pg + kRowBlock - 1) / kRowBlock;
  p.n_tiles = (a.n_keys + kKeyTile - 1) / kKeyTile;
  const int units = ctx.cfg.n_kv_heads * p.n_rb;
  int segs = ctx.sm_count / units;
  if (segs < 1) segs = 1;
  if (segs > p.n_tiles) segs = p.n_tiles;
  if (segs > kMaxParts) segs = kMaxParts;
  p.segs = segs;
  p.c2 = a.scale * kLog2e;
  p.row_part = ctx.ws.row_part;
  p.row_lse2 = ctx.ws.row_lse2;
  p.cols = a.cols;
  p.col_stride = a.col_stride;
  p.status = ctx.ws.status;
  *parts_out = segs;
  const int grid = units * segs;
  const int d = ctx.cfg.head_dim, w = ctx.cfg.window;
  if (d == 128) return pass == 1 ? launch_w<128, 1>(w, mq, mk, p, grid, st) : launch_w<128, 2>(w, mq, mk, p, grid, st);
  return pass == 1 ? launch_w<64, 1>(w, mq, mk, p, grid, st) : launch_w<64, 2>(w, mq, mk, p, grid, st);
}

}  // namespace skv
