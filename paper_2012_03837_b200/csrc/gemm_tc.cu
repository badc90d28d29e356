// Grouped bf16 GEMM on the 5th-generation tensor cores (tcgen05) for sm_100a.
//
// Persistent CTAs walk a flat list of output tiles that spans every problem of the launch (all
// chunks' forward, input-gradient and weight-gradient products of one phase: Sec. 3 makes them
// independent).  Two variants of one kernel template:
//   CG = 2 (default): a cluster of two CTAs on neighbouring SMs owns a 256x256 tile
//          (tcgen05 cta_group::2, M = 256, N = 256, K = 16 per instruction, issued by the leader);
//   CG = 1: one CTA per 128x256 tile (launches that hold a problem with M <= 128).
// Per tile, 64-deep k slices of A and B are brought into a shared-memory ring (6 stages of 32 KB,
// or 4 of 48 KB) by TMA (128-byte swizzle; out-of-range rows/columns read as zero, so ragged M, N,
// K need no special case; operand panels carry an evict-last L2 hint), one elected thread issues
// the MMAs into one of two 256-column TMEM accumulators, and eight epilogue warps read the finished
// accumulator back with tcgen05.ld, apply the fused epilogue (bias, residual, ReLU/GELU, ReLU mask,
// GELU', softmax statistics of the logits) and hand bf16 or fp32 blocks, staged in swizzled shared
// memory, to TMA stores (evict-first) while the next tile's main loop already runs on the other
// accumulator.  Tiles of a problem are walked in bands of 8 row tiles so that the tiles in flight
// share operand panels in L2.
//
// Operands may be K-major (reduction index contiguous) or MN-major (row/column index contiguous),
// per problem: forward uses K/K, the input gradient K/MN, the weight gradient MN/MN, so no
// transposed copy of a weight or an activation is ever materialised.
//
// Every wait on an mbarrier is bounded (about two seconds): on expiry the thread raises the
// TIMEOUT bit of the status word, all roles leave their loops, TMEM is freed and the kernel returns.
// No TMA load uses cluster multicast.
#include <cuda.h>

#include <algorithm>
#include <queue>
#include <vector>
#include <cstdio>
#include <cstdlib>

#include "common.cuh"
#include "gemm_tc.h"
#include "tc_prims.cuh"

namespace lp {
namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int A_BYTES = BM * BK * 2;              // 16 KB of A per CTA and stage
// CG = 1: one CTA per 128x256 tile, B tile 256x64 (32 KB), 4 stages of 48 KB.
// CG = 2: a pair of CTAs (cluster of 2, tcgen05 cta_group::2) per 256x256 tile; each CTA holds its own
//         128 rows of A and HALF of the B tile (128x64, 16 KB), so every SM pulls a third fewer bytes per
//         FLOP through its L2 port and the ring is 6 stages of 32 KB.
// W = 1 ("wide", CTA pairs only): a 256x512 tile per pair, computed as two MMAs per k-step that share the A
//         slice: 16 KB of A and two 16 KB B halves per stage (4 stages of 48 KB).  Per FLOP a CTA then moves
//         20 % less through shared memory than with the 256x256 tile; both accumulators belong to the one
//         tile, so the epilogue is not overlapped with the next main loop -- worth it only for long reductions.
template <int CG, int W = 0> struct Cfg {
  static constexpr int TN = W ? 2 * BN : BN;                // tile columns
  static constexpr int NB = W ? 2 : 1;                      // B sub-tiles = MMAs per k-step
  static constexpr int BNL = BN / CG;                       // rows of one B sub-tile this CTA loads
  static constexpr int B_SUB_BYTES = BNL * BK * 2;
  static constexpr int B_BYTES = NB * B_SUB_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = CG == 1 ? 4 : (W ? 4 : 6);
};
constexpr int MAX_STAGES = 6;
constexpr int EPI_WARPS = 8;                      // two warps per TMEM lane quarter, each takes half of the 256 columns
// Warps 0-3 form the control warpgroup (0: TMA producer, 1: MMA issuer, 2-3: idle); warps 4-11 are
// the two epilogue warpgroups.  After set-up the control warpgroup hands most of its registers to
// the epilogue warpgroups (setmaxnreg), whose threads each hold 64 accumulator values, the prefetched
// side input and the converted outputs.
constexpr int EPI_FIRST = 4;
constexpr int NTHREADS = 32 * (EPI_FIRST + EPI_WARPS);
// The pool that setmaxnreg redistributes is what the launch allocated: 384 threads x 168 registers.
constexpr int CTRL_REGS = 56, EPI_REGS = 224;     // 128 * 56 + 256 * 224 = 384 * 168
constexpr uint32_t TMEM_COLS = 512;

struct __align__(8) Shared {
  uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

using namespace tc;

// Bounded wait on a barrier of this block (see tc::mbar_wait); on expiry all roles leave their loops.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Shared* sh, int* status) {
  return tc::mbar_wait(bar, parity, &sh->abort_flag, status);
}
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, bool mn_major) { return tc::make_desc(saddr, mn_major, BK * 128); }

// Which problem a tile of the launch's flat tile list belongs to.  Tiles are visited in increasing
// order, so the cursor only moves forward; seek() touches global memory only when the problem changes.
struct ProbCursor {
  const GemmProb* probs;
  int nprob, pi, next_start;
  __device__ __forceinline__ ProbCursor(const GemmProb* pr, int n) : probs(pr), nprob(n), pi(-1), next_start(0) {}
  // Moves to the problem holding `tile`; true if the problem changed (always on the first call).
  __device__ __forceinline__ bool seek(int tile) {
    if (tile < next_start) return false;
    do {
      ++pi;
      next_start = pi + 1 < nprob ? probs[pi + 1].tile_start : 0x7fffffff;
    } while (tile >= next_start);                 // problems without tiles are stepped over
    return true;
  }
};
// Tile t of a problem -> (row tile, column tile).  Tiles are walked in bands of `raster` row tiles,
// row tile fastest inside a band, so that the tiles in flight at any time share a few operand
// panels of each kind instead of one row panel and all column panels; the band is as high as
// lets its row panels stay in L2 while the column panels stream past once.
struct TileWalk {
  int tile_start, tiles_m, tiles_n, raster;
  __device__ __forceinline__ void set(const GemmProb& p, int tile_m) {
    tile_start = p.tile_start; tiles_n = p.tiles_n; raster = p.raster;
    tiles_m = (p.M + tile_m - 1) / tile_m;
  }
  __device__ __forceinline__ void coords(int tile, int& mt, int& nt) const {
    const int t = tile - tile_start;
    const int per_band = raster * tiles_n;
    const int band = t / per_band;
    const int m_base = band * raster;
    const int gm = min(raster, tiles_m - m_base);
    const int r = t - band * per_band;
    nt = r / gm;
    mt = m_base + r - nt * gm;
  }
};

// Fused epilogue for 32 consecutive columns (n0 ..) of one accumulator row (row m, held by this lane).
// Output path: if `stg` is non-null the warp's 32x32 block is written to a 4 KB shared-memory staging
// buffer in the swizzled layout of the output tensor map and leaves through ONE TMA store (full-line
// writes, clipped at the matrix edge by the hardware); otherwise every lane stores its own row.
// VEC: all 32 columns exist and resid / aux / C are 16-byte aligned (128-bit accesses).
// GELU x*Phi(x) and its derivative for the epilogue, where 128 values per thread and tile have to
// fit under the tile's main loop (16 k-slices for the feed-forward products).  Phi is evaluated as
// the logistic function of an odd quintic:  Phi(x) ~ 1 / (1 + 2^(-z)),  z = x (k0 + k1 s + k2 s^2),
// s = min(x^2, 64), fitted to 2 log2(e) atanh(erf(x / sqrt 2)) on |x| <= 8 (beyond it z keeps growing
// linearly and Phi is 0 or 1 to fp32 precision).  Largest deviation from the erf form: 6e-5 in Phi,
// 3e-5 in GELU, 1e-4 in GELU' -- below the bf16 rounding step (2^-9 relative) of the values the
// epilogue stores.  One ex2, one rcp and five FMA-class operations per value; the derivative
// d/dx [x Phi] = Phi + x Phi (1 - Phi) z'(x) ln 2 reuses Phi and needs no further special function.
constexpr float GELU_K0 = 2.30104886f, GELU_K1 = 0.106717206f, GELU_K2 = -1.00029423e-3f;   // 2 log2(e) * (c0, c1, c2)
__device__ __forceinline__ float phi_logistic(float x, float& s) {
  s = fminf(x * x, 64.f);
  const float z = x * fmaf(fmaf(GELU_K2, s, GELU_K1), s, GELU_K0);
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + ex2_approx(-z)));
  return r;
}
__device__ __forceinline__ float gelu_fast(float x) {
  float s;
  return x * phi_logistic(x, s);
}
__device__ __forceinline__ float gelu_grad_fast(float x) {
  float s;
  const float cdf = phi_logistic(x, s);
  // z'(x) ln 2 = ln 2 (k0 + 3 k1 s + 5 k2 s^2); the clamp of s only acts where Phi (1 - Phi) has vanished
  const float dz = fmaf(fmaf(5.f * 0.69314718f * GELU_K2, s, 3.f * 0.69314718f * GELU_K1), s, 0.69314718f * GELU_K0);
  return fmaf(x * fmaf(-cdf, cdf, cdf), dz, cdf);
}
template <bool VEC>
__device__ __forceinline__ void epilogue_row32(const GemmProb& p, const CUtensorMap* mapC, const CUtensorMap* mapC2,
                                               uint8_t* stg, int m, int m_warp0, int n0, const uint32_t* acc, int lane,
                                               int chunk, float2& run, const void* side, const uint4* side_pre) {
  float v[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(acc[j]);
  const bool row_ok = m < p.M;
  const size_t off = (size_t)m * p.ldc + n0;
  const int nvalid = min(32, p.N - n0);
  if (p.bias) {
    if (VEC && (((uintptr_t)p.bias & 15) == 0)) {
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float4 b4 = *(const float4*)(p.bias + n0 + 4 * q);
        v[4 * q] += b4.x; v[4 * q + 1] += b4.y; v[4 * q + 2] += b4.z; v[4 * q + 3] += b4.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (VEC || j < nvalid) v[j] += p.bias[n0 + j];
    }
  }
  // `side` (resid or aux, when only one of them is set) arrives already loaded in side_pre on the 128-bit path
  auto load32 = [&](const void* base, float* o) {
    const bf16* src = (const bf16*)base + off;
    if (!row_ok) {
#pragma unroll
      for (int j = 0; j < 32; ++j) o[j] = 0.f;
    } else if (VEC) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint4 u = (side_pre && base == side) ? side_pre[q] : *(const uint4*)(src + q * 8);
        const __nv_bfloat162* h = (const __nv_bfloat162*)&u;
#pragma unroll
        for (int t = 0; t < 4; ++t) { float2 f = __bfloat1622float2(h[t]); o[q * 8 + 2 * t] = f.x; o[q * 8 + 2 * t + 1] = f.y; }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) o[j] = j < nvalid ? __bfloat162float(src[j]) : 0.f;
    }
  };
  // 32 values -> 16 packed bf16 pairs (round to nearest even), and the values as stored
  auto pack32 = [](const float* o, uint32_t* pk) {
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      __nv_bfloat162 h = __floats2bfloat162_rn(o[2 * t], o[2 * t + 1]);
      pk[t] = *(uint32_t*)&h;
    }
  };
  auto unpack32 = [](const uint32_t* pk, float* o) {
#pragma unroll
    for (int t = 0; t < 16; ++t) { o[2 * t] = __uint_as_float(pk[t] << 16); o[2 * t + 1] = __uint_as_float(pk[t] & 0xffff0000u); }
  };
  // One output block of this warp: 32 rows x 32 columns, bf16 (pk: 16 packed pairs per lane) or fp32 (o).
  // With TMA stores the block is staged in this warp's 4 KB buffer.  `slot` selects the 2 KB half a
  // narrow bf16 block uses; only a block in slot 0 waits for the buffer's previous stores to have been
  // read, so the two outputs of the GELU epilogue are in flight together.
  auto put = [&](void* base, const CUtensorMap* map, const uint32_t* pk, const float* o, bool f32, int slot) {
    if (stg && p.store_tma == 2) {
      // bf16, two neighbouring 32-column blocks share one store of 128-byte rows: the even block
      // fills 16-byte units 0-3 of every row, the odd one units 4-7 (128-byte swizzle)
      const int half = chunk & 1;
      if (half == 0) {
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
        *(uint4*)(stg + lane * 128 + (((half * 4 + q) ^ (lane & 7)) << 4)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
      if (half == 1 || n0 + 32 >= p.N) {          // the pair is complete (or has no second block)
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(map, n0 - half * 32, m_warp0, stg);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
    } else if (stg) {
      if (slot == 0) {
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // staging buffer free again
        __syncwarp();
      }
      uint8_t* dst = stg + slot * 2048;
      if (f32) {
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *(float4*)(dst + lane * 128 + ((q ^ (lane & 7)) << 4)) = make_float4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *(uint4*)(dst + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        tma_store_2d(map, n0, m_warp0, dst);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    } else if (row_ok) {
      if (f32) {
        float* dst = (float*)base + off;
        if (VEC) {
#pragma unroll
          for (int q = 0; q < 8; ++q) *(float4*)(dst + q * 4) = make_float4(o[q * 4], o[q * 4 + 1], o[q * 4 + 2], o[q * 4 + 3]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = o[j];
        }
      } else {
        bf16* dst = (bf16*)base + off;
        if (VEC) {
#pragma unroll
          for (int q = 0; q < 4; ++q) *(uint4*)(dst + q * 8) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (j < nvalid) ((uint16_t*)dst)[j] = (uint16_t)((j & 1) ? (pk[j >> 1] >> 16) : (pk[j >> 1] & 0xffffu));
        }
      }
    }
  };
  float t[32];
  uint32_t pk[16];
  if (p.resid) {
    load32(p.resid, t);
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] += t[j];
  }
  switch (p.act) {
    case EPI_RELU:
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = relu_f(v[j]);
      break;
    case EPI_GELU:
      // the pre-activation is stored (C2) and the activation is taken of the value as stored
      pack32(v, pk);
      unpack32(pk, v);
      if (p.aux_blocked) {
        // blocked layout: this warp's 32x32 block is 2 KB of its own; four coalesced 512-byte stores
        uint4* blk = (uint4*)((bf16*)p.C2 + (((size_t)(m_warp0 >> 5) * (p.ldc >> 5) + (n0 >> 5)) << 10));
#pragma unroll
        for (int q = 0; q < 4; ++q) blk[q * 32 + lane] = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
      } else {
        put(p.C2, mapC2, pk, nullptr, false, 0);
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = gelu_fast(v[j]);
      pack32(v, pk);
      put(p.C, mapC, pk, nullptr, false, p.aux_blocked ? 0 : 1);
      return;
    case EPI_RELU_MASK:
      load32(p.aux, t);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = t[j] > 0.f ? v[j] : 0.f;
      break;
    case EPI_GELU_GRAD:
      load32(p.aux, t);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] *= gelu_grad_fast(t[j]);
      break;
    case EPI_LOGIT_STATS: {
      // running (max, sum of exp(z - max)) of this row over the warp's columns, on the values as stored
      const float L2E = 1.4426950408889634f;
      pack32(v, pk);
      unpack32(pk, v);
      float cm = -INFINITY;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (VEC || j < nvalid) cm = fmaxf(cm, v[j]);
      const float nm = fmaxf(run.x, cm), nml = nm * L2E;
      float cs = 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j) if (VEC || j < nvalid) cs += ex2_approx(fmaf(v[j], L2E, -nml));
      run.y = (run.x == -INFINITY ? 0.f : run.y * ex2_approx((run.x - nm) * L2E)) + cs;
      run.x = nm;
      put(p.C, mapC, pk, nullptr, false, 0);
      return;
    }
    default: break;
  }
  if (p.out_f32) {
    put(p.C, mapC, nullptr, v, true, 0);
  } else {
    pack32(v, pk);
    put(p.C, mapC, pk, nullptr, false, 0);
  }
}

// ---- cluster helpers (CG = 2)
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {   // same offset in CTA `rank` of the cluster
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t bar_caddr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_caddr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_caddr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_caddr) : "memory");
}
// TMA load whose completion is signalled on a barrier given by cluster address (the pair leader's).
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint32_t bar_caddr) {
  // operand panels are re-read by the neighbouring tiles: keep them in L2 ahead of the streamed outputs
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(bar_caddr), "l"(policy_evict_last()) : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar_caddr) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar_caddr), "l"(policy_evict_last()) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {   // arrives on this barrier in both CTAs of the pair
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

template <int CG, int W>
__global__ void __launch_bounds__(NTHREADS, 1)
gemm_tc_kernel(const GemmProb* __restrict__ probs, const CUtensorMap* __restrict__ maps, int nprob, int total_tiles,
               int* status, const int* __restrict__ sched, const int* __restrict__ sched_off) {
  using C = Cfg<CG, W>;
  constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES, BNL = C::BNL, TN = C::TN, NB = C::NB,
                B_SUB_BYTES = C::B_SUB_BYTES;
  constexpr int TILE_M = BM * CG;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* staging = tiles + STAGES * STAGE_BYTES;                     // EPI_WARPS x 4 KB, 1024-byte aligned
  Shared* sh = (Shared*)(staging + EPI_WARPS * 4096);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = CG == 2 ? cluster_rank() : 0;          // 0 = the CTA that issues the pair's MMAs
  const int first_tile = blockIdx.x / CG, tile_step = gridDim.x / CG;
  // The tiles of this CTA (pair), in increasing order: every tile_step-th tile of the launch, or -- when the
  // launch mixes tiles of very different lengths -- the list a host-side balancer made for it (gemm_tc_schedule).
  // All roles, and both CTAs of a pair, walk the same list.
  const int my_begin = sched ? sched_off[first_tile] : 0;
  const int my_count = sched ? sched_off[first_tile + 1] - my_begin
                             : (first_tile < total_tiles ? (total_tiles - first_tile + tile_step - 1) / tile_step : 0);
  auto tile_at = [&](int i) { return sched ? sched[my_begin + i] : first_tile + i * tile_step; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh->full[s], CG); mbar_init(&sh->empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh->tmem_full[a], 1); mbar_init(&sh->tmem_empty[a], CG * EPI_WARPS); }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (CG == 1) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();             // the partner's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *(volatile uint32_t*)&sh->tmem_base;

  if (warp < EPI_FIRST) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CTRL_REGS));
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one per CTA)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      ProbCursor cur(probs, nprob);
      TileWalk walk;
      bool a_mn = false, b_mn = false;
      int kb_n = 0;
      int conv = 0;
      int bnl = BNL;                                 // B rows (columns of the tile) this CTA loads per sub-tile
      uint32_t stage_tx = STAGE_BYTES;               // bytes a stage receives: less for a narrow tile
      int tile_next = my_count > 0 ? tile_at(0) : 0;
      for (int ti = 0; ti < my_count && ok; ++ti) {
        const int tile = tile_next;
        if (ti + 1 < my_count) tile_next = tile_at(ti + 1);   // on its way while this tile's loads are issued
        if (cur.seek(tile)) {                        // problem changed: re-read its fields (once per problem, not per tile)
          const GemmProb& p = probs[cur.pi];
          walk.set(p, TILE_M);
          a_mn = p.a_ms == 1; b_mn = p.b_ns == 1;
          kb_n = (p.K + BK - 1) / BK;
          conv = p.conv;
          bnl = p.tile_n / CG;
          stage_tx = (uint32_t)(A_BYTES + NB * bnl * BK * 2);
        }
        const CUtensorMap* mapA = maps + 4 * cur.pi;
        const CUtensorMap* mapB = mapA + 1;
        int mt, nt;
        walk.coords(tile, mt, nt);
        int m0 = mt * TILE_M + (int)rank * BM, n0 = nt * (TN / BN) * (bnl * CG) + (int)rank * bnl;
        if (conv == CONV_NONE) {
          // ---- ordinary operands: 2-D boxes of the A and B matrices
          for (int kb = 0; kb < kb_n; ++kb) {
            if (!(ok = mbar_wait(&sh->empty[stage], phase ^ 1, sh, status))) break;
            uint8_t* a_dst = tiles + stage * STAGE_BYTES;
            uint8_t* b_dst = a_dst + A_BYTES;
            int k0 = kb * BK;
            if (CG == 1) {
              uint64_t* bar = &sh->full[stage];
              mbar_expect_tx(bar, stage_tx);
              if (a_mn) {
#pragma unroll
                for (int i = 0; i < BM / 64; ++i) tma_load_2d(a_dst + i * (BK * 128), mapA, m0 + i * 64, k0, bar);
              } else {
                tma_load_2d(a_dst, mapA, k0, m0, bar);
              }
#pragma unroll
              for (int sb = 0; sb < NB; ++sb) {
                uint8_t* b_sub = b_dst + sb * B_SUB_BYTES;
                const int ns = n0 + sb * BN;
                if (b_mn) {
                  for (int i = 0; i < bnl / 64; ++i) tma_load_2d(b_sub + i * (BK * 128), mapB, ns + i * 64, k0, bar);
                } else {
                  tma_load_2d(b_sub, mapB, k0, ns, bar);
                }
              }
            } else {
              // both CTAs' bytes are counted on the leader's barrier
              uint32_t bar = map_to_rank(smem_u32(&sh->full[stage]), 0);
              mbar_expect_tx_cluster(bar, stage_tx);
              if (a_mn) {
#pragma unroll
                for (int i = 0; i < BM / 64; ++i) tma_load_2d_pair(a_dst + i * (BK * 128), mapA, m0 + i * 64, k0, bar);
              } else {
                tma_load_2d_pair(a_dst, mapA, k0, m0, bar);
              }
#pragma unroll
              for (int sb = 0; sb < NB; ++sb) {
                uint8_t* b_sub = b_dst + sb * B_SUB_BYTES;
                const int ns = n0 + sb * BN;
                if (b_mn) {
                  for (int i = 0; i < bnl / 64; ++i) tma_load_2d_pair(b_sub + i * (BK * 128), mapB, ns + i * 64, k0, bar);
                } else {
                  tma_load_2d_pair(b_sub, mapB, k0, ns, bar);
                }
              }
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          continue;
        }
        // ---- implicit convolution: one operand is fetched as shifted boxes of the activation tensor
        const GemmProb& p = probs[cur.pi];
        const int cv_c = p.conv_c, cv_w = p.conv_w, cv_hw = p.conv_h * p.conv_w, cv_n = p.conv_n, cv_k0 = p.conv_k0, p_n = p.N;
        const int cv_s = p.conv_stride > 1 ? p.conv_stride : 1, cv_taps = p.conv_taps ? p.conv_taps : 9;
        // tap t of the filter -> offset of the input pixel (3x3 with padding 1, or the single tap of a 1x1 filter)
        auto tap_di = [&](int t) { return cv_taps == 1 ? 0 : t / 3 - 1; };
        auto tap_dj = [&](int t) { return cv_taps == 1 ? 0 : t - (t / 3) * 3 - 1; };
        // this CTA's 128 output pixels start at row a_h0 of image a_img (whole rows)
        int a_img = 0, a_h0 = 0;
        if (conv != CONV_WGRAD) { a_img = m0 / cv_hw; a_h0 = (m0 - a_img * cv_hw) / cv_w; }
        // Filter gradient: 64-row boxes that lie wholly beyond the problem's rows (M = C_out of 64: the second A
        // box) or beyond the last filter tap are not fetched at all.  What the stage then holds there feeds only
        // accumulator rows >= M and columns >= N, which the epilogue never stores.
        uint32_t tx_tile = stage_tx;
        const int p_m = p.M;
        if (conv == CONV_WGRAD) {
          int boxes = 0;
          for (int i = 0; i < BM / 64; ++i) boxes += (m0 + i * 64 < p_m) ? 1 : 0;
          for (int i = 0; i < bnl / 64; ++i) boxes += ((n0 + i * 64) / cv_c < cv_taps) ? 1 : 0;
          tx_tile = (uint32_t)boxes * (BK * 128);
        }
        for (int kb = 0; kb < kb_n; ++kb) {
          if (!(ok = mbar_wait(&sh->empty[stage], phase ^ 1, sh, status))) break;
          uint8_t* a_dst = tiles + stage * STAGE_BYTES;
          uint8_t* b_dst = a_dst + A_BYTES;
          int k0 = kb * BK;
          uint64_t* bar1 = &sh->full[stage];
          uint32_t bar2 = 0;
          if (CG == 1) mbar_expect_tx(bar1, tx_tile);
          else { bar2 = map_to_rank(smem_u32(bar1), 0); mbar_expect_tx_cluster(bar2, tx_tile); }
          auto ld2 = [&](void* dst, const CUtensorMap* map, int x, int y) {
            if (CG == 1) tma_load_2d(dst, map, x, y, bar1); else tma_load_2d_pair(dst, map, x, y, bar2);
          };
          auto ld4 = [&](void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3) {
            if (CG == 1) tma_load_4d(dst, map, c0, c1, c2, c3, bar1); else tma_load_4d_pair(dst, map, c0, c1, c2, c3, bar2);
          };
          if (conv == CONV_WGRAD) {
            // A: dy as an ordinary MN-major operand; B: 64 pixels (whole rows) of x per 64-column block, each
            // column block with the shift of its own filter tap
#pragma unroll
            for (int i = 0; i < BM / 64; ++i)
              if (m0 + i * 64 < p_m) ld2(a_dst + i * (BK * 128), mapA, m0 + i * 64, k0);
            const int kp = cv_k0 + k0;
            const int img = kp / cv_hw, h0 = (kp - img * cv_hw) / cv_w;
            for (int i = 0; i < bnl / 64; ++i) {
              const int col = n0 + i * 64;
              const int t = col / cv_c, c0 = col - t * cv_c;
              if (t < cv_taps) ld4(b_dst + i * (BK * 128), mapB, c0, tap_dj(t), h0 * cv_s + tap_di(t), img);
            }
          } else {
            // k-slice -> (filter tap, channel block); A: 128 pixels shifted by the tap (mirrored for the input gradient)
            const int cb = cv_c >> 6, tap = kb / cb, ch0 = (kb - tap * cb) << 6;
            int di = tap_di(tap), dj = tap_dj(tap);
            if (conv == CONV_DGRAD) { di = -di; dj = -dj; }
            ld4(a_dst, mapA, ch0, dj, a_h0 * cv_s + di, a_img);
            if (conv == CONV_FWD) {
              ld2(b_dst, mapB, k0, n0);                  // filters [N, 9 conv_c], reduction index contiguous
            } else {
              // filters [conv_c, 3, 3, N] read in place: rows = output channel (the reduction), columns (tap, n)
              for (int i = 0; i < bnl / 64; ++i) ld2(b_dst + i * (BK * 128), mapB, tap * p_n + n0 + i * 64, ch0);
            }
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        // copies already issued still land in this CTA's shared memory: give them a bounded time
        unsigned long long t0 = gtime_ns();
        while (gtime_ns() - t0 < 2000000ull) { }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (the pair's leader only)
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      // The issuer runs only a few k-slices ahead of the tensor pipe, so whatever it does between two tiles
      // must be short: the problem's fields stay in registers and are re-read only when the problem changes.
      ProbCursor cur(probs, nprob);
      bool a_mn = false, b_mn = false;
      int kb_n = 0;
      uint32_t idesc = 0;
      int tile_next = my_count > 0 ? tile_at(0) : 0;
      for (; it < my_count && ok; ++it) {
        const int tile = tile_next;
        if (it + 1 < my_count) tile_next = tile_at(it + 1);
        if (cur.seek(tile)) {
          const GemmProb& p = probs[cur.pi];
          a_mn = p.a_ms == 1; b_mn = p.b_ns == 1;
          kb_n = (p.K + BK - 1) / BK;
          idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
                  ((uint32_t)(p.tile_n >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
        }
        // wide tiles own both accumulators (barrier set 0); otherwise the two alternate from tile to tile
        int ab = W ? 0 : (it & 1);
        uint32_t use = W ? (uint32_t)it : (uint32_t)(it >> 1);
        if (!(ok = mbar_wait(&sh->tmem_empty[ab], (use & 1) ^ 1, sh, status))) break;
        tc_fence_after();
        uint32_t d_tmem = tmem_base + ab * BN;
        for (int kb = 0; kb < kb_n; ++kb) {
          if (!(ok = mbar_wait(&sh->full[stage], phase, sh, status))) break;
          tc_fence_after();
          uint32_t a_addr = smem_u32(tiles + stage * STAGE_BYTES);
          uint32_t b_addr = a_addr + A_BYTES;
          uint64_t adesc = make_desc(a_addr, a_mn), bdesc = make_desc(b_addr, b_mn);
          uint32_t a_step = a_mn ? (16 * 128) >> 4 : 32 >> 4;
          uint32_t b_step = b_mn ? (16 * 128) >> 4 : 32 >> 4;
#pragma unroll
          for (int k4 = 0; k4 < BK / 16; ++k4) {
            if (CG == 1) tc_mma(d_tmem, adesc + (uint64_t)(k4 * a_step), bdesc + (uint64_t)(k4 * b_step), idesc, (kb | k4) != 0);
            else {
              // wide: the two column halves of the tile take the same A slice back to back
#pragma unroll
              for (int sb = 0; sb < NB; ++sb)
                tc_mma_pair(d_tmem + sb * BN, adesc + (uint64_t)(k4 * a_step),
                            bdesc + (uint64_t)((sb * B_SUB_BYTES) >> 4) + (uint64_t)(k4 * b_step), idesc, (kb | k4) != 0);
            }
          }
          if (CG == 1) tc_commit(&sh->empty[stage]); else tc_commit_pair(&sh->empty[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) { if (CG == 1) tc_commit(&sh->tmem_full[ab]); else tc_commit_pair(&sh->tmem_full[ab]); }
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(EPI_REGS));
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;            // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    int it = 0;
    bool ok = true;
    ProbCursor cur(probs, nprob);
    TileWalk walk;
    int tile_next = my_count > 0 ? tile_at(0) : 0;
    for (; it < my_count && ok; ++it) {
      const int tile = tile_next;
      if (it + 1 < my_count) tile_next = tile_at(it + 1);
      if (cur.seek(tile)) walk.set(probs[cur.pi], TILE_M);
      const int pi = cur.pi;
      const GemmProb p = probs[pi];          // read-only table: fields are fetched where they are used
      int mt, nt;
      walk.coords(tile, mt, nt);
      int m0 = mt * TILE_M + (int)rank * BM, n0 = nt * (TN / BN) * p.tile_n;
      int ab = W ? 0 : (it & 1);
      uint32_t use = W ? (uint32_t)it : (uint32_t)(it >> 1);
      // Each thread owns one accumulator row and walks this warp's half of the columns 32 at a time;
      // the TMEM load of the next 32 columns and the global load of the next block of the side input
      // (residual or activation-derivative operand) are in flight while the current block is stored.
      const int m = m0 + quarter * 32 + lane;
      const int col0 = ((warp - EPI_FIRST) >> 2) * (TN / 2);
      // 32-column blocks of this warp's half that the tile has: all of them, or for a narrow tile (one MMA of
      // 64 or 128 columns) those of the first half only; always an even number
      const int nblk32 = W ? TN / 64 : max(0, min(TN / 2, p.tile_n - col0)) >> 5;
      const bool vec_ok = (p.ldc % 8 == 0) && (((uintptr_t)p.C & 15) == 0) && (!p.C2 || ((uintptr_t)p.C2 & 15) == 0) &&
                          (!p.resid || ((uintptr_t)p.resid & 15) == 0) && (!p.aux || ((uintptr_t)p.aux & 15) == 0);
      const void* side = (p.resid && !p.aux) ? p.resid : (p.aux && !p.resid) ? p.aux : nullptr;
      uint4 side0[4], side1[4];
      auto fetch_side = [&](uint4* dst, int c) {
        const int nc = n0 + col0 + c * 32;
        if (side && vec_ok && m < p.M && nc + 32 <= p.N) {
          if (p.aux_blocked && side == p.aux) {
            const uint4* blk = (const uint4*)((const bf16*)side + (((size_t)((m0 + quarter * 32) >> 5) * (p.ldc >> 5) + (nc >> 5)) << 10));
#pragma unroll
            for (int q = 0; q < 4; ++q) dst[q] = blk[q * 32 + lane];
          } else {
            const uint4* src = (const uint4*)((const bf16*)side + (size_t)m * p.ldc + nc);
#pragma unroll
            for (int q = 0; q < 4; ++q) dst[q] = src[q];
          }
        }
      };
      fetch_side(side0, 0);                    // on its way while the accumulator is still being produced
      ok = lane == 0 ? mbar_wait(&sh->tmem_full[ab], use & 1, sh, status) : true;   // one poller per warp
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(ab * BN + col0);
      const CUtensorMap* mapC = maps + 4 * pi + 2;
      uint8_t* stg = p.store_tma ? staging + (warp - EPI_FIRST) * 4096 : nullptr;
      const int m_warp0 = m0 + quarter * 32;
      float2 run = make_float2(-INFINITY, 0.f);          // EPI_LOGIT_STATS: this row's statistics over the warp's columns
      auto emit = [&](const uint32_t* a, int c, const uint4* sp) {
        const int nc = n0 + col0 + c * 32;
        if (nc >= p.N || m_warp0 >= p.M) return;            // warp-uniform
        if (vec_ok && nc + 32 <= p.N) epilogue_row32<true>(p, mapC, mapC + 1, stg, m, m_warp0, nc, a, lane, c, run, side, side ? sp : nullptr);
        else epilogue_row32<false>(p, mapC, mapC + 1, stg, m, m_warp0, nc, a, lane, c, run, nullptr, nullptr);
      };
      uint32_t acc0[32], acc1[32];
      if (nblk32 > 0) tc_ld32(trow, acc0);
#pragma unroll 1
      for (int c = 0; c < nblk32; c += 2) {
        tc_wait_ld();
        tc_ld32(trow + (c + 1) * 32, acc1);
        fetch_side(side1, c + 1);
        emit(acc0, c, side0);
        tc_wait_ld();
        if (c + 2 < nblk32) { tc_ld32(trow + (c + 2) * 32, acc0); fetch_side(side0, c + 2); }
        emit(acc1, c + 1, side1);
      }
      if (p.act == EPI_LOGIT_STATS && m < p.M && n0 + col0 < p.N)
        ((float2*)p.C2)[(size_t)m * ((p.N + 127) >> 7) + ((n0 + col0) >> 7)] = run;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CG == 1) mbar_arrive(&sh->tmem_empty[ab]);
        else mbar_arrive_cluster(map_to_rank(smem_u32(&sh->tmem_empty[ab]), 0));   // the leader's MMA warp waits for both CTAs
      }
    }
  }

  if (warp >= EPI_FIRST && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // this warp's TMA stores are done
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();             // neither CTA frees TMEM or exits while the partner may still touch it
  if (warp == 1) {
    tc_fence_after();
    if (CG == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// 2-D bf16 tensor map: inner extent `inner` (contiguous), outer extent `outer` with a row pitch of
// `pitch` elements, box = 64 x box_outer, 128-byte swizzle, zero fill outside the tensor.
bool encode_map(CUtensorMap* out, const void* base, long long inner, long long outer, long long pitch, int box_outer) {
  EncodeFn fn = get_encode();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// 4-D bf16 tensor map of an NHWC activation tensor [n, h, w, c] for the implicit convolution: boxes of
// 64 channels x whole image rows that hold `pixels` pixels (128: a K-major A tile; 64: one k-slice of an
// MN-major B tile), i.e. (w, pixels / w, 1) inside an image or (w, h, pixels / (h w)) across small images.
// 128-byte swizzle; everything outside the tensor (the padding ring of the convolution) reads as zero.
// The boxes are counted in pixels of the OUTPUT image h x w; with a stride s the tensor is the input image
// hin x win and a box steps through it s pixels at a time (traversed extent s times the pixels it delivers).
bool encode_map4(CUtensorMap* out, const void* base, int n, int h, int w, int c, int pixels, int hin, int win, int s) {
  EncodeFn fn = get_encode();
  if (!fn) return false;
  const long long hw = (long long)h * w;
  cuuint32_t bw = (cuuint32_t)w, bh, bn;
  if (hw >= pixels) { bh = (cuuint32_t)(pixels / w); bn = 1; }
  else { bh = (cuuint32_t)h; bn = (cuuint32_t)(pixels / hw); }
  if (bw * s > 256 || bh * s > 256) return false;
  cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)win, (cuuint64_t)hin, (cuuint64_t)n};
  cuuint64_t strides[3] = {(cuuint64_t)c * 2, (cuuint64_t)win * c * 2, (cuuint64_t)hin * win * c * 2};
  cuuint32_t box[4] = {64u, bw * (cuuint32_t)s, bh * (cuuint32_t)s, bn};
  cuuint32_t estr[4] = {1u, (cuuint32_t)s, (cuuint32_t)s, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

bool gemm_tc_eligible(const GemmProb& g) {
  if (g.M < 1 || g.N < 1 || g.K < 1) return false;
  if (g.aux_blocked) {
    const void* u = g.act == EPI_GELU ? g.C2 : g.aux;
    if ((g.act != EPI_GELU && g.act != EPI_GELU_GRAD) || g.resid || g.out_f32 || !u || ((uintptr_t)u & 15) ||
        g.M % 32 || g.N % 32 || g.ldc % 32 || ((uintptr_t)g.C & 15))
      return false;
  }
  if (g.conv != CONV_NONE) {
    // implicit convolution: whole-row boxes, 64-channel k-slices, filters with 16-byte pitches
    if (g.conv_c < 64 || g.conv_c % 64 || g.conv_n < 1 || !conv_boxes_ok(g.conv_h, g.conv_w)) return false;
    if (((uintptr_t)g.A & 15) || ((uintptr_t)g.B & 15)) return false;
    const int s = g.conv_stride > 1 ? g.conv_stride : 1, taps = g.conv_taps ? g.conv_taps : 9;
    const int hin = g.conv_hin ? g.conv_hin : g.conv_h, win = g.conv_win ? g.conv_win : g.conv_w;
    if (s > 2 || (taps != 9 && taps != 1) || g.conv_w * s > 256) return false;
    // the output image is what a convolution with this stride makes of the input image
    // (3x3 with padding 1 and 1x1 without padding give the same size)
    if (g.conv_h != (hin - 1) / s + 1 || g.conv_w != (win - 1) / s + 1) return false;
    const long long pixels = (long long)g.conv_n * g.conv_h * g.conv_w;
    if (g.conv == CONV_FWD) return g.K == taps * g.conv_c && g.M == pixels && g.b_ks == 1 && g.b_ns % 8 == 0 && get_encode() != nullptr;
    if (g.conv == CONV_DGRAD) return s == 1 && taps == 9 && g.K == 9 * g.conv_c && g.M == pixels && g.N % 8 == 0 && get_encode() != nullptr;
    if (g.conv == CONV_WGRAD)
      return g.N == taps * g.conv_c && g.a_ms == 1 && g.a_ks % 8 == 0 && g.conv_k0 % 64 == 0 && g.conv_k0 + g.K <= pixels &&
             get_encode() != nullptr;
    return false;
  }
  if ((long long)g.M * g.N < 64 * 64 || g.K < 32) return false;          // too small to pay for a 128x256 tile
  if (((uintptr_t)g.A & 15) || ((uintptr_t)g.B & 15)) return false;
  long long a_pitch = g.a_ms == 1 ? g.a_ks : g.a_ms, b_pitch = g.b_ns == 1 ? g.b_ks : g.b_ns;
  if (a_pitch % 8 || b_pitch % 8) return false;                          // TMA: pitches are multiples of 16 bytes
  if (g.a_ms != 1 && g.a_ks != 1) return false;
  if (g.b_ns != 1 && g.b_ks != 1) return false;
  return get_encode() != nullptr;
}

int gemm_tc_choose_cg(const GemmProb* probs, int n) {
  for (int i = 0; i < n; ++i)
    if (probs[i].M <= BM) return 1;            // a 256-row pair tile would be half empty
  return 2;
}

bool gemm_tc_wide_ok(const GemmProb& g) {
  // long reductions only (the epilogue of a wide tile is exposed), plain epilogue, columns that fill 512-wide tiles
  return g.K >= 8192 && g.M > BM && g.N % (2 * BN) == 0 && g.act == EPI_NONE && !g.bias && !g.resid && !g.aux &&
         g.conv == CONV_NONE && !g.aux_blocked;
}

int gemm_tc_tiles(GemmProb& g, int tile_start, int cg, int wide) {
  g.tile_start = tile_start;
  // A problem with at most 128 columns (the 64- and 128-channel convolutions of the early ResNet stages) gets
  // one column tile of 64 or 128 instead of 256: the MMA, the B boxes and the accumulator read-back shrink with
  // it.  Every CTA must still receive whole boxes: 64 columns where B arrives in 64-column blocks (MN-major B,
  // the implicit input and filter gradients), 32 rows otherwise.
  g.tile_n = BN;
  if (!wide && g.act != EPI_LOGIT_STATS && g.conv != CONV_WGRAD) {
    const bool blocks64 = g.conv == CONV_NONE ? g.b_ns == 1 : g.conv != CONV_FWD;
    const int unit = (blocks64 ? 64 : 32) * cg;
    if (g.N <= 64 && unit <= 64) g.tile_n = 64;
    else if (g.N <= 128 && unit <= 128) g.tile_n = 128;
  }
  g.tiles_n = (g.N + (wide ? 2 : 1) * g.tile_n - 1) / ((wide ? 2 : 1) * g.tile_n);
  // band height: at least 8 row tiles, more while the band's row panels (tile rows x K) stay within ~32 MB of L2
  const long long panel = (long long)BM * cg * g.K * 2;
  g.raster = (int)std::max(8LL, std::min(4096LL, (32LL << 20) / std::max(panel, 1LL)));
  return ((g.M + BM * cg - 1) / (BM * cg)) * g.tiles_n;
}

// Output map: [M, N] with a pitch of ldc elements, 32x32 boxes, swizzled like the epilogue's staging buffer
// (64-byte rows for bf16, 128-byte rows for fp32).
// `wide`: bf16 boxes of 64 columns (128-byte rows, 128-byte swizzle) filled by two neighbouring column blocks.
bool encode_out_map(CUtensorMap* out, const void* base, long long N, long long M, long long ldc, bool f32, bool wide) {
  EncodeFn fn = get_encode();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  cuuint64_t strides[1] = {(cuuint64_t)ldc * (f32 ? 4 : 2)};
  cuuint32_t box[2] = {wide ? 64u : 32u, 32u};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(out, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  (f32 || wide) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// maps: 4 consecutive 128-byte tensor maps [A, B, C, C2].  Sets g.store_tma.
bool gemm_tc_encode(GemmProb& g, void* maps, int cg) {
  CUtensorMap* mapA = (CUtensorMap*)maps;
  CUtensorMap* mapB = mapA + 1;
  const long long esz = g.out_f32 ? 4 : 2;
  g.store_tma = ((g.ldc * esz) % 16 == 0) && (((uintptr_t)g.C & 15) == 0) &&
                (g.act != EPI_GELU || (((uintptr_t)g.C2 & 15) == 0 && (g.ldc * 2) % 16 == 0));
  if (g.store_tma) {
    // one bf16 output through the staging buffer: pairs of column blocks leave in one store of full 128-byte
    // rows (mode 2); the GELU epilogue's second output shares the buffer unless it is stored in blocks
    const bool two_staged = g.act == EPI_GELU && !g.aux_blocked;
    const bool wide = !g.out_f32 && !two_staged;
    bool ok = encode_out_map(mapA + 2, g.C, g.N, g.M, g.ldc, g.out_f32 != 0, wide);
    if (ok && two_staged) ok = encode_out_map(mapA + 3, g.C2, g.N, g.M, g.ldc, false, false);
    g.store_tma = ok ? (wide ? 2 : 1) : 0;
  }
  bool okA, okB;
  const int cs = g.conv_stride > 1 ? g.conv_stride : 1;
  const int chin = g.conv_hin ? g.conv_hin : g.conv_h, cwin = g.conv_win ? g.conv_win : g.conv_w;
  if (g.conv == CONV_FWD || g.conv == CONV_DGRAD) okA = encode_map4(mapA, g.A, g.conv_n, g.conv_h, g.conv_w, g.conv_c, BM, chin, cwin, cs);
  else if (g.a_ms == 1) okA = encode_map(mapA, g.A, g.M, g.K, g.a_ks, BK);       // MN-major: rows are k
  else okA = encode_map(mapA, g.A, g.K, g.M, g.a_ms, BM);
  if (g.conv == CONV_WGRAD) okB = encode_map4(mapB, g.B, g.conv_n, g.conv_h, g.conv_w, g.conv_c, BK, chin, cwin, cs);
  else if (g.conv == CONV_DGRAD) okB = encode_map(mapB, g.B, 9LL * g.N, g.conv_c, 9LL * g.N, BK);   // rows: output channel
  else if (g.b_ns == 1) okB = encode_map(mapB, g.B, g.N, g.K, g.b_ks, BK);
  else okB = encode_map(mapB, g.B, g.K, g.N, g.b_ns, (g.tile_n ? g.tile_n : BN) / cg);
  return okA && okB;
}

int gemm_tc_grid_units(int total_tiles, int num_sms, int cg) {
  const int units = cg == 1 ? num_sms : num_sms / 2;
  return total_tiles < units ? total_tiles : units;
}

// Longest-processing-time assignment of the launch's tiles to its CTAs (pairs).  A tile costs its k-slices plus a
// few for the epilogue.  Tiles are taken in index order (the caller lists long problems first) and each goes to
// the least loaded unit, the lowest index among equals: for tiles of one length this is exactly the round-robin
// walk of the kernel, so a uniform launch needs no schedule and gets none; nor does a launch whose busiest unit
// would gain less than a tenth.
bool gemm_tc_schedule(const GemmProb* probs, int nprob, int total_tiles, int num_sms, int cg, std::vector<int>& sched,
                      std::vector<int>& off) {
  sched.clear(); off.clear();
  const int units = gemm_tc_grid_units(total_tiles, num_sms, cg);
  if (nprob < 2 || units < 1 || total_tiles <= units) return false;
  std::vector<int> cost(total_tiles);
  int lo = 1 << 30, hi = 0;
  for (int i = 0; i < nprob; ++i) {
    const int end = i + 1 < nprob ? probs[i + 1].tile_start : total_tiles;
    const int c = (probs[i].K + BK - 1) / BK + 4;
    for (int t = probs[i].tile_start; t < end; ++t) cost[t] = c;
    if (end > probs[i].tile_start) { lo = std::min(lo, c); hi = std::max(hi, c); }
  }
  if (hi <= lo + lo / 4) return false;                 // lengths within 25 %: the round-robin walk is as good
  // what the kernel's own walk (unit u takes tiles u, u + units, ...) would make the busiest unit do
  std::vector<long long> rr(units, 0);
  for (int t = 0; t < total_tiles; ++t) rr[t % units] += cost[t];
  const long long rr_max = *std::max_element(rr.begin(), rr.end());
  std::vector<std::vector<int>> lists(units);
  typedef std::pair<long long, int> Load;                // (load, unit): smallest load first, lowest unit among equals
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> q;
  for (int u = 0; u < units; ++u) q.push(Load(0, u));
  for (int t = 0; t < total_tiles; ++t) {
    Load l = q.top(); q.pop();
    lists[l.second].push_back(t);
    q.push(Load(l.first + cost[t], l.second));
  }
  long long lpt_max = 0;
  while (!q.empty()) { lpt_max = std::max(lpt_max, q.top().first); q.pop(); }
  if (lpt_max * 10 > rr_max * 9) return false;          // less than a tenth to gain: keep the walk (and its L2 locality)
  off.push_back(0);
  for (auto& l : lists) { sched.insert(sched.end(), l.begin(), l.end()); off.push_back((int)sched.size()); }
  return true;
}

cudaError_t launch_gemm_tc(const GemmProb* d_probs, const void* d_maps, int nprob, int total_tiles, int* d_status,
                           int num_sms, cudaStream_t s, int cg, int wide, const int* d_sched, const int* d_sched_off) {
  // function attributes belong to a device's context: set once per device and variant
  static bool attr_set_dev[64][4] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  bool* attr_set = attr_set_dev[dev];
  const int which = cg == 1 ? 1 : (wide ? 3 : 2);
  const size_t ring = cg == 1 ? (size_t)Cfg<1, 0>::STAGES * Cfg<1, 0>::STAGE_BYTES
                              : (wide ? (size_t)Cfg<2, 1>::STAGES * Cfg<2, 1>::STAGE_BYTES : (size_t)Cfg<2, 0>::STAGES * Cfg<2, 0>::STAGE_BYTES);
  size_t smem = ring + EPI_WARPS * 4096 + 1024 + sizeof(Shared);
  if (cg == 1 && wide) return cudaErrorInvalidValue;
  if (!attr_set[which]) {
    const void* fn = which == 1 ? (const void*)gemm_tc_kernel<1, 0> : which == 2 ? (const void*)gemm_tc_kernel<2, 0> : (const void*)gemm_tc_kernel<2, 1>;
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // The epilogue warpgroups' register increase must fit into what the launch allocates (threads x
    // compiled register count); otherwise it would wait forever.  Refuse to launch instead.
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, fn);
    if (e != cudaSuccess) return e;
    if (32 * EPI_FIRST * CTRL_REGS + 32 * EPI_WARPS * EPI_REGS > NTHREADS * fa.numRegs) return cudaErrorLaunchOutOfResources;
    attr_set[which] = true;
  }
  if (total_tiles == 0) return cudaSuccess;
  if (cg == 1) {
    int grid = gemm_tc_grid_units(total_tiles, num_sms, 1);
    gemm_tc_kernel<1, 0><<<grid, NTHREADS, smem, s>>>(d_probs, (const CUtensorMap*)d_maps, nprob, total_tiles, d_status,
                                                      d_sched, d_sched_off);
    return cudaGetLastError();
  }
  int pairs = gemm_tc_grid_units(total_tiles, num_sms, 2);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(NTHREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (wide) return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, 1>, d_probs, (const CUtensorMap*)d_maps, nprob, total_tiles, d_status,
                                      d_sched, d_sched_off);
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, 0>, d_probs, (const CUtensorMap*)d_maps, nprob, total_tiles, d_status,
                            d_sched, d_sched_off);
}

}  // namespace lp

#include "../../include/lp.h"

// ---------------------------------------------------------------------------------------------
// lp_gemm_bf16_static: the grouped GEMM for callers that must not allocate device memory.
//
// The grouped kernels read their problem table (and, for the tensor-core kernel, two TMA tensor
// maps per problem and a status word) from global memory.  lp_gemm_bf16 keeps that table in a
// cudaMalloc'ed buffer that grows on demand.  Some callers cannot afford that: serving and
// real-time loops that must not take the driver's allocation lock or the device-wide
// synchronisation cudaMalloc and cudaFree imply, code that runs inside a region whose memory a
// pool manager has already handed out, and hosts whose device-memory budget is fixed up front.
// This variant keeps the table in the file-scope array below instead: a fixed LP_GEMM_STATIC_MAX
// problems, about 58 KB that every GPU loading this library holds until the process exits.
// ---------------------------------------------------------------------------------------------
#include <mutex>

#include "gemm_desc_check.h"

namespace {
using namespace lp;

struct alignas(64) TMap { unsigned char b[128]; };
struct StaticLayout {
  int status;                                   // sticky: kernels OR bits into it, lp_gemm_static_poll clears it
  int pad[63];
  GemmProb tc[LP_GEMM_STATIC_MAX];
  GemmProb alu[LP_GEMM_STATIC_MAX];
  alignas(64) TMap maps[4 * LP_GEMM_STATIC_MAX];
};

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticLayout)];

constexpr int MAX_DEVICES = 64;
StaticLayout* g_static_ptr[MAX_DEVICES] = {};
int g_static_sms[MAX_DEVICES] = {};
thread_local char g_static_err[256] = "";
// Host-side staging of one call's tables (process-wide, so it costs the calling thread no stack);
// the mutex orders calls from different host threads while they fill and upload it.
struct HostStage {
  GemmProb tc[LP_GEMM_STATIC_MAX], alu[LP_GEMM_STATIC_MAX];
  TMap maps[4 * LP_GEMM_STATIC_MAX];
};
HostStage g_stage;
std::mutex g_stage_mutex;

lp_status static_fail(lp_status code, const char* msg, cudaError_t e = cudaSuccess) {
  if (e != cudaSuccess) snprintf(g_static_err, sizeof(g_static_err), "%s: %s", msg, cudaGetErrorString(e));
  else snprintf(g_static_err, sizeof(g_static_err), "%s", msg);
  return code;
}

// Set-up, once per device, with that device current: resolve the array's device address.
lp_status static_setup(int* dev_out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return static_fail(LP_ERR_CUDA, "cudaGetDevice", e);
  if (dev < 0 || dev >= MAX_DEVICES) return static_fail(LP_ERR_UNSUPPORTED, "lp_gemm_bf16_static: device ordinal above 63");
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) return static_fail(LP_ERR_CUDA, "cudaGetSymbolAddress", e);
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return static_fail(LP_ERR_CUDA, "cudaDeviceGetAttribute", e);
    g_static_sms[dev] = sms;
    g_static_ptr[dev] = (StaticLayout*)p;
  }
  *dev_out = dev;
  return LP_OK;
}
}  // namespace

extern "C" const char* lp_gemm_static_last_error(void) { return g_static_err; }

extern "C" lp_status lp_gemm_bf16_static(int n, const lp_gemm_desc* in, void* stream) {
  if (n < 1 || !in) return static_fail(LP_ERR_INVALID_ARG, "lp_gemm_bf16_static: no problems");
  if (n > LP_GEMM_STATIC_MAX) return static_fail(LP_ERR_SHAPE, "lp_gemm_bf16_static: more than LP_GEMM_STATIC_MAX (64) problems in one call");
  for (int i = 0; i < n; ++i)
    if (const char* why = gemm_desc_problem(in[i])) {
      snprintf(g_static_err, sizeof(g_static_err), "lp_gemm_bf16_static: problem %d: %s", i, why);
      return LP_ERR_INVALID_ARG;
    }
  cudaStream_t s = (cudaStream_t)stream;
  int dev = 0;
  lp_status st = static_setup(&dev);
  if (st != LP_OK) return st;
  StaticLayout* sc = g_static_ptr[dev];

  std::lock_guard<std::mutex> lock(g_stage_mutex);
  GemmProb* tc = g_stage.tc;
  GemmProb* alu = g_stage.alu;
  TMap* maps = g_stage.maps;
  int ntc = 0, nalu = 0, tc_tiles = 0, alu_tiles = 0;
  for (int i = 0; i < n; ++i) {
    const lp_gemm_desc& q = in[i];
    GemmProb g{};
    g.A = q.A; g.B = q.B; g.C = q.C; g.C2 = q.C2; g.bias = q.bias; g.resid = q.resid; g.aux = q.aux;
    g.M = q.M; g.N = q.N; g.K = q.K; g.a_ms = q.a_ms; g.a_ks = q.a_ks; g.b_ns = q.b_ns; g.b_ks = q.b_ks;
    g.ldc = q.ldc; g.act = q.act; g.out_f32 = q.out_f32;
    if (gemm_tc_eligible(g)) {
      tc_tiles += gemm_tc_tiles(g, tc_tiles);
      if (!gemm_tc_encode(g, &maps[4 * ntc], 1)) return static_fail(LP_ERR_CUDA, "cuTensorMapEncodeTiled failed");
      tc[ntc++] = g;
    } else {
      g.tiles_n = (g.N + 63) / 64;
      g.tile_start = alu_tiles;
      alu_tiles += ((g.M + 63) / 64) * g.tiles_n;
      alu[nalu++] = g;
    }
  }
  // The device array keeps whatever the previous call left; the table entries this call uses are
  // overwritten.  The staging table is pageable host memory: the runtime has copied it out by the
  // time cudaMemcpyAsync returns, so the next call may refill it.
  cudaError_t e = cudaSuccess;
  if (ntc) {
    e = cudaMemcpyAsync(sc->tc, tc, ntc * sizeof(GemmProb), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sc->maps, maps, 4 * ntc * sizeof(TMap), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = launch_gemm_tc(sc->tc, sc->maps, ntc, tc_tiles, &sc->status, g_static_sms[dev], s);
    if (e != cudaSuccess) return static_fail(LP_ERR_CUDA, "tensor-core launch", e);
  }
  if (nalu) {
    e = cudaMemcpyAsync(sc->alu, alu, nalu * sizeof(GemmProb), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return static_fail(LP_ERR_CUDA, "cudaMemcpyAsync", e);
    launch_gemm_simt(sc->alu, alu, nalu, true, s);
    e = cudaGetLastError();
    if (e != cudaSuccess) return static_fail(LP_ERR_CUDA, "FP32-ALU launch", e);
  }
  return LP_OK;
}

extern "C" lp_status lp_gemm_static_poll(void* stream) {
  int dev = 0;
  lp_status st = static_setup(&dev);
  if (st != LP_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  int w = 0;
  cudaError_t e = cudaMemcpyAsync(&w, &g_static_ptr[dev]->status, sizeof(int), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(&g_static_ptr[dev]->status, 0, sizeof(int), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return static_fail(LP_ERR_CUDA, "lp_gemm_static_poll", e);
  if (w & ST_TIMEOUT) return static_fail(LP_ERR_TIMEOUT, "lp_gemm_static_poll: a device-side wait gave up; outputs of the calls since the last poll are not valid");
  return LP_OK;
}
