// Causal multi-head attention for bf16 activations (App. B.2's transformer layers), heads of 64, on the
// 5th-generation tensor cores (tcgen05) with the score tiles in tensor memory.
//
// Three kernels, all flash-style (no T x T matrix ever reaches global memory) and free of atomics:
//   forward : one block per (sequence, head, 128 query rows).  Per 128-key tile: S = Q K^T is formed in tensor
//             memory by one elected thread (tcgen05.mma, operands staged by TMA); 128 row threads -- thread r owns
//             query row r, which is lane r of tensor memory, so a row's maximum and sum need no shuffles -- read
//             S with tcgen05.ld, keep the running maximum and sum of the online softmax, and write the
//             probabilities back to tensor memory as bf16 (tcgen05.st), where the second product O_tile = P V
//             reads them as its A operand; the row threads add O_tile into their fp32 output row, rescaled when
//             the maximum moved.  Saves the row's log-sum-exp (base 2) for the backward kernels.
//   dQ      : one block per 128 query rows, 64-key tiles.  S = Q K^T and dP = dO V^T in tensor memory; the row
//             threads recompute P = exp2(S - lse), form dS = P (dP - delta) and write it back as bf16; dQ += dS K
//             accumulates in tensor memory over all key tiles.  Also writes delta = rowsum(dO * O).
//   dK, dV  : one block per 128 key rows, 64-query tiles, on the transposed tiles: S^T = K Q^T, dP^T = V dO^T;
//             the row threads (one key each) write P^T and dS^T over S^T and dP^T; dV += P^T dO and
//             dK += dS^T Q accumulate in tensor memory over all query tiles that see these keys.
// Blocks hold 256 of the 512 tensor-memory columns and under 100 KB of shared memory, so two are resident per SM:
// one block's softmax runs while the other's products do.
//
// qkv is [B, T, 3*H*64]: columns [0, d) queries, [d, 2d) keys, [2d, 3d) values, head h at h*64.  Tiles are
// fetched through 3-D tensor maps (column, position, sequence) in boxes of 64 positions; positions past the
// end of a sequence read as zero.  Every wait on an mbarrier is bounded (see tc::mbar_wait): on expiry the
// TIMEOUT bit of the status word is raised, all roles leave their loops, tensor memory is freed and the kernel
// returns.
#include <algorithm>
#include <cstring>

#include "common.cuh"
#include "tc_prims.cuh"

namespace lp {
namespace {
using namespace tc;

constexpr int DH = 64;
constexpr float SCALE = 0.125f;                     // 1/sqrt(64)
constexpr float LOG2E = 1.4426950408889634f;
constexpr float SL2 = SCALE * LOG2E;                // scores are used in base-2 units: s2 = s * SL2
constexpr int NTHREADS = 192;                       // warps 0-3: row threads; warp 4: TMA producer; warp 5: MMA issuer
constexpr int ROW_WARPS = 4;
constexpr uint32_t TMEM_COLS = 256;
constexpr int BOX_BYTES = 64 * 128;                 // one TMA box: 64 positions x 64 bf16
constexpr size_t MIN_SMEM = 78 * 1024;              // no third block fits on an SM beside two of these

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) { return (uint8_t*)(((uintptr_t)p + 1023) & ~(uintptr_t)1023); }
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&v;
}
// One poller per warp; the whole warp learns the outcome.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, int* abort_flag, int* status, int lane) {
  bool ok = lane == 0 ? mbar_wait(bar, parity, abort_flag, status) : true;
  return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(TMEM_COLS) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t base) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(TMEM_COLS) : "memory");
}
// Copies already issued by an aborting producer still land in this block's shared memory: give them time.
__device__ __forceinline__ void drain_copies() {
  unsigned long long t0 = gtime_ns();
  while (gtime_ns() - t0 < 2000000ull) { }
}
// Row `row` of a [*, ld] bf16 matrix: 64 values scaled by `mul`, as eight 16-byte stores.
__device__ __forceinline__ void store_row64(bf16* dst, const float* v, float mul) {
#pragma unroll
  for (int q = 0; q < 8; ++q)
    *(uint4*)(dst + q * 8) = make_uint4(pack2(v[8 * q] * mul, v[8 * q + 1] * mul), pack2(v[8 * q + 2] * mul, v[8 * q + 3] * mul),
                                        pack2(v[8 * q + 4] * mul, v[8 * q + 5] * mul), pack2(v[8 * q + 6] * mul, v[8 * q + 7] * mul));
}

// ------------------------------------------------------------------------------------------ forward
struct __align__(8) FwdShared {
  uint64_t q_full, kv_full[2], kv_empty[2], s_full, p_full, o_full;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int FWD_TILES = 16384 + 2 * 16384 + 2 * 16384;     // Q, two stages of K, two stages of V
constexpr uint32_t F_S = 0, F_O = 128, F_P = 192;            // tensor-memory columns: S (128 fp32), O tile (64), P (64 packed)

__global__ void __launch_bounds__(NTHREADS, 2) attn_fwd_tc_kernel(const AttnTcProb* __restrict__ probs, int* status) {
  const AttnTcProb& pb = probs[blockIdx.z];
  const AttnProb pr = pb.p;
  const int qt = gridDim.x - 1 - blockIdx.x, q0 = qt * 128;    // heaviest query tiles (most keys) first
  if ((int)blockIdx.y >= pr.B * pr.H || q0 >= pr.T) return;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sQ = align1024(smem_raw);
  uint8_t* sK = sQ + 16384;
  uint8_t* sV = sK + 2 * 16384;
  FwdShared* sh = (FwdShared*)(sV + 2 * 16384);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const int nk = qt + 1;                                       // 128-key tiles this query tile sees
  const CUtensorMap* map = (const CUtensorMap*)pb.map_qkv;

  if (threadIdx.x == 0) {
    mbar_init(&sh->q_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&sh->kv_full[s], 1); mbar_init(&sh->kv_empty[s], 1); }
    mbar_init(&sh->s_full, 1); mbar_init(&sh->p_full, ROW_WARPS); mbar_init(&sh->o_full, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(&sh->tmem_base);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)&sh->tmem_base;

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(&sh->q_full, 16384);
      tma_load_3d(sQ, map, h * DH, q0, b, &sh->q_full);
      tma_load_3d(sQ + BOX_BYTES, map, h * DH, q0 + 64, b, &sh->q_full);
      for (int j = 0; j < nk && ok; ++j) {
        const int st = j & 1;
        if (!(ok = mbar_wait(&sh->kv_empty[st], ((j >> 1) & 1) ^ 1, &sh->abort_flag, status))) break;
        mbar_expect_tx(&sh->kv_full[st], 32768);
        tma_load_3d(sK + st * 16384, map, d + h * DH, j * 128, b, &sh->kv_full[st]);
        tma_load_3d(sK + st * 16384 + BOX_BYTES, map, d + h * DH, j * 128 + 64, b, &sh->kv_full[st]);
        tma_load_3d(sV + st * 16384, map, 2 * d + h * DH, j * 128, b, &sh->kv_full[st]);
        tma_load_3d(sV + st * 16384 + BOX_BYTES, map, 2 * d + h * DH, j * 128 + 64, b, &sh->kv_full[st]);
      }
      if (!ok) drain_copies();
    }
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = make_idesc(128, 128, false, false), idesc_pv = make_idesc(128, 64, false, true);
      bool ok = mbar_wait(&sh->q_full, 0, &sh->abort_flag, status);
      const uint64_t dq = make_desc(smem_u32(sQ), false, 0);
      for (int j = 0; j < nk && ok; ++j) {
        const int st = j & 1;
        if (!(ok = mbar_wait(&sh->kv_full[st], (j >> 1) & 1, &sh->abort_flag, status))) break;
        tc_fence_after();
        const uint64_t dk = make_desc(smem_u32(sK + st * 16384), false, 0);
        const uint64_t dv = make_desc(smem_u32(sV + st * 16384), true, 16384);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + F_S, dq + (uint64_t)(k4 * 2), dk + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
        tc_commit(&sh->s_full);
        // the row threads have read S, written P and taken the previous O tile
        if (!(ok = mbar_wait(&sh->p_full, j & 1, &sh->abort_flag, status))) break;
        tc_fence_after();
#pragma unroll
        for (int k8 = 0; k8 < 8; ++k8) tc_mma_ts(tmem + F_O, tmem + F_P + k8 * 8, dv + (uint64_t)(k8 * 128), idesc_pv, k8 != 0);
        tc_commit(&sh->kv_empty[st]);
        tc_commit(&sh->o_full);
      }
    }
  } else {
    // ---------------------------------------------------------------- row threads: thread r owns query row q0 + r
    const int row = warp * 32 + lane, grow = q0 + row;
    const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
    float o[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) o[i] = 0.f;
    float m_run = -INFINITY, l = 0.f, c_prev = 0.f;
    bool ok = true;
    uint32_t v[32];
    auto take_o_tile = [&](float c) {                       // o = o * c + O tile
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        tc_ld32(trow + F_O + hh * 32, v);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[hh * 32 + i] = fmaf(o[hh * 32 + i], c, __uint_as_float(v[i]));
      }
    };
    for (int j = 0; j < nk; ++j) {
      if (!(ok = warp_wait(&sh->s_full, j & 1, &sh->abort_flag, status, lane))) break;
      tc_fence_after();
      const bool diag = j == qt;                             // only the last key tile crosses the diagonal
      const int rel = grow - j * 128;                        // columns above `rel` are in the future of this row
      float mx = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        tc_ld32(trow + F_S + c * 32, v);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float s = __uint_as_float(v[i]);
          if (diag && c * 32 + i > rel) s = -INFINITY;
          mx = fmaxf(mx, s);
        }
      }
      const float m_new = fmaxf(m_run, mx * SL2);            // column 0 of the diagonal tile is never masked: finite
      const float cfac = ex2_approx(m_run - m_new);
      float rowsum = 0.f;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        tc_ld32(trow + F_S + c * 32, v);
        tc_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float s0 = __uint_as_float(v[i]), s1 = __uint_as_float(v[i + 1]);
          if (diag && c * 32 + i > rel) s0 = -INFINITY;
          if (diag && c * 32 + i + 1 > rel) s1 = -INFINITY;
          const float p0 = ex2_approx(fmaf(s0, SL2, -m_new)), p1 = ex2_approx(fmaf(s1, SL2, -m_new));
          rowsum += p0 + p1;
          pk[i >> 1] = pack2(p0, p1);
        }
        tc_st16(trow + F_P + c * 16, pk);
      }
      l = fmaf(l, cfac, rowsum);
      if (j > 0) {
        // the previous tile's product has completed (the tensor pipe runs in order and S of this tile is there)
        if (!(ok = warp_wait(&sh->o_full, (j - 1) & 1, &sh->abort_flag, status, lane))) break;
        tc_fence_after();
        take_o_tile(c_prev);
      }
      c_prev = cfac;
      m_run = m_new;
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->p_full);
    }
    if (ok) ok = warp_wait(&sh->o_full, (nk - 1) & 1, &sh->abort_flag, status, lane);
    if (ok) {
      tc_fence_after();
      take_o_tile(c_prev);
      if (grow < T) {
        store_row64((bf16*)pr.o + ((size_t)b * T + grow) * d + (size_t)h * DH, o, 1.f / l);
        pr.lse[((size_t)b * pr.H + h) * T + grow] = m_run + log2f(l);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_free(tmem); }
}

// ------------------------------------------------------------------------------------------ backward: dQ
struct __align__(8) DqShared {
  uint64_t qdo_full, kv_full[2], kv_empty[2], sdp_full, ds_full, dq_full;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int DQ_TILES = 2 * 16384 + 4 * BOX_BYTES;          // Q, dO, two stages of (K, V) boxes
constexpr uint32_t Q_S = 0, Q_DP = 64, Q_DS = 128, Q_DQ = 192;   // S (64 fp32), dP (64), dS (32 packed), dQ (64)

__global__ void __launch_bounds__(NTHREADS, 2) attn_bwd_dq_tc_kernel(const AttnTcProb* __restrict__ probs, int* status) {
  const AttnTcProb& pb = probs[blockIdx.z];
  const AttnProb pr = pb.p;
  const int qt = gridDim.x - 1 - blockIdx.x, q0 = qt * 128;
  if ((int)blockIdx.y >= pr.B * pr.H || q0 >= pr.T) return;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sQ = align1024(smem_raw);
  uint8_t* sdO = sQ + 16384;
  uint8_t* sK = sdO + 16384;                                   // stage st at + st * BOX_BYTES
  uint8_t* sV = sK + 2 * BOX_BYTES;
  DqShared* sh = (DqShared*)(sV + 2 * BOX_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const int nk = (min(T, q0 + 128) + 63) >> 6;                 // 64-key tiles up to the diagonal
  const CUtensorMap* map = (const CUtensorMap*)pb.map_qkv;
  const CUtensorMap* map_do = (const CUtensorMap*)pb.map_do;

  if (threadIdx.x == 0) {
    mbar_init(&sh->qdo_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&sh->kv_full[s], 1); mbar_init(&sh->kv_empty[s], 1); }
    mbar_init(&sh->sdp_full, 1); mbar_init(&sh->ds_full, ROW_WARPS); mbar_init(&sh->dq_full, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(&sh->tmem_base);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)&sh->tmem_base;

  if (warp == 4) {
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(&sh->qdo_full, 32768);
      tma_load_3d(sQ, map, h * DH, q0, b, &sh->qdo_full);
      tma_load_3d(sQ + BOX_BYTES, map, h * DH, q0 + 64, b, &sh->qdo_full);
      tma_load_3d(sdO, map_do, h * DH, q0, b, &sh->qdo_full);
      tma_load_3d(sdO + BOX_BYTES, map_do, h * DH, q0 + 64, b, &sh->qdo_full);
      for (int j = 0; j < nk && ok; ++j) {
        const int st = j & 1;
        if (!(ok = mbar_wait(&sh->kv_empty[st], ((j >> 1) & 1) ^ 1, &sh->abort_flag, status))) break;
        mbar_expect_tx(&sh->kv_full[st], 2 * BOX_BYTES);
        tma_load_3d(sK + st * BOX_BYTES, map, d + h * DH, j * 64, b, &sh->kv_full[st]);
        tma_load_3d(sV + st * BOX_BYTES, map, 2 * d + h * DH, j * 64, b, &sh->kv_full[st]);
      }
      if (!ok) drain_copies();
    }
  } else if (warp == 5) {
    if (lane == 0) {
      const uint32_t idesc_s = make_idesc(128, 64, false, false), idesc_acc = make_idesc(128, 64, false, true);
      bool ok = mbar_wait(&sh->qdo_full, 0, &sh->abort_flag, status);
      const uint64_t dq = make_desc(smem_u32(sQ), false, 0), ddo = make_desc(smem_u32(sdO), false, 0);
      for (int j = 0; j < nk && ok; ++j) {
        const int st = j & 1;
        if (!(ok = mbar_wait(&sh->kv_full[st], (j >> 1) & 1, &sh->abort_flag, status))) break;
        tc_fence_after();
        const uint64_t dk = make_desc(smem_u32(sK + st * BOX_BYTES), false, 0), dv = make_desc(smem_u32(sV + st * BOX_BYTES), false, 0);
        const uint64_t dk_mn = make_desc(smem_u32(sK + st * BOX_BYTES), true, BOX_BYTES);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + Q_S, dq + (uint64_t)(k4 * 2), dk + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + Q_DP, ddo + (uint64_t)(k4 * 2), dv + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
        tc_commit(&sh->sdp_full);
        if (!(ok = mbar_wait(&sh->ds_full, j & 1, &sh->abort_flag, status))) break;
        tc_fence_after();
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma_ts(tmem + Q_DQ, tmem + Q_DS + k4 * 8, dk_mn + (uint64_t)(k4 * 128), idesc_acc, (j | k4) != 0);
        tc_commit(&sh->kv_empty[st]);
      }
      if (ok) tc_commit(&sh->dq_full);
    }
  } else {
    const int row = warp * 32 + lane, grow = q0 + row;
    const bool live = grow < T;
    const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
    // delta = sum_c dO[row, c] * O[row, c] (read from global memory: 128 contiguous bytes each), and the row's log-sum-exp
    float delta = 0.f, lse = 0.f;
    if (live) {
      const uint4* gdo = (const uint4*)((const bf16*)pr.dout + ((size_t)b * T + grow) * d + (size_t)h * DH);
      const uint4* go = (const uint4*)((const bf16*)pr.o + ((size_t)b * T + grow) * d + (size_t)h * DH);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        uint4 a = gdo[q], c = go[q];
        const __nv_bfloat162* ha = (const __nv_bfloat162*)&a;
        const __nv_bfloat162* hc = (const __nv_bfloat162*)&c;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          float2 fa = __bfloat1622float2(ha[t]), fc = __bfloat1622float2(hc[t]);
          delta = fmaf(fa.x, fc.x, delta);
          delta = fmaf(fa.y, fc.y, delta);
        }
      }
      lse = pr.lse[((size_t)b * pr.H + h) * T + grow];
      pr.delta[((size_t)b * pr.H + h) * T + grow] = delta;
    }
    bool ok = true;
    uint32_t vs[32], vd[32];
    for (int j = 0; j < nk; ++j) {
      if (!(ok = warp_wait(&sh->sdp_full, j & 1, &sh->abort_flag, status, lane))) break;
      tc_fence_after();
      const bool edge = j * 64 + 63 > q0;                     // some column of this tile lies above some row's diagonal
      const int rel = grow - j * 64;
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        tc_ld32(trow + Q_S + c * 32, vs);
        tc_ld32(trow + Q_DP + c * 32, vd);
        tc_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float p0 = ex2_approx(fmaf(__uint_as_float(vs[i]), SL2, -lse)), p1 = ex2_approx(fmaf(__uint_as_float(vs[i + 1]), SL2, -lse));
          if (!live || (edge && c * 32 + i > rel)) p0 = 0.f;
          if (!live || (edge && c * 32 + i + 1 > rel)) p1 = 0.f;
          pk[i >> 1] = pack2(p0 * (__uint_as_float(vd[i]) - delta), p1 * (__uint_as_float(vd[i + 1]) - delta));
        }
        tc_st16(trow + Q_DS + c * 16, pk);
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->ds_full);
    }
    if (ok) ok = warp_wait(&sh->dq_full, 0, &sh->abort_flag, status, lane);
    if (ok) {
      tc_fence_after();
      float acc[64];
      tc_ld32(trow + Q_DQ, vs);
      tc_ld32(trow + Q_DQ + 32, vd);
      tc_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) { acc[i] = __uint_as_float(vs[i]); acc[32 + i] = __uint_as_float(vd[i]); }
      if (live) store_row64((bf16*)pr.dqkv + ((size_t)b * T + grow) * 3 * d + (size_t)h * DH, acc, SCALE);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_free(tmem); }
}

// ------------------------------------------------------------------------------------------ backward: dK, dV
struct __align__(8) DkvShared {
  uint64_t kv_full, q_full[2], q_empty[2], sdp_full, ps_full, dkv_full, ld_full[2];
  uint32_t tmem_base;
  int abort_flag;
  float lse[2][64], delta[2][64];
};
constexpr int DKV_TILES = 2 * 16384 + 4 * BOX_BYTES;         // K, V, two stages of (Q, dO) boxes
// S^T (64 fp32; P^T is written over its first 32 columns), dP^T (64; dS^T over its first 32), dV (64), dK (64)
constexpr uint32_t K_ST = 0, K_DPT = 64, K_DV = 128, K_DK = 192;

__global__ void __launch_bounds__(NTHREADS, 2) attn_bwd_dkv_tc_kernel(const AttnTcProb* __restrict__ probs, int* status) {
  const AttnTcProb& pb = probs[blockIdx.z];
  const AttnProb pr = pb.p;
  const int kt = blockIdx.x, k0 = kt * 128;                    // the first key tile is seen by all queries: heaviest first
  if ((int)blockIdx.y >= pr.B * pr.H || k0 >= pr.T) return;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sK = align1024(smem_raw);
  uint8_t* sV = sK + 16384;
  uint8_t* sQ = sV + 16384;                                    // stage st at + st * BOX_BYTES
  uint8_t* sdO = sQ + 2 * BOX_BYTES;
  DkvShared* sh = (DkvShared*)(sdO + 2 * BOX_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const int j0 = k0 >> 6, nq = ((T + 63) >> 6) - j0;           // 64-query tiles from the diagonal to the end
  const CUtensorMap* map = (const CUtensorMap*)pb.map_qkv;
  const CUtensorMap* map_do = (const CUtensorMap*)pb.map_do;

  if (threadIdx.x == 0) {
    mbar_init(&sh->kv_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&sh->q_full[s], 1); mbar_init(&sh->q_empty[s], 1); mbar_init(&sh->ld_full[s], 32 * ROW_WARPS); }
    mbar_init(&sh->sdp_full, 1); mbar_init(&sh->ps_full, ROW_WARPS); mbar_init(&sh->dkv_full, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(&sh->tmem_base);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)&sh->tmem_base;

  if (warp == 4) {
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(&sh->kv_full, 32768);
      tma_load_3d(sK, map, d + h * DH, k0, b, &sh->kv_full);
      tma_load_3d(sK + BOX_BYTES, map, d + h * DH, k0 + 64, b, &sh->kv_full);
      tma_load_3d(sV, map, 2 * d + h * DH, k0, b, &sh->kv_full);
      tma_load_3d(sV + BOX_BYTES, map, 2 * d + h * DH, k0 + 64, b, &sh->kv_full);
      for (int jj = 0; jj < nq && ok; ++jj) {
        const int st = jj & 1;
        if (!(ok = mbar_wait(&sh->q_empty[st], ((jj >> 1) & 1) ^ 1, &sh->abort_flag, status))) break;
        mbar_expect_tx(&sh->q_full[st], 2 * BOX_BYTES);
        tma_load_3d(sQ + st * BOX_BYTES, map, h * DH, (j0 + jj) * 64, b, &sh->q_full[st]);
        tma_load_3d(sdO + st * BOX_BYTES, map_do, h * DH, (j0 + jj) * 64, b, &sh->q_full[st]);
      }
      if (!ok) drain_copies();
    }
  } else if (warp == 5) {
    if (lane == 0) {
      const uint32_t idesc_s = make_idesc(128, 64, false, false), idesc_acc = make_idesc(128, 64, false, true);
      bool ok = mbar_wait(&sh->kv_full, 0, &sh->abort_flag, status);
      const uint64_t dk = make_desc(smem_u32(sK), false, 0), dv = make_desc(smem_u32(sV), false, 0);
      for (int jj = 0; jj < nq && ok; ++jj) {
        const int st = jj & 1;
        if (!(ok = mbar_wait(&sh->q_full[st], (jj >> 1) & 1, &sh->abort_flag, status))) break;
        tc_fence_after();
        const uint32_t aq = smem_u32(sQ + st * BOX_BYTES), ado = smem_u32(sdO + st * BOX_BYTES);
        const uint64_t dq = make_desc(aq, false, 0), ddo = make_desc(ado, false, 0);
        const uint64_t dq_mn = make_desc(aq, true, BOX_BYTES), ddo_mn = make_desc(ado, true, BOX_BYTES);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + K_ST, dk + (uint64_t)(k4 * 2), dq + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + K_DPT, dv + (uint64_t)(k4 * 2), ddo + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
        tc_commit(&sh->sdp_full);
        if (!(ok = mbar_wait(&sh->ps_full, jj & 1, &sh->abort_flag, status))) break;
        tc_fence_after();
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma_ts(tmem + K_DV, tmem + K_ST + k4 * 8, ddo_mn + (uint64_t)(k4 * 128), idesc_acc, (jj | k4) != 0);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) tc_mma_ts(tmem + K_DK, tmem + K_DPT + k4 * 8, dq_mn + (uint64_t)(k4 * 128), idesc_acc, (jj | k4) != 0);
        tc_commit(&sh->q_empty[st]);
      }
      if (ok) tc_commit(&sh->dkv_full);
    }
  } else {
    const int row = warp * 32 + lane, gkey = k0 + row;
    const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
    // the 128 row threads fetch the query tile's log-sum-exp (threads 0-63) and delta (64-127) one tile ahead
    const int idx = threadIdx.x & 63;
    const float* src = (threadIdx.x < 64 ? pr.lse : pr.delta) + ((size_t)b * pr.H + h) * T;
    auto fetch = [&](int j) { const int q = j * 64 + idx; return q < T ? src[q] : 0.f; };
    float nxt = fetch(j0);
    bool ok = true;
    uint32_t vs[32], vd[32];
    for (int jj = 0; jj < nq; ++jj) {
      const int buf = jj & 1, q0j = (j0 + jj) * 64;
      (threadIdx.x < 64 ? sh->lse[buf] : sh->delta[buf])[idx] = nxt;
      mbar_arrive(&sh->ld_full[buf]);
      if (jj + 1 < nq) nxt = fetch(j0 + jj + 1);
      if (!(ok = warp_wait(&sh->ld_full[buf], (jj >> 1) & 1, &sh->abort_flag, status, lane))) break;
      if (!(ok = warp_wait(&sh->sdp_full, jj & 1, &sh->abort_flag, status, lane))) break;
      tc_fence_after();
      const bool edge = q0j < k0 + 128 || q0j + 64 > T;       // the tile crosses the diagonal or the end of the sequence
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        tc_ld32(trow + K_ST + c * 32, vs);
        tc_ld32(trow + K_DPT + c * 32, vd);
        tc_wait_ld();
        uint32_t pp[16], pd[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float2 ls = *(const float2*)&sh->lse[buf][c * 32 + i], dl = *(const float2*)&sh->delta[buf][c * 32 + i];
          float p0 = ex2_approx(fmaf(__uint_as_float(vs[i]), SL2, -ls.x)), p1 = ex2_approx(fmaf(__uint_as_float(vs[i + 1]), SL2, -ls.y));
          if (edge) {
            const int q = q0j + c * 32 + i;
            if (gkey > q || q >= T) p0 = 0.f;
            if (gkey > q + 1 || q + 1 >= T) p1 = 0.f;
          }
          pp[i >> 1] = pack2(p0, p1);
          pd[i >> 1] = pack2(p0 * (__uint_as_float(vd[i]) - dl.x), p1 * (__uint_as_float(vd[i + 1]) - dl.y));
        }
        tc_st16(trow + K_ST + c * 16, pp);                   // P^T over the part of S^T already read
        tc_st16(trow + K_DPT + c * 16, pd);                  // dS^T over the part of dP^T already read
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->ps_full);
    }
    if (ok) ok = warp_wait(&sh->dkv_full, 0, &sh->abort_flag, status, lane);
    if (ok) {
      tc_fence_after();
      float acc[64];
      bf16* out = (bf16*)pr.dqkv + ((size_t)b * T + gkey) * 3 * d + (size_t)h * DH;
      tc_ld32(trow + K_DV, vs);
      tc_ld32(trow + K_DV + 32, vd);
      tc_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) { acc[i] = __uint_as_float(vs[i]); acc[32 + i] = __uint_as_float(vd[i]); }
      if (gkey < T) store_row64(out + 2 * d, acc, 1.f);
      tc_ld32(trow + K_DK, vs);
      tc_ld32(trow + K_DK + 32, vd);
      tc_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) { acc[i] = __uint_as_float(vs[i]); acc[32 + i] = __uint_as_float(vd[i]); }
      if (gkey < T) store_row64(out + d, acc, SCALE);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_free(tmem); }
}

// 3-D bf16 tensor map of a [B, T, width] activation: boxes of 64 columns x 64 positions of one sequence,
// 128-byte swizzle, zero fill outside the tensor.
bool encode_seq_map(void* out, const void* base, int B, int T, long long width) {
  EncodeFn fn = get_encode();
  if (!fn || ((uintptr_t)base & 15) || (width * 2) % 16) return false;
  cuuint64_t dims[3] = {(cuuint64_t)width, (cuuint64_t)T, (cuuint64_t)B};
  cuuint64_t strides[2] = {(cuuint64_t)width * 2, (cuuint64_t)T * width * 2};
  cuuint32_t box[3] = {64u, 64u, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = fn((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int KERNEL_ID>
cudaError_t prepare(const void* kern, size_t smem) {
  // function attributes belong to a device's context: set once per device and kernel
  static bool done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (done[dev]) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess) done[dev] = true;
  return e;
}

}  // namespace

bool attn_tc_encode(AttnTcProb& out, const AttnProb& p) {
  memset(&out, 0, sizeof(out));
  out.p = p;
  const long long d = (long long)p.H * DH;
  if (p.B < 1 || p.T < 1 || p.H < 1 || !p.qkv) return false;
  if (!encode_seq_map(out.map_qkv, p.qkv, p.B, p.T, 3 * d)) return false;
  if (p.dout && !encode_seq_map(out.map_do, p.dout, p.B, p.T, d)) return false;
  return true;
}

cudaError_t launch_attn_fwd_tc(const AttnTcProb* d, int n, int maxB, int maxT, int maxH, int* status, cudaStream_t s) {
  const size_t smem = std::max(MIN_SMEM, (size_t)FWD_TILES + 1024 + sizeof(FwdShared));
  cudaError_t e = prepare<0>((const void*)attn_fwd_tc_kernel, smem);
  if (e != cudaSuccess) return e;
  dim3 grid((maxT + 127) / 128, maxB * maxH, n);
  attn_fwd_tc_kernel<<<grid, NTHREADS, smem, s>>>(d, status);
  return cudaGetLastError();
}

cudaError_t launch_attn_bwd_tc(const AttnTcProb* d, int n, int maxB, int maxT, int maxH, int* status, cudaStream_t s) {
  const size_t smem_q = std::max(MIN_SMEM, (size_t)DQ_TILES + 1024 + sizeof(DqShared));
  const size_t smem_kv = std::max(MIN_SMEM, (size_t)DKV_TILES + 1024 + sizeof(DkvShared));
  cudaError_t e = prepare<1>((const void*)attn_bwd_dq_tc_kernel, smem_q);
  if (e == cudaSuccess) e = prepare<2>((const void*)attn_bwd_dkv_tc_kernel, smem_kv);
  if (e != cudaSuccess) return e;
  dim3 grid((maxT + 127) / 128, maxB * maxH, n);
  attn_bwd_dq_tc_kernel<<<grid, NTHREADS, smem_q, s>>>(d, status);     // writes delta, which the second kernel reads
  attn_bwd_dkv_tc_kernel<<<grid, NTHREADS, smem_kv, s>>>(d, status);
  return cudaGetLastError();
}

}  // namespace lp
