// Causal multi-head attention for bf16 activations on the tensor cores (warp-level mma through
// the wmma interface), heads of 64, flash-style: 64x64 score tiles live only in shared memory.
//
// Forward runs two passes over the visible key tiles: pass 1 finds each row's log-sum-exp with an
// online (max, sum) update, pass 2 forms P = exp(S - lse) (already normalised, so the output
// accumulators never need rescaling) and O += P V.  Backward recomputes P from Q, K and the saved
// log-sum-exp: one kernel per query tile for dQ, one per key tile for dK and dV; no atomics, every
// sum has a fixed order.
//
// qkv is [B*T, 3*H*64]: columns [0, d) queries, [d, 2d) keys, [2d, 3d) values, head h at h*64.
#include <mma.h>

#include "common.cuh"

namespace lp {
namespace {
using namespace nvcuda;

constexpr int DH = 64, TQ = 64, TK = 64;
constexpr int LDB = 72;   // bf16 tile pitch (elements)
constexpr int LDF = 68;   // fp32 tile pitch
constexpr float SCALE = 0.125f;

typedef wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> FragA;
typedef wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::col_major> FragAT;
typedef wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> FragB;
typedef wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::col_major> FragBT;
typedef wmma::fragment<wmma::accumulator, 16, 16, 16, float> FragC;

// Copy a 64x64 bf16 tile (rows r0.., row pitch ld elements) into shared memory; rows >= rmax read as zero.
__device__ __forceinline__ void load_tile_bf16(bf16* dst, const bf16* src, size_t ld, int r0, int rmax) {
  for (int e = threadIdx.x; e < 64 * 8; e += blockDim.x) {
    int r = e >> 3, c = (e & 7) * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r0 + r < rmax) v = *(const uint4*)(src + (size_t)(r0 + r) * ld + c);
    *(uint4*)(dst + r * LDB + c) = v;
  }
}

// C[16 x 64] (rows m0..m0+15 of an fp32 tile) = A[16 x 64] * B^T, A rows from `a` (pitch LDB), B given as
// [n][k] (pitch LDB): the QK^T / dO V^T shape.
__device__ __forceinline__ void mma_abt_to_smem(float* c, const bf16* a, const bf16* b) {
#pragma unroll
  for (int n = 0; n < 4; ++n) {
    FragC acc;
    wmma::fill_fragment(acc, 0.f);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      FragA fa;
      FragBT fb;
      wmma::load_matrix_sync(fa, a + k * 16, LDB);
      wmma::load_matrix_sync(fb, b + n * 16 * LDB + k * 16, LDB);
      wmma::mma_sync(acc, fa, fb, acc);
    }
    wmma::store_matrix_sync(c + n * 16, acc, LDF, wmma::mem_row_major);
  }
}

struct FwdSmem {
  bf16 q[TQ * LDB], k[TK * LDB], v[TK * LDB], p[TQ * LDB];
  float s[TQ * LDF];
};

__global__ void __launch_bounds__(128) attn_fwd_tc_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb pr = probs[blockIdx.z];
  if ((int)blockIdx.y >= pr.B * pr.H || (int)blockIdx.x * TQ >= pr.T) return;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  FwdSmem& sm = *(FwdSmem*)smem_raw;
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const size_t ld = 3 * (size_t)d;
  const bf16* base = (const bf16*)pr.qkv + (size_t)b * T * ld + (size_t)h * DH;
  const int qt = blockIdx.x, q0 = qt * TQ;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = warp * 16 + (lane >> 1), half = lane & 1;   // this lane's row of the tile, and its 32-column half
  const int qi = q0 + row;

  load_tile_bf16(sm.q, base, ld, q0, T);
  float m = -INFINITY, l = 0.f;
  // ---- pass 1: row log-sum-exp
  for (int kt = 0; kt <= qt; ++kt) {
    __syncthreads();
    load_tile_bf16(sm.k, base + d, ld, kt * TK, T);
    __syncthreads();
    mma_abt_to_smem(sm.s + warp * 16 * LDF, sm.q + warp * 16 * LDB, sm.k);
    __syncwarp();
    const float* srow = sm.s + row * LDF + half * 32;
    int jmax = min(32, min(T, qi + 1) - (kt * TK + half * 32));   // visible keys in this half
    float tm = -INFINITY;
    for (int j = 0; j < jmax; ++j) tm = fmaxf(tm, srow[j] * SCALE);
    tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 1));
    float mn = fmaxf(m, tm);
    float ts = 0.f;
    for (int j = 0; j < jmax; ++j) ts += __expf(srow[j] * SCALE - mn);
    ts += __shfl_xor_sync(0xffffffffu, ts, 1);
    if (mn > -INFINITY) { l = l * __expf(m - mn) + ts; m = mn; }
    __syncwarp();
  }
  const float lse = m + logf(l);
  // ---- pass 2: O = sum_tiles exp(S - lse) V
  FragC o[4];
#pragma unroll
  for (int n = 0; n < 4; ++n) wmma::fill_fragment(o[n], 0.f);
  for (int kt = 0; kt <= qt; ++kt) {
    __syncthreads();
    load_tile_bf16(sm.k, base + d, ld, kt * TK, T);
    load_tile_bf16(sm.v, base + 2 * d, ld, kt * TK, T);
    __syncthreads();
    mma_abt_to_smem(sm.s + warp * 16 * LDF, sm.q + warp * 16 * LDB, sm.k);
    __syncwarp();
    const float* srow = sm.s + row * LDF + half * 32;
    bf16* prow = sm.p + row * LDB + half * 32;
    int jmax = min(32, min(T, qi + 1) - (kt * TK + half * 32));
    for (int j = 0; j < 32; ++j) prow[j] = __float2bfloat16_rn(j < jmax ? __expf(srow[j] * SCALE - lse) : 0.f);
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      FragA fa;
      wmma::load_matrix_sync(fa, sm.p + warp * 16 * LDB + k * 16, LDB);
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        FragB fb;
        wmma::load_matrix_sync(fb, sm.v + k * 16 * LDB + n * 16, LDB);
        wmma::mma_sync(o[n], fa, fb, o[n]);
      }
    }
  }
  __syncwarp();
#pragma unroll
  for (int n = 0; n < 4; ++n) wmma::store_matrix_sync(sm.s + warp * 16 * LDF + n * 16, o[n], LDF, wmma::mem_row_major);
  __syncwarp();
  if (qi < T) {
    const float* orow = sm.s + row * LDF + half * 32;
    bf16* out = (bf16*)pr.o + ((size_t)b * T + qi) * d + (size_t)h * DH + half * 32;
#pragma unroll
    for (int c = 0; c < 32; c += 8) {
      uint4 u;
      __nv_bfloat162* hh = (__nv_bfloat162*)&u;
#pragma unroll
      for (int t = 0; t < 4; ++t) hh[t] = __floats2bfloat162_rn(orow[c + 2 * t], orow[c + 2 * t + 1]);
      *(uint4*)(out + c) = u;
    }
    if (half == 0) pr.lse[((size_t)b * pr.H + h) * T + qi] = lse;
  }
}

struct DqSmem {
  bf16 q[TQ * LDB], go[TQ * LDB], k[TK * LDB], v[TK * LDB], ds[TQ * LDB];
  float s[TQ * LDF], dp[TQ * LDF];
};

// dQ for one query tile; also writes delta[row] = sum_c dO[row,c] O[row,c].
__global__ void __launch_bounds__(128) attn_bwd_dq_tc_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb pr = probs[blockIdx.z];
  if ((int)blockIdx.y >= pr.B * pr.H || (int)blockIdx.x * TQ >= pr.T) return;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  DqSmem& sm = *(DqSmem*)smem_raw;
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const size_t ld = 3 * (size_t)d;
  const bf16* base = (const bf16*)pr.qkv + (size_t)b * T * ld + (size_t)h * DH;
  const bf16* gob = (const bf16*)pr.dout + (size_t)b * T * d + (size_t)h * DH;
  const bf16* ob = (const bf16*)pr.o + (size_t)b * T * d + (size_t)h * DH;
  const int qt = blockIdx.x, q0 = qt * TQ;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = warp * 16 + (lane >> 1), half = lane & 1;
  const int qi = q0 + row;

  load_tile_bf16(sm.q, base, ld, q0, T);
  load_tile_bf16(sm.go, gob, (size_t)d, q0, T);
  float delta = 0.f, lse = 0.f;
  if (qi < T) {
    const bf16* orow = ob + (size_t)qi * d + half * 32;
    const bf16* grow = gob + (size_t)qi * d + half * 32;
    for (int c = 0; c < 32; ++c) delta = fmaf(__bfloat162float(grow[c]), __bfloat162float(orow[c]), delta);
    lse = pr.lse[((size_t)b * pr.H + h) * T + qi];
  }
  delta += __shfl_xor_sync(0xffffffffu, delta, 1);
  if (qi < T && half == 0) pr.delta[((size_t)b * pr.H + h) * T + qi] = delta;

  FragC dq[4];
#pragma unroll
  for (int n = 0; n < 4; ++n) wmma::fill_fragment(dq[n], 0.f);
  for (int kt = 0; kt <= qt; ++kt) {
    __syncthreads();
    load_tile_bf16(sm.k, base + d, ld, kt * TK, T);
    load_tile_bf16(sm.v, base + 2 * d, ld, kt * TK, T);
    __syncthreads();
    mma_abt_to_smem(sm.s + warp * 16 * LDF, sm.q + warp * 16 * LDB, sm.k);
    mma_abt_to_smem(sm.dp + warp * 16 * LDF, sm.go + warp * 16 * LDB, sm.v);
    __syncwarp();
    const float* srow = sm.s + row * LDF + half * 32;
    const float* dprow = sm.dp + row * LDF + half * 32;
    bf16* dsrow = sm.ds + row * LDB + half * 32;
    int jmax = min(32, min(T, qi + 1) - (kt * TK + half * 32));
    for (int j = 0; j < 32; ++j) {
      float v = j < jmax ? __expf(srow[j] * SCALE - lse) * (dprow[j] - delta) : 0.f;
      dsrow[j] = __float2bfloat16_rn(v);
    }
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      FragA fa;
      wmma::load_matrix_sync(fa, sm.ds + warp * 16 * LDB + k * 16, LDB);
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        FragB fb;
        wmma::load_matrix_sync(fb, sm.k + k * 16 * LDB + n * 16, LDB);
        wmma::mma_sync(dq[n], fa, fb, dq[n]);
      }
    }
  }
  __syncwarp();
#pragma unroll
  for (int n = 0; n < 4; ++n) wmma::store_matrix_sync(sm.s + warp * 16 * LDF + n * 16, dq[n], LDF, wmma::mem_row_major);
  __syncwarp();
  if (qi < T) {
    const float* r = sm.s + row * LDF + half * 32;
    bf16* out = (bf16*)pr.dqkv + ((size_t)b * T + qi) * ld + (size_t)h * DH + half * 32;
#pragma unroll
    for (int c = 0; c < 32; c += 8) {
      uint4 u;
      __nv_bfloat162* hh = (__nv_bfloat162*)&u;
#pragma unroll
      for (int t = 0; t < 4; ++t) hh[t] = __floats2bfloat162_rn(r[c + 2 * t] * SCALE, r[c + 2 * t + 1] * SCALE);
      *(uint4*)(out + c) = u;
    }
  }
}

struct DkvSmem {
  bf16 k[TK * LDB], v[TK * LDB], q[TQ * LDB], go[TQ * LDB], p[TQ * LDB], ds[TQ * LDB];
  float s[TQ * LDF], dp[TQ * LDF];
  float lse[TQ], delta[TQ];
};

// dK and dV for one key tile: loops over the query tiles that can see it.
__global__ void __launch_bounds__(128) attn_bwd_dkv_tc_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb pr = probs[blockIdx.z];
  if ((int)blockIdx.y >= pr.B * pr.H || (int)blockIdx.x * TK >= pr.T) return;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  DkvSmem& sm = *(DkvSmem*)smem_raw;
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const size_t ld = 3 * (size_t)d;
  const bf16* base = (const bf16*)pr.qkv + (size_t)b * T * ld + (size_t)h * DH;
  const bf16* gob = (const bf16*)pr.dout + (size_t)b * T * d + (size_t)h * DH;
  const int kt = blockIdx.x, k0 = kt * TK;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = (T + TQ - 1) / TQ;

  load_tile_bf16(sm.k, base + d, ld, k0, T);
  load_tile_bf16(sm.v, base + 2 * d, ld, k0, T);
  FragC dk[4], dv[4];
#pragma unroll
  for (int n = 0; n < 4; ++n) { wmma::fill_fragment(dk[n], 0.f); wmma::fill_fragment(dv[n], 0.f); }
  for (int qt = kt; qt < nq; ++qt) {
    int q0 = qt * TQ;
    __syncthreads();
    load_tile_bf16(sm.q, base, ld, q0, T);
    load_tile_bf16(sm.go, gob, (size_t)d, q0, T);
    if (threadIdx.x < TQ) {
      int qi = q0 + threadIdx.x;
      sm.lse[threadIdx.x] = qi < T ? pr.lse[((size_t)b * pr.H + h) * T + qi] : 0.f;
      sm.delta[threadIdx.x] = qi < T ? pr.delta[((size_t)b * pr.H + h) * T + qi] : 0.f;
    }
    __syncthreads();
    // scores and dP for query rows [16*warp, 16*warp+16) against all 64 keys of this tile
    mma_abt_to_smem(sm.s + warp * 16 * LDF, sm.q + warp * 16 * LDB, sm.k);
    mma_abt_to_smem(sm.dp + warp * 16 * LDF, sm.go + warp * 16 * LDB, sm.v);
    __syncwarp();
    {
      int row = warp * 16 + (lane >> 1), half = lane & 1;
      int qi = q0 + row;
      const float* srow = sm.s + row * LDF + half * 32;
      const float* dprow = sm.dp + row * LDF + half * 32;
      bf16* prow = sm.p + row * LDB + half * 32;
      bf16* dsrow = sm.ds + row * LDB + half * 32;
      float lse = sm.lse[row], delta = sm.delta[row];
      int jmax = qi < T ? min(32, min(T, qi + 1) - (k0 + half * 32)) : 0;
      for (int j = 0; j < 32; ++j) {
        float pv = j < jmax ? __expf(srow[j] * SCALE - lse) : 0.f;
        prow[j] = __float2bfloat16_rn(pv);
        dsrow[j] = __float2bfloat16_rn(pv * (dprow[j] - delta));
      }
    }
    __syncthreads();
    // dV[keys of this warp] += P^T dO ; dK[keys of this warp] += dS^T Q
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      FragAT fp, fds;
      wmma::load_matrix_sync(fp, sm.p + k * 16 * LDB + warp * 16, LDB);
      wmma::load_matrix_sync(fds, sm.ds + k * 16 * LDB + warp * 16, LDB);
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        FragB fgo, fq;
        wmma::load_matrix_sync(fgo, sm.go + k * 16 * LDB + n * 16, LDB);
        wmma::load_matrix_sync(fq, sm.q + k * 16 * LDB + n * 16, LDB);
        wmma::mma_sync(dv[n], fp, fgo, dv[n]);
        wmma::mma_sync(dk[n], fds, fq, dk[n]);
      }
    }
  }
  __syncthreads();
  const int row = warp * 16 + (lane >> 1), half = lane & 1;
  const int ki = k0 + row;
  for (int which = 0; which < 2; ++which) {
#pragma unroll
    for (int n = 0; n < 4; ++n)
      wmma::store_matrix_sync(sm.s + warp * 16 * LDF + n * 16, which == 0 ? dk[n] : dv[n], LDF, wmma::mem_row_major);
    __syncwarp();
    if (ki < T) {
      const float* r = sm.s + row * LDF + half * 32;
      float sc = which == 0 ? SCALE : 1.f;
      bf16* out = (bf16*)pr.dqkv + ((size_t)b * T + ki) * ld + (size_t)(which + 1) * d + (size_t)h * DH + half * 32;
#pragma unroll
      for (int c = 0; c < 32; c += 8) {
        uint4 u;
        __nv_bfloat162* hh = (__nv_bfloat162*)&u;
#pragma unroll
        for (int t = 0; t < 4; ++t) hh[t] = __floats2bfloat162_rn(r[c + 2 * t] * sc, r[c + 2 * t + 1] * sc);
        *(uint4*)(out + c) = u;
      }
    }
    __syncwarp();
  }
}

template <typename K>
cudaError_t ensure_smem(K kernel, size_t bytes, bool* done) {
  if (*done) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) *done = true;
  return e;
}

}  // namespace

// Requirements of the tensor-core path: bf16, qkv / o / dout / dqkv rows 16-byte aligned (d multiple of 8: always, d = 64 H).
void launch_attn_fwd_tc(const AttnProb* d, int n, int maxB, int maxT, int maxH, cudaStream_t s) {
  static bool set = false;
  if (ensure_smem(attn_fwd_tc_kernel, sizeof(FwdSmem), &set) != cudaSuccess) return;
  dim3 grid((maxT + TQ - 1) / TQ, maxB * maxH, n);
  attn_fwd_tc_kernel<<<grid, 128, sizeof(FwdSmem), s>>>(d);
}

void launch_attn_bwd_tc(const AttnProb* d, int n, int maxB, int maxT, int maxH, cudaStream_t s) {
  static bool set1 = false, set2 = false;
  if (ensure_smem(attn_bwd_dq_tc_kernel, sizeof(DqSmem), &set1) != cudaSuccess) return;
  if (ensure_smem(attn_bwd_dkv_tc_kernel, sizeof(DkvSmem), &set2) != cudaSuccess) return;
  dim3 grid((maxT + TQ - 1) / TQ, maxB * maxH, n);
  attn_bwd_dq_tc_kernel<<<grid, 128, sizeof(DqSmem), s>>>(d);
  attn_bwd_dkv_tc_kernel<<<grid, 128, sizeof(DkvSmem), s>>>(d);
}

}  // namespace lp
