// Causal multi-head softmax attention (App. B.2's transformer layers), heads of 64, forward and
// backward, flash-style: keys/values are streamed through shared memory in tiles of 64 with an
// online softmax, the T x T score matrix is never stored; backward recomputes the probabilities
// from Q, K and the saved log-sum-exp.  FP32-ALU version for fp32 activations: one thread per query
// row (forward, dQ), two threads per key row (dK, dV).  All sums run in a fixed order (no atomics).
// bf16 activations take the tensor-core kernels of attn_tc.cu.
//
// qkv is [B*T, 3*H*64]: columns [0, d) queries, [d, 2d) keys, [2d, 3d) values, head h at h*64.
#include "common.cuh"

namespace lp {
namespace {
constexpr int DH = 64, TILE = 64;
constexpr float SCALE = 0.125f;   // 1/sqrt(64)

template <typename T>
__device__ __forceinline__ void load_tile(float (*dst)[DH], const T* base, size_t ld, int r0, int rmax, int nthreads) {
  for (int e = threadIdx.x; e < TILE * DH; e += nthreads) {
    int r = e / DH, c = e % DH;
    dst[r][c] = (r0 + r < rmax) ? to_f(base[(size_t)(r0 + r) * ld + c]) : 0.f;
  }
}

template <typename T>
__global__ void __launch_bounds__(64) attn_fwd_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb p = probs[blockIdx.z];
  if ((int)blockIdx.y >= p.B * p.H || (int)blockIdx.x * TILE >= p.T) return;
  __shared__ float Ks[TILE][DH];
  __shared__ float Vs[TILE][DH];
  __shared__ float Ss[TILE][TILE];   // [key][query thread]: conflict-free
  int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
  int d = p.H * DH;
  size_t ld = 3 * (size_t)d;
  const T* base = (const T*)p.qkv + (size_t)b * p.T * ld + (size_t)h * DH;
  int r = blockIdx.x * TILE + threadIdx.x;
  bool live = r < p.T;
  float q[DH], acc[DH];
#pragma unroll
  for (int c = 0; c < DH; ++c) { q[c] = live ? to_f(base[(size_t)r * ld + c]) * SCALE : 0.f; acc[c] = 0.f; }
  float m = -INFINITY, l = 0.f;
  for (int kt = 0; kt <= (int)blockIdx.x; ++kt) {
    __syncthreads();
    load_tile(Ks, base + d, ld, kt * TILE, p.T, 64);
    load_tile(Vs, base + 2 * d, ld, kt * TILE, p.T, 64);
    __syncthreads();
    int jmax = min(TILE, min(p.T, r + 1) - kt * TILE);   // keys kt*TILE + j, j < jmax, are visible to row r
    if (!live) jmax = 0;
    float tm = m;
    for (int j = 0; j < jmax; ++j) {
      float s = 0.f;
#pragma unroll
      for (int c = 0; c < DH; ++c) s = fmaf(q[c], Ks[j][c], s);
      Ss[j][threadIdx.x] = s;
      tm = fmaxf(tm, s);
    }
    if (jmax > 0) {
      float corr = __expf(m - tm);
      l *= corr;
#pragma unroll
      for (int c = 0; c < DH; ++c) acc[c] *= corr;
      for (int j = 0; j < jmax; ++j) {
        float pj = __expf(Ss[j][threadIdx.x] - tm);
        l += pj;
#pragma unroll
        for (int c = 0; c < DH; ++c) acc[c] = fmaf(pj, Vs[j][c], acc[c]);
      }
      m = tm;
    }
  }
  if (live) {
    float inv = 1.f / l;
    T* o = (T*)p.o + ((size_t)b * p.T + r) * d + (size_t)h * DH;
#pragma unroll
    for (int c = 0; c < DH; ++c) o[c] = from_f<T>(acc[c] * inv);
    p.lse[((size_t)b * p.H + h) * p.T + r] = m + logf(l);
  }
}

// dQ: thread per query row.  Also writes delta[r] = sum_c dO[r,c] * O[r,c].
template <typename T>
__global__ void __launch_bounds__(64) attn_bwd_dq_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb p = probs[blockIdx.z];
  if ((int)blockIdx.y >= p.B * p.H || (int)blockIdx.x * TILE >= p.T) return;
  __shared__ float Ks[TILE][DH];
  __shared__ float Vs[TILE][DH];
  int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
  int d = p.H * DH;
  size_t ld = 3 * (size_t)d;
  const T* base = (const T*)p.qkv + (size_t)b * p.T * ld + (size_t)h * DH;
  int r = blockIdx.x * TILE + threadIdx.x;
  bool live = r < p.T;
  float q[DH], dO[DH], dq[DH];
  float delta = 0.f, lse = 0.f;
  {
    const T* o = (const T*)p.o + ((size_t)b * p.T + r) * d + (size_t)h * DH;
    const T* go = (const T*)p.dout + ((size_t)b * p.T + r) * d + (size_t)h * DH;
#pragma unroll
    for (int c = 0; c < DH; ++c) {
      q[c] = live ? to_f(base[(size_t)r * ld + c]) * SCALE : 0.f;
      dO[c] = live ? to_f(go[c]) : 0.f;
      dq[c] = 0.f;
      if (live) delta = fmaf(dO[c], to_f(o[c]), delta);
    }
    if (live) {
      lse = p.lse[((size_t)b * p.H + h) * p.T + r];
      p.delta[((size_t)b * p.H + h) * p.T + r] = delta;
    }
  }
  for (int kt = 0; kt <= (int)blockIdx.x; ++kt) {
    __syncthreads();
    load_tile(Ks, base + d, ld, kt * TILE, p.T, 64);
    load_tile(Vs, base + 2 * d, ld, kt * TILE, p.T, 64);
    __syncthreads();
    int jmax = live ? min(TILE, min(p.T, r + 1) - kt * TILE) : 0;
    for (int j = 0; j < jmax; ++j) {
      float s = 0.f, dp = 0.f;
#pragma unroll
      for (int c = 0; c < DH; ++c) { s = fmaf(q[c], Ks[j][c], s); dp = fmaf(dO[c], Vs[j][c], dp); }
      float ds = __expf(s - lse) * (dp - delta);
#pragma unroll
      for (int c = 0; c < DH; ++c) dq[c] = fmaf(ds, Ks[j][c], dq[c]);
    }
  }
  if (live) {
    T* out = (T*)p.dqkv + ((size_t)b * p.T + r) * ld + (size_t)h * DH;
#pragma unroll
    for (int c = 0; c < DH; ++c) out[c] = from_f<T>(dq[c] * SCALE);
  }
}

// dK, dV: two threads per key row, each owning 32 of the 64 columns; dot products are completed
// with one shuffle between the two partners.
template <typename T>
__global__ void __launch_bounds__(128) attn_bwd_dkv_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb p = probs[blockIdx.z];
  if ((int)blockIdx.y >= p.B * p.H || (int)blockIdx.x * TILE >= p.T) return;
  __shared__ float Qs[TILE][DH];
  __shared__ float Os[TILE][DH];
  __shared__ float Ls[TILE], Ds[TILE];
  int b = blockIdx.y / p.H, h = blockIdx.y % p.H;
  int d = p.H * DH;
  size_t ld = 3 * (size_t)d;
  const T* base = (const T*)p.qkv + (size_t)b * p.T * ld + (size_t)h * DH;
  const T* gob = (const T*)p.dout + (size_t)b * p.T * d + (size_t)h * DH;
  int jrow = threadIdx.x >> 1, half = threadIdx.x & 1;
  int j = blockIdx.x * TILE + jrow;
  bool live = j < p.T;
  constexpr int HC = DH / 2;
  float k[HC], v[HC], dk[HC], dv[HC];
#pragma unroll
  for (int c = 0; c < HC; ++c) {
    k[c] = live ? to_f(base[(size_t)j * ld + d + half * HC + c]) : 0.f;
    v[c] = live ? to_f(base[(size_t)j * ld + 2 * d + half * HC + c]) : 0.f;
    dk[c] = 0.f; dv[c] = 0.f;
  }
  int ntiles = (p.T + TILE - 1) / TILE;
  for (int qt = blockIdx.x; qt < ntiles; ++qt) {
    __syncthreads();
    load_tile(Qs, base, ld, qt * TILE, p.T, 128);
    load_tile(Os, gob, (size_t)d, qt * TILE, p.T, 128);
    if (threadIdx.x < TILE) {
      int i = qt * TILE + threadIdx.x;
      Ls[threadIdx.x] = i < p.T ? p.lse[((size_t)b * p.H + h) * p.T + i] : 0.f;
      Ds[threadIdx.x] = i < p.T ? p.delta[((size_t)b * p.H + h) * p.T + i] : 0.f;
    }
    __syncthreads();
    int imax = min(TILE, p.T - qt * TILE);
    for (int ii = 0; ii < imax; ++ii) {
      int i = qt * TILE + ii;
      float s = 0.f, dp = 0.f;
#pragma unroll
      for (int c = 0; c < HC; ++c) {
        s = fmaf(Qs[ii][half * HC + c], k[c], s);
        dp = fmaf(Os[ii][half * HC + c], v[c], dp);
      }
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      dp += __shfl_xor_sync(0xffffffffu, dp, 1);
      if (live && i >= j) {
        float pr = __expf(s * SCALE - Ls[ii]);
        float ds = pr * (dp - Ds[ii]);
#pragma unroll
        for (int c = 0; c < HC; ++c) {
          dv[c] = fmaf(pr, Os[ii][half * HC + c], dv[c]);
          dk[c] = fmaf(ds, Qs[ii][half * HC + c], dk[c]);
        }
      }
    }
  }
  if (live) {
    T* out = (T*)p.dqkv + ((size_t)b * p.T + j) * ld + (size_t)h * DH + half * HC;
#pragma unroll
    for (int c = 0; c < HC; ++c) {
      out[d + c] = from_f<T>(dk[c] * SCALE);
      out[2 * d + c] = from_f<T>(dv[c]);
    }
  }
}

}  // namespace

void launch_attn_fwd(const AttnProb* d, int n, int maxB, int maxT, int maxH, bool is_bf16, cudaStream_t s) {
  dim3 grid((maxT + TILE - 1) / TILE, maxB * maxH, n);
  if (is_bf16) attn_fwd_kernel<bf16><<<grid, 64, 0, s>>>(d);
  else attn_fwd_kernel<float><<<grid, 64, 0, s>>>(d);
}

void launch_attn_bwd(const AttnProb* d, int n, int maxB, int maxT, int maxH, bool is_bf16, cudaStream_t s) {
  dim3 grid((maxT + TILE - 1) / TILE, maxB * maxH, n);
  if (is_bf16) {
    attn_bwd_dq_kernel<bf16><<<grid, 64, 0, s>>>(d);
    attn_bwd_dkv_kernel<bf16><<<grid, 128, 0, s>>>(d);
    return;
  }
  attn_bwd_dq_kernel<float><<<grid, 64, 0, s>>>(d);
  attn_bwd_dkv_kernel<float><<<grid, 128, 0, s>>>(d);
}

}  // namespace lp
