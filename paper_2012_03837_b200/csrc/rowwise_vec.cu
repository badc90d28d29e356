// 128-bit vectorised bf16 versions of the HBM-bound row kernels (LayerNorm forward/backward,
// softmax cross-entropy with in-place dlogits).  Each row is read from HBM exactly once and kept in
// registers; outputs are written once.  Used when every row is 16-byte aligned and its length fits
// the register budget; otherwise the generic kernels of rowwise.cu run.  Fixed reduction orders.
#include "common.cuh"

namespace lp {
namespace {

__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
  const __nv_bfloat162* h = (const __nv_bfloat162*)&u;
#pragma unroll
  for (int t = 0; t < 4; ++t) { float2 v = __bfloat1622float2(h[t]); f[2 * t] = v.x; f[2 * t + 1] = v.y; }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
  uint4 u;
  __nv_bfloat162* h = (__nv_bfloat162*)&u;
#pragma unroll
  for (int t = 0; t < 4; ++t) h[t] = __floats2bfloat162_rn(f[2 * t], f[2 * t + 1]);
  return u;
}

// ------------------------------------------------------------------ LayerNorm forward
// Block = 8 warps over LN_FWD_ROWS rows (warp w takes rows w, w+8, ...); a lane owns the 8-element
// vectors j*32 + lane, j < NV (d = NV * 256).  The warp's next row is loaded while the current one
// is normalised.
enum { LN_FWD_ROWS = 64 };
template <int NV>
__global__ void __launch_bounds__(256, 2) ln_fwd_vec_kernel(const LnProb* __restrict__ probs) {
  const LnProb p = probs[blockIdx.y];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int r0 = blockIdx.x * LN_FWD_ROWS;
  if (r0 >= p.rows) return;
  const int r1 = min(r0 + LN_FWD_ROWS, p.rows);
  const float inv_d = 1.0f / p.d;
  uint4 nxt[NV];
  if (r0 + w < r1) {
    const uint4* x = (const uint4*)((const bf16*)p.x + (size_t)(r0 + w) * p.d);
#pragma unroll
    for (int j = 0; j < NV; ++j) nxt[j] = x[j * 32 + lane];
  }
  // scale and shift of this lane's columns stay in registers for all rows of the warp
  float g[NV][8], b[NV][8];
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int c0 = (j * 32 + lane) * 8;
    float4 g0 = *(const float4*)(p.g + c0), g1 = *(const float4*)(p.g + c0 + 4);
    float4 b0 = *(const float4*)(p.b + c0), b1 = *(const float4*)(p.b + c0 + 4);
    g[j][0] = g0.x; g[j][1] = g0.y; g[j][2] = g0.z; g[j][3] = g0.w; g[j][4] = g1.x; g[j][5] = g1.y; g[j][6] = g1.z; g[j][7] = g1.w;
    b[j][0] = b0.x; b[j][1] = b0.y; b[j][2] = b0.z; b[j][3] = b0.w; b[j][4] = b1.x; b[j][5] = b1.y; b[j][6] = b1.z; b[j][7] = b1.w;
  }
  for (int row = r0 + w; row < r1; row += 8) {
    float v[NV][8];
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      unpack8(nxt[j], v[j]);
#pragma unroll
      for (int t = 0; t < 8; ++t) s += v[j][t];
    }
    if (row + 8 < r1) {
      const uint4* x = (const uint4*)((const bf16*)p.x + (size_t)(row + 8) * p.d);
#pragma unroll
      for (int j = 0; j < NV; ++j) nxt[j] = x[j * 32 + lane];
    }
    float mu = warp_sum(s) * inv_d;
    float q = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j)
#pragma unroll
      for (int t = 0; t < 8; ++t) { v[j][t] -= mu; q += v[j][t] * v[j][t]; }
    float rstd = rsqrtf(warp_sum(q) * inv_d + 1e-5f);
    uint4* y = (uint4*)((bf16*)p.y + (size_t)row * p.d);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      float o[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) o[t] = v[j][t] * rstd * g[j][t] + b[j][t];
      y[j * 32 + lane] = pack8(o);
    }
    if (lane == 0) { p.mean[row] = mu; p.rstd[row] = rstd; }
  }
}

// ------------------------------------------------------------------ LayerNorm backward
// Block = 8 warps over LN_BWD_ROWS rows (warp w takes rows w, w+8, ...).  Each warp streams its
// rows of x and dy (and of the residual-path gradient) through its own three-deep ring of
// shared-memory buffers filled by cp.async, so two rows are in flight while one is reduced.  Each
// lane accumulates the scale/shift gradient of its own columns over the warp's rows in registers;
// the 8 warps are then summed through shared memory in warp order and the block writes one
// partial row.
enum { LN_RING = 3 };
__device__ __forceinline__ void cp_async_16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src));
}
template <int NV>
__global__ void __launch_bounds__(256) ln_bwd_vec_kernel(const LnBwdProb* __restrict__ probs) {
  extern __shared__ __align__(16) float red[];   // [8][2][d] floats, then the rings: [8 warps][LN_RING][3][d] bf16
  const LnBwdProb p = probs[blockIdx.y];
  int r0 = blockIdx.x * LN_BWD_ROWS;
  if (r0 >= p.rows) return;
  int r1 = min(r0 + LN_BWD_ROWS, p.rows);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  constexpr int D = NV * 256;
  uint4* ring = (uint4*)(red + 8 * 2 * D) + (size_t)w * LN_RING * 3 * (D / 8);
  const bool has_res = p.dx && p.dres;
  auto fetch = [&](int row, int slot) {
    if (row < r1) {
      const uint4* x = (const uint4*)((const bf16*)p.x + (size_t)row * D);
      const uint4* dy = (const uint4*)((const bf16*)p.dy + (size_t)row * D);
      uint4* dst = ring + (size_t)slot * 3 * (D / 8);
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        cp_async_16(dst + j * 32 + lane, x + j * 32 + lane);
        cp_async_16(dst + D / 8 + j * 32 + lane, dy + j * 32 + lane);
      }
      if (has_res) {
        const uint4* dr = (const uint4*)((const bf16*)p.dres + (size_t)row * D);
#pragma unroll
        for (int j = 0; j < NV; ++j) cp_async_16(dst + 2 * (D / 8) + j * 32 + lane, dr + j * 32 + lane);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  float ag[NV][8], ab[NV][8], g[NV][8];
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int c0 = (j * 32 + lane) * 8;
    float4 g0 = *(const float4*)(p.g + c0), g1 = *(const float4*)(p.g + c0 + 4);
    g[j][0] = g0.x; g[j][1] = g0.y; g[j][2] = g0.z; g[j][3] = g0.w; g[j][4] = g1.x; g[j][5] = g1.y; g[j][6] = g1.z; g[j][7] = g1.w;
#pragma unroll
    for (int t = 0; t < 8; ++t) { ag[j][t] = 0.f; ab[j][t] = 0.f; }
  }
  fetch(r0 + w, 0);
  fetch(r0 + w + 8, 1);
  // lane k holds the statistics of the warp's k-th row (rows r0 + w + 8k, k < LN_BWD_ROWS / 8 <= 32)
  static_assert(LN_BWD_ROWS / 8 <= 32, "one row per lane");
  float mu_mine = 0.f, rs_mine = 0.f;
  if (r0 + w + 8 * lane < r1) { mu_mine = p.mean[r0 + w + 8 * lane]; rs_mine = p.rstd[r0 + w + 8 * lane]; }
  int slot = 0, kk = 0;
  const float inv_d = 1.0f / D;
  for (int row = r0 + w; row < r1; row += 8, ++kk) {
    fetch(row + 16, slot == 0 ? 2 : slot - 1);      // the slot freed by the previous row
    asm volatile("cp.async.wait_group 2;" ::: "memory");
    __syncwarp();
    const uint4* buf = ring + (size_t)slot * 3 * (D / 8);
    const float mu = __shfl_sync(0xffffffffu, mu_mine, kk), rs = __shfl_sync(0xffffffffu, rs_mine, kk);
    float xh[NV][8], dv[NV][8];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      unpack8(buf[j * 32 + lane], xh[j]);
      unpack8(buf[D / 8 + j * 32 + lane], dv[j]);
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        xh[j][t] = (xh[j][t] - mu) * rs;
        ag[j][t] += dv[j][t] * xh[j][t];
        ab[j][t] += dv[j][t];
        dv[j][t] *= g[j][t];                          // from here on: gradient w.r.t. the normalised value
        s1 += dv[j][t];
        s2 += dv[j][t] * xh[j][t];
      }
    }
    if (p.dx) {
      s1 = warp_sum(s1) * inv_d;
      s2 = warp_sum(s2) * inv_d;
      uint4* dx = (uint4*)((bf16*)p.dx + (size_t)row * D);
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        float o[8], r[8];
        if (has_res) unpack8(buf[2 * (D / 8) + j * 32 + lane], r);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          o[t] = rs * (dv[j][t] - s1 - xh[j][t] * s2);
          if (has_res) o[t] += r[t];
        }
        dx[j * 32 + lane] = pack8(o);
      }
    }
    __syncwarp();                                     // all lanes are done with this slot before it is refilled
    slot = slot == LN_RING - 1 ? 0 : slot + 1;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int c0 = (j * 32 + lane) * 8;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      red[(w * 2 + 0) * D + c0 + t] = ag[j][t];
      red[(w * 2 + 1) * D + c0 + t] = ab[j][t];
    }
  }
  __syncthreads();
  float* part = p.part + (size_t)blockIdx.x * 2 * D;
  for (int c = threadIdx.x; c < 2 * D; c += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int ww = 0; ww < 8; ++ww) s += red[ww * 2 * D + c];
    part[c] = s;
  }
}

// ------------------------------------------------------------------ softmax cross-entropy
// Block (NT threads) per row; thread owns vectors j*NT + tid, j < NV.  Long rows use 1024 threads
// with few vectors each, so that two blocks fit an SM and one block's loads overlap the other's math.
template <int NV, int NT>
__global__ void __launch_bounds__(NT) xent_vec_kernel(const XentProb* __restrict__ probs) {
  __shared__ float red[33];
  const XentProb p = probs[blockIdx.y];
  int row = blockIdx.x;
  if (row >= p.rows) return;
  uint4* z = (uint4*)((bf16*)p.z + (size_t)row * p.ld);
  const int nvec = p.classes >> 3;
  int y = p.y[row];
  bool valid = (y >= 0 && y < p.classes);
  if (!valid) {
    for (int i = threadIdx.x; i < nvec; i += NT) z[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) p.row_loss[row] = 0.f;
    return;
  }
  uint4 raw[NV];
  float m = -INFINITY;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int i = j * NT + threadIdx.x;
    if (i < nvec) {
      raw[j] = z[i];
      float f[8];
      unpack8(raw[j], f);
#pragma unroll
      for (int t = 0; t < 8; ++t) m = fmaxf(m, f[t]);
    }
  }
  float M = block_max(m, red);
  // One exponential per logit: e = exp(z - max) is summed in fp32 and kept (as bf16, the precision
  // the stored dlogits have anyway) in the registers that held z; the label's logit is saved first.
  float s = 0.f, zy = 0.f;
  const float ML2 = M * 1.4426950408889634f;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int i = j * NT + threadIdx.x;
    if (i < nvec) {
      float f[8];
      unpack8(raw[j], f);
      int c0 = i * 8;
      if (y >= c0 && y < c0 + 8) {
#pragma unroll
        for (int t = 0; t < 8; ++t) if (c0 + t == y) zy = f[t];
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) { f[t] = exp2f(fmaf(f[t], 1.4426950408889634f, -ML2)); s += f[t]; }
      raw[j] = pack8(f);
    }
  }
  float S = block_sum(s, red);
  float lse = M + logf(S);
  float inv = 1.0f / (float)(*p.n_valid);
  float scale = inv / S;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int i = j * NT + threadIdx.x;
    if (i < nvec) {
      float f[8];
      unpack8(raw[j], f);
      int c0 = i * 8;
#pragma unroll
      for (int t = 0; t < 8; ++t) f[t] *= scale;
      if (y >= c0 && y < c0 + 8) {
        p.row_loss[row] = lse - zy;
#pragma unroll
        for (int t = 0; t < 8; ++t) if (c0 + t == y) f[t] -= inv;
      }
      z[i] = pack8(f);
    }
  }
}

// ------------------------------------------------------------------ cross-entropy over blocks of rows
// One block of NT threads walks XENT_ROWS consecutive rows; thread t owns the 8-column vectors
// j*NT + t.  Per row: packed bf16 max over the thread's logits and a shuffle max over the warp; then
// e = exp(z - warp max) (one exponential per logit; kept as bf16 in the registers that held z) and
// its sum; the per-warp (max, sum) pairs are merged over the block through double-buffered shared
// memory, so a row costs a single block barrier.  The next row is loaded while the current one is
// reduced; labels and the logits at the labels are fetched once per block.  The label's "- 1/n" is
// applied by the one thread that owns that column after the vector stores, which keeps the inner
// loops free of label tests.  The column sums of the written dlogits (the head's bias gradient)
// accumulate in shared memory (each thread only touches its own columns) and are written once per
// block: the logits are read once and written once per step.
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Warp reductions in one instruction each.  The maximum is the hardware's fp32 reduction; the sum
// goes through fixed point (integer adds: exact and order-free), `scale` being a power of two that
// keeps the warp's total below 2^32.  A non-finite addend makes the result NaN.
__device__ __forceinline__ float warp_max_f(float v) {
  float m;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(m) : "f"(v));
  return m;
}
__device__ __forceinline__ float warp_sum_fixed(float v, float scale, float inv_scale) {
  unsigned q = __float2uint_rn(v * scale), bad = (v >= 0.f && v <= 3.0e38f) ? 0u : 1u, s, b;
  asm volatile("redux.sync.add.u32 %0, %1, 0xffffffff;" : "=r"(s) : "r"(q));
  asm volatile("redux.sync.or.b32 %0, %1, 0xffffffff;" : "=r"(b) : "r"(bad));
  return b ? __int_as_float(0x7fc00000) : (float)s * inv_scale;
}

template <int NV, int NT>
__global__ void __launch_bounds__(NT) xent_rows_kernel(const XentProb* __restrict__ probs) {
  // column sums, two planes of float4 per 8-column vector (conflict-free 16-byte lane stride):
  // plane 0 = columns 8i..8i+3 at csum4[i], plane 1 = columns 8i+4..8i+7 at csum4[nvec + i]
  extern __shared__ float4 csum4[];
  __shared__ float2 wred[2][32];             // per-warp (max, sum), double-buffered by row parity
  __shared__ int ys[XENT_ROWS];
  __shared__ float zys[XENT_ROWS];
  const float L2E = 1.4426950408889634f;
  const XentProb p = probs[blockIdx.y];
  const int r0 = blockIdx.x * XENT_ROWS;
  if (r0 >= p.rows) return;
  const int r1 = min(r0 + XENT_ROWS, p.rows);
  const int nvec = p.classes >> 3;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int NW = NT / 32;
  const float inv = 1.0f / (float)(*p.n_valid);
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    int i = j * NT + threadIdx.x;
    if (i < nvec) { csum4[i] = make_float4(0, 0, 0, 0); csum4[nvec + i] = make_float4(0, 0, 0, 0); }
  }
  uint4 nxt[NV];
  {
    const uint4* z = (const uint4*)((const bf16*)p.z + (size_t)r0 * p.ld);
#pragma unroll
    for (int j = 0; j < NV; ++j) { int i = j * NT + threadIdx.x; if (i < nvec) nxt[j] = z[i]; }
  }
  if (threadIdx.x < r1 - r0) {
    int y = p.y[r0 + threadIdx.x];
    bool ok = y >= 0 && y < p.classes;
    ys[threadIdx.x] = ok ? y : -1;
    zys[threadIdx.x] = ok ? __bfloat162float(((const bf16*)p.z)[(size_t)(r0 + threadIdx.x) * p.ld + y]) : 0.f;
  }
  __syncthreads();
  int par = 0;
  for (int row = r0; row < r1; ++row) {
    uint4 raw[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) raw[j] = nxt[j];
    if (row + 1 < r1) {
      const uint4* zn = (const uint4*)((const bf16*)p.z + (size_t)(row + 1) * p.ld);
#pragma unroll
      for (int j = 0; j < NV; ++j) { int i = j * NT + threadIdx.x; if (i < nvec) nxt[j] = zn[i]; }
    }
    uint4* z = (uint4*)((bf16*)p.z + (size_t)row * p.ld);
    const int y = ys[row - r0];
    if (y < 0) {                               // ignored row: no loss, zero gradient (uniform over the block)
#pragma unroll
      for (int j = 0; j < NV; ++j) { int i = j * NT + threadIdx.x; if (i < nvec) z[i] = make_uint4(0, 0, 0, 0); }
      if (threadIdx.x == 0) p.row_loss[row] = 0.f;
      continue;
    }
    const float zy = zys[row - r0];
    // max: packed bf16 over the thread's vectors, then over the warp
    __nv_bfloat162 mx2 = __float2bfloat162_rn(-INFINITY);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int i = j * NT + threadIdx.x;
      if (i < nvec) {
        const __nv_bfloat162* h2 = (const __nv_bfloat162*)&raw[j];
        mx2 = __hmax2(mx2, __hmax2(__hmax2(h2[0], h2[1]), __hmax2(h2[2], h2[3])));
      }
    }
    const float wm = warp_max_f(fmaxf(__low2float(mx2), __high2float(mx2)));   // -inf only for a warp without columns
    const float wml = wm * L2E;
    float st = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int i = j * NT + threadIdx.x;
      if (i < nvec) {
        float f[8];
        unpack8(raw[j], f);
#pragma unroll
        for (int t = 0; t < 8; ++t) { f[t] = fast_exp2(fmaf(f[t], L2E, -wml)); st += f[t]; }
        raw[j] = pack8(f);
      }
    }
    st = warp_sum_fixed(st, 2097152.f, 1.f / 2097152.f);          // <= 32 lanes x 32 terms <= 1 each, x 2^21
    if (lane == 0) wred[par][warp] = make_float2(wm, st);
    __syncthreads();
    const float2 v = lane < NW ? wred[par][lane] : make_float2(-INFINITY, 0.f);
    par ^= 1;
    const float M = warp_max_f(v.x);
    const float S = warp_sum_fixed(v.x == -INFINITY ? 0.f : v.y * fast_exp2((v.x - M) * L2E), 65536.f, 1.f / 65536.f);   // <= 32 x 1024, x 2^16
    const float lse = M + logf(S);
    const float scale = wm == -INFINITY ? 0.f : fast_exp2((wm - M) * L2E) * inv / S;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int i = j * NT + threadIdx.x;
      if (i < nvec) {
        float f[8];
        unpack8(raw[j], f);
#pragma unroll
        for (int t = 0; t < 8; ++t) f[t] *= scale;
        z[i] = pack8(f);
        if (p.colsum_part) {
          float4 a = csum4[i], b = csum4[nvec + i];
          a.x += f[0]; a.y += f[1]; a.z += f[2]; a.w += f[3];
          b.x += f[4]; b.y += f[5]; b.z += f[6]; b.w += f[7];
          csum4[i] = a; csum4[nvec + i] = b;
        }
      }
    }
    if (threadIdx.x == ((y >> 3) % NT)) {      // the thread that owns the label's column
      float ey = __bfloat162float(__float2bfloat16(fast_exp2(fmaf(zy, L2E, -wml))));
      ((bf16*)z)[y] = __float2bfloat16(ey * scale - inv);
      if (p.colsum_part) {
        float* c = (float*)csum4 + (((y >> 2) & 1) ? (size_t)(nvec + (y >> 3)) * 4 : (size_t)(y >> 3) * 4) + (y & 3);
        *c -= inv;
      }
    }
    if (threadIdx.x == 0) p.row_loss[row] = lse - zy;
  }
  if (p.colsum_part) {
    float* part = p.colsum_part + (size_t)blockIdx.x * p.classes;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      int i = j * NT + threadIdx.x;
      if (i < nvec) { *(float4*)(part + i * 8) = csum4[i]; *(float4*)(part + i * 8 + 4) = csum4[nvec + i]; }
    }
  }
}

// ------------------------------------------------------------------ cross-entropy from GEMM-side statistics
// Warp per row: merge the (max, sum-exp) pairs of the row's column groups; row_c is the base-2 constant
// with exp2(z*log2(e) - row_c) = softmax(z) / n_valid (+inf for ignored rows: zero gradient).
__global__ void __launch_bounds__(256) xent_merge_kernel(const XentStatsProb* __restrict__ probs) {
  const float L2E = 1.4426950408889634f;
  const XentStatsProb p = probs[blockIdx.y];
  const int lane = threadIdx.x & 31, row = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  const int y = p.y[row];
  if (!(y >= 0 && y < p.classes)) {
    if (lane == 0) { p.row_loss[row] = 0.f; p.row_c[row] = INFINITY; }
    return;
  }
  const float2* st = p.stats + (size_t)row * p.groups;
  float m = -INFINITY;
  for (int g = lane; g < p.groups; g += 32) m = fmaxf(m, st[g].x);
  m = warp_max_f(m);
  float s = 0.f;
  for (int g = lane; g < p.groups; g += 32) { float2 v = st[g]; s += v.y * fast_exp2((v.x - m) * L2E); }
  s = warp_sum(s);
  if (lane == 0) {
    float lse = m + logf(s);
    float zy = __bfloat162float(((const bf16*)p.z)[(size_t)row * p.ld + y]);
    p.row_loss[row] = lse - zy;
    p.row_c[row] = lse * L2E + log2f((float)(*p.n_valid));
  }
}

__device__ __forceinline__ void xent_apply_row(uint4 raw, float c, int y, int vec, float inv, bool col_ok, float (&cs)[8],
                                               bf16* out) {
  const float L2E = 1.4426950408889634f;
  float f[8];
  unpack8(raw, f);
#pragma unroll
  for (int t = 0; t < 8; ++t) f[t] = fast_exp2(fmaf(f[t], L2E, -c));
  if ((y >> 3) == vec && c != INFINITY) {
    const int ty = y & 7;
#pragma unroll
    for (int t = 0; t < 8; ++t) f[t] -= (t == ty) ? inv : 0.f;
  }
  if (col_ok) {
#pragma unroll
    for (int t = 0; t < 8; ++t) cs[t] += f[t];
    *(uint4*)out = pack8(f);
  }
}

// Block = 32 column lanes (8 columns each: a strip of 256 columns) x 8 row lanes over XENT_APPLY_ROWS
// rows; four rows per row lane in flight.  A thread keeps the column sums of its 8 columns in
// registers; the 8 row lanes are added in order at the end.
__global__ void __launch_bounds__(256) xent_apply_kernel(const XentStatsProb* __restrict__ probs) {
  __shared__ float red[8][32][9];
  const float L2E = 1.4426950408889634f;
  const XentStatsProb p = probs[blockIdx.z];
  const int r0 = blockIdx.y * XENT_APPLY_ROWS;
  if (r0 >= p.rows || (int)blockIdx.x * 256 >= p.classes) return;
  const int r1 = min(r0 + XENT_APPLY_ROWS, p.rows);
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int vec = blockIdx.x * 32 + cx, c0 = vec * 8;
  const bool col_ok = c0 < p.classes;
  const float inv = 1.0f / (float)(*p.n_valid);
  float cs[8];
#pragma unroll
  for (int t = 0; t < 8; ++t) cs[t] = 0.f;
  // the warp's rows are r0 + ry + 8*k, k < 32: lane k fetches row k's constant and label once, the
  // loop broadcasts them with shuffles (no per-element loads besides the logits themselves)
  static_assert(XENT_APPLY_ROWS == 256, "one row per lane of each of the 8 row-lane warps");
  float c_mine = INFINITY;
  int y_mine = -1;
  {
    int r = r0 + ry + 8 * cx;
    if (r < r1) { c_mine = p.row_c[r]; y_mine = p.y[r]; }
  }
  auto one = [&](uint4 raw, int r, int k) {
    xent_apply_row(raw, __shfl_sync(0xffffffffu, c_mine, k), __shfl_sync(0xffffffffu, y_mine, k), vec, inv, col_ok, cs,
                   (bf16*)p.z + (size_t)r * p.ld + c0);
  };
  {
    const bf16* base = (const bf16*)p.z + (col_ok ? c0 : 0);
    const uint4 zero = make_uint4(0, 0, 0, 0);
    int r = r0 + ry, k = 0;
    for (; r + 24 < r1; r += 32, k += 4) {
      uint4 a0 = zero, a1 = zero, a2 = zero, a3 = zero;
      if (col_ok) {
        a0 = *(const uint4*)(base + (size_t)r * p.ld); a1 = *(const uint4*)(base + (size_t)(r + 8) * p.ld);
        a2 = *(const uint4*)(base + (size_t)(r + 16) * p.ld); a3 = *(const uint4*)(base + (size_t)(r + 24) * p.ld);
      }
      one(a0, r, k); one(a1, r + 8, k + 1); one(a2, r + 16, k + 2); one(a3, r + 24, k + 3);
    }
    for (; r < r1; r += 8, ++k) one(col_ok ? *(const uint4*)(base + (size_t)r * p.ld) : zero, r, k);
  }
  if (!p.colsum_part) return;
#pragma unroll
  for (int t = 0; t < 8; ++t) red[ry][cx][t] = cs[t];
  __syncthreads();
  const int col = threadIdx.x, gc = blockIdx.x * 256 + col;
  if (gc < p.classes) {
    float v = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) v += red[k][col >> 3][col & 7];
    p.colsum_part[(size_t)blockIdx.y * p.classes + gc] = v;
  }
}

}  // namespace

// d must equal nv*256 with nv in {1, 2, 4}; rows, scale and shift 16-byte aligned.
void launch_ln_fwd_vec(const LnProb* d, int n, int max_rows, int nv, cudaStream_t s) {
  dim3 grid((max_rows + LN_FWD_ROWS - 1) / LN_FWD_ROWS, n);
  switch (nv) {
    case 1: ln_fwd_vec_kernel<1><<<grid, 256, 0, s>>>(d); break;
    case 2: ln_fwd_vec_kernel<2><<<grid, 256, 0, s>>>(d); break;
    default: ln_fwd_vec_kernel<4><<<grid, 256, 0, s>>>(d); break;
  }
}
void launch_ln_bwd_vec(const LnBwdProb* d, int n, int max_rows, int nv, cudaStream_t s) {
  dim3 grid((max_rows + LN_BWD_ROWS - 1) / LN_BWD_ROWS, n);
  // [8][2][d] fp32 for the final reduction + 8 warps x LN_RING slots x 3 rows of d bf16
  auto bytes = [](int v) { return (size_t)8 * 2 * v * 256 * sizeof(float) + (size_t)8 * LN_RING * 3 * v * 256 * 2; };
  size_t smem = bytes(nv == 1 || nv == 2 ? nv : 4);
  static bool set = false;
  if (!set) {
    cudaFuncSetAttribute(ln_bwd_vec_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes(1));
    cudaFuncSetAttribute(ln_bwd_vec_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes(2));
    cudaFuncSetAttribute(ln_bwd_vec_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes(4));
    set = true;
  }
  switch (nv) {
    case 1: ln_bwd_vec_kernel<1><<<grid, 256, smem, s>>>(d); break;
    case 2: ln_bwd_vec_kernel<2><<<grid, 256, smem, s>>>(d); break;
    default: ln_bwd_vec_kernel<4><<<grid, 256, smem, s>>>(d); break;
  }
}
// classes and ld multiples of 8, z 16-byte aligned, classes <= nv*2048, nv in {1,2,4,8,16}
// (nv*2048 elements are covered either by 256 threads x nv vectors or by 1024 threads x nv/4).
void launch_xent_vec(const XentProb* d, int n, int max_rows, int nv, cudaStream_t s) {
  dim3 grid(max_rows, n);
  switch (nv) {
    case 1: xent_vec_kernel<1, 256><<<grid, 256, 0, s>>>(d); break;
    case 2: xent_vec_kernel<2, 256><<<grid, 256, 0, s>>>(d); break;
    case 4: xent_vec_kernel<1, 1024><<<grid, 1024, 0, s>>>(d); break;
    case 8: xent_vec_kernel<2, 1024><<<grid, 1024, 0, s>>>(d); break;
    default: xent_vec_kernel<4, 1024><<<grid, 1024, 0, s>>>(d); break;
  }
}

void launch_xent_rows(const XentProb* d, int n, int max_rows, int classes, cudaStream_t s) {
  dim3 grid((max_rows + XENT_ROWS - 1) / XENT_ROWS, n);
  size_t smem = (size_t)classes * sizeof(float);
  static bool set = false;
  if (!set) {
    cudaFuncSetAttribute(xent_rows_kernel<4, 1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4);
    cudaFuncSetAttribute(xent_rows_kernel<2, 1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16384 * 4);
    set = true;
  }
  int nvec = classes / 8;
  if (nvec <= 512) xent_rows_kernel<1, 512><<<grid, 512, smem, s>>>(d);
  else if (nvec <= 1024) xent_rows_kernel<1, 1024><<<grid, 1024, smem, s>>>(d);
  else if (nvec <= 2048) xent_rows_kernel<2, 1024><<<grid, 1024, smem, s>>>(d);
  else xent_rows_kernel<4, 1024><<<grid, 1024, smem, s>>>(d);
}

// classes and ld multiples of 8, z 16-byte aligned
void launch_xent_from_stats(const XentStatsProb* d, int n, int max_rows, int classes, cudaStream_t s) {
  xent_merge_kernel<<<dim3((max_rows + 7) / 8, n), 256, 0, s>>>(d);
  dim3 grid((classes + 255) / 256, (max_rows + XENT_APPLY_ROWS - 1) / XENT_APPLY_ROWS, n);
  xent_apply_kernel<<<grid, 256, 0, s>>>(d);
}

}  // namespace lp
