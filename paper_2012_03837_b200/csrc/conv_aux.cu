// HBM-bound kernels around the convolution GEMMs of the ResNet family (App. B.3): layout change,
// im2col / col2im (gather form, no atomics), train-mode BatchNorm (statistics, apply, backward) with
// fp32 statistics, global average pool.  Activations are NHWC: [N*H*W, C] row-major, so a
// convolution is the GEMM  y[M, C_out] = cols[M, kh*kw*C_in] * W[C_out, kh*kw*C_in]^T.
// blockIdx.y selects the problem.  All reductions have a fixed order.
#include "common.cuh"
#include "grid_barrier.cuh"

namespace lp {
namespace {

template <typename T>
__global__ void __launch_bounds__(256) nchw_to_nhwc_kernel(LayoutProb p) {
  long long total = (long long)p.N * p.C * p.H * p.W;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    int c = (int)(i % p.C);
    long long r = i / p.C;
    int w = (int)(r % p.W); r /= p.W;
    int h = (int)(r % p.H);
    int n = (int)(r / p.H);
    ((T*)p.out)[i] = ((const T*)p.in)[(((long long)n * p.C + c) * p.H + h) * p.W + w];
  }
}

// cols[(n,ho,wo), (i*kw+j)*C + c] = x[n, ho*s+i-pad, wo*s+j-pad, c] (0 outside the image)
template <typename T>
__global__ void __launch_bounds__(256) im2col_kernel(const Im2colProb* __restrict__ probs) {
  const Im2colProb p = probs[blockIdx.y];
  const int K = p.kh * p.kw * p.C;
  long long total = (long long)p.N * p.Ho * p.Wo * K;
  const T* x = (const T*)p.x;
  T* cols = (T*)p.cols;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    int kk = (int)(e % K);
    long long m = e / K;
    int c = kk % p.C, tap = kk / p.C;
    int i = tap / p.kw, j = tap % p.kw;
    int wo = (int)(m % p.Wo);
    long long r = m / p.Wo;
    int ho = (int)(r % p.Ho);
    int n = (int)(r / p.Ho);
    int h = ho * p.stride + i - p.pad, w = wo * p.stride + j - p.pad;
    T v = from_f<T>(0.f);
    if (h >= 0 && h < p.H && w >= 0 && w < p.W) v = x[(((long long)n * p.H + h) * p.W + w) * p.C + c];
    cols[m * p.ldk + kk] = v;
  }
}

// dx[n,h,w,c] = sum over taps (i,j) with h = ho*s+i-pad, w = wo*s+j-pad of dcols[(n,ho,wo), (i*kw+j)*C+c]
template <typename T>
__global__ void __launch_bounds__(256) col2im_kernel(const Im2colProb* __restrict__ probs) {
  const Im2colProb p = probs[blockIdx.y];
  long long total = (long long)p.N * p.H * p.W * p.C;
  const T* cols = (const T*)p.cols;
  T* dx = (T*)p.x;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    int c = (int)(e % p.C);
    long long r = e / p.C;
    int w = (int)(r % p.W); r /= p.W;
    int h = (int)(r % p.H);
    int n = (int)(r / p.H);
    float s = 0.f;
    for (int i = 0; i < p.kh; ++i) {
      int hh = h + p.pad - i;
      if (hh < 0 || hh % p.stride) continue;
      int ho = hh / p.stride;
      if (ho >= p.Ho) continue;
      for (int j = 0; j < p.kw; ++j) {
        int ww = w + p.pad - j;
        if (ww < 0 || ww % p.stride) continue;
        int wo = ww / p.stride;
        if (wo >= p.Wo) continue;
        long long m = ((long long)n * p.Ho + ho) * p.Wo + wo;
        s += to_f(cols[m * p.ldk + (i * p.kw + j) * p.C + c]);
      }
    }
    dx[e] = from_f<T>(s);
  }
}

// Per-channel partial sums over a block of bn_rows_per_block(rows) rows.
//   forward : part[blk][0][c] = sum x,   part[blk][1][c] = sum x^2
//   backward: part[blk][0][c] = sum dyr * xhat, part[blk][1][c] = sum dyr, dyr = dy * [relu_out > 0]
template <typename T, bool BWD>
__global__ void __launch_bounds__(256) bn_stat_kernel(const BnStatProb* __restrict__ probs) {
  const BnStatProb p = probs[blockIdx.z];
  const int rpb = bn_rows_per_block(p.rows);
  int r0 = blockIdx.y * rpb;
  if (r0 >= p.rows) return;
  int r1 = min(r0 + rpb, p.rows);
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= p.C) return;
  const T* x = (const T*)p.x;
  float a = 0.f, b = 0.f;
  if (BWD) {
    const T* dy = (const T*)p.dy;
    const T* ro = (const T*)p.relu_out;
    float mu = p.mean[c], rs = p.rstd[c];
    for (int r = r0; r < r1; ++r) {
      size_t off = (size_t)r * p.C + c;
      float g = to_f(dy[off]);
      if (ro && !(to_f(ro[off]) > 0.f)) g = 0.f;
      a += g * (to_f(x[off]) - mu) * rs;
      b += g;
    }
  } else {
    for (int r = r0; r < r1; ++r) {
      float v = to_f(x[(size_t)r * p.C + c]);
      a += v;
      b += v * v;
    }
  }
  float* part = p.part + (size_t)blockIdx.y * 2 * p.C;
  part[c] = a;
  part[p.C + c] = b;
}

// forward: mean and 1/sqrt(biased variance + eps); backward: dgamma, dbeta.  One warp per channel:
// lane l sums partial blocks l, l+32, ... in double, then a fixed shuffle tree combines the lanes.
template <bool BWD>
__device__ __forceinline__ void bn_finalize_channel(const BnFinalProb& p, int c, int lane) {
  if (!BWD && p.use_running) {                 // evaluation mode: normalise with the running statistics
    if (lane == 0) {
      p.mean[c] = p.run_mean[c];
      p.rstd[c] = (float)(1.0 / sqrt((double)p.run_var[c] + (double)p.eps));
    }
    return;
  }
  double a = 0.0, b = 0.0;
  int k = lane;
  for (; k + 7 * 32 < p.nblk; k += 8 * 32) {     // eight partial blocks per pass: sixteen loads in flight, same order of sums
    float va[8], vb[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      va[u] = __ldcg(p.part + (size_t)(k + u * 32) * 2 * p.C + c);
      vb[u] = __ldcg(p.part + (size_t)(k + u * 32) * 2 * p.C + p.C + c);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) { a += (double)va[u]; b += (double)vb[u]; }
  }
  for (; k < p.nblk; k += 32) {
    a += (double)__ldcg(p.part + (size_t)k * 2 * p.C + c);
    b += (double)__ldcg(p.part + (size_t)k * 2 * p.C + p.C + c);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, o);
    b += __shfl_xor_sync(0xffffffffu, b, o);
  }
  if (lane != 0) return;
  if (BWD) {
    p.dgamma[c] = (float)a;
    p.dbeta[c] = (float)b;
  } else {
    double mu = a / p.rows;
    double var = b / p.rows - mu * mu;
    if (var < 0.0) var = 0.0;
    p.mean[c] = (float)mu;
    p.rstd[c] = (float)(1.0 / sqrt(var + (double)p.eps));
    if (p.run_mean && !(p.chunk_tab && p.chunk_tab[p.chunk].x == 0.f)) {   // training step: exponential averages
      const double m = (double)p.momentum, unb = var * ((double)p.rows / (double)(p.rows > 1 ? p.rows - 1 : 1));
      p.run_mean[c] = (float)((1.0 - m) * (double)p.run_mean[c] + m * mu);
      p.run_var[c] = (float)((1.0 - m) * (double)p.run_var[c] + m * unb);
    }
  }
}
template <bool BWD>
__global__ void __launch_bounds__(256) bn_finalize_kernel(const BnFinalProb* __restrict__ probs) {
  const BnFinalProb p = probs[blockIdx.y];
  const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (c < p.C) bn_finalize_channel<BWD>(p, c, threadIdx.x & 31);
}

template <typename T, bool BWD>
__global__ void __launch_bounds__(256) bn_apply_kernel(const BnApplyProb* __restrict__ probs) {
  const BnApplyProb p = probs[blockIdx.y];
  long long total = (long long)p.rows * p.C;
  const T* x = (const T*)p.x;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    int c = (int)(e % p.C);
    float xh = (to_f(x[e]) - p.mean[c]) * p.rstd[c];
    if (!BWD) {
      float v = xh * p.g[c] + p.b[c];
      if (p.res) v += to_f(((const T*)p.res)[e]);
      if (p.relu) v = relu_f(v);
      ((T*)p.y)[e] = from_f<T>(v);
    } else {
      float g = to_f(((const T*)p.dy)[e]);
      if (p.relu_out && !(to_f(((const T*)p.relu_out)[e]) > 0.f)) g = 0.f;
      if (p.dres_out) ((T*)p.dres_out)[e] = from_f<T>(g);
      float inv = 1.0f / (float)p.rows;
      float v = p.rstd[c] * p.g[c] * (g - p.dbeta[c] * inv - xh * p.dgamma[c] * inv);
      ((T*)p.dx)[e] = from_f<T>(v);
    }
  }
}

// y[n, c] = mean over hw of x[n, hw, c]
template <typename T>
__global__ void __launch_bounds__(256) gap_fwd_kernel(const GapProb* __restrict__ probs) {
  const GapProb p = probs[blockIdx.z];
  int n = blockIdx.y;
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= p.N || c >= p.C) return;
  const T* x = (const T*)p.x + (size_t)n * p.HW * p.C;
  float s = 0.f;
  for (int i = 0; i < p.HW; ++i) s += to_f(x[(size_t)i * p.C + c]);
  ((T*)p.y)[(size_t)n * p.C + c] = from_f<T>(s / p.HW);
}
template <typename T>
__global__ void __launch_bounds__(256) gap_bwd_kernel(const GapProb* __restrict__ probs) {
  const GapProb p = probs[blockIdx.y];
  long long total = (long long)p.N * p.HW * p.C;
  float inv = 1.0f / p.HW;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    int c = (int)(e % p.C);
    int n = (int)(e / ((long long)p.HW * p.C));
    ((T*)p.dx)[e] = from_f<T>(to_f(((const T*)p.dy)[(size_t)n * p.C + c]) * inv);
  }
}

// ------------------------------------------------------------------ 128-bit bf16 variants (C % 8 == 0)
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

__global__ void __launch_bounds__(256) im2col_vec_kernel(const Im2colProb* __restrict__ probs) {
  const Im2colProb p = probs[blockIdx.y];
  const int cv = p.C >> 3, taps = p.kh * p.kw;
  long long total = (long long)p.N * p.Ho * p.Wo * taps * cv;
  const bf16* x = (const bf16*)p.x;
  bf16* cols = (bf16*)p.cols;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    int c8 = (int)(e % cv);
    long long r = e / cv;
    int tap = (int)(r % taps);
    long long m = r / taps;
    int i = tap / p.kw, j = tap % p.kw;
    int wo = (int)(m % p.Wo);
    long long q = m / p.Wo;
    int ho = (int)(q % p.Ho);
    int n = (int)(q / p.Ho);
    int h = ho * p.stride + i - p.pad, w = wo * p.stride + j - p.pad;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (h >= 0 && h < p.H && w >= 0 && w < p.W) v = *(const uint4*)(x + (((long long)n * p.H + h) * p.W + w) * p.C + c8 * 8);
    *(uint4*)(cols + m * p.ldk + tap * p.C + c8 * 8) = v;
  }
}

__global__ void __launch_bounds__(256) col2im_vec_kernel(const Im2colProb* __restrict__ probs) {
  const Im2colProb p = probs[blockIdx.y];
  const int cv = p.C >> 3;
  long long total = (long long)p.N * p.H * p.W * cv;
  const bf16* cols = (const bf16*)p.cols;
  bf16* dx = (bf16*)p.x;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    int c8 = (int)(e % cv);
    long long r = e / cv;
    int w = (int)(r % p.W); r /= p.W;
    int h = (int)(r % p.H);
    int n = (int)(r / p.H);
    float s[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int i = 0; i < p.kh; ++i) {
      int hh = h + p.pad - i;
      if (hh < 0 || hh % p.stride) continue;
      int ho = hh / p.stride;
      if (ho >= p.Ho) continue;
      for (int j = 0; j < p.kw; ++j) {
        int ww = w + p.pad - j;
        if (ww < 0 || ww % p.stride) continue;
        int wo = ww / p.stride;
        if (wo >= p.Wo) continue;
        long long m = ((long long)n * p.Ho + ho) * p.Wo + wo;
        float f[8];
        unpack8(*(const uint4*)(cols + m * p.ldk + (i * p.kw + j) * p.C + c8 * 8), f);
#pragma unroll
        for (int t = 0; t < 8; ++t) s[t] += f[t];
      }
    }
    *(uint4*)(dx + e * 8) = pack8(s);
  }
}

// Block of 256 threads = (C/8 channel vectors) x (256 / (C/8) row lanes) over the block's rows; the row
// lanes are summed through shared memory in lane order.  Requires C % 8 == 0 and C/8 <= 256.
// Thread (tx, ty) of the block adds rows r0 + ty, r0 + ty + ny, ... of its channel vector tx to a / b.
template <bool BWD, int U>
__device__ __forceinline__ void bn_stat_vec_accum(const BnStatProb& p, int row_block, float (&a)[8], float (&b)[8]) {
  const int rpb = bn_rows_per_block(p.rows);
  const int r0 = row_block * rpb;
  const int r1 = min(r0 + rpb, p.rows);
  const int cv = p.C >> 3, ny = 256 / cv;
  const int tx = threadIdx.x % cv, ty = threadIdx.x / cv;
  if (ty >= ny) return;
  const bf16* x = (const bf16*)p.x;
  float mu[8], rs[8];
  if (BWD) {
#pragma unroll
    for (int t = 0; t < 8; ++t) { mu[t] = p.mean[tx * 8 + t]; rs[t] = p.rstd[tx * 8 + t]; }
  }
  // several rows per pass, every load of a pass issued before the first sum (the rows are added in their order)
  for (int r = r0 + ty; r < r1; r += U * ny) {
    uint4 xr[U], gr[U], rr[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int ru = r + u * ny;
      if (ru < r1) {
        const size_t off = (size_t)ru * p.C + tx * 8;
        xr[u] = *(const uint4*)(x + off);
        if (BWD) {
          gr[u] = *(const uint4*)((const bf16*)p.dy + off);
          if (p.relu_out) rr[u] = *(const uint4*)((const bf16*)p.relu_out + off);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (r + u * ny >= r1) break;
      float xv[8];
      unpack8(xr[u], xv);
      if (BWD) {
        float g[8];
        unpack8(gr[u], g);
        if (p.relu_out) {
          float ro[8];
          unpack8(rr[u], ro);
#pragma unroll
          for (int t = 0; t < 8; ++t) if (!(ro[t] > 0.f)) g[t] = 0.f;
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) { a[t] += g[t] * (xv[t] - mu[t]) * rs[t]; b[t] += g[t]; }
      } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) { a[t] += xv[t]; b[t] += xv[t] * xv[t]; }
      }
    }
  }
}
// The block's row lanes summed through shared memory in lane order; row `out_row` of the partial sums [.][2][C].
__device__ __forceinline__ void bn_stat_vec_reduce(const BnStatProb& p, int out_row, const float (&a)[8], const float (&b)[8],
                                                   float* red) {   // red: 256 * 16 floats
  const int cv = p.C >> 3, ny = 256 / cv;
  // red[value][thread]: the 16 partial values of a thread go to 16 different rows, so that a warp's stores, and
  // the loads below (channel vectors of one value and line side by side), touch 32 different banks.
#pragma unroll
  for (int t = 0; t < 8; ++t) { red[t * 256 + threadIdx.x] = a[t]; red[(8 + t) * 256 + threadIdx.x] = b[t]; }
  __syncthreads();
  // thread (which, t, j) sums lane 0..ny-1 for channel j * 8 + t, in lane order
  for (int idx = threadIdx.x; idx < 2 * p.C; idx += 256) {
    const int j = idx % cv, vt = idx / cv;             // vt = which * 8 + t
    float s = 0.f;
    for (int l = 0; l < ny; ++l) s += red[vt * 256 + l * cv + j];
    p.part[(size_t)out_row * 2 * p.C + (vt >> 3) * p.C + j * 8 + (vt & 7)] = s;
  }
}
template <bool BWD>
__global__ void __launch_bounds__(256) bn_stat_vec_kernel(const BnStatProb* __restrict__ probs) {
  __shared__ float red[256 * 16];
  const BnStatProb p = probs[blockIdx.z];
  if ((long long)blockIdx.y * bn_rows_per_block(p.rows) >= p.rows) return;
  float a[8], b[8];
#pragma unroll
  for (int t = 0; t < 8; ++t) { a[t] = 0.f; b[t] = 0.f; }
  bn_stat_vec_accum<BWD, BWD ? 2 : 4>(p, blockIdx.y, a, b);
  bn_stat_vec_reduce(p, blockIdx.y, a, b, red);
}

// dx[n, hw, c] = dy[n, c] / HW, bf16 with C % 8 == 0: eight channels per access
__global__ void __launch_bounds__(256) gap_bwd_vec_kernel(const GapProb* __restrict__ probs) {
  const GapProb p = probs[blockIdx.y];
  const int cv = p.C >> 3;
  const long long per_image = (long long)p.HW * cv, total = (long long)p.N * per_image;
  const float inv = 1.0f / p.HW;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(e / per_image), j = (int)(e % cv);
    float g[8];
    unpack8(*(const uint4*)((const bf16*)p.dy + (size_t)n * p.C + j * 8), g);
#pragma unroll
    for (int t = 0; t < 8; ++t) g[t] *= inv;
    *(uint4*)((bf16*)p.dx + e * 8) = pack8(g);
  }
}

// y[n, c] = mean over hw of x[n, hw, c], bf16: one block per image.  With C % 8 == 0 and C / 8 <= 256 the block
// is (C/8 channel vectors) x (256 / (C/8) pixel lanes) reading 16 bytes at a time, the pixel lanes summed through
// shared memory in lane order; otherwise each thread walks the pixels of its channels.
__global__ void __launch_bounds__(256) gap_fwd_vec_kernel(const GapProb* __restrict__ probs) {
  __shared__ float red[256 * 8];
  const GapProb p = probs[blockIdx.z];
  const int n = blockIdx.y;
  if (n >= p.N) return;
  const bf16* x = (const bf16*)p.x + (size_t)n * p.HW * p.C;
  bf16* y = (bf16*)p.y + (size_t)n * p.C;
  const float inv = 1.0f / p.HW;
  if ((p.C & 7) != 0 || (p.C >> 3) > 256) {
    for (int c = threadIdx.x; c < p.C; c += 256) {
      float s = 0.f;
      for (int i = 0; i < p.HW; ++i) s += __bfloat162float(x[(size_t)i * p.C + c]);
      y[c] = __float2bfloat16(s * inv);
    }
    return;
  }
  const int cv = p.C >> 3, ny = 256 / cv;
  const int tx = threadIdx.x % cv, ty = threadIdx.x / cv;
  float a[8];
#pragma unroll
  for (int t = 0; t < 8; ++t) a[t] = 0.f;
  if (ty < ny)
    for (int i = ty; i < p.HW; i += ny) {
      float v[8];
      unpack8(*(const uint4*)(x + (size_t)i * p.C + tx * 8), v);
#pragma unroll
      for (int t = 0; t < 8; ++t) a[t] += v[t];
    }
#pragma unroll
  for (int t = 0; t < 8; ++t) red[t * 256 + threadIdx.x] = a[t];
  __syncthreads();
  for (int idx = threadIdx.x; idx < p.C; idx += 256) {
    const int j = idx % cv, t = idx / cv;
    float s = 0.f;
    for (int l = 0; l < ny; ++l) s += red[t * 256 + l * cv + j];
    y[j * 8 + t] = __float2bfloat16(s * inv);
  }
}

// The per-channel constants are formed once per block in shared memory (a thread would otherwise issue some
// thirty scalar loads for every 16 bytes of data).  A thread's channel vector is the same in every pass of the
// grid-stride loop when the stride is a multiple of C / 8 (always so for power-of-two channel counts): it then
// keeps its constants in registers.
// Elements first, first + stride, ... (in 16-byte vectors) of one problem; every thread of the block calls it
// (the constants are formed by the whole block).
template <bool BWD, int U>
__device__ __forceinline__ void bn_apply_vec_range(const BnApplyProb& p, long long first, long long stride, float (*cst)[2048]) {
  const int cv = p.C >> 3;
  const long long total = (long long)p.rows * cv;
  const bool fixed = stride % cv == 0;
  const bf16* x = (const bf16*)p.x;
  const float inv = 1.0f / (float)p.rows;
  // forward: y = (x - mu) * ka + kb;  backward: dx = ka * (dyr - kb - (x - mu) * kc)
  for (int c = threadIdx.x; c < p.C; c += 256) {
    const float rs = __ldcg(p.rstd + c);
    cst[0][c] = __ldcg(p.mean + c);
    cst[1][c] = rs * p.g[c];
    cst[2][c] = BWD ? __ldcg(p.dbeta + c) * inv : p.b[c];
    cst[3][c] = BWD ? rs * __ldcg(p.dgamma + c) * inv : 0.f;
  }
  __syncthreads();
  float mu[8], ka[8], kb[8], kc[8];
  auto constants = [&](int c0) {
    *(float4*)&mu[0] = *(const float4*)&cst[0][c0]; *(float4*)&mu[4] = *(const float4*)&cst[0][c0 + 4];
    *(float4*)&ka[0] = *(const float4*)&cst[1][c0]; *(float4*)&ka[4] = *(const float4*)&cst[1][c0 + 4];
    *(float4*)&kb[0] = *(const float4*)&cst[2][c0]; *(float4*)&kb[4] = *(const float4*)&cst[2][c0 + 4];
    if (BWD) { *(float4*)&kc[0] = *(const float4*)&cst[3][c0]; *(float4*)&kc[4] = *(const float4*)&cst[3][c0 + 4]; }
  };
  long long e = first;
  if (fixed && e < total) constants((int)(e % cv) * 8);
  // U vectors per pass, every load of a pass issued before the first store: enough bytes in flight per SM to
  // cover the memory latency with two or three blocks of 256 threads
  for (; e < total; e += stride * U) {
    uint4 xr[U], ar[U], rr[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long eu = e + u * stride;
      if (eu < total) {
        xr[u] = *(const uint4*)(x + eu * 8);
        if (!BWD) {
          if (p.res) ar[u] = *(const uint4*)((const bf16*)p.res + eu * 8);
        } else {
          ar[u] = *(const uint4*)((const bf16*)p.dy + eu * 8);
          if (p.relu_out) rr[u] = *(const uint4*)((const bf16*)p.relu_out + eu * 8);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long eu = e + u * stride;
      if (eu >= total) break;
      if (!fixed) constants((int)(eu % cv) * 8);
      float xv[8], o[8];
      unpack8(xr[u], xv);
      if (!BWD) {
        float r[8];
        if (p.res) unpack8(ar[u], r);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          float v = (xv[t] - mu[t]) * ka[t] + kb[t];
          if (p.res) v += r[t];
          o[t] = p.relu ? relu_f(v) : v;
        }
        *(uint4*)((bf16*)p.y + eu * 8) = pack8(o);
      } else {
        float g[8];
        unpack8(ar[u], g);
        if (p.relu_out) {
          float ro[8];
          unpack8(rr[u], ro);
#pragma unroll
          for (int t = 0; t < 8; ++t) if (!(ro[t] > 0.f)) g[t] = 0.f;
        }
        if (p.dres_out) *(uint4*)((bf16*)p.dres_out + eu * 8) = pack8(g);
#pragma unroll
        for (int t = 0; t < 8; ++t) o[t] = ka[t] * (g[t] - kb[t] - (xv[t] - mu[t]) * kc[t]);
        *(uint4*)((bf16*)p.dx + eu * 8) = pack8(o);
      }
    }
  }
}
template <bool BWD>
__global__ void __launch_bounds__(256, 3) bn_apply_vec_kernel(const BnApplyProb* __restrict__ probs) {
  __shared__ __align__(16) float cst[4][2048];          // C <= 2048 (C / 8 <= 256)
  const BnApplyProb p = probs[blockIdx.y];
  if ((long long)blockIdx.x * blockDim.x >= (long long)p.rows * (p.C >> 3)) return;
  bn_apply_vec_range<BWD, BWD ? 2 : 4>(p, (long long)blockIdx.x * blockDim.x + threadIdx.x, (long long)gridDim.x * blockDim.x, cst);
}

// Per-channel totals of the fused kernel: one block per tile of 8 channels (a 32-byte sector of a row of the
// partial sums [nrow][2][C]).  Lane (channel cs, row lane rl) of warp w takes rows 4 w + rl, + 32, + 64, ...; both
// sums of up to 16 rows are in flight at once.  A lane adds its rows in double in row order, then the four row
// lanes and the eight warps are added in a fixed order.
template <bool BWD>
__device__ __forceinline__ void bn_finalize_tile(const BnFinalProb& p, int tile, double (*wsum)[2][8]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int cs = lane & 7, rl = lane >> 3;
  const int c = tile * 8 + cs;                 // < C: C is a multiple of 8
  if (!BWD && p.use_running) {                 // evaluation mode: normalise with the running statistics
    if (warp == 0 && rl == 0) {
      p.mean[c] = p.run_mean[c];
      p.rstd[c] = (float)(1.0 / sqrt((double)p.run_var[c] + (double)p.eps));
    }
    return;
  }
  constexpr int PER = 16;                      // rows of each sum a lane has in flight at once
  double sa = 0.0, sb = 0.0;
  for (int k0 = warp * 4 + rl; k0 < p.nblk; k0 += 32 * PER) {
    float va[PER], vb[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int k = k0 + 32 * i;
      va[i] = k < p.nblk ? __ldcg(p.part + (size_t)k * 2 * p.C + c) : 0.0f;
      vb[i] = k < p.nblk ? __ldcg(p.part + (size_t)k * 2 * p.C + p.C + c) : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) { sa += (double)va[i]; sb += (double)vb[i]; }
  }
  sa += __shfl_xor_sync(0xffffffffu, sa, 8);  sb += __shfl_xor_sync(0xffffffffu, sb, 8);
  sa += __shfl_xor_sync(0xffffffffu, sa, 16); sb += __shfl_xor_sync(0xffffffffu, sb, 16);
  if (rl == 0) { wsum[warp][0][cs] = sa; wsum[warp][1][cs] = sb; }
  __syncthreads();
  if (warp == 0 && rl == 0) {
    double a = 0.0, b = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { a += wsum[w][0][cs]; b += wsum[w][1][cs]; }
    if (BWD) {
      p.dgamma[c] = (float)a;
      p.dbeta[c] = (float)b;
    } else {
      double mu = a / p.rows;
      double var = b / p.rows - mu * mu;
      if (var < 0.0) var = 0.0;
      p.mean[c] = (float)mu;
      p.rstd[c] = (float)(1.0 / sqrt(var + (double)p.eps));
      if (p.run_mean && !(p.chunk_tab && p.chunk_tab[p.chunk].x == 0.f)) {   // training step: exponential averages
        const double m = (double)p.momentum, unb = var * ((double)p.rows / (double)(p.rows > 1 ? p.rows - 1 : 1));
        p.run_mean[c] = (float)((1.0 - m) * (double)p.run_mean[c] + m * mu);
        p.run_var[c] = (float)((1.0 - m) * (double)p.run_var[c] + m * unb);
      }
    }
  }
  __syncthreads();
}

// BatchNorm of a whole launch group in ONE cooperative launch (bf16, C % 8 == 0): the three passes above --
// partial sums, per-channel totals, normalisation -- separated by grid-wide barriers instead of kernel
// boundaries.  The tensor the first pass has just pulled through L2 is still there for the third (a 33 MB
// activation of the first stage is read from HBM once, not twice), two launch latencies go away, and since the
// blocks are known to be co-resident each of them sums ALL its blocks of rows into one partial row, so the
// second pass adds a few hundred rows per channel instead of a thousand.  fin.nblk of a problem is the number
// of partial rows the launch produces for it: min(blocks of rows, blocks of the launch).
template <bool BWD>
__global__ void __launch_bounds__(256, BWD ? 2 : 3) bn_fused_kernel(const BnFusedProb* __restrict__ probs, int n, int stats,
                                                                    unsigned long long* counter, int* status) {
  __shared__ __align__(16) float buf[4][2048];
  __shared__ double wsum[8][2][8];
  constexpr int U = 4;
  bool alive = true;
  if (stats) {
    int item = blockIdx.x;
    for (int i = 0; i < n; ++i) {                        // (problem, block of rows) pairs, round-robin over the blocks
      const BnStatProb p = probs[i].st;
      const int nblk = bn_blocks(p.rows);
      if (item < nblk) {
        const int out_row = item;                        // < gridDim.x
        float a[8], b[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) { a[t] = 0.f; b[t] = 0.f; }
        for (; item < nblk; item += gridDim.x) bn_stat_vec_accum<BWD, U>(p, item, a, b);
        bn_stat_vec_reduce(p, out_row, a, b, &buf[0][0]);
        __syncthreads();
      }
      item -= nblk;
    }
    alive = grid_barrier(counter, (unsigned long long)gridDim.x, status);
  }
  if (alive) {
    int tile = blockIdx.x;
    for (int i = 0; i < n; ++i) {                        // one block per (problem, tile of 8 channels)
      const int tiles = probs[i].fin.C >> 3;
      if (tile < tiles) {
        const BnFinalProb p = probs[i].fin;
        for (; tile < tiles; tile += gridDim.x) bn_finalize_tile<BWD>(p, tile, wsum);
      }
      tile -= tiles;
    }
    alive = grid_barrier(counter, (unsigned long long)(stats ? 2 : 1) * gridDim.x, status);
  }
  if (alive) {
    for (int i = 0; i < n; ++i) {
      const BnApplyProb p = probs[i].ap;
      bn_apply_vec_range<BWD, U>(p, (long long)blockIdx.x * blockDim.x + threadIdx.x, (long long)gridDim.x * blockDim.x, buf);
      __syncthreads();
    }
  }
  grid_barrier_leave(counter);
}

// ------------------------------------------------------------------ few-channel 3x3 convolution (the stem)
// Both kernels stage, for a group of consecutive pixels, the 9 * Cin input values around each pixel (zero outside
// the image) in shared memory as fp32, padded to 32 per pixel, and work on register tiles from there: a thread
// re-reads from shared memory one value per four to eight multiply-adds instead of one per multiply-add.
constexpr int SC_KP = 32;                             // staged reduction length per pixel: 9 * Cin <= 32, zero padded

// patch[pl][k] for pixels base .. base + NPIX - 1 (k = tap * Cin + c), row pitch SC_KP + 4 floats.  blockDim.x / NPIX
// threads share a pixel; each stages the same SC_KP / (threads per pixel) values of k for every pixel it meets, so
// the tap offsets of those k are worked out once (StageTaps) and a pixel's coordinates once per thread and group:
// no division per staged value.
template <int NPIX>
struct StageTaps {
  static constexpr int TPP = 256 / NPIX, KPER = SC_KP / TPP;
  int pl, k0;
  signed char dh[KPER], dw[KPER], c[KPER];            // c < 0: k beyond 9 * Cin (stays zero)
  __device__ __forceinline__ void init(int Cin) {
    pl = threadIdx.x / TPP; k0 = (threadIdx.x % TPP) * KPER;
#pragma unroll
    for (int j = 0; j < KPER; ++j) {
      const int k = k0 + j, tap = k / Cin;
      dh[j] = (signed char)(tap / 3 - 1); dw[j] = (signed char)(tap % 3 - 1);
      c[j] = (signed char)(k < 9 * Cin ? k - tap * Cin : -1);
    }
  }
};
template <typename T, int NPIX>
__device__ __forceinline__ void stage_patch(const SmallConvProb& p, const StageTaps<NPIX>& st, long long base, long long total,
                                            float* patch) {
  const T* x = (const T*)p.x;
  const int pix = (int)base + st.pl;                   // the pixel count of a problem is below 2^31 (checked by the launchers)
  const bool in = pix < total;
  const int row = in ? pix / p.W : 0;
  const int w0 = in ? pix - row * p.W : 0;
  const int h0 = row % p.H;
  const T* img = x + (size_t)(row - h0) * p.W * p.Cin;   // first pixel of the image
  float* dst = patch + st.pl * (SC_KP + 4) + st.k0;
#pragma unroll
  for (int j = 0; j < StageTaps<NPIX>::KPER; ++j) {
    const int hh = h0 + st.dh[j], ww = w0 + st.dw[j];
    float v = 0.f;
    if (in && st.c[j] >= 0 && hh >= 0 && hh < p.H && ww >= 0 && ww < p.W) v = to_f(img[((size_t)hh * p.W + ww) * p.Cin + st.c[j]]);
    dst[j] = v;
  }
}

// Forward: a block of 256 threads takes groups of 64 pixels; thread (pixel pair, group of 8 output channels)
// holds 2 x 8 sums.  Filters transposed to [k][COUT] in shared memory once per block.  COUT is a template
// parameter (8, 16, 32 or 64): the index computations are shifts and the pair loop has a fixed trip count.
constexpr int SCF_PIX = 64;
template <typename T, typename WT, int COUT>
__global__ void __launch_bounds__(256) small_conv_fwd_kernel(SmallConvProb p) {
  extern __shared__ __align__(16) float sc_smem[];    // [9 * Cin][COUT] filters, then [SCF_PIX][SC_KP + 4] patch
  const int K = 9 * p.Cin;
  float* ws = sc_smem;
  float* patch = sc_smem + K * COUT;
  for (int i = threadIdx.x; i < K * COUT; i += blockDim.x) {
    int co = i / K, k = i - co * K;
    ws[k * COUT + co] = to_f(((const WT*)p.w)[i]);
  }
  constexpr int GROUPS = COUT / 8;                    // threads per pixel pair
  constexpr int PAIRS = 256 / GROUPS;                 // pixel pairs a pass of the block covers
  const int g = threadIdx.x % GROUPS, pp = threadIdx.x / GROUPS;
  const long long total = (long long)p.N * p.H * p.W;
  StageTaps<SCF_PIX> taps;
  taps.init(p.Cin);
  for (long long base = (long long)blockIdx.x * SCF_PIX; base < total; base += (long long)gridDim.x * SCF_PIX) {
    __syncthreads();                                  // filters staged / the previous group's patch has been read
    stage_patch<T, SCF_PIX>(p, taps, base, total, patch);
    __syncthreads();
#pragma unroll
    for (int q0 = 0; q0 < SCF_PIX / 2; q0 += PAIRS) {
      const int q = q0 + pp;
      if (q >= SCF_PIX / 2) break;
      const float* x0 = patch + (2 * q) * (SC_KP + 4);
      const float* x1 = x0 + (SC_KP + 4);
      float a0[8], a1[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) { a0[t] = 0.f; a1[t] = 0.f; }
      for (int k4 = 0; k4 < K; k4 += 4) {             // the patch is zero beyond K, the filter rows are not read there
        const float4 u4 = *(const float4*)(x0 + k4), v4 = *(const float4*)(x1 + k4);
        const float uu[4] = {u4.x, u4.y, u4.z, u4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (k4 + j >= K) break;
          const float4* wr = (const float4*)(ws + (k4 + j) * COUT + g * 8);
          const float4 w0 = wr[0], w1 = wr[1];
          const float u = uu[j], v = vv[j];
          a0[0] = fmaf(u, w0.x, a0[0]); a0[1] = fmaf(u, w0.y, a0[1]); a0[2] = fmaf(u, w0.z, a0[2]); a0[3] = fmaf(u, w0.w, a0[3]);
          a0[4] = fmaf(u, w1.x, a0[4]); a0[5] = fmaf(u, w1.y, a0[5]); a0[6] = fmaf(u, w1.z, a0[6]); a0[7] = fmaf(u, w1.w, a0[7]);
          a1[0] = fmaf(v, w0.x, a1[0]); a1[1] = fmaf(v, w0.y, a1[1]); a1[2] = fmaf(v, w0.z, a1[2]); a1[3] = fmaf(v, w0.w, a1[3]);
          a1[4] = fmaf(v, w1.x, a1[4]); a1[5] = fmaf(v, w1.y, a1[5]); a1[6] = fmaf(v, w1.z, a1[6]); a1[7] = fmaf(v, w1.w, a1[7]);
        }
      }
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        const long long pix = base + 2 * q + h2;
        if (pix >= total) continue;
        const float* a = h2 ? a1 : a0;
        T* y = (T*)p.y + pix * COUT + g * 8;
        if (sizeof(T) == 2) {
          *(uint4*)y = pack8(a);                      // COUT % 8 == 0: 16-byte aligned
        } else {
#pragma unroll
          for (int t = 0; t < 8; ++t) y[t] = from_f<T>(a[t]);
        }
      }
    }
  }
}

// Filter gradient: part[blk][co * 9 Cin + k] = sum over block blk's SMALLCONV_PIXELS pixels of dy[pixel, co] *
// patch[pixel, k].  Thread (pixel lane, group of 8 k, group of 4 output channels) holds 4 x 8 sums over the pixels
// of its lane (pixel index mod lanes) of each staged group of 32; the lanes are added in lane order at the end.
// COUT is a template parameter (8, 16, 32 or 64): every index computation is a shift and the loops unroll.
template <typename T, int COUT>
__global__ void __launch_bounds__(256) small_conv_wgrad_kernel(SmallConvProb p) {
  extern __shared__ __align__(16) float sc_smem[];    // [32][SC_KP + 4] patch, [32][COUT] dy; later [lanes][COUT * 32] sums
  const int K = 9 * p.Cin;
  float* patch = sc_smem;
  float* dys = sc_smem + 32 * (SC_KP + 4);
  constexpr int CG4 = COUT / 4;                       // threads along the output channels
  constexpr int PER_LANE = CG4 * (SC_KP / 8);         // threads of one pixel lane
  constexpr int LANES = 256 / PER_LANE;               // 4 for COUT = 64
  const int lane_q = threadIdx.x / PER_LANE, r = threadIdx.x % PER_LANE;
  const int kq = r / CG4, c4 = r % CG4;
  const long long total = (long long)p.N * p.H * p.W;
  const long long p0 = (long long)blockIdx.x * SMALLCONV_PIXELS;
  float acc[4][8];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  const T* dy = (const T*)p.dy;
  StageTaps<32> taps;
  taps.init(p.Cin);
  for (long long base = p0; base < p0 + SMALLCONV_PIXELS && base < total; base += 32) {
    __syncthreads();
    stage_patch<T, 32>(p, taps, base, total, patch);
    // the 32 x COUT output gradients of the group are contiguous in memory: eight values per thread
    for (int i8 = threadIdx.x; i8 < 32 * COUT / 8; i8 += 256) {
      const long long pix = base + (i8 * 8) / COUT;
      float v[8];
      if (pix < total) {
        if (sizeof(T) == 2) {
          unpack8(*(const uint4*)((const bf16*)p.dy + (size_t)base * COUT + i8 * 8), v);
        } else {
#pragma unroll
          for (int t = 0; t < 8; ++t) v[t] = to_f(dy[(size_t)base * COUT + i8 * 8 + t]);
        }
      } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) v[t] = 0.f;
      }
      *(float4*)(dys + i8 * 8) = make_float4(v[0], v[1], v[2], v[3]);
      *(float4*)(dys + i8 * 8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
    }
    __syncthreads();
#pragma unroll
    for (int pl = lane_q; pl < 32; pl += LANES) {
      const float4 d = *(const float4*)(dys + pl * COUT + c4 * 4);
      const float4 u0 = *(const float4*)(patch + pl * (SC_KP + 4) + kq * 8);
      const float4 u1 = *(const float4*)(patch + pl * (SC_KP + 4) + kq * 8 + 4);
      const float dv[4] = {d.x, d.y, d.z, d.w};
      const float uv[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(dv[i], uv[j], acc[i][j]);
    }
  }
  __syncthreads();
  float* red = sc_smem;                               // [LANES][COUT][32]
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float* dst = red + (lane_q * COUT + c4 * 4 + i) * SC_KP + kq * 8;
    *(float4*)dst = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    *(float4*)(dst + 4) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
  }
  __syncthreads();
  float* out = p.part + (size_t)blockIdx.x * COUT * K;
  for (int o = threadIdx.x; o < COUT * K; o += blockDim.x) {
    const int co = o / K, k = o - co * K;
    float sum = 0.f;
#pragma unroll
    for (int l = 0; l < LANES; ++l) sum += red[(l * COUT + co) * SC_KP + k];
    out[o] = sum;
  }
}

unsigned grid_for(long long elems) {
  long long b = (elems + 255) / 256;
  long long cap = 148LL * 32;
  return (unsigned)(b < 1 ? 1 : (b > cap ? cap : b));
}

}  // namespace

void launch_nchw_to_nhwc(const LayoutProb& p, bool is_bf16, cudaStream_t s) {
  unsigned g = grid_for((long long)p.N * p.C * p.H * p.W);
  if (is_bf16) nchw_to_nhwc_kernel<bf16><<<g, 256, 0, s>>>(p);
  else nchw_to_nhwc_kernel<float><<<g, 256, 0, s>>>(p);
}
void launch_im2col(const Im2colProb* d, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8) {
  dim3 grid(grid_for(vec8 ? max_elems / 8 : max_elems), n);
  if (vec8) im2col_vec_kernel<<<grid, 256, 0, s>>>(d);
  else if (is_bf16) im2col_kernel<bf16><<<grid, 256, 0, s>>>(d);
  else im2col_kernel<float><<<grid, 256, 0, s>>>(d);
}
void launch_col2im(const Im2colProb* d, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8) {
  dim3 grid(grid_for(vec8 ? max_elems / 8 : max_elems), n);
  if (vec8) col2im_vec_kernel<<<grid, 256, 0, s>>>(d);
  else if (is_bf16) col2im_kernel<bf16><<<grid, 256, 0, s>>>(d);
  else col2im_kernel<float><<<grid, 256, 0, s>>>(d);
}
void launch_bn_stat_partial(const BnStatProb* d, int n, int max_blocks, int max_c, bool bwd, bool is_bf16, cudaStream_t s,
                            bool vec8) {
  dim3 grid((max_c + 255) / 256, max_blocks, n);
  if (vec8) {
    grid.x = 1;
    if (bwd) bn_stat_vec_kernel<true><<<grid, 256, 0, s>>>(d); else bn_stat_vec_kernel<false><<<grid, 256, 0, s>>>(d);
  } else if (is_bf16) { if (bwd) bn_stat_kernel<bf16, true><<<grid, 256, 0, s>>>(d); else bn_stat_kernel<bf16, false><<<grid, 256, 0, s>>>(d); }
  else { if (bwd) bn_stat_kernel<float, true><<<grid, 256, 0, s>>>(d); else bn_stat_kernel<float, false><<<grid, 256, 0, s>>>(d); }
}
void launch_bn_finalize(const BnFinalProb* d, int n, int max_c, bool bwd, cudaStream_t s) {
  dim3 grid((max_c + 7) / 8, n);
  if (bwd) bn_finalize_kernel<true><<<grid, 256, 0, s>>>(d);
  else bn_finalize_kernel<false><<<grid, 256, 0, s>>>(d);
}
void launch_bn_apply(const BnApplyProb* d, int n, long long max_elems, bool bwd, bool is_bf16, cudaStream_t s, bool vec8) {
  dim3 grid(grid_for(vec8 ? max_elems / 8 : max_elems), n);
  if (vec8) {
    if (bwd) bn_apply_vec_kernel<true><<<grid, 256, 0, s>>>(d); else bn_apply_vec_kernel<false><<<grid, 256, 0, s>>>(d);
  } else if (is_bf16) { if (bwd) bn_apply_kernel<bf16, true><<<grid, 256, 0, s>>>(d); else bn_apply_kernel<bf16, false><<<grid, 256, 0, s>>>(d); }
  else { if (bwd) bn_apply_kernel<float, true><<<grid, 256, 0, s>>>(d); else bn_apply_kernel<float, false><<<grid, 256, 0, s>>>(d); }
}
int bn_fused_max_blocks(int num_sms, bool bwd) {
  int per_sm = 0;
  const cudaError_t e = bwd ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bn_fused_kernel<true>, 256, 0)
                            : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bn_fused_kernel<false>, 256, 0);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return num_sms * per_sm;
}
cudaError_t launch_bn_fused(const BnFusedProb* d, int n, bool bwd, bool stats, int blocks, unsigned long long* counter,
                            int* d_status, cudaStream_t s) {
  int st = stats ? 1 : 0;
  void* params[] = {(void*)&d, (void*)&n, (void*)&st, (void*)&counter, (void*)&d_status};
  const void* fn = bwd ? (const void*)bn_fused_kernel<true> : (const void*)bn_fused_kernel<false>;
  return cudaLaunchCooperativeKernel(fn, dim3(blocks), dim3(256), params, 0, s);
}
void launch_gap_fwd(const GapProb* d, int n, int max_n, int max_c, bool is_bf16, cudaStream_t s) {
  dim3 grid((max_c + 255) / 256, max_n, n);
  if (is_bf16) gap_fwd_vec_kernel<<<dim3(1, max_n, n), 256, 0, s>>>(d);
  else gap_fwd_kernel<float><<<grid, 256, 0, s>>>(d);
}
void launch_small_conv_fwd(const SmallConvProb& p, bool w_is_bf16, bool is_bf16, cudaStream_t s) {
  const long long total = (long long)p.N * p.H * p.W;
  if (total >= (1LL << 31) - 64) return;               // the builder does not choose these kernels for such an input
  long long groups = (total + SCF_PIX - 1) / SCF_PIX;
  const unsigned grid = (unsigned)std::min<long long>(groups, 148LL * 8);
  const size_t smem = ((size_t)9 * p.Cin * p.Cout + (size_t)SCF_PIX * (SC_KP + 4)) * sizeof(float);
#define LP_FWD(CO)                                                                                    \
  do {                                                                                                \
    if (is_bf16) {                                                                                    \
      if (w_is_bf16) small_conv_fwd_kernel<bf16, bf16, CO><<<grid, 256, smem, s>>>(p);                \
      else small_conv_fwd_kernel<bf16, float, CO><<<grid, 256, smem, s>>>(p);                         \
    } else {                                                                                          \
      small_conv_fwd_kernel<float, float, CO><<<grid, 256, smem, s>>>(p);                             \
    }                                                                                                 \
  } while (0)
  switch (p.Cout) {
    case 8: LP_FWD(8); break;
    case 16: LP_FWD(16); break;
    case 32: LP_FWD(32); break;
    case 64: LP_FWD(64); break;
    default: break;                                      // the builder chooses these kernels for these widths only
  }
#undef LP_FWD
}
void launch_small_conv_wgrad(const SmallConvProb& p, bool is_bf16, cudaStream_t s) {
  const long long total = (long long)p.N * p.H * p.W;
  if (total >= (1LL << 31) - 64) return;
  const unsigned grid = (unsigned)((total + SMALLCONV_PIXELS - 1) / SMALLCONV_PIXELS);
  const int lanes = 256 / ((p.Cout / 4) * (SC_KP / 8));
  const size_t stage = (size_t)32 * (SC_KP + 4) + (size_t)32 * p.Cout, red = (size_t)lanes * p.Cout * SC_KP;
  const size_t smem = std::max(stage, red) * sizeof(float);
#define LP_WGRAD(CO)                                                                      \
  do {                                                                                    \
    if (is_bf16) small_conv_wgrad_kernel<bf16, CO><<<grid, 256, smem, s>>>(p);            \
    else small_conv_wgrad_kernel<float, CO><<<grid, 256, smem, s>>>(p);                   \
  } while (0)
  switch (p.Cout) {
    case 8: LP_WGRAD(8); break;
    case 16: LP_WGRAD(16); break;
    case 32: LP_WGRAD(32); break;
    case 64: LP_WGRAD(64); break;
    default: break;                                      // the builder chooses these kernels for these widths only
  }
#undef LP_WGRAD
}
void launch_gap_bwd(const GapProb* d, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8) {
  if (vec8 && is_bf16) {
    gap_bwd_vec_kernel<<<dim3(grid_for(max_elems / 8), n), 256, 0, s>>>(d);
    return;
  }
  dim3 grid(grid_for(max_elems), n);
  if (is_bf16) gap_bwd_kernel<bf16><<<grid, 256, 0, s>>>(d);
  else gap_bwd_kernel<float><<<grid, 256, 0, s>>>(d);
}

}  // namespace lp
