// HBM-bound grouped kernels: LayerNorm forward/backward, column reductions, label preparation,
// softmax cross-entropy with in-place dlogits (App. A.1: the auxiliary classifier's loss), loss
// reduction, element-wise add.  blockIdx.y (or .z) selects the problem (= chunk).
// All reductions use fixed trees and fixed orders: results are bit-reproducible run to run.
#include "common.cuh"

namespace lp {
namespace {

// ------------------------------------------------------------------ LayerNorm forward
// One warp per row; mean and biased variance in two passes over the (cache-resident) row.
template <typename T>
__global__ void __launch_bounds__(256) ln_fwd_kernel(const LnProb* __restrict__ probs) {
  const LnProb p = probs[blockIdx.y];
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int row = blockIdx.x * 8 + w;
  if (row >= p.rows) return;
  const T* x = (const T*)p.x + (size_t)row * p.d;
  T* y = (T*)p.y + (size_t)row * p.d;
  float s = 0.f;
  for (int c = lane; c < p.d; c += 32) s += to_f(x[c]);
  float mu = warp_sum(s) / p.d;
  float v = 0.f;
  for (int c = lane; c < p.d; c += 32) { float t = to_f(x[c]) - mu; v += t * t; }
  float rstd = rsqrtf(warp_sum(v) / p.d + 1e-5f);
  for (int c = lane; c < p.d; c += 32) y[c] = from_f<T>((to_f(x[c]) - mu) * rstd * p.g[c] + p.b[c]);
  if (lane == 0) { p.mean[row] = mu; p.rstd[row] = rstd; }
}

// ------------------------------------------------------------------ LayerNorm backward
// Phase A: warp per row, dx = rstd*(dxhat - mean(dxhat) - xhat*mean(dxhat*xhat)) (+ dres).
// Phase B: thread per column over this block's rows: partial sums of dy*xhat and dy.
template <typename T>
__global__ void __launch_bounds__(256) ln_bwd_kernel(const LnBwdProb* __restrict__ probs) {
  const LnBwdProb p = probs[blockIdx.y];
  int r0 = blockIdx.x * LN_BWD_ROWS;
  if (r0 >= p.rows) return;
  int r1 = min(r0 + LN_BWD_ROWS, p.rows);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (p.dx) {
    for (int row = r0 + w; row < r1; row += 8) {
      const T* dy = (const T*)p.dy + (size_t)row * p.d;
      const T* x = (const T*)p.x + (size_t)row * p.d;
      float mu = p.mean[row], rs = p.rstd[row];
      float s1 = 0.f, s2 = 0.f;
      for (int c = lane; c < p.d; c += 32) {
        float dxh = to_f(dy[c]) * p.g[c];
        s1 += dxh;
        s2 += dxh * (to_f(x[c]) - mu) * rs;
      }
      s1 = warp_sum(s1) / p.d;
      s2 = warp_sum(s2) / p.d;
      T* dx = (T*)p.dx + (size_t)row * p.d;
      const T* dres = p.dres ? (const T*)p.dres + (size_t)row * p.d : nullptr;
      for (int c = lane; c < p.d; c += 32) {
        float xh = (to_f(x[c]) - mu) * rs;
        float v = rs * (to_f(dy[c]) * p.g[c] - s1 - xh * s2);
        if (dres) v += to_f(dres[c]);
        dx[c] = from_f<T>(v);
      }
    }
  }
  float* part = p.part + (size_t)blockIdx.x * 2 * p.d;
  for (int c = threadIdx.x; c < p.d; c += blockDim.x) {
    float a = 0.f, b = 0.f;
    for (int row = r0; row < r1; ++row) {
      float dyv = to_f(((const T*)p.dy)[(size_t)row * p.d + c]);
      float xh = (to_f(((const T*)p.x)[(size_t)row * p.d + c]) - p.mean[row]) * p.rstd[row];
      a += dyv * xh;
      b += dyv;
    }
    part[c] = a;
    part[p.d + c] = b;
  }
}

// ------------------------------------------------------------------ column reductions
// Block = 32 column lanes x 8 row lanes.  A row lane sums every 8th row with four independent
// loads in flight; the 8 row lanes are then added in lane order through shared memory, so the sum
// of a column always has the same order.  A column lane covers 4 (fp32) or 8 (bf16) adjacent
// columns with one 128-bit load when the matrix allows it, one column otherwise.
__global__ void __launch_bounds__(256) col_reduce_kernel(const ColReduceProb* __restrict__ probs, const int2* __restrict__ blocks) {
  __shared__ float4 red[8][32];
  const int2 blk = blocks[blockIdx.x];
  const ColReduceProb p = probs[blk.x];
  const int bx = blk.y;
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const bool vec = (p.cols % 4 == 0) && (p.ld % 4 == 0) && (((uintptr_t)p.in & 15) == 0);
  if (vec) {
    const int c = (bx * 32 + cx) * 4;
    float4 s = make_float4(0, 0, 0, 0);
    if (c < p.cols) {
      const float* base = p.in + c;
      int r = ry;
      for (; r + 24 < p.rows; r += 32) {
        float4 a0 = *(const float4*)(base + (size_t)r * p.ld), a1 = *(const float4*)(base + (size_t)(r + 8) * p.ld);
        float4 a2 = *(const float4*)(base + (size_t)(r + 16) * p.ld), a3 = *(const float4*)(base + (size_t)(r + 24) * p.ld);
        s.x += a0.x; s.y += a0.y; s.z += a0.z; s.w += a0.w;
        s.x += a1.x; s.y += a1.y; s.z += a1.z; s.w += a1.w;
        s.x += a2.x; s.y += a2.y; s.z += a2.z; s.w += a2.w;
        s.x += a3.x; s.y += a3.y; s.z += a3.z; s.w += a3.w;
      }
      for (; r < p.rows; r += 8) {
        float4 a0 = *(const float4*)(base + (size_t)r * p.ld);
        s.x += a0.x; s.y += a0.y; s.z += a0.z; s.w += a0.w;
      }
    }
    red[ry][cx] = s;
    __syncthreads();
    if (ry == 0 && c < p.cols) {
#pragma unroll
      for (int k = 1; k < 8; ++k) { float4 a = red[k][cx]; s.x += a.x; s.y += a.y; s.z += a.z; s.w += a.w; }
      if (((uintptr_t)p.out & 15) == 0) *(float4*)(p.out + c) = s;
      else { p.out[c] = s.x; p.out[c + 1] = s.y; p.out[c + 2] = s.z; p.out[c + 3] = s.w; }
    }
  } else {
    // one column per thread, 128 columns per block
    if (threadIdx.x >= 128) return;
    const int c = bx * 128 + threadIdx.x;
    if (c >= p.cols) return;
    float s = 0.f;
    for (int r = 0; r < p.rows; ++r) s += p.in[(size_t)r * p.ld + c];
    p.out[c] = s;
  }
}

template <typename T>
__global__ void __launch_bounds__(256) colsum_partial_kernel(const ColSumProb* __restrict__ probs) {
  const ColSumProb p = probs[blockIdx.z];
  int r0 = blockIdx.y * COLSUM_ROWS;
  if (r0 >= p.rows) return;
  int r1 = min(r0 + COLSUM_ROWS, p.rows);
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= p.cols) return;
  const T* x = (const T*)p.x;
  float s = 0.f;
  for (int r = r0; r < r1; ++r) s += to_f(x[(size_t)r * p.ld + c]);
  p.part[(size_t)blockIdx.y * p.cols + c] = s;
}

// bf16, cols % 8 == 0, ld % 8 == 0, 16-byte aligned x: 256 columns x COLSUM_ROWS rows per block
__global__ void __launch_bounds__(256) colsum_partial_vec_kernel(const ColSumProb* __restrict__ probs) {
  __shared__ float red[8][32][9];
  const ColSumProb p = probs[blockIdx.z];
  const int r0 = blockIdx.y * COLSUM_ROWS;
  if (r0 >= p.rows || (int)blockIdx.x * 256 >= p.cols) return;
  const int r1 = min(r0 + COLSUM_ROWS, p.rows);
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int c = (blockIdx.x * 32 + cx) * 8;
  float s[8];
#pragma unroll
  for (int t = 0; t < 8; ++t) s[t] = 0.f;
  auto acc = [&](uint4 u) {
    const __nv_bfloat162* h = (const __nv_bfloat162*)&u;
#pragma unroll
    for (int t = 0; t < 4; ++t) { float2 f = __bfloat1622float2(h[t]); s[2 * t] += f.x; s[2 * t + 1] += f.y; }
  };
  if (c < p.cols) {
    const bf16* base = (const bf16*)p.x + c;
    int r = r0 + ry;
    for (; r + 24 < r1; r += 32) {
      uint4 a0 = *(const uint4*)(base + (size_t)r * p.ld), a1 = *(const uint4*)(base + (size_t)(r + 8) * p.ld);
      uint4 a2 = *(const uint4*)(base + (size_t)(r + 16) * p.ld), a3 = *(const uint4*)(base + (size_t)(r + 24) * p.ld);
      acc(a0); acc(a1); acc(a2); acc(a3);
    }
    for (; r < r1; r += 8) acc(*(const uint4*)(base + (size_t)r * p.ld));
  }
#pragma unroll
  for (int t = 0; t < 8; ++t) red[ry][cx][t] = s[t];
  __syncthreads();
  // thread -> one column of the block's 256: add the 8 row lanes in order
  const int col = threadIdx.x, gc = blockIdx.x * 256 + col;
  if (gc < p.cols) {
    float v = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) v += red[k][col >> 3][col & 7];
    p.part[(size_t)blockIdx.y * p.cols + gc] = v;
  }
}

// ------------------------------------------------------------------ labels
__global__ void __launch_bounds__(256) label_prep_kernel(const LabelProb* __restrict__ probs, int* status) {
  __shared__ float red[33];
  const LabelProb p = probs[blockIdx.x];
  int cnt = 0, bad = 0;
  for (int r = threadIdx.x; r < p.rows; r += blockDim.x) {
    int y = p.y[r];
    if (y >= 0 && y < p.classes) ++cnt;
    else if (y != -1) bad = 1;
    if (p.y_out) p.y_out[r] = y;
  }
  float tot = block_sum((float)cnt, red);   // exact: counts are far below 2^24
  if (bad) atomicOr(status, ST_LABEL_RANGE);
  if (threadIdx.x == 0) *p.n_valid = (int)tot;
}

// ------------------------------------------------------------------ softmax cross-entropy
// One block per row.  Pass 1: online (max, sum of exponentials) per thread, merged over the block.
// Pass 2: dz = (exp(z - lse) - [j == y]) / n_valid written over z.  Rows whose label is outside
// [0, classes) contribute no loss and a zero gradient.
template <typename T>
__global__ void __launch_bounds__(256) xent_kernel(const XentProb* __restrict__ probs) {
  __shared__ float red[33];
  const XentProb p = probs[blockIdx.y];
  int row = blockIdx.x;
  if (row >= p.rows) return;
  T* z = (T*)p.z + (size_t)row * p.ld;
  int y = p.y[row];
  bool valid = (y >= 0 && y < p.classes);
  if (!valid) {
    for (int c = threadIdx.x; c < p.classes; c += blockDim.x) z[c] = from_f<T>(0.f);
    if (threadIdx.x == 0) p.row_loss[row] = 0.f;
    return;
  }
  float m = -INFINITY, s = 0.f;
  for (int c = threadIdx.x; c < p.classes; c += blockDim.x) {
    float v = to_f(z[c]);
    if (v > m) { s = s * __expf(m - v) + 1.f; m = v; }
    else s += __expf(v - m);
  }
  float M = block_max(m, red);
  float S = block_sum(m == -INFINITY ? 0.f : s * __expf(m - M), red);
  float lse = M + logf(S);
  float inv = 1.0f / (float)(*p.n_valid);
  if (threadIdx.x == 0) p.row_loss[row] = lse - to_f(z[y]);
  __syncthreads();
  for (int c = threadIdx.x; c < p.classes; c += blockDim.x) {
    float pr = __expf(to_f(z[c]) - lse);
    z[c] = from_f<T>((pr - (c == y ? 1.f : 0.f)) * inv);
  }
}

__global__ void __launch_bounds__(256) loss_reduce_kernel(const LossProb* __restrict__ probs, float* losses,
                                                          int* status) {
  __shared__ float red[33];
  const LossProb p = probs[blockIdx.x];
  float s = 0.f;
  for (int r = threadIdx.x; r < p.rows; r += blockDim.x) s += p.row_loss[r];
  float tot = block_sum(s, red);
  if (threadIdx.x == 0) {
    float l = tot / (float)(*p.n_valid);
    losses[p.out_index] = l;
    if (!isfinite(l)) atomicOr(status, ST_NONFINITE);
  }
}

// One block per row.  A candidate (value, index) beats another if its value is larger, or equal with a
// smaller index; threads scan their columns in increasing order, so "strictly larger" keeps the first.
template <typename T>
__global__ void __launch_bounds__(256) argmax_kernel(const ArgmaxProb* __restrict__ probs, int* pred, int pred_stride,
                                                     int* correct) {
  __shared__ float sv[8];
  __shared__ int si[8];
  const ArgmaxProb p = probs[blockIdx.y];
  const int r = blockIdx.x;
  if (r >= p.rows) return;
  const T* z = (const T*)p.z + (size_t)r * p.ld;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int c = threadIdx.x; c < p.classes; c += blockDim.x) {
    float v = to_f(z[c]);
    if (v > best) { best = v; bi = c; }
  }
  auto merge = [](float& v, int& i, float ov, int oi) {
    if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
  };
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) merge(best, bi, __shfl_xor_sync(0xffffffffu, best, o), __shfl_xor_sync(0xffffffffu, bi, o));
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) merge(best, bi, sv[w], si[w]);
    if (bi == 0x7fffffff) bi = 0;              // no finite value in the row
    if (pred) pred[(size_t)p.chunk * pred_stride + r] = bi;
    if (correct) {
      const int lab = p.y[r];
      if (lab >= 0 && lab == bi) atomicAdd(&correct[p.chunk], 1);   // integer sum: order does not matter
    }
  }
}

__global__ void __launch_bounds__(256) average_f32_kernel(const AvgProb* __restrict__ probs) {
  const AvgProb p = probs[blockIdx.y];
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < p.n; i += (long long)gridDim.x * blockDim.x)
    p.a[i] = (p.a[i] + p.b[i]) * 0.5f;
}

// bf16, element count a multiple of 8, 16-byte aligned tensors: eight elements per access
__global__ void __launch_bounds__(256) add_vec_kernel(const AddProb* __restrict__ probs) {
  const AddProb p = probs[blockIdx.y];
  const long long nv = p.n >> 3;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nv; i += (long long)gridDim.x * blockDim.x) {
    const uint4 ua = ((const uint4*)p.a)[i], ub = ((const uint4*)p.b)[i];
    const __nv_bfloat162* xa = (const __nv_bfloat162*)&ua;
    const __nv_bfloat162* xb = (const __nv_bfloat162*)&ub;
    uint4 uo;
    __nv_bfloat162* xo = (__nv_bfloat162*)&uo;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 fa = __bfloat1622float2(xa[t]), fb = __bfloat1622float2(xb[t]);
      xo[t] = __floats2bfloat162_rn(fa.x + fb.x, fa.y + fb.y);
    }
    ((uint4*)p.out)[i] = uo;
  }
}

template <typename T>
__global__ void __launch_bounds__(256) add_kernel(const AddProb* __restrict__ probs) {
  const AddProb p = probs[blockIdx.y];
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < p.n; i += (long long)gridDim.x * blockDim.x)
    ((T*)p.out)[i] = from_f<T>(to_f(((const T*)p.a)[i]) + to_f(((const T*)p.b)[i]));
}

}  // namespace

#define DISPATCH_T(is_bf16, KERNEL, grid, block, s, ...)                   \
  do {                                                                      \
    if (is_bf16) KERNEL<bf16><<<grid, block, 0, s>>>(__VA_ARGS__);          \
    else KERNEL<float><<<grid, block, 0, s>>>(__VA_ARGS__);                 \
  } while (0)

void launch_ln_fwd(const LnProb* d, int n, int max_rows, bool is_bf16, cudaStream_t s) {
  dim3 grid((max_rows + 7) / 8, n);
  DISPATCH_T(is_bf16, ln_fwd_kernel, grid, 256, s, d);
}
void launch_ln_bwd(const LnBwdProb* d, int n, int max_rows, bool is_bf16, cudaStream_t s) {
  dim3 grid((max_rows + LN_BWD_ROWS - 1) / LN_BWD_ROWS, n);
  DISPATCH_T(is_bf16, ln_bwd_kernel, grid, 256, s, d);
}
void launch_col_reduce_f32(const ColReduceProb* d, const int2* blocks, int n_blocks, cudaStream_t s) {
  if (n_blocks > 0) col_reduce_kernel<<<n_blocks, 256, 0, s>>>(d, blocks);
}
void launch_colsum_partial(const ColSumProb* d, int n, int max_rows, int max_cols, bool is_bf16, cudaStream_t s, bool vec8) {
  dim3 grid((max_cols + 255) / 256, (max_rows + COLSUM_ROWS - 1) / COLSUM_ROWS, n);
  if (is_bf16 && vec8) colsum_partial_vec_kernel<<<grid, 256, 0, s>>>(d);
  else DISPATCH_T(is_bf16, colsum_partial_kernel, grid, 256, s, d);
}
void launch_label_prep(const LabelProb* d, int n, int* d_status, cudaStream_t s) {
  label_prep_kernel<<<n, 256, 0, s>>>(d, d_status);
}
void launch_xent(const XentProb* d, int n, int max_rows, bool is_bf16, cudaStream_t s) {
  dim3 grid(max_rows, n);
  DISPATCH_T(is_bf16, xent_kernel, grid, 256, s, d);
}
void launch_loss_reduce(const LossProb* d, int n, float* d_losses, int* d_status, cudaStream_t s) {
  loss_reduce_kernel<<<n, 256, 0, s>>>(d, d_losses, d_status);
}
void launch_argmax(const ArgmaxProb* d, int n, int max_rows, bool is_bf16, int* pred, int pred_stride, int* correct,
                   cudaStream_t s) {
  if (n < 1 || max_rows < 1) return;
  dim3 grid(max_rows, n);
  DISPATCH_T(is_bf16, argmax_kernel, grid, 256, s, d, pred, pred_stride, correct);
}
void launch_average_f32(const AvgProb* d, int n, long long max_elems, cudaStream_t s) {
  if (n < 1 || max_elems < 1) return;
  long long blocks = (max_elems + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  average_f32_kernel<<<dim3((unsigned)blocks, n), 256, 0, s>>>(d);
}
void launch_add(const AddProb* d, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8) {
  if (vec8 && is_bf16) {
    long long blocks = (max_elems / 8 + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    add_vec_kernel<<<dim3((unsigned)blocks, n), 256, 0, s>>>(d);
    return;
  }
  long long blocks = (max_elems + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  dim3 grid((unsigned)blocks, n);
  DISPATCH_T(is_bf16, add_kernel, grid, 256, s, d);
}

}  // namespace lp
