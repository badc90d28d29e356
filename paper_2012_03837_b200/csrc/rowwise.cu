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
__global__ void __launch_bounds__(256) col_reduce_kernel(const ColReduceProb* __restrict__ probs) {
  const ColReduceProb p = probs[blockIdx.y];
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= p.cols) return;
  float s = 0.f;
  for (int r = 0; r < p.rows; ++r) s += p.in[(size_t)r * p.ld + c];
  p.out[c] = s;
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
void launch_col_reduce_f32(const ColReduceProb* d, int n, int max_cols, cudaStream_t s) {
  dim3 grid((max_cols + 255) / 256, n);
  col_reduce_kernel<<<grid, 256, 0, s>>>(d);
}
void launch_colsum_partial(const ColSumProb* d, int n, int max_rows, int max_cols, bool is_bf16, cudaStream_t s) {
  dim3 grid((max_cols + 255) / 256, (max_rows + COLSUM_ROWS - 1) / COLSUM_ROWS, n);
  DISPATCH_T(is_bf16, colsum_partial_kernel, grid, 256, s, d);
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
void launch_add(const AddProb* d, int n, long long max_elems, bool is_bf16, cudaStream_t s) {
  long long blocks = (max_elems + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  dim3 grid((unsigned)blocks, n);
  DISPATCH_T(is_bf16, add_kernel, grid, 256, s, d);
}

}  // namespace lp
