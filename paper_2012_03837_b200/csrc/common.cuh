// Small device helpers shared by the kernels: type conversion, activation functions, reductions.
#pragma once
#include "lp_kernels.h"

namespace lp {

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// ReLU that keeps a NaN (fmaxf would turn it into 0 and hide a non-finite input from the loss check).
__device__ __forceinline__ float relu_f(float v) { return v < 0.0f ? 0.0f : v; }

// Exact GELU x*Phi(x) and its derivative Phi(x) + x*phi(x).
__device__ __forceinline__ float gelu_f(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_grad_f(float x) {
  float cdf = 0.5f * (1.0f + erff(x * 0.70710678118654752f));
  float pdf = 0.39894228040143268f * __expf(-0.5f * x * x);
  return cdf + x * pdf;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum for blockDim.x <= 1024 (multiple of 32); every thread receives the total.
// `red` is shared memory of at least 33 floats.  Deterministic: fixed shuffle tree, fixed warp order.
__device__ __forceinline__ float block_sum(float v, float* red) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  if (w == 0) {
    float t = lane < nw ? red[lane] : 0.0f;
    t = warp_sum(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}
__device__ __forceinline__ float block_max(float v, float* red) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  if (w == 0) {
    float t = lane < nw ? red[lane] : -INFINITY;
    t = warp_max(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}

// One output element of a GEMM epilogue (see GemmProb).
template <typename T>
__device__ __forceinline__ void gemm_epilogue_store(const GemmProb& p, int m, int n, float v) {
  size_t off = (size_t)m * p.ldc + n;
  if (p.bias) v += p.bias[n];
  if (p.resid) v += to_f(((const T*)p.resid)[off]);
  switch (p.act) {
    case EPI_RELU: v = relu_f(v); break;
    case EPI_GELU: ((T*)p.C2)[off] = from_f<T>(v); v = gelu_f(to_f(from_f<T>(v))); break;
    case EPI_RELU_MASK: v = to_f(((const T*)p.aux)[off]) > 0.0f ? v : 0.0f; break;
    case EPI_GELU_GRAD: v *= gelu_grad_f(to_f(((const T*)p.aux)[off])); break;
    default: break;
  }
  if (p.out_f32) ((float*)p.C)[off] = v;
  else ((T*)p.C)[off] = from_f<T>(v);
}

}  // namespace lp
