// Grouped GEMM on the FP32 ALUs: any sizes, any operand strides, fp32 accumulation in k order.
// Serves the fp32 workload (its 1e-4 tolerance rules out reduced-precision tensor-core paths) and
// the problems whose sizes the tensor-core kernel does not take (tiny or unaligned, e.g. a
// 10-class head).  64x64 output tile per CTA, 16-deep k slices staged in shared memory, 4x4
// accumulators per thread.
#include "common.cuh"

namespace lp {

namespace {
constexpr int TM = 64, TN = 64, TK = 16, NT = 256;

template <typename T>
__global__ void __launch_bounds__(NT) gemm_simt_kernel(const GemmProb* __restrict__ probs, int nprob) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  int tile = blockIdx.x;
  int pi = 0;
  while (pi + 1 < nprob && probs[pi + 1].tile_start <= tile) ++pi;
  const GemmProb p = probs[pi];
  int t = tile - p.tile_start;
  int m0 = (t / p.tiles_n) * TM, n0 = (t % p.tiles_n) * TN;
  const T* A = (const T*)p.A;
  const T* B = (const T*)p.B;
  int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

  for (int k0 = 0; k0 < p.K; k0 += TK) {
#pragma unroll
    for (int r = 0; r < (TM * TK) / NT; ++r) {
      int idx = threadIdx.x + r * NT;
      int mm, kk;
      if (p.a_ks == 1) { mm = idx / TK; kk = idx % TK; } else { kk = idx / TM; mm = idx % TM; }
      int m = m0 + mm, k = k0 + kk;
      As[kk][mm] = (m < p.M && k < p.K) ? to_f(A[(size_t)m * p.a_ms + (size_t)k * p.a_ks]) : 0.0f;
      int nn;
      if (p.b_ks == 1) { nn = idx / TK; kk = idx % TK; } else { kk = idx / TN; nn = idx % TN; }
      int n = n0 + nn;
      k = k0 + kk;
      Bs[kk][nn] = (n < p.N && k < p.K) ? to_f(B[(size_t)n * p.b_ns + (size_t)k * p.b_ks]) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= p.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n < p.N) gemm_epilogue_store<T>(p, m, n, acc[i][j]);
    }
  }
}
}  // namespace

// h_probs must already carry tile_start / tiles_n for 64x64 tiles (see simt_tile_counts).
void launch_gemm_simt(const GemmProb* d_probs, const GemmProb* h_probs, int n, bool is_bf16, cudaStream_t s) {
  int total = 0;
  for (int i = 0; i < n; ++i) total += ((h_probs[i].M + TM - 1) / TM) * h_probs[i].tiles_n;
  if (total == 0) return;
  if (is_bf16) gemm_simt_kernel<bf16><<<total, NT, 0, s>>>(d_probs, n);
  else gemm_simt_kernel<float><<<total, NT, 0, s>>>(d_probs, n);
}

}  // namespace lp
