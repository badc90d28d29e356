// A whole local-update step of a small fp32 MLP in ONE launch (Sec. 3: forward of every chunk, auxiliary heads and
// losses, backward inside each chunk, per-chunk optimizer update).  A network of a few 256-wide layers is a few tens
// of MFLOP per step; as a dozen dependent launches it is bound by launch and drain latency, not by arithmetic.  Here
// the step is a list of phases; all thread blocks of a cooperative launch walk the list together, sharing the work
// units of a phase round-robin and meeting at a grid-wide barrier between phases.  A phase holds the tasks that do
// not depend on one another: the layers of one depth of every chunk (pipelined schedule) or of one chunk
// (synchronous), all head products, all softmax cross-entropy rows, all weight / input gradients of one depth, the
// optimizer sweep.
//
// Arithmetic: fp32 throughout, every sum in a fixed order (a tile's reduction index is split over groups of the
// block's sixteen warps in contiguous pieces, the pieces are added in group order), so a step is bit-reproducible.
#include <algorithm>

#include "common.cuh"
#include "grid_barrier.cuh"
#include "optim_update.cuh"

namespace lp {
namespace {

constexpr int NT = FUSED_THREADS, NW = NT / 32;
constexpr int SMEM_FLOATS = 10240;         // dynamic shared memory: the staged operands of a tile, later its partial tiles
// One TM x TN tile of C = epilogue(A B^T).  The sixteen warps form KS groups; group g takes the g-th of KS
// contiguous pieces of each staged slice of the reduction index, and the NW / KS warps of a group share the rows
// of the tile among them, each lane owning an RM x RN patch.  The KS partial tiles are added in group order.
// AK / BK: the operand's reduction index is the contiguous one in memory.  Such an operand is staged as
// [rows][KC + 4] and read four reduction steps at a time (one 128-bit access per row); the other kind is staged
// as [KC][rows + 4] and read along its rows.  Either way a lane needs about one shared-memory access per four
// multiply-adds instead of one per multiply-add.
template <int TM, int TN, int RM, int RN, int KC, int KS, bool AK, bool BK>
__device__ void gemm_tile_impl(const FusedGemm& p, const float* __restrict__ A, const float* __restrict__ B, int m0,
                               int n0, float* sm) {
  constexpr int WG = NW / KS;                // warps that share a piece of the reduction index
  static_assert((TM / WG / RM) * (TN / RN) == 32, "one patch per lane");
  static_assert(RN == 8 && (RM == 1 || RM == 2) && KC % 4 == 0, "patch shapes the loads below are written for");
  constexpr int LDA = AK ? KC + 4 : TM + 4, LDB = BK ? KC + 4 : TN + 4;
  constexpr int A_FLOATS = AK ? TM * LDA : KC * LDA, B_FLOATS = BK ? TN * LDB : KC * LDB;
  static_assert(A_FLOATS + B_FLOATS <= SMEM_FLOATS && KS * TM * TN <= SMEM_FLOATS, "shared memory");
  float* As = sm;
  float* Bs = sm + A_FLOATS;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ks = warp / WG;
  const int lr = (warp % WG) * (TM / WG) + (lane / (TN / RN)) * RM, lc = (lane % (TN / RN)) * RN;
  float acc[RM][RN];
#pragma unroll
  for (int i = 0; i < RM; ++i)
#pragma unroll
    for (int j = 0; j < RN; ++j) acc[i][j] = 0.0f;

  for (int k0 = 0; k0 < p.K; k0 += KC) {
    const int kc = min(KC, p.K - k0), kc4 = (kc + 3) & ~3;   // staged up to a multiple of four, zero-filled
    __syncthreads();                         // the previous slice (or the previous tile's partials) has been read
    // every load of the slice is issued before the first store to shared memory
    constexpr int PER_A = TM * KC / NT, PER_B = TN * KC / NT;
    float va[PER_A], vb[PER_B];
#pragma unroll
    for (int r = 0; r < PER_A; ++r) {
      const int idx = tid + r * NT;
      const int mm = AK ? idx / KC : idx % TM, kk = AK ? idx % KC : idx / TM, m = m0 + mm;
      va[r] = (m < p.M && kk < kc) ? __ldcg(A + (size_t)m * p.a_ms + (size_t)(k0 + kk) * p.a_ks) : 0.0f;
    }
#pragma unroll
    for (int r = 0; r < PER_B; ++r) {
      const int idx = tid + r * NT;
      const int nn = BK ? idx / KC : idx % TN, kk = BK ? idx % KC : idx / TN, n = n0 + nn;
      vb[r] = (n < p.N && kk < kc) ? __ldcg(B + (size_t)n * p.b_ns + (size_t)(k0 + kk) * p.b_ks) : 0.0f;
    }
#pragma unroll
    for (int r = 0; r < PER_A; ++r) {
      const int idx = tid + r * NT;
      const int mm = AK ? idx / KC : idx % TM, kk = AK ? idx % KC : idx / TM;
      if (kk < kc4) As[AK ? mm * LDA + kk : kk * LDA + mm] = va[r];
    }
#pragma unroll
    for (int r = 0; r < PER_B; ++r) {
      const int idx = tid + r * NT;
      const int nn = BK ? idx / KC : idx % TN, kk = BK ? idx % KC : idx / TN;
      if (kk < kc4) Bs[BK ? nn * LDB + kk : kk * LDB + nn] = vb[r];
    }
    __syncthreads();
    const int per = (((kc4 >> 2) + KS - 1) / KS) << 2;         // reduction steps per group, a multiple of four
    const int kb = ks * per, ke = min(kb + per, kc4);
    for (int kk = kb; kk < ke; kk += 4) {
      float a[RM][4], b[RN][4];
      if (AK) {
#pragma unroll
        for (int i = 0; i < RM; ++i) {
          const float4 v = *(const float4*)&As[(lr + i) * LDA + kk];
          a[i][0] = v.x; a[i][1] = v.y; a[i][2] = v.z; a[i][3] = v.w;
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (RM == 2) {
            const float2 v = *(const float2*)&As[(kk + q) * LDA + lr];
            a[0][q] = v.x; a[RM - 1][q] = v.y;
          } else {
            a[0][q] = As[(kk + q) * LDA + lr];
          }
        }
      }
      if (BK) {
#pragma unroll
        for (int j = 0; j < RN; ++j) {
          const float4 v = *(const float4*)&Bs[(lc + j) * LDB + kk];
          b[j][0] = v.x; b[j][1] = v.y; b[j][2] = v.z; b[j][3] = v.w;
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 v0 = *(const float4*)&Bs[(kk + q) * LDB + lc], v1 = *(const float4*)&Bs[(kk + q) * LDB + lc + 4];
          b[0][q] = v0.x; b[1][q] = v0.y; b[2][q] = v0.z; b[3][q] = v0.w;
          b[4][q] = v1.x; b[5][q] = v1.y; b[6][q] = v1.z; b[7][q] = v1.w;
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)            // reduction index in increasing order
#pragma unroll
        for (int i = 0; i < RM; ++i)
#pragma unroll
          for (int j = 0; j < RN; ++j) acc[i][j] = fmaf(a[i][q], b[j][q], acc[i][j]);
    }
  }
  __syncthreads();
  float* red = sm;                           // [KS][TM * TN]
#pragma unroll
  for (int i = 0; i < RM; ++i) {
    float* dst = red + ks * (TM * TN) + (lr + i) * TN + lc;
    *(float4*)dst = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    *(float4*)(dst + 4) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
  }
  __syncthreads();
  for (int o = tid; o < TM * TN; o += NT) {
    const int m = m0 + o / TN, n = n0 + o % TN;
    const bool in = m < p.M && n < p.N;
    const size_t off = (size_t)m * p.ldc + n;
    const float bias = (in && p.bias) ? p.bias[n] : 0.0f;
    const float aux = (in && p.act == EPI_RELU_MASK) ? __ldcg(p.aux + off) : 1.0f;
    float s = red[o];
#pragma unroll
    for (int w = 1; w < KS; ++w) s += red[w * (TM * TN) + o];
    if (in) {
      s += bias;
      if (p.act == EPI_RELU) s = relu_f(s);
      else if (p.act == EPI_RELU_MASK) s = aux > 0.0f ? s : 0.0f;
      p.C[off] = s;
    }
  }
}

template <int TM, int TN, int RM, int RN, int KS>
__device__ void gemm_tile(const FusedGemm& p, const float* A, const float* B, int m0, int n0, float* sm) {
  // 256 reduction steps per slice unless both operands are staged along their rows (that layout is larger)
  const bool ak = p.a_ks == 1, bk = p.b_ks == 1;
  constexpr int KC = TM == 16 ? 256 : 128;
  if (ak && bk) gemm_tile_impl<TM, TN, RM, RN, KC, KS, true, true>(p, A, B, m0, n0, sm);
  else if (ak) gemm_tile_impl<TM, TN, RM, RN, KC, KS, true, false>(p, A, B, m0, n0, sm);
  else if (bk) gemm_tile_impl<TM, TN, RM, RN, KC, KS, false, true>(p, A, B, m0, n0, sm);
  else gemm_tile_impl<TM, TN, RM, RN, 128, KS, false, false>(p, A, B, m0, n0, sm);
}

// Softmax cross-entropy of one row by one warp (App. A.1): loss of the row, dz = (softmax - onehot) / n_valid
// over z.  A row whose label is outside [0, classes) gives no loss and a zero gradient.
__device__ void xent_row(const FusedXent& p, const int* y_ptr, int row) {
  const int lane = threadIdx.x & 31;
  float* z = p.z + (size_t)row * p.ld;
  const int y = y_ptr[row];
  if (y < 0 || y >= p.classes) {
    for (int c = lane; c < p.classes; c += 32) z[c] = 0.0f;
    if (lane == 0) p.row_loss[row] = 0.0f;
    return;
  }
  float m = -INFINITY, s = 0.0f;
  for (int c = lane; c < p.classes; c += 32) {
    const float v = z[c];
    if (v > m) { s = s * __expf(m - v) + 1.0f; m = v; }
    else s += __expf(v - m);
  }
  const float M = warp_max(m);
  const float S = warp_sum(m == -INFINITY ? 0.0f : s * __expf(m - M));
  const float lse = M + logf(S);
  const float inv = 1.0f / (float)(*p.n_valid);
  const float zy = z[y];
  __syncwarp();
  if (lane == 0) p.row_loss[row] = lse - zy;
  for (int c = lane; c < p.classes; c += 32) z[c] = (__expf(z[c] - lse) - (c == y ? 1.0f : 0.0f)) * inv;
}

__global__ void __launch_bounds__(NT, 1) fused_mlp_step_kernel(FusedArgs a) {
  extern __shared__ __align__(16) float sm[];
  __shared__ float red[33];
  __shared__ FusedPhase s_phases[FUSED_MAX_PHASES];
  __shared__ FusedTask s_tasks[FUSED_MAX_TASKS];
  __shared__ FusedGemm s_gemms[FUSED_MAX_GEMMS];
  const int tid = threadIdx.x;
  // the step's tables, held in shared memory when they fit: three dependent global reads less per work unit
  const bool cached = a.n_phases <= FUSED_MAX_PHASES && a.n_tasks <= FUSED_MAX_TASKS && a.n_gemms <= FUSED_MAX_GEMMS;
  if (cached) {
    for (int i = tid; i < a.n_phases * (int)(sizeof(FusedPhase) / 4); i += NT) ((int*)s_phases)[i] = ((const int*)a.phases)[i];
    for (int i = tid; i < a.n_tasks * (int)(sizeof(FusedTask) / 4); i += NT) ((int*)s_tasks)[i] = ((const int*)a.tasks)[i];
    for (int i = tid; i < a.n_gemms * (int)(sizeof(FusedGemm) / 4); i += NT) ((int*)s_gemms)[i] = ((const int*)a.gemms)[i];
    __syncthreads();
  }
  const FusedPhase* phases = cached ? s_phases : a.phases;
  const FusedTask* tasks = cached ? s_tasks : a.tasks;
  const FusedGemm* gemms = cached ? s_gemms : a.gemms;
  auto in_x = [&](const void* q) { return (const float*)(q == a.x_slot ? a.x : q); };
  auto in_y = [&](const int* q) { return q == a.y_slot ? a.y : q; };
  bool alive = true;
  for (int ph = 0; ph < a.n_phases && alive; ++ph) {
    const FusedPhase phase = phases[ph];
    for (int u = blockIdx.x; u < phase.units; u += gridDim.x) {
      int ti = phase.task_begin;
      while (ti + 1 < phase.task_end && tasks[ti + 1].unit_start <= u) ++ti;
      const FusedTask t = tasks[ti];
      const int local = u - t.unit_start;
      switch (t.type) {
        case FT_GEMM16: {
          const FusedGemm p = gemms[t.index];
          gemm_tile<16, 16, 1, 8, 16>(p, in_x(p.A), in_x(p.B), (local / p.tiles_n) * 16, (local % p.tiles_n) * 16, sm);
          break;
        }
        case FT_GEMM32: {
          const FusedGemm p = gemms[t.index];
          gemm_tile<32, 32, 2, 8, 8>(p, in_x(p.A), in_x(p.B), (local / p.tiles_n) * 32, (local % p.tiles_n) * 32, sm);
          break;
        }
        case FT_XENT: {
          const FusedXent p = a.xents[t.index];
          const int row = local * (NT / 32) + (tid >> 5);
          if (row < p.rows) xent_row(p, in_y(p.y), row);
          break;
        }
        case FT_COLSUM: {                    // out[c] = sum over the rows, in row order
          const FusedColSum p = a.colsums[t.index];
          const int c = local * NT + tid;
          if (c < p.cols) {
            float s = 0.0f;
            for (int r = 0; r < p.rows; ++r) s += __ldcg(p.x + (size_t)r * p.ld + c);
            p.out[c] = s;
          }
          break;
        }
        case FT_LOSS: {                      // mean loss of a chunk over its valid rows; NaN for an idle chunk
          const LossProb p = a.losses[t.index];
          float s = 0.0f;
          for (int r = tid; r < p.rows; r += NT) s += __ldcg(p.row_loss + r);
          const float tot = block_sum(s, red);
          if (tid == 0) {
            float l = tot / (float)(*p.n_valid);
            if (!isfinite(l)) atomicOr(a.status, ST_NONFINITE);
            if (a.opt.chunk_tab && a.opt.chunk_tab[p.out_index].x == 0.0f) l = __int_as_float(0x7fc00000);
            a.d_losses[p.out_index] = l;
          }
          break;
        }
        case FT_LABELS: {                    // count the valid labels, flag the others, carry the labels on
          const LabelProb p = a.labels[t.index];
          const int* y = in_y(p.y);
          int cnt = 0, bad = 0;
          for (int r = tid; r < p.rows; r += NT) {
            const int v = y[r];
            if (v >= 0 && v < p.classes) ++cnt;
            else if (v != -1) bad = 1;
            if (p.y_out) p.y_out[r] = v;
          }
          const float tot = block_sum((float)cnt, red);     // exact: counts are far below 2^24
          if (bad) atomicOr(a.status, ST_LABEL_RANGE);
          if (tid == 0) *p.n_valid = (int)tot;
          break;
        }
        case FT_OPTIM: {
          const long long i4 = ((long long)local * NT + tid) * 4;
          if (i4 < a.opt.n_total) {
            if (a.opt.seg_end) optim_update4<true>(a.opt, i4);
            else optim_update4<false>(a.opt, i4);
          }
          break;
        }
        default: {                           // FT_PREFETCH: one 128-byte line per thread towards L2
          const FusedPrefetch p = a.prefetches[t.index];
          const long long off = ((long long)local * NT + tid) * 128;
          if (off < p.bytes) asm volatile("prefetch.global.L2 [%0];" ::"l"((const char*)p.p + off));
          break;
        }
      }
    }
    if (ph + 1 < a.n_phases) alive = grid_barrier(a.counter, (unsigned long long)(ph + 1) * gridDim.x, a.status);
  }
  grid_barrier_leave(a.counter);
}

}  // namespace

int fused_mlp_max_blocks(int num_sms) {
  int per_sm = 0;
  if (cudaFuncSetAttribute(fused_mlp_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           SMEM_FLOATS * (int)sizeof(float)) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_mlp_step_kernel, NT, SMEM_FLOATS * sizeof(float)) !=
          cudaSuccess ||
      per_sm < 1) {
    cudaGetLastError();
    return 0;
  }
  return num_sms;                            // one block per SM: the blocks are co-resident by construction
}

cudaError_t launch_fused_mlp_step(const FusedArgs& args, int blocks, cudaStream_t s) {
  FusedArgs a = args;
  void* params[] = {&a};
  return cudaLaunchCooperativeKernel((const void*)fused_mlp_step_kernel, dim3(blocks), dim3(NT), params,
                                     SMEM_FLOATS * sizeof(float), s);
}

}  // namespace lp
