// Causal multi-head attention for bf16 activations (App. B.2's transformer layers), heads of 64,
// flash-style with register-resident score tiles: warp-level tensor-core MMAs (m16n8k16, bf16 in,
// fp32 accumulate) fed by ldmatrix from bf16 Q/K/V tiles in shared memory; the scores, the
// probabilities and their gradients never leave registers (the accumulator fragment of one MMA is
// re-packed as the A fragment of the next).  Forward keeps an online softmax (running max and sum per
// row); backward recomputes the probabilities from Q, K and the saved log-sum-exp: one kernel per
// query tile for dQ, one per key tile for dK and dV.  No atomics: every sum has a fixed order.
//
// qkv is [B*T, 3*H*64]: columns [0, d) queries, [d, 2d) keys, [2d, 3d) values, head h at h*64.
#include "common.cuh"

namespace lp {
namespace {

constexpr int DH = 64, TILE = 64, PITCH = 72;     // bf16 tile rows of 144 bytes: ldmatrix rows hit distinct banks
constexpr float SCALE = 0.125f;                    // 1/sqrt(64)
constexpr float LOG2E = 1.4426950408889634f;
constexpr float SL2 = SCALE * LOG2E;               // scores are kept in base-2 units: s2 = s * SL2
constexpr float LN2 = 0.6931471805599453f;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ldsm_x4(uint32_t* r, const bf16* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(p)));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t* r, const bf16* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(p)));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&v;
}

// 64x64 bf16 tile global -> shared; rows >= rmax read as zero.  128 threads.
__device__ __forceinline__ void load_tile(bf16* dst, const bf16* src, size_t ld, int r0, int rmax) {
  for (int e = threadIdx.x; e < 64 * 8; e += 128) {
    int r = e >> 3, c = (e & 7) * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r0 + r < rmax) v = *(const uint4*)(src + (size_t)(r0 + r) * ld + c);
    *(uint4*)(dst + r * PITCH + c) = v;
  }
}

// A fragments (16 rows x 64 k) of rows [row0, row0+16) of a row-major tile: 4 k-steps x 4 registers.
// Lane l addresses row row0 + l%16, column block (l/16)*8: matrices (rows 0-7, k 0-7), (rows 8-15,
// k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 8-15) = a0..a3.
__device__ __forceinline__ void load_a_frags(uint32_t (*a)[4], const bf16* tile, int row0, int lane) {
#pragma unroll
  for (int ks = 0; ks < 4; ++ks) ldsm_x4(a[ks], tile + (row0 + (lane & 15)) * PITCH + ks * 16 + (lane >> 4) * 8);
}

// acc[j] (j = 8 n-tiles of 8 columns) += A[16 x 64] * X^T where X is a row-major [64 n][64 k] tile
// (scores: A = Q rows, X = K; dP: A = dO rows, X = V).  One ldmatrix.x4 yields the B fragments of two
// neighbouring n-tiles: (n 0-7, k 0-7), (n 0-7, k 8-15), (n 8-15, k 0-7), (n 8-15, k 8-15).
__device__ __forceinline__ void mma_a_xt(float (*acc)[4], const uint32_t (*a)[4], const bf16* x, int lane) {
#pragma unroll
  for (int ks = 0; ks < 4; ++ks)
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t b[4];
      ldsm_x4(b, x + (np * 16 + (lane & 7) + (lane >> 4) * 8) * PITCH + ks * 16 + ((lane >> 3) & 1) * 8);
      mma16816(acc[2 * np], a[ks], b[0], b[1]);
      mma16816(acc[2 * np + 1], a[ks], b[2], b[3]);
    }
}

// acc[j] (8 n-tiles over the 64 columns of X) += P[16 x 64] * X where P comes as packed A fragments
// (4 k-steps of 16 rows of X) and X is a row-major [64 k][64 n] tile (O += P V, dQ += dS K,
// dV += P^T dO, dK += dS^T Q).  Transposing ldmatrix: (k 0-7, n 0-7), (k 8-15, n 0-7), (k 0-7, n 8-15),
// (k 8-15, n 8-15).
__device__ __forceinline__ void mma_p_x(float (*acc)[4], const uint32_t (*pa)[4], const bf16* x, int lane) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk)
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t b[4];
      ldsm_x4_t(b, x + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + np * 16 + (lane >> 4) * 8);
      mma16816(acc[2 * np], pa[kk], b[0], b[1]);
      mma16816(acc[2 * np + 1], pa[kk], b[2], b[3]);
    }
}

// Accumulator fragments of a 16x64 tile -> A fragments of the same tile (bf16).
__device__ __forceinline__ void acc_to_a(uint32_t (*pa)[4], const float (*c)[4]) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    pa[kk][0] = pack2(c[2 * kk][0], c[2 * kk][1]);
    pa[kk][1] = pack2(c[2 * kk][2], c[2 * kk][3]);
    pa[kk][2] = pack2(c[2 * kk + 1][0], c[2 * kk + 1][1]);
    pa[kk][3] = pack2(c[2 * kk + 1][2], c[2 * kk + 1][3]);
  }
}

// Store a 16x64 accumulator tile (rows row_lo and row_lo + 8 of this thread) as bf16 into a row-major matrix.
__device__ __forceinline__ void store_acc(bf16* out, size_t ld, int row_lo, int rmax, const float (*c)[4], float mul_lo,
                                          float mul_hi, int lane) {
  int t = lane & 3;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    int col = j * 8 + 2 * t;
    if (row_lo < rmax) *(uint32_t*)(out + (size_t)row_lo * ld + col) = pack2(c[j][0] * mul_lo, c[j][1] * mul_lo);
    if (row_lo + 8 < rmax) *(uint32_t*)(out + (size_t)(row_lo + 8) * ld + col) = pack2(c[j][2] * mul_hi, c[j][3] * mul_hi);
  }
}

// cp.async copy of a 64x64 bf16 tile global -> shared; rows >= rmax are zero-filled (source size 0).
__device__ __forceinline__ void load_tile_async(bf16* dst, const bf16* src, size_t ld, int r0, int rmax) {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    int e = threadIdx.x + k * 128;
    int r = e >> 3, c = (e & 7) * 8;
    bool ok = r0 + r < rmax;
    const bf16* g = ok ? src + (size_t)(r0 + r) * ld + c : src;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr(dst + r * PITCH + c)), "l"(g), "r"(ok ? 16 : 0));
  }
}
__device__ __forceinline__ void cp_async_f32(float* dst, const float* src, bool ok) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_addr(dst)), "l"(src), "r"(ok ? 4 : 0));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The log-sum-exp saved by the forward kernel for the two backward kernels is in base-2 units.
// Query tiles are taken heaviest first (the last tile sees all keys).
__global__ void __launch_bounds__(128) attn_fwd_mma_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb pr = probs[blockIdx.z];
  const int qt = gridDim.x - 1 - blockIdx.x, q0 = qt * TILE;
  if ((int)blockIdx.y >= pr.B * pr.H || q0 >= pr.T) return;
  __shared__ __align__(16) bf16 sq[TILE * PITCH], sk[2][TILE * PITCH], sv[2][TILE * PITCH];
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const size_t ld = 3 * (size_t)d;
  const bf16* base = (const bf16*)pr.qkv + (size_t)b * T * ld + (size_t)h * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int row_lo = q0 + warp * 16 + g;          // this thread's two rows: row_lo and row_lo + 8

  load_tile_async(sq, base, ld, q0, T);
  load_tile_async(sk[0], base + d, ld, 0, T);
  load_tile_async(sv[0], base + 2 * d, ld, 0, T);
  cp_async_commit();
  uint32_t qa[4][4];
  float o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  for (int kt = 0; kt <= qt; ++kt) {
    const int st = kt & 1;
    if (kt < qt) {                                  // next key tile in flight while this one is used
      load_tile_async(sk[st ^ 1], base + d, ld, (kt + 1) * TILE, T);
      load_tile_async(sv[st ^ 1], base + 2 * d, ld, (kt + 1) * TILE, T);
    }
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (kt == 0) load_a_frags(qa, sq, warp * 16, lane);
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
    mma_a_xt(s, qa, sk[st], lane);
    const bool edge = (kt == qt) || ((kt + 1) * TILE > T);
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[j][e] * SL2;
        if (edge) {
          int col = kt * TILE + j * 8 + 2 * t + (e & 1);
          int row = row_lo + (e >> 1) * 8;
          if (col > row || col >= T) v = -INFINITY;
        }
        s[j][e] = v;
        if (e < 2) mx_lo = fmaxf(mx_lo, v); else mx_hi = fmaxf(mx_hi, v);
      }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    float c_lo = ex2(m_lo - mn_lo), c_hi = ex2(m_hi - mn_hi);
    m_lo = mn_lo; m_hi = mn_hi;
    float ps_lo = 0.f, ps_hi = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      s[j][0] = ex2(s[j][0] - mn_lo); s[j][1] = ex2(s[j][1] - mn_lo);
      s[j][2] = ex2(s[j][2] - mn_hi); s[j][3] = ex2(s[j][3] - mn_hi);
      ps_lo += s[j][0] + s[j][1];
      ps_hi += s[j][2] + s[j][3];
      o[j][0] *= c_lo; o[j][1] *= c_lo; o[j][2] *= c_hi; o[j][3] *= c_hi;
    }
    l_lo = l_lo * c_lo + ps_lo;
    l_hi = l_hi * c_hi + ps_hi;
    uint32_t pa[4][4];
    acc_to_a(pa, s);
    mma_p_x(o, pa, sv[st], lane);
    __syncthreads();                                // stage st is overwritten by the loads of the next iteration
  }
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  bf16* out = (bf16*)pr.o + (size_t)b * T * d + (size_t)h * DH;
  store_acc(out, (size_t)d, row_lo, T, o, 1.f / l_lo, 1.f / l_hi, lane);
  if (t == 0) {
    float* lse = pr.lse + ((size_t)b * pr.H + h) * T;
    if (row_lo < T) lse[row_lo] = m_lo + log2f(l_lo);
    if (row_lo + 8 < T) lse[row_lo + 8] = m_hi + log2f(l_hi);
  }
}

// dQ for one query tile; also writes delta[row] = sum_c dO[row,c] O[row,c].
__global__ void __launch_bounds__(128) attn_bwd_dq_mma_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb pr = probs[blockIdx.z];
  const int qt = gridDim.x - 1 - blockIdx.x, q0 = qt * TILE;
  if ((int)blockIdx.y >= pr.B * pr.H || q0 >= pr.T) return;
  // buf 0: Q, then keys of odd tiles; buf 1: dO, then values of odd tiles; buf 2: O (for delta);
  // buf 3 / 4: keys / values of even tiles
  __shared__ __align__(16) bf16 buf[5][TILE * PITCH];
  __shared__ float sdelta[TILE];
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const size_t ld = 3 * (size_t)d;
  const bf16* base = (const bf16*)pr.qkv + (size_t)b * T * ld + (size_t)h * DH;
  const bf16* gob = (const bf16*)pr.dout + (size_t)b * T * d + (size_t)h * DH;
  const bf16* ob = (const bf16*)pr.o + (size_t)b * T * d + (size_t)h * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int row_lo = q0 + warp * 16 + g;

  load_tile_async(buf[0], base, ld, q0, T);
  load_tile_async(buf[1], gob, (size_t)d, q0, T);
  load_tile_async(buf[2], ob, (size_t)d, q0, T);
  load_tile_async(buf[3], base + d, ld, 0, T);
  load_tile_async(buf[4], base + 2 * d, ld, 0, T);
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();
  {
    int r = threadIdx.x >> 1, half = threadIdx.x & 1;
    float dl = 0.f;
    for (int c = 0; c < 32; ++c)
      dl = fmaf(__bfloat162float(buf[1][r * PITCH + half * 32 + c]), __bfloat162float(buf[2][r * PITCH + half * 32 + c]), dl);
    dl += __shfl_xor_sync(0xffffffffu, dl, 1);
    if (half == 0) {
      sdelta[r] = dl;
      if (q0 + r < T) pr.delta[((size_t)b * pr.H + h) * T + q0 + r] = dl;
    }
  }
  uint32_t qa[4][4], ga[4][4];
  load_a_frags(qa, buf[0], warp * 16, lane);
  load_a_frags(ga, buf[1], warp * 16, lane);
  __syncthreads();
  const float* lsep = pr.lse + ((size_t)b * pr.H + h) * T;
  const float lse_lo = row_lo < T ? lsep[row_lo] : 0.f, lse_hi = row_lo + 8 < T ? lsep[row_lo + 8] : 0.f;
  const float dl_lo = sdelta[warp * 16 + g], dl_hi = sdelta[warp * 16 + g + 8];
  float dq[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) { dq[j][0] = dq[j][1] = dq[j][2] = dq[j][3] = 0.f; }

  for (int kt = 0; kt <= qt; ++kt) {
    const bf16* sk = (kt & 1) ? buf[0] : buf[3];
    const bf16* sv = (kt & 1) ? buf[1] : buf[4];
    if (kt < qt) {
      load_tile_async((kt & 1) ? buf[3] : buf[0], base + d, ld, (kt + 1) * TILE, T);
      load_tile_async((kt & 1) ? buf[4] : buf[1], base + 2 * d, ld, (kt + 1) * TILE, T);
    }
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    float s[8][4], dp[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; dp[j][0] = dp[j][1] = dp[j][2] = dp[j][3] = 0.f; }
    mma_a_xt(s, qa, sk, lane);
    mma_a_xt(dp, ga, sv, lane);
    const bool edge = (kt == qt) || ((kt + 1) * TILE > T);
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float p = ex2(fmaf(s[j][e], SL2, -(e < 2 ? lse_lo : lse_hi)));
        if (edge) {
          int col = kt * TILE + j * 8 + 2 * t + (e & 1);
          int row = row_lo + (e >> 1) * 8;
          if (col > row || col >= T || row >= T) p = 0.f;
        }
        s[j][e] = p * (dp[j][e] - (e < 2 ? dl_lo : dl_hi));
      }
    uint32_t dsa[4][4];
    acc_to_a(dsa, s);
    mma_p_x(dq, dsa, sk, lane);
    __syncthreads();
  }
  bf16* out = (bf16*)pr.dqkv + (size_t)b * T * ld + (size_t)h * DH;
  store_acc(out, ld, row_lo, T, dq, SCALE, SCALE, lane);
}

// dK and dV for one key tile: loops over the query tiles that can see it.  Works on the transposed
// score tile (rows = keys of this warp, columns = queries).  Key tiles are taken heaviest first
// (the first tile is seen by all queries).
__global__ void __launch_bounds__(128) attn_bwd_dkv_mma_kernel(const AttnProb* __restrict__ probs) {
  const AttnProb pr = probs[blockIdx.z];
  if ((int)blockIdx.y >= pr.B * pr.H || (int)blockIdx.x * TILE >= pr.T) return;
  // buf 0: K, then Q of odd steps; buf 1: V, then dO of odd steps; buf 2 / 3: Q / dO of even steps
  __shared__ __align__(16) bf16 buf[4][TILE * PITCH];
  __shared__ float slse[2][TILE], sdelta[2][TILE];
  const int b = blockIdx.y / pr.H, h = blockIdx.y % pr.H, d = pr.H * DH, T = pr.T;
  const size_t ld = 3 * (size_t)d;
  const bf16* base = (const bf16*)pr.qkv + (size_t)b * T * ld + (size_t)h * DH;
  const bf16* gob = (const bf16*)pr.dout + (size_t)b * T * d + (size_t)h * DH;
  const float* lsep = pr.lse + ((size_t)b * pr.H + h) * T;
  const float* delp = pr.delta + ((size_t)b * pr.H + h) * T;
  const int kt = blockIdx.x, k0 = kt * TILE;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int key_lo = k0 + warp * 16 + g;
  const int nq = (T + TILE - 1) / TILE;

  auto load_q = [&](int qt, int stage) {
    const int q0 = qt * TILE;
    load_tile_async(stage ? buf[0] : buf[2], base, ld, q0, T);
    load_tile_async(stage ? buf[1] : buf[3], gob, (size_t)d, q0, T);
    int i = threadIdx.x & 63, qi = q0 + i;
    if (threadIdx.x < 64) cp_async_f32(&slse[stage][i], qi < T ? lsep + qi : lsep, qi < T);
    else cp_async_f32(&sdelta[stage][i], qi < T ? delp + qi : delp, qi < T);
  };
  load_tile_async(buf[0], base + d, ld, k0, T);
  load_tile_async(buf[1], base + 2 * d, ld, k0, T);
  load_q(kt, 0);
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();
  uint32_t ka[4][4], va[4][4];
  load_a_frags(ka, buf[0], warp * 16, lane);
  load_a_frags(va, buf[1], warp * 16, lane);
  __syncthreads();
  float dk[8][4], dv[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) { dk[j][0] = dk[j][1] = dk[j][2] = dk[j][3] = 0.f; dv[j][0] = dv[j][1] = dv[j][2] = dv[j][3] = 0.f; }

  for (int qt = kt; qt < nq; ++qt) {
    const int q0 = qt * TILE, stage = (qt - kt) & 1;
    const bf16* sq = stage ? buf[0] : buf[2];
    const bf16* sgo = stage ? buf[1] : buf[3];
    if (qt + 1 < nq) load_q(qt + 1, stage ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    float st[8][4], dpt[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { st[j][0] = st[j][1] = st[j][2] = st[j][3] = 0.f; dpt[j][0] = dpt[j][1] = dpt[j][2] = dpt[j][3] = 0.f; }
    mma_a_xt(st, ka, sq, lane);       // S^T = K Q^T
    mma_a_xt(dpt, va, sgo, lane);     // dP^T = V dO^T
    const bool edge = (qt == kt) || ((qt + 1) * TILE > T);
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int qc = j * 8 + 2 * t + (e & 1);                  // query column inside the tile
        float pv = ex2(fmaf(st[j][e], SL2, -slse[stage][qc]));
        if (edge) {
          int qi = q0 + qc, key = key_lo + (e >> 1) * 8;
          if (key > qi || qi >= T || key >= T) pv = 0.f;
        }
        st[j][e] = pv * (dpt[j][e] - sdelta[stage][qc]);   // dS^T
        dpt[j][e] = pv;                                    // P^T
      }
    uint32_t pa[4][4], dsa[4][4];
    acc_to_a(pa, dpt);
    acc_to_a(dsa, st);
    mma_p_x(dv, pa, sgo, lane);       // dV += P^T dO
    mma_p_x(dk, dsa, sq, lane);       // dK += dS^T Q
    __syncthreads();
  }
  bf16* out = (bf16*)pr.dqkv + (size_t)b * T * ld + (size_t)h * DH;
  store_acc(out + d, ld, key_lo, T, dk, SCALE, SCALE, lane);
  store_acc(out + 2 * d, ld, key_lo, T, dv, 1.f, 1.f, lane);
}

}  // namespace

void launch_attn_fwd_tc(const AttnProb* d, int n, int maxB, int maxT, int maxH, cudaStream_t s) {
  dim3 grid((maxT + TILE - 1) / TILE, maxB * maxH, n);
  attn_fwd_mma_kernel<<<grid, 128, 0, s>>>(d);
}

void launch_attn_bwd_tc(const AttnProb* d, int n, int maxB, int maxT, int maxH, cudaStream_t s) {
  dim3 grid((maxT + TILE - 1) / TILE, maxB * maxH, n);
  attn_bwd_dq_mma_kernel<<<grid, 128, 0, s>>>(d);
  attn_bwd_dkv_mma_kernel<<<grid, 128, 0, s>>>(d);
}

}  // namespace lp
