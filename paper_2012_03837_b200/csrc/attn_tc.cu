// Causal multi-head attention for bf16 activations (App. B.2's transformer layers), heads of 64, on the
// 5th-generation tensor cores (tcgen05) with the score tiles in tensor memory.
//
// Kernels, all flash-style (no T x T matrix ever reaches global memory) and free of atomics:
//   forward : a 128-row query tile per work item, 64-key tiles.  S = Q K^T is formed in tensor memory by an elected
//             thread (tcgen05.mma, operands staged by TMA); 128 row threads -- thread r owns query row r, which is
//             lane r of tensor memory, so a row's maximum and sum need no shuffles -- copy S into registers with
//             tcgen05.ld and release the S columns at once, so the next tile's S is formed while they work; they
//             keep the running sum of the online softmax and write the probabilities back to tensor memory as bf16
//             (tcgen05.st), where the second product O += P V reads them as its A operand.  O accumulates in tensor
//             memory relative to a reference maximum that is raised (and O rescaled) only when a tile exceeds it by
//             a factor of 2^8.  Saves the row's log-sum-exp (base 2) for the backward kernels.
//   delta   : delta = rowsum(dO * O), a streaming pre-pass of the backward.
//   dQ      : S = Q K^T and dP = dO V^T in tensor memory; the row threads recompute P = exp2(S - lse), form
//             dS = P (dP - delta) and write it back as bf16; dQ += dS K accumulates in tensor memory over all key
//             tiles.
//   dK, dV  : one key per row thread, 64-query tiles, on the transposed tiles: S^T = K Q^T, dP^T = V dO^T; the row
//             threads write P^T and dS^T as swizzled bf16 rows of two shared-memory tiles, the A operands of
//             dV += P^T dO and dK += dS^T Q, which accumulate in tensor memory over all query tiles that see
//             these keys.
// The three tensor-core kernels are persistent (two blocks per SM, 256 of the 512 tensor-memory columns each, so
// one block's softmax runs while the other's products do): a block walks a list of (problem, sequence, head, row
// tile) items, heaviest first, with the TMA producer running ahead across items.  A tcgen05.mma costs its issuing
// thread about a hundred clocks whatever its size, so a tile's products are issued by up to three threads; all
// ordering between them goes through mbarriers.
//
// qkv is [B, T, 3*H*64]: columns [0, d) queries, [d, 2d) keys, [2d, 3d) values, head h at h*64.  Tiles are
// fetched through 3-D tensor maps (column, position, sequence) in boxes of 64 positions; positions past the
// end of a sequence read as zero.  Every wait on an mbarrier is bounded (see tc::mbar_wait): on expiry the
// TIMEOUT bit of the status word is raised, all roles leave their loops, tensor memory is freed and the kernel
// returns.
#include <algorithm>
#include <cstring>

#include "common.cuh"
#include "tc_prims.cuh"

namespace lp {
namespace {
using namespace tc;

constexpr int DH = 64;
constexpr float SCALE = 0.125f;                     // 1/sqrt(64)
constexpr float LOG2E = 1.4426950408889634f;
constexpr float SL2 = SCALE * LOG2E;                // scores are used in base-2 units: s2 = s * SL2
constexpr int NTHREADS = 256;                       // warps 0-3: row threads; warp 4: TMA producer; warps 5-7: MMA issuers
constexpr int ROW_WARPS = 4;
constexpr uint32_t TMEM_COLS = 256;
constexpr int BOX_BYTES = 64 * 128;                 // one TMA box: 64 positions x 64 bf16
constexpr size_t MIN_SMEM = 78 * 1024;              // no third block fits on an SM beside two of these

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) { return (uint8_t*)(((uintptr_t)p + 1023) & ~(uintptr_t)1023); }
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&v;
}
// One poller per warp; the whole warp learns the outcome.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, int* abort_flag, int* status, int lane) {
  bool ok = lane == 0 ? mbar_wait_hint(bar, parity, abort_flag, status) : true;
  return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(TMEM_COLS) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t base) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(TMEM_COLS) : "memory");
}
// Copies already issued by an aborting producer still land in this block's shared memory: give them time.
__device__ __forceinline__ void drain_copies() {
  unsigned long long t0 = gtime_ns();
  while (gtime_ns() - t0 < 2000000ull) { }
}
// Row `row` of a [*, ld] bf16 matrix: 64 values scaled by `mul`, as eight 16-byte stores.
__device__ __forceinline__ void store_row64(bf16* dst, const float* v, float mul) {
#pragma unroll
  for (int q = 0; q < 8; ++q)
    *(uint4*)(dst + q * 8) = make_uint4(pack2(v[8 * q] * mul, v[8 * q + 1] * mul), pack2(v[8 * q + 2] * mul, v[8 * q + 3] * mul),
                                        pack2(v[8 * q + 4] * mul, v[8 * q + 5] * mul), pack2(v[8 * q + 6] * mul, v[8 * q + 7] * mul));
}

// ------------------------------------------------------------------------------------------ work items
// The kernels are persistent: block c takes work items c, c + gridDim.x, ...  An item is (problem z, sequence-head
// y, 128-row tile t); items are numbered so that the heaviest row tiles come first.  All roles of a block walk the
// same list, so their barrier phase counters stay in step.  The problems' sizes and pointers are copied to shared
// memory once (at most MAX_PROBS per launch).
constexpr int MAX_PROBS = 32;
struct WorkList {
  int total, per_tile, bh, ntile;
  bool descending;                       // tile index falls with the item number (query tiles: the last sees most keys)
  __device__ __forceinline__ WorkList(int nprob, int max_bh, int ntile_, bool desc)
      : total(nprob * max_bh * ntile_), per_tile(nprob * max_bh), bh(max_bh), ntile(ntile_), descending(desc) {}
  __device__ __forceinline__ void decode(int w, int& z, int& y, int& t) const {
    const int ti = w / per_tile, rem = w - ti * per_tile;
    t = descending ? ntile - 1 - ti : ti;
    z = rem / bh;
    y = rem - z * bh;
  }
};
// Fields of a problem every role needs, and whether item (y, t) exists in it.
struct Item {
  int b, h, d, T, H, r0;                 // r0: first row of the 128-row tile
  __device__ __forceinline__ bool set(const AttnProb& pr, int y, int t) {
    H = pr.H; T = pr.T; d = pr.H * DH; r0 = t * 128;
    if (y >= pr.B * pr.H || r0 >= pr.T) return false;
    b = y / pr.H; h = y - b * pr.H;
    return true;
  }
};
// One tcgen05.mma costs its issuing thread about a hundred clocks whatever its size (measured: 64 back-to-back
// instructions of M = 128, N = 64 or 128 take 100-120 clocks each from one thread, 36 each from four threads), so
// the products of a tile are spread over up to three issuing threads (warps 5-7).  Instructions of different
// threads are not ordered against each other: every dependency between them goes through an mbarrier.
// Register split (setmaxnreg): the block is launched with 256 threads x 128 registers; the row warpgroup takes
// 192 per thread, the control warpgroup keeps 64.
constexpr int ROW_REGS = 192, CTRL_REGS = 64, LAUNCH_REGS = 128;
static_assert(128 * ROW_REGS + 128 * CTRL_REGS == NTHREADS * LAUNCH_REGS, "the split must add up to what the launch allocates");
#define ATTN_SETUP_COMMON(SH)                                                                         \
  for (int i = threadIdx.x; i < nprob * (int)(sizeof(AttnProb) / 4); i += NTHREADS)                   \
    ((uint32_t*)SH->prob)[i] = ((const uint32_t*)&probs[i / (sizeof(AttnProb) / 4)].p)[i % (sizeof(AttnProb) / 4)]; \
  if (warp == 5) tmem_alloc(&SH->tmem_base);                                                          \
  tc_fence_before();                                                                                  \
  __syncthreads();                                                                                    \
  tc_fence_after();                                                                                   \
  const uint32_t tmem = *(volatile uint32_t*)&SH->tmem_base;                                          \
  int* const abortp = &SH->abort_flag;

// ------------------------------------------------------------------------------------------ forward
// Per 64-key tile n (counted over all items of the block): warp 5 forms S_n = Q K_n^T in tensor memory; the row
// threads copy their row of S_n into registers and release the S columns at once (s_free), so S_{n+1} is formed
// while they work on tile n; they write P_n (bf16) into one of two P buffers (free again once P_{n-2} V_{n-2} has
// completed: o_full) and signal p_full; warp 6 then adds P_n V_n to O.
constexpr int F_NS = 4;                                      // stages of (K tile, V tile)
struct __align__(8) FwdShared {
  uint64_t q_full[2], q_empty[2], kv_full[F_NS], kv_empty[F_NS], s_full, s_free, p_full[2], o_full[2];
  uint32_t tmem_base;
  int abort_flag;
  AttnProb prob[MAX_PROBS];
};
constexpr int FWD_TILES = 2 * 16384 + F_NS * 2 * BOX_BYTES;  // two Q buffers, stages of one K and one V box
constexpr uint32_t F_S = 0, F_P = 64, F_O = 128;             // tensor-memory columns: S (64 fp32), P (2 x 32 packed), O (64 fp32)

__global__ void __launch_bounds__(NTHREADS, 2) attn_fwd_tc_kernel(const AttnTcProb* __restrict__ probs, int nprob, int max_bh,
                                                                   int ntile, int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sQ = align1024(smem_raw);                           // buffer qb at + qb * 16384
  uint8_t* sKV = sQ + 2 * 16384;                               // stage s at + s * 2 * BOX_BYTES: K box, V box
  FwdShared* sh = (FwdShared*)(sKV + F_NS * 2 * BOX_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WorkList wl(nprob, max_bh, ntile, true);

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->q_full[s], 1); mbar_init(&sh->q_empty[s], 1); mbar_init(&sh->p_full[s], ROW_WARPS); mbar_init(&sh->o_full[s], 1);
    }
    for (int s = 0; s < F_NS; ++s) { mbar_init(&sh->kv_full[s], 1); mbar_init(&sh->kv_empty[s], 2); }
    mbar_init(&sh->s_full, 1); mbar_init(&sh->s_free, ROW_WARPS);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  ATTN_SETUP_COMMON(sh)

  if (warp >= ROW_WARPS) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CTRL_REGS));
    if (lane != 0 || warp == 7) {
      // idle lanes and the spare warp
    } else if (warp == 4) {
      // ---------------------------------------------------------------- TMA producer
      bool ok = true;
      int n = 0, it = 0;
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const CUtensorMap* map = (const CUtensorMap*)probs[z].map_qkv;
        const int nk = (min(im.T, im.r0 + 128) + 63) >> 6, qb = it & 1;
        if (!(ok = mbar_wait_hint(&sh->q_empty[qb], ((it >> 1) & 1) ^ 1, abortp, status))) break;
        mbar_expect_tx(&sh->q_full[qb], 16384);
        tma_load_3d(sQ + qb * 16384, map, im.h * DH, im.r0, im.b, &sh->q_full[qb]);
        tma_load_3d(sQ + qb * 16384 + BOX_BYTES, map, im.h * DH, im.r0 + 64, im.b, &sh->q_full[qb]);
        for (int j = 0; j < nk; ++j, ++n) {
          const int st = n % F_NS;
          if (!(ok = mbar_wait_hint(&sh->kv_empty[st], ((n / F_NS) & 1) ^ 1, abortp, status))) break;
          mbar_expect_tx(&sh->kv_full[st], 2 * BOX_BYTES);
          tma_load_3d(sKV + st * 2 * BOX_BYTES, map, im.d + im.h * DH, j * 64, im.b, &sh->kv_full[st]);
          tma_load_3d(sKV + st * 2 * BOX_BYTES + BOX_BYTES, map, 2 * im.d + im.h * DH, j * 64, im.b, &sh->kv_full[st]);
        }
        ++it;
      }
      if (!ok) drain_copies();
    } else if (warp == 5) {
      // ---------------------------------------------------------------- issuer of S = Q K^T
      const uint32_t idesc_s = make_idesc(128, 64, false, false);
      bool ok = true;
      int n = 0, it = 0;
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const int nk = (min(im.T, im.r0 + 128) + 63) >> 6, qb = it & 1;
        if (!(ok = mbar_wait_hint(&sh->q_full[qb], (it >> 1) & 1, abortp, status))) break;
        const uint64_t dq = make_desc(smem_u32(sQ + qb * 16384), false, 0);
        for (int j = 0; j < nk; ++j, ++n) {
          const int st = n % F_NS;
          if (!(ok = mbar_wait_hint(&sh->kv_full[st], (n / F_NS) & 1, abortp, status))) break;
          if (n > 0 && !(ok = mbar_wait_hint(&sh->s_free, (n - 1) & 1, abortp, status))) break;
          tc_fence_after();
          const uint64_t dk = make_desc(smem_u32(sKV + st * 2 * BOX_BYTES), false, 0);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + F_S, dq + (uint64_t)(k4 * 2), dk + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
          tc_commit(&sh->s_full);
          tc_commit(&sh->kv_empty[st]);
        }
        if (!ok) break;
        tc_commit(&sh->q_empty[qb]);
        ++it;
      }
    } else {
      // ---------------------------------------------------------------- issuer of O += P V (warp 6)
      const uint32_t idesc_pv = make_idesc(128, 64, false, true);
      bool ok = true;
      int n = 0;
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const int nk = (min(im.T, im.r0 + 128) + 63) >> 6;
        for (int j = 0; j < nk; ++j, ++n) {
          const int st = n % F_NS;
          if (!(ok = mbar_wait_hint(&sh->kv_full[st], (n / F_NS) & 1, abortp, status))) break;
          if (!(ok = mbar_wait_hint(&sh->p_full[n & 1], (n >> 1) & 1, abortp, status))) break;
          tc_fence_after();
          const uint64_t dv = make_desc(smem_u32(sKV + st * 2 * BOX_BYTES + BOX_BYTES), true, BOX_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            tc_mma_ts(tmem + F_O, tmem + F_P + (n & 1) * 32 + k4 * 8, dv + (uint64_t)(k4 * 128), idesc_pv, (j | k4) != 0);
          tc_commit(&sh->kv_empty[st]);
          tc_commit(&sh->o_full[n & 1]);
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(ROW_REGS));
    // ---------------------------------------------------------------- row threads: thread r owns query row r0 + r
    // The output row accumulates in tensor memory (O += P V) relative to a reference maximum m_used that is
    // only raised -- with O and the running sum rescaled -- when a tile's maximum exceeds it by more than 8 in
    // base-2 units, so probabilities stay below 2^8 and most tiles need no rescale.  The decision depends on
    // the data alone.
    const int row = warp * 32 + lane;
    const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
    bool ok = true;
    int n = 0;
    uint32_t v[64];
    for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
      int z, y, t;
      wl.decode(w, z, y, t);
      Item im;
      const AttnProb& pr = sh->prob[z];
      if (!im.set(pr, y, t)) continue;
      const int nk = (min(im.T, im.r0 + 128) + 63) >> 6, grow = im.r0 + row;
      float m_used = -INFINITY, l = 0.f;
      for (int j = 0; j < nk; ++j, ++n) {
        if (!(ok = warp_wait(&sh->s_full, n & 1, abortp, status, lane))) break;
        tc_fence_after();
        tc_ld32(trow + F_S, v);
        tc_ld32(trow + F_S + 32, v + 32);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->s_free);               // the next tile's S may be formed now
        if (j * 64 + 63 > im.r0) {                             // some column lies above some row's diagonal
          const int rel = grow - j * 64;                       // columns above `rel` are in the future of this row
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (i > rel) v[i] = 0xff800000u;                   // -inf
        }
        float mx = __uint_as_float(v[0]);
#pragma unroll
        for (int i = 1; i < 64; ++i) mx = fmaxf(mx, __uint_as_float(v[i]));
        const float m_tile = mx * SL2;                         // -inf if the whole tile is in this row's future
        const bool raise = m_tile > m_used + 8.f;              // always on an item's first tile (m_used = -inf, column 0 visible)
        if (__any_sync(0xffffffffu, raise)) {
          const float m_new = raise ? m_tile : m_used;
          const float fac = ex2_approx(m_used - m_new);        // 1 for the rows whose reference stays
          if (j > 0) {
            // O must hold all earlier products of this item: wait for the one of tile n-1
            if (!(ok = warp_wait(&sh->o_full[(n - 1) & 1], ((n - 1) >> 1) & 1, abortp, status, lane))) break;
            tc_fence_after();
            uint32_t tt[32];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              tc_ld32(trow + F_O + hh * 32, tt);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) tt[i] = __float_as_uint(__uint_as_float(tt[i]) * fac);
              tc_st32(trow + F_O + hh * 32, tt);
            }
          }
          l *= fac;
          m_used = m_new;
        }
        // the product of tile n-2 has read the P buffer this tile writes
        if (n >= 2 && !(ok = warp_wait(&sh->o_full[n & 1], ((n - 2) >> 1) & 1, abortp, status, lane))) break;
        float rowsum = 0.f;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(v[c * 32 + i]), SL2, -m_used));
            const float p1 = ex2_approx(fmaf(__uint_as_float(v[c * 32 + i + 1]), SL2, -m_used));
            rowsum += p0 + p1;
            pk[i >> 1] = pack2(p0, p1);
          }
          tc_st16(trow + F_P + (n & 1) * 32 + c * 16, pk);
        }
        l += rowsum;
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->p_full[n & 1]);
      }
      if (!ok) break;
      if (!(ok = warp_wait(&sh->o_full[(n - 1) & 1], ((n - 1) >> 1) & 1, abortp, status, lane))) break;
      tc_fence_after();
      tc_ld32(trow + F_O, v);
      tc_ld32(trow + F_O + 32, v + 32);
      tc_wait_ld();
      if (grow < im.T) {
        float o[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) o[i] = __uint_as_float(v[i]);
        store_row64((bf16*)pr.o + ((size_t)im.b * im.T + grow) * im.d + (size_t)im.h * DH, o, 1.f / l);
        pr.lse[((size_t)im.b * im.H + im.h) * im.T + grow] = m_used + log2f(l);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_free(tmem); }
}

// ------------------------------------------------------------------------------------------ backward: delta
// delta[b, h, t] = sum_c dO[b, t, h*64 + c] * O[b, t, h*64 + c].  Eight consecutive threads share one (position,
// head): each reads one 16-byte piece of the 128 contiguous bytes of either tensor (a warp reads 512 contiguous
// bytes per instruction), then three shuffles add the partial sums.
__global__ void __launch_bounds__(256) attn_delta_kernel(const AttnTcProb* __restrict__ probs) {
  const AttnProb pr = probs[blockIdx.y].p;
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // 16-byte piece
  const long long i = g >> 3, total = (long long)pr.B * pr.T * pr.H;      // (position, head)
  float part = 0.f;
  if (i < total) {
    const uint4 a = ((const uint4*)pr.dout)[g], c = ((const uint4*)pr.o)[g];
    const __nv_bfloat162* ha = (const __nv_bfloat162*)&a;
    const __nv_bfloat162* hc = (const __nv_bfloat162*)&c;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float2 fa = __bfloat1622float2(ha[u]), fc = __bfloat1622float2(hc[u]);
      part = fmaf(fa.x, fc.x, part);
      part = fmaf(fa.y, fc.y, part);
    }
  }
  part += __shfl_xor_sync(0xffffffffu, part, 1);
  part += __shfl_xor_sync(0xffffffffu, part, 2);
  part += __shfl_xor_sync(0xffffffffu, part, 4);
  if (i < total && (threadIdx.x & 7) == 0) {
    const int h = (int)(i % pr.H);
    const long long bt = i / pr.H;
    const int t = (int)(bt % pr.T), b = (int)(bt / pr.T);
    pr.delta[((size_t)b * pr.H + h) * pr.T + t] = part;
  }
}

// ------------------------------------------------------------------------------------------ backward: dQ
// Same pipeline: S_n = Q K_n^T (warp 5) and dP_n = dO V_n^T (warp 6) are copied into registers and released at once;
// dS_n goes to one of two buffers (free again once dS_{n-2} K_{n-2} has completed: ds_free); warp 7 adds dS_n K_n to dQ.
constexpr int Q_NK = 3, Q_NV = 2;                            // K tiles live until dQ += dS K has read them, V tiles until dP is formed
struct __align__(8) DqShared {
  uint64_t qdo_full[2], qdo_empty[2], k_full[Q_NK], k_empty[Q_NK], v_full[Q_NV], v_empty[Q_NV], sdp_full, s_free, ds_full[2], ds_free[2], dq_full;
  uint32_t tmem_base;
  int abort_flag;
  AttnProb prob[MAX_PROBS];
};
constexpr int DQ_TILES = 4 * 16384 + (Q_NK + Q_NV) * BOX_BYTES;   // two (Q, dO) buffers, K ring, V ring
constexpr uint32_t Q_S = 0, Q_DP = 64, Q_DS = 128, Q_DQ = 192;    // S (64 fp32), dP (64), dS (2 x 32 packed), dQ (64)

__global__ void __launch_bounds__(NTHREADS, 2) attn_bwd_dq_tc_kernel(const AttnTcProb* __restrict__ probs, int nprob, int max_bh,
                                                                      int ntile, int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sQ = align1024(smem_raw);                           // buffer qb: Q at + qb * 32768, dO 16384 further
  uint8_t* sK = sQ + 4 * 16384;
  uint8_t* sV = sK + Q_NK * BOX_BYTES;
  DqShared* sh = (DqShared*)(sV + Q_NV * BOX_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WorkList wl(nprob, max_bh, ntile, true);

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->qdo_full[s], 1); mbar_init(&sh->qdo_empty[s], 2); mbar_init(&sh->ds_full[s], ROW_WARPS); mbar_init(&sh->ds_free[s], 1);
    }
    for (int s = 0; s < Q_NK; ++s) { mbar_init(&sh->k_full[s], 1); mbar_init(&sh->k_empty[s], 2); }
    for (int s = 0; s < Q_NV; ++s) { mbar_init(&sh->v_full[s], 1); mbar_init(&sh->v_empty[s], 1); }
    mbar_init(&sh->sdp_full, 2); mbar_init(&sh->s_free, ROW_WARPS); mbar_init(&sh->dq_full, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  ATTN_SETUP_COMMON(sh)

  if (warp >= ROW_WARPS) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CTRL_REGS));
    if (lane != 0) {
      // idle lanes
    } else if (warp == 4) {
      bool ok = true;
      int n = 0, it = 0;
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const CUtensorMap* map = (const CUtensorMap*)probs[z].map_qkv;
        const CUtensorMap* map_do = (const CUtensorMap*)probs[z].map_do;
        const int nk = (min(im.T, im.r0 + 128) + 63) >> 6, qb = it & 1;
        if (!(ok = mbar_wait_hint(&sh->qdo_empty[qb], ((it >> 1) & 1) ^ 1, abortp, status))) break;
        uint8_t* q = sQ + qb * 32768;
        mbar_expect_tx(&sh->qdo_full[qb], 32768);
        tma_load_3d(q, map, im.h * DH, im.r0, im.b, &sh->qdo_full[qb]);
        tma_load_3d(q + BOX_BYTES, map, im.h * DH, im.r0 + 64, im.b, &sh->qdo_full[qb]);
        tma_load_3d(q + 16384, map_do, im.h * DH, im.r0, im.b, &sh->qdo_full[qb]);
        tma_load_3d(q + 16384 + BOX_BYTES, map_do, im.h * DH, im.r0 + 64, im.b, &sh->qdo_full[qb]);
        for (int j = 0; j < nk; ++j, ++n) {
          const int sk = n % Q_NK, sv = n % Q_NV;
          if (!(ok = mbar_wait_hint(&sh->k_empty[sk], ((n / Q_NK) & 1) ^ 1, abortp, status))) break;
          mbar_expect_tx(&sh->k_full[sk], BOX_BYTES);
          tma_load_3d(sK + sk * BOX_BYTES, map, im.d + im.h * DH, j * 64, im.b, &sh->k_full[sk]);
          if (!(ok = mbar_wait_hint(&sh->v_empty[sv], ((n / Q_NV) & 1) ^ 1, abortp, status))) break;
          mbar_expect_tx(&sh->v_full[sv], BOX_BYTES);
          tma_load_3d(sV + sv * BOX_BYTES, map, 2 * im.d + im.h * DH, j * 64, im.b, &sh->v_full[sv]);
        }
        ++it;
      }
      if (!ok) drain_copies();
    } else if (warp == 5 || warp == 6) {
      // ---------------------------------------------------------------- issuers of S = Q K^T (warp 5) and dP = dO V^T (warp 6)
      const bool is_s = warp == 5;
      const uint32_t idesc_s = make_idesc(128, 64, false, false);
      bool ok = true;
      int n = 0, it = 0;
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const int nk = (min(im.T, im.r0 + 128) + 63) >> 6, qb = it & 1;
        if (!(ok = mbar_wait_hint(&sh->qdo_full[qb], (it >> 1) & 1, abortp, status))) break;
        const uint64_t da = make_desc(smem_u32(sQ + qb * 32768 + (is_s ? 0 : 16384)), false, 0);
        for (int j = 0; j < nk; ++j, ++n) {
          const int st = is_s ? n % Q_NK : n % Q_NV;
          uint64_t* full = is_s ? &sh->k_full[st] : &sh->v_full[st];
          if (!(ok = mbar_wait_hint(full, (is_s ? n / Q_NK : n / Q_NV) & 1, abortp, status))) break;
          if (n > 0 && !(ok = mbar_wait_hint(&sh->s_free, (n - 1) & 1, abortp, status))) break;
          tc_fence_after();
          const uint64_t db = make_desc(smem_u32((is_s ? sK : sV) + st * BOX_BYTES), false, 0);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + (is_s ? Q_S : Q_DP), da + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
          tc_commit(&sh->sdp_full);
          tc_commit(is_s ? &sh->k_empty[st] : &sh->v_empty[st]);
        }
        if (!ok) break;
        tc_commit(&sh->qdo_empty[qb]);
        ++it;
      }
    } else {
      // ---------------------------------------------------------------- issuer of dQ += dS K (warp 7)
      const uint32_t idesc_acc = make_idesc(128, 64, false, true);
      bool ok = true;
      int n = 0;
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const int nk = (min(im.T, im.r0 + 128) + 63) >> 6;
        for (int j = 0; j < nk; ++j, ++n) {
          const int sk = n % Q_NK;
          if (!(ok = mbar_wait_hint(&sh->k_full[sk], (n / Q_NK) & 1, abortp, status))) break;
          if (!(ok = mbar_wait_hint(&sh->ds_full[n & 1], (n >> 1) & 1, abortp, status))) break;
          tc_fence_after();
          const uint64_t dk_mn = make_desc(smem_u32(sK + sk * BOX_BYTES), true, BOX_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            tc_mma_ts(tmem + Q_DQ, tmem + Q_DS + (n & 1) * 32 + k4 * 8, dk_mn + (uint64_t)(k4 * 128), idesc_acc, (j | k4) != 0);
          tc_commit(&sh->k_empty[sk]);
          tc_commit(&sh->ds_free[n & 1]);
        }
        if (!ok) break;
        tc_commit(&sh->dq_full);
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(ROW_REGS));
    const int row = warp * 32 + lane;
    const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
    bool ok = true;
    int n = 0, it = 0;
    uint32_t vs[64], vd[64];
    // this row's log-sum-exp and delta, fetched one item ahead; rows past the end get lse = +inf: every probability
    // becomes exp2(-inf) = 0
    auto fetch = [&](int w, float& lse, float& delta) {
      lse = INFINITY; delta = 0.f;
      if (w >= wl.total) return;
      int z, y, t;
      wl.decode(w, z, y, t);
      Item im;
      const AttnProb& pr = sh->prob[z];
      if (!im.set(pr, y, t) || im.r0 + row >= im.T) return;
      const size_t at = ((size_t)im.b * im.H + im.h) * im.T + im.r0 + row;
      lse = pr.lse[at];
      delta = pr.delta[at];
    };
    float lse_nx, delta_nx;
    fetch(blockIdx.x, lse_nx, delta_nx);
    for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
      const float lse = lse_nx, delta = delta_nx;
      fetch(w + gridDim.x, lse_nx, delta_nx);
      int z, y, t;
      wl.decode(w, z, y, t);
      Item im;
      const AttnProb& pr = sh->prob[z];
      if (!im.set(pr, y, t)) continue;
      const int nk = (min(im.T, im.r0 + 128) + 63) >> 6, grow = im.r0 + row;
      for (int j = 0; j < nk; ++j, ++n) {
        if (!(ok = warp_wait(&sh->sdp_full, n & 1, abortp, status, lane))) break;
        tc_fence_after();
        tc_ld32(trow + Q_S, vs);
        tc_ld32(trow + Q_S + 32, vs + 32);
        tc_ld32(trow + Q_DP, vd);
        tc_ld32(trow + Q_DP + 32, vd + 32);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->s_free);
        if (j * 64 + 63 > im.r0) {
          const int rel = grow - j * 64;
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (i > rel) vs[i] = 0xff800000u;                  // -inf: probability 0
        }
        // the product of tile n-2 has read the dS buffer this tile writes
        if (n >= 2 && !(ok = warp_wait(&sh->ds_free[n & 1], ((n - 2) >> 1) & 1, abortp, status, lane))) break;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(vs[c * 32 + i]), SL2, -lse));
            const float p1 = ex2_approx(fmaf(__uint_as_float(vs[c * 32 + i + 1]), SL2, -lse));
            pk[i >> 1] = pack2(p0 * (__uint_as_float(vd[c * 32 + i]) - delta), p1 * (__uint_as_float(vd[c * 32 + i + 1]) - delta));
          }
          tc_st16(trow + Q_DS + (n & 1) * 32 + c * 16, pk);
        }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->ds_full[n & 1]);
      }
      if (!ok) break;
      if (!(ok = warp_wait(&sh->dq_full, it & 1, abortp, status, lane))) break;
      tc_fence_after();
      tc_ld32(trow + Q_DQ, vs);
      tc_ld32(trow + Q_DQ + 32, vs + 32);
      tc_wait_ld();
      if (grow < im.T) {
        float acc[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] = __uint_as_float(vs[i]);
        store_row64((bf16*)pr.dqkv + ((size_t)im.b * im.T + grow) * 3 * im.d + (size_t)im.h * DH, acc, SCALE);
      }
      ++it;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_free(tmem); }
}

// ------------------------------------------------------------------------------------------ backward: dK, dV
// One key per row thread, 64-query tiles.  S^T_n = K Q_n^T (warp 5) and dP^T_n = V dO_n^T (warp 6) are copied into
// registers and released at once; the row threads write P^T_n and dS^T_n as bf16 rows of two shared-memory tiles
// (128 keys x 64 queries, 128-byte swizzle: the A operands of dV += P^T dO_n and dK += dS^T Q_n), which the products
// of tile n-1 must have finished reading (acc_done).  Warp 5 issues S^T_n, then dK of tile n-1; warp 6 issues
// dP^T_n, then dV of tile n-1.
constexpr int K_NQ = 2;                                      // stages of (Q tile, dO tile)
struct __align__(8) DkvShared {
  uint64_t kv_full, kv_empty, q_full[K_NQ], q_empty[K_NQ], sdp_full, s_free, ps_full, acc_done, dkv_full, ld_full[2];
  uint32_t tmem_base;
  int abort_flag;
  float lse[2][64], delta[2][64];
  AttnProb prob[MAX_PROBS];
};
constexpr int DKV_TILES = 2 * 16384 + K_NQ * 2 * BOX_BYTES + 2 * 16384;   // K, V, stages of (Q, dO) boxes, P^T, dS^T
constexpr uint32_t K_ST = 0, K_DPT = 64, K_DV = 128, K_DK = 192;         // S^T (64 fp32), dP^T (64), dV (64), dK (64)

__global__ void __launch_bounds__(NTHREADS, 2) attn_bwd_dkv_tc_kernel(const AttnTcProb* __restrict__ probs, int nprob, int max_bh,
                                                                       int ntile, int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sK = align1024(smem_raw);
  uint8_t* sV = sK + 16384;
  uint8_t* sQ = sV + 16384;                                    // stage st at + st * 2 * BOX_BYTES: Q box, dO box
  uint8_t* sP = sQ + K_NQ * 2 * BOX_BYTES;
  uint8_t* sdS = sP + 16384;
  DkvShared* sh = (DkvShared*)(sdS + 16384);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WorkList wl(nprob, max_bh, ntile, false);              // the first key tile is seen by all queries: heaviest first

  if (threadIdx.x == 0) {
    mbar_init(&sh->kv_full, 1); mbar_init(&sh->kv_empty, 2);
    for (int s = 0; s < K_NQ; ++s) { mbar_init(&sh->q_full[s], 1); mbar_init(&sh->q_empty[s], 4); }
    for (int s = 0; s < 2; ++s) mbar_init(&sh->ld_full[s], 32 * ROW_WARPS);
    mbar_init(&sh->sdp_full, 2); mbar_init(&sh->s_free, ROW_WARPS); mbar_init(&sh->ps_full, ROW_WARPS);
    mbar_init(&sh->acc_done, 2); mbar_init(&sh->dkv_full, 2);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  ATTN_SETUP_COMMON(sh)

  if (warp >= ROW_WARPS) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CTRL_REGS));
    if (lane != 0 || warp == 7) {
      // idle lanes and the spare warp
    } else if (warp == 4) {
      bool ok = true;
      int n = 0, it = 0;
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const CUtensorMap* map = (const CUtensorMap*)probs[z].map_qkv;
        const CUtensorMap* map_do = (const CUtensorMap*)probs[z].map_do;
        const int j0 = im.r0 >> 6, nq = ((im.T + 63) >> 6) - j0;
        if (!(ok = mbar_wait_hint(&sh->kv_empty, (it & 1) ^ 1, abortp, status))) break;
        mbar_expect_tx(&sh->kv_full, 32768);
        tma_load_3d(sK, map, im.d + im.h * DH, im.r0, im.b, &sh->kv_full);
        tma_load_3d(sK + BOX_BYTES, map, im.d + im.h * DH, im.r0 + 64, im.b, &sh->kv_full);
        tma_load_3d(sV, map, 2 * im.d + im.h * DH, im.r0, im.b, &sh->kv_full);
        tma_load_3d(sV + BOX_BYTES, map, 2 * im.d + im.h * DH, im.r0 + 64, im.b, &sh->kv_full);
        for (int jj = 0; jj < nq; ++jj, ++n) {
          const int st = n % K_NQ;
          if (!(ok = mbar_wait_hint(&sh->q_empty[st], ((n / K_NQ) & 1) ^ 1, abortp, status))) break;
          mbar_expect_tx(&sh->q_full[st], 2 * BOX_BYTES);
          tma_load_3d(sQ + st * 2 * BOX_BYTES, map, im.h * DH, (j0 + jj) * 64, im.b, &sh->q_full[st]);
          tma_load_3d(sQ + st * 2 * BOX_BYTES + BOX_BYTES, map_do, im.h * DH, (j0 + jj) * 64, im.b, &sh->q_full[st]);
        }
        ++it;
      }
      if (!ok) drain_copies();
    } else {
      // ---------------------------------------------------------------- issuers: warp 5 (S^T = K Q^T, dK += dS^T Q), warp 6 (dP^T = V dO^T, dV += P^T dO)
      const bool is_k = warp == 5;
      const uint32_t idesc_s = make_idesc(128, 64, false, false), idesc_acc = make_idesc(128, 64, false, true);
      const uint64_t da = make_desc(smem_u32(is_k ? sK : sV), false, 0);          // K (or V) as the A operand of the first product
      const uint64_t dacc = make_desc(smem_u32(is_k ? sdS : sP), false, 0);       // dS^T (or P^T) as the A operand of the second
      const uint32_t box = is_k ? 0 : BOX_BYTES;                                  // Q (or dO) box of a stage
      bool ok = true;
      int n = 0, it = 0;
      // dK (+)= dS^T_m Q_m or dV (+)= P^T_m dO_m for tile m, whose row threads have signalled ps_full
      auto issue_acc = [&](int m, bool first) {
        if (!(ok = mbar_wait_hint(&sh->ps_full, m & 1, abortp, status))) return;
        tc_fence_after();
        const int st = m % K_NQ;
        const uint64_t db_mn = make_desc(smem_u32(sQ + st * 2 * BOX_BYTES + box), true, BOX_BYTES);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
          tc_mma(tmem + (is_k ? K_DK : K_DV), dacc + (uint64_t)(k4 * 2), db_mn + (uint64_t)(k4 * 128), idesc_acc, !first || k4 != 0);
        tc_commit(&sh->q_empty[st]);
        tc_commit(&sh->acc_done);
      };
      for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
        int z, y, t;
        wl.decode(w, z, y, t);
        Item im;
        if (!im.set(sh->prob[z], y, t)) continue;
        const int j0 = im.r0 >> 6, nq = ((im.T + 63) >> 6) - j0;
        if (!(ok = mbar_wait_hint(&sh->kv_full, it & 1, abortp, status))) break;
        for (int jj = 0; jj < nq && ok; ++jj, ++n) {
          const int st = n % K_NQ;
          if (!(ok = mbar_wait_hint(&sh->q_full[st], (n / K_NQ) & 1, abortp, status))) break;
          if (n > 0 && !(ok = mbar_wait_hint(&sh->s_free, (n - 1) & 1, abortp, status))) break;
          tc_fence_after();
          const uint64_t db = make_desc(smem_u32(sQ + st * 2 * BOX_BYTES + box), false, 0);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) tc_mma(tmem + (is_k ? K_ST : K_DPT), da + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), idesc_s, k4 != 0);
          tc_commit(&sh->sdp_full);
          tc_commit(&sh->q_empty[st]);
          if (jj == nq - 1) tc_commit(&sh->kv_empty);            // K (or V) has been read for the last time
          if (jj > 0) issue_acc(n - 1, jj == 1);
        }
        if (!ok) break;
        issue_acc(n - 1, nq == 1);
        if (!ok) break;
        tc_commit(&sh->dkv_full);
        ++it;
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(ROW_REGS));
    const int row = warp * 32 + lane;
    const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
    // the 128 row threads fetch the query tile's log-sum-exp (threads 0-63) and delta (64-127) one tile ahead
    const int idx = threadIdx.x & 63;
    bool ok = true;
    int n = 0, it = 0;
    uint32_t vs[64], vd[64];
    for (int w = blockIdx.x; w < wl.total && ok; w += gridDim.x) {
      int z, y, t;
      wl.decode(w, z, y, t);
      Item im;
      const AttnProb& pr = sh->prob[z];
      if (!im.set(pr, y, t)) continue;
      const int k0 = im.r0, gkey = k0 + row, T = im.T;
      const int j0 = k0 >> 6, nq = ((T + 63) >> 6) - j0;
      const float* src = (threadIdx.x < 64 ? pr.lse : pr.delta) + ((size_t)im.b * im.H + im.h) * T;
      auto fetch = [&](int j) { const int q = j * 64 + idx; return q < T ? src[q] : 0.f; };
      float nxt = fetch(j0);
      for (int jj = 0; jj < nq; ++jj, ++n) {
        const int buf = n & 1, q0j = (j0 + jj) * 64;
        (threadIdx.x < 64 ? sh->lse[buf] : sh->delta[buf])[idx] = nxt;
        mbar_arrive(&sh->ld_full[buf]);
        if (jj + 1 < nq) nxt = fetch(j0 + jj + 1);
        if (!(ok = warp_wait(&sh->ld_full[buf], (n >> 1) & 1, abortp, status, lane))) break;
        if (!(ok = warp_wait(&sh->sdp_full, n & 1, abortp, status, lane))) break;
        tc_fence_after();
        tc_ld32(trow + K_ST, vs);
        tc_ld32(trow + K_ST + 32, vs + 32);
        tc_ld32(trow + K_DPT, vd);
        tc_ld32(trow + K_DPT + 32, vd + 32);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->s_free);
        if (q0j < k0 + 128 || q0j + 64 > T) {                   // the tile crosses the diagonal or the end of the sequence
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (gkey > q0j + i || q0j + i >= T) vs[i] = 0xff800000u;   // -inf: probability 0
        }
        // the products of the previous tile have read the two shared-memory tiles
        if (n > 0 && !(ok = warp_wait(&sh->acc_done, (n - 1) & 1, abortp, status, lane))) break;
        // this key's row of P^T and of dS^T: 64 bf16 = eight 16-byte pieces, piece q of row r at (q ^ (r & 7))
        uint8_t* prow = sP + row * 128;
        uint8_t* drow = sdS + row * 128;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          uint32_t pp[4], pd[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = q * 8 + 2 * u;
            const float2 ls = *(const float2*)&sh->lse[buf][i], dl = *(const float2*)&sh->delta[buf][i];
            const float p0 = ex2_approx(fmaf(__uint_as_float(vs[i]), SL2, -ls.x));
            const float p1 = ex2_approx(fmaf(__uint_as_float(vs[i + 1]), SL2, -ls.y));
            pp[u] = pack2(p0, p1);
            pd[u] = pack2(p0 * (__uint_as_float(vd[i]) - dl.x), p1 * (__uint_as_float(vd[i + 1]) - dl.y));
          }
          const int off = (q ^ (row & 7)) << 4;
          *(uint4*)(prow + off) = make_uint4(pp[0], pp[1], pp[2], pp[3]);
          *(uint4*)(drow + off) = make_uint4(pd[0], pd[1], pd[2], pd[3]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads these tiles through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->ps_full);
      }
      if (!ok) break;
      if (!(ok = warp_wait(&sh->dkv_full, it & 1, abortp, status, lane))) break;
      tc_fence_after();
      tc_ld32(trow + K_DV, vs);
      tc_ld32(trow + K_DV + 32, vs + 32);
      tc_ld32(trow + K_DK, vd);
      tc_ld32(trow + K_DK + 32, vd + 32);
      tc_wait_ld();
      if (gkey < T) {
        float acc[64];
        bf16* out = (bf16*)pr.dqkv + ((size_t)im.b * T + gkey) * 3 * im.d + (size_t)im.h * DH;
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] = __uint_as_float(vs[i]);
        store_row64(out + 2 * im.d, acc, 1.f);
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] = __uint_as_float(vd[i]);
        store_row64(out + im.d, acc, SCALE);
      }
      ++it;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) { tc_fence_after(); tmem_free(tmem); }
}

// 3-D bf16 tensor map of a [B, T, width] activation: boxes of 64 columns x 64 positions of one sequence,
// 128-byte swizzle, zero fill outside the tensor.
bool encode_seq_map(void* out, const void* base, int B, int T, long long width) {
  EncodeFn fn = get_encode();
  if (!fn || ((uintptr_t)base & 15) || (width * 2) % 16) return false;
  cuuint64_t dims[3] = {(cuuint64_t)width, (cuuint64_t)T, (cuuint64_t)B};
  cuuint64_t strides[2] = {(cuuint64_t)width * 2, (cuuint64_t)T * width * 2};
  cuuint32_t box[3] = {64u, 64u, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = fn((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int KERNEL_ID>
cudaError_t prepare(const void* kern, size_t smem) {
  // function attributes belong to a device's context: set once per device and kernel
  static bool done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (done[dev]) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // The row warpgroup's register increase must fit into what the launch allocates (threads x compiled register
  // count); otherwise it would wait forever.  Refuse to launch instead.
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, kern);
  if (e != cudaSuccess) return e;
  if (fa.numRegs < LAUNCH_REGS) return cudaErrorLaunchOutOfResources;
  done[dev] = true;
  return cudaSuccess;
}

}  // namespace

bool attn_tc_encode(AttnTcProb& out, const AttnProb& p) {
  memset(&out, 0, sizeof(out));
  out.p = p;
  const long long d = (long long)p.H * DH;
  if (p.B < 1 || p.T < 1 || p.H < 1 || !p.qkv) return false;
  if (!encode_seq_map(out.map_qkv, p.qkv, p.B, p.T, 3 * d)) return false;
  if (p.dout && !encode_seq_map(out.map_do, p.dout, p.B, p.T, d)) return false;
  return true;
}

// Persistent grid: two blocks per SM (or fewer when there is less work).
static int attn_grid(int total) {
  static int sms[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
  if (!sms[dev]) cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
  return std::max(1, std::min(total, 2 * sms[dev]));
}

cudaError_t launch_attn_fwd_tc(const AttnTcProb* d, int n, int maxB, int maxT, int maxH, int* status, cudaStream_t s) {
  const size_t smem = std::max(MIN_SMEM, (size_t)FWD_TILES + 1024 + sizeof(FwdShared));
  cudaError_t e = prepare<0>((const void*)attn_fwd_tc_kernel, smem);
  if (e != cudaSuccess) return e;
  const int ntile = (maxT + 127) / 128;
  for (int i = 0; i < n; i += MAX_PROBS) {
    const int m = std::min(MAX_PROBS, n - i);
    attn_fwd_tc_kernel<<<attn_grid(m * maxB * maxH * ntile), NTHREADS, smem, s>>>(d + i, m, maxB * maxH, ntile, status);
  }
  return cudaGetLastError();
}

cudaError_t launch_attn_bwd_tc(const AttnTcProb* d, int n, int maxB, int maxT, int maxH, int* status, cudaStream_t s) {
  const size_t smem_q = std::max(MIN_SMEM, (size_t)DQ_TILES + 1024 + sizeof(DqShared));
  const size_t smem_kv = std::max(MIN_SMEM, (size_t)DKV_TILES + 1024 + sizeof(DkvShared));
  cudaError_t e = prepare<1>((const void*)attn_bwd_dq_tc_kernel, smem_q);
  if (e == cudaSuccess) e = prepare<2>((const void*)attn_bwd_dkv_tc_kernel, smem_kv);
  if (e != cudaSuccess) return e;
  const int ntile = (maxT + 127) / 128;
  {
    const long long pieces = 8LL * maxB * maxT * maxH;         // 16-byte pieces of the largest problem
    dim3 grid((unsigned)((pieces + 255) / 256), n);
    attn_delta_kernel<<<grid, 256, 0, s>>>(d);                  // delta = rowsum(dO * O), read by both kernels below
  }
  for (int i = 0; i < n; i += MAX_PROBS) {
    const int m = std::min(MAX_PROBS, n - i), grid = attn_grid(m * maxB * maxH * ntile);
    attn_bwd_dq_tc_kernel<<<grid, NTHREADS, smem_q, s>>>(d + i, m, maxB * maxH, ntile, status);
    attn_bwd_dkv_tc_kernel<<<grid, NTHREADS, smem_kv, s>>>(d + i, m, maxB * maxH, ntile, status);
  }
  return cudaGetLastError();
}

}  // namespace lp
