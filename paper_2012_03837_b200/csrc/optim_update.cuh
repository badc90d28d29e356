// The optimizer's update of four consecutive arena elements (Sec. 1 / Sec. 6: every chunk's parameters are
// updated from that chunk's own gradients only; the update is element-wise).  Shared by the stand-alone
// optimizer sweep and the single-launch MLP step.
#pragma once
#include "common.cuh"

namespace lp {

// Reads master, moments, gradient; writes master, moments and (for the leading n_matrix elements) the bf16
// working copy re-rounded from master.  i4 is a multiple of 4 below a.n_total.
template <bool PER_CHUNK>
__device__ __forceinline__ void optim_update4(OptimArgs a, long long i4) {
  if (PER_CHUNK) {
    // segment holding element i4 (segments start on multiples of 4, so the four elements share it)
    int lo = 0, hi = a.n_seg - 1;
    while (lo < hi) {
      int mid = (lo + hi) >> 1;
      if (i4 < a.seg_end[mid]) hi = mid; else lo = mid + 1;
    }
    const float4 tab = a.chunk_tab[a.seg_chunk[lo]];
    if (tab.x == 0.f) return;    // idle chunk: parameters, moments and working copy stay as they are
    a.bc1 = tab.y; a.bc2 = tab.z;
  }
  float4 w = *(const float4*)(a.master + i4);
  float4 g = *(const float4*)(a.grad + i4);
  float4 m1 = *(const float4*)(a.m1 + i4);
  float wv[4] = {w.x, w.y, w.z, w.w}, gv[4] = {g.x, g.y, g.z, g.w}, mv[4] = {m1.x, m1.y, m1.z, m1.w};
  bool is_mat = i4 < a.n_matrix;   // the matrix region length is a multiple of 4
  if (a.kind == 0) {               // SGD with momentum
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float gg = gv[j];
      if (is_mat && a.weight_decay != 0.f) gg += a.weight_decay * wv[j];
      mv[j] = a.momentum * mv[j] + gg;
      wv[j] -= a.lr * mv[j];
    }
  } else {                         // Adam
    float4 m2 = *(const float4*)(a.m2 + i4);
    float vv[4] = {m2.x, m2.y, m2.z, m2.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      mv[j] = a.beta1 * mv[j] + a.omb1 * gv[j];
      vv[j] = a.beta2 * vv[j] + a.omb2 * gv[j] * gv[j];
      float mh = mv[j] / a.bc1, vh = vv[j] / a.bc2;
      wv[j] -= a.lr * mh / (sqrtf(vh) + a.eps);
    }
    *(float4*)(a.m2 + i4) = make_float4(vv[0], vv[1], vv[2], vv[3]);
  }
  *(float4*)(a.m1 + i4) = make_float4(mv[0], mv[1], mv[2], mv[3]);
  *(float4*)(a.master + i4) = make_float4(wv[0], wv[1], wv[2], wv[3]);
  if (a.working && is_mat) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(wv[0], wv[1]);
    __nv_bfloat162 hi = __floats2bfloat162_rn(wv[2], wv[3]);
    uint2 pk;
    pk.x = *(uint32_t*)&lo;
    pk.y = *(uint32_t*)&hi;
    *(uint2*)(a.working + i4) = pk;
  }
}

}  // namespace lp
