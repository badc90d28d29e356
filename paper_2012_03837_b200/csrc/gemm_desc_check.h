// Host-side argument check shared by the kernel-level GEMM entries (lp_gemm_bf16, lp_gemm_bf16_static):
// everything that would otherwise reach a kernel as a null or out-of-bounds access is refused here.
#pragma once
#include "../../include/lp.h"

namespace lp {

// Null if the descriptor is usable, otherwise what is wrong with it.
inline const char* gemm_desc_problem(const lp_gemm_desc& q) {
  if (!q.A || !q.B || !q.C) return "null operand or output pointer";
  if (q.M < 1 || q.N < 1 || q.K < 1) return "M, N and K must be positive";
  if (q.a_ms < 1 || q.a_ks < 1 || q.b_ns < 1 || q.b_ks < 1) return "strides must be positive";
  if ((q.a_ms != 1 && q.a_ks != 1) || (q.b_ns != 1 && q.b_ks != 1)) return "one stride per operand must be 1";
  if (q.ldc < q.N) return "ldc is smaller than N";
  if (q.act < 0 || q.act > 4) return "act must be 0..4";
  if (q.out_f32 != 0 && q.out_f32 != 1) return "out_f32 must be 0 or 1";
  if (q.act == 2 && !q.C2) return "act 2 (GELU) needs C2 for the pre-activation";
  if ((q.act == 3 || q.act == 4) && !q.aux) return "act 3 and 4 need aux";
  if (q.act == 2 && q.out_f32) return "act 2 (GELU) writes operand-type outputs only";
  return nullptr;
}

}  // namespace lp
