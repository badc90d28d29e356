// Host interface of the tcgen05 grouped GEMM (gemm_tc.cu).
#pragma once
#include <vector>

#include "lp_kernels.h"

namespace lp {

// True if the problem can run on the tensor-core kernel: bf16 operands, 16-byte aligned bases,
// pitches that are multiples of 8 elements, and enough work to fill a 128x256 tile.
bool gemm_tc_eligible(const GemmProb& g);
// Fill tile_start / tiles_n for 128x256 tiles; returns the number of tiles of this problem.
// cg = 1: one CTA per 128x256 tile; cg = 2: a pair of CTAs per 256x256 tile (tcgen05 cta_group::2).
int gemm_tc_choose_cg(const GemmProb* probs, int n);
int gemm_tc_tiles(GemmProb& g, int tile_start, int cg = 1, int wide = 0);
// True if the problem may run with 256x512 tiles per CTA pair (wide = 1): a long reduction (K >= 8192) with a
// plain epilogue and N a multiple of 512; such problems go into a launch of their own with cg = 2.
bool gemm_tc_wide_ok(const GemmProb& g);
// Encode the four TMA tensor maps [A, B, C, C2] of a problem (128 bytes each, 64-byte aligned host memory);
// sets g.store_tma when the output's pitch lets the epilogue leave through TMA stores.
bool gemm_tc_encode(GemmProb& g, void* maps4, int cg = 1);
// A launch whose tiles differ much in length (grouped weight and input gradients of networks whose stages differ
// in every size) is balanced on the host: sched lists the tiles of CTA (pair) 0, then of 1, ..., each in
// increasing order, off[u] .. off[u + 1] being unit u's part (off has units + 1 entries, units =
// gemm_tc_grid_units).  probs must carry tile_start (gemm_tc_tiles).  Returns false, leaving both empty, when the
// kernel's own walk (every units-th tile) is as good.
int gemm_tc_grid_units(int total_tiles, int num_sms, int cg);
bool gemm_tc_schedule(const GemmProb* probs, int nprob, int total_tiles, int num_sms, int cg, std::vector<int>& sched,
                      std::vector<int>& off);
// d_maps: device array of 4*nprob tensor maps, [A0, B0, C0, C2_0, A1, ...].  d_sched / d_sched_off: device copies
// of a schedule made by gemm_tc_schedule for this launch, or null.
cudaError_t launch_gemm_tc(const GemmProb* d_probs, const void* d_maps, int nprob, int total_tiles, int* d_status,
                           int num_sms, cudaStream_t s, int cg = 1, int wide = 0, const int* d_sched = nullptr,
                           const int* d_sched_off = nullptr);

}  // namespace lp
