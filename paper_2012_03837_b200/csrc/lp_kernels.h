// Device-side problem tables and host launchers of the kernels behind the local update step.
// Every kernel is "grouped": one launch serves a list of independent problems (one per chunk,
// Sec. 3: chunks are trained independently), selected by blockIdx.y or by a tile scheduler.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lp {

typedef __nv_bfloat16 bf16;

// Bits of the device status word.
enum { ST_LABEL_RANGE = 1, ST_NONFINITE = 2, ST_TIMEOUT = 4 };

// ---------------------------------------------------------------------------- GEMM
// C[m,n] = epilogue( sum_k A(m,k) * B(n,k) ),  A(m,k) = A[m*a_ms + k*a_ks], B(n,k) = B[n*b_ns + k*b_ks].
// Exactly one stride of each operand is 1.  Forward of a Linear layer (App. A.1): A = x [M,K],
// B = W [N,K].  Input gradient: A = dy, B(n,k) = W[k,n].  Weight gradient: A(m,k) = dy[k,m],
// B(n,k) = x[k,n] (the reduction runs over the rows of the minibatch).
// EPI_LOGIT_STATS (tensor-core kernel only): no activation; besides C (bf16 logits), C2 receives, as
// float2 [M, ceil(N/128)], the maximum and the sum of exp(z - max) over every group of 128 columns of
// the stored (rounded) logits: the first pass of the softmax cross-entropy (App. A.1) done where the
// logits are produced.
enum EpiAct { EPI_NONE = 0, EPI_RELU = 1, EPI_GELU = 2, EPI_RELU_MASK = 3, EPI_GELU_GRAD = 4, EPI_LOGIT_STATS = 5 };

struct GemmProb {
  const void* A;
  const void* B;
  void* C;            // [M, ldc] output, element type = operand type, or float if out_f32
  void* C2;           // EPI_GELU: receives the pre-activation (operand type); else unused
  const float* bias;  // [N] added to every row, or null
  const void* resid;  // [M, ldc] operand type, added before the activation, or null
  const void* aux;    // [M, ldc] operand type: EPI_RELU_MASK: layer output y (mask y>0);
                      // EPI_GELU_GRAD: pre-activation u (multiply by gelu'(u))
  int M, N, K;
  long long a_ms, a_ks, b_ns, b_ks;
  int ldc;
  int act;
  int out_f32;
  int tile_start;  // first tile index of this problem in the launch (filled by the launcher)
  int tiles_n;
  int tile_n;      // tensor-core kernel: columns of a tile and of its MMA, 64 / 128 / 256 (set by the launcher)
  int store_tma;   // tensor-core kernel: outputs leave through TMA stores (set by the launcher when C's pitch allows)
  int raster;      // tensor-core kernel: row tiles per band of the tile walk (set by the launcher)
  // Implicit convolution over NHWC activations (tensor-core kernel only; App. B.3's residual blocks): 3x3 with
  // padding 1 (conv_taps = 9) or 1x1 without padding (conv_taps = 1), stride conv_stride = 1 or 2.  One operand
  // is never materialised as a matrix: its tiles are fetched as boxes of the activation tensor
  // [conv_n, conv_hin, conv_win, conv_c] that step through it with the stride, one shifted box per filter tap
  // (i, j), rows and columns outside the image reading as zero.  conv_h x conv_w is the OUTPUT image (the rows of
  // the GEMM are its pixels); for stride 1 it equals the input image.  The formulas below are written for the
  // 3x3, stride-1 case; with a stride s the input pixel of output pixel (p, q) and tap (i, j) is
  // (s p + i - 1, s q + j - 1), for 1x1 it is (s p, s q).  CONV_DGRAD exists for stride 1 only.
  //   CONV_FWD   : A(m, k) = x[pixel m shifted by (i-1, j-1)][c],  k = (3i + j) conv_c + c;  K = 9 conv_c;
  //                B = filters [N, 9 conv_c] (reduction index contiguous).
  //   CONV_DGRAD : A(m, k) = dy[pixel m shifted by (1-i, 1-j)][co], k = (3i + j) conv_c + co; K = 9 conv_c;
  //                B(n, k) = filters[co][(3i + j) N + n]  (the filter tensor [conv_c, 3, 3, N] read in place).
  //   CONV_WGRAD : B(n, k) = x[pixel conv_k0 + k shifted by (i-1, j-1)][ci], n = (3i + j) conv_c + ci;
  //                N = 9 conv_c; A(m, k) = dy[pixel k][m] as an ordinary MN-major operand; K = pixels.
  // A is the activation tensor for CONV_FWD / CONV_DGRAD, B for CONV_WGRAD.
  // Tensor-core kernel only.  The pre-activation that EPI_GELU writes (C2) and EPI_GELU_GRAD reads (aux) has no
  // other reader, so its layout is free: with aux_blocked it is stored as 32x32 blocks of 2 KB, block
  // (m / 32, n / 32) at ((m / 32) * (ldc / 32) + n / 32) * 1024 elements, inside a block 16-byte piece q of
  // row r at q * 256 + r * 8 elements.  A warp's epilogue owns exactly such a block (one row per lane), so
  // it writes and reads it with four fully coalesced 512-byte accesses instead of 32 scattered row pieces
  // per access.  Needs M, N and ldc multiples of 32 and a 16-byte aligned buffer.
  int aux_blocked;
  int conv;
  int conv_n, conv_h, conv_w, conv_c;
  int conv_k0;     // CONV_WGRAD: first pixel of this slice of the reduction (split-K)
  int conv_hin, conv_win, conv_stride, conv_taps;   // 0 = defaults: input image = output image, stride 1, 9 taps
};
enum { CONV_NONE = 0, CONV_FWD = 1, CONV_DGRAD = 2, CONV_WGRAD = 3 };
// True if an image of h x w pixels can be walked in whole-row boxes of 128 and of 64 pixels.
inline bool conv_boxes_ok(int h, int w) {
  const long long hw = (long long)h * w;
  return w >= 1 && 64 % w == 0 && (hw % 128 == 0 || 128 % hw == 0);
}

// FP32-ALU GEMM (any sizes and strides).  T = float or bf16 operands, fp32 accumulation.
void launch_gemm_simt(const GemmProb* d_probs, const GemmProb* h_probs, int n, bool is_bf16,
                      cudaStream_t s);

// ---------------------------------------------------------------------------- row-wise kernels
struct LnProb {       // LayerNorm over the last axis of x [rows, d]
  const void* x; void* y; const float* g; const float* b; float* mean; float* rstd;
  int rows, d;
};
void launch_ln_fwd(const LnProb* d_probs, int n, int max_rows, bool is_bf16, cudaStream_t s);

struct LnBwdProb {    // dx = LN'(dy) (+ dres); partial dgamma/dbeta per row block
  const void* dy; const void* x; const float* g; const float* mean; const float* rstd;
  void* dx;            // may be null: parameter gradients only (chunk input is a constant, Sec. 3)
  const void* dres;    // optional gradient arriving over the residual path, added to dx
  float* part;         // [nblk, 2, d] partial sums, nblk = ceil(rows / LN_BWD_ROWS)
  int rows, d;
};
enum { LN_BWD_ROWS = 64 };
void launch_ln_bwd(const LnBwdProb* d_probs, int n, int max_rows, bool is_bf16, cudaStream_t s);

struct ColReduceProb { // out[c] = sum_r in[r, c] over r < rows, for c < cols; in is fp32 [rows, ld]
  const float* in; float* out; int rows, cols, ld;
};
// d_blocks[i] = (problem, block of 128 columns inside it): one thread block each
void launch_col_reduce_f32(const ColReduceProb* d_probs, const int2* d_blocks, int n_blocks, cudaStream_t s);

struct ColSumProb {   // part[blk, c] = sum over a block of rows of x[r, c]; x is [rows, ld]
  const void* x; float* part; int rows, cols, ld;
};
enum { COLSUM_ROWS = 128 };
// vec8: bf16 with cols % 8 == 0, ld % 8 == 0 and 16-byte aligned x in every problem (128-bit loads)
void launch_colsum_partial(const ColSumProb* d_probs, int n, int max_rows, int max_cols, bool is_bf16,
                           cudaStream_t s, bool vec8 = false);

struct LabelProb {    // count valid labels, check range, (pipelined) carry labels to the next chunk
  const int* y; int* y_out; int rows; int classes; int* n_valid;
};
void launch_label_prep(const LabelProb* d_probs, int n, int* d_status, cudaStream_t s);

struct XentProb {     // softmax cross-entropy rows (App. A.1): z [rows, ld] -> dz in place, row losses
  void* z; const int* y; const int* n_valid; float* row_loss; int rows, classes, ld;
  float* colsum_part;   // optional [ceil(rows / XENT_ROWS), classes]: per-row-block column sums of dz (bias gradient)
};
enum { XENT_ROWS = 64 };
void launch_xent(const XentProb* d_probs, int n, int max_rows, bool is_bf16, cudaStream_t s);

// 128-bit vectorised bf16 variants (rowwise_vec.cu); nv = compile-time vectors per lane / thread.
void launch_ln_fwd_vec(const LnProb* d_probs, int n, int max_rows, int nv, cudaStream_t s);
void launch_ln_bwd_vec(const LnBwdProb* d_probs, int n, int max_rows, int nv, cudaStream_t s);
void launch_xent_vec(const XentProb* d_probs, int n, int max_rows, int nv, cudaStream_t s);
// Blocks of XENT_ROWS rows, dlogits in place plus per-block column sums; classes % 8 == 0, classes <= 32768.
void launch_xent_rows(const XentProb* d_probs, int n, int max_rows, int classes, cudaStream_t s);

// Cross-entropy from per-group softmax statistics (EPI_LOGIT_STATS): a merge kernel turns the groups
// of a row into its log-sum-exp and loss, then dlogits = softmax/n - onehot/n are written in place by
// column strips with no reduction left inside a row; the strips' column sums (bias gradient) go to
// colsum_part [ceil(rows / XENT_APPLY_ROWS), classes] when it is non-null.
struct XentStatsProb {
  void* z; const int* y; const int* n_valid; float* row_loss; const float2* stats; float* row_c;
  float* colsum_part; int rows, classes, ld, groups;
};
enum { XENT_APPLY_ROWS = 256 };
void launch_xent_from_stats(const XentStatsProb* d_probs, int n, int max_rows, int classes, cudaStream_t s);

// Prediction of every row: the index of its largest logit, the lowest index among equal values (an
// integer result: exact).  pred[chunk * pred_stride + r] receives it; correct[chunk] counts the rows
// whose prediction equals the label (rows with a negative label are not counted).  Either may be null.
struct ArgmaxProb { const void* z; const int* y; int rows, classes, ld, chunk; };
void launch_argmax(const ArgmaxProb* d_probs, int n, int max_rows, bool is_bf16, int* pred, int pred_stride,
                   int* correct, cudaStream_t s);

struct LossProb { const float* row_loss; const int* n_valid; int rows; int out_index; };
void launch_loss_reduce(const LossProb* d_probs, int n, float* d_losses, int* d_status, cudaStream_t s);

// ---------------------------------------------------------------------------- LM-specific
struct EmbedProb { const int* ids; const void* tok; const void* pos; void* h; int rows, T, d, vocab; };
void launch_embed_fwd(const EmbedProb& p, int* d_status, bool is_bf16, cudaStream_t s);
struct EmbedBwdProb {
  const int* ids; const void* dh; float* dtok; float* dpos; int* next; int* first; int rows, T, d, vocab, B;
};
void launch_embed_bwd(const EmbedBwdProb& p, bool is_bf16, cudaStream_t s);

struct AttnProb {     // causal attention over qkv [B*T, 3d], heads of 64
  const void* qkv; void* o; float* lse; const void* dout; void* dqkv; float* delta; int B, T, H;
};
void launch_attn_fwd(const AttnProb* d_probs, int n, int maxB, int maxT, int maxH, bool is_bf16, cudaStream_t s);
void launch_attn_bwd(const AttnProb* d_probs, int n, int maxB, int maxT, int maxH, bool is_bf16, cudaStream_t s);
// bf16 path (attn_tc.cu): tcgen05 kernels with the score tiles in tensor memory.  A problem carries the TMA tensor
// maps of its qkv tensor and (backward) of dout, [B, T, width] in boxes of 64 columns x 64 positions; the table of
// problems lives in device memory, 64-byte aligned.  attn_tc_encode fills one entry on the host (false: the tensor
// maps could not be encoded -- base addresses must be 16-byte aligned).  status: device status word (ST_TIMEOUT).
struct alignas(64) AttnTcProb { unsigned char map_qkv[128]; unsigned char map_do[128]; AttnProb p; };
bool attn_tc_encode(AttnTcProb& out, const AttnProb& p);
cudaError_t launch_attn_fwd_tc(const AttnTcProb* d_probs, int n, int maxB, int maxT, int maxH, int* status, cudaStream_t s);
cudaError_t launch_attn_bwd_tc(const AttnTcProb* d_probs, int n, int maxB, int maxT, int maxH, int* status, cudaStream_t s);

// ---------------------------------------------------------------------------- ResNet-specific
struct LayoutProb { const void* in; void* out; int N, C, H, W; };
void launch_nchw_to_nhwc(const LayoutProb& p, bool is_bf16, cudaStream_t s);

struct Im2colProb {   // x NHWC [N,H,W,C] -> cols [N*Ho*Wo, ldk], column (i*kw + j)*C + c, zero padded
  const void* x; void* cols; int N, H, W, C, kh, kw, stride, pad, Ho, Wo, ldk;
};
// vec8: bf16 with channel counts that are multiples of 8 (128-bit accesses)
void launch_im2col(const Im2colProb* d_probs, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8 = false);
// dx[n,h,w,c] = sum over the filter taps that read this pixel of dcols (gather form: no atomics)
void launch_col2im(const Im2colProb* d_probs, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8 = false);

struct BnStatProb {   // per-channel partial sums of x and x^2 (fwd) or of dy and dy*xhat (bwd)
  const void* x; const void* dy; const float* mean; const float* rstd; const void* relu_out;
  float* part; int rows, C;
};
// Rows summed by one block of the statistics kernels: 256 where that still leaves four blocks per SM of a
// 148-SM device, fewer (down to 32) for the short tensors of the late stages, whose sums would otherwise
// run as a few long serial loops on a handful of SMs.
#if defined(__CUDACC__)
__host__ __device__
#endif
inline int bn_rows_per_block(long long rows) {
  int rpb = 256;
  while (rpb > 32 && rows / rpb < 592) rpb >>= 1;
  return rpb;
}
#if defined(__CUDACC__)
__host__ __device__
#endif
inline int bn_blocks(long long rows) { int rpb = bn_rows_per_block(rows); return (int)((rows + rpb - 1) / rpb); }
// max_blocks: the largest bn_blocks(rows) among the n problems
void launch_bn_stat_partial(const BnStatProb* d_probs, int n, int max_blocks, int max_c, bool bwd, bool is_bf16,
                            cudaStream_t s, bool vec8 = false);
struct BnFinalProb {  // fwd: sums -> mean, rstd.  part is [nblk, 2, C]
  const float* part; int nblk; int rows; int C; float* mean; float* rstd; float* dgamma; float* dbeta; float eps;
  // Running statistics (fwd only, nullable): with use_running == 0 they are moved towards this minibatch's
  // mean and unbiased variance by `momentum` (training steps); with use_running == 1 nothing is summed and
  // mean / rstd are taken from them (evaluation mode).
  float* run_mean; float* run_var; float momentum; int use_running;
  // the update of the running statistics is skipped while the chunk idles (chunk_tab[chunk].x == 0; see OptimArgs)
  const float4* chunk_tab; int chunk;
};
void launch_bn_finalize(const BnFinalProb* d_probs, int n, int max_c, bool bwd, cudaStream_t s);
struct BnApplyProb {
  // fwd: y = relu?( (x-mean)*rstd*g + b (+ res) ).
  // bwd: dx = rstd*g*( dyr - sum_dy/rows - xhat*sum_dyxhat/rows ), dyr = dy masked by relu_out>0;
  //      dres_out (optional) receives dyr (gradient of the residual branch).
  const void* x; void* y; const void* res; const float* g; const float* b; const float* mean; const float* rstd;
  const void* dy; const void* relu_out; void* dx; void* dres_out; const float* dgamma; const float* dbeta;
  int rows, C, relu;
};
void launch_bn_apply(const BnApplyProb* d_probs, int n, long long max_elems, bool bwd, bool is_bf16, cudaStream_t s, bool vec8 = false);
// The three passes of a group of BatchNorms (bf16, C % 8 == 0, C / 8 <= 256 in every problem) as one cooperative
// launch with bounded grid-wide barriers in between.  Every block of the launch sums all its blocks of rows into
// ONE row of the partial sums, so fin.nblk must be min(bn_blocks(rows), blocks) -- deterministic, but not the
// summation order of the separate launches.  stats = false: the statistics pass is left out (evaluation mode: the
// finalize pass takes the running ones).  blocks = bn_fused_max_blocks(SM count, bwd) (0: the kernel cannot be
// co-resident; use the separate launches); counter: two zeroed 64-bit words owned by the caller, shared by all
// launches of one stream.
struct BnFusedProb { BnStatProb st; BnFinalProb fin; BnApplyProb ap; };
int bn_fused_max_blocks(int num_sms, bool bwd);
cudaError_t launch_bn_fused(const BnFusedProb* d_probs, int n, bool bwd, bool stats, int blocks, unsigned long long* counter,
                            int* d_status, cudaStream_t s);

// 3x3 stride-1 convolution of an image with very few channels (9 * Cin <= 32: the stem of App. B.3's
// networks, which a 64-deep tensor-core k-slice would leave mostly empty), on the FP32 ALUs with fp32
// accumulation.  x [N,H,W,Cin] NHWC, filters w [Cout,3,3,Cin], y / dy [N,H,W,Cout]; Cout % 8 == 0.
//   forward: y = conv(x, w).
//   filter gradient: part[blk][co*9*Cin + k] = sum over block blk's SMALLCONV_PIXELS pixels of
//     dy[pixel, co] * x[pixel shifted by tap(k), channel(k)]  (needs 256 % Cout == 0); the blocks'
//     partial sums are added up in block order by the caller's column reduction.
struct SmallConvProb { const void* x; const void* w; void* y; const void* dy; float* part; int N, H, W, Cin, Cout; };
enum { SMALLCONV_PIXELS = 512 };
void launch_small_conv_fwd(const SmallConvProb& p, bool w_is_bf16, bool is_bf16, cudaStream_t s);
void launch_small_conv_wgrad(const SmallConvProb& p, bool is_bf16, cudaStream_t s);

struct GapProb { const void* x; void* y; const void* dy; void* dx; int N, HW, C; };
void launch_gap_fwd(const GapProb* d_probs, int n, int max_n, int max_c, bool is_bf16, cudaStream_t s);
void launch_gap_bwd(const GapProb* d_probs, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8 = false);

struct AddProb { const void* a; const void* b; void* out; long long n; };
// a[i] = (a[i] + b[i]) / 2 in fp32: the averaged gradient of a layer shared by two overlapping blocks (App. A.2)
struct AvgProb { float* a; const float* b; long long n; };
void launch_average_f32(const AvgProb* d_probs, int n, long long max_elems, cudaStream_t s);
// vec8: bf16, every problem's element count a multiple of 8 and its tensors 16-byte aligned
void launch_add(const AddProb* d_probs, int n, long long max_elems, bool is_bf16, cudaStream_t s, bool vec8 = false);

// ---------------------------------------------------------------------------- optimizer
struct OptimArgs {
  float* master; float* m1; float* m2; const float* grad; bf16* working;  // working may be null
  long long n_total;    // elements in the arena
  long long n_matrix;   // leading elements that are matrices (weight decay + bf16 working copy)
  int kind; float lr, momentum, weight_decay, beta1, beta2, eps;
  float omb1, omb2;     // 1 - beta, rounded from double
  float bc1, bc2;       // 1 - beta^t, rounded from double
  // Per-chunk mode (idle ramp-up of the pipelined schedule, Sec. 6: a chunk that no minibatch has reached
  // yet makes no update, so the chunks' step counts differ).  seg_end[i] = one past the last arena element
  // of segment i (segments in arena order), seg_chunk[i] = its chunk, chunk_tab[k] = (active ? 1 : 0,
  // 1 - beta1^t_k, 1 - beta2^t_k, unused).  Null seg_end: all chunks share bc1 / bc2 and are updated.
  const long long* seg_end; const int* seg_chunk; int n_seg;
  const float4* chunk_tab;
};
void launch_optim(const OptimArgs& a, cudaStream_t s);

// ---------------------------------------------------------------------------- single-launch MLP step (fp32)
// A step as a list of phases; the blocks of one cooperative launch share a phase's work units round-robin and
// meet at a grid-wide barrier between phases.  A task is a run of units of one kind, a unit being what one block
// of FUSED_THREADS threads does at a time: a 16x16 or 32x32 output tile of a GEMM, one softmax cross-entropy row
// per warp, one column of a column sum per thread, one loss reduction, one label check, four arena elements of
// the optimizer sweep per thread, one 128-byte line per thread of a range to be brought into L2 ahead of its use.
enum { FUSED_THREADS = 512 };
enum FusedTaskType { FT_GEMM16 = 0, FT_GEMM32, FT_XENT, FT_COLSUM, FT_LOSS, FT_LABELS, FT_OPTIM, FT_PREFETCH };
struct FusedTask { int type, index, unit_start, units; };      // index into the array of its kind
struct FusedPhase { int task_begin, task_end, units; };
// C[m,n] = epilogue(sum_k A(m,k) B(n,k)) with the operand conventions of GemmProb, fp32 throughout; act is
// EPI_NONE, EPI_RELU (after the bias) or EPI_RELU_MASK (aux = the layer's output, [M, ldc])
struct FusedGemm {
  const float* A; const float* B; float* C; const float* bias; const float* aux;
  int M, N, K, ldc, act, tiles_n;
  int a_ms, a_ks, b_ns, b_ks;
};
struct FusedXent { float* z; const int* y; const int* n_valid; float* row_loss; int rows, classes, ld; };
struct FusedColSum { const float* x; float* out; int rows, cols, ld; };
struct FusedPrefetch { const void* p; long long bytes; };
enum { FUSED_MAX_PHASES = 64, FUSED_MAX_TASKS = 256, FUSED_MAX_GEMMS = 64 };   // tables that are held in shared memory
struct FusedArgs {
  const FusedPhase* phases; int n_phases;
  const FusedTask* tasks; int n_tasks;
  const FusedGemm* gemms; int n_gemms;
  const FusedXent* xents; const FusedColSum* colsums; const LossProb* losses; const LabelProb* labels;
  const FusedPrefetch* prefetches;
  OptimArgs opt;                      // chunk_tab non-null: per-chunk mode (idle chunks make no update, read NaN)
  float* d_losses; int* status;
  unsigned long long* counter;        // [2], zero between launches: barrier arrivals, blocks that have left
  // the step's inputs are read where the caller holds them: an operand or label pointer equal to x_slot /
  // y_slot (the handle's own input buffers, which the task tables name) is replaced by x / y
  const void* x_slot; const int* y_slot; const void* x; const int* y;
};
// Blocks of one cooperative launch (one per SM), or 0 if the kernel cannot be resident.
int fused_mlp_max_blocks(int num_sms);
cudaError_t launch_fused_mlp_step(const FusedArgs& args, int blocks, cudaStream_t s);
// losses[k] = NaN for the chunks whose chunk_tab entry is inactive
void launch_mask_losses(float* losses, const float4* chunk_tab, int K, cudaStream_t s);

}  // namespace lp
