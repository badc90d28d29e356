/*
 * lp.h -- C ABI of the local-update training step on one NVIDIA B200 (sm_100a).
 *
 * The method (paper Sec. 3, "Local Parallelism"): a network is cut into a sequence of K chunks.
 * Chunk k runs its layers on the output of chunk k-1 (chunk 0 on the minibatch), feeds the result
 * to an auxiliary head whose loss has the same form as the global objective, back-propagates that
 * loss into its own layers only (the activation handed to the next chunk carries no gradient), and
 * applies its own optimizer update (Sec. 1, Sec. 6: updates need not wait for the rest of the
 * network).  Back-propagation is the case K = 1.
 *
 * All pointers named "device" are CUDA device pointers owned by the caller; "host" pointers are
 * ordinary host memory.  Nothing here takes or returns a framework type.  Every entry point
 * returns an lp_status (0 = LP_OK, negative = error) and never throws, aborts or traps; after an
 * error lp_last_error(h) gives a message.  One handle may be used by one thread at a time.
 */
#ifndef LP_H_
#define LP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lp_handle_s* lp_handle;
typedef int lp_status;

enum {
  LP_OK = 0,
  LP_ERR_INVALID_ARG = -1, /* null pointer, bad enum, bad index                                  */
  LP_ERR_SHAPE = -2,       /* sizes that the model family cannot take (see lp_model_spec)        */
  LP_ERR_UNSUPPORTED = -3, /* valid request that the library does not implement                 */
  LP_ERR_ALLOC = -4,       /* device allocation failed                                           */
  LP_ERR_CUDA = -5,        /* a CUDA call failed; message holds the CUDA error string            */
  LP_ERR_STATE = -6,       /* call not allowed in the handle's current state                     */
  LP_ERR_LABEL_RANGE = -7, /* lp_status_poll: a label or token id was outside its range          */
  LP_ERR_NONFINITE = -8,   /* lp_status_poll: a loss was NaN or infinite                         */
  LP_ERR_TIMEOUT = -9      /* lp_status_poll: a device-side wait gave up (kernel returned early)  */
};

enum { LP_FAMILY_MLP = 0, LP_FAMILY_LM = 1, LP_FAMILY_RESNET = 2 };
enum { LP_BLOCK_BASIC = 0, LP_BLOCK_BOTTLENECK = 1 };
enum { LP_FP32 = 0, LP_BF16 = 1 }; /* LP_BF16: bf16 matrices and activations, fp32 master weights,
                                      fp32 accumulation, fp32 normalisation statistics and loss  */
enum { LP_HEAD_LINEAR = 0, LP_HEAD_LN_LINEAR = 1, LP_HEAD_GAP_LINEAR = 2, LP_HEAD_BN_RELU_GAP_LINEAR = 3 };
enum { LP_OPT_SGDM = 0, LP_OPT_ADAM = 1 };
enum { LP_SYNC = 0, LP_PIPELINED = 1 };
enum { LP_MASTER = 0, LP_WORKING = 1, LP_MOMENT1 = 2, LP_MOMENT2 = 3, LP_GRAD = 4 };

/*
 * Model description.  Only the fields of the chosen family are read.  Arrays are host pointers
 * read during lp_create only.
 *
 *  MLP (App. A.1: matrix product, bias add, ReLU per layer): n_layers Linear+ReLU layers of widths
 *    layer_widths[], input width d_in; chunk k holds layers_per_chunk[k] consecutive layers.
 *  LM (App. B.2: decoder-only transformer, one or more layers per chunk): learned token and
 *    position embeddings (in chunk 0), pre-LayerNorm blocks with causal softmax attention
 *    (n_heads heads of d_model/n_heads = 64) and a GELU feed-forward of width d_ffn; chunk k holds
 *    blocks_per_chunk[k] blocks.
 *  RESNET (App. B.3): 3x3 stem convolution + BatchNorm + ReLU (in chunk 0), then K stages of
 *    blocks_per_stage (or stage_blocks[k]) BasicBlocks with stage_channels[k] channels, or bottleneck
 *    blocks (block_kind); stages after the first start with stride 2 and a 1x1-convolution + BatchNorm
 *    shortcut.  BatchNorm uses batch statistics
 *    (and keeps running statistics, which lp_evaluate can use).
 */
typedef struct {
  int family;
  int dtype;
  int batch;
  /* MLP */
  int d_in;
  int n_layers;
  const int* layer_widths;     /* [n_layers] */
  const int* layers_per_chunk; /* [K] */
  /* LM */
  int vocab, seq_len, d_model, n_heads, d_ffn;
  const int* blocks_per_chunk; /* [K] */
  /* RESNET */
  int in_channels, height, width, stem_channels;
  const int* stage_channels; /* [K] */
  int blocks_per_stage;
  /* 0: tensor-core GEMMs wherever a problem's sizes allow (default); 1: plain FP32-ALU GEMMs
     everywhere (diagnostic).  The fp32 dtype always uses the FP32-ALU GEMMs. */
  int gemm_backend;
  /* 0: x is raw data (token ids, NCHW images, MLP rows).  1: the model is an inner piece of a longer chain,
     placed on its own GPU (Sec. 6: one block per device), and x is the activation the previous piece
     produced, in the compute dtype: LM -- [batch, seq_len, d_model], no embedding tables; RESNET --
     NHWC [batch, height, width, in_channels], no stem, and the first stage already starts with stride 2
     and a 1x1 shortcut; MLP -- no difference.  No gradient is formed for x (Sec. 3). */
  int input_is_activation;
  /* RESNET: LP_BLOCK_BASIC (0, default): BasicBlocks, two 3x3 convolutions.  LP_BLOCK_BOTTLENECK: the blocks of the
     deeper networks (Sec. 4.3 trains a ResNet-50): 1x1 convolution to stage_channels[k], 3x3 convolution (it
     carries the stage's stride), 1x1 convolution to 4 * stage_channels[k], each followed by BatchNorm and the first
     two by ReLU; identity shortcut, or 1x1 convolution + BatchNorm where the shape changes; ReLU after the sum.
     A stage's output then has 4 * stage_channels[k] channels. */
  int block_kind;
  /* RESNET, nullable: [K] blocks per stage (a ResNet-50 has 3, 4, 6, 3); NULL: blocks_per_stage in every stage. */
  const int* stage_blocks;
} lp_model_spec;

/* Auxiliary head of every chunk (Sec. 3: same form as the global objective): softmax
 * cross-entropy over `classes` on top of Linear (MLP), LayerNorm+Linear (LM; classes = vocab) or
 * global-average-pool+Linear (RESNET).  RESNET also takes LP_HEAD_BN_RELU_GAP_LINEAR, the head of
 * App. B.3: BatchNorm (own scale, shift and running statistics per chunk, tensors
 * "c<k>.head.bn.{g,b,rm,rv}") and ReLU on the stage output before the spatial mean. */
typedef struct {
  int kind;
  int classes;
} lp_head_spec;

/* Per-chunk optimizer (App. B: Adam, SGD with momentum).  SGDM: g += weight_decay*w on matrices,
 * filters and embedding tables only; v = momentum*v + g; w -= lr*v.  ADAM: bias-corrected, step
 * count from 1, eps added outside the square root. */
typedef struct {
  int kind;
  float lr, momentum, weight_decay, beta1, beta2, eps;
} lp_optim_spec;

/* Optional allocator for the handle's device memory (e.g. backed by a framework's caching
 * allocator).  alloc returns a device pointer aligned to 256 bytes or NULL.  If the lp_alloc
 * pointer given to lp_create is NULL, cudaMalloc/cudaFree are used. */
typedef struct {
  void* (*alloc)(size_t bytes, void* user);
  void (*release)(void* ptr, void* user);
  void* user;
} lp_alloc;

typedef struct {
  char name[48]; /* e.g. "c3.b3.Wqkv", "c0.head.W" */
  int chunk;
  int ndim;
  int64_t shape[4]; /* Linear [out,in]; convolution filter [C_out,kh,kw,C_in]; embedding [rows,d] */
  int64_t numel;
  int has_working_bf16; /* 1 if a bf16 working copy exists (matrices under LP_BF16) */
} lp_tensor_info;

/*
 * lp_create: build the K-chunk model, its heads and optimizer state on the current CUDA device
 * (Sec. 3).  All parameters, optimizer state, saved activations and the boundary buffers are
 * allocated here and owned by the handle.  Parameters start at zero: the caller installs initial
 * values with lp_set_tensor.  Errors: INVALID_ARG, SHAPE (e.g. d_model/n_heads != 64, sizes not
 * accepted by the family), UNSUPPORTED, ALLOC, CUDA.  On error *out is NULL.
 */
lp_status lp_create(const lp_model_spec* model, int K, const lp_head_spec* head,
                    const lp_optim_spec* optim, const lp_alloc* alloc, lp_handle* out);

/*
 * lp_step: one local update step (Sec. 3; schedules: App. E.1 for the synchronous order, Sec. 6
 * for the pipelined steady state).
 *   x: device.  MLP: [batch, d_in] fp32 (LP_FP32) or bf16 (LP_BF16), row-major.  LM: int32 token
 *      ids [batch, seq_len].  RESNET: [batch, C, H, W] (NCHW) fp32 or bf16.
 *   y: device int32 labels.  MLP/RESNET: [batch].  LM: [batch, seq_len], -1 = position ignored.
 *   schedule: LP_SYNC -- chunk k reads the output chunk k-1 produced in this step from the same
 *      minibatch.  LP_PIPELINED -- chunk k reads the output chunk k-1 produced in the previous
 *      step, with the labels of that older minibatch; the first pipelined step after lp_create or
 *      lp_reset_pipeline fills the boundary buffers by a forward pass of (x, y).
 *   stream: cudaStream_t (as void*) all work is issued on; no host synchronisation happens.
 *   out_losses: device, K floats: each chunk's mean auxiliary loss for the minibatch it trained on.
 * x, y and out_losses must stay valid until the caller synchronises `stream`.
 * Errors: INVALID_ARG, STATE (sync step while a pipeline is in flight needs lp_reset_pipeline), CUDA.
 */
lp_status lp_step(lp_handle h, const void* x, const void* y, int schedule, void* stream,
                  float* out_losses);

/* lp_step_host: the same step with HOST buffers: copies x and y to the device, runs lp_step,
 * copies the K losses back to out_losses_host and synchronises `stream` before returning. */
lp_status lp_step_host(lp_handle h, const void* x_host, const void* y_host, int schedule,
                       void* stream, float* out_losses_host);

/*
 * lp_forward: forward chain through all chunks with the current weights; no gradient, no update.
 *   y may be NULL (then out_losses must be NULL).  out_logits (device, nullable) receives the last
 *   chunk's head logits, [rows, classes] in the activation dtype, rows = batch (MLP, RESNET) or
 *   batch*seq_len (LM).  out_losses (device, nullable): K floats.
 */
lp_status lp_forward(lp_handle h, const void* x, const void* y, void* stream, void* out_logits,
                     float* out_losses);

/*
 * lp_evaluate: the forward chain of lp_forward on a labelled minibatch, reporting how well every chunk's
 * auxiliary head predicts it (Sec. 3: each block is trained to predict the target on its own; the last
 * chunk's head is the network's output).  No gradient, no update.
 *   out_losses  (device, nullable): K floats, each chunk's mean auxiliary loss.
 *   out_correct (device, nullable): K int32, the number of rows whose prediction equals the label.
 *   out_pred    (device, nullable): K x rows int32 (rows = batch, or batch*seq_len for LM), the predicted
 *     class of every row: the index of its largest logit, the lowest index among equal logits, taken on
 *     the logits as the head stores them (activation dtype).  Rows with label -1 get a prediction but
 *     are not counted in out_correct.
 *   bn_mode: what BatchNorm (RESNET) normalises with.  LP_BN_BATCH: the statistics of this minibatch, as in
 *     training.  LP_BN_RUNNING: its running mean and variance -- exponential averages (momentum 0.1) of the
 *     batch mean and the unbiased batch variance that every training step of a chunk updates (tensors
 *     "<bn>.rm" and "<bn>.rv", starting from 0 and 1; the optimizer never changes them).  Ignored by the
 *     other families.
 * Errors: INVALID_ARG, CUDA.
 */
enum { LP_BN_BATCH = 0, LP_BN_RUNNING = 1 };
lp_status lp_evaluate(lp_handle h, const void* x, const void* y, void* stream, int bn_mode, float* out_losses,
                      int* out_correct, int* out_pred);

/* lp_destroy: release everything the handle owns.  NULL is accepted. */
lp_status lp_destroy(lp_handle h);

/* Parameter access (host buffers; these calls synchronise `stream`).  `which` selects the fp32
 * master copy, the bf16 working copy (uint16 bit patterns), the optimizer moments (fp32) or the
 * last step's gradient (fp32).  Setting LP_MASTER also refreshes the bf16 working copy. `bytes`
 * must equal numel * element size, else LP_ERR_SHAPE. */
int lp_num_tensors(lp_handle h);
lp_status lp_tensor_info_get(lp_handle h, int i, lp_tensor_info* out);
lp_status lp_get_tensor(lp_handle h, int i, int which, void* host_dst, size_t bytes, void* stream);
lp_status lp_set_tensor(lp_handle h, int i, int which, const void* host_src, size_t bytes,
                        void* stream);

/* Forget the activations in flight between chunks; the next pipelined step starts the ramp-up again. */
lp_status lp_reset_pipeline(lp_handle h);

/*
 * Output activation of chunk k as the last lp_step left it (the tensor the next chunk reads; Sec. 3: it
 * carries no gradient), for handing it to the piece of the chain that lives on another GPU (Sec. 6).
 * lp_chunk_output_bytes gives its size; layout: MLP [batch, width], LM [batch, seq_len, d_model], RESNET
 * NHWC [batch, H_k, W_k, C_k], compute dtype.  lp_chunk_output copies it device-to-device into dst
 * (device, caller-owned, at least that many bytes) on `stream`, without host synchronisation.
 * Errors: INVALID_ARG (null, k outside [0, K), bytes too small), STATE (no step has run yet), CUDA.
 */
size_t lp_chunk_output_bytes(lp_handle h, int k);
lp_status lp_chunk_output(lp_handle h, int k, void* dst, size_t bytes, void* stream);

/*
 * lp_set_ramp: how the pipelined schedule starts after lp_create or lp_reset_pipeline (Sec. 6 speaks only
 * of "an initial ramp-up phase"; both readings are offered).
 *   LP_RAMP_PRIME (default): the first pipelined step fills every boundary buffer by a forward pass of its
 *     own minibatch; every chunk then trains in every step, and that first step equals a synchronous step.
 *   LP_RAMP_IDLE: nothing is filled.  In the s-th pipelined step after the reset (s = 0, 1, ...) only chunks
 *     0..s train: chunk k waits until an activation produced from real data reaches it, as a pipeline of K
 *     processors would.  An idle chunk's parameters, optimizer state and step count do not change, and its
 *     entry of out_losses is NaN.  (Idle chunks still execute, on stale buffer contents; the cost of a step
 *     is the same.)
 * Allowed only while no pipeline is in flight.  Errors: INVALID_ARG, STATE.
 */
enum { LP_RAMP_PRIME = 0, LP_RAMP_IDLE = 1 };
lp_status lp_set_ramp(lp_handle h, int ramp);

/*
 * lp_set_drain: the end of a pipelined run (Sec. 6: each stage works on the minibatch its predecessor finished one
 * iteration earlier, so the last minibatch leaves chunk k only k iterations after it entered chunk 0).  In
 * pipelined steps that follow, chunks 0 .. idle_first-1 idle: their minibatches are exhausted, so their parameters,
 * optimizer state and step counts stay as they are and their entry of out_losses is NaN, while the chunks behind
 * them go on with what the boundary buffers still hold.  (Like the chunks that idle during the ramp-up they still
 * execute; what they publish is not read by a training chunk.)  idle_first = 0 ends the drain.  Pipelined steps
 * only.  Errors: INVALID_ARG (idle_first outside [0, K]).
 */
lp_status lp_set_drain(lp_handle h, int idle_first);

/*
 * lp_set_fused_step: the single-launch form of the step.  A small MLP with fp32 storage (a step of at most a few
 * GFLOP, K <= 64) is bound by the latency of its dependent launches, not by arithmetic; for such a handle the
 * whole step of Sec. 3 -- label check, forward of every chunk, heads, losses, backward inside each chunk,
 * per-chunk optimizer update -- runs as ONE cooperative launch whose thread blocks walk the phases of the step
 * together, with a grid-wide barrier (bounded wait: LP_ERR_TIMEOUT at the next lp_status_poll) between phases.
 * Same arithmetic as the grouped launches up to the order of fp32 sums; every sum has a fixed order, so a step
 * is bit-reproducible.  lp_step then reads x and y where the caller holds them (no copy into the handle).  It is
 * on by default where it is available and never used with overlapping updates (lp_set_overlap).  on = 0 selects
 * the grouped launches.  Errors: UNSUPPORTED (on != 0 for a handle that has no single-launch form: another
 * family, bf16 storage, a larger network).
 */
lp_status lp_set_fused_step(lp_handle h, int on);

/*
 * lp_set_overlap: overlapping local parallelism (Sec. 3, Fig. 2 c; cost in App. A.2).  With on != 0 the
 * block trained by chunk k's loss also contains the last layer of chunk k-1: that loss is propagated one
 * layer past the chunk boundary and stops at that layer's input.  The shared layer exists once (one forward
 * pass); it receives a gradient from its own chunk's loss and one from the next chunk's, and its update
 * uses their mean.  All other parameters are updated as without overlap.  LP_GRAD of a shared layer then
 * holds the mean.  Synchronous steps only (a pipelined lp_step returns LP_ERR_UNSUPPORTED while overlap is
 * on).  The shared layer is the previous chunk's last Linear+ReLU (MLP), its last transformer block (LM; App.
 * B.2 trains layer-wise blocks) or its last BasicBlock (RESNET).  Needs K >= 2, otherwise LP_ERR_UNSUPPORTED.
 */
lp_status lp_set_overlap(lp_handle h, int on);

/* Read the device status word (synchronises `stream`): LP_OK, or LABEL_RANGE / NONFINITE /
 * TIMEOUT if any kernel since the last poll flagged it.  The word is cleared. */
lp_status lp_status_poll(lp_handle h, void* stream);

/* Checkpoint: master weights, moments, step count, boundary buffers and their labels.
 * lp_save_state / lp_load_state synchronise the device.  A handle restored into an identically
 * created handle continues bit-for-bit. */
size_t lp_state_size(lp_handle h);
lp_status lp_save_state(lp_handle h, void* host_dst, size_t bytes);
lp_status lp_load_state(lp_handle h, const void* host_src, size_t bytes);

/*
 * Kernel-level entry for tests and profiling: one grouped launch of n bf16 GEMM problems
 *   C[m,n] = epilogue( sum_k A(m,k) * B(n,k) ),  A(m,k) = A[m*a_ms + k*a_ks], B(n,k) = B[n*b_ns + k*b_ks]
 * (the products of a Linear layer, App. A.1, in forward, input-gradient and weight-gradient form).
 * All pointers inside the descriptors are device pointers; `probs` itself is a host array.
 * Exactly one stride of each operand must be 1.  act: 0 none, 1 ReLU, 2 GELU (C2 receives the
 * pre-activation), 3 multiply by [aux > 0], 4 multiply by GELU'(aux).  out_f32: C is float, else bf16.
 * backend: 0 = tensor cores where the sizes allow, 1 = FP32 ALUs.  *used_tensor_cores (nullable)
 * receives how many of the problems ran on the tensor-core kernel.  Asynchronous on `stream`
 * except for the upload of the descriptor table.  Refused before anything is uploaded or launched
 * (INVALID_ARG): null A, B or C; non-positive sizes or strides; no unit stride in an operand;
 * ldc < N; act outside 0..4; act 2 without C2 or with out_f32; act 3 or 4 without aux.  This entry
 * and lp_conv3x3_bf16 keep their scratch on the device that was current at their first call and
 * return UNSUPPORTED on any other device of the process.  Errors: INVALID_ARG, UNSUPPORTED, ALLOC, CUDA.
 */
typedef struct {
  const void* A; const void* B; void* C; void* C2;
  const float* bias; const void* resid; const void* aux;
  int M, N, K;
  long long a_ms, a_ks, b_ns, b_ks;
  int ldc, act, out_f32;
} lp_gemm_desc;
lp_status lp_gemm_bf16(int n, const lp_gemm_desc* probs, int backend, void* stream, int* used_tensor_cores);

/*
 * lp_conv3x3_bf16: kernel-level entry for tests and profiling: one 3x3 convolution, stride 1, zero padding 1,
 * no bias, over bf16 NHWC activations (the residual blocks of App. B.3), as an implicit GEMM on the tensor
 * cores: the activation tensor itself is the GEMM operand, fetched as one shifted box per filter tap; no
 * im2col matrix exists.  All pointers are device pointers.
 *   LP_CONV_FORWARD:     act = x  [n,h,w,c_in],  other = filters [c_out,3,3,c_in] bf16, out = y  [n,h,w,c_out] bf16
 *                        y[n,p,q,o] = sum_{i,j,c} x[n,p+i-1,q+j-1,c] * filters[o,i,j,c]
 *   LP_CONV_INPUT_GRAD:  act = dy [n,h,w,c_out], other = filters,                     out = dx [n,h,w,c_in]  bf16
 *   LP_CONV_FILTER_GRAD: act = x  [n,h,w,c_in],  other = dy [n,h,w,c_out] bf16,       out = dW [c_out,3,3,c_in] fp32
 * Accepted sizes: the channel count of `act` a multiple of 64, the other channel count a multiple of 8,
 * w a divisor of 64, h*w a divisor or a multiple of 128, 16-byte aligned tensors; otherwise
 * LP_ERR_UNSUPPORTED and nothing is launched.  Asynchronous on `stream` except for the upload of the
 * descriptor table.  Errors: INVALID_ARG, SHAPE, UNSUPPORTED, ALLOC, CUDA (message: lp_last_error(NULL)).
 */
enum { LP_CONV_FORWARD = 0, LP_CONV_INPUT_GRAD = 1, LP_CONV_FILTER_GRAD = 2 };
lp_status lp_conv3x3_bf16(int form, const void* act, const void* other, void* out, int n, int h, int w,
                          int c_in, int c_out, void* stream);

/*
 * lp_conv2d_bf16: the same entry for all convolutions of App. B.3's residual networks that run as implicit GEMMs:
 * ksize 3 (zero padding 1) or 1 (no padding), stride 1 or 2.  h x w is the INPUT image; the output image is
 * ho x wo with ho = (h - 1) / stride + 1, wo = (w - 1) / stride + 1.  The operand tiles are TMA boxes that step
 * through the input activation with the stride, one shifted box per filter tap.
 *   LP_CONV_FORWARD:     act = x [n,h,w,c_in], other = filters [c_out,ksize,ksize,c_in] bf16, out = y [n,ho,wo,c_out] bf16
 *                        y[n,p,q,o] = sum_{i,j,c} x[n, stride p + i - pad, stride q + j - pad, c] * filters[o,i,j,c]
 *   LP_CONV_FILTER_GRAD: act = x, other = dy [n,ho,wo,c_out] bf16, out = dW [c_out,ksize,ksize,c_in] fp32
 *   LP_CONV_INPUT_GRAD:  ksize 3, stride 1 only (otherwise LP_ERR_UNSUPPORTED): as lp_conv3x3_bf16.
 * Accepted sizes: as for lp_conv3x3_bf16, with wo and ho*wo in place of w and h*w.  Errors: as lp_conv3x3_bf16.
 */
lp_status lp_conv2d_bf16(int form, const void* act, const void* other, void* out, int n, int h, int w,
                         int c_in, int c_out, int ksize, int stride, void* stream);

/*
 * lp_attention_bf16: kernel-level entry for tests and profiling: causal multi-head softmax attention with heads
 * of 64 over bf16 activations (the attention of App. B.2's transformer layers), on the tensor cores with the
 * score tiles held in tensor memory.  All pointers are device pointers.
 *   qkv  [batch, seq_len, 3*d], d = 64*n_heads: columns [0, d) queries, [d, 2d) keys, [2d, 3d) values, head h
 *        at columns h*64 of each third.  Position t attends to positions <= t; scores are scaled by 1/8.
 *   LP_ATTN_FORWARD:  reads qkv; writes o [batch, seq_len, d] bf16 and lse [batch, n_heads, seq_len] fp32, each
 *        row's log2 of the sum of 2^(score * log2(e) / 8) over the keys it sees.  dout, dqkv, delta are ignored.
 *   LP_ATTN_BACKWARD: reads qkv, o and lse as the forward call left them and dout [batch, seq_len, d] bf16 (the
 *        gradient of o); writes dqkv [batch, seq_len, 3*d] bf16 and delta [batch, n_heads, seq_len] fp32 (row
 *        sums of dout * o).
 * The call synchronises `stream` before it returns.  Errors: INVALID_ARG (null pointer, unknown form), SHAPE
 * (non-positive sizes), UNSUPPORTED (tensors not 16-byte aligned; a device other than the one of the first
 * call), ALLOC, CUDA, TIMEOUT (a bounded device-side wait gave up: outputs are not valid).
 */
enum { LP_ATTN_FORWARD = 0, LP_ATTN_BACKWARD = 1 };
lp_status lp_attention_bf16(int form, const void* qkv, void* o, float* lse, const void* dout, void* dqkv, float* delta,
                            int batch, int seq_len, int n_heads, void* stream);

/*
 * lp_gemm_bf16_static: lp_gemm_bf16 for callers that cannot allocate device memory.  (The paper
 * has no counterpart to this entry point; it exists for the library's users.)
 *
 * Who needs it: code that may not call cudaMalloc or cudaFree at the point where it launches work --
 * a serving or real-time loop that must never take the driver's allocator lock nor the device-wide
 * synchronisation those calls imply, a plug-in inside a host program that handed out the whole
 * device-memory budget up front, code running under a memory-pool manager that forbids outside
 * allocations.  lp_gemm_bf16 keeps its problem table, its TMA tensor maps and its status word in a
 * cudaMalloc'ed buffer that grows on demand; this variant keeps them in a fixed array that is part of
 * the library image (about 58 KB of device memory on every GPU that loads the library, held until the
 * process exits) and calls no cudaMalloc, cudaFree or any other allocating routine.
 *
 *   n: 1 .. LP_GEMM_STATIC_MAX problems; more is rejected with LP_ERR_SHAPE and nothing is launched.
 *   probs: host array, same meaning and the same checks as for lp_gemm_bf16 (device pointers inside).
 *     Each problem runs on the tensor-core kernel if its sizes allow, otherwise on the FP32-ALU kernel.
 *   stream: the problems are uploaded and launched on this stream, asynchronously.
 *
 * The first call on a device looks up the array's device address (one-time set-up, with that
 * device current); make that first call before any stream capture begins.  All calls on a device
 * share the one array, which keeps the previous call's contents: each call overwrites the table
 * entries it uses.  Two calls whose work may overlap on the GPU (different streams without an
 * ordering between them) race on the array; calls on one stream are ordered.  Host threads are
 * serialised by a lock while they fill the (process-wide, host-side) staging table.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED (device ordinal above 63), CUDA; the message is returned
 * by lp_gemm_static_last_error().
 *
 * lp_gemm_static_poll: synchronises `stream`, reads and clears the array's status word on the current
 * device.  LP_OK, or LP_ERR_TIMEOUT if a bounded device-side wait of any call since the last poll gave
 * up (those calls' outputs are then not valid).  Allocates nothing.
 */
#define LP_GEMM_STATIC_MAX 64
lp_status lp_gemm_bf16_static(int n, const lp_gemm_desc* probs, void* stream);
lp_status lp_gemm_static_poll(void* stream);
const char* lp_gemm_static_last_error(void);

/*
 * Per-kernel-class timing for benchmarks.  While enabled, every grouped launch of lp_step is
 * bracketed by a pair of CUDA events on the caller's stream.  lp_profile_read synchronises the
 * device and returns, for each class and summed over the steps since the last read: device
 * milliseconds, algorithmic work (FLOPs for the GEMM and attention classes, bytes for the others)
 * and kernel launches.  Each output array has LP_KIND_COUNT entries.
 */
enum {
  LP_KIND_OTHER = 0, LP_KIND_GEMM_TC = 1, LP_KIND_GEMM_ALU = 2, LP_KIND_NORM = 3, LP_KIND_XENT = 4,
  LP_KIND_ATTN = 5, LP_KIND_OPTIM = 6, LP_KIND_REDUCE = 7, LP_KIND_EMBED = 8, LP_KIND_CONV_AUX = 9,
  LP_KIND_COUNT = 10
};
lp_status lp_profile_enable(lp_handle h, int on);
lp_status lp_profile_read(lp_handle h, double* ms, double* work, int* launches);

/*
 * FLOP cost model (App. A): what a training run costs in total FLOPs and in sequential FLOPs, the
 * paper's stand-in for time on ideal hardware.  Host arithmetic only; no device is touched.
 *
 * App. A.2 describes a model by its layer count, the forward cost of one layer per example, the cost
 * of one auxiliary loss per example, the backward multiplier (backward cost / forward cost) and its
 * parameter count (the optimizer costs ten FLOPs per parameter per step).  The methods:
 *   BACKPROP     one forward and backward pass, one loss; examples are the only parallelism.
 *   GREEDY       one auxiliary loss per layer; layers and examples run in parallel.
 *   OVERLAPPING  as GREEDY, with a second backward pass through all layers but the last and two more
 *                FLOPs per parameter per step for averaging the two gradients.
 *   CHUNKED      `chunks` blocks, one auxiliary loss each; blocks and examples run in parallel.
 *   LAST_LAYERS  back-propagation through the last `chunks` layers only.
 * Two of the printed per-example formulas are garbled (CHUNKED lacks the layer count, LAST_LAYERS an
 * addition sign); they are read by analogy with BACKPROP.
 * total_flops = cost_per_example * steps * batch_size + steps * optimizer cost;
 * sequential_flops = total_flops / (batch_size * parallelism).
 * Errors: INVALID_ARG (null pointer, unknown method), SHAPE (negative sizes, chunks outside
 * [1, layers] for the two methods that use it).
 *
 * lp_mlp_layer_flops / lp_mlp_aux_flops are App. A.1's per-example counts for one fully connected
 * layer with ReLU (input_size -> units) and for a linear classifier with softmax cross-entropy
 * (units -> classes); they give forward_cost and aux_cost for the MLP family.
 */
enum { LP_COST_BACKPROP = 0, LP_COST_GREEDY = 1, LP_COST_OVERLAPPING = 2, LP_COST_CHUNKED = 3,
       LP_COST_LAST_LAYERS = 4 };
typedef struct {
  int method;                 /* LP_COST_*                                        */
  long long layers;           /* layers (or residual / transformer blocks)        */
  long long chunks;           /* K for CHUNKED and LAST_LAYERS, ignored otherwise */
  long long batch_size;       /* examples per step                                */
  long long steps;            /* optimizer steps of the run                       */
  double forward_cost;        /* FLOPs of one layer's forward pass, per example   */
  double aux_cost;            /* FLOPs of one auxiliary loss, per example         */
  double backward_multiplier; /* backward FLOPs / forward FLOPs                   */
  double parameters;          /* parameters of the whole model                    */
} lp_cost_spec;
typedef struct {
  double cost_per_example; /* FLOPs of one step for one example, optimizer excluded */
  double total_flops;
  double parallelism;      /* units of work that can run at once, per example       */
  double sequential_flops;
} lp_cost_result;
lp_status lp_cost_model(const lp_cost_spec* spec, lp_cost_result* out);
double lp_mlp_layer_flops(long long input_size, long long units);
double lp_mlp_aux_flops(long long units, long long classes);

/* Number of kernel launches the last lp_step issued (for reporting). */
int lp_last_step_launches(lp_handle h);
/* Device bytes owned by the handle. */
size_t lp_device_bytes(lp_handle h);
/* Message of the last error on this handle (or of the last failed lp_create if h is NULL). */
const char* lp_last_error(lp_handle h);

#ifdef __cplusplus
}
#endif
#endif /* LP_H_ */
