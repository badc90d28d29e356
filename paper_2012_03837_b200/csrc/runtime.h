// Host runtime behind the C ABI: the handle, its device memory, the parameter arena, and "plans"
// (ordered lists of grouped kernel launches with device-resident problem tables, built once at
// lp_create because every buffer a step touches is owned by the handle).
#pragma once
#include <functional>
#include <string>
#include <vector>

#include "../../include/lp.h"
#include "lp_kernels.h"

namespace lp {

struct TensorRec {
  std::string name;
  int chunk = 0;
  std::vector<int64_t> shape;
  int64_t numel = 0;
  bool matrix = false;   // Linear weight, convolution filter or embedding table
  int64_t off = 0;       // element offset in the arena
};

// Kernel classes for the optional per-class timing (lp_profile_*): values of LP_KIND_* in lp.h.
enum { KIND_OTHER = 0, KIND_GEMM_TC = 1, KIND_GEMM_ALU = 2, KIND_NORM = 3, KIND_XENT = 4, KIND_ATTN = 5,
       KIND_OPTIM = 6, KIND_REDUCE = 7, KIND_EMBED = 8, KIND_CONV_AUX = 9, KIND_COUNT = 10 };

struct ProfRecord { int kind; int launches; double work; cudaEvent_t e0, e1; };

struct RunCtx {
  cudaStream_t stream;
  void* out_logits;                      // lp_forward only
  std::vector<ProfRecord>* prof;         // non-null: bracket every op with events
  int* out_pred = nullptr;               // lp_evaluate only: per-row predictions [K, rows]
  int* out_correct = nullptr;            // lp_evaluate only: per-chunk count of correct predictions
  const void* x = nullptr;               // training step: where the caller holds the step's inputs (device), when the
  const int* y = nullptr;                // step may read them in place; null: the handle's own input buffers
};

struct PlanOp {
  std::function<void(const RunCtx&)> fn;
  int kind, launches;
  double work;                           // algorithmic FLOPs (GEMM, attention) or bytes (the rest)
};

struct Plan {
  std::vector<PlanOp> ops;
  int launches = 0;
  void add(int n_launches, std::function<void(const RunCtx&)> f, int kind = KIND_OTHER, double work = 0) {
    ops.push_back(PlanOp{std::move(f), kind, n_launches, work});
    launches += n_launches;
  }
  void run(const RunCtx& c) const {
    for (auto& op : ops) {
      if (c.prof && op.launches > 0) {
        ProfRecord r{op.kind, op.launches, op.work, nullptr, nullptr};
        cudaEventCreate(&r.e0);
        cudaEventCreate(&r.e1);
        cudaEventRecord(r.e0, c.stream);
        op.fn(c);
        cudaEventRecord(r.e1, c.stream);
        c.prof->push_back(r);
      } else {
        op.fn(c);
      }
    }
  }
};

struct Handle {
  // ---- specification
  lp_model_spec spec{};
  std::vector<int> layer_widths, per_chunk, stage_channels, stage_blocks;
  lp_head_spec head{};
  lp_optim_spec opt{};
  int K = 0;
  bool bf16_mode = false;
  bool force_simt = false;
  int num_sms = 148;
  int rows = 0;             // rows entering the head: batch (MLP, RESNET) or batch*seq_len (LM)
  // ---- memory
  lp_alloc alloc{};
  bool use_cuda_malloc = true;
  std::vector<void*> blocks;
  size_t device_bytes = 0;
  // ---- parameter arena: [matrices of all chunks | vectors of all chunks]
  std::vector<TensorRec> tensors;
  long long n_total = 0, n_matrix = 0;
  float *master = nullptr, *m1 = nullptr, *m2 = nullptr, *grad = nullptr;
  bf16* working = nullptr;
  // ---- step inputs / outputs
  void* x_in = nullptr;  size_t x_bytes = 0;
  int* y_in = nullptr;   size_t y_bytes = 0;
  float* d_losses = nullptr;
  int* d_status = nullptr;
  // ---- chunk boundaries: activation and labels, two halves each (Sec. 6 pipelining)
  std::vector<void*> bnd[2];
  std::vector<int*> lab[2];
  size_t bnd_bytes_total = 0;
  std::vector<size_t> bnd_bytes;
  std::vector<int*> n_valid;
  // ---- plans
  Plan sync_plan, pipe_plan[2], prime_plan[2], fwd_plan[2];
  Plan eval_plan[2];                           // RESNET: forward with BatchNorm on its running statistics
  bool has_eval_plan = false;
  Plan sync_overlap_plan;                      // synchronous step with overlapping local updates (Sec. 3)
  bool has_overlap_plan = false;
  bool overlap = false;
  std::vector<ColReduceProb> pending_reduce;   // collected while a plan is being built
  int parity = 0;
  int last_wr = -1;         // boundary-buffer slot the last training step wrote (-1: no step yet)
  bool primed = false;
  long long step_count = 0;
  // ---- ramp-up of the pipelined schedule (Sec. 6): LP_RAMP_PRIME fills the boundary buffers by a forward
  // pass; LP_RAMP_IDLE lets chunk k idle until the k-th pipelined step after a reset
  int ramp = 0;
  int drain_first = 0;                         // chunks below this index idle in pipelined steps (end of a run)
  long long pipe_steps = 0;                    // pipelined steps since create / reset
  std::vector<long long> updates;              // per chunk: optimizer updates made so far
  bool per_chunk_counts = false;               // some chunk has idled: the chunks' step counts differ
  const long long* d_seg_end = nullptr;        // arena segments (see OptimArgs), built on first use
  const int* d_seg_chunk = nullptr;
  int n_seg = 0;
  float4* d_chunk_tab = nullptr;
  // ---- single-launch step of a small fp32 MLP (fused_mlp.cu): the same work as sync_plan / pipe_plan[par]
  struct FusedProgram { FusedArgs args{}; double flops = 0; bool ok = false; };
  FusedProgram fused_sync, fused_pipe[2];
  int fused_blocks = 0;                        // blocks of the cooperative launch; 0: not available for this handle
  bool use_fused = false;                      // lp_set_fused_step; on by default where available
  // ---- cooperative launches with grid-wide barriers (grid_barrier.cuh): two zeroed words shared by the launches
  // of this handle (they run on one stream, one after the other), and the BatchNorm kernel's grid (0: unavailable)
  unsigned long long* d_grid_counter = nullptr;
  int bn_fused_blocks[2] = {0, 0};             // forward, backward
  int last_launches = 0;
  bool profiling = false;
  std::vector<ProfRecord> prof;
  std::string err;

  size_t esize() const { return bf16_mode ? 2 : 4; }
  // tensor lookup
  int find(const std::string& name) const;
  const void* W(const std::string& name) const;   // GEMM operand pointer (bf16 working copy or fp32 master)
  float* P32(const std::string& name) const;      // fp32 master (vectors: biases, norm scales)
  float* G(const std::string& name) const;        // fp32 gradient
  // device memory (zero-filled); throws std::runtime_error on failure
  void* dalloc(size_t bytes);
  template <typename T> const T* upload(const std::vector<T>& v) {
    if (v.empty()) return nullptr;
    void* d = dalloc(v.size() * sizeof(T));
    cudaMemcpy(d, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice);
    return (const T*)d;
  }
  void add_tensor(const std::string& name, int chunk, std::vector<int64_t> shape, bool matrix);
  void finalize_arena();
};

// ---- emitters: append one grouped launch (or a few) to a plan
void emit_gemm(Handle& h, Plan& p, std::vector<GemmProb> probs);
void emit_ln_fwd(Handle& h, Plan& p, const std::vector<LnProb>& probs);
// LayerNorm backward; the parameter-gradient partials are queued for the plan's final reduction
void emit_ln_bwd(Handle& h, Plan& p, std::vector<LnBwdProb> probs, const std::vector<float*>& dgamma,
                 const std::vector<float*>& dbeta);
// db[c] = sum_r x[r,c]: partial sums now, final reduction queued
void emit_colsum(Handle& h, Plan& p, const std::vector<ColSumProb>& probs_without_part, const std::vector<float*>& out);
void emit_pending_reduce(Handle& h, Plan& p);
void emit_labels(Handle& h, Plan& p, const std::vector<LabelProb>& probs);
// bias_grads (optional, one pointer per problem): where the column sums of dlogits go.  Returns true if the
// cross-entropy kernel produces them itself (then the caller needs no separate column-sum pass).
bool emit_xent_and_loss(Handle& h, Plan& p, std::vector<XentProb> probs, const std::vector<int>& chunk_of,
                        const std::vector<float*>* bias_grads = nullptr);
// Cross-entropy whose per-group softmax statistics were left by the head GEMM (EPI_LOGIT_STATS); classes of
// all problems equal.  The column sums of dlogits are queued for bias_grads when it is given.
void emit_xent_from_stats(Handle& h, Plan& p, std::vector<XentStatsProb> probs, const std::vector<int>& chunk_of,
                          const std::vector<float*>* bias_grads);
void emit_optimizer(Handle& h, Plan& p);
OptimArgs optimizer_args(const Handle& h);     // the optimizer sweep of the step about to run
// Causal attention of all problems of a phase in one grouped launch (forward) or two (backward: dQ, then dK and
// dV).  bf16 takes the tcgen05 kernels unless the handle was created with the FP32-ALU backend.
void emit_attention(Handle& h, Plan& p, const std::vector<AttnProb>& probs, bool backward);
// Predictions of the heads' logits (before the cross-entropy overwrites them); runs only under lp_evaluate
void emit_argmax(Handle& h, Plan& p, const std::vector<ArgmaxProb>& probs);

// GEMM problem constructors (x: [M,K] row-major, W: [N,K] row-major, dy: [M,N] row-major)
GemmProb gemm_fwd(const void* x, const void* W, void* y, int M, int N, int Kd, const float* bias, int act);
GemmProb gemm_dgrad(const void* dy, const void* W, void* dx, int M, int N, int Kd, int act, const void* aux);
GemmProb gemm_wgrad(const void* dy, const void* x, float* dW, int M, int N, int Kd);

// ---- per-family builders: register tensors, allocate buffers, build all plans
void build_mlp(Handle& h);
void build_lm(Handle& h);
void build_resnet(Handle& h);

}  // namespace lp
