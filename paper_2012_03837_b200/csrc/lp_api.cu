// C ABI of the local update step (include/lp.h): argument checks, handle life cycle, step
// drivers, parameter access, checkpointing.  No exception leaves this file.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <stdexcept>

#include "runtime.h"
#include "gemm_tc.h"
#include "gemm_desc_check.h"

using namespace lp;

struct lp_handle_s {
  Handle h;
};

static thread_local std::string g_create_error;

namespace {

struct ShapeError : std::runtime_error { using std::runtime_error::runtime_error; };
struct UnsupportedError : std::runtime_error { using std::runtime_error::runtime_error; };

lp_status fail(Handle* h, lp_status code, const std::string& msg) {
  if (h) h->err = msg;
  else g_create_error = msg;
  return code;
}

lp_status check_cuda(Handle* h, const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return LP_OK;
  return fail(h, LP_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

void validate(const lp_model_spec* m, int K, const lp_head_spec* hd, const lp_optim_spec* o) {
  if (K < 1 || K > 1024) throw ShapeError("K must be in [1, 1024]");
  if (m->batch < 1) throw ShapeError("batch must be positive");
  if (m->dtype != LP_FP32 && m->dtype != LP_BF16) throw std::invalid_argument("dtype");
  if (o->kind != LP_OPT_SGDM && o->kind != LP_OPT_ADAM) throw std::invalid_argument("optimizer kind");
  if (hd->classes < 2) throw ShapeError("classes must be at least 2");
  switch (m->family) {
    case LP_FAMILY_MLP: {
      if (hd->kind != LP_HEAD_LINEAR) throw std::invalid_argument("MLP takes LP_HEAD_LINEAR");
      if (!m->layer_widths || !m->layers_per_chunk) throw std::invalid_argument("null layer arrays");
      if (m->d_in < 1 || m->n_layers < 1) throw ShapeError("d_in and n_layers must be positive");
      int tot = 0;
      for (int k = 0; k < K; ++k) {
        if (m->layers_per_chunk[k] < 1) throw ShapeError("every chunk needs at least one layer");
        tot += m->layers_per_chunk[k];
      }
      if (tot != m->n_layers) throw ShapeError("layers_per_chunk does not sum to n_layers");
      for (int i = 0; i < m->n_layers; ++i)
        if (m->layer_widths[i] < 1) throw ShapeError("layer width must be positive");
      break;
    }
    case LP_FAMILY_LM: {
      if (hd->kind != LP_HEAD_LN_LINEAR) throw std::invalid_argument("LM takes LP_HEAD_LN_LINEAR");
      if (!m->blocks_per_chunk) throw std::invalid_argument("null blocks_per_chunk");
      if (m->vocab < 2 || m->seq_len < 1 || m->d_model < 1 || m->n_heads < 1 || m->d_ffn < 1)
        throw ShapeError("LM sizes must be positive");
      if (m->d_model != m->n_heads * 64) throw ShapeError("d_model / n_heads must be 64");
      if (hd->classes != m->vocab) throw ShapeError("LM head classes must equal vocab");
      for (int k = 0; k < K; ++k)
        if (m->blocks_per_chunk[k] < 1) throw ShapeError("every chunk needs at least one block");
      break;
    }
    case LP_FAMILY_RESNET: {
      if (hd->kind != LP_HEAD_GAP_LINEAR && hd->kind != LP_HEAD_BN_RELU_GAP_LINEAR)
        throw std::invalid_argument("RESNET takes LP_HEAD_GAP_LINEAR or LP_HEAD_BN_RELU_GAP_LINEAR");
      if (!m->stage_channels) throw std::invalid_argument("null stage_channels");
      if (m->in_channels < 1 || m->height < 1 || m->width < 1 || m->stem_channels < 1 || m->blocks_per_stage < 1)
        throw ShapeError("RESNET sizes must be positive");
      if ((m->height >> (K - 1)) < 1 || (m->width >> (K - 1)) < 1) throw ShapeError("image too small for K stages");
      if (m->block_kind != LP_BLOCK_BASIC && m->block_kind != LP_BLOCK_BOTTLENECK) throw std::invalid_argument("block_kind");
      for (int k = 0; k < K; ++k) {
        if (m->stage_channels[k] < 1) throw ShapeError("stage_channels must be positive");
        if (m->stage_blocks && m->stage_blocks[k] < 1) throw ShapeError("every stage needs at least one block");
      }
      break;
    }
    default: throw std::invalid_argument("family");
  }
}

// Copy a tensor between host and the arena.
lp_status tensor_io(lp_handle hh, int i, int which, void* host, size_t bytes, void* stream, bool set) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!host) return fail(&h, LP_ERR_INVALID_ARG, "null host pointer");
  if (i < 0 || i >= (int)h.tensors.size()) return fail(&h, LP_ERR_INVALID_ARG, "tensor index out of range");
  const TensorRec& t = h.tensors[i];
  cudaStream_t s = (cudaStream_t)stream;
  void* dev = nullptr;
  size_t es = 4;
  switch (which) {
    case LP_MASTER: dev = h.master + t.off; break;
    case LP_MOMENT1: dev = h.m1 + t.off; break;
    case LP_MOMENT2:
      if (!h.m2) return fail(&h, LP_ERR_STATE, "no second moment for this optimizer");
      dev = h.m2 + t.off; break;
    case LP_GRAD: dev = h.grad + t.off; break;
    case LP_WORKING:
      if (!h.bf16_mode || !t.matrix) return fail(&h, LP_ERR_STATE, "tensor has no bf16 working copy");
      dev = h.working + t.off; es = 2; break;
    default: return fail(&h, LP_ERR_INVALID_ARG, "bad `which`");
  }
  if (bytes != (size_t)t.numel * es) return fail(&h, LP_ERR_SHAPE, "byte count does not match the tensor");
  if (set) {
    cudaMemcpyAsync(dev, host, bytes, cudaMemcpyHostToDevice, s);
    if (which == LP_MASTER && h.bf16_mode && t.matrix) {
      // refresh the working copy: round to nearest even on the host, same rule as the device update
      std::vector<uint16_t> w(t.numel);
      const uint32_t* src = (const uint32_t*)host;
      for (int64_t j = 0; j < t.numel; ++j) {
        uint32_t u = src[j];
        if ((u & 0x7fffffffu) > 0x7f800000u) w[j] = (uint16_t)((u >> 16) | 0x40);
        else w[j] = (uint16_t)((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
      }
      cudaMemcpyAsync(h.working + t.off, w.data(), t.numel * 2, cudaMemcpyHostToDevice, s);
      cudaStreamSynchronize(s);
    }
  } else {
    cudaMemcpyAsync(host, dev, bytes, cudaMemcpyDeviceToHost, s);
  }
  cudaStreamSynchronize(s);
  return check_cuda(&h, set ? "lp_set_tensor" : "lp_get_tensor");
}

lp_status copy_inputs(Handle& h, const void* x, const void* y, cudaMemcpyKind kind, cudaStream_t s) {
  cudaMemcpyAsync(h.x_in, x, h.x_bytes, kind, s);
  if (y) cudaMemcpyAsync(h.y_in, y, h.y_bytes, kind, s);
  return check_cuda(&h, "input copy");
}

// Arena segments for the optimizer's per-chunk mode: one per tensor, in arena order; a tensor's
// alignment padding belongs to it (its gradient there is zero).
void build_segments(Handle& h) {
  std::vector<const TensorRec*> order;
  for (auto& t : h.tensors) order.push_back(&t);
  std::sort(order.begin(), order.end(), [](const TensorRec* a, const TensorRec* b) { return a->off < b->off; });
  std::vector<long long> ends;
  std::vector<int> chunks;
  for (size_t i = 0; i < order.size(); ++i) {
    ends.push_back(i + 1 < order.size() ? (long long)order[i + 1]->off : h.n_total);
    chunks.push_back(order[i]->chunk);
  }
  h.d_seg_end = h.upload(ends);
  h.d_seg_chunk = h.upload(chunks);
  h.n_seg = (int)ends.size();
  h.updates.assign(h.K, 0);
}

// Which chunks take part in this step (Sec. 6: with the idle ramp-up, chunk k waits until the k-th
// pipelined step after a reset has brought it an activation), and the per-chunk optimizer table when
// the chunks' step counts differ.  Returns true if some chunk idles.
bool prepare_chunks(Handle& h, int schedule, cudaStream_t s, std::vector<char>& active) {
  const int K = h.K;
  active.assign(K, 1);
  bool any_idle = false, differ = false;
  if (schedule == LP_PIPELINED && h.ramp == LP_RAMP_IDLE)
    for (int k = 0; k < K; ++k)
      if (k > h.pipe_steps) { active[k] = 0; any_idle = true; }
  if (schedule == LP_PIPELINED)
    for (int k = 0; k < h.drain_first && k < K; ++k) { active[k] = 0; any_idle = true; }
  for (int k = 1; k < K; ++k) differ |= h.updates[k] != h.updates[0];
  h.per_chunk_counts = any_idle || differ;
  if (h.per_chunk_counts || h.spec.family == LP_FAMILY_RESNET) {   // BatchNorm reads the active flags every step
    std::vector<float4> tab(K);
    for (int k = 0; k < K; ++k) {
      const double t = (double)(h.updates[k] + 1);
      tab[k] = make_float4(active[k] ? 1.f : 0.f, (float)(1.0 - pow((double)h.opt.beta1, t)),
                           (float)(1.0 - pow((double)h.opt.beta2, t)), 0.f);
    }
    // pageable source: the runtime stages it before the call returns, so the vector may go out of scope
    cudaMemcpyAsync(h.d_chunk_tab, tab.data(), sizeof(float4) * K, cudaMemcpyHostToDevice, s);
  }
  return any_idle;
}

// Whether this step runs as the single cooperative launch (small fp32 MLP), and whether that launch may read
// the caller's device buffers in place (not when a priming pass, which reads the handle's own, comes first).
bool step_is_fused(const Handle& h) { return h.use_fused && h.fused_blocks > 0 && !h.overlap; }
bool step_reads_in_place(const Handle& h, int schedule) {
  return step_is_fused(h) && !(schedule == LP_PIPELINED && !h.primed && h.ramp == LP_RAMP_PRIME);
}

int run_fused(Handle& h, const Handle::FusedProgram& fp, const RunCtx& c) {
  FusedArgs a = fp.args;
  a.opt = optimizer_args(h);
  a.x = c.x ? c.x : h.x_in;
  a.y = c.y ? c.y : h.y_in;
  ProfRecord r{KIND_GEMM_ALU, 1, fp.flops, nullptr, nullptr};
  if (c.prof) {
    cudaEventCreate(&r.e0);
    cudaEventCreate(&r.e1);
    cudaEventRecord(r.e0, c.stream);
  }
  const bool launched = launch_fused_mlp_step(a, h.fused_blocks, c.stream) == cudaSuccess;
  if (!launched) cudaGetLastError();          // the device cannot hold the cooperative grid right now
  if (c.prof) {
    cudaEventRecord(r.e1, c.stream);
    c.prof->push_back(r);
  }
  return launched ? 1 : 0;
}

lp_status run_step(Handle& h, int schedule, cudaStream_t s, const void* x = nullptr, const int* y = nullptr) {
  RunCtx ctx{s, nullptr, h.profiling ? &h.prof : nullptr};
  const bool fused = step_is_fused(h);
  if (x && step_reads_in_place(h, schedule)) { ctx.x = x; ctx.y = y; }
  int launches = 0;
  std::vector<char> active;
  const bool any_idle = prepare_chunks(h, schedule, s, active);
  if (schedule == LP_SYNC) {
    if (h.primed) return fail(&h, LP_ERR_STATE, "a pipeline is in flight: call lp_reset_pipeline before a synchronous step");
    if (fused) launches = run_fused(h, h.fused_sync, ctx);
    if (fused && launches == 0) {               // refused: the grouped launches do the same step
      if (ctx.x) { copy_inputs(h, ctx.x, ctx.y, cudaMemcpyDeviceToDevice, s); ctx.x = nullptr; ctx.y = nullptr; }
      h.sync_plan.run(ctx);
      launches = h.sync_plan.launches;
    } else if (!fused) {
      const Plan& plan = h.overlap ? h.sync_overlap_plan : h.sync_plan;
      plan.run(ctx);
      launches = plan.launches;
    }
    h.last_wr = 0;
  } else {
    if (!h.primed && h.ramp == LP_RAMP_PRIME) {
      h.prime_plan[h.parity].run(ctx);
      launches += h.prime_plan[h.parity].launches;
    }
    h.primed = true;
    // Idle chunks run through the plan as well, on whatever their boundary buffer holds (finite values:
    // zeros after lp_create); the optimizer leaves their parameters alone, their losses read NaN, and
    // what they publish is overwritten before an active chunk reads it.
    int fused_done = 0;
    if (fused) fused_done = run_fused(h, h.fused_pipe[h.parity], ctx);   // masks the idle chunks' losses itself
    launches += fused_done;
    if (fused && fused_done == 0 && ctx.x) { copy_inputs(h, ctx.x, ctx.y, cudaMemcpyDeviceToDevice, s); ctx.x = nullptr; ctx.y = nullptr; }
    if (!fused || fused_done == 0) {
      h.pipe_plan[h.parity].run(ctx);
      launches += h.pipe_plan[h.parity].launches;
      if (any_idle) { launch_mask_losses(h.d_losses, h.d_chunk_tab, h.K, s); launches += 1; }
    }
    h.last_wr = 1 - h.parity;
    h.parity ^= 1;
    h.pipe_steps += 1;
  }
  for (int k = 0; k < h.K; ++k) h.updates[k] += active[k] ? 1 : 0;
  h.step_count += 1;
  h.last_launches = launches;
  return check_cuda(&h, "lp_step launch");
}

}  // namespace

extern "C" {

lp_status lp_create(const lp_model_spec* model, int K, const lp_head_spec* head, const lp_optim_spec* optim,
                    const lp_alloc* alloc, lp_handle* out) {
  if (out) *out = nullptr;
  if (!model || !head || !optim || !out) return fail(nullptr, LP_ERR_INVALID_ARG, "null argument");
  if (alloc && (!alloc->alloc || !alloc->release)) return fail(nullptr, LP_ERR_INVALID_ARG, "allocator needs both callbacks");
  lp_handle hh = nullptr;
  try {
    validate(model, K, head, optim);
    int dev_count = 0;
    if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count == 0) {
      cudaGetLastError();
      return fail(nullptr, LP_ERR_CUDA, "no CUDA device available");
    }
    hh = new lp_handle_s();
    Handle& h = hh->h;
    h.spec = *model;
    h.head = *head;
    h.opt = *optim;
    h.K = K;
    h.bf16_mode = model->dtype == LP_BF16;
    h.force_simt = model->gemm_backend == 1 || !h.bf16_mode;
    if (alloc) { h.alloc = *alloc; h.use_cuda_malloc = false; }
    {
      int dev = 0;
      cudaGetDevice(&dev);
      cudaDeviceGetAttribute(&h.num_sms, cudaDevAttrMultiProcessorCount, dev);
    }
    h.d_losses = (float*)h.dalloc(sizeof(float) * K);
    h.d_status = (int*)h.dalloc(sizeof(int));
    h.d_chunk_tab = (float4*)h.dalloc(sizeof(float4) * K);
    switch (model->family) {
      case LP_FAMILY_MLP:
        h.layer_widths.assign(model->layer_widths, model->layer_widths + model->n_layers);
        h.per_chunk.assign(model->layers_per_chunk, model->layers_per_chunk + K);
        h.spec.layer_widths = nullptr; h.spec.layers_per_chunk = nullptr;
        build_mlp(h);
        break;
      case LP_FAMILY_LM:
        h.per_chunk.assign(model->blocks_per_chunk, model->blocks_per_chunk + K);
        h.spec.blocks_per_chunk = nullptr;
        build_lm(h);
        break;
      default:
        h.stage_channels.assign(model->stage_channels, model->stage_channels + K);
        h.spec.stage_channels = nullptr;
        for (int k = 0; k < K; ++k) h.stage_blocks.push_back(model->stage_blocks ? model->stage_blocks[k] : model->blocks_per_stage);
        h.spec.stage_blocks = nullptr;
        build_resnet(h);
        break;
    }
    build_segments(h);
    cudaDeviceSynchronize();
    lp_status st = check_cuda(nullptr, "lp_create");
    if (st != LP_OK) { lp_destroy(hh); return st; }
    *out = hh;
    return LP_OK;
  } catch (const ShapeError& e) {
    if (hh) lp_destroy(hh);
    return fail(nullptr, LP_ERR_SHAPE, e.what());
  } catch (const UnsupportedError& e) {
    if (hh) lp_destroy(hh);
    return fail(nullptr, LP_ERR_UNSUPPORTED, e.what());
  } catch (const std::invalid_argument& e) {
    if (hh) lp_destroy(hh);
    return fail(nullptr, LP_ERR_INVALID_ARG, e.what());
  } catch (const std::bad_alloc&) {
    if (hh) lp_destroy(hh);
    return fail(nullptr, LP_ERR_ALLOC, "host allocation failed");
  } catch (const std::exception& e) {
    std::string m = e.what();
    if (hh) lp_destroy(hh);
    lp_status code = m.rfind("alloc:", 0) == 0 ? LP_ERR_ALLOC
                     : m.rfind("unsupported:", 0) == 0 ? LP_ERR_UNSUPPORTED
                     : m.rfind("shape:", 0) == 0 ? LP_ERR_SHAPE : LP_ERR_CUDA;
    return fail(nullptr, code, m);
  }
}

lp_status lp_destroy(lp_handle hh) {
  if (!hh) return LP_OK;
  Handle& h = hh->h;
  cudaDeviceSynchronize();
  for (void* p : h.blocks) {
    if (h.use_cuda_malloc) cudaFree(p);
    else h.alloc.release(p, h.alloc.user);
  }
  cudaGetLastError();
  delete hh;
  return LP_OK;
}

lp_status lp_step(lp_handle hh, const void* x, const void* y, int schedule, void* stream, float* out_losses) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!x || !y || !out_losses) return fail(&h, LP_ERR_INVALID_ARG, "null pointer");
  if (schedule != LP_SYNC && schedule != LP_PIPELINED) return fail(&h, LP_ERR_INVALID_ARG, "bad schedule");
  if (schedule == LP_SYNC && h.primed) return fail(&h, LP_ERR_STATE, "a pipeline is in flight: call lp_reset_pipeline before a synchronous step");
  if (schedule == LP_PIPELINED && h.overlap) return fail(&h, LP_ERR_UNSUPPORTED, "overlapping updates take both gradients of a shared layer from one minibatch: synchronous schedule only");
  cudaStream_t s = (cudaStream_t)stream;
  lp_status st = LP_OK;
  if (step_reads_in_place(h, schedule)) {
    st = run_step(h, schedule, s, x, (const int*)y);
  } else {
    st = copy_inputs(h, x, y, cudaMemcpyDeviceToDevice, s);
    if (st != LP_OK) return st;
    st = run_step(h, schedule, s);
  }
  if (st != LP_OK) return st;
  cudaMemcpyAsync(out_losses, h.d_losses, sizeof(float) * h.K, cudaMemcpyDeviceToDevice, s);
  return check_cuda(&h, "lp_step");
}

lp_status lp_step_host(lp_handle hh, const void* x_host, const void* y_host, int schedule, void* stream,
                       float* out_losses_host) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!x_host || !y_host || !out_losses_host) return fail(&h, LP_ERR_INVALID_ARG, "null pointer");
  if (schedule != LP_SYNC && schedule != LP_PIPELINED) return fail(&h, LP_ERR_INVALID_ARG, "bad schedule");
  if (schedule == LP_SYNC && h.primed) return fail(&h, LP_ERR_STATE, "a pipeline is in flight: call lp_reset_pipeline before a synchronous step");
  if (schedule == LP_PIPELINED && h.overlap) return fail(&h, LP_ERR_UNSUPPORTED, "overlapping updates take both gradients of a shared layer from one minibatch: synchronous schedule only");
  cudaStream_t s = (cudaStream_t)stream;
  lp_status st = copy_inputs(h, x_host, y_host, cudaMemcpyHostToDevice, s);
  if (st != LP_OK) return st;
  st = run_step(h, schedule, s);
  if (st != LP_OK) return st;
  cudaMemcpyAsync(out_losses_host, h.d_losses, sizeof(float) * h.K, cudaMemcpyDeviceToHost, s);
  cudaStreamSynchronize(s);
  return check_cuda(&h, "lp_step_host");
}

lp_status lp_forward(lp_handle hh, const void* x, const void* y, void* stream, void* out_logits, float* out_losses) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!x) return fail(&h, LP_ERR_INVALID_ARG, "null x");
  if (!y && out_losses) return fail(&h, LP_ERR_INVALID_ARG, "losses need labels");
  cudaStream_t s = (cudaStream_t)stream;
  lp_status st = copy_inputs(h, x, y, cudaMemcpyDeviceToDevice, s);
  if (st != LP_OK) return st;
  if (!y) cudaMemsetAsync(h.y_in, 0xff, h.y_bytes, s);   // all labels -1: no row is valid
  RunCtx ctx{s, out_logits};
  int half = h.primed ? h.parity ^ 1 : 0;                 // the half no chunk will read next step
  h.fwd_plan[half].run(ctx);
  if (out_losses) cudaMemcpyAsync(out_losses, h.d_losses, sizeof(float) * h.K, cudaMemcpyDeviceToDevice, s);
  if (!y) cudaMemsetAsync(h.d_status, 0, sizeof(int), s); // the unlabeled pass yields NaN losses by design
  return check_cuda(&h, "lp_forward");
}

lp_status lp_evaluate(lp_handle hh, const void* x, const void* y, void* stream, int bn_mode, float* out_losses,
                      int* out_correct, int* out_pred) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!x || !y) return fail(&h, LP_ERR_INVALID_ARG, "null x or y");
  if (!out_losses && !out_correct && !out_pred) return fail(&h, LP_ERR_INVALID_ARG, "no output requested");
  if (bn_mode != LP_BN_BATCH && bn_mode != LP_BN_RUNNING) return fail(&h, LP_ERR_INVALID_ARG, "bad bn_mode");
  cudaStream_t s = (cudaStream_t)stream;
  lp_status st = copy_inputs(h, x, y, cudaMemcpyDeviceToDevice, s);
  if (st != LP_OK) return st;
  if (out_correct) cudaMemsetAsync(out_correct, 0, sizeof(int) * h.K, s);
  RunCtx ctx{s, nullptr, nullptr};
  ctx.out_pred = out_pred;
  ctx.out_correct = out_correct;
  int half = h.primed ? h.parity ^ 1 : 0;                 // the half no chunk will read next step
  if (bn_mode == LP_BN_RUNNING && h.has_eval_plan) h.eval_plan[half].run(ctx);
  else h.fwd_plan[half].run(ctx);
  if (out_losses) cudaMemcpyAsync(out_losses, h.d_losses, sizeof(float) * h.K, cudaMemcpyDeviceToDevice, s);
  return check_cuda(&h, "lp_evaluate");
}

int lp_num_tensors(lp_handle hh) { return hh ? (int)hh->h.tensors.size() : 0; }

lp_status lp_tensor_info_get(lp_handle hh, int i, lp_tensor_info* out) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!out || i < 0 || i >= (int)h.tensors.size()) return fail(&h, LP_ERR_INVALID_ARG, "bad tensor index or null output");
  const TensorRec& t = h.tensors[i];
  memset(out, 0, sizeof(*out));
  strncpy(out->name, t.name.c_str(), sizeof(out->name) - 1);
  out->chunk = t.chunk;
  out->ndim = (int)t.shape.size();
  for (size_t j = 0; j < t.shape.size() && j < 4; ++j) out->shape[j] = t.shape[j];
  out->numel = t.numel;
  out->has_working_bf16 = (h.bf16_mode && t.matrix) ? 1 : 0;
  return LP_OK;
}

lp_status lp_get_tensor(lp_handle hh, int i, int which, void* host_dst, size_t bytes, void* stream) {
  return tensor_io(hh, i, which, host_dst, bytes, stream, false);
}
lp_status lp_set_tensor(lp_handle hh, int i, int which, const void* host_src, size_t bytes, void* stream) {
  return tensor_io(hh, i, which, const_cast<void*>(host_src), bytes, stream, true);
}

lp_status lp_reset_pipeline(lp_handle hh) {
  if (!hh) return LP_ERR_INVALID_ARG;
  hh->h.primed = false;
  hh->h.parity = 0;
  hh->h.pipe_steps = 0;
  hh->h.drain_first = 0;
  return LP_OK;
}

size_t lp_chunk_output_bytes(lp_handle hh, int k) {
  if (!hh || k < 0 || k >= hh->h.K) return 0;
  return hh->h.bnd_bytes[k];
}

lp_status lp_chunk_output(lp_handle hh, int k, void* dst, size_t bytes, void* stream) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!dst || k < 0 || k >= h.K) return fail(&h, LP_ERR_INVALID_ARG, "lp_chunk_output: null destination or chunk index out of range");
  if (bytes < h.bnd_bytes[k]) return fail(&h, LP_ERR_INVALID_ARG, "lp_chunk_output: destination smaller than lp_chunk_output_bytes");
  if (h.last_wr < 0) return fail(&h, LP_ERR_STATE, "lp_chunk_output: no training step has run yet");
  cudaMemcpyAsync(dst, h.bnd[h.last_wr][k], h.bnd_bytes[k], cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  return check_cuda(&h, "lp_chunk_output");
}

lp_status lp_set_overlap(lp_handle hh, int on) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (on && !h.has_overlap_plan)
    return fail(&h, LP_ERR_UNSUPPORTED, "overlapping updates need at least two chunks");
  h.overlap = on != 0;
  return LP_OK;
}

lp_status lp_set_drain(lp_handle hh, int idle_first) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (idle_first < 0 || idle_first > h.K) return fail(&h, LP_ERR_INVALID_ARG, "lp_set_drain: idle_first outside [0, K]");
  h.drain_first = idle_first;
  return LP_OK;
}

lp_status lp_set_fused_step(lp_handle hh, int on) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (on && h.fused_blocks <= 0) return fail(&h, LP_ERR_UNSUPPORTED, "lp_set_fused_step: this handle has no single-launch form of the step");
  h.use_fused = on != 0;
  return LP_OK;
}

lp_status lp_set_ramp(lp_handle hh, int ramp) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (ramp != LP_RAMP_PRIME && ramp != LP_RAMP_IDLE) return fail(&h, LP_ERR_INVALID_ARG, "bad ramp mode");
  if (h.primed) return fail(&h, LP_ERR_STATE, "a pipeline is in flight: call lp_reset_pipeline before changing the ramp-up");
  h.ramp = ramp;
  return LP_OK;
}

lp_status lp_status_poll(lp_handle hh, void* stream) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  cudaStream_t s = (cudaStream_t)stream;
  int w = 0;
  cudaMemcpyAsync(&w, h.d_status, sizeof(int), cudaMemcpyDeviceToHost, s);
  cudaMemsetAsync(h.d_status, 0, sizeof(int), s);
  cudaStreamSynchronize(s);
  lp_status st = check_cuda(&h, "lp_status_poll");
  if (st != LP_OK) return st;
  if (w & ST_TIMEOUT) return fail(&h, LP_ERR_TIMEOUT, "a device-side wait gave up");
  if (w & ST_LABEL_RANGE) return fail(&h, LP_ERR_LABEL_RANGE, "a label or token id was out of range");
  if (w & ST_NONFINITE) return fail(&h, LP_ERR_NONFINITE, "a loss was not finite");
  return LP_OK;
}

// Checkpoint layout: header {magic, n_total, K, step_count, parity, primed, ramp, pipe_steps}, the K per-chunk
// update counts, master, m1, [m2], then for each half and chunk: boundary activation, labels.
struct StateHeader {
  uint64_t magic; int64_t n_total; int64_t K; int64_t step_count; int64_t parity; int64_t primed;
  int64_t ramp; int64_t pipe_steps;
};
static const uint64_t kMagic = 0x4c50535441544532ull;

size_t lp_state_size(lp_handle hh) {
  if (!hh) return 0;
  Handle& h = hh->h;
  size_t n = sizeof(StateHeader) + sizeof(int64_t) * h.K + (size_t)h.n_total * 4 * (h.m2 ? 3 : 2);
  for (int s = 0; s < 2; ++s)
    for (int k = 0; k < h.K; ++k) n += h.bnd_bytes[k] + h.y_bytes;
  return n;
}

static lp_status state_io(lp_handle hh, void* host, size_t bytes, bool save) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!host) return fail(&h, LP_ERR_INVALID_ARG, "null host pointer");
  if (bytes != lp_state_size(hh)) return fail(&h, LP_ERR_SHAPE, "state size mismatch");
  cudaDeviceSynchronize();
  char* p = (char*)host;
  StateHeader hd{kMagic, h.n_total, h.K, h.step_count, h.parity, h.primed ? 1 : 0, h.ramp, h.pipe_steps};
  if (save) memcpy(p, &hd, sizeof(hd));
  else {
    memcpy(&hd, p, sizeof(hd));
    if (hd.magic != kMagic || hd.n_total != h.n_total || hd.K != h.K) return fail(&h, LP_ERR_STATE, "state blob does not match this handle");
    h.step_count = hd.step_count; h.parity = (int)hd.parity; h.primed = hd.primed != 0;
    h.last_wr = h.step_count == 0 ? -1 : (h.primed ? h.parity : 0);
    h.ramp = (int)hd.ramp; h.pipe_steps = hd.pipe_steps;
  }
  p += sizeof(hd);
  for (int k = 0; k < h.K; ++k) {
    int64_t u = h.updates[k];
    if (save) memcpy(p, &u, sizeof(u));
    else { memcpy(&u, p, sizeof(u)); h.updates[k] = u; }
    p += sizeof(u);
  }
  auto io = [&](void* dev, size_t n) {
    if (save) cudaMemcpy(p, dev, n, cudaMemcpyDeviceToHost);
    else cudaMemcpy(dev, p, n, cudaMemcpyHostToDevice);
    p += n;
  };
  io(h.master, (size_t)h.n_total * 4);
  io(h.m1, (size_t)h.n_total * 4);
  if (h.m2) io(h.m2, (size_t)h.n_total * 4);
  for (int s = 0; s < 2; ++s)
    for (int k = 0; k < h.K; ++k) { io(h.bnd[s][k], h.bnd_bytes[k]); io(h.lab[s][k], h.y_bytes); }
  if (!save && h.bf16_mode) {
    // working copies follow the restored masters: one optimizer-free refresh on the host side
    std::vector<float> m((size_t)h.n_matrix);
    cudaMemcpy(m.data(), h.master, (size_t)h.n_matrix * 4, cudaMemcpyDeviceToHost);
    std::vector<uint16_t> w((size_t)h.n_matrix);
    for (long long j = 0; j < h.n_matrix; ++j) {
      uint32_t u; memcpy(&u, &m[j], 4);
      w[j] = ((u & 0x7fffffffu) > 0x7f800000u) ? (uint16_t)((u >> 16) | 0x40) : (uint16_t)((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
    }
    cudaMemcpy(h.working, w.data(), (size_t)h.n_matrix * 2, cudaMemcpyHostToDevice);
  }
  return check_cuda(&h, save ? "lp_save_state" : "lp_load_state");
}

lp_status lp_save_state(lp_handle hh, void* host_dst, size_t bytes) { return state_io(hh, host_dst, bytes, true); }
lp_status lp_load_state(lp_handle hh, const void* host_src, size_t bytes) { return state_io(hh, const_cast<void*>(host_src), bytes, false); }

lp_status lp_gemm_bf16(int n, const lp_gemm_desc* in, int backend, void* stream, int* used_tc) {
  if (n < 1 || !in) return fail(nullptr, LP_ERR_INVALID_ARG, "lp_gemm_bf16: no problems");
  if (backend != 0 && backend != 1) return fail(nullptr, LP_ERR_INVALID_ARG, "lp_gemm_bf16: backend must be 0 or 1");
  for (int i = 0; i < n; ++i)
    if (const char* why = gemm_desc_problem(in[i]))
      return fail(nullptr, LP_ERR_INVALID_ARG, "lp_gemm_bf16: problem " + std::to_string(i) + ": " + why);
  cudaStream_t s = (cudaStream_t)stream;
  // the scratch of this entry belongs to the device that was current at its first call
  static int* d_status = nullptr;
  static int num_sms = 0;
  static int first_dev = -1;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return fail(nullptr, LP_ERR_CUDA, "lp_gemm_bf16: no CUDA device"); }
    if (first_dev >= 0 && dev != first_dev)
      return fail(nullptr, LP_ERR_UNSUPPORTED, "lp_gemm_bf16: one device per process (the first one it was called on)");
    if (!d_status) {
      if (cudaMalloc(&d_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return fail(nullptr, LP_ERR_ALLOC, "status word"); }
      cudaMemset(d_status, 0, sizeof(int));
      cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
      first_dev = dev;
    }
  }
  std::vector<GemmProb> tc, simt;
  for (int i = 0; i < n; ++i) {
    const lp_gemm_desc& q = in[i];
    GemmProb g{};
    g.A = q.A; g.B = q.B; g.C = q.C; g.C2 = q.C2; g.bias = q.bias; g.resid = q.resid; g.aux = q.aux;
    g.M = q.M; g.N = q.N; g.K = q.K; g.a_ms = q.a_ms; g.a_ks = q.a_ks; g.b_ns = q.b_ns; g.b_ks = q.b_ks;
    g.ldc = q.ldc; g.act = q.act; g.out_f32 = q.out_f32;
    if (backend == 0 && gemm_tc_eligible(g)) tc.push_back(g);
    else simt.push_back(g);
  }
  if (used_tc) *used_tc = (int)tc.size();
  // descriptor tables live in a per-process scratch buffer that grows on demand
  static void* d_tab = nullptr;
  static size_t d_cap = 0;
  struct alignas(64) Map { unsigned char b[128]; };
  size_t need = 1024 + tc.size() * sizeof(GemmProb) + 256 + 4 * tc.size() * sizeof(Map) + simt.size() * sizeof(GemmProb) + 256;
  if (need > d_cap) {
    cudaStreamSynchronize(s);
    if (d_tab) cudaFree(d_tab);
    if (cudaMalloc(&d_tab, need * 2) != cudaSuccess) { cudaGetLastError(); d_tab = nullptr; d_cap = 0; return fail(nullptr, LP_ERR_ALLOC, "descriptor table"); }
    d_cap = need * 2;
  }
  char* cur = (char*)d_tab;
  auto take = [&](size_t bytes) { char* r = cur; cur += (bytes + 255) / 256 * 256; return r; };
  std::vector<GemmProb> lists[2];                       // [1]: long reductions that take the wide tiles
  for (auto& g : tc) lists[gemm_tc_wide_ok(g) ? 1 : 0].push_back(g);
  for (int wide = 0; wide < 2; ++wide) {
    std::vector<GemmProb>& list = lists[wide];
    if (list.empty()) continue;
    int total = 0;
    const int cg = wide ? 2 : gemm_tc_choose_cg(list.data(), (int)list.size());
    for (auto& g : list) total += gemm_tc_tiles(g, total, cg, wide);
    std::vector<Map> maps(4 * list.size());
    for (size_t i = 0; i < list.size(); ++i)
      if (!gemm_tc_encode(list[i], &maps[4 * i], cg)) return fail(nullptr, LP_ERR_CUDA, "cuTensorMapEncodeTiled failed");
    GemmProb* dp = (GemmProb*)take(list.size() * sizeof(GemmProb));
    Map* dm = (Map*)take(maps.size() * sizeof(Map));
    cudaMemcpyAsync(dp, list.data(), list.size() * sizeof(GemmProb), cudaMemcpyHostToDevice, s);
    cudaMemcpyAsync(dm, maps.data(), maps.size() * sizeof(Map), cudaMemcpyHostToDevice, s);
    cudaStreamSynchronize(s);
    launch_gemm_tc(dp, dm, (int)list.size(), total, d_status, num_sms, s, cg, wide);
  }
  if (!simt.empty()) {
    int t = 0;
    for (auto& g : simt) { g.tiles_n = (g.N + 63) / 64; g.tile_start = t; t += ((g.M + 63) / 64) * g.tiles_n; }
    GemmProb* dp = (GemmProb*)take(simt.size() * sizeof(GemmProb));
    cudaMemcpyAsync(dp, simt.data(), simt.size() * sizeof(GemmProb), cudaMemcpyHostToDevice, s);
    cudaStreamSynchronize(s);
    launch_gemm_simt(dp, simt.data(), (int)simt.size(), true, s);
  }
  return check_cuda(nullptr, "lp_gemm_bf16");
}

lp_status lp_conv3x3_bf16(int form, const void* act, const void* other, void* out, int n, int hgt, int wid, int c_in,
                          int c_out, void* stream) {
  return lp_conv2d_bf16(form, act, other, out, n, hgt, wid, c_in, c_out, 3, 1, stream);
}

lp_status lp_conv2d_bf16(int form, const void* act, const void* other, void* out, int n, int hgt, int wid, int c_in,
                         int c_out, int ksize, int stride, void* stream) {
  if (!act || !other || !out) return fail(nullptr, LP_ERR_INVALID_ARG, "lp_conv2d_bf16: null pointer");
  if (n < 1 || hgt < 1 || wid < 1 || c_in < 1 || c_out < 1) return fail(nullptr, LP_ERR_SHAPE, "lp_conv2d_bf16: sizes must be positive");
  if ((ksize != 3 && ksize != 1) || (stride != 1 && stride != 2))
    return fail(nullptr, LP_ERR_UNSUPPORTED, "lp_conv2d_bf16: 3x3 (padding 1) or 1x1 filters, stride 1 or 2");
  const int ho = (hgt - 1) / stride + 1, wo = (wid - 1) / stride + 1, taps = ksize * ksize;
  const long long pixels = (long long)n * ho * wo;
  if ((long long)n * hgt * wid > 0x7fffffffLL) return fail(nullptr, LP_ERR_SHAPE, "lp_conv2d_bf16: too many pixels");
  GemmProb g{};
  g.conv_n = n; g.conv_h = ho; g.conv_w = wo; g.conv_hin = hgt; g.conv_win = wid; g.conv_stride = stride; g.conv_taps = taps;
  switch (form) {
    case LP_CONV_FORWARD:        // act = x [n,h,w,c_in], other = filters [c_out,k,k,c_in], out = y [n,ho,wo,c_out]
      g.A = act; g.B = other; g.C = out; g.M = (int)pixels; g.N = c_out; g.K = taps * c_in;
      g.a_ms = c_in; g.a_ks = 1; g.b_ns = (long long)taps * c_in; g.b_ks = 1; g.ldc = c_out;
      g.conv = CONV_FWD; g.conv_c = c_in;
      break;
    case LP_CONV_INPUT_GRAD:     // act = dy [n,h,w,c_out], other = filters, out = dx [n,h,w,c_in]
      if (ksize != 3 || stride != 1) return fail(nullptr, LP_ERR_UNSUPPORTED, "lp_conv2d_bf16: the input gradient exists for 3x3, stride 1");
      g.A = act; g.B = other; g.C = out; g.M = (int)pixels; g.N = c_in; g.K = 9 * c_out;
      g.a_ms = c_out; g.a_ks = 1; g.b_ns = 1; g.b_ks = 9LL * c_in; g.ldc = c_in;
      g.conv = CONV_DGRAD; g.conv_c = c_out;
      break;
    case LP_CONV_FILTER_GRAD:    // act = x [n,h,w,c_in], other = dy [n,ho,wo,c_out], out = dW [c_out,k,k,c_in] fp32
      g.A = other; g.B = act; g.C = out; g.M = c_out; g.N = taps * c_in; g.K = (int)pixels;
      g.a_ms = 1; g.a_ks = c_out; g.b_ns = 1; g.b_ks = c_in; g.ldc = taps * c_in; g.out_f32 = 1;
      g.conv = CONV_WGRAD; g.conv_c = c_in;
      break;
    default: return fail(nullptr, LP_ERR_INVALID_ARG, "lp_conv2d_bf16: unknown form");
  }
  if (!gemm_tc_eligible(g))
    return fail(nullptr, LP_ERR_UNSUPPORTED, "lp_conv2d_bf16: needs 16-byte aligned tensors, the shifted operand's channels a multiple of 64, "
                                             "the other channel count a multiple of 8, an output width dividing 64 and output h*w dividing or "
                                             "divisible by 128");
  cudaStream_t s = (cudaStream_t)stream;
  static int* d_status = nullptr;
  static void* d_tab = nullptr;
  static int num_sms = 0;
  struct alignas(64) Map { unsigned char b[128]; };
  static int first_dev = -1;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return fail(nullptr, LP_ERR_CUDA, "lp_conv2d_bf16: no CUDA device"); }
  if (first_dev >= 0 && dev != first_dev)
    return fail(nullptr, LP_ERR_UNSUPPORTED, "lp_conv2d_bf16: one device per process (the first one it was called on)");
  if (!d_tab) {
    if (cudaMalloc(&d_tab, 1024 + 4 * sizeof(Map)) != cudaSuccess) { cudaGetLastError(); d_tab = nullptr; return fail(nullptr, LP_ERR_ALLOC, "descriptor table"); }
    d_status = (int*)d_tab;
    cudaMemset(d_status, 0, sizeof(int));
    cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
    first_dev = dev;
  }
  const int cg = gemm_tc_choose_cg(&g, 1);
  const int total = gemm_tc_tiles(g, 0, cg);
  Map maps[4];
  if (!gemm_tc_encode(g, maps, cg)) return fail(nullptr, LP_ERR_CUDA, "cuTensorMapEncodeTiled failed");
  GemmProb* dp = (GemmProb*)((char*)d_tab + 256);
  Map* dm = (Map*)((char*)d_tab + 1024);
  cudaMemcpyAsync(dp, &g, sizeof(GemmProb), cudaMemcpyHostToDevice, s);
  cudaMemcpyAsync(dm, maps, sizeof(maps), cudaMemcpyHostToDevice, s);
  cudaStreamSynchronize(s);                      // the tables above are host stack memory
  launch_gemm_tc(dp, dm, 1, total, d_status, num_sms, s, cg);
  return check_cuda(nullptr, "lp_conv2d_bf16");
}

lp_status lp_attention_bf16(int form, const void* qkv, void* o, float* lse, const void* dout, void* dqkv, float* delta,
                            int batch, int seq_len, int n_heads, void* stream) {
  if (form != LP_ATTN_FORWARD && form != LP_ATTN_BACKWARD) return fail(nullptr, LP_ERR_INVALID_ARG, "lp_attention_bf16: unknown form");
  if (!qkv || !o || !lse || (form == LP_ATTN_BACKWARD && (!dout || !dqkv || !delta)))
    return fail(nullptr, LP_ERR_INVALID_ARG, "lp_attention_bf16: null pointer");
  if (batch < 1 || seq_len < 1 || n_heads < 1 || (long long)batch * seq_len > 0x7fffffffLL / (192LL * n_heads))
    return fail(nullptr, LP_ERR_SHAPE, "lp_attention_bf16: sizes must be positive (and batch*seq_len*3*d below 2^31)");
  cudaStream_t s = (cudaStream_t)stream;
  static void* d_tab = nullptr;                  // status word at 0, the problem at 256
  static int first_dev = -1;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return fail(nullptr, LP_ERR_CUDA, "lp_attention_bf16: no CUDA device"); }
  if (first_dev >= 0 && dev != first_dev)
    return fail(nullptr, LP_ERR_UNSUPPORTED, "lp_attention_bf16: one device per process (the first one it was called on)");
  AttnTcProb tab;
  AttnProb ap{qkv, o, lse, form == LP_ATTN_BACKWARD ? dout : nullptr, dqkv, delta, batch, seq_len, n_heads};
  if (((uintptr_t)o & 15) || ((uintptr_t)dqkv & 15) || !attn_tc_encode(tab, ap))
    return fail(nullptr, LP_ERR_UNSUPPORTED, "lp_attention_bf16: tensors must be 16-byte aligned");
  if (!d_tab) {
    if (cudaMalloc(&d_tab, 256 + sizeof(AttnTcProb)) != cudaSuccess) { cudaGetLastError(); d_tab = nullptr; return fail(nullptr, LP_ERR_ALLOC, "descriptor table"); }
    cudaMemset(d_tab, 0, 256);
    first_dev = dev;
  }
  int* d_status = (int*)d_tab;
  AttnTcProb* dp = (AttnTcProb*)((char*)d_tab + 256);
  cudaMemcpyAsync(dp, &tab, sizeof(tab), cudaMemcpyHostToDevice, s);
  cudaStreamSynchronize(s);                      // the table above is host stack memory
  cudaError_t e = form == LP_ATTN_FORWARD ? launch_attn_fwd_tc(dp, 1, batch, seq_len, n_heads, d_status, s)
                                          : launch_attn_bwd_tc(dp, 1, batch, seq_len, n_heads, d_status, s);
  if (e != cudaSuccess) return fail(nullptr, LP_ERR_CUDA, std::string("lp_attention_bf16: launch: ") + cudaGetErrorString(e));
  int w = 0;
  cudaMemcpyAsync(&w, d_status, sizeof(int), cudaMemcpyDeviceToHost, s);
  cudaMemsetAsync(d_status, 0, sizeof(int), s);
  cudaStreamSynchronize(s);
  lp_status st = check_cuda(nullptr, "lp_attention_bf16");
  if (st != LP_OK) return st;
  if (w & ST_TIMEOUT) return fail(nullptr, LP_ERR_TIMEOUT, "lp_attention_bf16: a device-side wait gave up");
  return LP_OK;
}

lp_status lp_profile_enable(lp_handle hh, int on) {
  if (!hh) return LP_ERR_INVALID_ARG;
  hh->h.profiling = on != 0;
  return LP_OK;
}

lp_status lp_profile_read(lp_handle hh, double* ms, double* work, int* launches) {
  if (!hh) return LP_ERR_INVALID_ARG;
  Handle& h = hh->h;
  if (!ms || !work || !launches) return fail(&h, LP_ERR_INVALID_ARG, "null output");
  cudaDeviceSynchronize();
  for (int k = 0; k < LP_KIND_COUNT; ++k) { ms[k] = 0; work[k] = 0; launches[k] = 0; }
  for (auto& r : h.prof) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.e0, r.e1) == cudaSuccess && r.kind >= 0 && r.kind < LP_KIND_COUNT) {
      ms[r.kind] += t; work[r.kind] += r.work; launches[r.kind] += r.launches;
    }
    cudaEventDestroy(r.e0);
    cudaEventDestroy(r.e1);
  }
  h.prof.clear();
  return check_cuda(&h, "lp_profile_read");
}

int lp_last_step_launches(lp_handle hh) { return hh ? hh->h.last_launches : 0; }
size_t lp_device_bytes(lp_handle hh) { return hh ? hh->h.device_bytes : 0; }
const char* lp_last_error(lp_handle hh) { return hh ? hh->h.err.c_str() : g_create_error.c_str(); }

}  // extern "C"
