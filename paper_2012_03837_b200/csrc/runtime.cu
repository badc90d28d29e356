// Handle memory, parameter arena and launch emitters (see runtime.h).
#include "runtime.h"
#include "gemm_tc.h"

#include <algorithm>
#include <cmath>
#include <stdexcept>

namespace lp {

// ------------------------------------------------------------------ memory
void* Handle::dalloc(size_t bytes) {
  if (bytes == 0) bytes = 256;
  bytes = (bytes + 255) / 256 * 256;
  void* p = nullptr;
  if (use_cuda_malloc) {
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { cudaGetLastError(); p = nullptr; }
  } else {
    p = alloc.alloc(bytes, alloc.user);
  }
  if (!p) throw std::runtime_error("alloc: device allocation of " + std::to_string(bytes) + " bytes failed");
  blocks.push_back(p);
  device_bytes += bytes;
  cudaError_t e = cudaMemset(p, 0, bytes);
  if (e != cudaSuccess) throw std::runtime_error(std::string("cuda: memset: ") + cudaGetErrorString(e));
  return p;
}

// ------------------------------------------------------------------ arena
void Handle::add_tensor(const std::string& name, int chunk, std::vector<int64_t> shape, bool matrix) {
  TensorRec t;
  t.name = name;
  t.chunk = chunk;
  t.shape = shape;
  t.numel = 1;
  for (auto s : shape) t.numel *= s;
  t.matrix = matrix;
  tensors.push_back(t);
}

// Arena order: every matrix first, then every vector; each tensor starts on a 128-element
// boundary (256 bytes in bf16, 512 in fp32), padding stays zero under every update rule.
void Handle::finalize_arena() {
  long long off = 0;
  for (int pass = 0; pass < 2; ++pass) {
    for (auto& t : tensors) {
      if (t.matrix != (pass == 0)) continue;
      t.off = off;
      off += (t.numel + 127) / 128 * 128;
    }
    if (pass == 0) n_matrix = off;
  }
  n_total = off;
  master = (float*)dalloc(n_total * sizeof(float));
  m1 = (float*)dalloc(n_total * sizeof(float));
  if (opt.kind == LP_OPT_ADAM) m2 = (float*)dalloc(n_total * sizeof(float));
  grad = (float*)dalloc(n_total * sizeof(float));
  if (bf16_mode) working = (bf16*)dalloc(std::max<long long>(n_matrix, 128) * sizeof(bf16));
}

int Handle::find(const std::string& name) const {
  for (size_t i = 0; i < tensors.size(); ++i)
    if (tensors[i].name == name) return (int)i;
  throw std::runtime_error("internal: no tensor named " + name);
}
const void* Handle::W(const std::string& name) const {
  const TensorRec& t = tensors[find(name)];
  if (bf16_mode && t.matrix) return working + t.off;
  return master + t.off;
}
float* Handle::P32(const std::string& name) const { return master + tensors[find(name)].off; }
float* Handle::G(const std::string& name) const { return grad + tensors[find(name)].off; }

// ------------------------------------------------------------------ GEMM problems
GemmProb gemm_fwd(const void* x, const void* W, void* y, int M, int N, int Kd, const float* bias, int act) {
  GemmProb g{};
  g.A = x; g.B = W; g.C = y; g.bias = bias; g.act = act;
  g.M = M; g.N = N; g.K = Kd;
  g.a_ms = Kd; g.a_ks = 1; g.b_ns = Kd; g.b_ks = 1; g.ldc = N;
  return g;
}
// dx[M,Kd] = dy[M,N] * W[N,Kd]  (reduction over N)
GemmProb gemm_dgrad(const void* dy, const void* W, void* dx, int M, int N, int Kd, int act, const void* aux) {
  GemmProb g{};
  g.A = dy; g.B = W; g.C = dx; g.act = act; g.aux = aux;
  g.M = M; g.N = Kd; g.K = N;
  g.a_ms = N; g.a_ks = 1; g.b_ns = 1; g.b_ks = Kd; g.ldc = Kd;
  return g;
}
// dW[N,Kd] = dy[M,N]^T * x[M,Kd]  (reduction over the M rows of the minibatch), fp32 output
GemmProb gemm_wgrad(const void* dy, const void* x, float* dW, int M, int N, int Kd) {
  GemmProb g{};
  g.A = dy; g.B = x; g.C = dW; g.out_f32 = 1;
  g.M = N; g.N = Kd; g.K = M;
  g.a_ms = 1; g.a_ks = N; g.b_ns = 1; g.b_ks = Kd; g.ldc = Kd;
  return g;
}

// ------------------------------------------------------------------ emitters
void emit_gemm(Handle& h, Plan& p, std::vector<GemmProb> probs) {
  if (probs.empty()) return;
  // Weight gradients whose output is a handful of tiles but whose reduction runs over very many
  // rows (first-stage convolutions, the stem) would keep only a few SMs busy: split the reduction
  // into slices that write fp32 partial outputs, summed in slice order by the plan's final
  // column reduction (deterministic; no atomics).
  {
    std::vector<GemmProb> expanded;
    const size_t es = h.esize();
    // Work of the whole grouped launch in k-slices (tiles x 64-deep slices per tile) and what one SM gets if
    // it is spread evenly: a problem whose single tile is longer than that share would be the launch's tail.
    double launch_slices = 0;
    for (auto& g : probs) launch_slices += (double)((g.M + 127) / 128) * ((g.N + 255) / 256) * ((g.K + 63) / 64);
    const double share = std::max(32.0, launch_slices / h.num_sms);
    for (auto& g : probs) {
      bool plain = g.out_f32 && g.act == EPI_NONE && !g.bias && !g.resid && g.ldc == g.N;
      long long S = 1;
      if (plain && g.K >= 8192 && (g.K + 63) / 64 > share)
        S = std::max(1LL, std::min<long long>({(long long)std::ceil(((g.K + 63) / 64) / share), g.K / 2048LL, 64LL}));
      if (S == 1) { expanded.push_back(g); continue; }
      size_t mn = (size_t)g.M * g.N;
      float* part = (float*)h.dalloc((size_t)S * mn * sizeof(float));
      int kc = (int)(((g.K + S - 1) / S + 63) / 64 * 64);
      int made = 0;
      for (int k0 = 0; k0 < g.K; k0 += kc, ++made) {
        GemmProb q = g;
        q.K = std::min(kc, g.K - k0);
        q.A = (const char*)g.A + (size_t)k0 * g.a_ks * es;
        if (g.conv == CONV_WGRAD) q.conv_k0 = g.conv_k0 + k0;     // the implicit operand is addressed by pixel, not by pointer
        else q.B = (const char*)g.B + (size_t)k0 * g.b_ks * es;
        q.C = part + (size_t)made * mn;
        expanded.push_back(q);
      }
      h.pending_reduce.push_back(ColReduceProb{part, (float*)g.C, made, (int)mn, (int)mn});
    }
    probs.swap(expanded);
  }
  // Problems the tensor-core kernel takes go into one grouped launch, the rest into another.
  std::vector<GemmProb> tc, simt;
  for (auto& g : probs) {
    if (!h.force_simt && gemm_tc_eligible(g)) tc.push_back(g);
    else if (g.conv != CONV_NONE) throw std::runtime_error("internal: implicit convolution problem not accepted by the tensor-core kernel");
    else simt.push_back(g);
  }
  // Long reductions with a plain epilogue run with 256x512 tiles per CTA pair in a launch of their own
  std::vector<GemmProb> wide_list, normal_list;
  for (auto& g : tc) (gemm_tc_wide_ok(g) ? wide_list : normal_list).push_back(g);
  {
    // ... provided they fill the CTA pairs for a few even waves; a short or ragged wide launch loses more to its
    // tail than the tile shape gains
    long long tiles = 0;
    for (auto& g : wide_list) tiles += (long long)((g.M + 255) / 256) * ((g.N + 511) / 512);
    const long long pairs = std::max(1, h.num_sms / 2), waves = (tiles + pairs - 1) / pairs;
    if (!wide_list.empty() && (waves < 3 || (double)tiles / (double)(waves * pairs) < 0.9)) {
      normal_list.insert(normal_list.end(), wide_list.begin(), wide_list.end());
      wide_list.clear();
    }
  }
  for (int wide = 0; wide < 2; ++wide) {
    std::vector<GemmProb>& list = wide ? wide_list : normal_list;
    if (list.empty()) continue;
    // Longest tiles (largest K) first: the persistent CTAs take tiles in list order, so the long ones do not
    // end up in the tail, and products that walk the same operand in different directions (a weight
    // gradient and an input gradient reading the same dy) are not interleaved in the cache.
    std::stable_sort(list.begin(), list.end(), [](const GemmProb& a, const GemmProb& b) { return a.K > b.K; });
    int total = 0;
    const int cg = wide ? 2 : gemm_tc_choose_cg(list.data(), (int)list.size());
    for (auto& g : list) total += gemm_tc_tiles(g, total, cg, wide);
    struct alignas(64) Map { unsigned char b[128]; };
    std::vector<Map> maps(4 * list.size());
    for (size_t i = 0; i < list.size(); ++i)
      if (!gemm_tc_encode(list[i], &maps[4 * i], cg)) throw std::runtime_error("cuda: cuTensorMapEncodeTiled failed");
    const GemmProb* d = h.upload(list);
    const void* dm = h.upload(maps);
    int n = (int)list.size();
    int* st = h.d_status;
    int sms = h.num_sms;
    double fl = 0;
    for (auto& g : list) fl += 2.0 * g.M * g.N * g.K;
    // tiles of very different lengths in one launch: a balanced assignment to the CTAs, made once here
    std::vector<int> sched, off;
    const int *dsched = nullptr, *doff = nullptr;
    if (gemm_tc_schedule(list.data(), n, total, sms, cg, sched, off)) { dsched = h.upload(sched); doff = h.upload(off); }
    p.add(1, [=](const RunCtx& c) { launch_gemm_tc(d, dm, n, total, st, sms, c.stream, cg, wide, dsched, doff); }, KIND_GEMM_TC, fl);
  }
  if (!simt.empty()) {
    int t = 0;
    for (auto& g : simt) {
      g.tiles_n = (g.N + 63) / 64;
      g.tile_start = t;
      t += ((g.M + 63) / 64) * g.tiles_n;
    }
    const GemmProb* d = h.upload(simt);
    bool bf = h.bf16_mode;
    int n = (int)simt.size();
    double fl = 0;
    for (auto& g : simt) fl += 2.0 * g.M * g.N * g.K;
    p.add(1, [d, simt, n, bf](const RunCtx& c) { launch_gemm_simt(d, simt.data(), n, bf, c.stream); }, KIND_GEMM_ALU, fl);
  }
}

// Vectors per lane for the register-resident LayerNorm kernels (rows of 256, 512 or 1024 bf16), else 0.
static int ln_vec_width(const Handle& h, int d) {
  if (!h.bf16_mode) return 0;
  return d == 256 ? 1 : d == 512 ? 2 : d == 1024 ? 4 : 0;
}

void emit_ln_fwd(Handle& h, Plan& p, const std::vector<LnProb>& probs) {
  if (probs.empty()) return;
  int mr = 0;
  for (auto& q : probs) mr = std::max(mr, q.rows);
  const LnProb* d = h.upload(probs);
  int n = (int)probs.size();
  bool bf = h.bf16_mode;
  double by = 0;
  for (auto& q : probs) by += 2.0 * q.rows * q.d * h.esize();
  int nv = ln_vec_width(h, probs[0].d);
  for (auto& q : probs) if (q.d != probs[0].d) nv = 0;
  if (nv) p.add(1, [=](const RunCtx& c) { launch_ln_fwd_vec(d, n, mr, nv, c.stream); }, KIND_NORM, by);
  else p.add(1, [=](const RunCtx& c) { launch_ln_fwd(d, n, mr, bf, c.stream); }, KIND_NORM, by);
}

void emit_ln_bwd(Handle& h, Plan& p, std::vector<LnBwdProb> probs, const std::vector<float*>& dgamma,
                 const std::vector<float*>& dbeta) {
  if (probs.empty()) return;
  int mr = 0;
  for (size_t i = 0; i < probs.size(); ++i) {
    auto& q = probs[i];
    mr = std::max(mr, q.rows);
    int nblk = (q.rows + LN_BWD_ROWS - 1) / LN_BWD_ROWS;
    q.part = (float*)h.dalloc((size_t)nblk * 2 * q.d * sizeof(float));
    h.pending_reduce.push_back(ColReduceProb{q.part, dgamma[i], nblk, q.d, 2 * q.d});
    h.pending_reduce.push_back(ColReduceProb{q.part + q.d, dbeta[i], nblk, q.d, 2 * q.d});
  }
  const LnBwdProb* d = h.upload(probs);
  int n = (int)probs.size();
  bool bf = h.bf16_mode;
  double by = 0;
  for (auto& q : probs) by += (double)q.rows * q.d * h.esize() * (2 + (q.dx ? 1 : 0) + (q.dres ? 1 : 0));
  int nv = ln_vec_width(h, probs[0].d);
  for (auto& q : probs) if (q.d != probs[0].d) nv = 0;
  if (nv) p.add(1, [=](const RunCtx& c) { launch_ln_bwd_vec(d, n, mr, nv, c.stream); }, KIND_NORM, by);
  else p.add(1, [=](const RunCtx& c) { launch_ln_bwd(d, n, mr, bf, c.stream); }, KIND_NORM, by);
}

void emit_colsum(Handle& h, Plan& p, const std::vector<ColSumProb>& in, const std::vector<float*>& out) {
  if (in.empty()) return;
  std::vector<ColSumProb> probs = in;
  int mr = 0, mc = 0;
  for (size_t i = 0; i < probs.size(); ++i) {
    auto& q = probs[i];
    mr = std::max(mr, q.rows);
    mc = std::max(mc, q.cols);
    int nblk = (q.rows + COLSUM_ROWS - 1) / COLSUM_ROWS;
    q.part = (float*)h.dalloc((size_t)nblk * q.cols * sizeof(float));
    h.pending_reduce.push_back(ColReduceProb{q.part, out[i], nblk, q.cols, q.cols});
  }
  const ColSumProb* d = h.upload(probs);
  int n = (int)probs.size();
  bool bf = h.bf16_mode;
  double by = 0;
  bool vec8 = bf;
  for (auto& q : probs) {
    by += (double)q.rows * q.cols * h.esize();
    if (q.cols % 8 || q.ld % 8 || ((uintptr_t)q.x & 15)) vec8 = false;
  }
  p.add(1, [=](const RunCtx& c) { launch_colsum_partial(d, n, mr, mc, bf, c.stream, vec8); }, KIND_REDUCE, by);
}

void emit_pending_reduce(Handle& h, Plan& p) {
  if (h.pending_reduce.empty()) return;
  // flat list of blocks: (problem, block of 128 columns inside it)
  std::vector<int2> blocks;
  for (size_t i = 0; i < h.pending_reduce.size(); ++i)
    for (int b = 0; b * 128 < h.pending_reduce[i].cols; ++b) blocks.push_back(make_int2((int)i, b));
  const ColReduceProb* d = h.upload(h.pending_reduce);
  const int2* db = h.upload(blocks);
  int nb = (int)blocks.size();
  double by = 0;
  for (auto& q : h.pending_reduce) by += (double)q.rows * q.cols * 4;
  h.pending_reduce.clear();
  p.add(1, [=](const RunCtx& c) { launch_col_reduce_f32(d, db, nb, c.stream); }, KIND_REDUCE, by);
}

void emit_labels(Handle& h, Plan& p, const std::vector<LabelProb>& probs) {
  const LabelProb* d = h.upload(probs);
  int n = (int)probs.size();
  int* st = h.d_status;
  p.add(1, [=](const RunCtx& c) { launch_label_prep(d, n, st, c.stream); });
}

bool emit_xent_and_loss(Handle& h, Plan& p, std::vector<XentProb> probs, const std::vector<int>& chunk_of,
                        const std::vector<float*>* bias_grads) {
  if (probs.empty()) return false;
  int mr = 0;
  std::vector<LossProb> lps;
  for (size_t i = 0; i < probs.size(); ++i) {
    mr = std::max(mr, probs[i].rows);
    lps.push_back(LossProb{probs[i].row_loss, probs[i].n_valid, probs[i].rows, chunk_of[i]});
  }
  double by = 0;
  for (auto& q : probs) by += 2.0 * q.rows * q.classes * h.esize();
  bool bf = h.bf16_mode;
  int nv = 0;
  if (bf && probs[0].classes % 8 == 0 && probs[0].classes <= 32768) {
    nv = 1;
    while (nv * 2048 < probs[0].classes) nv *= 2;
    for (auto& q : probs)
      if (q.classes != probs[0].classes || q.ld % 8 != 0 || ((uintptr_t)q.z & 15)) nv = 0;
  }
  // Long rows: blocks of XENT_ROWS rows with the next row prefetched, and the bias gradient on the way.
  const bool rows_kernel = nv != 0 && probs[0].classes >= 2048;
  const int classes = probs[0].classes;
  if (rows_kernel && bias_grads) {
    for (size_t i = 0; i < probs.size(); ++i) {
      int nblk = (probs[i].rows + XENT_ROWS - 1) / XENT_ROWS;
      probs[i].colsum_part = (float*)h.dalloc((size_t)nblk * classes * sizeof(float));
      h.pending_reduce.push_back(ColReduceProb{probs[i].colsum_part, (*bias_grads)[i], nblk, classes, classes});
    }
  }
  const XentProb* d = h.upload(probs);
  const LossProb* dl = h.upload(lps);
  int n = (int)probs.size();
  float* losses = h.d_losses;
  int* st = h.d_status;
  p.add(2, [=](const RunCtx& c) {
    if (rows_kernel) launch_xent_rows(d, n, mr, classes, c.stream);
    else if (nv) launch_xent_vec(d, n, mr, nv, c.stream);
    else launch_xent(d, n, mr, bf, c.stream);
    launch_loss_reduce(dl, n, losses, st, c.stream);
  }, KIND_XENT, by);
  return rows_kernel && bias_grads;
}

void emit_xent_from_stats(Handle& h, Plan& p, std::vector<XentStatsProb> probs, const std::vector<int>& chunk_of,
                          const std::vector<float*>* bias_grads) {
  if (probs.empty()) return;
  int mr = 0;
  const int classes = probs[0].classes;
  std::vector<LossProb> lps;
  double by = 0;
  for (size_t i = 0; i < probs.size(); ++i) {
    auto& q = probs[i];
    mr = std::max(mr, q.rows);
    lps.push_back(LossProb{q.row_loss, q.n_valid, q.rows, chunk_of[i]});
    by += 2.0 * q.rows * q.classes * h.esize();
    q.row_c = (float*)h.dalloc((size_t)q.rows * sizeof(float));
    if (bias_grads) {
      int nblk = (q.rows + XENT_APPLY_ROWS - 1) / XENT_APPLY_ROWS;
      q.colsum_part = (float*)h.dalloc((size_t)nblk * classes * sizeof(float));
      h.pending_reduce.push_back(ColReduceProb{q.colsum_part, (*bias_grads)[i], nblk, classes, classes});
    }
  }
  const XentStatsProb* d = h.upload(probs);
  const LossProb* dl = h.upload(lps);
  int n = (int)probs.size();
  float* losses = h.d_losses;
  int* st = h.d_status;
  p.add(3, [=](const RunCtx& c) {
    launch_xent_from_stats(d, n, mr, classes, c.stream);
    launch_loss_reduce(dl, n, losses, st, c.stream);
  }, KIND_XENT, by);
}

void emit_argmax(Handle& h, Plan& p, const std::vector<ArgmaxProb>& probs) {
  if (probs.empty()) return;
  const ArgmaxProb* d = h.upload(probs);
  int n = (int)probs.size(), mr = 0, stride = h.rows;
  for (auto& q : probs) mr = std::max(mr, q.rows);
  bool bf = h.bf16_mode;
  p.add(0, [=](const RunCtx& c) {
    if (c.out_pred || c.out_correct) launch_argmax(d, n, mr, bf, c.out_pred, stride, c.out_correct, c.stream);
  });
}

OptimArgs optimizer_args(const Handle& h) {
  OptimArgs a{};
  a.master = h.master; a.m1 = h.m1; a.m2 = h.m2; a.grad = h.grad; a.working = h.working;
  a.n_total = h.n_total; a.n_matrix = h.n_matrix;
  a.kind = h.opt.kind; a.lr = h.opt.lr; a.momentum = h.opt.momentum; a.weight_decay = h.opt.weight_decay;
  a.beta1 = h.opt.beta1; a.beta2 = h.opt.beta2; a.eps = h.opt.eps;
  // all chunks share one step count here (otherwise the per-chunk table below carries theirs)
  double t = (double)((h.updates.empty() ? h.step_count : h.updates[0]) + 1);
  a.omb1 = (float)(1.0 - (double)h.opt.beta1);
  a.omb2 = (float)(1.0 - (double)h.opt.beta2);
  a.bc1 = (float)(1.0 - pow((double)h.opt.beta1, t));
  a.bc2 = (float)(1.0 - pow((double)h.opt.beta2, t));
  if (h.per_chunk_counts) {   // the step driver has filled d_chunk_tab for this step
    a.seg_end = h.d_seg_end; a.seg_chunk = h.d_seg_chunk; a.n_seg = h.n_seg; a.chunk_tab = h.d_chunk_tab;
  }
  return a;
}

void emit_optimizer(Handle& h, Plan& p) {
  Handle* hp = &h;
  p.add(1, [hp](const RunCtx& c) { launch_optim(optimizer_args(*hp), c.stream); }, KIND_OPTIM,
        (double)h.n_total * (h.opt.kind == LP_OPT_ADAM ? 28.0 : 20.0) + (h.bf16_mode ? 2.0 * h.n_matrix : 0.0));
}

void emit_attention(Handle& h, Plan& p, const std::vector<AttnProb>& probs, bool backward) {
  if (probs.empty()) return;
  const int n = (int)probs.size();
  int B = 0, T = 0, H = 0;
  for (auto& a : probs) { B = std::max(B, a.B); T = std::max(T, a.T); H = std::max(H, a.H); }
  double pairs = 0;                                     // causal (query, key) pairs x head width
  for (auto& a : probs) pairs += (double)a.B * a.H * 64.0 * a.T * (a.T + 1) / 2;
  const double work = (backward ? 10.0 : 4.0) * pairs;
  const bool bf = h.bf16_mode;
  if (bf && !h.force_simt) {
    std::vector<AttnTcProb> tab(n);
    for (int i = 0; i < n; ++i)
      if (!attn_tc_encode(tab[i], probs[i])) throw std::runtime_error("cuda: cuTensorMapEncodeTiled failed for an attention operand");
    const AttnTcProb* dp = h.upload(tab);
    int* st = h.d_status;
    if (backward) p.add(2, [=](const RunCtx& c) { launch_attn_bwd_tc(dp, n, B, T, H, st, c.stream); }, KIND_ATTN, work);
    else p.add(1, [=](const RunCtx& c) { launch_attn_fwd_tc(dp, n, B, T, H, st, c.stream); }, KIND_ATTN, work);
    return;
  }
  const AttnProb* dp = h.upload(probs);
  if (backward) p.add(2, [=](const RunCtx& c) { launch_attn_bwd(dp, n, B, T, H, bf, c.stream); }, KIND_ATTN, work);
  else p.add(1, [=](const RunCtx& c) { launch_attn_fwd(dp, n, B, T, H, bf, c.stream); }, KIND_ATTN, work);
}

}  // namespace lp
