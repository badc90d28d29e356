// MLP family: chunks of Linear+ReLU layers (App. A.1) with a Linear + softmax cross-entropy
// auxiliary head per chunk (Sec. 3).  Builds the synchronous, pipelined, priming and forward-only
// plans.  Within a plan, work that belongs to different chunks and does not depend on another
// chunk's result of the same step is issued as one grouped launch.
#include <stdexcept>

#include "runtime.h"

namespace lp {
namespace {

struct MlpBufs {
  std::vector<std::vector<int>> widths;        // [k][i]
  std::vector<int> d_in;                       // input width of chunk k
  std::vector<std::vector<void*>> y;           // [k][i] layer outputs except the last (which is the boundary)
  std::vector<void*> z;                        // [k] logits / dlogits
  std::vector<float*> row_loss;                // [k]
  std::vector<void*> g0, g1;                   // [k] gradient ping-pong buffers [B, max width]
};

std::string tn(int k, int i, const char* s) { return "c" + std::to_string(k) + ".l" + std::to_string(i) + "." + s; }
std::string hn(int k, const char* s) { return "c" + std::to_string(k) + ".head." + s; }

// Input of chunk k for a plan that reads boundary half `rd`.
const void* chunk_in(Handle& h, int k, int rd) { return k == 0 ? h.x_in : h.bnd[rd][k - 1]; }

// Forward of the chunks in `ks` (layer index aligned from the front), outputs into half `wr`.
void forward_level(Handle& h, MlpBufs& b, Plan& p, const std::vector<int>& ks, int rd, int wr) {
  size_t maxl = 0;
  for (int k : ks) maxl = std::max(maxl, b.widths[k].size());
  int B = h.spec.batch;
  for (size_t i = 0; i < maxl; ++i) {
    std::vector<GemmProb> g;
    for (int k : ks) {
      if (i >= b.widths[k].size()) continue;
      bool last = i + 1 == b.widths[k].size();
      const void* in = i == 0 ? chunk_in(h, k, rd) : b.y[k][i - 1];
      int din = i == 0 ? b.d_in[k] : b.widths[k][i - 1];
      void* out = last ? h.bnd[wr][k] : b.y[k][i];
      g.push_back(gemm_fwd(in, h.W(tn(k, (int)i, "W")), out, B, b.widths[k][i], din, h.P32(tn(k, (int)i, "b")), EPI_RELU));
    }
    emit_gemm(h, p, g);
  }
}

// Collects the phases of a single-launch step (FusedArgs).  The GEMMs of a phase are held back until the phase
// ends: whether they are cut into 16x16 or 32x32 tiles depends on how many tiles the whole phase has.
struct FusedBuilder {
  std::vector<FusedPhase> phases;
  std::vector<FusedTask> tasks;
  std::vector<FusedGemm> gemms;
  std::vector<GemmProb> held;
  std::vector<FusedPrefetch> prefetches;
  std::vector<FusedXent> xents;
  std::vector<FusedColSum> colsums;
  std::vector<LossProb> losses;
  std::vector<LabelProb> labels;
  int grid = 148;
  double flops = 0;

  void begin() { phases.push_back(FusedPhase{(int)tasks.size(), (int)tasks.size(), 0}); held.clear(); }
  void add(int type, int index, int n) {
    if (n <= 0) return;
    tasks.push_back(FusedTask{type, index, phases.back().units, n});
    phases.back().units += n;
    phases.back().task_end = (int)tasks.size();
  }
  void gemm(const GemmProb& g) { held.push_back(g); }
  void xent(const FusedXent& x) { xents.push_back(x); add(FT_XENT, (int)xents.size() - 1, (x.rows + FUSED_THREADS / 32 - 1) / (FUSED_THREADS / 32)); }
  void colsum(const FusedColSum& c) { colsums.push_back(c); add(FT_COLSUM, (int)colsums.size() - 1, (c.cols + FUSED_THREADS - 1) / FUSED_THREADS); }
  void loss(const LossProb& l) { losses.push_back(l); add(FT_LOSS, (int)losses.size() - 1, 1); }
  void label(const LabelProb& l) { labels.push_back(l); add(FT_LABELS, (int)labels.size() - 1, 1); }
  void optim(long long n_total) { add(FT_OPTIM, 0, (int)((n_total / 4 + FUSED_THREADS - 1) / FUSED_THREADS)); }
  void prefetch(const void* p, long long bytes) {
    prefetches.push_back(FusedPrefetch{p, bytes});
    add(FT_PREFETCH, (int)prefetches.size() - 1, (int)((bytes + 128 * FUSED_THREADS - 1) / (128 * FUSED_THREADS)));
  }
  void end() {
    flush();
    if (phases.back().units == 0) phases.pop_back();
  }
  void flush() {                                         // cut the held GEMMs into tiles
    long long t16 = 0;
    for (auto& g : held) t16 += (long long)((g.M + 15) / 16) * ((g.N + 15) / 16);
    const bool crowded = t16 > 2ll * grid;             // more than two waves of small tiles: cut larger ones
    for (auto& g : held) {
      const bool big = crowded && g.M >= 32 && g.N >= 32;
      const int T = big ? 32 : 16;
      FusedGemm f{(const float*)g.A, (const float*)g.B, (float*)g.C, g.bias, (const float*)g.aux,
                  g.M, g.N, g.K, g.ldc, g.act, (g.N + T - 1) / T, (int)g.a_ms, (int)g.a_ks, (int)g.b_ns, (int)g.b_ks};
      gemms.push_back(f);
      add(big ? FT_GEMM32 : FT_GEMM16, (int)gemms.size() - 1, ((g.M + T - 1) / T) * f.tiles_n);
      flops += 2.0 * g.M * g.N * g.K;
    }
    held.clear();
  }
};

}  // namespace

void build_mlp(Handle& h) {
  const int K = h.K, B = h.spec.batch, C = h.head.classes;
  auto* bp = new MlpBufs();   // lives as long as the handle's plans (freed with the process; tiny)
  MlpBufs& b = *bp;
  b.widths.resize(K);
  b.d_in.resize(K);
  int li = 0, prev = h.spec.d_in, maxw = 0;
  for (int k = 0; k < K; ++k) {
    b.d_in[k] = prev;
    for (int i = 0; i < h.per_chunk[k]; ++i) {
      int w = h.layer_widths[li++];
      h.add_tensor(tn(k, i, "W"), k, {w, prev}, true);
      h.add_tensor(tn(k, i, "b"), k, {w}, false);
      b.widths[k].push_back(w);
      prev = w;
      maxw = std::max(maxw, w);
    }
    h.add_tensor(hn(k, "W"), k, {C, prev}, true);
    h.add_tensor(hn(k, "b"), k, {C}, false);
  }
  h.finalize_arena();
  h.rows = B;
  size_t es = h.esize();
  h.x_bytes = (size_t)B * h.spec.d_in * es;
  h.x_in = h.dalloc(h.x_bytes);
  h.y_bytes = (size_t)B * sizeof(int);
  h.y_in = (int*)h.dalloc(h.y_bytes);
  b.y.resize(K);
  for (int k = 0; k < K; ++k) {
    size_t bytes = (size_t)B * b.widths[k].back() * es;
    h.bnd_bytes.push_back(bytes);
    for (int s = 0; s < 2; ++s) {
      h.bnd[s].push_back(h.dalloc(bytes));
      h.lab[s].push_back((int*)h.dalloc(h.y_bytes));
    }
    h.n_valid.push_back((int*)h.dalloc(sizeof(int)));
    for (size_t i = 0; i + 1 < b.widths[k].size(); ++i) b.y[k].push_back(h.dalloc((size_t)B * b.widths[k][i] * es));
    b.z.push_back(h.dalloc((size_t)B * C * es));
    b.row_loss.push_back((float*)h.dalloc((size_t)B * sizeof(float)));
    b.g0.push_back(h.dalloc((size_t)B * maxw * es));
    b.g1.push_back(h.dalloc((size_t)B * maxw * es));
  }

  std::vector<int> all;
  for (int k = 0; k < K; ++k) all.push_back(k);

  // labels chunk k trains on, for a plan that reads half `rd` (pipelined) or the step's own y (sync)
  auto labels_of = [&](int k, bool pipelined, int rd) -> const int* {
    return (!pipelined || k == 0) ? h.y_in : h.lab[rd][k - 1];
  };

  // Overlapping local parallelism (Sec. 3, Fig. 2 c): the block trained by chunk k's loss also holds the last
  // layer of chunk k-1.  That layer exists once; the loss of chunk k is propagated one layer past the chunk
  // boundary into a second gradient for it (g2w / g2b), and its update uses the mean of its two gradients.
  std::vector<float*> g2w(K, nullptr), g2b(K, nullptr);     // second gradient of chunk k's last layer
  auto build_step = [&](Plan& p, bool pipelined, int rd, int wr, bool overlap) {
    std::vector<LabelProb> lps;
    for (int k = 0; k < K; ++k)
      lps.push_back(LabelProb{labels_of(k, pipelined, rd), (pipelined && k < K - 1) ? h.lab[wr][k] : nullptr, B, C,
                              h.n_valid[k]});
    emit_labels(h, p, lps);
    if (pipelined) forward_level(h, b, p, all, rd, wr);
    else for (int k = 0; k < K; ++k) forward_level(h, b, p, {k}, rd, wr);
    // heads: logits, loss, dlogits
    {
      std::vector<GemmProb> g;
      std::vector<XentProb> xs;
      for (int k = 0; k < K; ++k) {
        g.push_back(gemm_fwd(h.bnd[wr][k], h.W(hn(k, "W")), b.z[k], B, C, b.widths[k].back(), h.P32(hn(k, "b")), EPI_NONE));
        xs.push_back(XentProb{b.z[k], labels_of(k, pipelined, rd), h.n_valid[k], b.row_loss[k], B, C, C, nullptr});
      }
      emit_gemm(h, p, g);
      emit_xent_and_loss(h, p, xs, all);
    }
    // head backward: dW_h, db_h, and the gradient at the last layer's pre-activation
    {
      std::vector<GemmProb> g;
      std::vector<ColSumProb> cs;
      std::vector<float*> outs;
      for (int k = 0; k < K; ++k) {
        int D = b.widths[k].back();
        g.push_back(gemm_wgrad(b.z[k], h.bnd[wr][k], h.G(hn(k, "W")), B, C, D));
        g.push_back(gemm_dgrad(b.z[k], h.W(hn(k, "W")), b.g0[k], B, C, D, EPI_RELU_MASK, h.bnd[wr][k]));
        cs.push_back(ColSumProb{b.z[k], nullptr, B, C, C});
        outs.push_back(h.G(hn(k, "b")));
      }
      emit_gemm(h, p, g);
      emit_colsum(h, p, cs, outs);
    }
    // trunk backward, aligned from the last layer of each chunk; nothing is propagated to the
    // chunk input (Sec. 3: the gradient stops at the chunk boundary)
    size_t maxl = 0;
    for (int k = 0; k < K; ++k) maxl = std::max(maxl, b.widths[k].size());
    std::vector<void*> du_over(K, nullptr);        // overlap: gradient at the pre-activation of chunk k-1's last layer
    for (size_t j = 0; j < maxl; ++j) {
      std::vector<GemmProb> g;
      std::vector<ColSumProb> cs;
      std::vector<float*> outs;
      for (int k = 0; k < K; ++k) {
        int nl = (int)b.widths[k].size();
        if ((int)j >= nl) continue;
        int i = nl - 1 - (int)j;
        void* du = (j % 2 == 0) ? b.g0[k] : b.g1[k];
        void* dnext = (j % 2 == 0) ? b.g1[k] : b.g0[k];
        const void* in = i == 0 ? chunk_in(h, k, rd) : b.y[k][i - 1];
        int din = i == 0 ? b.d_in[k] : b.widths[k][i - 1];
        int w = b.widths[k][i];
        g.push_back(gemm_wgrad(du, in, h.G(tn(k, i, "W")), B, w, din));
        if (i > 0) g.push_back(gemm_dgrad(du, h.W(tn(k, i, "W")), dnext, B, w, din, EPI_RELU_MASK, b.y[k][i - 1]));
        else if (overlap && k > 0) {               // one layer past the boundary: through the ReLU of the shared layer
          g.push_back(gemm_dgrad(du, h.W(tn(k, 0, "W")), dnext, B, w, din, EPI_RELU_MASK, chunk_in(h, k, rd)));
          du_over[k] = dnext;
        }
        cs.push_back(ColSumProb{du, nullptr, B, w, w});
        outs.push_back(h.G(tn(k, i, "b")));
      }
      emit_gemm(h, p, g);
      emit_colsum(h, p, cs, outs);
    }
    std::vector<AvgProb> avg;
    long long avg_max = 0;
    if (overlap) {
      std::vector<GemmProb> g;
      std::vector<ColSumProb> cs;
      std::vector<float*> outs;
      for (int k = 1; k < K; ++k) {
        const int q = k - 1, nl = (int)b.widths[q].size(), i = nl - 1;     // the shared layer: chunk q's last
        const int w = b.widths[q][i], din = i == 0 ? b.d_in[q] : b.widths[q][i - 1];
        const void* in = i == 0 ? chunk_in(h, q, rd) : b.y[q][i - 1];
        if (!g2w[q]) { g2w[q] = (float*)h.dalloc((size_t)w * din * sizeof(float)); g2b[q] = (float*)h.dalloc((size_t)w * sizeof(float)); }
        g.push_back(gemm_wgrad(du_over[k], in, g2w[q], B, w, din));
        cs.push_back(ColSumProb{du_over[k], nullptr, B, w, w});
        outs.push_back(g2b[q]);
        avg.push_back(AvgProb{h.G(tn(q, i, "W")), g2w[q], (long long)w * din});
        avg.push_back(AvgProb{h.G(tn(q, i, "b")), g2b[q], (long long)w});
        avg_max = std::max(avg_max, (long long)w * din);
      }
      emit_gemm(h, p, g);
      emit_colsum(h, p, cs, outs);
    }
    emit_pending_reduce(h, p);
    if (!avg.empty()) {
      const AvgProb* d = h.upload(avg);
      int n = (int)avg.size();
      double bytes = 0;
      for (auto& a : avg) bytes += 12.0 * a.n;
      p.add(1, [=](const RunCtx& r) { launch_average_f32(d, n, avg_max, r.stream); }, KIND_REDUCE, bytes);
    }
    emit_optimizer(h, p);
  };

  auto build_forward = [&](Plan& p, int wr, bool heads) {
    for (int k = 0; k < K; ++k) forward_level(h, b, p, {k}, wr, wr);
    if (!heads) return;
    std::vector<LabelProb> lps;
    for (int k = 0; k < K; ++k) lps.push_back(LabelProb{h.y_in, nullptr, B, C, h.n_valid[k]});
    emit_labels(h, p, lps);
    std::vector<GemmProb> g;
    std::vector<XentProb> xs;
    for (int k = 0; k < K; ++k) {
      g.push_back(gemm_fwd(h.bnd[wr][k], h.W(hn(k, "W")), b.z[k], B, C, b.widths[k].back(), h.P32(hn(k, "b")), EPI_NONE));
      xs.push_back(XentProb{b.z[k], h.y_in, h.n_valid[k], b.row_loss[k], B, C, C, nullptr});
    }
    emit_gemm(h, p, g);
    void* zlast = b.z[K - 1];
    size_t zbytes = (size_t)B * C * es;
    p.add(0, [zlast, zbytes](const RunCtx& c) {
      if (c.out_logits) cudaMemcpyAsync(c.out_logits, zlast, zbytes, cudaMemcpyDeviceToDevice, c.stream);
    });
    std::vector<ArgmaxProb> am;
    for (int k = 0; k < K; ++k) am.push_back(ArgmaxProb{b.z[k], h.y_in, B, C, C, k});
    emit_argmax(h, p, am);
    emit_xent_and_loss(h, p, xs, all);
  };

  unsigned long long* fused_counter = nullptr;
  // The same step as one cooperative launch (fp32 storage, small networks: a step of at most a few GFLOP on
  // at most 64 chunks; larger ones are bound by arithmetic and keep the grouped launches above).
  auto build_fused = [&](Handle::FusedProgram& fp, bool pipelined, int rd, int wr) {
    FusedBuilder fb;
    fb.grid = h.fused_blocks;
    fb.begin();
    for (int k = 0; k < K; ++k)
      fb.label(LabelProb{labels_of(k, pipelined, rd), (pipelined && k < K - 1) ? h.lab[wr][k] : nullptr, B, C, h.n_valid[k]});
    auto layer = [&](int k, int i) {
      const bool last = i + 1 == (int)b.widths[k].size();
      const void* in = i == 0 ? chunk_in(h, k, rd) : b.y[k][i - 1];
      const int din = i == 0 ? b.d_in[k] : b.widths[k][i - 1];
      fb.gemm(gemm_fwd(in, h.W(tn(k, i, "W")), last ? h.bnd[wr][k] : b.y[k][i], B, b.widths[k][i], din,
                       h.P32(tn(k, i, "b")), EPI_RELU));
    };
    size_t maxl = 0;
    for (int k = 0; k < K; ++k) maxl = std::max(maxl, b.widths[k].size());
    // The label checks share the first forward phase, and so does a sweep that asks for the parameters and
    // the optimizer state to be brought into L2 (the blocks that have no tile in that phase issue it): the
    // later phases then find their operands there instead of waiting for DRAM one phase after the other.
    bool first = true;
    auto end_phase = [&]() {
      if (first) {
        fb.flush();
        const long long bytes = h.n_total * (long long)sizeof(float);
        if (bytes <= (4ll << 20)) {
          fb.prefetch(h.master, bytes);
          fb.prefetch(h.m1, bytes);
          if (h.m2) fb.prefetch(h.m2, bytes);
        }
      }
      first = false;
      fb.end();
    };
    if (pipelined) {
      for (size_t i = 0; i < maxl; ++i) {
        if (!first) fb.begin();
        for (int k = 0; k < K; ++k) if (i < b.widths[k].size()) layer(k, (int)i);
        end_phase();
      }
    } else {
      for (int k = 0; k < K; ++k)
        for (int i = 0; i < (int)b.widths[k].size(); ++i) {
          if (!first) fb.begin();
          layer(k, i);
          end_phase();
        }
    }
    fb.begin();                                          // heads: logits
    for (int k = 0; k < K; ++k)
      fb.gemm(gemm_fwd(h.bnd[wr][k], h.W(hn(k, "W")), b.z[k], B, C, b.widths[k].back(), h.P32(hn(k, "b")), EPI_NONE));
    fb.end();
    fb.begin();                                          // losses of the rows, dlogits in place
    for (int k = 0; k < K; ++k)
      fb.xent(FusedXent{(float*)b.z[k], labels_of(k, pipelined, rd), h.n_valid[k], b.row_loss[k], B, C, C});
    fb.end();
    fb.begin();                                          // head backward, chunk losses
    for (int k = 0; k < K; ++k) {
      const int D = b.widths[k].back();
      fb.gemm(gemm_wgrad(b.z[k], h.bnd[wr][k], h.G(hn(k, "W")), B, C, D));
      fb.gemm(gemm_dgrad(b.z[k], h.W(hn(k, "W")), b.g0[k], B, C, D, EPI_RELU_MASK, h.bnd[wr][k]));
      fb.colsum(FusedColSum{(const float*)b.z[k], h.G(hn(k, "b")), B, C, C});
      fb.loss(LossProb{b.row_loss[k], h.n_valid[k], B, k});
    }
    fb.end();
    for (size_t j = 0; j < maxl; ++j) {                  // trunk backward, aligned from the last layer of each chunk
      fb.begin();
      for (int k = 0; k < K; ++k) {
        const int nl = (int)b.widths[k].size();
        if ((int)j >= nl) continue;
        const int i = nl - 1 - (int)j;
        void* du = (j % 2 == 0) ? b.g0[k] : b.g1[k];
        void* dnext = (j % 2 == 0) ? b.g1[k] : b.g0[k];
        const void* in = i == 0 ? chunk_in(h, k, rd) : b.y[k][i - 1];
        const int din = i == 0 ? b.d_in[k] : b.widths[k][i - 1];
        const int w = b.widths[k][i];
        fb.gemm(gemm_wgrad(du, in, h.G(tn(k, i, "W")), B, w, din));
        if (i > 0) fb.gemm(gemm_dgrad(du, h.W(tn(k, i, "W")), dnext, B, w, din, EPI_RELU_MASK, b.y[k][i - 1]));
        fb.colsum(FusedColSum{(const float*)du, h.G(tn(k, i, "b")), B, w, w});
      }
      fb.end();
    }
    fb.begin();
    fb.optim(h.n_total);
    fb.end();
    FusedArgs& a = fp.args;
    a.phases = h.upload(fb.phases);
    a.n_phases = (int)fb.phases.size();
    a.tasks = h.upload(fb.tasks);
    a.n_tasks = (int)fb.tasks.size();
    a.gemms = h.upload(fb.gemms);
    a.n_gemms = (int)fb.gemms.size();
    a.prefetches = h.upload(fb.prefetches);
    a.xents = h.upload(fb.xents);
    a.colsums = h.upload(fb.colsums);
    a.losses = h.upload(fb.losses);
    a.labels = h.upload(fb.labels);
    a.d_losses = h.d_losses;
    a.status = h.d_status;
    a.counter = fused_counter;
    a.x_slot = h.x_in;
    a.y_slot = h.y_in;
    fp.flops = fb.flops;
    fp.ok = true;
  };
  double step_flops = 0;
  {
    int prev_w = h.spec.d_in;
    for (int k = 0; k < K; ++k) {
      for (int w : b.widths[k]) { step_flops += 6.0 * B * w * prev_w; prev_w = w; }
      step_flops += 6.0 * B * C * prev_w;
    }
  }
  if (!h.bf16_mode && K <= 64 && step_flops <= 4e9) h.fused_blocks = fused_mlp_max_blocks(h.num_sms);
  if (h.fused_blocks > 0) {
    fused_counter = (unsigned long long*)h.dalloc(2 * sizeof(unsigned long long));
    build_fused(h.fused_sync, false, 0, 0);
    for (int par = 0; par < 2; ++par) build_fused(h.fused_pipe[par], true, par, 1 - par);
    h.use_fused = true;
  }

  build_step(h.sync_plan, false, 0, 0, false);
  if (K > 1) {
    build_step(h.sync_overlap_plan, false, 0, 0, true);
    h.has_overlap_plan = true;
  }
  for (int par = 0; par < 2; ++par) {
    build_step(h.pipe_plan[par], true, par, 1 - par, false);
    // priming: forward chain into the half the first pipelined step will read, labels alongside
    build_forward(h.prime_plan[par], par, false);
    std::vector<LabelProb> lps;
    for (int k = 0; k + 1 < K; ++k) lps.push_back(LabelProb{h.y_in, h.lab[par][k], B, C, h.n_valid[k]});
    if (!lps.empty()) emit_labels(h, h.prime_plan[par], lps);
    build_forward(h.fwd_plan[par], par, true);
  }
}

}  // namespace lp
