// Decoder-only transformer LM family (App. B.2): token + position embeddings in chunk 0, pre-LayerNorm
// blocks (causal attention, GELU feed-forward), and a LayerNorm + vocabulary projection + softmax
// cross-entropy auxiliary head on every chunk (Sec. 3; App. B.2 for the head's form).
//
// Forward of one block:  a1 = LN1(h); qkv = a1 Wqkv^T + b; o = Attn(qkv); h1 = h + o Wo^T + b;
//                        a2 = LN2(h1); u = a2 W1^T + b; g = GELU(u); h' = h1 + g W2^T + b.
// Backward is truncated at the chunk input: for the first block of a chunk k > 0 only LN1's scale
// and shift gradients are formed, not the gradient of the chunk input (Sec. 3).
#include <map>
#include <stdexcept>

#include "gemm_tc.h"
#include "runtime.h"

namespace lp {
namespace {

struct BlockBufs {
  std::string name;
  const void* hin = nullptr;   // set per plan
  void *a1, *qkv, *o, *h1, *a2, *u, *g;
  void* hout_internal;         // output when this is not the chunk's last block
  float *mean1, *rstd1, *mean2, *rstd2, *lse, *delta;
};
struct ChunkBufs {
  std::vector<BlockBufs> blocks;
  void* emb = nullptr;         // chunk 0: embedding output
  void *ah, *z;                // head LayerNorm output, logits / dlogits
  float *meanh, *rstdh, *row_loss;
  float2* zstats = nullptr;    // per-row softmax statistics of the logits' column groups (training, tensor-core path)
  void *G0, *G1, *G2, *Gf, *Gq;   // gradient scratch: [M,d] x3, [M,ffn], [M,3d]
};

std::string hn(int k, const char* s) { return "c" + std::to_string(k) + ".head." + s; }

}  // namespace

void build_lm(Handle& h) {
  const int K = h.K, B = h.spec.batch, T = h.spec.seq_len, d = h.spec.d_model, F = h.spec.d_ffn, V = h.spec.vocab,
            H = h.spec.n_heads;
  const int M = B * T;
  // an inner piece of a chain spread over several GPUs: x is the previous piece's activation, no embeddings
  const bool inner = h.spec.input_is_activation != 0;
  h.rows = M;
  std::vector<ChunkBufs> cb(K);
  int blk = 0;
  for (int k = 0; k < K; ++k) {
    if (k == 0 && !inner) {
      h.add_tensor("c0.tok", 0, {V, d}, true);
      h.add_tensor("c0.pos", 0, {T, d}, true);
    }
    for (int j = 0; j < h.per_chunk[k]; ++j, ++blk) {
      BlockBufs bb;
      bb.name = "c" + std::to_string(k) + ".b" + std::to_string(blk);
      const std::string& n = bb.name;
      h.add_tensor(n + ".ln1.g", k, {d}, false);
      h.add_tensor(n + ".ln1.b", k, {d}, false);
      h.add_tensor(n + ".Wqkv", k, {3 * d, d}, true);
      h.add_tensor(n + ".bqkv", k, {3 * d}, false);
      h.add_tensor(n + ".Wo", k, {d, d}, true);
      h.add_tensor(n + ".bo", k, {d}, false);
      h.add_tensor(n + ".ln2.g", k, {d}, false);
      h.add_tensor(n + ".ln2.b", k, {d}, false);
      h.add_tensor(n + ".W1", k, {F, d}, true);
      h.add_tensor(n + ".b1", k, {F}, false);
      h.add_tensor(n + ".W2", k, {d, F}, true);
      h.add_tensor(n + ".b2", k, {d}, false);
      cb[k].blocks.push_back(bb);
    }
    h.add_tensor(hn(k, "ln.g"), k, {d}, false);
    h.add_tensor(hn(k, "ln.b"), k, {d}, false);
    h.add_tensor(hn(k, "W"), k, {V, d}, true);
    h.add_tensor(hn(k, "b"), k, {V}, false);
  }
  h.finalize_arena();

  const size_t es = h.esize();
  const size_t md = (size_t)M * d * es;
  h.x_bytes = inner ? md : (size_t)M * sizeof(int);
  h.x_in = h.dalloc(h.x_bytes);
  h.y_bytes = (size_t)M * sizeof(int);
  h.y_in = (int*)h.dalloc(h.y_bytes);
  int* emb_next = (int*)h.dalloc((size_t)M * sizeof(int));
  int* emb_first = (int*)h.dalloc((size_t)M * sizeof(int));
  auto fal = [&](size_t n) { return (float*)h.dalloc(n * sizeof(float)); };
  for (int k = 0; k < K; ++k) {
    h.bnd_bytes.push_back(md);
    for (int s = 0; s < 2; ++s) {
      h.bnd[s].push_back(h.dalloc(md));
      h.lab[s].push_back((int*)h.dalloc(h.y_bytes));
    }
    h.n_valid.push_back((int*)h.dalloc(sizeof(int)));
    ChunkBufs& c = cb[k];
    if (k == 0) c.emb = inner ? h.x_in : h.dalloc(md);
    for (size_t j = 0; j < c.blocks.size(); ++j) {
      BlockBufs& b = c.blocks[j];
      b.a1 = h.dalloc(md); b.qkv = h.dalloc(3 * md); b.o = h.dalloc(md); b.h1 = h.dalloc(md); b.a2 = h.dalloc(md);
      b.u = h.dalloc((size_t)M * F * es); b.g = h.dalloc((size_t)M * F * es);
      b.hout_internal = (j + 1 < c.blocks.size()) ? h.dalloc(md) : nullptr;
      b.mean1 = fal(M); b.rstd1 = fal(M); b.mean2 = fal(M); b.rstd2 = fal(M);
      b.lse = fal((size_t)B * H * T); b.delta = fal((size_t)B * H * T);
    }
    c.ah = h.dalloc(md);
    c.z = h.dalloc((size_t)M * V * es);
    c.meanh = fal(M); c.rstdh = fal(M); c.row_loss = fal(M);
    c.G0 = h.dalloc(md); c.G1 = h.dalloc(md); c.G2 = h.dalloc(md);
    c.Gf = h.dalloc((size_t)M * F * es); c.Gq = h.dalloc(3 * md);
  }

  std::vector<int> all;
  for (int k = 0; k < K; ++k) all.push_back(k);
  const bool bf = h.bf16_mode;
  int* st = h.d_status;
  // The feed-forward pre-activation u is written by the first feed-forward product's epilogue and read only by
  // the epilogue of the second one's input gradient.  When both run on the tensor-core kernel, u is kept in
  // 32x32 blocks (see GemmProb::aux_blocked) so that both touch it with coalesced accesses.
  bool u_blocked = bf && !h.force_simt && M % 32 == 0 && F % 32 == 0 && !cb.empty() && !cb[0].blocks.empty();
  if (u_blocked) {
    BlockBufs& b0 = cb[0].blocks[0];
    GemmProb f = gemm_fwd(b0.a2, h.W(b0.name + ".W1"), b0.g, M, F, d, h.P32(b0.name + ".b1"), EPI_GELU);
    f.C2 = b0.u; f.aux_blocked = 1;
    GemmProb g2 = gemm_dgrad(cb[0].G0, h.W(b0.name + ".W2"), cb[0].Gf, M, d, F, EPI_GELU_GRAD, b0.u);
    g2.aux_blocked = 1;
    u_blocked = gemm_tc_eligible(f) && gemm_tc_eligible(g2);
  }

  auto chunk_in = [&](int k, int rd) -> const void* { return k == 0 ? cb[0].emb : h.bnd[rd][k - 1]; };
  auto block_in = [&](int k, size_t j, int rd) -> const void* {
    return j == 0 ? chunk_in(k, rd) : cb[k].blocks[j - 1].hout_internal;
  };
  auto block_out = [&](int k, size_t j, int wr) -> void* {
    return (j + 1 < cb[k].blocks.size()) ? cb[k].blocks[j].hout_internal : h.bnd[wr][k];
  };
  auto labels_of = [&](int k, bool pipelined, int rd) -> const int* {
    return (!pipelined || k == 0) ? h.y_in : h.lab[rd][k - 1];
  };

  // ---- forward of the trunks of chunks `ks`
  auto forward = [&](Plan& p, const std::vector<int>& ks, int rd, int wr) {
    for (int k : ks)
      if (k == 0 && !inner) {
        EmbedProb e{(const int*)h.x_in, h.W("c0.tok"), h.W("c0.pos"), cb[0].emb, M, T, d, V};
        p.add(1, [e, st, bf](const RunCtx& c) { launch_embed_fwd(e, st, bf, c.stream); }, KIND_EMBED, 3.0 * M * d * es);
      }
    size_t maxb = 0;
    for (int k : ks) maxb = std::max(maxb, cb[k].blocks.size());
    for (size_t j = 0; j < maxb; ++j) {
      std::vector<int> act;
      for (int k : ks) if (j < cb[k].blocks.size()) act.push_back(k);
      std::vector<LnProb> ln;
      std::vector<GemmProb> g;
      std::vector<AttnProb> at;
      for (int k : act) {
        BlockBufs& b = cb[k].blocks[j];
        ln.push_back(LnProb{block_in(k, j, rd), b.a1, h.P32(b.name + ".ln1.g"), h.P32(b.name + ".ln1.b"), b.mean1, b.rstd1, M, d});
        g.push_back(gemm_fwd(b.a1, h.W(b.name + ".Wqkv"), b.qkv, M, 3 * d, d, h.P32(b.name + ".bqkv"), EPI_NONE));
        at.push_back(AttnProb{b.qkv, b.o, b.lse, nullptr, nullptr, b.delta, B, T, H});
      }
      emit_ln_fwd(h, p, ln);
      emit_gemm(h, p, g);
      emit_attention(h, p, at, false);
      g.clear(); ln.clear();
      for (int k : act) {
        BlockBufs& b = cb[k].blocks[j];
        GemmProb q = gemm_fwd(b.o, h.W(b.name + ".Wo"), b.h1, M, d, d, h.P32(b.name + ".bo"), EPI_NONE);
        q.resid = block_in(k, j, rd);
        g.push_back(q);
        ln.push_back(LnProb{b.h1, b.a2, h.P32(b.name + ".ln2.g"), h.P32(b.name + ".ln2.b"), b.mean2, b.rstd2, M, d});
      }
      emit_gemm(h, p, g);
      emit_ln_fwd(h, p, ln);
      g.clear();
      for (int k : act) {
        BlockBufs& b = cb[k].blocks[j];
        GemmProb q = gemm_fwd(b.a2, h.W(b.name + ".W1"), b.g, M, F, d, h.P32(b.name + ".b1"), EPI_GELU);
        q.C2 = b.u;
        q.aux_blocked = u_blocked ? 1 : 0;
        g.push_back(q);
      }
      emit_gemm(h, p, g);
      g.clear();
      for (int k : act) {
        BlockBufs& b = cb[k].blocks[j];
        GemmProb q = gemm_fwd(b.g, h.W(b.name + ".W2"), block_out(k, j, wr), M, d, F, h.P32(b.name + ".b2"), EPI_NONE);
        q.resid = b.h1;
        g.push_back(q);
      }
      emit_gemm(h, p, g);
    }
  };

  // ---- heads: LayerNorm, logits, loss (+ dlogits in place)
  bool head_bias_done = false;   // the cross-entropy kernel already produced the head bias gradients
  auto heads_forward = [&](Plan& p, int wr, bool pipelined, int rd, bool copy_logits, bool train) {
    std::vector<LnProb> ln;
    std::vector<GemmProb> g;
    std::vector<XentProb> xs;
    std::vector<XentStatsProb> xst;
    // Training steps on the tensor-core path: the head GEMM leaves per-group softmax statistics next
    // to the logits, so the cross-entropy needs no reduction pass over the logits of its own.
    bool fused = train && h.bf16_mode && !h.force_simt && V % 8 == 0;
    for (int k = 0; k < K && fused; ++k) {
      GemmProb probe = gemm_fwd(cb[k].ah, h.W(hn(k, "W")), cb[k].z, M, V, d, h.P32(hn(k, "b")), EPI_LOGIT_STATS);
      fused = gemm_tc_eligible(probe) && (((uintptr_t)cb[k].z & 15) == 0);
    }
    const int groups = (V + 127) / 128;
    for (int k = 0; k < K; ++k) {
      ChunkBufs& c = cb[k];
      ln.push_back(LnProb{h.bnd[wr][k], c.ah, h.P32(hn(k, "ln.g")), h.P32(hn(k, "ln.b")), c.meanh, c.rstdh, M, d});
      g.push_back(gemm_fwd(c.ah, h.W(hn(k, "W")), c.z, M, V, d, h.P32(hn(k, "b")), fused ? EPI_LOGIT_STATS : EPI_NONE));
      if (fused) {
        if (!c.zstats) c.zstats = (float2*)h.dalloc((size_t)M * groups * sizeof(float2));
        g.back().C2 = c.zstats;
        xst.push_back(XentStatsProb{c.z, labels_of(k, pipelined, rd), h.n_valid[k], c.row_loss, c.zstats, nullptr, nullptr,
                                    M, V, V, groups});
      } else {
        xs.push_back(XentProb{c.z, labels_of(k, pipelined, rd), h.n_valid[k], c.row_loss, M, V, V, nullptr});
      }
    }
    emit_ln_fwd(h, p, ln);
    emit_gemm(h, p, g);
    if (copy_logits) {
      void* zlast = cb[K - 1].z;
      size_t zbytes = (size_t)M * V * es;
      p.add(0, [zlast, zbytes](const RunCtx& c) {
        if (c.out_logits) cudaMemcpyAsync(c.out_logits, zlast, zbytes, cudaMemcpyDeviceToDevice, c.stream);
      });
      std::vector<ArgmaxProb> am;
      for (int k = 0; k < K; ++k) am.push_back(ArgmaxProb{cb[k].z, labels_of(k, pipelined, rd), M, V, V, k});
      emit_argmax(h, p, am);
    }
    std::vector<float*> bgs;
    for (int k = 0; k < K; ++k) bgs.push_back(h.G(hn(k, "b")));
    if (fused) {
      emit_xent_from_stats(h, p, xst, all, &bgs);
      head_bias_done = true;
    } else {
      head_bias_done = emit_xent_and_loss(h, p, xs, all, train ? &bgs : nullptr);
    }
  };

  // Backward of one transformer block for a list of independent (scratch, block) pairs, as grouped launches.
  // On entry the gradient at the block output is in the scratch G0; parameter gradients go to the arena, or to
  // `second` (name -> buffer) when that is given; the gradient at the block input is left in G0 if need_dx.
  struct BwdItem {
    ChunkBufs* c; BlockBufs* b; const void* blk_in; bool need_dx; std::map<std::string, float*>* second;
  };
  auto GR = [&](const BwdItem& it, const std::string& name) -> float* {
    return it.second ? it.second->at(name) : h.G(name);
  };
  auto block_backward = [&](Plan& p, const std::vector<BwdItem>& items) {
    if (items.empty()) return;
    std::vector<GemmProb> g;
    std::vector<ColSumProb> cs;
    std::vector<float*> outs;
    // 1. feed-forward second matrix: dW2, db2, du = (dout W2) * gelu'(u)
    for (auto& it : items) {
      ChunkBufs& c = *it.c; BlockBufs& b = *it.b;
      g.push_back(gemm_wgrad(c.G0, b.g, GR(it, b.name + ".W2"), M, d, F));
      g.push_back(gemm_dgrad(c.G0, h.W(b.name + ".W2"), c.Gf, M, d, F, EPI_GELU_GRAD, b.u));
      g.back().aux_blocked = u_blocked ? 1 : 0;
      cs.push_back(ColSumProb{c.G0, nullptr, M, d, d});
      outs.push_back(GR(it, b.name + ".b2"));
    }
    emit_gemm(h, p, g); emit_colsum(h, p, cs, outs);
    g.clear(); cs.clear(); outs.clear();
    // 2. feed-forward first matrix: dW1, db1, da2
    for (auto& it : items) {
      ChunkBufs& c = *it.c; BlockBufs& b = *it.b;
      g.push_back(gemm_wgrad(c.Gf, b.a2, GR(it, b.name + ".W1"), M, F, d));
      g.push_back(gemm_dgrad(c.Gf, h.W(b.name + ".W1"), c.G1, M, F, d, EPI_NONE, nullptr));
      cs.push_back(ColSumProb{c.Gf, nullptr, M, F, F});
      outs.push_back(GR(it, b.name + ".b1"));
    }
    emit_gemm(h, p, g); emit_colsum(h, p, cs, outs);
    g.clear(); cs.clear(); outs.clear();
    // 3. LN2 backward; the residual path adds dout: dh1 -> G2
    {
      std::vector<LnBwdProb> lb;
      std::vector<float*> dgs, dbs;
      for (auto& it : items) {
        ChunkBufs& c = *it.c; BlockBufs& b = *it.b;
        lb.push_back(LnBwdProb{c.G1, b.h1, h.P32(b.name + ".ln2.g"), b.mean2, b.rstd2, c.G2, c.G0, nullptr, M, d});
        dgs.push_back(GR(it, b.name + ".ln2.g"));
        dbs.push_back(GR(it, b.name + ".ln2.b"));
      }
      emit_ln_bwd(h, p, lb, dgs, dbs);
    }
    // 4. attention output projection: dWo, dbo, do -> G1
    for (auto& it : items) {
      ChunkBufs& c = *it.c; BlockBufs& b = *it.b;
      g.push_back(gemm_wgrad(c.G2, b.o, GR(it, b.name + ".Wo"), M, d, d));
      g.push_back(gemm_dgrad(c.G2, h.W(b.name + ".Wo"), c.G1, M, d, d, EPI_NONE, nullptr));
      cs.push_back(ColSumProb{c.G2, nullptr, M, d, d});
      outs.push_back(GR(it, b.name + ".bo"));
    }
    emit_gemm(h, p, g); emit_colsum(h, p, cs, outs);
    g.clear(); cs.clear(); outs.clear();
    // 5. attention backward: dqkv -> Gq
    {
      std::vector<AttnProb> at;
      for (auto& it : items) {
        ChunkBufs& c = *it.c; BlockBufs& b = *it.b;
        at.push_back(AttnProb{b.qkv, b.o, b.lse, c.G1, c.Gq, b.delta, B, T, H});
      }
      emit_attention(h, p, at, true);
    }
    // 6. qkv projection: dWqkv, dbqkv, da1 -> G1 (needed for LN1's own parameters in every case)
    for (auto& it : items) {
      ChunkBufs& c = *it.c; BlockBufs& b = *it.b;
      g.push_back(gemm_wgrad(c.Gq, b.a1, GR(it, b.name + ".Wqkv"), M, 3 * d, d));
      g.push_back(gemm_dgrad(c.Gq, h.W(b.name + ".Wqkv"), c.G1, M, 3 * d, d, EPI_NONE, nullptr));
      cs.push_back(ColSumProb{c.Gq, nullptr, M, 3 * d, 3 * d});
      outs.push_back(GR(it, b.name + ".bqkv"));
    }
    emit_gemm(h, p, g); emit_colsum(h, p, cs, outs);
    g.clear(); cs.clear(); outs.clear();
    // 7. LN1 backward.  The block-input gradient (dh1 + LN1 path -> G0) is formed only if a
    //    caller asks for it.
    {
      std::vector<LnBwdProb> lb;
      std::vector<float*> dgs, dbs;
      for (auto& it : items) {
        ChunkBufs& c = *it.c; BlockBufs& b = *it.b;
        const bool need_dx = it.need_dx;
        lb.push_back(LnBwdProb{c.G1, it.blk_in, h.P32(b.name + ".ln1.g"), b.mean1, b.rstd1,
                               need_dx ? c.G0 : nullptr, need_dx ? c.G2 : nullptr, nullptr, M, d});
        dgs.push_back(GR(it, b.name + ".ln1.g"));
        dbs.push_back(GR(it, b.name + ".ln1.b"));
      }
      emit_ln_bwd(h, p, lb, dgs, dbs);
    }
  };

  std::vector<std::map<std::string, float*>> second_grads(K);   // overlapping updates: second gradients of chunk k's last block
  auto build_step = [&](Plan& p, bool pipelined, int rd, int wr, bool overlap) {
    std::vector<LabelProb> lps;
    for (int k = 0; k < K; ++k)
      lps.push_back(LabelProb{labels_of(k, pipelined, rd), (pipelined && k < K - 1) ? h.lab[wr][k] : nullptr, M, V,
                              h.n_valid[k]});
    emit_labels(h, p, lps);
    if (pipelined) forward(p, all, rd, wr);
    else for (int k = 0; k < K; ++k) forward(p, {k}, rd, wr);
    heads_forward(p, wr, pipelined, rd, false, true);

    // ---- head backward -> gradient at the trunk output in G0
    {
      std::vector<GemmProb> g;
      std::vector<ColSumProb> cs;
      std::vector<float*> outs;
      for (int k = 0; k < K; ++k) {
        ChunkBufs& c = cb[k];
        g.push_back(gemm_wgrad(c.z, c.ah, h.G(hn(k, "W")), M, V, d));
        g.push_back(gemm_dgrad(c.z, h.W(hn(k, "W")), c.G1, M, V, d, EPI_NONE, nullptr));
        if (!head_bias_done) {
          cs.push_back(ColSumProb{c.z, nullptr, M, V, V});
          outs.push_back(h.G(hn(k, "b")));
        }
      }
      emit_gemm(h, p, g);
      emit_colsum(h, p, cs, outs);
      std::vector<LnBwdProb> lb;
      std::vector<float*> dgs, dbs;
      for (int k = 0; k < K; ++k) {
        ChunkBufs& c = cb[k];
        lb.push_back(LnBwdProb{c.G1, h.bnd[wr][k], h.P32(hn(k, "ln.g")), c.meanh, c.rstdh, c.G0, nullptr, nullptr, M, d});
        dgs.push_back(h.G(hn(k, "ln.g")));
        dbs.push_back(h.G(hn(k, "ln.b")));
      }
      emit_ln_bwd(h, p, lb, dgs, dbs);
    }

    // ---- trunk backward, blocks aligned from the back of each chunk
    size_t maxb = 0;
    for (int k = 0; k < K; ++k) maxb = std::max(maxb, cb[k].blocks.size());
    for (size_t jj = 0; jj < maxb; ++jj) {
      std::vector<BwdItem> items;
      for (int k = 0; k < K; ++k) {
        if (jj >= cb[k].blocks.size()) continue;
        const size_t j = cb[k].blocks.size() - 1 - jj;
        // The block-input gradient is formed only if something consumes it: an earlier block of the same
        // chunk, chunk 0's embeddings, or (overlapping updates) the previous chunk's last block.
        const bool need_dx = (j > 0) || (k == 0 && !inner) || overlap;
        items.push_back(BwdItem{&cb[k], &cb[k].blocks[j], block_in(k, j, rd), need_dx, nullptr});
      }
      block_backward(p, items);
      // chunk 0, first block: embedding tables
      for (auto& it : items)
        if (!inner && it.c == &cb[0] && it.b == &cb[0].blocks[0]) {
          EmbedBwdProb e{(const int*)h.x_in, cb[0].G0, h.G("c0.tok"), h.G("c0.pos"), emb_next, emb_first, M, T, d, V, B};
          p.add(6, [e, bf](const RunCtx& c) { launch_embed_bwd(e, bf, c.stream); }, KIND_EMBED, (double)M * d * es + 4.0 * V * d);
        }
    }
    // ---- overlapping updates (Sec. 3, Fig. 2 c): chunk k's loss, whose gradient at the chunk input now sits in
    // chunk k's G0, goes on through the last block of chunk k-1 (saved activations of this very minibatch),
    // into second gradients of that block's parameters; it stops at that block's input.  The block's update
    // uses the mean of its two gradients.
    std::vector<AvgProb> avg;
    long long avg_max = 0;
    if (overlap) {
      std::vector<BwdItem> items;
      for (int k = 1; k < K; ++k) {
        const size_t j = cb[k - 1].blocks.size() - 1;
        BlockBufs* sb = &cb[k - 1].blocks[j];
        auto& second = second_grads[k - 1];
        if (second.empty())
          for (const char* suf : {".ln1.g", ".ln1.b", ".Wqkv", ".bqkv", ".Wo", ".bo", ".ln2.g", ".ln2.b", ".W1", ".b1", ".W2", ".b2"})
            second[sb->name + suf] = fal((size_t)h.tensors[h.find(sb->name + suf)].numel);
        items.push_back(BwdItem{&cb[k], sb, block_in(k - 1, j, rd), false, &second});
        for (auto& kv : second) {
          const long long n = h.tensors[h.find(kv.first)].numel;
          avg.push_back(AvgProb{h.G(kv.first), kv.second, n});
          avg_max = std::max(avg_max, n);
        }
      }
      block_backward(p, items);
    }
    emit_pending_reduce(h, p);
    if (!avg.empty()) {
      const AvgProb* dp = h.upload(avg);
      int n = (int)avg.size();
      double bytes = 0;
      for (auto& a : avg) bytes += 12.0 * a.n;
      p.add(1, [=](const RunCtx& r) { launch_average_f32(dp, n, avg_max, r.stream); }, KIND_REDUCE, bytes);
    }
    emit_optimizer(h, p);
  };

  auto build_forward = [&](Plan& p, int wr, bool heads) {
    for (int k = 0; k < K; ++k) forward(p, {k}, wr, wr);
    if (!heads) return;
    std::vector<LabelProb> lps;
    for (int k = 0; k < K; ++k) lps.push_back(LabelProb{h.y_in, nullptr, M, V, h.n_valid[k]});
    emit_labels(h, p, lps);
    heads_forward(p, wr, false, wr, true, false);
  };

  build_step(h.sync_plan, false, 0, 0, false);
  if (K > 1) {
    build_step(h.sync_overlap_plan, false, 0, 0, true);
    h.has_overlap_plan = true;
  }
  for (int par = 0; par < 2; ++par) {
    build_step(h.pipe_plan[par], true, par, 1 - par, false);
    build_forward(h.prime_plan[par], par, false);
    std::vector<LabelProb> lps;
    for (int k = 0; k + 1 < K; ++k) lps.push_back(LabelProb{h.y_in, h.lab[par][k], M, V, h.n_valid[k]});
    if (!lps.empty()) emit_labels(h, h.prime_plan[par], lps);
    build_forward(h.fwd_plan[par], par, true);
  }
}

}  // namespace lp
