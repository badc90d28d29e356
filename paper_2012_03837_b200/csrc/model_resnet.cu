// ResNet family (App. B.3): a 3x3 stem convolution + BatchNorm + ReLU in chunk 0, then one stage of residual
// blocks per chunk -- BasicBlocks (conv3x3-BN-ReLU-conv3x3-BN) or bottleneck blocks (1x1 - 3x3 - 1x1, expansion
// 4), identity or 1x1-stride-2 conv+BN shortcut, ReLU -- BatchNorm with batch statistics, and a global-average-
// pool + Linear + softmax cross-entropy auxiliary head per chunk (Sec. 3).  Activations are NHWC.  In bf16 the
// 3x3 and 1x1 convolutions with channel counts that are multiples of 64 are implicit GEMMs on the tensor cores
// (no im2col), 1x1 stride-1 convolutions plain GEMMs over [pixels, C], the few-channel stem a direct FP32-ALU
// kernel; everything else (fp32, the FP32-ALU backend, other channel counts) is im2col + GEMM with the cols kept
// for the weight gradient and a GEMM + col2im gather for an input gradient.  BatchNorm is one cooperative launch
// per layer (forward) and per grouped position (backward) in bf16, three launches otherwise.
//
// Backward is truncated at the chunk input (Sec. 3): the first block of a stage k > 0 forms no input
// gradient (no dgrad for its first convolution and its shortcut convolution), nor does the stem.
// The synchronous schedule is the natural one here; the pipelined plans are built too.
#include <map>
#include <stdexcept>

#include "runtime.h"

namespace lp {
namespace {

struct Conv {
  std::string w;
  int Cin, Cout, k, stride, pad, H, W, Ho, Wo, N;
  long long M;   // N*Ho*Wo
  int K;         // k*k*Cin
  int ldk;       // pitch of the cols matrix: K rounded up to 8 elements (16 bytes for bf16), pad columns stay zero
  void* cols = nullptr;
  void* y = nullptr;
  // implicit GEMM on the tensor-core kernel (no im2col / col2im): forward and weight gradient, input gradient
  bool imp_fwd = false, imp_dgrad = false;
  // few-channel direct convolution on the FP32 ALUs (the stem): forward and filter gradient, no im2col
  bool small = false;
  // 1x1, stride 1: the NHWC activation [pixels, Cin] is the GEMM operand as it stands, in every backend
  bool pointwise = false;
};
struct Bn {
  std::string g, b;
  int C;
  long long rows;
  float *mean, *rstd;
};
struct Block {
  Conv c1, c2, c3, cs;                                   // c3: third convolution of a bottleneck block
  Bn b1, b2, b3, bs;
  bool has_sc = false, bottleneck = false;
  void *a1 = nullptr, *a2 = nullptr, *sc = nullptr, *out = nullptr;   // out is null for the chunk's last block (boundary buffer)
  const Conv& last() const { return bottleneck ? c3 : c2; }
  const Bn& last_bn() const { return bottleneck ? b3 : b2; }
};
struct Chunk {
  bool has_stem = false;
  Conv stem;
  Bn stem_bn;
  void *x_nhwc = nullptr, *stem_out = nullptr;
  std::vector<Block> blocks;
  int C, Hout, Wout;
  void *pool, *z, *dpool;
  Bn head_bn;                                  // LP_HEAD_BN_RELU_GAP_LINEAR: BatchNorm + ReLU in front of the pool
  void* hact = nullptr;                        // its output
  float* row_loss;
  void* G[4];
  void* dcols;
  // overlapping updates: scratch for the second backward pass through the previous stage's last block
  void* GO[3] = {nullptr, nullptr, nullptr};
  void* dcolsO = nullptr;
  std::map<std::string, float*> second;        // second gradients of THIS chunk's last block (filled by chunk k+1's loss)
};

// Backward passes of the chunks are independent of one another (Sec. 3): each chunk records its backward
// as a list of ops, and the lists are emitted in lockstep, ops of the same kind at the same position
// sharing one grouped launch.
enum OpKind { OP_NOP = 0, OP_GEMM, OP_COLSUM, OP_GAP_BWD, OP_BN_BWD, OP_ADD, OP_RAW };
struct Op {
  OpKind kind = OP_NOP;
  std::vector<GemmProb> gemms;                       // OP_GEMM
  ColSumProb colsum{}; float* colsum_out = nullptr;  // OP_COLSUM
  GapProb gap{}; long long elems = 0;                // OP_GAP_BWD (elems also: OP_BN_BWD, OP_ADD)
  BnStatProb bn_stat{}; BnFinalProb bn_final{}; BnApplyProb bn_apply{}; bool v8 = false; double work = 0;  // OP_BN_BWD
  AddProb add{};                                     // OP_ADD
  std::function<void(Plan&)> raw;                    // OP_RAW: emitted on its own
};
typedef std::vector<Op> OpList;

Conv make_conv(const std::string& w, int N, int H, int W, int Cin, int Cout, int k, int stride) {
  Conv c;
  c.w = w; c.N = N; c.H = H; c.W = W; c.Cin = Cin; c.Cout = Cout; c.k = k; c.stride = stride; c.pad = k / 2;
  c.Ho = (H + 2 * c.pad - k) / stride + 1;
  c.Wo = (W + 2 * c.pad - k) / stride + 1;
  c.M = (long long)N * c.Ho * c.Wo;
  c.K = k * k * Cin;
  c.ldk = (c.K + 7) / 8 * 8;
  c.pointwise = k == 1 && stride == 1;
  return c;
}

}  // namespace

void build_resnet(Handle& h) {
  const int K = h.K, B = h.spec.batch, NC = h.head.classes;
  const bool bf = h.bf16_mode;
  const bool head_bn = h.head.kind == LP_HEAD_BN_RELU_GAP_LINEAR;   // App. B.3's head
  const size_t es = h.esize();
  // an inner piece of a chain spread over several GPUs: x is the previous stage's NHWC activation, there is no
  // stem, and the first stage is a later stage of the network (stride 2, 1x1 shortcut)
  const bool inner = h.spec.input_is_activation != 0;
  std::vector<Chunk> ch(K);
  int H = h.spec.height, W = h.spec.width, cprev = inner ? h.spec.in_channels : h.spec.stem_channels;
  for (int k = 0; k < K; ++k) {
    Chunk& c = ch[k];
    const std::string ck = "c" + std::to_string(k);
    if (k == 0 && !inner) {
      c.has_stem = true;
      c.stem = make_conv("c0.stem.conv", B, H, W, h.spec.in_channels, cprev, 3, 1);
      h.add_tensor("c0.stem.conv", 0, {cprev, 3, 3, h.spec.in_channels}, true);
      h.add_tensor("c0.stem.bn.g", 0, {cprev}, false);
      h.add_tensor("c0.stem.bn.b", 0, {cprev}, false);
      c.stem_bn = Bn{"c0.stem.bn.g", "c0.stem.bn.b", cprev, c.stem.M, nullptr, nullptr};
    }
    const bool bottleneck = h.spec.block_kind == LP_BLOCK_BOTTLENECK;
    const int cmid = h.stage_channels[k];
    int cout = bottleneck ? 4 * cmid : cmid;                 // a bottleneck block leaves four times its inner width
    for (int j = 0; j < h.stage_blocks[k]; ++j) {
      Block b;
      b.bottleneck = bottleneck;
      const std::string p = ck + ".r" + std::to_string(j);
      int stride = (j == 0 && (k > 0 || inner)) ? 2 : 1;
      int cin = j == 0 ? cprev : cout;
      auto add_bn = [&](const std::string& n, int C, long long rows) {
        h.add_tensor(n + ".g", k, {C}, false);
        h.add_tensor(n + ".b", k, {C}, false);
        return Bn{n + ".g", n + ".b", C, rows, nullptr, nullptr};
      };
      if (bottleneck) {
        b.c1 = make_conv(p + ".conv1", B, H, W, cin, cmid, 1, 1);
        h.add_tensor(p + ".conv1", k, {cmid, 1, 1, cin}, true);
        b.b1 = add_bn(p + ".bn1", cmid, b.c1.M);
        b.c2 = make_conv(p + ".conv2", B, H, W, cmid, cmid, 3, stride);
        h.add_tensor(p + ".conv2", k, {cmid, 3, 3, cmid}, true);
        b.b2 = add_bn(p + ".bn2", cmid, b.c2.M);
        b.c3 = make_conv(p + ".conv3", B, b.c2.Ho, b.c2.Wo, cmid, cout, 1, 1);
        h.add_tensor(p + ".conv3", k, {cout, 1, 1, cmid}, true);
        b.b3 = add_bn(p + ".bn3", cout, b.c3.M);
      } else {
        b.c1 = make_conv(p + ".conv1", B, H, W, cin, cout, 3, stride);
        h.add_tensor(p + ".conv1", k, {cout, 3, 3, cin}, true);
        b.b1 = add_bn(p + ".bn1", cout, b.c1.M);
        b.c2 = make_conv(p + ".conv2", B, b.c1.Ho, b.c1.Wo, cout, cout, 3, 1);
        h.add_tensor(p + ".conv2", k, {cout, 3, 3, cout}, true);
        b.b2 = add_bn(p + ".bn2", cout, b.c2.M);
      }
      b.has_sc = j == 0 && (stride != 1 || cin != cout);
      if (b.has_sc) {
        b.cs = make_conv(p + ".sc.conv", B, H, W, cin, cout, 1, stride);
        h.add_tensor(p + ".sc.conv", k, {cout, 1, 1, cin}, true);
        h.add_tensor(p + ".sc.bn.g", k, {cout}, false);
        h.add_tensor(p + ".sc.bn.b", k, {cout}, false);
        b.bs = Bn{p + ".sc.bn.g", p + ".sc.bn.b", cout, b.cs.M, nullptr, nullptr};
      }
      H = b.last().Ho; W = b.last().Wo;
      c.blocks.push_back(b);
    }
    cprev = cout;
    c.C = cout; c.Hout = H; c.Wout = W;
    h.add_tensor(ck + ".head.W", k, {NC, cout}, true);
    h.add_tensor(ck + ".head.b", k, {NC}, false);
    if (head_bn) {
      h.add_tensor(ck + ".head.bn.g", k, {cout}, false);
      h.add_tensor(ck + ".head.bn.b", k, {cout}, false);
      c.head_bn = Bn{ck + ".head.bn.g", ck + ".head.bn.b", cout, (long long)B * H * W, nullptr, nullptr};
    }
  }
  // running mean / variance of every BatchNorm: state no gradient reaches (their gradient entries stay
  // zero, so the optimizer sweep leaves them alone); they live in the arena so that tensor access and
  // checkpoints cover them
  {
    std::vector<std::pair<std::string, std::pair<int, int64_t>>> bns;
    for (auto& t : h.tensors)
      if (t.name.size() > 2 && t.name.compare(t.name.size() - 2, 2, ".g") == 0 && t.name.find(".bn") != std::string::npos)
        bns.push_back({t.name.substr(0, t.name.size() - 2), {t.chunk, t.numel}});
    for (auto& b : bns) {
      h.add_tensor(b.first + ".rm", b.second.first, {b.second.second}, false);
      h.add_tensor(b.first + ".rv", b.second.first, {b.second.second}, false);
    }
  }
  h.finalize_arena();
  h.rows = B;

  // ---- buffers
  const size_t in_elems = (size_t)B * h.spec.in_channels * h.spec.height * h.spec.width;
  h.x_bytes = in_elems * es;
  h.x_in = h.dalloc(h.x_bytes);
  h.y_bytes = (size_t)B * sizeof(int);
  h.y_in = (int*)h.dalloc(h.y_bytes);
  auto fal = [&](size_t n) { return (float*)h.dalloc(n * sizeof(float)); };
  if (bf) {
    h.bn_fused_blocks[0] = bn_fused_max_blocks(h.num_sms, false);
    h.bn_fused_blocks[1] = bn_fused_max_blocks(h.num_sms, true);
    h.d_grid_counter = (unsigned long long*)h.dalloc(2 * sizeof(unsigned long long));
  }
  const int bn_blocks_fused = h.bn_fused_blocks[0], bn_blocks_fused_bwd = h.bn_fused_blocks[1];
  unsigned long long* const grid_counter = h.d_grid_counter;
  int* const d_status = h.d_status;
  // 3x3 (padding 1) and 1x1 convolutions with stride 1 or 2 whose input channel count is a multiple of 64 run
  // as implicit GEMMs: the activation tensor itself is the operand (TMA boxes that step through it with the
  // stride, one shifted box per filter tap), nothing 9 times its size is written.  Forward and filter gradient
  // for both strides; the input gradient in this form for the 3x3 stride-1 convolutions (the stride-2
  // convolutions open a stage, so their input gradient is only needed by the overlapping variant).
  auto set_implicit = [&](Conv& c) {
    const bool shape = (c.k == 3 && c.pad == 1) || (c.k == 1 && c.pad == 0);
    const bool base = bf && !h.force_simt && shape && (c.stride == 1 || c.stride == 2) && conv_boxes_ok(c.Ho, c.Wo) &&
                      c.Wo * c.stride <= 256;
    c.imp_fwd = base && c.Cin % 64 == 0 && c.Cout % 8 == 0;
    c.imp_dgrad = base && c.k == 3 && c.stride == 1 && c.Cout % 64 == 0 && c.Cin % 8 == 0;
  };
  auto alloc_conv = [&](Conv& c) {
    set_implicit(c);
    if (!c.imp_fwd && !c.small && !c.pointwise) c.cols = h.dalloc((size_t)c.M * c.ldk * es);
    c.y = h.dalloc((size_t)c.M * c.Cout * es);
  };
  auto alloc_bn = [&](Bn& b) { b.mean = fal(b.C); b.rstd = fal(b.C); };
  for (int k = 0; k < K; ++k) {
    Chunk& c = ch[k];
    size_t out_bytes = (size_t)B * c.Hout * c.Wout * c.C * es;
    h.bnd_bytes.push_back(out_bytes);
    for (int s = 0; s < 2; ++s) {
      h.bnd[s].push_back(h.dalloc(out_bytes));
      h.lab[s].push_back((int*)h.dalloc(h.y_bytes));
    }
    h.n_valid.push_back((int*)h.dalloc(sizeof(int)));
    size_t max_act = 0, max_cols = 0;
    auto track = [&](const Conv& cv) {
      max_act = std::max(max_act, (size_t)cv.M * cv.Cout);
      max_act = std::max(max_act, (size_t)cv.N * cv.H * cv.W * cv.Cin);
      if (!cv.imp_dgrad && !cv.pointwise) max_cols = std::max(max_cols, (size_t)cv.M * cv.ldk);
    };
    if (c.has_stem) {
      c.x_nhwc = h.dalloc(in_elems * es);
      c.stem.small = c.stem.k == 3 && c.stem.stride == 1 && 9 * c.stem.Cin <= 32 && c.stem.Cout % 8 == 0 &&
                     c.stem.Cout <= 64 && 256 % c.stem.Cout == 0 && c.stem.M < (1LL << 30);
      alloc_conv(c.stem); alloc_bn(c.stem_bn); track(c.stem);
      c.stem_out = h.dalloc((size_t)c.stem.M * c.stem.Cout * es);
    }
    for (size_t j = 0; j < c.blocks.size(); ++j) {
      Block& b = c.blocks[j];
      alloc_conv(b.c1); alloc_bn(b.b1); track(b.c1);
      alloc_conv(b.c2); alloc_bn(b.b2); track(b.c2);
      b.a1 = h.dalloc((size_t)b.c1.M * b.c1.Cout * es);
      if (b.bottleneck) {
        alloc_conv(b.c3); alloc_bn(b.b3); track(b.c3);
        b.a2 = h.dalloc((size_t)b.c2.M * b.c2.Cout * es);
      }
      if (b.has_sc) { alloc_conv(b.cs); alloc_bn(b.bs); track(b.cs); b.sc = h.dalloc((size_t)b.cs.M * b.cs.Cout * es); }
      if (j + 1 < c.blocks.size()) b.out = h.dalloc((size_t)b.last().M * b.last().Cout * es);
    }
    if (head_bn) { alloc_bn(c.head_bn); c.hact = h.dalloc(out_bytes); }
    c.pool = h.dalloc((size_t)B * c.C * es);
    c.dpool = h.dalloc((size_t)B * c.C * es);
    c.z = h.dalloc((size_t)B * NC * es);
    c.row_loss = fal(B);
    for (int i = 0; i < 4; ++i) c.G[i] = h.dalloc(max_act * es);
    c.dcols = max_cols ? h.dalloc(max_cols * es) : nullptr;
  }

  // ---- op emitters (one problem per launch: the stages differ in every size)
  auto conv_fields = [&](GemmProb& g, const Conv& c, int mode, int channels) {
    g.conv = mode; g.conv_n = c.N; g.conv_h = c.Ho; g.conv_w = c.Wo; g.conv_c = channels; g.conv_k0 = 0;
    g.conv_hin = c.H; g.conv_win = c.W; g.conv_stride = c.stride; g.conv_taps = c.k * c.k;
  };
  auto conv_fwd = [&](Plan& p, const Conv& c, const void* x) {
    if (c.small) {
      SmallConvProb sp{x, h.W(c.w), c.y, nullptr, nullptr, c.N, c.H, c.W, c.Cin, c.Cout};
      p.add(1, [=](const RunCtx& r) { launch_small_conv_fwd(sp, bf, bf, r.stream); }, KIND_GEMM_ALU, 2.0 * c.M * c.Cout * c.K);
      return;
    }
    if (c.pointwise) {                                       // y [pixels, Cout] = x [pixels, Cin] W^T
      emit_gemm(h, p, {gemm_fwd(x, h.W(c.w), c.y, (int)c.M, c.Cout, c.Cin, nullptr, EPI_NONE)});
      return;
    }
    if (c.imp_fwd) {
      GemmProb g = gemm_fwd(x, h.W(c.w), c.y, (int)c.M, c.Cout, c.K, nullptr, EPI_NONE);
      g.a_ms = c.Cin;
      conv_fields(g, c, CONV_FWD, c.Cin);
      emit_gemm(h, p, {g});
      return;
    }
    Im2colProb ip{x, c.cols, c.N, c.H, c.W, c.Cin, c.k, c.k, c.stride, c.pad, c.Ho, c.Wo, c.ldk};
    const Im2colProb* d = h.upload(std::vector<Im2colProb>{ip});
    long long elems = c.M * c.K;
    bool v8 = bf && c.Cin % 8 == 0;
    p.add(1, [=](const RunCtx& r) { launch_im2col(d, 1, elems, bf, r.stream, v8); }, KIND_CONV_AUX, (double)elems * es * (1.0 + 1.0 / (c.k * c.k)));
    GemmProb g = gemm_fwd(c.cols, h.W(c.w), c.y, (int)c.M, c.Cout, c.K, nullptr, EPI_NONE);
    g.a_ms = c.ldk;
    emit_gemm(h, p, {g});
  };
  // BatchNorm modes of a forward pass: batch statistics only (priming, lp_forward), batch statistics that
  // also move the running averages (training steps), running statistics (evaluation)
  enum { BN_BATCH = 0, BN_TRAIN = 1, BN_RUNNING = 2 };
  auto bn_fwd = [&](Plan& p, const Bn& b, const void* x, void* y, const void* res, bool relu, int mode) {
    int nblk = bn_blocks(b.rows);
    float* part = mode == BN_RUNNING ? nullptr : fal((size_t)nblk * 2 * b.C);
    float *rm = nullptr, *rv = nullptr;
    if (mode != BN_BATCH) {
      const std::string stem = b.g.substr(0, b.g.size() - 2);      // "...bn.g" -> "...bn"
      rm = h.P32(stem + ".rm"); rv = h.P32(stem + ".rv");
    }
    BnStatProb sp{x, nullptr, nullptr, nullptr, nullptr, part, (int)b.rows, b.C};
    BnFinalProb fp{part, nblk, (int)b.rows, b.C, b.mean, b.rstd, nullptr, nullptr, 1e-5f, rm, rv, 0.1f, mode == BN_RUNNING ? 1 : 0,
                   mode == BN_TRAIN ? h.d_chunk_tab : nullptr, h.tensors[h.find(b.g)].chunk};
    BnApplyProb ap{x, y, res, h.P32(b.g), h.P32(b.b), b.mean, b.rstd, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                   (int)b.rows, b.C, relu ? 1 : 0};
    const BnStatProb* ds = h.upload(std::vector<BnStatProb>{sp});
    const BnFinalProb* df = h.upload(std::vector<BnFinalProb>{fp});
    const BnApplyProb* da = h.upload(std::vector<BnApplyProb>{ap});
    int C = b.C;
    bool v8 = bf && C % 8 == 0 && C / 8 <= 256;
    long long elems = b.rows * b.C;
    const bool stats = mode != BN_RUNNING;
    if (v8 && bn_blocks_fused > 0) {                     // the three passes as one cooperative launch
      BnFinalProb ff = fp;
      ff.nblk = std::min(nblk, bn_blocks_fused);         // one partial row per block of the launch
      const BnFusedProb* dfp = h.upload(std::vector<BnFusedProb>{BnFusedProb{sp, ff, ap}});
      // (should the cooperative launch be refused -- the device cannot hold the grid right now -- the three
      // separate launches do the same work; their partial sums use one row per block of rows)
      p.add(1, [=](const RunCtx& r) {
        if (launch_bn_fused(dfp, 1, false, stats, bn_blocks_fused, grid_counter, d_status, r.stream) == cudaSuccess) return;
        cudaGetLastError();
        if (stats) launch_bn_stat_partial(ds, 1, nblk, C, false, bf, r.stream, v8);
        launch_bn_finalize(df, 1, C, false, r.stream);
        launch_bn_apply(da, 1, elems, false, bf, r.stream, v8);
      }, KIND_NORM, (double)elems * es * ((stats ? 3 : 2) + (res ? 1 : 0)));
      return;
    }
    p.add(stats ? 3 : 2, [=](const RunCtx& r) {
      if (stats) launch_bn_stat_partial(ds, 1, nblk, C, false, bf, r.stream, v8);
      launch_bn_finalize(df, 1, C, false, r.stream);
      launch_bn_apply(da, 1, elems, false, bf, r.stream, v8);
    }, KIND_NORM, (double)elems * es * ((stats ? 3 : 2) + (res ? 1 : 0)));
  };

  auto chunk_in = [&](int k, int rd) -> const void* { return k == 0 ? (inner ? h.x_in : ch[0].stem_out) : h.bnd[rd][k - 1]; };
  auto labels_of = [&](int k, bool pipelined, int rd) -> const int* {
    return (!pipelined || k == 0) ? h.y_in : h.lab[rd][k - 1];
  };

  auto forward_chunk = [&](Plan& p, int k, int rd, int wr, int mode) {
    Chunk& c = ch[k];
    if (c.has_stem) {
      LayoutProb lp{h.x_in, c.x_nhwc, B, h.spec.in_channels, h.spec.height, h.spec.width};
      p.add(1, [=](const RunCtx& r) { launch_nchw_to_nhwc(lp, bf, r.stream); }, KIND_CONV_AUX, 2.0 * in_elems * es);
      conv_fwd(p, c.stem, c.x_nhwc);
      bn_fwd(p, c.stem_bn, c.stem.y, c.stem_out, nullptr, true, mode);
    }
    const void* x = chunk_in(k, rd);
    for (size_t j = 0; j < c.blocks.size(); ++j) {
      Block& b = c.blocks[j];
      void* out = b.out ? b.out : h.bnd[wr][k];
      conv_fwd(p, b.c1, x);
      bn_fwd(p, b.b1, b.c1.y, b.a1, nullptr, true, mode);
      conv_fwd(p, b.c2, b.a1);
      if (b.bottleneck) {
        bn_fwd(p, b.b2, b.c2.y, b.a2, nullptr, true, mode);
        conv_fwd(p, b.c3, b.a2);
      }
      const void* res = x;
      if (b.has_sc) {
        conv_fwd(p, b.cs, x);
        bn_fwd(p, b.bs, b.cs.y, b.sc, nullptr, false, mode);
        res = b.sc;
      }
      bn_fwd(p, b.last_bn(), b.last().y, out, res, true, mode);
      x = out;
    }
  };

  // The heads of all chunks (Sec. 3: each reads only its own chunk's output): one grouped launch per step of the
  // head -- spatial means, logits, predictions (evaluation), cross-entropy and losses.
  auto heads_forward = [&](Plan& p, int wr, const std::function<const int*(int)>& labels, bool copy_logits, int mode) {
    std::vector<GapProb> gaps;
    std::vector<GemmProb> logits;
    std::vector<ArgmaxProb> am;
    std::vector<XentProb> xs;
    std::vector<int> all_chunks;
    double gap_bytes = 0;
    int gap_c = 0;
    for (int k = 0; k < K; ++k) {
      Chunk& c = ch[k];
      const std::string ck = "c" + std::to_string(k);
      if (head_bn) bn_fwd(p, c.head_bn, h.bnd[wr][k], c.hact, nullptr, true, mode);
      gaps.push_back(GapProb{head_bn ? c.hact : h.bnd[wr][k], c.pool, nullptr, nullptr, B, c.Hout * c.Wout, c.C});
      gap_bytes += (double)B * c.Hout * c.Wout * c.C * es;
      gap_c = std::max(gap_c, c.C);
      logits.push_back(gemm_fwd(c.pool, h.W(ck + ".head.W"), c.z, B, NC, c.C, h.P32(ck + ".head.b"), EPI_NONE));
      am.push_back(ArgmaxProb{c.z, labels(k), B, NC, NC, k});
      xs.push_back(XentProb{c.z, labels(k), h.n_valid[k], c.row_loss, B, NC, NC, nullptr});
      all_chunks.push_back(k);
    }
    const GapProb* dg = h.upload(gaps);
    p.add(1, [=](const RunCtx& r) { launch_gap_fwd(dg, K, B, gap_c, bf, r.stream); }, KIND_CONV_AUX, gap_bytes);
    emit_gemm(h, p, logits);
    if (copy_logits) {
      void* zlast = ch[K - 1].z;
      size_t zbytes = (size_t)B * NC * es;
      p.add(0, [zlast, zbytes](const RunCtx& r) {
        if (r.out_logits) cudaMemcpyAsync(r.out_logits, zlast, zbytes, cudaMemcpyDeviceToDevice, r.stream);
      });
      emit_argmax(h, p, am);
    }
    emit_xent_and_loss(h, p, xs, all_chunks);
  };

  // ---- backward, recorded per chunk and emitted in lockstep
  // where a parameter gradient goes: the arena, or a second buffer (overlapping updates)
  typedef std::map<std::string, float*> GradMap;
  auto GD = [&](const GradMap* second, const std::string& name) -> float* { return second ? second->at(name) : h.G(name); };
  auto wgrad_prob = [&](const Conv& c, const void* dy, const void* x, const GradMap* second = nullptr) {
    if (c.pointwise) return gemm_wgrad(dy, x, GD(second, c.w), (int)c.M, c.Cout, c.Cin);
    if (c.imp_fwd) {
      GemmProb g = gemm_wgrad(dy, x, GD(second, c.w), (int)c.M, c.Cout, c.K);
      g.b_ks = c.Cin;
      conv_fields(g, c, CONV_WGRAD, c.Cin);
      return g;
    }
    GemmProb g = gemm_wgrad(dy, c.cols, GD(second, c.w), (int)c.M, c.Cout, c.K);
    g.b_ks = c.ldk;
    return g;
  };
  // the input gradient of a convolution: its GEMM problem and, for the explicit form, the col2im gather after it
  auto dgrad_prob = [&](const Conv& c, const void* dy, void* dx, void* dcols, Op& gather) {
    gather = Op{};
    if (c.pointwise) return gemm_dgrad(dy, h.W(c.w), dx, (int)c.M, c.Cout, c.Cin, EPI_NONE, nullptr);
    if (c.imp_dgrad) {
      GemmProb g{};
      g.A = dy; g.B = h.W(c.w); g.C = dx;
      g.M = (int)c.M; g.N = c.Cin; g.K = 9 * c.Cout;
      g.a_ms = c.Cout; g.a_ks = 1; g.b_ns = 1; g.b_ks = 9LL * c.Cin; g.ldc = c.Cin;
      conv_fields(g, c, CONV_DGRAD, c.Cout);
      return g;
    }
    GemmProb g = gemm_dgrad(dy, h.W(c.w), dcols, (int)c.M, c.Cout, c.K, EPI_NONE, nullptr);
    g.ldc = c.ldk;
    Im2colProb ip{dx, dcols, c.N, c.H, c.W, c.Cin, c.k, c.k, c.stride, c.pad, c.Ho, c.Wo, c.ldk};
    long long elems = (long long)c.N * c.H * c.W * c.Cin;
    bool v8 = bf && c.Cin % 8 == 0;
    double work = (double)(elems + c.M * c.K) * es;
    gather.kind = OP_RAW;
    gather.raw = [=, &h](Plan& p) {
      const Im2colProb* d = h.upload(std::vector<Im2colProb>{ip});
      p.add(1, [=](const RunCtx& r) { launch_col2im(d, 1, elems, bf, r.stream, v8); }, KIND_CONV_AUX, work);
    };
    return g;
  };
  auto rec_gemm = [&](OpList& L, std::vector<GemmProb> g) {
    Op o; o.kind = OP_GEMM; o.gemms = std::move(g); L.push_back(std::move(o));
  };
  auto rec_nop = [&](OpList& L, int n = 1) { for (int i = 0; i < n; ++i) L.push_back(Op{}); };
  // dx = BN'(dy masked by relu_out > 0); dres (optional) receives the masked dy
  auto rec_bn_bwd = [&](OpList& L, const Bn& b, const void* x, const void* dy, const void* relu_out, void* dx, void* dres,
                        const GradMap* second = nullptr) {
    int nblk = bn_blocks(b.rows);
    float* part = fal((size_t)nblk * 2 * b.C);
    float *dg = GD(second, b.g), *db = GD(second, b.b);
    Op o; o.kind = OP_BN_BWD;
    o.bn_stat = BnStatProb{x, dy, b.mean, b.rstd, relu_out, part, (int)b.rows, b.C};
    o.bn_final = BnFinalProb{part, nblk, (int)b.rows, b.C, nullptr, nullptr, dg, db, 1e-5f, nullptr, nullptr, 0.f, 0, nullptr, 0};
    o.bn_apply = BnApplyProb{x, nullptr, nullptr, h.P32(b.g), h.P32(b.b), b.mean, b.rstd, dy, relu_out, dx, dres, dg, db,
                             (int)b.rows, b.C, 0};
    o.v8 = bf && b.C % 8 == 0 && b.C / 8 <= 256;
    o.elems = b.rows * b.C;
    o.work = (double)o.elems * es * (5 + (relu_out ? 2 : 0) + (dres ? 1 : 0));
    L.push_back(std::move(o));
  };
  auto rec_add = [&](OpList& L, void* acc, const void* other, long long n) {
    Op o; o.kind = OP_ADD; o.add = AddProb{acc, other, acc, n}; o.elems = n; L.push_back(std::move(o));
  };

  // Backward of one BasicBlock, recorded: on entry the gradient at the block output is in gin; parameter
  // gradients go to the arena or to `second`; if need_dx the gradient at the block input ends up in the
  // buffer returned (one of gin / gc), otherwise no input gradient is formed (Sec. 3).
  auto rec_block_bwd = [&](OpList& L, Block& b, const void* x, const void* out, bool need_dx, void* gin, void* ga, void* gb,
                           void* gc, void* dcols, const GradMap* second) -> void* {
    long long in_elems_blk = (long long)b.c1.N * b.c1.H * b.c1.W * b.c1.Cin;
    Op gather;
    if (b.bottleneck) {
      // out = relu(bn3(c3) + shortcut): ga <- d(c3), gb <- gradient of the shortcut branch
      rec_bn_bwd(L, b.b3, b.c3.y, gin, out, ga, gb, second);
      {                                                   // dW(c3) and gc <- d(a2)
        GemmProb dg = dgrad_prob(b.c3, ga, gc, dcols, gather);
        rec_gemm(L, {wgrad_prob(b.c3, ga, b.a2, second), dg});
        L.push_back(gather);
      }
      rec_bn_bwd(L, b.b2, b.c2.y, gc, b.a2, ga, nullptr, second);   // ga <- d(c2)
    } else {
      // out = relu(bn2(c2) + shortcut): ga <- d(c2), gb <- gradient of the shortcut branch
      rec_bn_bwd(L, b.b2, b.c2.y, gin, out, ga, gb, second);
    }
    {                                                     // dW(c2) and gc <- d(a1) read the same ga: one launch
      GemmProb dg = dgrad_prob(b.c2, ga, gc, dcols, gather);
      rec_gemm(L, {wgrad_prob(b.c2, ga, b.a1, second), dg});
      L.push_back(gather);
    }
    rec_bn_bwd(L, b.b1, b.c1.y, gc, b.a1, ga, nullptr, second);   // ga <- d(c1)
    if (need_dx) {                                        // gc <- d(x) through the main branch
      GemmProb dg = dgrad_prob(b.c1, ga, gc, dcols, gather);
      rec_gemm(L, {wgrad_prob(b.c1, ga, x, second), dg});
      L.push_back(gather);
    } else {
      rec_gemm(L, {wgrad_prob(b.c1, ga, x, second)});
      rec_nop(L);
    }
    if (b.has_sc) {
      rec_bn_bwd(L, b.bs, b.cs.y, gb, nullptr, ga, nullptr, second);   // ga <- d(cs)
      if (need_dx) {
        GemmProb dg = dgrad_prob(b.cs, ga, gin, dcols, gather);   // gin <- d(x) through the shortcut
        rec_gemm(L, {wgrad_prob(b.cs, ga, x, second), dg});
        L.push_back(gather);
        rec_add(L, gc, gin, in_elems_blk);
      } else {
        rec_gemm(L, {wgrad_prob(b.cs, ga, x, second)});
        rec_nop(L, 2);
      }
    } else {
      rec_nop(L, 3);
      if (need_dx) rec_add(L, gc, gb, in_elems_blk); else rec_nop(L);
    }
    return gc;                                            // the block-input gradient (if formed)
  };

  // Every chunk's list has the same kind (or a gap) at every position it shares with another chunk's.
  std::vector<AvgProb> overlap_avg;                       // filled while an overlapping plan is recorded
  auto record_backward = [&](OpList& L, int k, int rd, int wr, bool overlap) {
    Chunk& c = ch[k];
    const std::string ck = "c" + std::to_string(k);
    // head: dW_h, db_h, d(pool), then the pool's gradient spread over H*W -> G[0]
    rec_gemm(L, {gemm_wgrad(c.z, c.pool, h.G(ck + ".head.W"), B, NC, c.C),
                 gemm_dgrad(c.z, h.W(ck + ".head.W"), c.dpool, B, NC, c.C, EPI_NONE, nullptr)});
    { Op o; o.kind = OP_COLSUM; o.colsum = ColSumProb{c.z, nullptr, B, NC, NC}; o.colsum_out = h.G(ck + ".head.b"); L.push_back(std::move(o)); }
    { Op o; o.kind = OP_GAP_BWD; o.gap = GapProb{nullptr, nullptr, c.dpool, head_bn ? c.G[3] : c.G[0], B, c.Hout * c.Wout, c.C};
      o.elems = (long long)B * c.Hout * c.Wout * c.C; L.push_back(std::move(o)); }
    // head BatchNorm + ReLU: G[3] holds the gradient at their output, G[0] receives the one at the stage output
    if (head_bn) rec_bn_bwd(L, c.head_bn, h.bnd[wr][k], c.G[3], c.hact, c.G[0], nullptr);
    void *gin = c.G[0], *ga = c.G[1], *gb = c.G[2], *gc = c.G[3];
    for (int j = (int)c.blocks.size() - 1; j >= 0; --j) {
      Block& b = c.blocks[j];
      const void* x = j == 0 ? chunk_in(k, rd) : c.blocks[j - 1].out;
      const void* out = b.out ? b.out : h.bnd[wr][k];
      // the stage-input gradient is needed by the stem (chunk 0) or, with overlapping updates, by the previous
      // stage's last block
      bool need_dx = (j > 0) || c.has_stem || (overlap && k > 0);
      void* dxbuf = rec_block_bwd(L, b, x, out, need_dx, gin, ga, gb, gc, c.dcols, nullptr);
      gc = gin; gin = dxbuf;                                // the block-input gradient feeds the next (earlier) block
    }
    if (overlap && k > 0) {
      // Overlapping local parallelism (Sec. 3, Fig. 2 c): this stage's loss goes on through the last BasicBlock of
      // stage k-1 (activations of this very minibatch) into second gradients of its parameters and stops at
      // that block's input; the block's update uses the mean of its two gradients.
      Chunk& q = ch[k - 1];
      Block& sb = q.blocks.back();
      const size_t nb = q.blocks.size();
      const void* sx = nb == 1 ? chunk_in(k - 1, rd) : q.blocks[nb - 2].out;
      if (!c.GO[0]) {
        size_t act = 0, cols = 0;
        for (const Conv* cv : {&sb.c1, &sb.c2, &sb.c3, &sb.cs}) {
          if ((cv == &sb.cs && !sb.has_sc) || (cv == &sb.c3 && !sb.bottleneck)) continue;
          act = std::max(act, (size_t)cv->M * cv->Cout);
          act = std::max(act, (size_t)cv->N * cv->H * cv->W * cv->Cin);
          if (!cv->imp_dgrad && !cv->pointwise) cols = std::max(cols, (size_t)cv->M * cv->ldk);
        }
        for (int i = 0; i < 3; ++i) c.GO[i] = h.dalloc(act * es);
        if (cols) c.dcolsO = h.dalloc(cols * es);
        std::vector<std::string> names = {sb.c1.w, sb.b1.g, sb.b1.b, sb.c2.w, sb.b2.g, sb.b2.b};
        if (sb.bottleneck) { names.push_back(sb.c3.w); names.push_back(sb.b3.g); names.push_back(sb.b3.b); }
        if (sb.has_sc) { names.push_back(sb.cs.w); names.push_back(sb.bs.g); names.push_back(sb.bs.b); }
        for (auto& n : names) q.second[n] = fal((size_t)h.tensors[h.find(n)].numel);
      }
      rec_block_bwd(L, sb, sx, h.bnd[wr][k - 1], false, gin, c.GO[0], c.GO[1], c.GO[2], c.dcolsO, &q.second);
      for (auto& kv : q.second) overlap_avg.push_back(AvgProb{h.G(kv.first), kv.second, (long long)h.tensors[h.find(kv.first)].numel});
    }
    if (c.has_stem) {
      rec_bn_bwd(L, c.stem_bn, c.stem.y, gin, c.stem_out, ga, nullptr);
      if (c.stem.small) {
        const Conv& cv = c.stem;
        const int nblk = (int)((cv.M + SMALLCONV_PIXELS - 1) / SMALLCONV_PIXELS), cols = cv.Cout * cv.K;
        float* part = fal((size_t)nblk * cols);
        h.pending_reduce.push_back(ColReduceProb{part, h.G(cv.w), nblk, cols, cols});
        SmallConvProb sp{c.x_nhwc, nullptr, nullptr, ga, part, cv.N, cv.H, cv.W, cv.Cin, cv.Cout};
        const double work = 2.0 * cv.M * cv.Cout * cv.K;
        Op o; o.kind = OP_RAW;
        o.raw = [=](Plan& p) { p.add(1, [=](const RunCtx& r) { launch_small_conv_wgrad(sp, bf, r.stream); }, KIND_GEMM_ALU, work); };
        L.push_back(std::move(o));
      } else {
        rec_gemm(L, {wgrad_prob(c.stem, ga, c.x_nhwc)});
      }
    } else {
      rec_nop(L, 2);
    }
  };

  // Emit the recorded lists position by position; at a position, ops of one kind from all chunks form one
  // grouped launch (BatchNorm ops with different vector widths stay apart).  A chunk's own order is kept.
  auto flush_ops = [&](Plan& p, std::vector<OpList>& lists) {
    size_t len = 0;
    for (auto& L : lists) len = std::max(len, L.size());
    for (size_t i = 0; i < len; ++i) {
      std::vector<Op*> at;
      for (auto& L : lists) if (i < L.size() && L[i].kind != OP_NOP) at.push_back(&L[i]);
      std::vector<GemmProb> gemms;
      std::vector<ColSumProb> cs; std::vector<float*> cs_out;
      std::vector<GapProb> gaps; long long gap_max = 0; double gap_work = 0; bool gap_vec = bf;
      std::vector<AddProb> adds; long long add_max = 0; double add_work = 0; bool add_vec = bf;
      for (Op* o : at) {
        switch (o->kind) {
          case OP_GEMM: gemms.insert(gemms.end(), o->gemms.begin(), o->gemms.end()); break;
          case OP_COLSUM: cs.push_back(o->colsum); cs_out.push_back(o->colsum_out); break;
          case OP_GAP_BWD: gaps.push_back(o->gap); gap_vec = gap_vec && o->gap.C % 8 == 0; gap_max = std::max(gap_max, o->elems); gap_work += (double)o->elems * es; break;
          case OP_ADD: adds.push_back(o->add); add_vec = add_vec && o->elems % 8 == 0; add_max = std::max(add_max, o->elems); add_work += 3.0 * o->elems * es; break;
          default: break;
        }
      }
      if (!gemms.empty()) emit_gemm(h, p, gemms);
      if (!cs.empty()) emit_colsum(h, p, cs, cs_out);
      if (!gaps.empty()) {
        const GapProb* dg = h.upload(gaps);
        int n = (int)gaps.size();
        p.add(1, [=](const RunCtx& r) { launch_gap_bwd(dg, n, gap_max, bf, r.stream, gap_vec); }, KIND_CONV_AUX, gap_work);
      }
      for (int v8 = 0; v8 < 2; ++v8) {
        std::vector<BnStatProb> st; std::vector<BnFinalProb> fi; std::vector<BnApplyProb> ap;
        int nb = 0, C = 0; long long elems = 0; double work = 0;
        for (Op* o : at)
          if (o->kind == OP_BN_BWD && (int)o->v8 == v8) {
            st.push_back(o->bn_stat); fi.push_back(o->bn_final); ap.push_back(o->bn_apply);
            nb = std::max(nb, o->bn_final.nblk); C = std::max(C, o->bn_stat.C); elems = std::max(elems, o->elems); work += o->work;
          }
        if (st.empty()) continue;
        const BnStatProb* ds = h.upload(st);
        const BnFinalProb* df = h.upload(fi);
        const BnApplyProb* da = h.upload(ap);
        int n = (int)st.size();
        bool vec = v8 != 0;
        if (vec && bn_blocks_fused_bwd > 0) {
          std::vector<BnFusedProb> fu;
          for (int i = 0; i < n; ++i) {
            fu.push_back(BnFusedProb{st[i], fi[i], ap[i]});
            fu.back().fin.nblk = std::min(fi[i].nblk, bn_blocks_fused_bwd);   // one partial row per block of the launch
          }
          const BnFusedProb* dfp = h.upload(fu);
          p.add(1, [=](const RunCtx& r) {
            if (launch_bn_fused(dfp, n, true, true, bn_blocks_fused_bwd, grid_counter, d_status, r.stream) == cudaSuccess) return;
            cudaGetLastError();
            launch_bn_stat_partial(ds, n, nb, C, true, bf, r.stream, vec);
            launch_bn_finalize(df, n, C, true, r.stream);
            launch_bn_apply(da, n, elems, true, bf, r.stream, vec);
          }, KIND_NORM, work);
          continue;
        }
        p.add(3, [=](const RunCtx& r) {
          launch_bn_stat_partial(ds, n, nb, C, true, bf, r.stream, vec);
          launch_bn_finalize(df, n, C, true, r.stream);
          launch_bn_apply(da, n, elems, true, bf, r.stream, vec);
        }, KIND_NORM, work);
      }
      if (!adds.empty()) {
        const AddProb* d = h.upload(adds);
        int n = (int)adds.size();
        p.add(1, [=](const RunCtx& r) { launch_add(d, n, add_max, bf, r.stream, add_vec); }, KIND_CONV_AUX, add_work);
      }
      for (Op* o : at) if (o->kind == OP_RAW) o->raw(p);
    }
  };

  std::vector<int> all;
  for (int k = 0; k < K; ++k) all.push_back(k);

  auto build_step = [&](Plan& p, bool pipelined, int rd, int wr, bool overlap) {
    std::vector<LabelProb> lps;
    for (int k = 0; k < K; ++k)
      lps.push_back(LabelProb{labels_of(k, pipelined, rd), (pipelined && k < K - 1) ? h.lab[wr][k] : nullptr, B, NC, h.n_valid[k]});
    emit_labels(h, p, lps);
    for (int k = 0; k < K; ++k) forward_chunk(p, k, rd, wr, BN_TRAIN);
    heads_forward(p, wr, [&](int k) { return labels_of(k, pipelined, rd); }, false, BN_TRAIN);
    std::vector<OpList> lists(K);
    overlap_avg.clear();
    for (int k = 0; k < K; ++k) record_backward(lists[k], k, rd, wr, overlap);
    flush_ops(p, lists);
    emit_pending_reduce(h, p);
    if (!overlap_avg.empty()) {
      const AvgProb* d = h.upload(overlap_avg);
      int n = (int)overlap_avg.size();
      long long mx = 0;
      double bytes = 0;
      for (auto& a : overlap_avg) { mx = std::max(mx, a.n); bytes += 12.0 * a.n; }
      p.add(1, [=](const RunCtx& r) { launch_average_f32(d, n, mx, r.stream); }, KIND_REDUCE, bytes);
      overlap_avg.clear();
    }
    emit_optimizer(h, p);
  };
  auto build_forward = [&](Plan& p, int wr, bool heads, int mode) {
    for (int k = 0; k < K; ++k) forward_chunk(p, k, wr, wr, mode);
    if (!heads) return;
    std::vector<LabelProb> lps;
    for (int k = 0; k < K; ++k) lps.push_back(LabelProb{h.y_in, nullptr, B, NC, h.n_valid[k]});
    emit_labels(h, p, lps);
    heads_forward(p, wr, [&](int) { return (const int*)h.y_in; }, true, mode);
  };

  h.has_eval_plan = true;
  build_step(h.sync_plan, false, 0, 0, false);
  if (K > 1) {
    build_step(h.sync_overlap_plan, false, 0, 0, true);
    h.has_overlap_plan = true;
  }
  for (int par = 0; par < 2; ++par) {
    build_step(h.pipe_plan[par], true, par, 1 - par, false);
    build_forward(h.prime_plan[par], par, false, BN_BATCH);
    std::vector<LabelProb> lps;
    for (int k = 0; k + 1 < K; ++k) lps.push_back(LabelProb{h.y_in, h.lab[par][k], B, NC, h.n_valid[k]});
    if (!lps.empty()) emit_labels(h, h.prime_plan[par], lps);
    build_forward(h.fwd_plan[par], par, true, BN_BATCH);
    build_forward(h.eval_plan[par], par, true, BN_RUNNING);
  }
}

}  // namespace lp
