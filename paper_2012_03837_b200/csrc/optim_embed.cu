// Fused multi-tensor optimizer update over the whole parameter arena (each chunk's parameters are
// updated from that chunk's own gradients only, Sec. 1 / Sec. 6: the update is element-wise, so one
// flat sweep applies all K per-chunk updates), and the token/position embedding of LM chunk 0.
#include <climits>

#include "common.cuh"
#include "optim_update.cuh"

namespace lp {
namespace {

// 4 elements per thread, 128-bit accesses (optim_update4).
template <bool PER_CHUNK>
__global__ void __launch_bounds__(256) optim_kernel(OptimArgs a) {
  long long i4 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i4 >= a.n_total) return;   // the arena length is a multiple of 4
  optim_update4<PER_CHUNK>(a, i4);
}

__global__ void __launch_bounds__(256) mask_losses_kernel(float* losses, const float4* chunk_tab, int K) {
  int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < K && chunk_tab[k].x == 0.f) losses[k] = __int_as_float(0x7fc00000);
}

// h[r, :] = tok[ids[r], :] + pos[r % T, :]; ids outside [0, vocab) are flagged and clamped.
template <typename T>
__global__ void __launch_bounds__(256) embed_fwd_kernel(EmbedProb p, int* status) {
  int row = blockIdx.x;
  int id = p.ids[row];
  if (id < 0 || id >= p.vocab) {
    if (threadIdx.x == 0) atomicOr(status, ST_LABEL_RANGE);
    id = min(max(id, 0), p.vocab - 1);
  }
  const T* tok = (const T*)p.tok + (size_t)id * p.d;
  const T* pos = (const T*)p.pos + (size_t)(row % p.T) * p.d;
  T* h = (T*)p.h + (size_t)row * p.d;
  for (int c = threadIdx.x; c < p.d; c += blockDim.x) h[c] = from_f<T>(to_f(tok[c]) + to_f(pos[c]));
}

// next[i] = smallest j > i holding the same token id (or -1); first[i] = 1 unless some earlier
// position holds the same id.  Three steps: reset, one block per (tile of i, later tile of j) that
// takes an atomic minimum over the matches it finds (a minimum does not depend on the order of
// its arguments, so the result is deterministic), then the successors are marked.
__global__ void __launch_bounds__(256) embed_link_init_kernel(EmbedBwdProb p) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < p.rows) { p.next[i] = INT_MAX; p.first[i] = 1; }
}
__global__ void __launch_bounds__(256) embed_link_kernel(EmbedBwdProb p) {
  __shared__ int tile[256];
  if (blockIdx.x < blockIdx.y) return;         // only tiles of j at or after the tile of i
  const int i = blockIdx.y * 256 + threadIdx.x, j0 = blockIdx.x * 256;
  const int j = j0 + threadIdx.x;
  tile[threadIdx.x] = j < p.rows ? min(max(p.ids[j], 0), p.vocab - 1) : -2;
  const int my = i < p.rows ? min(max(p.ids[i], 0), p.vocab - 1) : -1;
  __syncthreads();
  if (my < 0) return;
  for (int t = 0; t < 256; ++t) {
    if (tile[t] == my && j0 + t > i) { atomicMin(&p.next[i], j0 + t); break; }
  }
}
__global__ void __launch_bounds__(256) embed_mark_kernel(EmbedBwdProb p) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= p.rows) return;
  int n = p.next[i];
  if (n == INT_MAX) p.next[i] = -1;
  else p.first[n] = 0;
}
// One block per position: the first holder of a token id sums dh over the chain of positions
// holding that id, in increasing position order (deterministic), and writes the table row.
template <typename T>
__global__ void __launch_bounds__(256) embed_bwd_tok_kernel(EmbedBwdProb p) {
  int i = blockIdx.x;
  if (!p.first[i]) return;
  int id = min(max(p.ids[i], 0), p.vocab - 1);
  const T* dh = (const T*)p.dh;
  for (int c = threadIdx.x; c < p.d; c += blockDim.x) {
    float s = 0.f;
    for (int j = i; j >= 0; j = p.next[j]) s += to_f(dh[(size_t)j * p.d + c]);
    p.dtok[(size_t)id * p.d + c] = s;
  }
}
template <typename T>
__global__ void __launch_bounds__(256) embed_bwd_pos_kernel(EmbedBwdProb p) {
  int t = blockIdx.x;
  const T* dh = (const T*)p.dh;
  for (int c = threadIdx.x; c < p.d; c += blockDim.x) {
    float s = 0.f;
    for (int b = 0; b < p.B; ++b) s += to_f(dh[((size_t)b * p.T + t) * p.d + c]);
    p.dpos[(size_t)t * p.d + c] = s;
  }
}

}  // namespace

void launch_optim(const OptimArgs& a, cudaStream_t s) {
  long long threads = (a.n_total + 3) / 4;
  if (threads == 0) return;
  if (a.seg_end) optim_kernel<true><<<(unsigned)((threads + 255) / 256), 256, 0, s>>>(a);
  else optim_kernel<false><<<(unsigned)((threads + 255) / 256), 256, 0, s>>>(a);
}

void launch_mask_losses(float* losses, const float4* chunk_tab, int K, cudaStream_t s) {
  mask_losses_kernel<<<(K + 255) / 256, 256, 0, s>>>(losses, chunk_tab, K);
}

void launch_embed_fwd(const EmbedProb& p, int* d_status, bool is_bf16, cudaStream_t s) {
  if (is_bf16) embed_fwd_kernel<bf16><<<p.rows, 256, 0, s>>>(p, d_status);
  else embed_fwd_kernel<float><<<p.rows, 256, 0, s>>>(p, d_status);
}

void launch_embed_bwd(const EmbedBwdProb& p, bool is_bf16, cudaStream_t s) {
  int nb = (p.rows + 255) / 256;
  embed_link_init_kernel<<<nb, 256, 0, s>>>(p);
  embed_link_kernel<<<dim3(nb, nb), 256, 0, s>>>(p);
  embed_mark_kernel<<<nb, 256, 0, s>>>(p);
  cudaMemsetAsync(p.dtok, 0, (size_t)p.vocab * p.d * sizeof(float), s);
  if (is_bf16) {
    embed_bwd_tok_kernel<bf16><<<p.rows, 256, 0, s>>>(p);
    embed_bwd_pos_kernel<bf16><<<p.T, 256, 0, s>>>(p);
  } else {
    embed_bwd_tok_kernel<float><<<p.rows, 256, 0, s>>>(p);
    embed_bwd_pos_kernel<float><<<p.T, 256, 0, s>>>(p);
  }
}

}  // namespace lp
