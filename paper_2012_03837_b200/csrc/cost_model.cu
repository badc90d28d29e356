// FLOP cost model of App. A: total FLOPs and sequential FLOPs ("time") of a training run for back-propagation
// and the local-update variants.  Host arithmetic only; nothing here touches a GPU.
//
// App. A.1 counts an MLP layer with input size I and N units as a matrix-vector product (2 I N - I), a bias
// add (N) and a ReLU (2 N), and an auxiliary classifier as a matrix-vector product to `classes` outputs
// (2 N classes - N), a bias add (classes) and a softmax cross-entropy at 5 FLOPs per class.  App. A.2 builds
// every method's cost from four numbers -- forward cost per layer, auxiliary cost, backward multiplier,
// optimizer cost (ten FLOPs per parameter) -- plus batch size and step count, and divides by the parallelism
// the method offers (every example and, for local methods, every block at once).
#include "../../include/lp.h"

extern "C" {

double lp_mlp_layer_flops(long long input_size, long long units) {
  return (double)(2 * input_size * units - input_size) + (double)units + 2.0 * (double)units;
}

double lp_mlp_aux_flops(long long units, long long classes) {
  return (double)(2 * units * classes - units) + (double)classes + 5.0 * (double)classes;
}

lp_status lp_cost_model(const lp_cost_spec* c, lp_cost_result* out) {
  if (!c || !out) return LP_ERR_INVALID_ARG;
  if (c->layers < 1 || c->batch_size < 1 || c->steps < 0 || c->forward_cost < 0 || c->aux_cost < 0 ||
      c->backward_multiplier < 0 || c->parameters < 0)
    return LP_ERR_SHAPE;
  const double f = c->forward_cost, a = c->aux_cost, bm = c->backward_multiplier, L = (double)c->layers;
  double per_example = 0, parallel = 1, optimizer = 10.0 * c->parameters;
  switch (c->method) {
    case LP_COST_BACKPROP:
      per_example = (1 + bm) * (f * L + a);
      parallel = 1;
      break;
    case LP_COST_GREEDY:
      per_example = (1 + bm) * ((f + a) * L);
      parallel = L;
      break;
    case LP_COST_OVERLAPPING:
      // one forward pass, two backward passes for every layer but the last, one auxiliary loss per layer,
      // and the averaging of the shared layers' gradients (two FLOPs per parameter on top of the optimizer)
      per_example = (f + a) * L + (L - 1) * bm * (2 * f + a) + bm * (f + a);
      parallel = L;
      optimizer += 2.0 * c->parameters;
      break;
    case LP_COST_CHUNKED: {
      // K chunks: one forward + backward pass through all layers, K auxiliary losses.  (The printed
      // formula drops the layer count; it is restored by analogy with the back-propagation one.)
      if (c->chunks < 1 || c->chunks > c->layers) return LP_ERR_SHAPE;
      const double K = (double)c->chunks;
      per_example = (1 + bm) * (f * L + K * a);
      parallel = K;
      break;
    }
    case LP_COST_LAST_LAYERS: {
      // full forward pass, one auxiliary loss, backward pass through the last K layers only.  (The printed
      // formula lacks a "+" between the forward and the auxiliary cost.)
      if (c->chunks < 1 || c->chunks > c->layers) return LP_ERR_SHAPE;
      const double K = (double)c->chunks;
      per_example = (L * f + a) + bm * (K * f + a);
      parallel = (L + K * bm) / (K * (1 + bm));
      break;
    }
    default:
      return LP_ERR_INVALID_ARG;
  }
  out->cost_per_example = per_example;
  out->total_flops = per_example * (double)c->steps * (double)c->batch_size + (double)c->steps * optimizer;
  out->parallelism = parallel;
  out->sequential_flops = out->total_flops / ((double)c->batch_size * parallel);
  return LP_OK;
}

}  // extern "C"
