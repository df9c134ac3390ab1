// Confidence-expansion truncation (Sec. 3.4, Eq. 12-14; Algorithm 1, the loop body around "stop drafting").
// Host-only bookkeeping: the predicted block-level verifier set U_hat is one bitmask per layer; a candidate's
// marginal expansion Delta_i is the number of (layer, expert) pairs its draft-router prediction adds.
#include <new>
#include <vector>

#include "dx_internal.cuh"

struct dx_controller {
  int L, E, words;
  std::vector<unsigned long long> mask;   // [L][words]
  int size;                               // |U_hat|
};

extern "C" dx_status dx_controller_create(int32_t n_layers, int32_t n_experts, dx_controller** out) {
  if (!out) return DX_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_layers < 1 || n_experts < 1) return DX_ERR_INVALID_ARG;
  dx_controller* c = new (std::nothrow) dx_controller();
  if (!c) return DX_ERR_OOM;
  c->L = n_layers;
  c->E = n_experts;
  c->words = (n_experts + 63) / 64;
  c->mask.assign((size_t)n_layers * c->words, 0ull);
  c->size = 0;
  *out = c;
  return DX_OK;
}

extern "C" dx_status dx_controller_destroy(dx_controller* c) {
  if (!c) return DX_ERR_INVALID_ARG;
  delete c;
  return DX_OK;
}

extern "C" dx_status dx_controller_reset(dx_controller* c) {
  if (!c) return DX_ERR_INVALID_ARG;
  c->mask.assign(c->mask.size(), 0ull);
  c->size = 0;
  return DX_OK;
}

extern "C" dx_status dx_controller_size(dx_controller* c, int32_t* size_out) {
  if (!c || !size_out) return DX_ERR_INVALID_ARG;
  *size_out = c->size;
  return DX_OK;
}

extern "C" dx_status dx_controller_propose(dx_controller* c, const int32_t* predicted, int32_t k, float q, float tau,
                                           int32_t budget, int32_t* delta_out, int32_t* stop_out,
                                           int32_t* new_layers_out, int32_t* new_experts_out, int32_t* n_new_out) {
  if (!c || !predicted || k < 1 || !delta_out || !stop_out) return DX_ERR_INVALID_ARG;
  for (int i = 0; i < c->L * k; ++i)
    if (predicted[i] < 0 || predicted[i] >= c->E) return DX_ERR_INVALID_ARG;
  // U_hat_i = U_hat  union  (union over layers of the candidate's predicted experts)
  std::vector<unsigned long long> next = c->mask;
  int delta = 0;
  std::vector<int> nl, ne;
  for (int l = 0; l < c->L; ++l)
    for (int j = 0; j < k; ++j) {
      const int e = predicted[l * k + j];
      unsigned long long& w = next[(size_t)l * c->words + e / 64];
      const unsigned long long bit = 1ull << (e % 64);
      if (!(w & bit)) {
        w |= bit;
        ++delta;
        nl.push_back(l);
        ne.push_back(e);
      }
    }
  *delta_out = delta;
  const bool stop = (q < tau) && (delta > budget);   // Eq. 14: unlikely to be accepted AND expensive to verify
  *stop_out = stop ? 1 : 0;
  if (stop) {
    if (n_new_out) *n_new_out = 0;
    return DX_OK;   // the candidate is dropped, U_hat is unchanged
  }
  c->mask.swap(next);
  c->size += delta;
  if (n_new_out) *n_new_out = delta;
  for (int i = 0; i < delta; ++i) {
    if (new_layers_out) new_layers_out[i] = nl[i];
    if (new_experts_out) new_experts_out[i] = ne[i];
  }
  return DX_OK;
}
