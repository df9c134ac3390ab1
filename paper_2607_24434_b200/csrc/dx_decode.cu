// One exact DraftExpert decode step (Algorithm 1) over an offloaded layer stack, as a host loop inside the library.
//
// Nothing is computed here: every arithmetic step is one of the library's own entry points -- the drafter's layers
// (Eq. 5, moe_draft_step_cached), the draft LM head with its confidence (spec_draft_token), the confidence-expansion
// stop rule (Sec. 3.4, dx_controller_propose), prefetching of the newly predicted verifier experts (Sec. 3.5,
// expert_cache_prefetch), the verifier's layers (Eq. 4 over the block's expert union, moe_verify_block_cached) and
// greedy exact acceptance (spec_accept) -- in the order Algorithm 1 gives.  What the loop adds is that it runs
// without an interpreter between two calls (a step is some 250 calls, each a few microseconds of device work
// apart), that token embeddings are gathered by a kernel from ids passed as launch parameters, and that every
// result the host has to look at (draft token, confidence, target tokens, accepted length) is written by the
// producing kernel into page-locked host memory.  Attention is not part of the path (pre-norm residual MoE
// sub-layers only), so a token's hidden states depend on its own embedding alone.
#include <cstring>
#include <new>
#include <vector>

#include <cuda_bf16.h>

#include "dx_internal.cuh"

int dx_cache_slots(const dx_cache* c);

namespace {

struct EmbedIds {
  int32_t id[DX_MAX_K];
};

// rows[i] = float(emb[ids.id[i]]), i < n; H a multiple of 8
__global__ void dx_embed_rows_kernel(const __nv_bfloat16* emb, EmbedIds ids, int n, int H, int V, float* rows) {
  const int per_row = H / 8;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n * per_row; i += gridDim.x * blockDim.x) {
    const int r = i / per_row, c = i - r * per_row;
    const int tok = min(max(ids.id[r], 0), V - 1);
    const uint4 v = *reinterpret_cast<const uint4*>(emb + (size_t)tok * H + 8 * c);
    const unsigned int w[4] = {v.x, v.y, v.z, v.w};
    float4 lo, hi;
    lo.x = __uint_as_float(w[0] << 16); lo.y = __uint_as_float(w[0] & 0xffff0000u);
    lo.z = __uint_as_float(w[1] << 16); lo.w = __uint_as_float(w[1] & 0xffff0000u);
    hi.x = __uint_as_float(w[2] << 16); hi.y = __uint_as_float(w[2] & 0xffff0000u);
    hi.z = __uint_as_float(w[3] << 16); hi.w = __uint_as_float(w[3] & 0xffff0000u);
    float* dst = rows + (size_t)r * H + 8 * c;
    *reinterpret_cast<float4*>(dst) = lo;
    *reinterpret_cast<float4*>(dst + 4) = hi;
  }
}

}  // namespace

struct dx_decoder {
  dx_ctx* ctx;
  int L, k_max, V, H, E, k, budget;
  float tau;
  std::vector<dx_layer*> layers;
  dx_cache* cache;
  const __nv_bfloat16* emb;
  const void* W_lm;
  dx_controller* ctl;
  float* hd[2];        // the drafter's hidden row, alternating (h_in and h_out of a residual layer are distinct)
  float* hv[2];        // the verifier's block rows, alternating
  int32_t* res_host;   // page-locked, mapped: [0] draft token, [1] its confidence (float bits), [2, 2 + k_max) target
                       // tokens, then accepted length, next token, then the drafted tokens the accept kernel reads
  int32_t* res_dev;    // its device mapping
  std::vector<int32_t> pred, new_l, new_e;
};

extern "C" dx_status dx_decoder_create(dx_ctx* ctx, dx_layer* const* layers, int32_t n_layers, dx_cache* cache,
                                       const void* emb, const void* W_lm, int32_t V, int32_t k_max, float tau,
                                       int32_t budget, dx_decoder** out) {
  if (!ctx || !layers || !cache || !emb || !W_lm || !out) return DX_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_layers < 1 || V < 1 || k_max < 1 || k_max > DX_MAX_K) return DX_ERR_INVALID_ARG;
  const dx_layer_desc& d0 = layers[0]->desc;
  for (int l = 0; l < n_layers; ++l) {
    const dx_layer* L = layers[l];
    if (!L || L->ctx != ctx || L->cache != cache || L->cache_layer != l) return DX_ERR_INVALID_ARG;
    if (L->desc.hidden != d0.hidden || L->desc.n_experts != d0.n_experts || L->desc.top_k != d0.top_k) return DX_ERR_SHAPE;
  }
  if (d0.hidden % 8 || ((uintptr_t)emb) % 16) return DX_ERR_INVALID_ARG;
  dx_decoder* d = new (std::nothrow) dx_decoder();
  if (!d) return DX_ERR_OOM;
  d->ctx = ctx; d->L = n_layers; d->k_max = k_max; d->V = V; d->H = d0.hidden; d->E = d0.n_experts; d->k = d0.top_k;
  d->budget = budget; d->tau = tau;
  d->layers.assign(layers, layers + n_layers);
  d->cache = cache;
  d->emb = reinterpret_cast<const __nv_bfloat16*>(emb);
  d->W_lm = W_lm;
  d->ctl = nullptr;
  d->hd[0] = d->hd[1] = d->hv[0] = d->hv[1] = nullptr;
  d->res_host = d->res_dev = nullptr;
  d->pred.assign((size_t)n_layers * d->k, 0);
  d->new_l.assign((size_t)n_layers * d->k, 0);
  d->new_e.assign((size_t)n_layers * d->k, 0);
  dx_status s = dx_controller_create(n_layers, d->E, &d->ctl);
  cudaError_t e = cudaSetDevice(ctx->device);
  const size_t row = sizeof(float) * (size_t)d->H;
  for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
    e = cudaMalloc(&d->hd[i], row);
    if (e == cudaSuccess) e = cudaMalloc(&d->hv[i], row * k_max);
  }
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&d->res_host, sizeof(int32_t) * (4 + 2 * DX_MAX_K), cudaHostAllocMapped);
  if (e == cudaSuccess) e = cudaHostGetDevicePointer((void**)&d->res_dev, d->res_host, 0);
  if (s != DX_OK || e != cudaSuccess) {
    if (e != cudaSuccess) ctx->last_cuda = e;
    dx_decoder_destroy(d);
    return s != DX_OK ? s : (e == cudaErrorMemoryAllocation ? DX_ERR_OOM : DX_ERR_CUDA);
  }
  *out = d;
  return DX_OK;
}

extern "C" dx_status dx_decoder_destroy(dx_decoder* d) {
  if (!d) return DX_ERR_INVALID_ARG;
  if (d->ctl) dx_controller_destroy(d->ctl);
  for (int i = 0; i < 2; ++i) { cudaFree(d->hd[i]); cudaFree(d->hv[i]); }
  if (d->res_host) cudaFreeHost(d->res_host);
  delete d;
  return DX_OK;
}

extern "C" dx_status dx_decoder_step(dx_decoder* d, int32_t t0, int32_t scripted_accept, int32_t* drafted,
                                     int32_t* n_drafted, int32_t* n_accept, int32_t* emitted, int32_t* n_emitted,
                                     int32_t* target, int32_t* union_sizes, void* stream) {
  if (!d || !drafted || !n_drafted || !n_accept || !emitted || !n_emitted) return DX_ERR_INVALID_ARG;
  dx_ctx* ctx = d->ctx;
  cudaStream_t st = (cudaStream_t)stream;
  const int L = d->L, H = d->H, k = d->k;
  int32_t* r_tok = d->res_host;            // draft token
  int32_t* r_conf = d->res_host + 1;       // its confidence, as float bits
  int32_t* r_target = d->res_host + 2;     // [DX_MAX_K]
  int32_t* r_n = d->res_host + 2 + DX_MAX_K;
  int32_t* r_next = r_n + 1;
  int32_t* r_draft = r_n + 2;              // [DX_MAX_K] what the accept kernel compares with
  auto dev = [&](int32_t* host) { return d->res_dev + (host - d->res_host); };
  auto embed = [&](const EmbedIds& ids, int n, float* rows) -> dx_status {
    const int threads = n * (H / 8);
    dx_embed_rows_kernel<<<(threads + 255) / 256, 256, 0, st>>>(d->emb, ids, n, H, d->V, rows);
    DX_CUDA(ctx, cudaGetLastError());
    ctx->launches++;
    return DX_OK;
  };
  dx_status s = expert_cache_begin_step(d->cache);
  if (s != DX_OK) return s;
  s = dx_controller_reset(d->ctl);
  if (s != DX_OK) return s;
  int nd = 0;
  int32_t prev = t0;
  for (int i = 0; i < d->k_max; ++i) {
    // ---- candidate i (Algorithm 1, drafting): the drafter's stack on the embedding of the previous token
    EmbedIds one{};
    one.id[0] = prev;
    s = embed(one, 1, d->hd[0]);
    if (s != DX_OK) return s;
    for (int l = 0; l < L; ++l) {
      s = moe_draft_step_cached(d->layers[l], d->hd[l & 1], d->hd[(l + 1) & 1], 1, nullptr, nullptr,
                                d->pred.data() + (size_t)l * k, stream);
      if (s != DX_OK) return s;
    }
    s = spec_draft_token(ctx, d->hd[L & 1], 1, d->W_lm, d->V, H, DX_DTYPE_BF16, 1, dev(r_tok),
                         reinterpret_cast<float*>(dev(r_conf)), stream);
    if (s != DX_OK) return s;
    DX_CUDA(ctx, cudaStreamSynchronize(st));
    const int32_t v = *r_tok;
    float q;
    memcpy(&q, r_conf, sizeof(float));
    // ---- its confidence, the experts its draft routers predict and what they add to the block's set: the stop rule
    int32_t size = 0;
    dx_controller_size(d->ctl, &size);
    const int32_t budget = d->budget < 0 ? L * dx_cache_slots(d->cache) - size : d->budget;
    int32_t delta = 0, stop = 0, n_new = 0;
    s = dx_controller_propose(d->ctl, d->pred.data(), k, q, d->tau, budget, &delta, &stop, d->new_l.data(),
                              d->new_e.data(), &n_new);
    if (s != DX_OK) return s;
    if (stop) break;
    drafted[nd++] = v;
    // ---- prefetch what the candidate adds and the cache does not hold or expect yet; the new pairs come layer by layer
    for (int a = 0; a < n_new;) {
      int b = a;
      while (b < n_new && d->new_l[b] == d->new_l[a]) ++b;
      s = expert_cache_prefetch(d->cache, d->new_l[a], d->new_e.data() + a, b - a);
      if (s != DX_OK) return s;
      a = b;
    }
    prev = v;
  }
  // ---- verify D with the full target MoE: the rows are the inputs that predict d_1 .. d_K
  const int K = nd > 0 ? nd : 1;
  EmbedIds in{};
  in.id[0] = t0;
  for (int i = 1; i < K; ++i) in.id[i] = drafted[i - 1];
  s = embed(in, K, d->hv[0]);
  if (s != DX_OK) return s;
  for (int l = 0; l < L; ++l) {
    int32_t cnt = 0;
    s = moe_verify_block_cached(d->layers[l], d->hv[l & 1], K, d->hv[(l + 1) & 1], 1, nullptr, nullptr, nullptr, nullptr,
                                nullptr, nullptr, nullptr, nullptr, &cnt, stream);
    if (s != DX_OK) return s;
    if (union_sizes) union_sizes[l] = cnt;
  }
  const int Kd = nd > 0 ? nd : 1;
  for (int i = 0; i < Kd; ++i) r_draft[i] = nd > 0 ? drafted[i] : -1;
  s = spec_accept(ctx, d->hv[L & 1], K, d->W_lm, d->V, H, DX_DTYPE_BF16, dev(r_draft), Kd, 1, dev(r_target), dev(r_n),
                  dev(r_next), stream);
  if (s != DX_OK) return s;
  DX_CUDA(ctx, cudaStreamSynchronize(st));
  int n = nd > 0 ? *r_n : 0;
  if (scripted_accept >= 0) n = scripted_accept < nd ? scripted_accept : nd;
  // the accepted prefix d_1 .. d_n, then the target's own token for position n + 1 if a row is left for it (with the
  // whole block accepted the next step starts from d_K)
  int ne = 0;
  for (int i = 0; i < n; ++i) emitted[ne++] = drafted[i];
  if (n < K) emitted[ne++] = r_target[n];
  if (target)
    for (int i = 0; i < K; ++i) target[i] = r_target[i];
  *n_drafted = nd;
  *n_accept = n;
  *n_emitted = ne;
  return DX_OK;
}
