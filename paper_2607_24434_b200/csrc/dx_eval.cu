// Evaluation terms of Sec. 3.3 that need no training: the router-agreement divergence of Eq. 10 with the top-k
// set agreement the section tracks beside it, and the squared error of Eq. 7.  (The missing residual of Eq. 6 and
// the draft-expert term of Eq. 7 run through the routing and expert kernels with two switches; see dx_api.cu.)
// Small, latency-bound kernels: one CTA per block row, nothing tuned.
#include "dx_internal.cuh"

namespace {

constexpr int kEvalThreads = 256;
constexpr int kEvalWarps = kEvalThreads / 32;

__device__ __forceinline__ float eval_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float eval_warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Block-wide sum / max over kEvalThreads threads; every thread gets the result.
__device__ __forceinline__ float eval_block_sum(float v, float* s_red) {
  v = eval_warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < kEvalWarps; ++w) t += s_red[w];
  return t;
}
__device__ __forceinline__ float eval_block_max(float v, float* s_red) {
  v = eval_warp_max(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = s_red[0];
#pragma unroll
  for (int w = 1; w < kEvalWarps; ++w) t = fmaxf(t, s_red[w]);
  return t;
}

__device__ __forceinline__ float eval_load(const float* p) { return *p; }
__device__ __forceinline__ float eval_load(const __nv_bfloat16* p) { return __bfloat162float(*p); }

struct AgreeParams {
  const float* h_star;
  const float* h_draft;
  const void* W_r;
  const float* bias;
  int H, E, k, score_fn;
  float* kl;
  int32_t* agree;
};

// log of R_l(h)_e as a distribution over the experts (softmax, or sigmoid scores divided by their sum), for the
// expert(s) this thread owns; `z` is the row's logit table in shared memory.
__device__ __forceinline__ void log_distribution(const float* z, int E, int score_fn, float* s_red, float (&lp)[2]) {
  const int e0 = threadIdx.x, e1 = threadIdx.x + kEvalThreads;   // E <= DX_MAX_E = 256: e1 is never in range
  (void)e1;
  const bool in = e0 < E;
  if (score_fn == DX_SCORE_SOFTMAX) {
    const float m = eval_block_max(in ? z[e0] : -INFINITY, s_red);
    const float s = eval_block_sum(in ? expf(z[e0] - m) : 0.f, s_red);
    lp[0] = in ? (z[e0] - m) - logf(s) : 0.f;
  } else {
    // log sigmoid(z) = -log(1 + exp(-z)), evaluated without overflow on either side
    const float zz = in ? z[e0] : 0.f;
    const float ls = zz >= 0.f ? -log1pf(expf(-zz)) : zz - log1pf(expf(zz));
    const float s = eval_block_sum(in ? expf(ls) : 0.f, s_red);
    lp[0] = in ? ls - logf(s) : 0.f;
  }
  lp[1] = 0.f;
}

template <typename WT>
__global__ void __launch_bounds__(kEvalThreads) dx_router_agreement_kernel(AgreeParams p) {
  __shared__ float s_zs[DX_MAX_E], s_zd[DX_MAX_E];
  __shared__ float s_red[kEvalWarps];
  __shared__ int s_cnt[kEvalWarps];
  const int t = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int H = p.H, E = p.E;
  const float* hs = p.h_star + (size_t)t * H;
  const float* hd = p.h_draft + (size_t)t * H;
  const WT* W = reinterpret_cast<const WT*>(p.W_r);
  // router logits of both hidden states: a warp per expert, lanes stride the columns
  for (int e = warp; e < E; e += kEvalWarps) {
    const WT* w = W + (size_t)e * H;
    float as = 0.f, ad = 0.f;
    for (int j = lane; j < H; j += 32) {
      const float wv = eval_load(w + j);
      as = fmaf(wv, hs[j], as);
      ad = fmaf(wv, hd[j], ad);
    }
    as = eval_warp_sum(as);
    ad = eval_warp_sum(ad);
    if (lane == 0) {
      const float b = p.bias ? p.bias[e] : 0.f;
      s_zs[e] = as + b;
      s_zd[e] = ad + b;
    }
  }
  __syncthreads();
  // Eq. 10: KL( R(h*) || R(h^d) ) = sum_e R*_e (log R*_e - log R^d_e)
  float ls[2], ld[2];
  log_distribution(s_zs, E, p.score_fn, s_red, ls);
  log_distribution(s_zd, E, p.score_fn, s_red, ld);
  const int e = threadIdx.x;
  const float term = e < E ? expf(ls[0]) * (ls[0] - ld[0]) : 0.f;
  const float kl = eval_block_sum(term, s_red);
  // top-k sets of both (rank = logits that are larger, or equal with a lower expert id) and their overlap
  int both = 0;
  if (e < E) {
    const float zs = s_zs[e], zd = s_zd[e];
    int rs = 0, rd = 0;
    for (int o = 0; o < E; ++o) {
      const float a = s_zs[o], b = s_zd[o];
      rs += (int)(a > zs) + ((int)(a == zs) & (int)(o < e));
      rd += (int)(b > zd) + ((int)(b == zd) & (int)(o < e));
    }
    both = (rs < p.k) & (rd < p.k);
  }
  const unsigned int bal = __ballot_sync(0xffffffffu, both);
  if (lane == 0) s_cnt[warp] = __popc(bal);
  __syncthreads();
  if (threadIdx.x == 0) {
    int c = 0;
    for (int w = 0; w < kEvalWarps; ++w) c += s_cnt[w];
    if (p.kl) p.kl[t] = kl;
    if (p.agree) p.agree[t] = c;
  }
}

// sum_i (a_i - b_i)^2 with one CTA, in a fixed order (the result does not depend on timing)
__global__ void __launch_bounds__(kEvalThreads) dx_squared_error_kernel(const float* a, const float* b, long long n,
                                                                        float* out) {
  __shared__ float s_red[kEvalWarps];
  float acc = 0.f;
  for (long long i = threadIdx.x; i < n; i += kEvalThreads) {
    const float d = a[i] - b[i];
    acc = fmaf(d, d, acc);
  }
  const float s = eval_block_sum(acc, s_red);
  if (threadIdx.x == 0) *out = s;
}

}  // namespace

cudaError_t dx_launch_router_agreement(const dx_layer* L, const float* h_star, const float* h_draft, int K, float* kl,
                                       int32_t* agree, cudaStream_t st) {
  const dx_layer_desc& d = L->desc;
  AgreeParams p{h_star, h_draft, L->W_r, L->bias, d.hidden, d.n_experts, d.top_k, d.score_fn, kl, agree};
  if (d.weight_dtype != DX_DTYPE_FP32)   // (layers with 4-bit or wide-layout experts have a bf16 router)
    dx_router_agreement_kernel<__nv_bfloat16><<<K, kEvalThreads, 0, st>>>(p);
  else
    dx_router_agreement_kernel<float><<<K, kEvalThreads, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t dx_launch_squared_error(const float* a, const float* b, long long n, float* out, cudaStream_t st) {
  dx_squared_error_kernel<<<1, kEvalThreads, 0, st>>>(a, b, n, out);
  return cudaGetLastError();
}
