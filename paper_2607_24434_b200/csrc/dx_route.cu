// Routing kernel: router logits, scores, top-k with gate weights (Eq. 1, the
// g_{l,e} of Eq. 4), the block's expert union and the pair permutation grouped
// by expert (Eq. 2 / Eq. 3), and the work list the expert kernels consume.
//
// Grid: one CTA per (token, group of 8 experts); each warp owns one router row
// and reduces its dot product with shuffles.  The CTA that takes the last
// ticket finalises: one warp per token runs k rounds of a warp-wide 64-bit max
// over (orderable logit, ~expert id) keys, then the CTA builds the union with
// ballot/popc compaction and a counting sort of the K*k (token, expert) pairs.
#include "dx_internal.cuh"

namespace {

__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  uint4 r = *reinterpret_cast<const uint4*>(p);
  unsigned int u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
    v = other > v ? other : v;
  }
  return v;
}

// Exclusive scan over the 256 threads of the CTA; `total` receives the sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* s_warp, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) {
    int c = s_warp[w];
    if (w < warp) base += c;
    tot += c;
  }
  __syncthreads();
  total = tot;
  return base + inc - v;
}

template <typename WT>
__global__ void __launch_bounds__(256) dx_route_kernel(DxRouteParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int EG = (p.E + 7) >> 3;
  const int t = blockIdx.x / EG, eg = blockIdx.x % EG;
  const int H = p.H;
  const float* hrow = p.h + (size_t)t * H;
  // everything this kernel reads or writes may still be in use by the previous kernel of the stream
  dx_pdl_wait();
  dx_pdl_trigger();

  // 1/rms of the row (every warp recomputes it: H floats from L1/L2)
  float rstd = 1.0f;
  if (p.rms_norm) {
    float ss = 0.f;
    for (int j = lane * 4; j < H; j += 128) {
      float4 v = *reinterpret_cast<const float4*>(hrow + j);
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    rstd = rsqrtf(ss / (float)H + 1e-6f);
  }

  const int e = eg * 8 + warp;
  if (e < p.E) {
    const WT* wrow = reinterpret_cast<const WT*>(p.W_r) + (size_t)e * H;
    float acc = 0.f;
#pragma unroll 4
    for (int j = lane * 8; j < H; j += 256) {
      float wv[8], hv[8];
      load8(wrow + j, wv);
      load8(hrow + j, hv);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc = fmaf(wv[i], hv[i], acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) p.z[t * p.E + e] = acc * rstd + (p.bias ? p.bias[e] : 0.f);
  }
  if (eg == 0) {
    // y starts at zero, or as a copy of the block in the residual form
    for (int j = threadIdx.x * 4; j < H; j += 1024) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (p.residual) v = *reinterpret_cast<const float4*>(hrow + j);
      *reinterpret_cast<float4*>(p.y + (size_t)t * H + j) = v;
    }
  }

  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int tk = atomicAdd(p.ticket, 1u);
    s_last = (tk == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  if (threadIdx.x == 0) *p.ticket = 0u;
  __threadfence();

  // ------------------------------------------------------------- finalise
  __shared__ int s_ids[DX_MAX_PAIRS];
  __shared__ float s_w[DX_MAX_PAIRS];
  __shared__ int s_scan[8];
  __shared__ unsigned int s_ballot[8];
  __shared__ int s_perm[DX_MAX_PAIRS];
  const int K = p.K, E = p.E, k = p.k, P = K * k;

  for (int tt = warp; tt < K; tt += 8) {
    unsigned long long key[8];
    float zv[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      int ee = lane + 32 * j;
      if (ee < E) {
        zv[j] = __ldcg(p.z + tt * E + ee);
        key[j] = ((unsigned long long)dx_orderable(zv[j]) << 32) | (unsigned long long)(0xffffffffu - (unsigned)ee);
      } else {
        zv[j] = 0.f;
        key[j] = 0ull;
      }
    }
    int my_e = 0;
    float my_z = 0.f, zmax = 0.f;
    for (int r = 0; r < k; ++r) {
      unsigned long long best = 0ull;
#pragma unroll
      for (int j = 0; j < 8; ++j) best = key[j] > best ? key[j] : best;
      best = warp_max_u64(best);
      int be = (int)(0xffffffffu - (unsigned)(best & 0xffffffffull));
      // the owning lane publishes the logit and retires the key
      float bz = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (lane + 32 * j == be) { bz = zv[j]; key[j] = 0ull; }
      bz = __shfl_sync(0xffffffffu, bz, be & 31);
      if (r == 0) zmax = bz;
      if (lane == r) { my_e = be; my_z = bz; }
    }
    float psel;
    if (p.score_fn == DX_SCORE_SOFTMAX) {
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (lane + 32 * j < E) s += expf(zv[j] - zmax);
      s = warp_sum(s);
      psel = expf(my_z - zmax) / s;
    } else {
      psel = 1.0f / (1.0f + expf(-my_z));
    }
    if (lane >= k) psel = 0.f;
    float denom = warp_sum(psel);
    float g = p.norm_topk ? psel / denom : psel;
    g *= p.scale;
    if (lane < k) {
      s_ids[tt * k + lane] = my_e;
      s_w[tt * k + lane] = g;
      if (p.topk_ids) p.topk_ids[tt * k + lane] = my_e;
      if (p.topk_w) p.topk_w[tt * k + lane] = g;
    }
  }
  __syncthreads();

  // counting sort of the pairs by expert; thread e owns expert e
  const int me = threadIdx.x;
  int cnt = 0;
  if (me < E)
    for (int q = 0; q < P; ++q) cnt += (s_ids[q] == me);
  int total;
  const int off = block_exclusive_scan(cnt, s_scan, total);
  const int flag = cnt > 0;
  const unsigned int bal = __ballot_sync(0xffffffffu, flag);
  if (lane == 0) s_ballot[warp] = bal;
  int ucount;
  const int upos = block_exclusive_scan(flag, s_scan, ucount);   // also orders s_ballot
  if (me < E) {
    if (p.offsets) p.offsets[me] = off;
    int i = 0;
    for (int q = 0; q < P; ++q)
      if (s_ids[q] == me) { s_perm[off + i] = q; ++i; }
    if (flag && p.union_ids) p.union_ids[upos] = me;
  }
  if (me == 0) {
    if (p.offsets) p.offsets[E] = P;
    if (p.union_count) *p.union_count = ucount;
  }
  if (p.union_mask && me < (E + 63) / 64) {
    unsigned long long lo = s_ballot[2 * me], hi = (2 * me + 1 < 8) ? s_ballot[2 * me + 1] : 0u;
    p.union_mask[me] = lo | (hi << 32);
  }
  __syncthreads();
  if (p.perm)
    for (int q = me; q < P; q += 256) p.perm[q] = s_perm[q];

  // work list
  DxWork* W = p.work;
  if (me < p.n_shared) {
    DxEntry& en = W->entries[me];
    en.table_index = me;
    en.n_tiles = p.shared_tiles;
    en.unit_begin = me * p.shared_tiles;
    en.m = K;
    for (int i = 0; i < K; ++i) { en.tok[i] = i; en.w[i] = 1.0f; }
  }
  int n_entries, total_units;
  const int routed_base = p.n_shared * p.shared_tiles;
  if (!p.draft_mode) {
    if (me < E && flag) {
      DxEntry& en = W->entries[p.n_shared + upos];
      en.table_index = p.n_shared + 1 + me;
      en.n_tiles = p.routed_tiles;
      en.unit_begin = routed_base + upos * p.routed_tiles;
      en.m = cnt;
      for (int i = 0; i < cnt; ++i) {
        int q = s_perm[off + i];
        en.tok[i] = q / k;
        en.w[i] = s_w[q];
      }
    }
    n_entries = p.n_shared + ucount;
    total_units = routed_base + ucount * p.routed_tiles;
  } else {
    int base = p.n_shared;
    if (p.draft_tiles > 0) {
      if (me == 0) {
        DxEntry& en = W->entries[base];
        en.table_index = p.n_shared;
        en.n_tiles = p.draft_tiles;
        en.unit_begin = routed_base;
        en.m = 1;
        en.tok[0] = 0;
        en.w[0] = p.gamma;
      }
      base += 1;
    }
    if (me < p.top_r) {
      DxEntry& en = W->entries[base + me];
      en.table_index = p.n_shared + 1 + s_ids[me];
      en.n_tiles = p.routed_tiles;
      en.unit_begin = routed_base + p.draft_tiles + me * p.routed_tiles;
      en.m = 1;
      en.tok[0] = 0;
      en.w[0] = s_w[me];
    }
    n_entries = base + p.top_r;
    total_units = routed_base + p.draft_tiles + p.top_r * p.routed_tiles;
  }
  if (me == 0) {
    W->n_entries = n_entries;
    W->total_units = total_units;
    W->K = K;
  }
}

}  // namespace

cudaError_t dx_launch_route(const DxRouteParams& p, int weight_dtype, cudaStream_t st) {
  const int grid = p.K * ((p.E + 7) / 8);
  if (weight_dtype == DX_DTYPE_BF16)
    return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, p);
  return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<float>, dim3(grid), dim3(256), 0, st, p);
}
