// Routing kernel: router logits, scores, top-k with gate weights (Eq. 1, the
// g_{l,e} of Eq. 4), the block's expert union and the pair permutation grouped
// by expert (Eq. 2 / Eq. 3), and the work list the expert kernels consume.
//
// One thread-block cluster of 8 CTAs does all of it.  Each CTA owns an eighth
// of the router rows: a warp loads a 2048-column slab of its row once (all
// loads in flight together) and dots it with every block row, which sit in
// shared memory.  The logits are written straight into CTA 0's shared memory
// through distributed shared memory, so the hand-over is one hardware cluster
// barrier: no fences, tickets or global round trips on the critical path.
// CTA 0 then runs, one warp per token, k rounds of a warp-wide 64-bit max over
// (orderable logit, ~expert id) keys, and builds the union with ballot/popc
// compaction and a counting sort of the K*k (token, expert) pairs.
#include <cooperative_groups.h>

#include "dx_internal.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kRouteThreads = 256;
constexpr int kRouteCluster = 8;
constexpr int kRouteWarps = kRouteThreads / 32;

__device__ __forceinline__ void unpack8(const uint4& r, float (&v)[8]) {
  const unsigned int u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
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

// Exclusive scan over the threads of the CTA; `total` receives the sum.
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
  for (int w = 0; w < kRouteWarps; ++w) {
    int c = s_warp[w];
    if (w < warp) base += c;
    tot += c;
  }
  __syncthreads();
  total = tot;
  return base + inc - v;
}

// Dot products of one router row with up to kTokGroup block rows (staged in
// shared memory, row stride H) over a slab of <= 2048 columns; the lane owns
// columns j0 + lane*8 + 256*i.
constexpr int kTokGroup = 8;
__device__ __forceinline__ void row_load(const __nv_bfloat16* wrow, int j0, int chunks, int lane, uint4 (&w)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (i < chunks) w[i] = ldg_stream(wrow + j0 + lane * 8 + 256 * i);
}
__device__ __forceinline__ void row_load(const float*, int, int, int, uint4 (&)[8]) {}
// Staged rows are stored so that a lane's eight columns of a 256-column chunk sit in two conflict-free halves:
// columns 8l..8l+3 at chunk*256 + 4l, columns 8l+4..8l+7 at chunk*256 + 128 + 4l.
__device__ __forceinline__ int staged_index(int col) {
  const int chunk = col >> 8, c4 = (col & 255) >> 2;   // float4 index inside the chunk
  return (chunk << 8) + ((c4 & 1) << 7) + ((c4 >> 1) << 2) + (col & 3);
}

template <int KT>
__device__ __forceinline__ void row_dots_kt(const float* h, int H, int K, int j0, int chunks, int lane,
                                            float (&acc)[kTokGroup], const float (&wv)[8][8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (i < chunks) {
      const float* hp = h + j0 + 256 * i + lane * 4;
#pragma unroll
      for (int t = 0; t < KT; ++t) {
        if (t < K) {
          const float4 a = *reinterpret_cast<const float4*>(hp + (size_t)t * H);
          const float4 b = *reinterpret_cast<const float4*>(hp + (size_t)t * H + 128);
          float s = acc[t];
          s = fmaf(wv[i][0], a.x, s); s = fmaf(wv[i][1], a.y, s); s = fmaf(wv[i][2], a.z, s);
          s = fmaf(wv[i][3], a.w, s); s = fmaf(wv[i][4], b.x, s); s = fmaf(wv[i][5], b.y, s);
          s = fmaf(wv[i][6], b.z, s); s = fmaf(wv[i][7], b.w, s);
          acc[t] = s;
        }
      }
    }
  }
}

__device__ __forceinline__ void row_dots_any(const float* h, int H, int K, int j0, int chunks, int lane,
                                             float (&acc)[kTokGroup], const float (&wv)[8][8]) {
  if (K <= 1) row_dots_kt<1>(h, H, K, j0, chunks, lane, acc, wv);
  else if (K <= 2) row_dots_kt<2>(h, H, K, j0, chunks, lane, acc, wv);
  else if (K <= 4) row_dots_kt<4>(h, H, K, j0, chunks, lane, acc, wv);
  else row_dots_kt<8>(h, H, K, j0, chunks, lane, acc, wv);
}

__device__ __forceinline__ void row_dots(const __nv_bfloat16*, const float* h, int H, int K, int j0, int chunks,
                                         int lane, float (&acc)[kTokGroup], const uint4 (&w)[8]) {
  float wv[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (i < chunks) unpack8(w[i], wv[i]);
  row_dots_any(h, H, K, j0, chunks, lane, acc, wv);
}

__device__ __forceinline__ void row_dots(const float* wrow, const float* h, int H, int K, int j0, int chunks, int lane,
                                         float (&acc)[kTokGroup], const uint4 (&)[8]) {
  // fp32 router rows (small layers): two passes of four chunks keep the register footprint down
  for (int half = 0; half < 2; ++half) {
    float wv[8][8];
    const int c0 = half * 4, nc = min(4, chunks - c0);
    if (nc <= 0) break;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (i < nc) {
        const float* wp = wrow + j0 + lane * 8 + 256 * (c0 + i);
        const uint4 u0 = ldg_stream(wp), u1 = ldg_stream(wp + 4);
        wv[i][0] = __uint_as_float(u0.x); wv[i][1] = __uint_as_float(u0.y); wv[i][2] = __uint_as_float(u0.z);
        wv[i][3] = __uint_as_float(u0.w); wv[i][4] = __uint_as_float(u1.x); wv[i][5] = __uint_as_float(u1.y);
        wv[i][6] = __uint_as_float(u1.z); wv[i][7] = __uint_as_float(u1.w);
      }
    }
    row_dots_any(h, H, K, j0 + 256 * c0, nc, lane, acc, wv);
  }
}

// Top-k of one token by one warp: k rounds of (lane-local best, warp max of the logit, warp min of the id among
// the holders of that maximum); then softmax / sigmoid scores of the selected experts and their gate weights.
template <int NK>
__device__ __forceinline__ void topk_token(const DxRouteParams& p, const float* s_z, int* s_ids, float* s_w,
                                           unsigned int* s_mask, int tt, int lane) {
  const int E = p.E, k = p.k;
    unsigned long long key[NK];
    float zv[NK];
#pragma unroll
    for (int j = 0; j < NK; ++j) {
      int ee = lane + 32 * j;
      if (ee < E) {
        zv[j] = s_z[tt * E + ee];
        key[j] = ((unsigned long long)dx_orderable(zv[j]) << 32) | (unsigned long long)(0xffffffffu - (unsigned)ee);
      } else {
        zv[j] = 0.f;
        key[j] = 0ull;
      }
    }
    int my_e = 0;
    float my_z = 0.f, zmax = 0.f;
    for (int r = 0; r < k; ++r) {
      // lane-local best (largest orderable logit, lowest id on ties), then two warp reductions:
      // the maximum logit, and the lowest expert id among the lanes that hold it
      unsigned int lbest = 0u, lid = 0xffffffffu;
#pragma unroll
      for (int j = 0; j < NK; ++j) {
        const unsigned int hi = (unsigned int)(key[j] >> 32);
        if (key[j] != 0ull && hi > lbest) { lbest = hi; lid = (unsigned int)(lane + 32 * j); }
      }
      const unsigned int wbest = __reduce_max_sync(0xffffffffu, lbest);
      const int be = (int)__reduce_min_sync(0xffffffffu, lbest == wbest ? lid : 0xffffffffu);
      // the owning lane publishes the logit and retires the key
      float bz = 0.f;
#pragma unroll
      for (int j = 0; j < NK; ++j)
        if (lane + 32 * j == be) { bz = zv[j]; key[j] = 0ull; }
      bz = __shfl_sync(0xffffffffu, bz, be & 31);
      if (r == 0) zmax = bz;
      if (lane == r) { my_e = be; my_z = bz; }
    }
    float psel;
    if (p.score_fn == DX_SCORE_SOFTMAX) {
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < NK; ++j)
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
      atomicOr(&s_mask[my_e >> 5], 1u << (my_e & 31));   // union of Eq. 2 / Eq. 3 as a bit mask
      if (p.topk_ids) p.topk_ids[tt * k + lane] = my_e;
      if (p.topk_w) p.topk_w[tt * k + lane] = g;
    }
}

template <typename WT>
__global__ void __launch_bounds__(kRouteThreads) dx_route_kernel(DxRouteParams p) {
  __shared__ float s_z[DX_MAX_K * DX_MAX_E];
  __shared__ float s_rstd[DX_MAX_K];
  __shared__ int s_ids[DX_MAX_PAIRS];
  __shared__ float s_w[DX_MAX_PAIRS];
  __shared__ int s_perm[DX_MAX_PAIRS];
  __shared__ int s_scan[kRouteWarps];
  __shared__ unsigned int s_mask[DX_MAX_E / 32];
  __shared__ const void* s_tab[DX_MAX_E];

  cg::cluster_group cluster = cg::this_cluster();
  const int crank = (int)cluster.block_rank();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int K = p.K, E = p.E, k = p.k, H = p.H, P = K * k;
  const int epc = (E + kRouteCluster - 1) / kRouteCluster;   // router rows per CTA
  const int e_lo = crank * epc, e_hi = min(E, e_lo + epc);
  // the router matrix is constant: pull this CTA's rows into L2 while the previous kernel of the stream drains
  if (e_lo < e_hi) {
    const char* wb = reinterpret_cast<const char*>(p.W_r) + (size_t)e_lo * H * sizeof(WT);
    const size_t bytes = (size_t)(e_hi - e_lo) * H * sizeof(WT);
    for (size_t o = (size_t)threadIdx.x * 128; o < bytes; o += (size_t)kRouteThreads * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(wb + o));
  }
  // Let the expert kernel be scheduled right away: its producers only touch constant weights, and its consumers
  // hold back until this kernel publishes that the block input is final.  Everything else this kernel reads or
  // writes may still be in use by the previous kernel of the stream, so wait for that kernel first.
  if (p.handover && crank == 0) {
    // words left set by the previous pair: every CTA of that pair's expert kernel is past them (it lets this
    // kernel start only then), and the expert kernel of this pair cannot start before the trigger below
    if (threadIdx.x == 0) {
      atomicExch(p.handover, 0u);
      atomicExch(p.handover + 1, 0u);
      __threadfence();
    }
    __syncthreads();
  }
  dx_pdl_trigger();
  dx_pdl_wait();
  if (p.handover && crank == 0 && threadIdx.x == 0) {
    __threadfence();
    atomicExch(p.handover, 1u);
  }
  // routed part of the blob table (final now), for the group list at the end
  if (crank == 0) {
    if (threadIdx.x < E) s_tab[threadIdx.x] = p.table[p.n_shared + 1 + threadIdx.x];
    if (threadIdx.x < DX_MAX_E / 32) s_mask[threadIdx.x] = 0u;
  }
  // bias of the first router row of this warp: requested now, used after the dot products
  float bias_first = 0.f;
  if (p.bias && e_lo + warp < e_hi) bias_first = p.bias[e_lo + warp];

  // the first router row of this warp is requested before anything else, so its latency overlaps the staging
  uint4 wreg[8];
  const int first_chunks = min(8, H / 256);
  if (e_lo + warp < e_hi)
    row_load(reinterpret_cast<const WT*>(p.W_r) + (size_t)(e_lo + warp) * H, 0, first_chunks, lane, wreg);

  // y starts at zero, or as a copy of the block in the residual form (stores only complete in the background)
  for (int j = (crank * kRouteThreads + threadIdx.x) * 4; j < K * H; j += kRouteCluster * kRouteThreads * 4) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (p.residual) v = *reinterpret_cast<const float4*>(p.h + j);
    *reinterpret_cast<float4*>(p.y + j) = v;
  }

  // router logits z[t,e]; block rows go through shared memory in groups of up to `tg` rows
  extern __shared__ __align__(16) float s_h[];
  float* z0 = cluster.map_shared_rank(s_z, 0);   // CTA 0's logit table
  const int tg = p.tok_group;
  for (int t0 = 0; t0 < K; t0 += tg) {
    const int kt = min(tg, K - t0);
    __syncthreads();
    // stage the rows with eight loads in flight per thread
    for (int base = threadIdx.x * 4; base < kt * H; base += kRouteThreads * 4 * 8) {
      float4 v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int j = base + i * kRouteThreads * 4;
        if (j < kt * H) v[i] = *reinterpret_cast<const float4*>(p.h + (size_t)t0 * H + j);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int j = base + i * kRouteThreads * 4;
        if (j < kt * H) *reinterpret_cast<float4*>(s_h + (j / H) * H + staged_index(j % H)) = v[i];
      }
    }
    __syncthreads();
    // 1/rms of the staged rows
    for (int t = warp; t < kt; t += kRouteWarps) {
      float rs = 1.0f;
      if (p.rms_norm) {
        float ss = 0.f;
        for (int j = lane * 4; j < H; j += 128) {
          const float4 v = *reinterpret_cast<const float4*>(s_h + (size_t)t * H + j);
          ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        rs = rsqrtf(warp_sum(ss) / (float)H + 1e-6f);
      }
      if (lane == 0) s_rstd[t0 + t] = rs;
    }
    __syncthreads();
    for (int e = e_lo + warp; e < e_hi; e += kRouteWarps) {
      const WT* wrow = reinterpret_cast<const WT*>(p.W_r) + (size_t)e * H;
      float acc[kTokGroup];
#pragma unroll
      for (int t = 0; t < kTokGroup; ++t) acc[t] = 0.f;
      for (int j0 = 0; j0 < H; j0 += 2048) {
        const int chunks = min(8, (H - j0) / 256);
        if (!(t0 == 0 && e == e_lo + warp && j0 == 0)) row_load(wrow, j0, chunks, lane, wreg);
        row_dots(wrow, s_h, H, kt, j0, chunks, lane, acc, wreg);
      }
      const float b = (e == e_lo + warp) ? bias_first : (p.bias ? p.bias[e] : 0.f);
#pragma unroll
      for (int t = 0; t < kTokGroup; ++t) {
        if (t < kt) {
          const float s = warp_sum(acc[t]);
          if (lane == 0) z0[(t0 + t) * E + e] = s * s_rstd[t0 + t] + b;
        }
      }
    }
  }
  cluster.sync();          // all logits have landed in CTA 0
  if (crank != 0) return;

  // top-k and gate weights, one warp per token (NK = keys per lane, a power of two covering E)
  for (int tt = warp; tt < K; tt += kRouteWarps) {
    if (E <= 32) topk_token<1>(p, s_z, s_ids, s_w, s_mask, tt, lane);
    else if (E <= 64) topk_token<2>(p, s_z, s_ids, s_w, s_mask, tt, lane);
    else if (E <= 128) topk_token<4>(p, s_z, s_ids, s_w, s_mask, tt, lane);
    else topk_token<8>(p, s_z, s_ids, s_w, s_mask, tt, lane);
  }
  __syncthreads();

  // ---- group list for the expert kernel (it is waiting for it); the caller's outputs come afterwards
  const int me = threadIdx.x;
  DxWork* W = p.work;
  int flag = 0, upos = 0, ucount = 0;
  {
    const unsigned int mine = me < E ? s_mask[me >> 5] : 0u;
    flag = (mine >> (me & 31)) & 1u;
    for (int w2 = 0; w2 < (E + 31) / 32; ++w2) {
      const int c = __popc(s_mask[w2]);
      ucount += c;
      if (w2 < (me >> 5)) upos += c;
    }
    upos += __popc(mine & ((1u << (me & 31)) - 1u));
  }
  if (!p.draft_mode) {
    if (flag) { W->gid[upos] = me; W->gblob[upos] = s_tab[me]; }
  } else if (me < p.top_r) {
    W->gid[me] = s_ids[me];
    W->gblob[me] = s_tab[s_ids[me]];
  }
  for (int q = me; q < P; q += kRouteThreads) { W->pair_id[q] = s_ids[q]; W->pair_w[q] = s_w[q]; }
  if (me == 0) {
    W->n_groups = p.draft_mode ? p.top_r : ucount;
    W->K = K;
    W->k = k;
  }
  __syncthreads();
  if (p.handover && me == 0) {
    __threadfence();   // cumulative: covers the other threads' stores ordered before the barrier
    atomicExch(p.handover + 1, 1u);
  }

  // ---- routing outputs for the caller: pairs sorted by expert (counting sort; thread e owns expert e)
  int cnt = 0;
  if (me < E) {
#pragma unroll 8
    for (int q = 0; q < P; ++q) cnt += (s_ids[q] == me);
  }
  int total;
  const int off = block_exclusive_scan(cnt, s_scan, total);
  if (me < E) {
    int i = 0;
    for (int q = 0; q < P; ++q)
      if (s_ids[q] == me) s_perm[off + i++] = q;
    if (p.offsets) p.offsets[me] = off;
    if (flag && p.union_ids) p.union_ids[upos] = me;
  }
  if (me == 0) {
    if (p.offsets) p.offsets[E] = P;
    if (p.union_count) *p.union_count = ucount;
  }
  if (p.union_mask && me < (E + 63) / 64) {
    const unsigned long long lo = s_mask[2 * me], hi = (2 * me + 1 < DX_MAX_E / 32) ? s_mask[2 * me + 1] : 0u;
    p.union_mask[me] = lo | (hi << 32);
  }
  __syncthreads();
  if (p.perm)
    for (int q = me; q < P; q += kRouteThreads) p.perm[q] = s_perm[q];
}

}  // namespace

cudaError_t dx_launch_route(const DxRouteParams& p_in, int weight_dtype, cudaStream_t st) {
  DxRouteParams p = p_in;
  // as many block rows per pass as fit in 64 KB of shared memory (at most kTokGroup)
  int tg = (64 * 1024) / (p.H * 4);
  if (tg > kTokGroup) tg = kTokGroup;
  if (tg > p.K) tg = p.K;
  if (tg < 1) tg = 1;
  p.tok_group = tg;
  const size_t smem = (size_t)tg * p.H * 4;
  cudaError_t e;
  if (weight_dtype == DX_DTYPE_BF16) {
    e = cudaFuncSetAttribute(dx_route_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    if (e != cudaSuccess) return e;
    return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<__nv_bfloat16>, dim3(kRouteCluster), dim3(kRouteThreads), smem,
                         st, kRouteCluster, p);
  }
  e = cudaFuncSetAttribute(dx_route_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
  if (e != cudaSuccess) return e;
  return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<float>, dim3(kRouteCluster), dim3(kRouteThreads), smem, st,
                       kRouteCluster, p);
}
