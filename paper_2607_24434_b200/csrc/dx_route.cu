// Routing kernel: router logits, scores, top-k with gate weights (Eq. 1, the
// g_{l,e} of Eq. 4), the block's expert union and the pair permutation grouped
// by expert (Eq. 2 / Eq. 3), and the work list the expert kernels consume.
//
// One thread-block cluster of 8 CTAs does all of it.  Each CTA owns an eighth
// of the router rows; a warp dots its row with every block row, reading both
// straight from global memory with all loads of a slab in flight together
// (the block rows are shared by the warps of a CTA through L1).  The logits
// are written into CTA 0's shared memory through distributed shared memory,
// so the hand-over is one hardware cluster barrier: no fences, tickets or
// global round trips on the critical path.  CTA 0 then selects, one warp per
// token, by ranking every logit against all others (no selection rounds),
// builds the union as a bit mask, publishes the group list the expert kernel
// is waiting for, and only then sorts the K*k (token, expert) pairs by expert
// for the caller's outputs.
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
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
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

// Dot products of one router row with TG block rows, everything read straight from global memory: the lane owns
// columns 256*c + 8*lane .. +7 of every 256-column chunk c, and NB chunks (one row slab and TG block-row slabs
// each, row stride hs) are requested together before any of them is used.  The block rows are shared by all warps of the CTA
// and come out of L1 after the first touch.  With `rms`, the sums of squares of the block rows ride along.
constexpr int kTokGroup = 8;
template <typename WT> struct RowRaw;
template <> struct RowRaw<__nv_bfloat16> {
  uint4 r;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { r = ldg_stream(p); }
  __device__ __forceinline__ void unpack(float (&v)[8]) const { unpack8(r, v); }
};
template <> struct RowRaw<float> {
  uint4 r0, r1;
  __device__ __forceinline__ void load(const float* p) { r0 = ldg_stream(p); r1 = ldg_stream(p + 4); }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
    v[0] = __uint_as_float(r0.x); v[1] = __uint_as_float(r0.y); v[2] = __uint_as_float(r0.z);
    v[3] = __uint_as_float(r0.w); v[4] = __uint_as_float(r1.x); v[5] = __uint_as_float(r1.y);
    v[6] = __uint_as_float(r1.z); v[7] = __uint_as_float(r1.w);
  }
};

template <typename WT, int TG>
__device__ __forceinline__ void row_dots_direct(const WT* wrow, const float* h, int hs, int H, int kt, int lane, bool rms,
                                                float (&acc)[kTokGroup], float (&ss)[kTokGroup]) {
  constexpr int NB = TG >= 8 ? 2 : (TG >= 4 ? 4 : 8);
  const int chunks = H / 256;
  for (int c0 = 0; c0 < chunks; c0 += NB) {
    RowRaw<WT> wr[NB];
    float4 ha[NB][TG], hb[NB][TG];
#pragma unroll
    for (int i = 0; i < NB; ++i) {
      if (c0 + i < chunks) {
        const int col = 256 * (c0 + i) + 8 * lane;
        wr[i].load(wrow + col);
#pragma unroll
        for (int t = 0; t < TG; ++t) {
          if (t < kt) {
            ha[i][t] = *reinterpret_cast<const float4*>(h + (size_t)t * hs + col);
            hb[i][t] = *reinterpret_cast<const float4*>(h + (size_t)t * hs + col + 4);
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < NB; ++i) {
      if (c0 + i < chunks) {
        float wv[8];
        wr[i].unpack(wv);
#pragma unroll
        for (int t = 0; t < TG; ++t) {
          if (t < kt) {
            const float4 a = ha[i][t], b = hb[i][t];
            float s = acc[t];
            s = fmaf(wv[0], a.x, s); s = fmaf(wv[1], a.y, s); s = fmaf(wv[2], a.z, s); s = fmaf(wv[3], a.w, s);
            s = fmaf(wv[4], b.x, s); s = fmaf(wv[5], b.y, s); s = fmaf(wv[6], b.z, s); s = fmaf(wv[7], b.w, s);
            acc[t] = s;
            if (rms) {
              float q = ss[t];
              q = fmaf(a.x, a.x, q); q = fmaf(a.y, a.y, q); q = fmaf(a.z, a.z, q); q = fmaf(a.w, a.w, q);
              q = fmaf(b.x, b.x, q); q = fmaf(b.y, b.y, q); q = fmaf(b.z, b.z, q); q = fmaf(b.w, b.w, q);
              ss[t] = q;
            }
          }
        }
      }
    }
  }
}

// Top-k of one token by one warp.  Every lane ranks its own logits against all E of them (rank = number of
// logits that are larger, or equal with a lower expert id), so there are no selection rounds: the k logits of
// rank < k are the selection, in order.  Then softmax / sigmoid scores of the selected experts and their gates.
template <int NK>
__device__ __forceinline__ void topk_token(const DxRouteParams& p, const float* s_z, int* s_ids, float* s_w,
                                           unsigned int* s_mask, int* s_sel_e, float* s_sel_z, int tt, int lane) {
  const int E = p.E, k = p.k;
  const float* zrow = s_z + tt * E;
  float zv[NK];
  int rank[NK];
#pragma unroll
  for (int j = 0; j < NK; ++j) {
    const int ee = lane + 32 * j;
    zv[j] = ee < E ? zrow[ee] : 0.f;
    rank[j] = 0;
  }
  for (int o = 0; o < E; ++o) {
    const float zo = zrow[o];
#pragma unroll
    for (int j = 0; j < NK; ++j) {
      const int ee = lane + 32 * j;
      rank[j] += (zo > zv[j]) || (zo == zv[j] && o < ee);
    }
  }
#pragma unroll
  for (int j = 0; j < NK; ++j) {
    const int ee = lane + 32 * j;
    if (ee < E && rank[j] < k) { s_sel_e[tt * DX_MAX_TOPK + rank[j]] = ee; s_sel_z[tt * DX_MAX_TOPK + rank[j]] = zv[j]; }
  }
  __syncwarp();
  const float zmax = s_sel_z[tt * DX_MAX_TOPK];
  int my_e = 0;
  float my_z = 0.f;
  if (lane < k) { my_e = s_sel_e[tt * DX_MAX_TOPK + lane]; my_z = s_sel_z[tt * DX_MAX_TOPK + lane]; }
  my_e = min(max(my_e, 0), E - 1);   // whatever the logits were (NaNs rank nowhere), stay in range
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
  const float denom = warp_sum(psel);
  float g = p.norm_topk ? psel / denom : psel;
  g *= p.scale;
  if (lane < k) {
    s_ids[tt * k + lane] = my_e;
    s_w[tt * k + lane] = g;
    atomicOr(&s_mask[my_e >> 5], 1u << (my_e & 31));   // union of Eq. 2 / Eq. 3 as a bit mask
    dx_word_store(&p.work->pair[tt * k + lane], dx_pair_word(my_e, g));   // what the expert kernel waits for
    if (p.topk_ids) p.topk_ids[tt * k + lane] = my_e;
    if (p.topk_w) p.topk_w[tt * k + lane] = g;
  }
}

// TG: block rows per pass of the logits phase (1, 2, 4 or 8; the launcher picks the smallest that covers K, or 8)
template <typename WT, int TG>
__global__ void __launch_bounds__(kRouteThreads) dx_route_kernel(DxRouteParams p) {
  __shared__ float s_z[DX_MAX_K * DX_MAX_E];
  __shared__ int s_sel_e[DX_MAX_K * DX_MAX_TOPK];
  __shared__ float s_sel_z[DX_MAX_K * DX_MAX_TOPK];
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
  // hold back until this kernel publishes that the block input is final.
  if (p.handover && crank == 0) {
    // words left set by the previous pair: every CTA of that pair's expert kernel is past them (it lets this
    // kernel start only then), and the expert kernel of this pair cannot start before the trigger below
    if (threadIdx.x == 0) { atomicExch(p.handover, 0u); dx_word_store(&p.work->head, 0ull); }
    if (threadIdx.x < DX_MAX_PAIRS) dx_word_store(&p.work->group[threadIdx.x], 0ull);
    else if (threadIdx.x < 2 * DX_MAX_PAIRS) dx_word_store(&p.work->pair[threadIdx.x - DX_MAX_PAIRS], 0ull);
    __threadfence();
    __syncthreads();
  }
  dx_pdl_trigger();
  for (int i = threadIdx.x; i < DX_MAX_K * DX_MAX_TOPK; i += kRouteThreads) { s_sel_e[i] = 0; s_sel_z[i] = 0.f; }

  float* z0 = cluster.map_shared_rank(s_z, 0);
  const bool rms = p.rms_norm != 0;
  const int me = threadIdx.x;
  DxWork* W = p.work;
  {
    // everything this kernel reads or writes from here on may have been in use by the previous kernel
    dx_pdl_wait();
    if (p.handover && crank == 0 && threadIdx.x == 0) {
      __threadfence();
      atomicExch(p.handover, 1u);
    }
    if (crank == 0) {
      // routed part of the blob table, for the group list at the end; empty union mask
      if (threadIdx.x < E) s_tab[threadIdx.x] = p.table[p.n_shared + 1 + threadIdx.x];
      if (threadIdx.x < DX_MAX_E / 32) s_mask[threadIdx.x] = 0u;
    }
    // router logits z[t,e], written into CTA 0's table through distributed shared memory
    for (int t0 = 0; t0 < K; t0 += TG) {
      const int kt = min(TG, K - t0);
      const float* hb = p.h + (size_t)t0 * H;
      const int hs = H;
      for (int e = e_lo + warp; e < e_hi; e += kRouteWarps) {
        const WT* wrow = reinterpret_cast<const WT*>(p.W_r) + (size_t)e * H;
        const float b = p.bias ? p.bias[e] : 0.f;
        float acc[kTokGroup], ss[kTokGroup];
#pragma unroll
        for (int t = 0; t < kTokGroup; ++t) { acc[t] = 0.f; ss[t] = 0.f; }
        row_dots_direct<WT, TG>(wrow, hb, hs, H, kt, lane, rms, acc, ss);
#pragma unroll
        for (int t = 0; t < TG; ++t) {
          if (t < kt) {
            const float s = warp_sum(acc[t]);
            const float rs = rms ? rsqrtf(warp_sum(ss[t]) / (float)H + 1e-6f) : 1.0f;
            if (lane == 0) z0[(t0 + t) * E + e] = s * rs + b;
          }
        }
      }
    }
    {
      // y starts at zero, or as a copy of the block in the residual form; nothing reads it before this kernel
      // is over
      for (int j = (crank * kRouteThreads + threadIdx.x) * 4; j < K * H; j += kRouteCluster * kRouteThreads * 4) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.residual) v = *reinterpret_cast<const float4*>(p.h + j);
        *reinterpret_cast<float4*>(p.y + j) = v;
      }
    }
    cluster.sync();          // all logits have landed in CTA 0
    if (crank == 0) {
      // top-k and gate weights, one warp per token (NK = logits per lane, a power of two covering E)
      for (int tt = warp; tt < K; tt += kRouteWarps) {
        if (E <= 32) topk_token<1>(p, s_z, s_ids, s_w, s_mask, s_sel_e, s_sel_z, tt, lane);
        else if (E <= 64) topk_token<2>(p, s_z, s_ids, s_w, s_mask, s_sel_e, s_sel_z, tt, lane);
        else if (E <= 128) topk_token<4>(p, s_z, s_ids, s_w, s_mask, s_sel_e, s_sel_z, tt, lane);
        else topk_token<8>(p, s_z, s_ids, s_w, s_mask, s_sel_e, s_sel_z, tt, lane);
      }
      __syncthreads();

      // ---- group list for the expert kernel (it is waiting for it); the caller's outputs come afterwards
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
        if (flag) dx_word_store(&W->group[upos], dx_group_word(me, s_tab[me]));
      } else if (me < p.top_r) {
        dx_word_store(&W->group[me], dx_group_word(s_ids[me], s_tab[s_ids[me]]));
      }
      if (me == 0) dx_word_store(&W->head, dx_head_word(K, k, p.draft_mode ? p.top_r : ucount));

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
  }
}

}  // namespace

template <typename WT>
static cudaError_t launch_route_tg(const DxRouteParams& p, cudaStream_t st) {
  const dim3 grid(kRouteCluster), block(kRouteThreads);
  if (p.K <= 1) return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<WT, 1>, grid, block, 0, st, kRouteCluster, p);
  if (p.K <= 2) return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<WT, 2>, grid, block, 0, st, kRouteCluster, p);
  if (p.K <= 4) return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<WT, 4>, grid, block, 0, st, kRouteCluster, p);
  return dx_launch_pdl(DX_PDL_ROUTE, dx_route_kernel<WT, 8>, grid, block, 0, st, kRouteCluster, p);
}

cudaError_t dx_launch_route(const DxRouteParams& p, int weight_dtype, cudaStream_t st) {
  if (weight_dtype == DX_DTYPE_BF16) return launch_route_tg<__nv_bfloat16>(p, st);
  return launch_route_tg<float>(p, st);
}
