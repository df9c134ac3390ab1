// Routing kernel: router logits, scores, top-k with gate weights (Eq. 1, the
// g_{l,e} of Eq. 4), the block's expert union and the pair permutation grouped
// by expert (Eq. 2 / Eq. 3), and the work list the expert kernels consume.
//
// One thread-block cluster of 4 CTAs does all of it (few SMs, because the
// expert kernel runs beside it on all the others).  The contraction is split
// over the hidden dimension: CTA c owns a slice of the columns (and, for narrow
// layers, a share of the router rows).  Its part of the router matrix is a
// constant and sits in registers before the previous kernel of the stream has
// finished; once the block is final a thread needs two 16-byte loads per block
// row and slab, so a single memory round trip separates "block ready" from the
// arithmetic.  For a bf16 router and blocks of more than two rows the products
// run on the tensor cores (block rows as bf16 high part + residual, so the
// logits keep fp32-like accuracy; one partial table per warp, added in a fixed
// order); one or two rows and fp32 routers use plain FMAs.  Partial logits go
// into CTA 0's shared memory through distributed shared memory (one table per
// slice, summed in a fixed order, so the result does not depend on timing); the
// hand-over is one hardware cluster barrier.  CTA 0 then selects, one warp per
// token, in k rounds of warp-wide maximum on orderable keys, builds the union
// as a bit mask, publishes the group list the expert kernel is waiting for, and
// only then works out the gates and sorts the K*k (token, expert) pairs by
// expert for the caller's outputs.
#include <cooperative_groups.h>

#include <type_traits>

#include "dx_internal.cuh"
#include "dx_stream.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kRouteThreads = 256;
constexpr int kRouteCluster = DX_ROUTE_CLUSTER;
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

// Eight router columns as stored (bf16: one 16-byte load, fp32: two).
constexpr int kRowsPerBatch = 8;   // router rows a warp carries through one pass over its slice
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

// Sum N = 8, 16 or 32 per-lane values across the warp so that lane j (< N) ends up with the total of value j:
// each step halves the number of live values by exchanging the half the partner lane keeps (N - 1 shuffles
// instead of 5 N), and the lanes that share j then fold their subtotals.
template <int N>
__device__ __forceinline__ float warp_transpose_sum(float (&v)[N], int lane) {
#pragma unroll
  for (int o = N / 2; o >= 1; o >>= 1) {
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float keep = upper ? v[i + o] : v[i];
      const float send = upper ? v[i] : v[i + o];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
  float r = v[0];
#pragma unroll
  for (int o = N; o < 32; o <<= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
  return r;
}

// Top-k, in two steps so that the expert ids (all the expert kernel's producers need) are out before the gate
// arithmetic starts.  Selection of one token by one warp: k rounds of (lane-local best, warp maximum of the
// orderable logit, lowest expert id among the lanes that hold it); NK = logits per lane.
template <int NK>
__device__ __forceinline__ void topk_select(const DxRouteParams& p, const float* s_z, int* s_ids, unsigned int* s_mask,
                                            float* s_sel_z, int tt, int lane) {
  const int E = p.E, k = p.k;
  const float* zrow = s_z + tt * E;
  unsigned int key[NK];   // orderable logit; 0 = retired or out of range (a real logit never maps to 0)
  float zv[NK];
#pragma unroll
  for (int j = 0; j < NK; ++j) {
    const int ee = lane + 32 * j;
    zv[j] = ee < E ? zrow[ee] : 0.f;
    key[j] = ee < E ? dx_orderable(zv[j]) : 0u;
    if (ee < E && key[j] == 0u) key[j] = 1u;   // (only a NaN pattern maps to 0; keep it selectable)
  }
  int my_e = 0;
  float my_z = 0.f;
  for (int r = 0; r < k; ++r) {
    unsigned int lbest = 0u, lid = 0xffffffffu;
#pragma unroll
    for (int j = 0; j < NK; ++j)
      if (key[j] > lbest) { lbest = key[j]; lid = (unsigned int)(lane + 32 * j); }
    const unsigned int wbest = __reduce_max_sync(0xffffffffu, lbest);
    const int be = (int)__reduce_min_sync(0xffffffffu, lbest == wbest ? lid : 0xffffffffu);
    // the owning lane publishes the logit and retires the key
    float bz = 0.f;
#pragma unroll
    for (int j = 0; j < NK; ++j)
      if (lane + 32 * j == be) { bz = zv[j]; key[j] = 0u; }
    bz = __shfl_sync(0xffffffffu, bz, be & 31);
    if (lane == r) { my_e = be; my_z = bz; }
  }
  if (lane < k) {
    my_e = min(max(my_e, 0), E - 1);   // whatever the logits were, stay in range
    if (!DX_BOUNDS(tt * k + lane < DX_MAX_PAIRS && tt * DX_MAX_TOPK + lane < DX_MAX_K * DX_MAX_TOPK, p.dev_status)) return;
    s_sel_z[tt * DX_MAX_TOPK + lane] = my_z;
    s_ids[tt * k + lane] = my_e;
    if (!(p.skip_top1 && lane == 0))
      atomicOr(&s_mask[my_e >> 5], 1u << (my_e & 31));   // union of Eq. 2 / Eq. 3 as a bit mask
    if (p.topk_ids) p.topk_ids[tt * k + lane] = my_e;
    if (p.host_mirror && tt == 0) p.host_mirror[DX_MAX_E + 1 + lane] = my_e;
  }
}

// Softmax / sigmoid scores of the selected experts and their gate weights (the g_{l,e} of Eq. 4).
template <int NK>
__device__ __forceinline__ void topk_gates(const DxRouteParams& p, const float* s_z, const int* s_ids, float* s_w,
                                           const float* s_sel_z, int tt, int lane) {
  const int E = p.E, k = p.k;
  const float* zrow = s_z + tt * E;
  const float zmax = s_sel_z[tt * DX_MAX_TOPK];
  const float my_z = lane < k ? s_sel_z[tt * DX_MAX_TOPK + lane] : 0.f;
  float psel;
  if (p.score_fn == DX_SCORE_SOFTMAX) {
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < NK; ++j)
      if (lane + 32 * j < E) s += expf(zrow[lane + 32 * j] - zmax);
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
    s_w[tt * k + lane] = g;
    // for the consumers (the missing residual of Eq. 6 leaves the first selected expert's term out)
    dx_word_store(&p.work->pair[tt * k + lane], dx_pair_word(s_ids[tt * k + lane], (p.skip_top1 && lane == 0) ? 0.0f : g));
    if (p.topk_w) p.topk_w[tt * k + lane] = g;
  }
}

// How the cluster divides the contraction: S column slices (the largest divisor of H/256 that is at most the
// cluster size) of C 256-column slabs each, times R = cluster size / S shares of the router rows.
struct RouteSplit {
  int S, R, C, slice, share, e_lo, e_hi;
  bool idle;
};
__device__ __forceinline__ RouteSplit route_split(int H, int E, int crank) {
  RouteSplit q;
  const int slabs = H / 256;
  q.S = 1;
  for (int s = 2; s <= kRouteCluster; ++s)
    if (slabs % s == 0) q.S = s;
  q.R = kRouteCluster / q.S;
  q.C = slabs / q.S;
  q.idle = crank >= q.S * q.R;
  q.slice = crank % q.S;
  q.share = crank / q.S;
  const int per = (E + q.R - 1) / q.R;
  q.e_lo = min(E, q.share * per);
  q.e_hi = q.idle ? q.e_lo : min(E, q.e_lo + per);
  return q;
}

// TG: block rows per pass of the logits phase (1, 2 or 4; the launcher picks the smallest that covers K, or 4)
template <typename WT, int TG>
__global__ void __launch_bounds__(kRouteThreads) dx_route_kernel(DxRouteParams p) {
  __shared__ __align__(16) float s_z[DX_MAX_K * DX_MAX_E];
  __shared__ float s_bias[DX_MAX_E];
  __shared__ float s_sel_z[DX_MAX_K * DX_MAX_TOPK];
  __shared__ int s_ids[DX_MAX_PAIRS];
  __shared__ float s_w[DX_MAX_PAIRS];
  __shared__ int s_perm[DX_MAX_PAIRS];
  __shared__ int s_scan[kRouteWarps];
  __shared__ unsigned int s_mask[DX_MAX_E / 32];
  __shared__ const void* s_tab[DX_MAX_E];
  extern __shared__ __align__(16) float s_part[];   // CTA 0: [S][K*E + K] partial logits and sums of squares

  cg::cluster_group cluster = cg::this_cluster();
  const int crank = (int)cluster.block_rank();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int K = p.K, E = p.E, k = p.k, H = p.H, P = K * k;
  const RouteSplit sp = route_split(H, E, crank);
  const int part_stride = K * E + K;
  const int col0 = sp.slice * sp.C * 256 + 8 * lane;   // this lane's first column; slab c adds 256 c
  const WT* Wr = reinterpret_cast<const WT*>(p.W_r);

  // bf16 router and blocks of more than two rows: the contraction runs on the tensor cores (one or two rows are
  // quicker on the plain path: its arithmetic is small and it has no partial tables to merge)
  constexpr bool kMma = std::is_same<WT, __nv_bfloat16>::value && TG == 4;
  // the first batch of this warp's router rows (first kPreSlabs slabs of the slice): constant data, fetched right away
  constexpr int kPreSlabs = 2;
  constexpr int kPreTiles = 4;   // (tensor-core path) 16-row tiles of the router kept in registers
  RowRaw<WT> wpre[kMma ? 1 : kPreSlabs][kMma ? 1 : kRowsPerBatch];
  uint4 wa[kMma ? kPreTiles : 1][kMma ? kPreSlabs : 1][2];
  const int mg = lane >> 2, mc = lane & 3;
  // (tensor-core path) warp w owns the 32 columns [32 w, 32 w + 32) of every slab of the slice; a lane loads the
  // 8 columns 8 mc .. 8 mc + 7 of rows mg and mg + 8 of a tile -- its operand fragment of two contraction steps
  const int mcol0 = sp.slice * sp.C * 256 + 32 * warp + 8 * mc;
  const int n_et = sp.idle ? 0 : (sp.e_hi - sp.e_lo + 15) / 16;
  if constexpr (kMma) {
#pragma unroll
    for (int et = 0; et < kPreTiles; ++et)
#pragma unroll
      for (int c = 0; c < kPreSlabs; ++c) {
        if (et < n_et && c < sp.C) {
          const int e0 = min(sp.e_lo + 16 * et + mg, sp.e_hi - 1), e1 = min(sp.e_lo + 16 * et + mg + 8, sp.e_hi - 1);
          wa[et][c][0] = ldg_stream(Wr + (size_t)e0 * H + mcol0 + 256 * c);
          wa[et][c][1] = ldg_stream(Wr + (size_t)e1 * H + mcol0 + 256 * c);
        }
      }
  } else {
#pragma unroll
    for (int c = 0; c < kPreSlabs; ++c)
#pragma unroll
      for (int i = 0; i < kRowsPerBatch; ++i) {
        const int e = sp.e_lo + warp + kRouteWarps * i;
        if (c < sp.C && e < sp.e_hi) wpre[c][i].load(Wr + (size_t)e * H + col0 + 256 * c);
      }
  }
  if (crank == 0)
    for (int e = threadIdx.x; e < E; e += kRouteThreads) s_bias[e] = p.bias ? p.bias[e] : 0.f;
  for (int i = threadIdx.x; i < DX_MAX_K * DX_MAX_TOPK; i += kRouteThreads) s_sel_z[i] = 0.f;
  for (int i = threadIdx.x; i < DX_MAX_PAIRS; i += kRouteThreads) s_ids[i] = 0;

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
  // everything this kernel reads or writes from here on may have been in use by the previous kernel
  dx_pdl_wait();
  // "the block is final", for the expert kernel that is already resident.  The fence in front of the word costs
  // most of a microsecond; on the tensor-core path it is issued behind this thread's loads of the block rows, so the
  // two latencies overlap instead of adding up on the way to the group list.
  auto publish_block_final = [&]() {
    if (p.handover && crank == 0 && threadIdx.x == 0) {
      __threadfence();
      atomicExch(p.handover, 1u);
    }
  };
  if (!kMma) publish_block_final();
  // routed part of the blob table, for the group list at the end: fetched here, put into shared memory after the
  // partial logits (a store right away would hold these warps back for a memory round trip, in front of the loads
  // of the block rows everything else waits for)
  const void* tab_mine = nullptr;
  if (crank == 0) {
    if (threadIdx.x < E && DX_BOUNDS(E <= DX_MAX_E && E <= kRouteThreads, p.dev_status))
      tab_mine = p.table[p.n_shared + 1 + threadIdx.x];
    if (threadIdx.x < DX_MAX_E / 32) s_mask[threadIdx.x] = 0u;   // empty union mask
  }

  // ---- partial logits of this CTA's slice, into CTA 0's table for the slice
  float* part0 = cluster.map_shared_rank(s_part, 0) + (size_t)sp.slice * part_stride;
  const bool rms = p.rms_norm != 0;
  if constexpr (kMma) {
    // Tensor-core contraction: the block rows are the eight (sixteen) token columns, split into bf16 high part and
    // residual so that the logits keep fp32-like accuracy; a warp's products over its columns of every slab give
    // one partial table per warp, the eight tables are added in a fixed order.
    const int NTK = K > 8 ? 2 : 1, kpad = NTK * 8;
    const int red_stride = ((E + 15) / 16) * 16 * kpad;
    float* s_red = s_part + (size_t)kRouteCluster * part_stride;       // [8 warps][tiles * 16 rows][kpad tokens]
    float* s_ssq = s_red + (size_t)kRouteWarps * red_stride;           // [8 warps][kpad]
    uint4 bh[2][2], bl[2][2];   // [slab][token tile]
    float ssq[2] = {0.f, 0.f};
    float4 raw[2][2][2];
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int tok = nt * 8 + mg;
        raw[c][nt][0] = raw[c][nt][1] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < sp.C && nt < NTK && tok < K && !sp.idle) {
          const float* hp = p.h + (size_t)tok * H + mcol0 + 256 * c;
          raw[c][nt][0] = *reinterpret_cast<const float4*>(hp);
          raw[c][nt][1] = *reinterpret_cast<const float4*>(hp + 4);
        }
      }
    publish_block_final();
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        bh[c][nt] = bl[c][nt] = make_uint4(0u, 0u, 0u, 0u);
        const int tok = nt * 8 + mg;
        if (c < sp.C && nt < NTK && tok < K && !sp.idle) {
          const float4 v0 = raw[c][nt][0], v1 = raw[c][nt][1];
          const float x[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
          __nv_bfloat16 hb[8], lb[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            ssq[nt] = fmaf(x[i], x[i], ssq[nt]);
            split_bf16(x[i], hb[i], lb[i]);
          }
          bh[c][nt] = make_uint4(pack2(hb[0], hb[1]), pack2(hb[2], hb[3]), pack2(hb[4], hb[5]), pack2(hb[6], hb[7]));
          bl[c][nt] = make_uint4(pack2(lb[0], lb[1]), pack2(lb[2], lb[3]), pack2(lb[4], lb[5]), pack2(lb[6], lb[7]));
        }
      }
    // one 16-row tile of the router: products over this warp's columns of every slab, into the warp's table
    auto do_tile = [&](int et, const uint4 (&aw)[2][2]) {
      float cacc[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) cacc[nt][r] = 0.f;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        if (c >= sp.C) continue;
        const uint4 a0 = aw[c][0], a1 = aw[c][1];
        const uint4 f0 = make_uint4(a0.x, a1.x, a0.y, a1.y), f1 = make_uint4(a0.z, a1.z, a0.w, a1.w);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          if (nt >= NTK) continue;
          mma_k16(cacc[nt], f0, bh[c][nt].x, bh[c][nt].y);
          mma_k16(cacc[nt], f0, bl[c][nt].x, bl[c][nt].y);
          mma_k16(cacc[nt], f1, bh[c][nt].z, bh[c][nt].w);
          mma_k16(cacc[nt], f1, bl[c][nt].z, bl[c][nt].w);
        }
      }
      // rows mg and mg + 8 of the tile, tokens 2 mc and 2 mc + 1 of each token tile
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        if (nt >= NTK) continue;
        float* dst = s_red + (size_t)warp * red_stride + (size_t)(16 * et + mg) * kpad + nt * 8 + 2 * mc;
        *reinterpret_cast<float2*>(dst) = make_float2(cacc[nt][0], cacc[nt][1]);
        *reinterpret_cast<float2*>(dst + 8 * kpad) = make_float2(cacc[nt][2], cacc[nt][3]);
      }
    };
    // The preloaded tiles (held in registers since before the wait) are multiplied together, one product of every
    // tile after the other: the eight products of a tile form one dependent chain on its accumulator, and four
    // chains side by side take a quarter of the time of four chains one after the other.
    {
      float cacc[kPreTiles][2][4];
#pragma unroll
      for (int et = 0; et < kPreTiles; ++et)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int r = 0; r < 4; ++r) cacc[et][nt][r] = 0.f;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        if (c >= sp.C) continue;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          if (nt >= NTK) continue;
#pragma unroll
          for (int part = 0; part < 4; ++part) {   // high / low part of the block rows, first / second contraction step
#pragma unroll
            for (int et = 0; et < kPreTiles; ++et) {
              if (et >= n_et) continue;
              const uint4 a0 = wa[et][c][0], a1 = wa[et][c][1];
              const uint4 f = part < 2 ? make_uint4(a0.x, a1.x, a0.y, a1.y) : make_uint4(a0.z, a1.z, a0.w, a1.w);
              const uint4& b = (part & 1) ? bl[c][nt] : bh[c][nt];
              if (part < 2) mma_k16(cacc[et][nt], f, b.x, b.y);
              else mma_k16(cacc[et][nt], f, b.z, b.w);
            }
          }
        }
      }
#pragma unroll
      for (int et = 0; et < kPreTiles; ++et) {
        if (et >= n_et) continue;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          if (nt >= NTK) continue;
          float* dst = s_red + (size_t)warp * red_stride + (size_t)(16 * et + mg) * kpad + nt * 8 + 2 * mc;
          *reinterpret_cast<float2*>(dst) = make_float2(cacc[et][nt][0], cacc[et][nt][1]);
          *reinterpret_cast<float2*>(dst + 8 * kpad) = make_float2(cacc[et][nt][2], cacc[et][nt][3]);
        }
      }
    }
    for (int et = kPreTiles; et < n_et; ++et) {
      uint4 aw[2][2];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        aw[c][0] = aw[c][1] = make_uint4(0u, 0u, 0u, 0u);
        if (c < sp.C) {
          const int e0 = min(sp.e_lo + 16 * et + mg, sp.e_hi - 1), e1 = min(sp.e_lo + 16 * et + mg + 8, sp.e_hi - 1);
          aw[c][0] = ldg_stream(Wr + (size_t)e0 * H + mcol0 + 256 * c);
          aw[c][1] = ldg_stream(Wr + (size_t)e1 * H + mcol0 + 256 * c);
        }
      }
      do_tile(et, aw);
    }
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      float q = ssq[nt];
      q += __shfl_xor_sync(0xffffffffu, q, 1);
      q += __shfl_xor_sync(0xffffffffu, q, 2);
      if (mc == 0 && nt < NTK) s_ssq[warp * kpad + nt * 8 + mg] = q;
    }
    __syncthreads();
    const int n_rows = sp.idle ? 0 : sp.e_hi - sp.e_lo;
    for (int i = threadIdx.x; i < n_rows * K; i += kRouteThreads) {
      const int el = i / K, t = i - el * K;
      float z = 0.f;
#pragma unroll
      for (int w = 0; w < kRouteWarps; ++w) z += s_red[(size_t)w * red_stride + (size_t)el * kpad + t];
      part0[t * E + sp.e_lo + el] = z;
    }
    if (rms && sp.share == 0 && !sp.idle && threadIdx.x < K) {
      float q = 0.f;
#pragma unroll
      for (int w = 0; w < kRouteWarps; ++w) q += s_ssq[w * kpad + threadIdx.x];
      part0[K * E + threadIdx.x] = q;
    }
  } else {
  for (int t0 = 0; t0 < K; t0 += TG) {
    const int kt = min(TG, K - t0);
    float ss[TG];
#pragma unroll
    for (int t = 0; t < TG; ++t) ss[t] = 0.f;
    for (int r0 = sp.e_lo + warp; r0 < sp.e_hi; r0 += kRouteWarps * kRowsPerBatch) {
      float acc[kRowsPerBatch * TG];
#pragma unroll
      for (int i = 0; i < kRowsPerBatch * TG; ++i) acc[i] = 0.f;
      const bool first_rows = r0 == sp.e_lo + warp;
      for (int c = 0; c < sp.C; ++c) {
        // the block rows' part of this slab: two 16-byte loads per row, all in flight together
        float4 ha[TG], hb[TG];
#pragma unroll
        for (int t = 0; t < TG; ++t) {
          if (t < kt) {
            const float* hp = p.h + (size_t)(t0 + t) * H + col0 + 256 * c;
            ha[t] = *reinterpret_cast<const float4*>(hp);
            hb[t] = *reinterpret_cast<const float4*>(hp + 4);
          } else {
            ha[t] = hb[t] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        RowRaw<WT> wr[kRowsPerBatch];
#pragma unroll
        for (int i = 0; i < kRowsPerBatch; ++i) {
          const int e = r0 + kRouteWarps * i;
          if (first_rows && c == 0) wr[i] = wpre[0][i];
          else if (first_rows && c == 1) wr[i] = wpre[1][i];
          else if (e < sp.e_hi) wr[i].load(Wr + (size_t)e * H + col0 + 256 * c);
        }
        if (rms && first_rows && warp == 0 && sp.share == 0) {
#pragma unroll
          for (int t = 0; t < TG; ++t) {
            float q = ss[t];
            q = fmaf(ha[t].x, ha[t].x, q); q = fmaf(ha[t].y, ha[t].y, q); q = fmaf(ha[t].z, ha[t].z, q);
            q = fmaf(ha[t].w, ha[t].w, q); q = fmaf(hb[t].x, hb[t].x, q); q = fmaf(hb[t].y, hb[t].y, q);
            q = fmaf(hb[t].z, hb[t].z, q); q = fmaf(hb[t].w, hb[t].w, q);
            ss[t] = q;
          }
        }
#pragma unroll
        for (int i = 0; i < kRowsPerBatch; ++i) {
          if (r0 + kRouteWarps * i < sp.e_hi) {
            float wv[8];
            wr[i].unpack(wv);
#pragma unroll
            for (int t = 0; t < TG; ++t) {
              float s = acc[i * TG + t];
              s = fmaf(wv[0], ha[t].x, s); s = fmaf(wv[1], ha[t].y, s); s = fmaf(wv[2], ha[t].z, s);
              s = fmaf(wv[3], ha[t].w, s); s = fmaf(wv[4], hb[t].x, s); s = fmaf(wv[5], hb[t].y, s);
              s = fmaf(wv[6], hb[t].z, s); s = fmaf(wv[7], hb[t].w, s);
              acc[i * TG + t] = s;
            }
          }
        }
      }
      // lane j now gets the warp total of (row r0 + 8 (j / TG), block row t0 + j % TG)
      const float tot = warp_transpose_sum<kRowsPerBatch * TG>(acc, lane);
      const int e = r0 + kRouteWarps * (lane / TG), t = lane % TG;
      if (lane < kRowsPerBatch * TG && e < sp.e_hi && t < kt) part0[(t0 + t) * E + e] = tot;
    }
    if (rms && warp == 0 && sp.share == 0 && !sp.idle) {
#pragma unroll
      for (int t = 0; t < TG; ++t) {
        const float q = warp_sum(ss[t]);
        if (lane == 0 && t < kt) part0[K * E + t0 + t] = q;
      }
    }
  }
  }
  if (crank == 0 && threadIdx.x < E && threadIdx.x < DX_MAX_E) s_tab[threadIdx.x] = tab_mine;
  cluster.sync();          // all partial logits have landed in CTA 0
  if (crank != 0) {
    // y starts at zero, or as a copy of the block in the residual form; nothing reads it before this kernel is over,
    // so the CTAs that are done fill it while CTA 0 selects (in front of the barrier the copy -- one memory round
    // trip per 16 bytes and thread -- held the group list back by up to 3 us at sixteen rows)
    constexpr int kFill = 4;
    const int n_fill = (kRouteCluster - 1) * kRouteThreads;
    for (int j0 = ((crank - 1) * kRouteThreads + threadIdx.x) * 4; j0 < K * H; j0 += n_fill * 4 * kFill) {
      float4 v[kFill];
#pragma unroll
      for (int i = 0; i < kFill; ++i) {
        const int j = j0 + i * n_fill * 4;
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.residual && j < K * H) v[i] = *reinterpret_cast<const float4*>(p.h + j);
      }
#pragma unroll
      for (int i = 0; i < kFill; ++i) {
        const int j = j0 + i * n_fill * 4;
        if (j < K * H) *reinterpret_cast<float4*>(p.y + j) = v[i];
      }
    }
    return;
  }

  // logits: slices summed in a fixed order, RMSNorm scale and bias applied
  for (int idx = threadIdx.x; idx < K * E; idx += kRouteThreads) {
    const int t = idx / E, e = idx - t * E;
    float z = 0.f, q = 0.f;
#pragma unroll 8
    for (int s2 = 0; s2 < sp.S; ++s2) {
      z += s_part[s2 * part_stride + idx];
      if (rms) q += s_part[s2 * part_stride + K * E + t];
    }
    const float rs = rms ? rsqrtf(q / (float)H + 1e-6f) : 1.0f;
    s_z[idx] = z * rs + s_bias[e];
  }
  __syncthreads();

  // selection, one warp per token
  for (int tt = warp; tt < K; tt += kRouteWarps) {
    if (E <= 32) topk_select<1>(p, s_z, s_ids, s_mask, s_sel_z, tt, lane);
    else if (E <= 64) topk_select<2>(p, s_z, s_ids, s_mask, s_sel_z, tt, lane);
    else if (E <= 128) topk_select<4>(p, s_z, s_ids, s_mask, s_sel_z, tt, lane);
    else topk_select<8>(p, s_z, s_ids, s_mask, s_sel_z, tt, lane);
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
    if (flag && DX_BOUNDS(upos < DX_MAX_PAIRS && upos < K * k, p.dev_status))
      dx_word_store(&W->group[upos], dx_group_word(me, s_tab[me]));
  } else if (me < p.top_r && DX_BOUNDS(me < DX_MAX_PAIRS && s_ids[me] >= 0 && s_ids[me] < E, p.dev_status)) {
    dx_word_store(&W->group[me], dx_group_word(s_ids[me], s_tab[s_ids[me]]));
  }
  if (me == 0) dx_word_store(&W->head, dx_head_word(K, k, p.draft_mode ? p.top_r : ucount));

  // ---- gate weights: the expert kernel's consumers pick the pairs up when they reach the first routed group
  for (int tt = warp; tt < K; tt += kRouteWarps) {
    if (E <= 32) topk_gates<1>(p, s_z, s_ids, s_w, s_sel_z, tt, lane);
    else if (E <= 64) topk_gates<2>(p, s_z, s_ids, s_w, s_sel_z, tt, lane);
    else if (E <= 128) topk_gates<4>(p, s_z, s_ids, s_w, s_sel_z, tt, lane);
    else topk_gates<8>(p, s_z, s_ids, s_w, s_sel_z, tt, lane);
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
      if (s_ids[q] == me && DX_BOUNDS(off + i < P, p.dev_status)) s_perm[off + i++] = q;
    if (p.offsets) p.offsets[me] = off;
    if (flag && p.union_ids && DX_BOUNDS(upos < min(E, P), p.dev_status)) p.union_ids[upos] = me;
    if (flag && p.host_mirror && DX_BOUNDS(upos < min(E, P), p.dev_status)) p.host_mirror[upos] = me;
  }
  if (me == 0) {
    if (p.offsets) p.offsets[E] = P;
    if (p.union_count) *p.union_count = ucount;
    if (p.host_mirror) p.host_mirror[DX_MAX_E] = ucount;
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

template <typename WT, int TG>
static cudaError_t launch_route_one(dx_ctx* ctx, const DxRouteParams& p, cudaStream_t st) {
  // CTA 0 holds one partial table per column slice (at most one per CTA of the cluster)
  size_t smem = (size_t)kRouteCluster * ((size_t)p.K * p.E + p.K) * sizeof(float);
  // (tensor-core path) one partial table per warp: [8][tiles of 16 router rows][8 or 16 token columns], sums of squares
  const size_t kpad = p.K > 8 ? 16 : 8;
  if (std::is_same<WT, __nv_bfloat16>::value && TG == 4)
    smem += (size_t)kRouteWarps * ((size_t)((p.E + 15) / 16) * 16 * kpad + kpad) * sizeof(float);
  // static + dynamic shared memory can pass the default 48 KB: opt in once per instantiation for the largest case
  static bool opted_in = false;
  if (!opted_in) {
    size_t most = (size_t)kRouteCluster * ((size_t)DX_MAX_K * DX_MAX_E + DX_MAX_K) * sizeof(float);
    if (std::is_same<WT, __nv_bfloat16>::value && TG == 4)
      most += (size_t)kRouteWarps * ((size_t)DX_MAX_E * 16 + 16) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(dx_route_kernel<WT, TG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
    if (e != cudaSuccess) return e;
    opted_in = true;
  }
  return dx_launch_pdl((ctx->pdl_mask & DX_PDL_ROUTE) != 0, dx_route_kernel<WT, TG>, dim3(kRouteCluster), dim3(kRouteThreads), smem, st,
                       kRouteCluster, p);
}

template <typename WT>
static cudaError_t launch_route_tg(dx_ctx* ctx, const DxRouteParams& p, cudaStream_t st) {
  if (p.K <= 1) return launch_route_one<WT, 1>(ctx, p, st);
  if (p.K <= 2) return launch_route_one<WT, 2>(ctx, p, st);
  return launch_route_one<WT, 4>(ctx, p, st);
}

cudaError_t dx_launch_route(dx_ctx* ctx, const DxRouteParams& p, int weight_dtype, cudaStream_t st) {
  if (weight_dtype == DX_DTYPE_BF16) return launch_route_tg<__nv_bfloat16>(ctx, p, st);
  return launch_route_tg<float>(ctx, p, st);
}
