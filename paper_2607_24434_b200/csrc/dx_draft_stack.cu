// Draft stack: Eq. 5 for one token through a whole stack of layers in ONE persistent kernel,
//     h_{l+1} = h_l + S_l(x) + g_{l,e1} E_{l,e1}(x) + gamma_l E^d_l(x),   x = RMSNorm(h_l),   l = 0 .. L-1.
//
// Per layer the drafter reads four experts' worth of weights (69 MB at the DeepSeek-V2-Lite shape) for a single
// token, so a layer lasts ~10 us at HBM speed and every microsecond between two layers shows.  One launch per layer
// pays a kernel boundary each time; here one cooperative grid (one CTA per SM) stays resident for all layers:
//   * every CTA keeps the hidden row in shared memory.  A layer's contributions are added (vector reductions in
//     L2) to that layer's own delta rows in global memory, zero at launch -- a few partial rows per layer, CTA c
//     into row c mod DX_STACK_COPIES, because additions to one address are serial in L2; once the layer's arrival
//     counter shows all CTAs, each CTA (all its warps but the producer) adds the partial rows to its copy.  No row
//     is ever initialised or copied between layers, and the counter is the only grid-wide wait of a layer;
//   * the producer warp of every CTA streams its share of the layer's routing-independent units (shared experts,
//     draft expert) and, because weights are constants, runs ahead into the next layer while the current one is
//     still being reduced -- the ring does not drain at a layer boundary;
//   * a router warp per CTA advances the hidden row, computes one router row of the layer (rows are dealt over the
//     CTAs; the weights are in registers before the row is final) and publishes the logit as a self-validating
//     64-bit word; every router warp polls the E words, selects the top-k itself (identical arithmetic, identical
//     result) and tells its CTA which routed expert to stream;
//   * eight consumer warps do the SwiGLU on the units' fragments (the grouped kernel's layout) with plain FMAs --
//     one token leaves the tensor cores nothing to amortise -- and keep the layer's partial output in registers
//     until the layer's flush.
// The kernel is launched cooperatively, which either places the whole grid at once or fails the launch.  Every
// wait on another CTA is bounded and ends in the device status word.
#include <cooperative_groups.h>
#include <cuda_fp16.h>

#include "dx_internal.cuh"
#include "dx_stream.cuh"


namespace {

constexpr int kStackConsumers = 8;
constexpr int kStackThreads = (kStackConsumers + 2) * 32;   // consumers, producer warp, router warp
constexpr int kStackMaxSlots = 48;
constexpr int kStackPartialBytes = 2 * 8 * 8 * 8;   // [2][warp][row] (gate, up) partial sums

struct StackSmem {
  unsigned long long full[kStackMaxSlots];
  unsigned long long empty[kStackMaxSlots];
  int abort_flag;
  float ssq[kStackConsumers];   // sums of squares of the current hidden row, one per consumer warp
  // what the router warp found for the current layer
  int r_have;                    // 0: the routed expert has no blob (reported; the layer goes on without it)
  float r_w;                     // its gate
  const unsigned char* r_blob;   // for the producer
};

__device__ __forceinline__ float stack_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// Bounded wait until a counter in global memory has reached `want`.
__device__ __forceinline__ bool counter_wait(const unsigned int* word, unsigned int want, uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(word) : "memory");
    if (v >= want) return true;
    __nanosleep(32);
  }
  return false;
}
__device__ __forceinline__ float bf_lo(unsigned int u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(unsigned int u) { return __uint_as_float(u & 0xffff0000u); }
// Two 4-bit codes (bits [0,4) and [16,20)) -> the bf16 pair (code - 8): 0x4300 | code is 128 + code in bf16.
__device__ __forceinline__ uint32_t q4s_pair(uint32_t w) {
  const uint32_t v = (w & 0x000F000Fu) | 0x43004300u;
  const __nv_bfloat162 r = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&v), __floats2bfloat162_rn(136.f, 136.f));
  return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ void unpack8(const uint4& r, float (&v)[8]) {
  const unsigned int u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
  }
}

// This CTA's units of a layer: [s_lo, s_hi) of the NS routing-independent units and [r_lo, r_hi) of the NR units of
// the routed expert, balanced together.
__device__ __forceinline__ void stack_shares(int NS, int NR, int G, int cta, int& s_lo, int& s_hi, int& r_lo, int& r_hi) {
  s_lo = (int)(((long long)NS * cta) / G);
  s_hi = (int)(((long long)NS * (cta + 1)) / G);
  const long long T = (long long)NS + NR;
  if (T / G >= (NS + G - 1) / G) {
    r_lo = (int)((T * cta) / G) - s_lo;
    r_hi = (int)((T * (cta + 1)) / G) - s_hi;
  } else {
    r_lo = (int)(((long long)NR * cta) / G);
    r_hi = (int)(((long long)NR * (cta + 1)) / G);
  }
  r_lo = min(max(r_lo, 0), NR);
  r_hi = min(max(r_hi, r_lo), NR);
}

// Q4: units of 4-bit codes and fp16 block scales (the grouped kernel's packed 4-bit layout), converted in registers.
template <int H, bool Q4>
__global__ void __launch_bounds__(kStackThreads, 1) dx_draft_stack_kernel(DxStackParams p, int n_slots) {
  constexpr int KW = H / 128;        // phase-1 contraction steps per consumer warp
  constexpr int PW = H / 256;        // phase-2 row-tile pairs per consumer warp
  constexpr uint32_t CHUNK = Q4 ? KW * 144u + PW * 192u : KW * 512u + PW * 512u;
  constexpr uint32_t UNIT_BYTES = 8u * CHUNK;

  extern __shared__ __align__(128) unsigned char smem[];
  StackSmem* hdr = reinterpret_cast<StackSmem*>(smem);
  constexpr size_t HDR = (sizeof(StackSmem) + 127) / 128 * 128;
  float2* partial = reinterpret_cast<float2*>(smem + HDR);                          // [2][8][8]
  constexpr size_t PART = kStackPartialBytes;
  float* x_s = reinterpret_cast<float*>(smem + HDR + PART);                         // [H] the hidden row
  unsigned char* ring = smem + HDR + PART + (size_t)H * 4;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  const int L = p.n_layers, E = p.E;
  const int NS = p.n_shared * p.shared_tiles + p.draft_tiles, NR = p.routed_tiles;
  volatile int* abort_flag = &hdr->abort_flag;
  int s_lo, s_hi, r_lo, r_hi;
  stack_shares(NS, NR, G, cta, s_lo, s_hi, r_lo, r_hi);

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_slots; ++s) {
      mbar_init(smem_u32(&hdr->full[s]), 1);
      mbar_init(smem_u32(&hdr->empty[s]), 1);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int j = threadIdx.x * 4; j < H; j += kStackThreads * 4)
    *reinterpret_cast<float4*>(x_s + j) = *reinterpret_cast<const float4*>(p.h_in + j);
  __syncthreads();

  // Advance the hidden row by the finished layer's partial rows (layer l - 1; nothing to add for l = 0) and collect
  // its sum of squares.  Done by the eight consumer warps together (they have nothing else to do at this point, and
  // the router warp keeps its registers for the router rows it has fetched): every thread owns one or two 16-byte
  // pieces of the row and has the pieces of all partial rows in flight at once (one memory round trip).
  constexpr int kAdvThreads = kStackConsumers * 32;
  constexpr int kAdvPieces = (H / 4 + kAdvThreads - 1) / kAdvThreads;
  auto advance_row = [&](int l, int q) {   // q: 0 .. kAdvThreads - 1 (the consumer's thread index)
    float4 part[kAdvPieces][DX_STACK_COPIES];
    if (l > 0) {
#pragma unroll
      for (int n = 0; n < kAdvPieces; ++n) {
        const int j = (q + n * kAdvThreads) * 4;
#pragma unroll
        for (int c = 0; c < DX_STACK_COPIES; ++c)
          part[n][c] = j < H ? __ldcg(reinterpret_cast<const float4*>(p.delta + ((size_t)(l - 1) * DX_STACK_COPIES + c) * H + j))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    float ss = 0.f;
#pragma unroll
    for (int n = 0; n < kAdvPieces; ++n) {
      const int j = (q + n * kAdvThreads) * 4;
      if (j < H) {
        float4 v = *reinterpret_cast<float4*>(x_s + j);
        if (l > 0) {
#pragma unroll
          for (int c = 0; c < DX_STACK_COPIES; ++c) { v.x += part[n][c].x; v.y += part[n][c].y; v.z += part[n][c].z; v.w += part[n][c].w; }
          *reinterpret_cast<float4*>(x_s + j) = v;
        }
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      }
    }
    ss = stack_warp_sum(ss);
    if ((q & 31) == 0) hdr->ssq[q >> 5] = ss;
  };
  auto row_rstd = [&]() {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kStackConsumers; ++w) t += hdr->ssq[w];
    return rsqrtf(t / (float)H + 1e-6f);
  };

  if (warp == kStackConsumers) {
    // ---------------------------------------------------------------- producer
    uint32_t it = 0, slot = 0, phase = 0;   // chunk counter, its ring slot and that slot's phase bit
    const uint64_t l2pol = l2_evict_first_policy();
    auto static_unit = [&](int l, int u) -> const unsigned char* {
      const int grp = u < p.n_shared * p.shared_tiles ? u / p.shared_tiles : p.n_shared;
      const int first = grp < p.n_shared ? grp * p.shared_tiles : p.n_shared * p.shared_tiles;
      const unsigned char* blob = reinterpret_cast<const unsigned char*>(p.layers[l].table[grp]);
      return blob ? blob + (size_t)(u - first) * UNIT_BYTES : nullptr;
    };
    auto push_chunk = [&](const unsigned char* src) {
      // nothing more is copied once anything has given up (see mbar_wait)
      if (!mbar_wait(smem_u32(&hdr->empty[slot]), phase ^ 1u, abort_flag, p.wait_limit)) return;
      const uint32_t fb = smem_u32(&hdr->full[slot]);
      mbar_arrive_expect_tx(fb, CHUNK);
      bulk_g2s(smem_u32(ring + (size_t)slot * CHUNK), src, CHUNK, fb, l2pol);
      ++it;
      if (++slot == (uint32_t)n_slots) { slot = 0; phase ^= 1u; }
    };
    for (int l = 0; l < L; ++l) {
      if (lane == 0) {
#pragma unroll 1
        for (int u = s_lo; u < s_hi; ++u) {
          const unsigned char* src = static_unit(l, u);
          if (src) {
#pragma unroll 1
            for (int w = 0; w < kStackConsumers; ++w) push_chunk(src + (size_t)w * CHUNK);
          } else {
            *abort_flag = 1;   // (the entry point refuses stacks with missing experts; never expected)
          }
        }
      }
      __syncwarp();
      asm volatile("bar.sync 2, 64;" ::: "memory");   // the router warp knows this layer's routed expert
      if (lane == 0) {
        const unsigned char* blob = hdr->r_blob;
        if (blob) {
#pragma unroll 1
          for (int c = r_lo * kStackConsumers; c < r_hi * kStackConsumers; ++c) push_chunk(blob + (size_t)c * CHUNK);
        }
      }
      __syncwarp();
    }
    if (lane == 0 && *abort_flag) {
      // something gave up: make sure no copy is still landing in this CTA's shared memory before it is released
      const uint32_t n_back = it < (uint32_t)n_slots ? it : (uint32_t)n_slots;
      for (uint32_t k = 1; k <= n_back; ++k) {
        const uint32_t j = it - k, s = j % (uint32_t)n_slots, ph = (j / (uint32_t)n_slots) & 1u;
        for (uint32_t spin = 0; spin < DX_WAIT_LIMIT_DEFAULT; ++spin)
          if (mbar_try_wait(smem_u32(&hdr->full[s]), ph)) break;
      }
      atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED);
    }
    return;
  }

  if (warp == kStackConsumers + 1) {
    // ---------------------------------------------------------------- router
    constexpr int WV = H / 256;   // 16-byte pieces of a router row per lane
    for (int l = 0; l <= L; ++l) {
      // the first of this CTA's router rows, on its way before the hidden row is final
      uint4 wreg[WV];
      if (l < L && cta < E) {
        const uint4* wrow = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.layers[l].W_r) +
                                                          (size_t)cta * H);
#pragma unroll
        for (int i = 0; i < WV; ++i) wreg[i] = wrow[lane + 32 * i];
      }
      bool ok = true;
      if (l > 0 && lane == 0) ok = counter_wait(p.sync + (l - 1), (unsigned int)G, p.wait_limit);   // layer l-1 is complete
      __syncwarp();   // orders the other lanes' reads of the delta row behind lane 0's acquire (a shuffle would not)
      ok = __shfl_sync(0xffffffffu, ok, 0);
      asm volatile("bar.sync 5, 288;" ::: "memory");   // the finished layer's sums are complete: the consumers advance the row
      asm volatile("bar.sync 3, 288;" ::: "memory");   // the row is advanced, its sums of squares are in place
      if (l == L) {   // past the last layer: the row is the result
        if (cta == 0) {
          for (int j = lane * 4; j < H; j += 128)
            *reinterpret_cast<float4*>(p.h_out + j) = *reinterpret_cast<const float4*>(x_s + j);
        }
        if (!ok && lane == 0) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
        break;
      }
      const DxStackLayer& ly = p.layers[l];
      const float rstd = row_rstd();
      // this CTA's router rows, each logit published as (1 << 32 | float bits)
      for (int e = cta; e < E; e += G) {
        float acc = 0.f;
        if (e != cta) {
          const uint4* wrow = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(ly.W_r) + (size_t)e * H);
#pragma unroll
          for (int i = 0; i < WV; ++i) wreg[i] = wrow[lane + 32 * i];
        }
#pragma unroll
        for (int i = 0; i < WV; ++i) {
          const int j = (lane + 32 * i) * 8;
          const float4 a = *reinterpret_cast<const float4*>(x_s + j);
          const float4 b = *reinterpret_cast<const float4*>(x_s + j + 4);
          float w8[8];
          unpack8(wreg[i], w8);
          acc = fmaf(w8[0], a.x, acc); acc = fmaf(w8[1], a.y, acc); acc = fmaf(w8[2], a.z, acc); acc = fmaf(w8[3], a.w, acc);
          acc = fmaf(w8[4], b.x, acc); acc = fmaf(w8[5], b.y, acc); acc = fmaf(w8[6], b.z, acc); acc = fmaf(w8[7], b.w, acc);
        }
        acc = stack_warp_sum(acc);
        if (lane == 0) {
          const float z = acc * rstd + (ly.bias ? ly.bias[e] : 0.f);
          dx_word_store(p.zword + (size_t)l * E + e, (1ull << 32) | (unsigned long long)__float_as_uint(z));
        }
      }
      // all E logits (E <= 256: up to eight per lane), polled until every word is there
      unsigned int key[8];
      float zv[8];
      {
        unsigned long long zw[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) zw[j] = 0ull;
        bool all = false;
        for (uint32_t spin = 0; spin < p.wait_limit && !all; ++spin) {
          bool mine = true;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int ee = lane + 32 * j;
            if (ee < E && zw[j] == 0ull) {
              zw[j] = dx_word_load(p.zword + (size_t)l * E + ee);
              mine = mine && zw[j] != 0ull;
            }
          }
          all = __all_sync(0xffffffffu, mine);
        }
        ok = ok && all;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int ee = lane + 32 * j;
          zv[j] = ee < E ? __uint_as_float((unsigned int)zw[j]) : 0.f;
          key[j] = ee < E ? max(dx_orderable(zv[j]), 1u) : 0u;
        }
      }
      // top-k: k rounds of (lane-local best, warp maximum of the orderable logit, lowest expert id among its
      // holders), then the gates of Eq. 4
      int my_e = 0;
      float my_z = 0.f, zmax = 0.f;
      for (int r = 0; r < p.k; ++r) {
        unsigned int lbest = 0u, lid = 0xffffffffu;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (key[j] > lbest) { lbest = key[j]; lid = (unsigned int)(lane + 32 * j); }
        const unsigned int wbest = __reduce_max_sync(0xffffffffu, lbest);
        const int be = (int)__reduce_min_sync(0xffffffffu, lbest == wbest ? lid : 0xffffffffu);
        float bz = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (lane + 32 * j == be) { bz = zv[j]; key[j] = 0u; }
        bz = __shfl_sync(0xffffffffu, bz, be & 31);
        if (r == 0) {
          // the routed expert is known: the producer goes on while the rest of the selection and the gates are
          // worked out
          zmax = bz;
          const int e1 = min(max(be, 0), E - 1);
          if (lane == 0) {
            const unsigned char* blob = reinterpret_cast<const unsigned char*>(ly.table[p.n_shared + 1 + e1]);
            hdr->r_blob = blob;
            hdr->r_have = blob != nullptr;
            if (!blob) atomicExch(p.dev_status, DX_DEV_BAD_EXPERT_ID);
            if (!ok) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
          }
          __threadfence_block();
          __syncwarp();
          asm volatile("bar.sync 2, 64;" ::: "memory");
        }
        if (lane == r) { my_e = be; my_z = bz; }
      }
      my_e = min(max(my_e, 0), E - 1);
      float psel;
      if (p.score_fn == DX_SCORE_SOFTMAX) {
        float sden = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (lane + 32 * j < E) sden += expf(zv[j] - zmax);
        sden = stack_warp_sum(sden);
        psel = expf(my_z - zmax) / sden;
      } else {
        psel = 1.0f / (1.0f + expf(-my_z));
      }
      if (lane >= p.k) psel = 0.f;
      const float denom = stack_warp_sum(psel);
      const float gate = (p.norm_topk ? psel / denom : psel) * p.scale;
      if (cta == 0 && lane < p.k) {
        if (p.topk_ids) p.topk_ids[l * p.k + lane] = my_e;
        if (p.topk_w) p.topk_w[l * p.k + lane] = gate;
      }
      const float g1 = __shfl_sync(0xffffffffu, gate, 0);
      if (lane == 0) hdr->r_w = g1;
      __threadfence_block();
      __syncwarp();
      asm volatile("bar.sync 4, 288;" ::: "memory");   // the consumers may weigh the routed expert
    }
    return;
  }

  // ------------------------------------------------------------------ consumers
  const int g = lane >> 2, c = lane & 3;
  uint32_t cslot = (uint32_t)warp, cphase = 0;   // ring slot (and its phase bit) of this warp's chunk of the next unit
  int buf = 0;
  for (int l = 0; l <= L; ++l) {
    asm volatile("bar.sync 5, 288;" ::: "memory");   // the router warp has seen every CTA's arrival for layer l - 1
    advance_row(l, threadIdx.x);
    asm volatile("bar.sync 3, 288;" ::: "memory");   // the hidden row stands at layer l
    if (l == L) break;   // (the router warp of CTA 0 writes the result)
    // the token fragments of this warp's contraction slice: token slot 0 is the normalised row, the other seven
    // slots are zero
    const float rs = row_rstd();
    // One token only: the tensor cores would spend seven of their eight token columns (and a second pass for the
    // low halves of the activations) on nothing, and at one token their issue rate, not the stream, sets the
    // pace.  The same fragments are consumed with plain FMAs instead: a lane holds rows g and g + 8 of a
    // 16-row tile at four hidden positions per contraction step, so it needs one float4 of the normalised row
    // per step, kept in registers for the whole layer.
    float4 xr[KW];
#pragma unroll
    for (int i = 0; i < KW; ++i) {
      const float4 v = *reinterpret_cast<const float4*>(x_s + 16 * (warp * KW + i) + 4 * c);
      xr[i] = make_float4(v.x * rs, v.y * rs, v.z * rs, v.w * rs);
    }
    float acc[2 * PW][2];   // [tile][row g | row g + 8]: this lane's two contraction columns of the down projection
#pragma unroll
    for (int j = 0; j < 2 * PW; ++j) acc[j][0] = acc[j][1] = 0.f;

    // one unit with weight wu
    auto unit = [&](float wu) {
      const uint32_t s = cslot, ph = cphase;
      cslot += kStackConsumers;   // (a ring has more slots than a unit has chunks: at most one wrap)
      if (cslot >= (uint32_t)n_slots) { cslot -= (uint32_t)n_slots; cphase ^= 1u; }
      const uint4* A = reinterpret_cast<const uint4*>(ring + (size_t)s * CHUNK) + lane;
      mbar_wait(smem_u32(&hdr->full[s]), ph, abort_flag, p.wait_limit);
      // gate (rows 0..7 of the tile) and up (rows 8..15) over this warp's slice of the hidden dimension
      float ga = 0.f, gb = 0.f, ua = 0.f, ub = 0.f;
      if constexpr (Q4) {
        // a 32-wide quantisation block is two contraction steps; its sums are scaled by the rows' block scales
        const unsigned char* Cq = ring + (size_t)s * CHUNK;
        const uint2* Aq = reinterpret_cast<const uint2*>(Cq) + lane;
        const __half2* S1 = reinterpret_cast<const __half2*>(Cq + KW * 128) + g;
#pragma unroll
        for (int b = 0; b < KW / 2; ++b) {
          const uint2 cw = Aq[b * 32];
          const float2 sc = __half22float2(S1[b * 8]);
          float gs = 0.f, us = 0.f;
#pragma unroll
          for (int ks = 0; ks < 2; ++ks) {
            const uint32_t w = ks ? cw.y : cw.x;
            const float4 x4 = xr[2 * b + ks];
            const uint32_t p0 = q4s_pair(w), p1 = q4s_pair(w >> 4), p2 = q4s_pair(w >> 8), p3 = q4s_pair(w >> 12);
            gs = fmaf(bf_lo(p0), x4.x, gs); gs = fmaf(bf_hi(p0), x4.y, gs);
            us = fmaf(bf_lo(p1), x4.x, us); us = fmaf(bf_hi(p1), x4.y, us);
            gs = fmaf(bf_lo(p2), x4.z, gs); gs = fmaf(bf_hi(p2), x4.w, gs);
            us = fmaf(bf_lo(p3), x4.z, us); us = fmaf(bf_hi(p3), x4.w, us);
          }
          if (b & 1) { gb = fmaf(sc.x, gs, gb); ub = fmaf(sc.y, us, ub); }
          else { ga = fmaf(sc.x, gs, ga); ua = fmaf(sc.y, us, ua); }
        }
      } else {
#pragma unroll
        for (int i = 0; i < KW; ++i) {
          const uint4 a = A[i * 32];
          ga = fmaf(bf_lo(a.x), xr[i].x, ga); gb = fmaf(bf_hi(a.x), xr[i].y, gb);
          ua = fmaf(bf_lo(a.y), xr[i].x, ua); ub = fmaf(bf_hi(a.y), xr[i].y, ub);
          ga = fmaf(bf_lo(a.z), xr[i].z, ga); gb = fmaf(bf_hi(a.z), xr[i].w, gb);
          ua = fmaf(bf_lo(a.w), xr[i].z, ua); ub = fmaf(bf_hi(a.w), xr[i].w, ub);
        }
      }
      float gt = ga + gb, ut = ua + ub;
      gt += __shfl_xor_sync(0xffffffffu, gt, 1); ut += __shfl_xor_sync(0xffffffffu, ut, 1);
      gt += __shfl_xor_sync(0xffffffffu, gt, 2); ut += __shfl_xor_sync(0xffffffffu, ut, 2);
      float2* part = partial + buf * 64;   // [warp][row]
      if (c == 0) part[warp * 8 + g] = make_float2(gt, ut);
      consumer_bar();
      // every warp sums the eight slices (fixed order) and activates: lane r < 8 holds intermediate row r
      float act = 0.f;
      if (lane < 8) {
        float2 t = part[lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) {
          const float2 q = part[w * 8 + lane];
          t.x += q.x; t.y += q.y;
        }
        act = fast_silu(t.x) * t.y * wu;
      }
      const float act0 = __shfl_sync(0xffffffffu, act, 2 * c), act1 = __shfl_sync(0xffffffffu, act, 2 * c + 1);
      buf ^= 1;
      // down projection: a lane holds rows g and g + 8 of two 16-row tiles at intermediate rows 2c and 2c + 1
      if constexpr (Q4) {
        // the eight columns of a unit lie in one quantisation block of W_d: one scale per output row
        const unsigned char* Cq = ring + (size_t)s * CHUNK + KW * 144;
        const uint32_t* Dq = reinterpret_cast<const uint32_t*>(Cq) + lane;
        const uint2* S2 = reinterpret_cast<const uint2*>(Cq + PW * 128) + g;
#pragma unroll
        for (int q2 = 0; q2 < PW; ++q2) {
          const uint32_t w = Dq[q2 * 32];
          const uint2 sw = S2[q2 * 8];
          const float2 s01 = __half22float2(*reinterpret_cast<const __half2*>(&sw.x));
          const float2 s23 = __half22float2(*reinterpret_cast<const __half2*>(&sw.y));
          const uint32_t p0 = q4s_pair(w), p1 = q4s_pair(w >> 4), p2 = q4s_pair(w >> 8), p3 = q4s_pair(w >> 12);
          acc[2 * q2][0] = fmaf(s01.x, fmaf(bf_hi(p0), act1, bf_lo(p0) * act0), acc[2 * q2][0]);
          acc[2 * q2][1] = fmaf(s01.y, fmaf(bf_hi(p1), act1, bf_lo(p1) * act0), acc[2 * q2][1]);
          acc[2 * q2 + 1][0] = fmaf(s23.x, fmaf(bf_hi(p2), act1, bf_lo(p2) * act0), acc[2 * q2 + 1][0]);
          acc[2 * q2 + 1][1] = fmaf(s23.y, fmaf(bf_hi(p3), act1, bf_lo(p3) * act0), acc[2 * q2 + 1][1]);
        }
      } else {
        const uint4* D = A + KW * 32;
#pragma unroll
        for (int q2 = 0; q2 < PW; ++q2) {
          const uint4 a = D[q2 * 32];
          acc[2 * q2][0] = fmaf(bf_hi(a.x), act1, fmaf(bf_lo(a.x), act0, acc[2 * q2][0]));
          acc[2 * q2][1] = fmaf(bf_hi(a.y), act1, fmaf(bf_lo(a.y), act0, acc[2 * q2][1]));
          acc[2 * q2 + 1][0] = fmaf(bf_hi(a.z), act1, fmaf(bf_lo(a.z), act0, acc[2 * q2 + 1][0]));
          acc[2 * q2 + 1][1] = fmaf(bf_hi(a.w), act1, fmaf(bf_lo(a.w), act0, acc[2 * q2 + 1][1]));
        }
      }
      __syncwarp();
      if (lane == 0 && !*abort_flag) mbar_arrive(smem_u32(&hdr->empty[s]));   // (no slot is released after a give-up)
    };

    const float gamma = p.layers[l].gamma;
    for (int u = s_lo; u < s_hi; ++u) unit(u < p.n_shared * p.shared_tiles ? 1.0f : gamma);
    asm volatile("bar.sync 4, 288;" ::: "memory");   // the router warp knows this layer's routed expert and its gate
    const float g1 = hdr->r_w;
    const bool have = hdr->r_have != 0;
    if (have)
      for (int u = r_lo; u < r_hi; ++u) unit(g1);
    // the layer's partial output row goes to the layer's delta row.  The four lanes of a row group first add
    // their contraction columns up (lane 4g then has rows g and g + 8 of each 16-row tile); four neighbouring
    // rows are gathered into one lane so that the additions go out as 16-byte vector reductions
    float* dl = p.delta + ((size_t)l * DX_STACK_COPIES + (cta % DX_STACK_COPIES)) * H;
    constexpr int NV = 4 * PW;   // (tile, half) values of this warp
#pragma unroll
    for (int v0 = 0; v0 < NV; v0 += 16) {
      float4 keep = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int vi = v0; vi < v0 + 16 && vi < NV; ++vi) {
        float val = acc[vi >> 1][vi & 1];
        val += __shfl_xor_sync(0xffffffffu, val, 1);
        val += __shfl_xor_sync(0xffffffffu, val, 2);
        const int from = 16 * (lane & 1);
        const float t0 = __shfl_sync(0xffffffffu, val, from), t1 = __shfl_sync(0xffffffffu, val, from + 4);
        const float t2 = __shfl_sync(0xffffffffu, val, from + 8), t3 = __shfl_sync(0xffffffffu, val, from + 12);
        if ((lane >> 1) == vi - v0) keep = make_float4(t0, t1, t2, t3);
      }
      const int vi = v0 + (lane >> 1);
      if (vi < NV) {
        float* dst = dl + (warp * 2 * PW + (vi >> 1)) * 16 + (vi & 1) * 8 + 4 * (lane & 1);
        asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                     :: "l"(dst), "f"(keep.x), "f"(keep.y), "f"(keep.z), "f"(keep.w) : "memory");
      }
    }
    consumer_bar();
    if (threadIdx.x == 0)   // release: the additions of all consumer threads (ordered by the barrier) come first
      asm volatile("red.release.gpu.global.add.u32 [%0], %1;" :: "l"(p.sync + l), "r"(1u) : "memory");
  }
  if (*abort_flag && threadIdx.x == 0) atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED);
}

template <int H, bool Q4>
cudaError_t launch_stack(dx_ctx* ctx, const DxStackParams& p, cudaStream_t st) {
  const size_t hdr = (sizeof(StackSmem) + 127) / 128 * 128;
  const size_t fixed = hdr + (size_t)kStackPartialBytes + (size_t)H * 4;
  const size_t chunk = dx_chunk_bytes(H, Q4);
  int n_slots = (int)(((size_t)ctx->smem_optin - fixed) / chunk);
  if (n_slots > kStackMaxSlots) n_slots = kStackMaxSlots;
  if (n_slots < kStackConsumers + 1) return cudaErrorInvalidConfiguration;
  const size_t smem = fixed + (size_t)n_slots * chunk;
  cudaError_t e = cudaFuncSetAttribute(dx_draft_stack_kernel<H, Q4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctx->sm_count);
  cfg.blockDim = dim3(kStackThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;   // the CTAs wait on one another: all of them must be resident
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, dx_draft_stack_kernel<H, Q4>, p, n_slots);
}

}  // namespace

cudaError_t dx_launch_draft_stack(dx_ctx* ctx, const DxStackParams& p, cudaStream_t st) {
  switch (p.H) {
    case 256: return p.q4 ? launch_stack<256, true>(ctx, p, st) : launch_stack<256, false>(ctx, p, st);
    case 512: return p.q4 ? launch_stack<512, true>(ctx, p, st) : launch_stack<512, false>(ctx, p, st);
    case 1024: return p.q4 ? launch_stack<1024, true>(ctx, p, st) : launch_stack<1024, false>(ctx, p, st);
    case 2048: return p.q4 ? launch_stack<2048, true>(ctx, p, st) : launch_stack<2048, false>(ctx, p, st);
    default: return cudaErrorInvalidConfiguration;
  }
}
