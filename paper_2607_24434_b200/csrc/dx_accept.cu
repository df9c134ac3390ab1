// Exact greedy verification (Algorithm 1, "verify" + "accept the
// target-consistent prefix"): target tokens t_i = argmax_v <W_lm[v], h_i> with
// the lowest v winning ties, accepted length n = longest prefix with
// t_i == d_i, next token = t_n.
//
// The LM head [V,H] is streamed from HBM exactly once for all M rows.  Two bf16
// kernels share the arithmetic described here; the ring variant further down
// (H = 1024 / 2048) brings the rows in through shared memory instead.  Register-
// direct kernel: each warp owns 16 vocabulary rows at a time and multiplies them with
// the M hidden rows on the tensor cores (mma.sync m16n8k16, vocabulary rows as
// the 16-row operand, hidden rows as the 8-column operand, hidden rows fed as
// bf16 high part + bf16 residual).  A lane loads 16 contiguous bytes of two
// rows per step straight from global memory; the contraction index is permuted
// consistently on both operands so those 16 bytes are exactly its fragment.
// Every lane tracks the running maximum of the logits it owns; maxima are
// merged as packed 64-bit keys (orderable logit << 32 | ~index) with
// atomicMax, and the CTA that takes the last ticket turns the keys into
// tokens, the accepted length and the next token.
#include <mutex>

#include "dx_internal.cuh"
#include "dx_stream.cuh"

namespace {

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}
__device__ __forceinline__ uint4 ldg_hint(const void* p, uint64_t pol) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.L2::256B.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p), "l"(pol));
  return r;
}
__device__ __forceinline__ void mma_k16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned long long make_key(float v, int idx) {
  return ((unsigned long long)dx_orderable(v) << 32) | (unsigned long long)(0xffffffffu - (unsigned)idx);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

struct AcceptParams {
  const float* h;
  int M, V, H;
  const void* W;
  const int32_t* draft;
  int K;
  int rms_norm;
  int32_t* target;
  int32_t* n_accept;
  int32_t* next_token;
  unsigned long long* keys;
  unsigned int* ticket;
  float* conf;          // [M] softmax probability of the argmax (only the CONF variants)
  float2* conf_part;    // [grid][DX_MAX_M] per-CTA (running max, sum of exp) pairs
  int keep_tiles;       // 16-row tiles at the head of the matrix that L2 is asked to retain from call to call
  int32_t* dev_status;  // the context's status word (null for the context-free entry point)
};

// online softmax bookkeeping: (m, s) with s = sum exp(l - m) over the logits seen so far
__device__ __forceinline__ void conf_push(float& m, float& s, float l) {
  if (l > m) { s = s * __expf(m - l) + 1.0f; m = l; }
  else s += __expf(l - m);
}
__device__ __forceinline__ void conf_merge(float& m, float& s, float m2, float s2) {
  if (s2 == 0.0f) return;
  if (s == 0.0f) { m = m2; s = s2; return; }
  const float mm = fmaxf(m, m2);
  s = s * __expf(m - mm) + s2 * __expf(m2 - mm);
  m = mm;
}

// Shared tail: merge CTA maxima into the global keys; the last CTA decodes.
template <bool CONF>
__device__ __forceinline__ void finish(const AcceptParams& p, unsigned long long* s_keys) {
  __shared__ int s_last;
  __syncthreads();
  if (threadIdx.x < p.M && s_keys[threadIdx.x] != 0ull) atomicMax(p.keys + threadIdx.x, s_keys[threadIdx.x]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(p.ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  __shared__ int s_tok[DX_MAX_M];
  if (threadIdx.x < p.M) {
    unsigned long long kk = __ldcg(p.keys + threadIdx.x);
    int tok = (int)(0xffffffffu - (unsigned)(kk & 0xffffffffull));
#ifdef DX_CHECKED
    if (p.dev_status && !(tok >= 0 && tok < p.V)) atomicExch(p.dev_status, (int32_t)DX_DEV_BOUNDS);
#endif
    s_tok[threadIdx.x] = tok;
    p.target[threadIdx.x] = tok;
    p.keys[threadIdx.x] = 0ull;
    if constexpr (CONF) {
      // max softmax probability = 1 / sum_v exp(l_v - l_max): merge every CTA's (max, sum) pair in CTA order
      float m = -INFINITY, sum = 0.0f;
      for (unsigned int cta = 0; cta < gridDim.x; ++cta) {
        const float2 part = __ldcg(p.conf_part + (size_t)cta * DX_MAX_M + threadIdx.x);
        conf_merge(m, sum, part.x, part.y);
      }
      p.conf[threadIdx.x] = 1.0f / sum;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = 0;
    while (n < p.K && n < p.M && p.draft[n] == s_tok[n]) ++n;
    *p.n_accept = n;
    *p.next_token = n < p.M ? s_tok[n] : -1;
    *p.ticket = 0u;
  }
}

template <int NT, bool CONF>
__global__ void __launch_bounds__(512, 1) dx_accept_bf16_kernel(AcceptParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ float s_rstd[DX_MAX_M];
  __shared__ unsigned long long s_keys[DX_MAX_M];
  const int H = p.H, Q = H / 32;
  uint4* hiF = reinterpret_cast<uint4*>(smem);        // [NT][Q][32]
  uint4* loF = hiF + (size_t)NT * Q * 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
  dx_pdl_wait();   // the hidden rows are usually the previous kernel's output
  dx_pdl_trigger();

  if (warp < DX_MAX_M) {
    float r = 1.0f;
    if (p.rms_norm && warp < p.M) {
      float ss = 0.f;
      for (int j = lane * 4; j < H; j += 128) {
        float4 v = *reinterpret_cast<const float4*>(p.h + (size_t)warp * H + j);
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      }
      r = rsqrtf(warp_sum(ss) / (float)H + 1e-6f);
    }
    if (lane == 0) { s_rstd[warp] = r; s_keys[warp] = 0ull; }
  }
  __syncthreads();
  // hidden-row fragments: lane (g,c) of column block q holds, for row nt*8+g,
  // columns 32q+8c..+7 split into bf16 high part and residual
  for (int idx = threadIdx.x; idx < NT * Q * 32; idx += blockDim.x) {
    const int l = idx & 31, q = (idx >> 5) % Q, nt = idx / (32 * Q);
    const int row = nt * 8 + (l >> 2);
    uint4 oh = make_uint4(0u, 0u, 0u, 0u), ol = oh;
    if (row < p.M) {
      const float* src = p.h + (size_t)row * H + 32 * q + 8 * (l & 3);
      const float4 v0 = *reinterpret_cast<const float4*>(src), v1 = *reinterpret_cast<const float4*>(src + 4);
      const float rs = s_rstd[row];
      const float x[8] = {v0.x * rs, v0.y * rs, v0.z * rs, v0.w * rs, v1.x * rs, v1.y * rs, v1.z * rs, v1.w * rs};
      __nv_bfloat16 hb[8], lb[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        hb[i] = __float2bfloat16_rn(x[i]);
        lb[i] = __float2bfloat16_rn(x[i] - __bfloat162float(hb[i]));
      }
      oh = make_uint4(pack2(hb[0], hb[1]), pack2(hb[2], hb[3]), pack2(hb[4], hb[5]), pack2(hb[6], hb[7]));
      ol = make_uint4(pack2(lb[0], lb[1]), pack2(lb[2], lb[3]), pack2(lb[4], lb[5]), pack2(lb[6], lb[7]));
    }
    hiF[idx] = oh;
    loF[idx] = ol;
  }
  __syncthreads();

  float best_v[NT][2];
  int best_i[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) { best_v[nt][0] = best_v[nt][1] = -INFINITY; best_i[nt][0] = best_i[nt][1] = -1; }
  float cm[NT][2], cs[NT][2];   // online softmax state of the two rows this lane owns per tile (CONF only)
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) { cm[nt][0] = cm[nt][1] = -INFINITY; cs[nt][0] = cs[nt][1] = 0.0f; }

  const int tiles = (p.V + 15) / 16;
  // Tiles are dealt to the CTAs first (tile t belongs to CTA t mod gridDim.x) and to the warps inside a CTA second,
  // so every CTA streams the same number of tiles to within one; dealing them warp by warp across the grid would
  // give the first CTAs one whole tile per warp more than the last ones.
  const int tiles_cta = gridDim.x;
  const __nv_bfloat16* Wb = reinterpret_cast<const __nv_bfloat16*>(p.W);
  // The LM head is the same matrix in every decode step and larger than L2, so a plain stream leaves nothing of it
  // behind.  The first keep_tiles tiles are read with an evict-last hint, everything else with evict-first: the
  // head of the matrix stays in L2 between two calls (expert weights are streamed evict-first as well) and only the
  // rest comes from HBM again.
  uint64_t pol_keep, pol_stream;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
  for (int tile = blockIdx.x + tiles_cta * warp; tile < tiles; tile += tiles_cta * (int)(blockDim.x >> 5)) {
    const uint64_t pol = tile < p.keep_tiles ? pol_keep : pol_stream;
    const int r0 = tile * 16 + g, r1 = r0 + 8;
    const __nv_bfloat16* w0 = Wb + (size_t)min(r0, p.V - 1) * H + 8 * c;
    const __nv_bfloat16* w1 = Wb + (size_t)min(r1, p.V - 1) * H + 8 * c;
    float ch[NT][4], cl[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int r = 0; r < 4; ++r) ch[nt][r] = cl[nt][r] = 0.f;
#pragma unroll 16
    for (int q = 0; q < Q; ++q) {
      const uint4 a0 = p.keep_tiles ? ldg_hint(w0 + 32 * q, pol) : ldg_stream(w0 + 32 * q);
      const uint4 a1 = p.keep_tiles ? ldg_hint(w1 + 32 * q, pol) : ldg_stream(w1 + 32 * q);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const uint4 bh = hiF[(nt * Q + q) * 32 + lane];
        const uint4 bl = loF[(nt * Q + q) * 32 + lane];
        mma_k16(ch[nt], a0.x, a1.x, a0.y, a1.y, bh.x, bh.y);
        mma_k16(cl[nt], a0.x, a1.x, a0.y, a1.y, bl.x, bl.y);
        mma_k16(ch[nt], a0.z, a1.z, a0.w, a1.w, bh.z, bh.w);
        mma_k16(cl[nt], a0.z, a1.z, a0.w, a1.w, bl.z, bl.w);
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float l00 = ch[nt][0] + cl[nt][0], l01 = ch[nt][1] + cl[nt][1];
      const float l10 = ch[nt][2] + cl[nt][2], l11 = ch[nt][3] + cl[nt][3];
      if (r0 < p.V) {
        if (l00 > best_v[nt][0]) { best_v[nt][0] = l00; best_i[nt][0] = r0; }
        if (l01 > best_v[nt][1]) { best_v[nt][1] = l01; best_i[nt][1] = r0; }
        if constexpr (CONF) { conf_push(cm[nt][0], cs[nt][0], l00); conf_push(cm[nt][1], cs[nt][1], l01); }
      }
      if (r1 < p.V) {
        if (l10 > best_v[nt][0]) { best_v[nt][0] = l10; best_i[nt][0] = r1; }
        if (l11 > best_v[nt][1]) { best_v[nt][1] = l11; best_i[nt][1] = r1; }
        if constexpr (CONF) { conf_push(cm[nt][0], cs[nt][0], l10); conf_push(cm[nt][1], cs[nt][1], l11); }
      }
    }
  }
  if constexpr (CONF) {
    __shared__ float2 s_conf[16][DX_MAX_M];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float m = cm[nt][j], sum = cs[nt][j];
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, sum, o);
          conf_merge(m, sum, m2, s2);
        }
        const int row = nt * 8 + 2 * c + j;
        if (g == 0 && row < DX_MAX_M) s_conf[warp][row] = make_float2(m, sum);
      }
    __syncthreads();
    if (threadIdx.x < p.M) {
      float m = -INFINITY, sum = 0.0f;
      for (int w = 0; w < 16; ++w) conf_merge(m, sum, s_conf[w][threadIdx.x].x, s_conf[w][threadIdx.x].y);
      p.conf_part[(size_t)blockIdx.x * DX_MAX_M + threadIdx.x] = make_float2(m, sum);
    }
  }
  // lanes with equal c hold the same token columns: merge over g
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      unsigned long long key = best_i[nt][j] >= 0 ? make_key(best_v[nt][j], best_i[nt][j]) : 0ull;
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
      }
      const int row = nt * 8 + 2 * c + j;
      if (g == 0 && row < p.M && key != 0ull) atomicMax(&s_keys[row], key);
    }
  finish<CONF>(p, s_keys);
}

// ---------------------------------------------------------------------------------------------------------
// Ring variant (H = 1024 / 2048; one or two tiles of eight block rows).  Same arithmetic as the
// kernel above; what differs is how the LM head reaches the tensor cores.  A producer thread streams whole
// vocabulary rows (one bulk asynchronous copy each) into a ring of three 16-row tiles in shared memory; the eight
// consumer warps split the contraction (warp w owns hidden columns [w H/8, (w+1) H/8), its hidden-row fragments
// live in registers), add their partial logits up through shared memory once per tile, and 128 threads per token
// tile keep the running maxima.  The LM head does not depend on the kernel in front, so when the launch is a programmatic one
// the producer fills the ring while that kernel's last CTAs are still working, and the consumers wait for the
// hidden rows only where they read them.  Loads that go to shared memory are also indifferent to how much of the
// SM's memory is left for L1 -- the register-direct kernel loses a third of its rate on an SM that an expert CTA
// has just left configured for 227 KB of shared memory.
constexpr int kRingConsumers = 8;
constexpr int kRingThreads = (kRingConsumers + 1) * 32;
constexpr int kRingSlots = 3;

struct RingHeader {
  unsigned long long full[kRingSlots];
  unsigned long long empty[kRingSlots];
  unsigned long long keys[DX_MAX_M];
  float ssq[kRingConsumers][DX_MAX_M];
  int abort_flag;
};
constexpr size_t kRingHdr = (sizeof(RingHeader) + 127) / 128 * 128;
constexpr size_t kRingPartial = (size_t)2 * kRingConsumers * 32 * 16;   // [2][warp][lane] float4, per token tile
// a row of the tile is padded by 64 bytes: the eight rows a quarter-warp reads side by side fall into distinct banks
template <int H> __host__ __device__ constexpr uint32_t ring_row_stride() { return (uint32_t)H * 2u + 64u; }
template <int H, int NT> constexpr size_t ring_smem_bytes() { return kRingHdr + (size_t)NT * kRingPartial + (size_t)kRingSlots * 16 * ring_row_stride<H>(); }

template <int H, int NT, bool CONF>
__global__ void __launch_bounds__(kRingThreads, 1) dx_accept_ring_kernel(AcceptParams p, uint32_t wait_limit) {
  constexpr int QW = H / 256;                    // 32-column steps of the contraction per consumer warp
  constexpr uint32_t ROW = (uint32_t)H * 2u, STRIDE = ring_row_stride<H>(), TILE = 16u * STRIDE;
  extern __shared__ __align__(128) unsigned char smem[];
  RingHeader* hdr = reinterpret_cast<RingHeader*>(smem);
  float4* partial = reinterpret_cast<float4*>(smem + kRingHdr);            // [2][warp][NT][lane]
  unsigned char* ring = smem + kRingHdr + (size_t)NT * kRingPartial;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
  const int tiles = (p.V + 15) / 16;
  volatile int* abort_flag = &hdr->abort_flag;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kRingSlots; ++s) {
      mbar_init(smem_u32(&hdr->full[s]), 1);
      mbar_init(smem_u32(&hdr->empty[s]), kRingConsumers);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < DX_MAX_M) hdr->keys[threadIdx.x] = 0ull;
  __syncthreads();
  dx_pdl_trigger();

  if (warp == kRingConsumers) {
    // ------------------------------------------------------------ producer: tile t of this CTA is tile blockIdx.x + t gridDim.x
    if (lane == 0) {
      // (tiles at the head of the matrix may be marked for retention in L2, see dx_set_accept_l2_keep)
      const uint64_t pol_stream = l2_evict_first_policy();
      uint64_t pol_keep;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
      const unsigned char* Wb = reinterpret_cast<const unsigned char*>(p.W);
      uint32_t issued = 0, slot = 0, phase = 0;
      for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++issued) {
        if (!mbar_wait(smem_u32(&hdr->empty[slot]), phase ^ 1u, abort_flag, wait_limit)) break;
        const int rows = min(16, p.V - tile * 16);
        if (!DX_BOUNDS(slot < (uint32_t)kRingSlots && rows >= 1 && (long long)tile * 16 + rows <= (long long)p.V, p.dev_status)) {
          *abort_flag = 1;
          break;
        }
        const uint32_t fb = smem_u32(&hdr->full[slot]);
        const uint64_t pol = tile < p.keep_tiles ? pol_keep : pol_stream;
        mbar_arrive_expect_tx(fb, (uint32_t)rows * ROW);
        for (int r = 0; r < rows; ++r)
          bulk_g2s(smem_u32(ring + (size_t)slot * TILE + (size_t)r * STRIDE), Wb + ((size_t)tile * 16 + r) * ROW, ROW, fb, pol);
        if (++slot == (uint32_t)kRingSlots) { slot = 0; phase ^= 1u; }
      }
      if (*abort_flag) {
        // something gave up: no copy may still be landing in this CTA's shared memory when it is released
        const uint32_t n_back = issued < (uint32_t)kRingSlots ? issued : (uint32_t)kRingSlots;
        for (uint32_t k = 1; k <= n_back; ++k) {
          const uint32_t j = issued - k, s = j % (uint32_t)kRingSlots, ph = (j / (uint32_t)kRingSlots) & 1u;
          for (uint32_t spin = 0; spin < DX_WAIT_LIMIT_DEFAULT; ++spin)
            if (mbar_try_wait(smem_u32(&hdr->full[s]), ph)) break;
        }
        if (p.dev_status) atomicExch(p.dev_status, (int32_t)DX_DEV_WAIT_EXPIRED);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ consumers
    dx_pdl_wait();   // the hidden rows are usually the previous kernel's output
    // this lane's fragments of hidden rows g (and 8 + g) over the warp's columns: values of columns 32 q + 8 c .. + 7,
    // as bf16 high part and residual (the contraction index is permuted the same way on both operands, see the
    // kernel above)
    uint4 bh[NT][QW], bl[NT][QW];
    if (p.rms_norm) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float ss = 0.f;
        if (nt * 8 + g < p.M) {
#pragma unroll
          for (int q = 0; q < QW; ++q) {
            const float* src = p.h + (size_t)(nt * 8 + g) * H + 32 * (warp * QW + q) + 8 * c;
            const float4 v0 = *reinterpret_cast<const float4*>(src), v1 = *reinterpret_cast<const float4*>(src + 4);
            ss += v0.x * v0.x + v0.y * v0.y + v0.z * v0.z + v0.w * v0.w + v1.x * v1.x + v1.y * v1.y + v1.z * v1.z + v1.w * v1.w;
          }
        }
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        ss += __shfl_xor_sync(0xffffffffu, ss, 2);
        if (c == 0) hdr->ssq[warp][nt * 8 + g] = ss;
      }
      consumer_bar();
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float rs = 1.0f;
      if (p.rms_norm) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kRingConsumers; ++w) tot += hdr->ssq[w][nt * 8 + g];
        rs = rsqrtf(tot / (float)H + 1e-6f);
      }
      const bool valid = nt * 8 + g < p.M;
#pragma unroll
      for (int q = 0; q < QW; ++q) {
        float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f), v1 = v0;
        if (valid) {
          const float* src = p.h + (size_t)(nt * 8 + g) * H + 32 * (warp * QW + q) + 8 * c;
          v0 = *reinterpret_cast<const float4*>(src);
          v1 = *reinterpret_cast<const float4*>(src + 4);
        }
        const float x[8] = {v0.x * rs, v0.y * rs, v0.z * rs, v0.w * rs, v1.x * rs, v1.y * rs, v1.z * rs, v1.w * rs};
        __nv_bfloat16 hb[8], lb[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) split_bf16(x[i], hb[i], lb[i]);
        bh[nt][q] = make_uint4(pack2(hb[0], hb[1]), pack2(hb[2], hb[3]), pack2(hb[4], hb[5]), pack2(hb[6], hb[7]));
        bl[nt][q] = make_uint4(pack2(lb[0], lb[1]), pack2(lb[2], lb[3]), pack2(lb[4], lb[5]), pack2(lb[6], lb[7]));
      }
    }
    // threads 0 .. 128 NT - 1 each own one (row within the tile, block row) pair of the summed logits: element e of
    // token tile nt's C fragments, e = 4 lane + r: tile row (lane >> 2) + 8 (r >> 1), block row 8 nt + 2 (lane & 3) + (r & 1)
    const int e_el = threadIdx.x & 127, e_nt = threadIdx.x >> 7;
    const int e_row = (e_el >> 4) + ((e_el & 2) ? 8 : 0), e_tok = 8 * e_nt + 2 * ((e_el >> 2) & 3) + (e_el & 1);
    const bool owner = threadIdx.x < 128 * NT;
    float best_v = -INFINITY;
    int best_i = -1;
    float cm = -INFINITY, cs = 0.0f;   // online softmax state of this thread's share of its block row (CONF only)
    uint32_t slot = 0, phase = 0;
    int buf = 0;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
      // (a slot out of range is reported and replaced: every warp has to keep taking part in the barriers below)
      if (!DX_BOUNDS(slot < (uint32_t)kRingSlots, p.dev_status)) { *abort_flag = 1; slot = 0; }
      mbar_wait(smem_u32(&hdr->full[slot]), phase, abort_flag, wait_limit);
      const unsigned char* T = ring + (size_t)slot * TILE + (size_t)g * STRIDE + (size_t)(warp * QW) * 64 + c * 16;
      float ch[NT][4], cl[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) ch[nt][r] = cl[nt][r] = 0.f;
#pragma unroll
      for (int q = 0; q < QW; ++q) {
        const uint4 a0 = *reinterpret_cast<const uint4*>(T + q * 64);
        const uint4 a1 = *reinterpret_cast<const uint4*>(T + 8 * STRIDE + q * 64);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          mma_k16(ch[nt], a0.x, a1.x, a0.y, a1.y, bh[nt][q].x, bh[nt][q].y);
          mma_k16(cl[nt], a0.x, a1.x, a0.y, a1.y, bl[nt][q].x, bl[nt][q].y);
          mma_k16(ch[nt], a0.z, a1.z, a0.w, a1.w, bh[nt][q].z, bh[nt][q].w);
          mma_k16(cl[nt], a0.z, a1.z, a0.w, a1.w, bl[nt][q].z, bl[nt][q].w);
        }
      }
      __syncwarp();
      if (lane == 0 && !*abort_flag) mbar_arrive(smem_u32(&hdr->empty[slot]));   // (no slot is released after a give-up)
      if (++slot == (uint32_t)kRingSlots) { slot = 0; phase ^= 1u; }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
        partial[((buf * kRingConsumers + warp) * NT + nt) * 32 + lane] =
            make_float4(ch[nt][0] + cl[nt][0], ch[nt][1] + cl[nt][1], ch[nt][2] + cl[nt][2], ch[nt][3] + cl[nt][3]);
      consumer_bar();
      if (owner) {
        const float* ps = reinterpret_cast<const float*>(partial) + ((size_t)buf * kRingConsumers * NT + e_nt) * 128 + e_el;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < kRingConsumers; ++w) v += ps[w * NT * 128];
        const int row = tile * 16 + e_row;
        if (row < p.V) {
          if (v > best_v) { best_v = v; best_i = row; }
          if constexpr (CONF) conf_push(cm, cs, v);
        }
      }
      buf ^= 1;
    }
    if (owner && e_tok < p.M && best_i >= 0 && DX_BOUNDS(e_tok < DX_MAX_M && best_i < p.V, p.dev_status))
      atomicMax(&hdr->keys[e_tok], make_key(best_v, best_i));
    if constexpr (CONF) {
      // sixteen threads share a block row: their (max, sum) pairs meet in the (now idle) partial buffer
      float2* sc = reinterpret_cast<float2*>(partial);
      consumer_bar();
      if (owner) sc[threadIdx.x] = make_float2(cm, cs);
      consumer_bar();
      if (threadIdx.x < p.M && threadIdx.x < 8 * NT) {
        float m = -INFINITY, sum = 0.0f;
        for (int e = 0; e < 128 * NT; ++e)
          if (8 * (e >> 7) + 2 * (((e & 127) >> 2) & 3) + (e & 1) == (int)threadIdx.x) conf_merge(m, sum, sc[e].x, sc[e].y);
        p.conf_part[(size_t)blockIdx.x * DX_MAX_M + threadIdx.x] = make_float2(m, sum);
      }
    }
  }
  finish<CONF>(p, hdr->keys);
}

// fp32 LM head (small vocabularies): one warp per vocabulary row.
template <bool CONF>
__global__ void __launch_bounds__(256) dx_accept_fp32_kernel(AcceptParams p) {
  __shared__ float s_rstd[DX_MAX_M];
  __shared__ unsigned long long s_keys[DX_MAX_M];
  const int H = p.H, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  dx_pdl_wait();
  dx_pdl_trigger();
  for (int row = warp; row < DX_MAX_M; row += 8) {
    float r = 1.0f;
    if (p.rms_norm && row < p.M) {
      float ss = 0.f;
      for (int j = lane; j < H; j += 32) { float v = p.h[(size_t)row * H + j]; ss += v * v; }
      r = rsqrtf(warp_sum(ss) / (float)H + 1e-6f);
    }
    if (lane == 0) { s_rstd[row] = r; s_keys[row] = 0ull; }
  }
  __syncthreads();
  const float* Wf = reinterpret_cast<const float*>(p.W);
  const int warps_total = gridDim.x * 8;
  unsigned long long best[DX_MAX_M];
  float cm[CONF ? DX_MAX_M : 1], cs[CONF ? DX_MAX_M : 1];
#pragma unroll
  for (int i = 0; i < DX_MAX_M; ++i) best[i] = 0ull;
  if constexpr (CONF) {
#pragma unroll
    for (int i = 0; i < DX_MAX_M; ++i) { cm[i] = -INFINITY; cs[i] = 0.0f; }
  }
  for (int v = blockIdx.x * 8 + warp; v < p.V; v += warps_total) {
    const float* wr = Wf + (size_t)v * H;
#pragma unroll
    for (int i = 0; i < DX_MAX_M; ++i) {
      if (i < p.M) {
        float acc = 0.f;
        for (int j = lane; j < H; j += 32) acc = fmaf(wr[j], p.h[(size_t)i * H + j] * s_rstd[i], acc);
        acc = warp_sum(acc);
        unsigned long long key = make_key(acc, v);
        best[i] = key > best[i] ? key : best[i];
        if constexpr (CONF) conf_push(cm[i], cs[i], acc);
      }
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < DX_MAX_M; ++i)
      if (i < p.M && best[i] != 0ull) atomicMax(&s_keys[i], best[i]);
  }
  if constexpr (CONF) {
    __shared__ float2 s_conf[8][DX_MAX_M];
    if (lane == 0) {
#pragma unroll
      for (int i = 0; i < DX_MAX_M; ++i) s_conf[warp][i] = make_float2(cm[i], cs[i]);
    }
    __syncthreads();
    if (threadIdx.x < p.M) {
      float m = -INFINITY, sum = 0.0f;
      for (int w = 0; w < 8; ++w) conf_merge(m, sum, s_conf[w][threadIdx.x].x, s_conf[w][threadIdx.x].y);
      p.conf_part[(size_t)blockIdx.x * DX_MAX_M + threadIdx.x] = make_float2(m, sum);
    }
  }
  finish<CONF>(p, s_keys);
}

}  // namespace

template <int NT, bool CONF>
static cudaError_t launch_accept_bf16(dx_ctx* ctx, const AcceptParams& p, size_t smem, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(dx_accept_bf16_kernel<NT, CONF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  return dx_launch_pdl((ctx->pdl_mask & DX_PDL_ACCEPT) != 0, dx_accept_bf16_kernel<NT, CONF>, dim3(ctx->sm_count), dim3(512), smem, st, 1, p);
}

template <int H, int NT, bool CONF>
static cudaError_t launch_accept_ring(dx_ctx* ctx, const AcceptParams& p, cudaStream_t st) {
  const size_t smem = ring_smem_bytes<H, NT>();
  cudaError_t e = cudaFuncSetAttribute(dx_accept_ring_kernel<H, NT, CONF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return dx_launch_pdl((ctx->pdl_mask & DX_PDL_ACCEPT) != 0, dx_accept_ring_kernel<H, NT, CONF>, dim3(ctx->sm_count), dim3(kRingThreads), smem,
                       st, 1, p, ctx->wait_limit);
}
template <int H>
static cudaError_t launch_accept_ring_h(dx_ctx* ctx, const AcceptParams& p, int NT, bool conf, cudaStream_t st) {
  if (NT == 1) return conf ? launch_accept_ring<H, 1, true>(ctx, p, st) : launch_accept_ring<H, 1, false>(ctx, p, st);
  return conf ? launch_accept_ring<H, 2, true>(ctx, p, st) : launch_accept_ring<H, 2, false>(ctx, p, st);
}

cudaError_t dx_launch_accept(dx_ctx* ctx, const float* h, int M, const void* W_lm, int V, int H, int w_dtype,
                             const int32_t* draft, int K, int rms_norm, int32_t* target, int32_t* n_accept,
                             int32_t* next_token, float* conf, cudaStream_t st) {
  AcceptParams p{h, M, V, H, W_lm, draft, K, rms_norm, target, n_accept, next_token, ctx->keys, ctx->ticket + 1,
                 conf, ctx->conf_part, 0, ctx->dev_status};
  if (w_dtype != DX_DTYPE_FP32) p.keep_tiles = (int)(ctx->accept_keep_bytes / ((size_t)16 * H * 2));
  if (w_dtype == DX_DTYPE_FP32) {
    int grid = (V + 7) / 8;
    if (grid > ctx->sm_count * 8) grid = ctx->sm_count * 8;
    if (conf) return dx_launch_pdl((ctx->pdl_mask & DX_PDL_ACCEPT) != 0, dx_accept_fp32_kernel<true>, dim3(grid), dim3(256), 0, st, 1, p);
    return dx_launch_pdl((ctx->pdl_mask & DX_PDL_ACCEPT) != 0, dx_accept_fp32_kernel<false>, dim3(grid), dim3(256), 0, st, 1, p);
  }
  const int NT = (M + 7) / 8;
  // the two large hidden sizes: the shared-memory ring variant
  if (H == 2048 && ring_smem_bytes<2048, 2>() <= (size_t)ctx->smem_optin) return launch_accept_ring_h<2048>(ctx, p, NT, conf != nullptr, st);
  if (H == 1024 && ring_smem_bytes<1024, 2>() <= (size_t)ctx->smem_optin) return launch_accept_ring_h<1024>(ctx, p, NT, conf != nullptr, st);
  const size_t smem = (size_t)NT * (H / 32) * 32 * 16 * 2;
  if (NT == 1) return conf ? launch_accept_bf16<1, true>(ctx, p, smem, st) : launch_accept_bf16<1, false>(ctx, p, smem, st);
  return conf ? launch_accept_bf16<2, true>(ctx, p, smem, st) : launch_accept_bf16<2, false>(ctx, p, smem, st);
}

// ---------------------------------------------------------------------------------------------------------
// spec_accept_noalloc: greedy verification for callers that must not allocate.
//
// Some callers cannot call cudaMalloc (or anything that does): a thread inside a serving loop whose memory
// pool was sized once at start-up (a late cudaMalloc is forbidden there, or would stall every stream), a
// plugin that is handed streams and buffers but no allocator.  For them this entry point needs no context handle: the scratch the
// kernels use (the packed 64-bit argmax key of every row and the "last CTA" ticket) lives in the file-scope
// device array below, which every GPU that loads the library holds until the process exits.
//
// The array's name is only a host-side stand-in in host code, not a device address, so the address is looked
// up once per device with cudaGetSymbolAddress and that pointer is what the kernels get.
constexpr int kNoAllocMaxRows = DX_MAX_M;                       // rows (M) the static scratch is sized for
static __device__ __align__(256) unsigned long long g_noalloc_scratch[kNoAllocMaxRows + 2];   // keys, then ticket

namespace {
struct NoAllocDevice {
  std::once_flag once;     // the set-up below runs once per device, whichever host thread gets there first
  bool ok = false;
  unsigned long long* scratch = nullptr;
  int sm_count = 0;
  int smem_optin = 0;
};
NoAllocDevice g_noalloc_dev[64];
}  // namespace

extern "C" dx_status spec_accept_noalloc(const float* h, int32_t M, const void* W_lm, int32_t V, int32_t H,
                                         int32_t w_dtype, const int32_t* draft, int32_t K, int32_t rms_norm,
                                         int32_t* target, int32_t* n_accept, int32_t* next_token, void* stream) {
  if (!h || !W_lm || !target || !n_accept || !next_token) return DX_ERR_INVALID_ARG;
  if (K > 0 && !draft) return DX_ERR_INVALID_ARG;
  if (M < 1 || V < 1 || K < 0) return DX_ERR_SHAPE;
  if (w_dtype != DX_DTYPE_FP32 && w_dtype != DX_DTYPE_BF16) return DX_ERR_INVALID_ARG;
  // sizes beyond what the static scratch (and the kernels) are built for are refused, never truncated
  if (M > kNoAllocMaxRows || K > DX_MAX_K || H <= 0 || H > DX_MAX_H || H % 256) return DX_ERR_UNSUPPORTED;
  if (((uintptr_t)h) % 16 || ((uintptr_t)W_lm) % 16) return DX_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DX_ERR_CUDA;
  NoAllocDevice& d = g_noalloc_dev[dev];
  // first call on this device (with this device current): resolve the device address of the scratch array.  Host
  // threads that arrive together are serialised here; the others see a fully initialised record.
  std::call_once(d.once, [&d, dev] {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
    if (cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return;
    d.scratch = static_cast<unsigned long long*>(ptr);
    d.ok = true;
  });
  if (!d.ok) return DX_ERR_CUDA;
  const int NT = (M + 7) / 8;
  const size_t smem = (size_t)NT * (H / 32) * 32 * 16 * 2;
  if (w_dtype == DX_DTYPE_BF16 && smem > (size_t)d.smem_optin) return DX_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps whatever the last call left; keys and ticket must start at zero
  if (cudaMemsetAsync(d.scratch, 0, sizeof(unsigned long long) * (kNoAllocMaxRows + 2), st) != cudaSuccess)
    return DX_ERR_CUDA;
  AcceptParams p{h, M, V, H, W_lm, draft, K, rms_norm, target, n_accept, next_token, d.scratch,
                 reinterpret_cast<unsigned int*>(d.scratch + kNoAllocMaxRows), nullptr, nullptr, 0, nullptr};
  cudaError_t e;
  if (w_dtype == DX_DTYPE_FP32) {
    int grid = (V + 7) / 8;
    if (grid > d.sm_count * 8) grid = d.sm_count * 8;
    dx_accept_fp32_kernel<false><<<grid, 256, 0, st>>>(p);
    e = cudaGetLastError();
  } else if (NT == 1) {
    e = cudaFuncSetAttribute(dx_accept_bf16_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) {
      dx_accept_bf16_kernel<1, false><<<d.sm_count, 512, smem, st>>>(p);
      e = cudaGetLastError();
    }
  } else {
    e = cudaFuncSetAttribute(dx_accept_bf16_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) {
      dx_accept_bf16_kernel<2, false><<<d.sm_count, 512, smem, st>>>(p);
      e = cudaGetLastError();
    }
  }
  return e == cudaSuccess ? DX_OK : DX_ERR_CUDA;
}
