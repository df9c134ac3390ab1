// Grouped SwiGLU over the work list built by the routing kernel: for every
// group (an expert plus the block tokens routed to it)
//     y[tok] += w[tok] * W_d ( silu(W_g x[tok]) * (W_u x[tok]) )            (the summands of Eq. 4 / Eq. 5)
// with each expert's weights streamed from HBM exactly once per block.
//
// Work decomposition.  An expert is cut into I/8 "units": 8 rows of W_g, the
// same 8 rows of W_u and the matching 8 columns of W_d.  A unit is
// self-contained (its 8 activations feed only its own 8 columns of W_d), so the
// down projection is fused in and nothing intermediate ever reaches HBM.  The
// global unit list is split into equal contiguous ranges, one per CTA, so a CTA
// touches at most a few experts and keeps its partial y in registers until the
// expert changes; partials are then added to y with fp32 reductions.
//
// bf16 path (sm_100a): one elected producer thread streams each unit through a
// shared-memory ring with bulk asynchronous copies (cp.async.bulk, completion on
// mbarriers); eight consumer warps read the tiles with conflict-free 128-bit
// shared loads and multiply on the tensor cores (mma.sync m16n8k16 / m16n8k8,
// weights as the 16-row operand, tokens as the 8-column operand, fp32
// accumulate).  Activations are fed as a bf16 high part plus a bf16 residual so
// the products carry ~16 mantissa bits.  The packed blob stores every tile in
// the exact per-lane fragment order, which is why no ldmatrix or swizzle is
// needed.  All waits are bounded; an expired wait sets the device status word.
#include "dx_internal.cuh"

namespace {

// ------------------------------------------------------------------ helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(bar),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when it gave up; callers raise the abort flag,
// after which every wait of the CTA falls through so the CTA still terminates.
#define DX_WAIT_LIMIT (1u << 22)
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < DX_WAIT_LIMIT; ++it) {
    if (mbar_try_wait(bar, parity)) return;
    if ((it & 63u) == 63u && *abort_flag) return;
  }
  *abort_flag = 1;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ void mma_k16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_k8(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(b0));
}
// x = hi + lo with hi, lo bf16 (lo is the rounding residual of hi)
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}
__device__ __forceinline__ uint32_t pack2(__nv_bfloat16 lo16, __nv_bfloat16 hi16) {
  return (uint32_t)__bfloat16_as_ushort(lo16) | ((uint32_t)__bfloat16_as_ushort(hi16) << 16);
}

__device__ __forceinline__ int find_entry(const DxWork* W, int n_entries, int u, int start) {
  int ei = start;
  while (ei + 1 < n_entries && u >= W->entries[ei + 1].unit_begin) ++ei;
  // entries with zero tiles share unit_begin with their successor; skip them
  while (ei + 1 < n_entries && W->entries[ei].n_tiles == 0) ++ei;
  return ei;
}

// ----------------------------------------------------- bf16 tensor-core path
constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;

struct SmemHeader {
  unsigned long long full[8];
  unsigned long long empty[8];
  int abort_flag;
  int pad[31];
};

template <int H, int NT>
__global__ void __launch_bounds__(kThreads, 1) dx_experts_bf16_kernel(DxExpertParams p, int n_stages) {
  constexpr int KW = H / 128;        // phase-1 k-steps per consumer warp
  constexpr int PW = H / 256;        // phase-2 row-tile pairs per consumer warp
  constexpr int KSTEPS = H / 16;
  constexpr uint32_t STAGE_BYTES = 16u * H;   // a third of a unit
  constexpr uint32_t UNIT_BYTES = 48u * H;

  extern __shared__ __align__(128) unsigned char smem[];
  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  float4* partial = reinterpret_cast<float4*>(smem + sizeof(SmemHeader));                // [2][8][NT][32]
  uint4* bfrag = reinterpret_cast<uint4*>(smem + sizeof(SmemHeader) + 2 * 8 * NT * 32 * 16);  // [NT][KSTEPS][32]
  unsigned char* ring = reinterpret_cast<unsigned char*>(bfrag) + (size_t)NT * KSTEPS * 32 * 16;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const DxWork* W = p.work;
  const int n_entries = W->n_entries;
  const long long total = W->total_units;
  const int u_lo = (int)((total * blockIdx.x) / gridDim.x);
  const int u_hi = (int)((total * (blockIdx.x + 1)) / gridDim.x);
  volatile int* abort_flag = &hdr->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(smem_u32(&hdr->full[s]), 1);
      mbar_init(smem_u32(&hdr->empty[s]), kConsumerWarps);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (u_lo >= u_hi) return;

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      int ei = 0;
      uint32_t it = 0;
      for (int u = u_lo; u < u_hi; ++u) {
        ei = find_entry(W, n_entries, u, ei);
        const DxEntry& en = W->entries[ei];
        const unsigned char* blob = reinterpret_cast<const unsigned char*>(p.table[en.table_index]);
        if (blob == nullptr) continue;
        const unsigned char* src = blob + (size_t)(u - en.unit_begin) * UNIT_BYTES;
#pragma unroll 1
        for (int part = 0; part < 3; ++part, ++it) {
          const uint32_t s = it % (uint32_t)n_stages, ph = (it / (uint32_t)n_stages) & 1u;
          mbar_wait(smem_u32(&hdr->empty[s]), ph ^ 1u, abort_flag);
          const uint32_t fb = smem_u32(&hdr->full[s]);
          mbar_arrive_expect_tx(fb, STAGE_BYTES);
          bulk_g2s(smem_u32(ring + (size_t)s * STAGE_BYTES), src + (size_t)part * STAGE_BYTES, STAGE_BYTES, fb);
        }
      }
      if (*abort_flag) {
        // something gave up: make sure no copy is still landing in this CTA's
        // shared memory before it is released (bounded, ignores the flag)
        const uint32_t n_back = it < (uint32_t)n_stages ? it : (uint32_t)n_stages;
        for (uint32_t b = 1; b <= n_back; ++b) {
          const uint32_t j = it - b, s = j % (uint32_t)n_stages, ph = (j / (uint32_t)n_stages) & 1u;
          for (uint32_t spin = 0; spin < DX_WAIT_LIMIT; ++spin)
            if (mbar_try_wait(smem_u32(&hdr->full[s]), ph)) break;
        }
        atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED);
      }
    }
    return;
  }

  // --------------------------------------------------------------- consumers
  const int g = lane >> 2, c = lane & 3;
  float acc[NT][2 * PW][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int j = 0; j < 2 * PW; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[nt][j][r] = 0.f;

  int ei = -1, cur_m = 0;
  uint32_t it = 0;
  int buf = 0;

  auto flush = [&](int e_idx) {
    const DxEntry& en = W->entries[e_idx];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int s0 = nt * 8 + 2 * c, s1 = s0 + 1;
      const bool v0 = s0 < en.m, v1 = s1 < en.m;
      if (!v0) continue;
      const float w0 = en.w[s0], w1 = v1 ? en.w[s1] : 0.f;
      float* y0 = p.y + (size_t)en.tok[s0] * H;
      float* y1 = v1 ? p.y + (size_t)en.tok[s1] * H : nullptr;
#pragma unroll
      for (int j = 0; j < 2 * PW; ++j) {
        const int hh = (warp * 2 * PW + j) * 16 + g;
        atomicAdd(y0 + hh, w0 * acc[nt][j][0]);
        atomicAdd(y0 + hh + 8, w0 * acc[nt][j][2]);
        if (v1) {
          atomicAdd(y1 + hh, w1 * acc[nt][j][1]);
          atomicAdd(y1 + hh + 8, w1 * acc[nt][j][3]);
        }
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int j = 0; j < 2 * PW; ++j)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[nt][j][r] = 0.f;
  };

  for (int u = u_lo; u < u_hi; ++u) {
    const int ne = find_entry(W, n_entries, u, ei < 0 ? 0 : ei);
    if (ne != ei) {
      if (ei >= 0 && cur_m > 0) flush(ei);
      ei = ne;
      const DxEntry& en = W->entries[ei];
      const bool present = p.table[en.table_index] != nullptr;
      if (!present && threadIdx.x == 0) atomicExch(p.dev_status, DX_DEV_BAD_EXPERT_ID);
      cur_m = present ? en.m : 0;
      if (cur_m > 0) {
        // token fragments of this group: lane (g,c) of k-step ks holds, for
        // token slot nt*8+g, columns 16ks+4c..+3 as {hi01, hi23, lo01, lo23}
        for (int idx = threadIdx.x; idx < NT * KSTEPS * 32; idx += kConsumerWarps * 32) {
          const int l = idx & 31, ks = (idx >> 5) % KSTEPS, nt = idx / (32 * KSTEPS);
          const int slot = nt * 8 + (l >> 2);
          uint4 o = make_uint4(0u, 0u, 0u, 0u);
          if (slot < cur_m) {
            const float4 v =
                *reinterpret_cast<const float4*>(p.x + (size_t)en.tok[slot] * H + 16 * ks + 4 * (l & 3));
            __nv_bfloat16 h0, h1, h2, h3, l0, l1, l2, l3;
            split_bf16(v.x, h0, l0); split_bf16(v.y, h1, l1); split_bf16(v.z, h2, l2); split_bf16(v.w, h3, l3);
            o = make_uint4(pack2(h0, h1), pack2(h2, h3), pack2(l0, l1), pack2(l2, l3));
          }
          bfrag[idx] = o;
        }
      }
      consumer_bar();
    }
    if (cur_m == 0) continue;   // expert without weights: the producer skipped this unit too

    // ---- phase 1: [8 gate rows ; 8 up rows] x tokens, k split over the warps
    const uint32_t itA = it + (warp >> 2);
    {
      const uint32_t s = itA % (uint32_t)n_stages, ph = (itA / (uint32_t)n_stages) & 1u;
      mbar_wait(smem_u32(&hdr->full[s]), ph, abort_flag);
      const uint4* A = reinterpret_cast<const uint4*>(ring + (size_t)s * STAGE_BYTES) + (warp & 3) * KW * 32 + lane;
      float cacc[NT][2][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) cacc[nt][0][r] = cacc[nt][1][r] = 0.f;
#pragma unroll
      for (int i = 0; i < KW; ++i) {
        const uint4 a = A[i * 32];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (nt > 0 && cur_m <= 8 * nt) continue;
          const uint4 b = bfrag[(nt * KSTEPS + warp * KW + i) * 32 + lane];
          mma_k16(cacc[nt][i & 1], a, b.x, b.y);
          mma_k16(cacc[nt][i & 1], a, b.z, b.w);
        }
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&hdr->empty[it % (uint32_t)n_stages]));
        mbar_arrive(smem_u32(&hdr->empty[(it + 1) % (uint32_t)n_stages]));
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
        partial[((buf * 8 + warp) * NT + nt) * 32 + lane] =
            make_float4(cacc[nt][0][0] + cacc[nt][1][0], cacc[nt][0][1] + cacc[nt][1][1],
                        cacc[nt][0][2] + cacc[nt][1][2], cacc[nt][0][3] + cacc[nt][1][3]);
    }
    consumer_bar();

    // ---- reduce the k-split partials, activation, re-fragment for phase 2:
    // lane (g,c) needs act[i = 2c, 2c+1][token slot g] which sits in source
    // lane (i*4 + g/2), component g&1 (gate) / 2+(g&1) (up)
    uint32_t bhi[NT], blo[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float G0 = 0.f, U0 = 0.f, G1 = 0.f, U1 = 0.f;
      const int src0 = (2 * c) * 4 + (g >> 1), src1 = src0 + 4;
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        const float4 v0 = partial[((buf * 8 + w) * NT + nt) * 32 + src0];
        const float4 v1 = partial[((buf * 8 + w) * NT + nt) * 32 + src1];
        G0 += (g & 1) ? v0.y : v0.x; U0 += (g & 1) ? v0.w : v0.z;
        G1 += (g & 1) ? v1.y : v1.x; U1 += (g & 1) ? v1.w : v1.z;
      }
      const float a0 = dx_silu(G0) * U0, a1 = dx_silu(G1) * U1;
      __nv_bfloat16 h0, l0, h1, l1;
      split_bf16(a0, h0, l0);
      split_bf16(a1, h1, l1);
      bhi[nt] = pack2(h0, h1);
      blo[nt] = pack2(l0, l1);
    }
    buf ^= 1;

    // ---- phase 2: 8 columns of W_d x activations, output rows split over the warps
    {
      const uint32_t itD = it + 2;
      const uint32_t s = itD % (uint32_t)n_stages, ph = (itD / (uint32_t)n_stages) & 1u;
      mbar_wait(smem_u32(&hdr->full[s]), ph, abort_flag);
      const uint4* D = reinterpret_cast<const uint4*>(ring + (size_t)s * STAGE_BYTES) + warp * PW * 32 + lane;
#pragma unroll
      for (int q = 0; q < PW; ++q) {
        const uint4 a = D[q * 32];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (nt > 0 && cur_m <= 8 * nt) continue;
          mma_k8(acc[nt][2 * q], a.x, a.y, bhi[nt]);
          mma_k8(acc[nt][2 * q], a.x, a.y, blo[nt]);
          mma_k8(acc[nt][2 * q + 1], a.z, a.w, bhi[nt]);
          mma_k8(acc[nt][2 * q + 1], a.z, a.w, blo[nt]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&hdr->empty[s]));
    }
    it += 3;
  }
  if (ei >= 0 && cur_m > 0) flush(ei);
  if (*abort_flag && threadIdx.x == 0) atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------- fp32 path
// Plain CUDA-core version for fp32 weights (small layers): one CTA per unit,
// warp w owns gate/up row w, then every thread owns output columns.
__global__ void __launch_bounds__(256) dx_experts_fp32_kernel(DxExpertParams p) {
  __shared__ float s_act[DX_MAX_K][DX_TILE_I];
  const DxWork* W = p.work;
  const int n_entries = W->n_entries, total = W->total_units, H = p.H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int ei = 0;
  for (int u = blockIdx.x; u < total; u += gridDim.x) {
    ei = find_entry(W, n_entries, u, ei);
    const DxEntry& en = W->entries[ei];
    const float* blob = reinterpret_cast<const float*>(p.table[en.table_index]);
    if (blob == nullptr) {
      if (threadIdx.x == 0) atomicExch(p.dev_status, DX_DEV_BAD_EXPERT_ID);
      continue;
    }
    const float* unit = blob + (size_t)(u - en.unit_begin) * 24 * H;
    const float* gr = unit + (size_t)warp * H;
    const float* ur = unit + (size_t)(8 + warp) * H;
    for (int t = 0; t < en.m; ++t) {
      const float* x = p.x + (size_t)en.tok[t] * H;
      float ag = 0.f, au = 0.f;
      for (int j = lane; j < H; j += 32) {
        const float xv = x[j];
        ag = fmaf(gr[j], xv, ag);
        au = fmaf(ur[j], xv, au);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ag += __shfl_xor_sync(0xffffffffu, ag, o);
        au += __shfl_xor_sync(0xffffffffu, au, o);
      }
      if (lane == 0) s_act[t][warp] = dx_silu(ag) * au;
    }
    __syncthreads();
    const float* dT = unit + (size_t)16 * H;
    for (int hh = threadIdx.x; hh < H; hh += 256) {
      float d[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) d[i] = dT[(size_t)i * H + hh];
      for (int t = 0; t < en.m; ++t) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) s = fmaf(s_act[t][i], d[i], s);
        atomicAdd(p.y + (size_t)en.tok[t] * H + hh, en.w[t] * s);
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------ pack kernels
// bf16 blob, unit j (24*H elements):
//   gate/up part (16*H): k-step s, lane l=(g,c): 8 elements
//       { Wg[8j+g][16s+4c+0..1], Wu[8j+g][16s+4c+0..1], Wg[8j+g][16s+4c+2..3], Wu[8j+g][16s+4c+2..3] }
//   down part (8*H): row-tile pair q, lane l=(g,c): 8 elements
//       { Wd[32q+g][8j+2c..+1], Wd[32q+8+g][..], Wd[32q+16+g][..], Wd[32q+24+g][..] }
__global__ void dx_pack_bf16_kernel(const __nv_bfloat16* Wg, const __nv_bfloat16* Wu, const __nv_bfloat16* Wd,
                                    __nv_bfloat16* blob, int H, int I) {
  const size_t n = (size_t)3 * H * I;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x) {
    const size_t unit = idx / (24 * (size_t)H);
    const int r = (int)(idx % (24 * (size_t)H));
    const int j = (int)unit;
    __nv_bfloat16 v;
    if (r < 16 * H) {
      const int s = r / 256, l = (r % 256) / 8, el = r % 8;
      const int g = l >> 2, c = l & 3;
      const int col = 16 * s + 4 * c + (el & 1) + ((el >> 2) << 1);
      const int row = 8 * j + g;
      v = ((el >> 1) & 1) ? Wu[(size_t)row * H + col] : Wg[(size_t)row * H + col];
    } else {
      const int r2 = r - 16 * H;
      const int q = r2 / 256, l = (r2 % 256) / 8, el = r2 % 8;
      const int g = l >> 2, c = l & 3;
      const int row = 32 * q + 8 * (el >> 1) + g;
      const int col = 8 * j + 2 * c + (el & 1);
      v = Wd[(size_t)row * I + col];
    }
    blob[idx] = v;
  }
}

// fp32 blob, unit j: Wg rows 8j..8j+7 [8][H], Wu rows [8][H], then W_d columns 8j..8j+7 transposed [8][H]
__global__ void dx_pack_fp32_kernel(const float* Wg, const float* Wu, const float* Wd, float* blob, int H, int I) {
  const size_t n = (size_t)3 * H * I;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(idx / (24 * (size_t)H));
    const int r = (int)(idx % (24 * (size_t)H));
    const int row = r / H, col = r % H;
    float v;
    if (row < 8) v = Wg[(size_t)(8 * j + row) * H + col];
    else if (row < 16) v = Wu[(size_t)(8 * j + row - 8) * H + col];
    else v = Wd[(size_t)col * I + 8 * j + (row - 16)];
    blob[idx] = v;
  }
}

template <int H, int NT>
size_t bf16_fixed_smem() {
  return sizeof(SmemHeader) + (size_t)2 * 8 * NT * 32 * 16 + (size_t)NT * (H / 16) * 32 * 16;
}

template <int H, int NT>
cudaError_t launch_bf16(dx_ctx* ctx, const DxExpertParams& p, cudaStream_t st) {
  const size_t fixed = bf16_fixed_smem<H, NT>();
  const size_t stage = (size_t)16 * H;
  int n_stages = (int)(((size_t)ctx->smem_optin - fixed) / stage);
  if (n_stages > 8) n_stages = 8;
  if (n_stages < 2) return cudaErrorInvalidConfiguration;
  const size_t smem = fixed + (size_t)n_stages * stage;
  cudaError_t e = cudaFuncSetAttribute(dx_experts_bf16_kernel<H, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  dx_experts_bf16_kernel<H, NT><<<ctx->sm_count, kThreads, smem, st>>>(p, n_stages);
  return cudaGetLastError();
}

template <int H>
cudaError_t launch_bf16_h(dx_ctx* ctx, const DxExpertParams& p, int K, cudaStream_t st) {
  return K > 8 ? launch_bf16<H, 2>(ctx, p, st) : launch_bf16<H, 1>(ctx, p, st);
}

}  // namespace

bool dx_bf16_hidden_supported(int H) { return H == 256 || H == 512 || H == 1024 || H == 2048; }

cudaError_t dx_launch_experts(dx_ctx* ctx, const DxExpertParams& p, int weight_dtype, int K, cudaStream_t st) {
  if (weight_dtype == DX_DTYPE_FP32) {
    dx_experts_fp32_kernel<<<ctx->sm_count * 4, 256, 0, st>>>(p);
    return cudaGetLastError();
  }
  switch (p.H) {
    case 256: return launch_bf16_h<256>(ctx, p, K, st);
    case 512: return launch_bf16_h<512>(ctx, p, K, st);
    case 1024: return launch_bf16_h<1024>(ctx, p, K, st);
    case 2048: return launch_bf16_h<2048>(ctx, p, K, st);
    default: return cudaErrorInvalidConfiguration;
  }
}

cudaError_t dx_launch_pack(int weight_dtype, int H, int I, const void* Wg, const void* Wu, const void* Wd,
                           void* blob, cudaStream_t st) {
  const size_t n = (size_t)3 * H * I;
  int grid = (int)((n + 255) / 256);
  if (grid > 4096) grid = 4096;
  if (weight_dtype == DX_DTYPE_BF16)
    dx_pack_bf16_kernel<<<grid, 256, 0, st>>>((const __nv_bfloat16*)Wg, (const __nv_bfloat16*)Wu,
                                              (const __nv_bfloat16*)Wd, (__nv_bfloat16*)blob, H, I);
  else
    dx_pack_fp32_kernel<<<grid, 256, 0, st>>>((const float*)Wg, (const float*)Wu, (const float*)Wd, (float*)blob, H,
                                              I);
  return cudaGetLastError();
}
