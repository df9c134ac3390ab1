// Grouped SwiGLU for blocks of up to 16 rows on the 5th-generation tensor cores (tcgen05, accumulators in tensor
// memory): the same summands of Eq. 4 / Eq. 5 as dx_grouped.cu,
//     y[tok] += w[tok] * W_d ( silu(W_g x[tok]) * (W_u x[tok]) ),
// with each expert streamed from HBM once per block, for layers packed in the "wide" blob layout
// (DX_DTYPE_BF16_WIDE).
//
// Why a second kernel.  With mma.sync the block rows are the 8-column operand: nine to sixteen rows double the
// tensor work of every consumer warp and either double the shared-memory traffic (two token tiles) or make two CTAs
// stream the same bytes.  Here the weights are the 128-row operand of tcgen05.mma, read from shared memory by the
// tensor core itself, the block rows are the 16-column operand, and one thread issues all products, so the number of
// block rows (1..16) changes nothing and no warp's dependent instruction chain sits between two weight tiles.
//
// Blob layout (dx_pack_expert for DX_DTYPE_BF16_WIDE; same bytes as the three matrices).  A unit is still 8
// intermediate indices (48 H bytes), so work is split between CTAs exactly as in dx_grouped.cu; 8 consecutive
// units of an expert form a macro-unit (MU; the last one of an expert may have fewer).  Everything is stored as 8 x 8
// "core matrices" (8 rows x 16 bytes, 128 contiguous bytes), the shared-memory image tcgen05 reads without a swizzle:
//   gate/up region of an MU with nq units: [s < H/64][rg < 2 nq][kg < 8]  core matrix = rows 8 (8 m + rg/2) .. + 7 of
//       W_g (rg even) or W_u (rg odd), columns 64 s + 8 kg .. + 7                    -- one "stage" per s
//   down region:                       [T < H/128][q < nq][hg < 16] core matrix = rows 128 T + 8 hg .. + 7 of W_d,
//       columns 8 (8 m + q) .. + 7                                                   -- one stage per T
// A stage is at most 16 KB and is one bulk copy (a CTA that owns only units q0..q1 of an MU copies that contiguous
// part of every stage, to the same offset of the shared-memory stage).
//
// Per MU piece: D1[128 x 16] = [gate rows; up rows] x block rows^T over H (accumulated in tensor memory over the
// H/64 stages), the epilogue warps read D1, form w * silu(g) * u in bf16 as the next operand in shared memory, and
// D2[T][128 x 16] += W_d tile x that, for every tile T of 128 output rows; D2 (H/128 tiles x 16 columns) stays in
// tensor memory across all pieces of the CTA and is added to y once, at the end.  Rows of a stage that were not
// copied hold older weights or zeros (the ring is cleared once): their products are finite and meet zero activations.
// The first product of piece p + 1 is issued before the second of piece p, so the epilogue's latency is covered.
//
// Warps: 0-3 epilogue (tensor-memory lanes 32 w .. 32 w + 31), 4 producer (one lane issues the bulk copies), 5 issues
// the tcgen05.mma (one lane) and owns the tensor-memory allocation.  Every wait is bounded (context's wait limit); a
// wait that runs out raises the CTA's abort flag, after which nothing more is copied or multiplied, the CTA waits
// (bounded) for what is in flight, frees its tensor memory and returns with DX_DEV_WAIT_EXPIRED in the status word.
#include "dx_internal.cuh"
#include "dx_stream.cuh"

namespace {

constexpr int kWideThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kStageBytes = 16384;
constexpr int kMaxStages = 12;
constexpr int kTok = 16;          // token columns of every product

struct WideHeader {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long d1_full[2];
  unsigned long long act_ready[2];
  unsigned long long d2_full;
  unsigned long long x_ready;
  uint32_t tmem_base;
  int abort_flag;
  int ph_e_lo[2], ph_e_hi[2], ph_u_lo[2], ph_u_hi[2];   // routing-independent groups, then routed groups
  int kk, n_pairs;
  float rstd[DX_MAX_K];
  int e_begin[DX_MAX_ENTRIES];
  int e_tiles[DX_MAX_ENTRIES];
  int e_gid[DX_MAX_ENTRIES];
  const unsigned char* e_blob[DX_MAX_ENTRIES];
  int pair_id[DX_MAX_PAIRS];
  float pair_w[DX_MAX_PAIRS];
  float roww[DX_MAX_ENTRIES][kTok];   // weight of every group in every block row (0: the row is not in the group)
};

struct Piece {
  int e;        // group
  int m;        // macro-unit of the group's expert
  int q0, q1;   // units of the macro-unit this CTA owns
  int nq;       // units the macro-unit has (8, or fewer for an expert's last one)
};

// The CTA's pieces in the order all three roles walk them.
template <class F>
__device__ __forceinline__ void for_each_piece(const WideHeader* hdr, F&& f) {
  for (int ph = 0; ph < 2; ++ph)
    for (int e = hdr->ph_e_lo[ph]; e < hdr->ph_e_hi[ph]; ++e) {
      const int b = hdr->e_begin[e], nt = hdr->e_tiles[e];
      const int lo = max(b, hdr->ph_u_lo[ph]), hi = min(b + nt, hdr->ph_u_hi[ph]);
      if (lo >= hi || hdr->e_blob[e] == nullptr) continue;
      for (int u = lo; u < hi;) {
        const int m = (u - b) >> 3;
        const int end = min(hi, b + 8 * (m + 1));
        Piece pc;
        pc.e = e; pc.m = m; pc.q0 = (u - b) & 7; pc.q1 = pc.q0 + (end - u); pc.nq = min(8, nt - 8 * m);
        f(pc);
        u = end;
      }
    }
}

// shared-memory matrix descriptor: no swizzle, K-major; lbo = bytes between the two core matrices of a product
// along the contraction, sbo = bytes between groups of eight rows
__device__ __forceinline__ uint64_t umma_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}
// D[128 x 16] (+)= A[128 x 16] B[16 x 16]^T, bf16 operands from shared memory, fp32 accumulator in tensor memory
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTok >> 3) << 17) | (8u << 24);
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d_tmem), "l"(da), "l"(db), "r"(kIdesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__host__ __device__ constexpr int tmem_columns(int H) {
  const int need = 32 + H / 8;   // two D1 buffers of 16 columns, H/128 D2 tiles of 16 columns
  return need <= 32 ? 32 : need <= 64 ? 64 : need <= 128 ? 128 : need <= 256 ? 256 : 512;
}

template <int H>
__global__ void __launch_bounds__(kWideThreads, 1) dx_experts_wide_kernel(DxExpertParams p, int n_stages) {
  constexpr int S1 = H / 64;            // gate/up stages of a piece
  constexpr int S2 = H / 128;           // down stages (output tiles) of a piece
  constexpr uint32_t UNIT_BYTES = 48u * H;
  constexpr uint32_t X_BYTES = 32u * H;   // [H/8][2][128 B]
  constexpr int TCOLS = tmem_columns(H);

  extern __shared__ __align__(128) unsigned char smem[];
  WideHeader* hdr = reinterpret_cast<WideHeader*>(smem);
  constexpr size_t HDR = (sizeof(WideHeader) + 127) / 128 * 128;
  unsigned char* xs = smem + HDR;                       // block rows as the bf16 16-column operand
  unsigned char* acts = xs + X_BYTES;                   // two SwiGLU-product operands [8 q][2][128 B]
  unsigned char* ring = acts + 2 * 2048;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const DxWork* W = p.work;
  const int G = gridDim.x, cta = blockIdx.x;
  const int n_static = p.n_shared + (p.draft_tiles > 0 ? 1 : 0);
  const int S0 = p.skip_shared ? p.n_shared * p.shared_tiles : 0;
  const int NS = p.do_static ? p.n_shared * p.shared_tiles + p.draft_tiles - S0 : 0;
  const int s_lo = S0 + (int)(((long long)NS * cta) / G), s_hi = S0 + (int)(((long long)NS * (cta + 1)) / G);
  volatile int* abort_flag = &hdr->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(smem_u32(&hdr->full[s]), 1);
      mbar_init(smem_u32(&hdr->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&hdr->d1_full[b]), 1);
      mbar_init(smem_u32(&hdr->act_ready[b]), 4);
    }
    mbar_init(smem_u32(&hdr->d2_full), 1);
    mbar_init(smem_u32(&hdr->x_ready), 4);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&hdr->tmem_base)),
                 "r"(TCOLS));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  // the ring starts out as zeros: rows of a stage that a partial piece does not copy must hold finite values
  for (uint32_t i = threadIdx.x; i < (uint32_t)n_stages * (kStageBytes / 16); i += kWideThreads)
    reinterpret_cast<uint4*>(ring)[i] = make_uint4(0u, 0u, 0u, 0u);
  proxy_fence();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  const uint32_t tm_d1 = tmem, tm_d2 = tmem + 32;

  // the routing kernel in front has completed once this returns: the work list is final and y is initialised
  dx_pdl_wait();

  // ---- the groups of this launch and this CTA's share of their units (as in dx_grouped.cu, without the hand-over)
  if (warp == 4) {
    if (lane < n_static) {
      const bool is_draft = lane >= p.n_shared;
      hdr->e_begin[lane] = is_draft ? p.n_shared * p.shared_tiles : lane * p.shared_tiles;
      hdr->e_tiles[lane] = is_draft ? p.draft_tiles : p.shared_tiles;
      hdr->e_gid[lane] = -1;
      hdr->e_blob[lane] = DX_BOUNDS(lane < p.table_len, p.dev_status)
                              ? reinterpret_cast<const unsigned char*>(p.table[lane]) : nullptr;
    }
    const unsigned long long head = dx_word_load(&W->head);
    int n_groups = 0, kk = 1, n_pairs = 0;
    if (head & DX_WORD_VALID) {
      n_groups = min((int)(head & 0xffffu), DX_MAX_PAIRS);
      kk = (int)((head >> 16) & 0xffu);
      n_pairs = min((int)((head >> 24) & 0xffu) * kk, DX_MAX_PAIRS);
    }
    constexpr int PER_LANE = DX_MAX_PAIRS / 32;
    unsigned long long gw[PER_LANE];
    int pos[PER_LANE];
    int n_sel = 0;
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) {
      const int idx = lane + 32 * i;
      gw[i] = idx < n_groups ? dx_word_load(&W->group[idx]) : 0ull;
      const int gid = dx_group_id(gw[i]);
      const bool in = idx < n_groups && (gw[i] & DX_WORD_VALID) &&
                      (!p.use_subset || (gid < DX_MAX_E && ((p.subset[gid >> 6] >> (gid & 63)) & 1ull)));
      const unsigned int b = __ballot_sync(0xffffffffu, in);
      pos[i] = in ? n_sel + __popc(b & ((1u << lane) - 1u)) : -1;
      n_sel += __popc(b);
    }
    n_groups = n_sel;
    int e_lo, e_hi, u_lo, u_hi;
    dx_routed_range(n_groups, p, n_static, NS, s_lo - S0, s_hi - S0, G, cta, e_lo, e_hi, u_lo, u_hi);
    const int unit_base = p.n_shared * p.shared_tiles + p.draft_tiles;
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) {
      const int idx = pos[i];
      if (idx < 0) continue;
      const int gid = dx_group_id(gw[i]);
      const unsigned char* blob = nullptr;
      if (gid < DX_MAX_E && DX_BOUNDS(p.n_shared + 1 + gid < p.table_len, p.dev_status))
        blob = reinterpret_cast<const unsigned char*>(p.table[p.n_shared + 1 + gid]);
      const int e = n_static + idx;
      if (!DX_BOUNDS(e < DX_MAX_ENTRIES, p.dev_status)) continue;
      hdr->e_begin[e] = unit_base + idx * p.routed_tiles;
      hdr->e_tiles[e] = p.routed_tiles;
      hdr->e_gid[e] = gid;
      hdr->e_blob[e] = blob;
      if (blob == nullptr && e >= e_lo && e < e_hi) atomicExch(p.dev_status, DX_DEV_BAD_EXPERT_ID);
    }
    for (int idx = lane; idx < n_pairs; idx += 32) {
      const unsigned long long w = dx_word_load(&W->pair[idx]);
      hdr->pair_id[idx] = dx_pair_id(w);
      hdr->pair_w[idx] = (w & DX_WORD_VALID) ? dx_pair_weight(w) : 0.0f;
    }
    if (lane == 0) {
      hdr->kk = kk;
      hdr->n_pairs = n_pairs;
      hdr->ph_e_lo[0] = 0; hdr->ph_e_hi[0] = p.do_static ? n_static : 0;
      hdr->ph_u_lo[0] = s_lo; hdr->ph_u_hi[0] = s_hi;
      hdr->ph_e_lo[1] = e_lo; hdr->ph_e_hi[1] = e_hi; hdr->ph_u_lo[1] = u_lo; hdr->ph_u_hi[1] = u_hi;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) dx_pdl_trigger();   // what follows on the stream may be scheduled (it waits for this grid to end)

  if (warp == 4) {
    // ------------------------------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t it = 0, slot = 0, phase = 0;
      bool alive = true;
      const uint64_t l2pol = l2_evict_first_policy();
      auto push = [&](const unsigned char* src, uint32_t bytes, uint32_t dst_off) {
        if (!alive) return;
        if (!mbar_wait(smem_u32(&hdr->empty[slot]), phase ^ 1u, abort_flag, p.wait_limit)) { alive = false; return; }
        const uint32_t fb = smem_u32(&hdr->full[slot]);
        mbar_arrive_expect_tx(fb, bytes);
        bulk_g2s(smem_u32(ring + (size_t)slot * kStageBytes + dst_off), src, bytes, fb, l2pol);
        ++it;
        if (++slot == (uint32_t)n_stages) { slot = 0; phase ^= 1u; }
      };
      auto gate_up = [&](const Piece& c) {
        const unsigned char* mu = hdr->e_blob[c.e] + (size_t)c.m * 8 * UNIT_BYTES;
        const uint32_t bytes = (uint32_t)(c.q1 - c.q0) * 2048u, off = (uint32_t)c.q0 * 2048u;
        for (int s = 0; s < S1; ++s) push(mu + (size_t)s * c.nq * 2048 + off, bytes, off);
      };
      auto down = [&](const Piece& c) {
        const unsigned char* mu = hdr->e_blob[c.e] + (size_t)c.m * 8 * UNIT_BYTES + (size_t)c.nq * 32 * H;
        const uint32_t bytes = (uint32_t)(c.q1 - c.q0) * 2048u, off = (uint32_t)c.q0 * 2048u;
        for (int t = 0; t < S2; ++t) push(mu + (size_t)t * c.nq * 2048 + off, bytes, off);
      };
      Piece prev;
      bool have_prev = false;
      for_each_piece(hdr, [&](const Piece& c) {
        gate_up(c);
        if (have_prev) down(prev);
        prev = c;
        have_prev = true;
      });
      if (have_prev) down(prev);
      if (*abort_flag) {
        // something gave up: no copy may still be landing when the CTA's shared memory is released
        const uint32_t n_back = it < (uint32_t)n_stages ? it : (uint32_t)n_stages;
        for (uint32_t k = 1; k <= n_back; ++k) {
          const uint32_t j = it - k, s = j % (uint32_t)n_stages, ph = (j / (uint32_t)n_stages) & 1u;
          for (uint32_t spin = 0; spin < DX_WAIT_LIMIT_DEFAULT; ++spin)
            if (mbar_try_wait(smem_u32(&hdr->full[s]), ph)) break;
        }
        atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------------------------------ tensor-core issue
    if (lane == 0) {
      uint32_t slot = 0, phase = 0;
      bool alive = mbar_wait(smem_u32(&hdr->x_ready), 0u, abort_flag, p.wait_limit);
      tc_fence_after();
      const uint32_t xs_addr = smem_u32(xs), act_addr = smem_u32(acts);
      uint32_t d2_started = 0u;    // bit T: tile T of D2 has been written
      int n_done = 0;
      auto next_stage = [&](uint32_t& stage_addr) -> bool {
        if (!alive) return false;
        if (!mbar_wait(smem_u32(&hdr->full[slot]), phase, abort_flag, p.wait_limit)) { alive = false; return false; }
        tc_fence_after();
        stage_addr = smem_u32(ring + (size_t)slot * kStageBytes);
        return true;
      };
      auto release_stage = [&]() {
        umma_commit(smem_u32(&hdr->empty[slot]));     // the slot is free again once the products above have read it
        if (++slot == (uint32_t)n_stages) { slot = 0; phase ^= 1u; }
      };
      auto gate_up = [&](const Piece& c, int pidx) {
        const uint32_t d1 = tm_d1 + (uint32_t)(pidx & 1) * kTok;
        for (int s = 0; s < S1; ++s) {
          uint32_t st;
          if (!next_stage(st)) return;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            umma(d1, umma_desc(st + j * 256, 128, 1024), umma_desc(xs_addr + (8 * s + 2 * j) * 256, 256, 128),
                 (s | j) != 0 ? 1u : 0u);
          release_stage();
        }
        umma_commit(smem_u32(&hdr->d1_full[pidx & 1]));
      };
      auto down = [&](const Piece& c, int pidx) {
        // the SwiGLU products of this piece, written by the epilogue warps
        if (alive && !mbar_wait(smem_u32(&hdr->act_ready[pidx & 1]), (uint32_t)(pidx >> 1) & 1u, abort_flag, p.wait_limit))
          alive = false;
        tc_fence_after();
        const uint32_t act = act_addr + (uint32_t)(pidx & 1) * 2048u;
        for (int t = 0; t < S2; ++t) {
          uint32_t st;
          if (!next_stage(st)) return;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (2 * j + 1 < c.q0 || 2 * j >= c.q1) continue;     // both units of this product lie outside the piece
            umma(tm_d2 + (uint32_t)t * kTok, umma_desc(st + j * 4096, 2048, 128), umma_desc(act + j * 512, 256, 128),
                 (d2_started >> t) & 1u);
            d2_started |= 1u << t;
          }
          release_stage();
        }
      };
      Piece prev;
      bool have_prev = false;
      for_each_piece(hdr, [&](const Piece& c) {
        gate_up(c, n_done);
        if (have_prev) down(prev, n_done - 1);
        prev = c;
        have_prev = true;
        ++n_done;
      });
      if (have_prev) down(prev, n_done - 1);
      umma_commit(smem_u32(&hdr->d2_full));   // (also what the epilogue waits for before it lets the memory go)
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int tid = threadIdx.x;   // 0..127 = tensor-memory lane
    // 1/rms of the block rows, then the rows as the bf16 operand [H/8][2][8 rows x 16 bytes]
    for (int r = warp; r < kTok; r += 4) {
      float rs = 1.0f;
      if (p.rms_norm && r < p.K) {
        float ss = 0.f;
        for (int j = lane * 4; j < H; j += 128) {
          const float4 v = *reinterpret_cast<const float4*>(p.x + (size_t)r * H + j);
          ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        rs = rsqrtf(ss / (float)H + 1e-6f);
      }
      if (lane == 0) hdr->rstd[r] = rs;
    }
    epi_bar();
    for (int idx = tid; idx < kTok * (H / 8); idx += kEpiThreads) {
      const int t = idx & 15, kg = idx >> 4;
      uint4 o = make_uint4(0u, 0u, 0u, 0u);
      if (t < p.K) {
        const float rs = hdr->rstd[t];
        const float* src = p.x + (size_t)t * H + 8 * kg;
        const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
        o.x = pack2(__float2bfloat16_rn(a.x * rs), __float2bfloat16_rn(a.y * rs));
        o.y = pack2(__float2bfloat16_rn(a.z * rs), __float2bfloat16_rn(a.w * rs));
        o.z = pack2(__float2bfloat16_rn(b.x * rs), __float2bfloat16_rn(b.y * rs));
        o.w = pack2(__float2bfloat16_rn(b.z * rs), __float2bfloat16_rn(b.w * rs));
      }
      *reinterpret_cast<uint4*>(xs + (size_t)kg * 256 + (t >> 3) * 128 + (t & 7) * 16) = o;
    }
    // every group's weight in every block row
    {
      const int n_entries = max(hdr->ph_e_hi[0], hdr->ph_e_hi[1]);
      const int kk = hdr->kk;
      for (int idx = tid; idx < n_entries * kTok; idx += kEpiThreads) {
        const int e = idx >> 4, row = idx & 15;
        float w = 0.0f;
        if (row < p.K) {
          if (e < n_static) w = e < p.n_shared ? 1.0f : p.gamma;
          else {
            const int gid = hdr->e_gid[e];
            for (int j = 0; j < kk; ++j)
              if (hdr->pair_id[row * kk + j] == gid) w = hdr->pair_w[row * kk + j];
          }
        }
        hdr->roww[e][row] = w;
      }
    }
    proxy_fence();            // the operand above was written with ordinary stores, the tensor core reads it
    epi_bar();
    if (lane == 0) mbar_arrive(smem_u32(&hdr->x_ready));

    // lane of tensor memory = row of D1: row group rg = tid / 8 = 2 q + (0 gate | 1 up), row r of the unit
    const int q = tid >> 4, gu = (tid >> 3) & 1, r = tid & 7;
    const uint32_t lane_base = (uint32_t)(32 * warp) << 16;
    int pidx = 0;
    bool alive = true;
    for_each_piece(hdr, [&](const Piece& c) {
      if (alive && !mbar_wait(smem_u32(&hdr->d1_full[pidx & 1]), (uint32_t)(pidx >> 1) & 1u, abort_flag, p.wait_limit))
        alive = false;
      tc_fence_after();
      float v[16];
      tmem_ld16(tm_d1 + lane_base + (uint32_t)(pidx & 1) * kTok, v);
      // a gate row takes block rows 0..7, its up row (8 lanes on) block rows 8..15: swap the halves each needs
      float other[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) other[i] = __shfl_xor_sync(0xffffffffu, gu ? v[i] : v[8 + i], 8);
      const bool mine = q >= c.q0 && q < c.q1;
      unsigned char* dst = acts + (size_t)(pidx & 1) * 2048 + (size_t)q * 256 + gu * 128 + r * 2;
      const float* wrow = hdr->roww[c.e] + 8 * gu;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float g = gu ? other[i] : v[i], u = gu ? v[8 + i] : other[i];
        const float a = mine ? fast_silu(g) * u * wrow[i] : 0.0f;
        *reinterpret_cast<__nv_bfloat16*>(dst + i * 16) = __float2bfloat16_rn(a);
      }
      proxy_fence();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&hdr->act_ready[pidx & 1]));
      ++pidx;
    });
    // ---- this CTA's partial output rows: D2 tile T, lane = output row 128 T + tid, columns = block rows
    if (alive && !mbar_wait(smem_u32(&hdr->d2_full), 0u, abort_flag, p.wait_limit)) alive = false;
    tc_fence_after();
    if (pidx > 0 && alive && !*abort_flag) {
      for (int t = 0; t < S2; ++t) {
        float v[16];
        tmem_ld16(tm_d2 + lane_base + (uint32_t)t * kTok, v);
        float* ycol = p.y + 128 * t + tid;
#pragma unroll
        for (int row = 0; row < kTok; ++row)
          if (row < p.K)
            asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(ycol + (size_t)row * H), "f"(v[row]) : "memory");
      }
    }
    tc_fence_before();
  }
  // ---- everything this CTA put in flight has landed (or has been waited for): the tensor memory goes back
  __syncthreads();
  if (warp == 5) {
    if (lane == 0 && *abort_flag) {
      // products may still be running if a wait gave up: the last commit covers all of them
      for (uint32_t spin = 0; spin < DX_WAIT_LIMIT_DEFAULT; ++spin)
        if (mbar_try_wait(smem_u32(&hdr->d2_full), 0u)) break;
      atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED);
    }
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TCOLS));
  }
}

// bf16 "wide" blob from the three canonical matrices: see the layout at the top of the file
__global__ void dx_pack_wide_kernel(const __nv_bfloat16* Wg, const __nv_bfloat16* Wu, const __nv_bfloat16* Wd,
                                    __nv_bfloat16* blob, int H, int I) {
  const size_t n = (size_t)3 * H * I;
  const size_t mu_elems = (size_t)8 * 24 * H;       // elements of a full macro-unit
  const int n_units = I / 8;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x) {
    const int m = (int)(idx / mu_elems);
    const size_t local = idx - (size_t)m * mu_elems;
    const int nq = min(8, n_units - 8 * m);
    const size_t gu_elems = (size_t)nq * 16 * H;
    __nv_bfloat16 v;
    if (local < gu_elems) {
      const size_t stage = (size_t)2 * nq * 512;
      const int s = (int)(local / stage);
      const int rem = (int)(local % stage);
      const int rg = rem / 512, rem2 = rem % 512;
      const int kg = rem2 / 64, r = (rem2 % 64) / 8, el = rem2 % 8;
      const int row = 8 * (8 * m + rg / 2) + r, col = 64 * s + 8 * kg + el;
      v = (rg & 1) ? Wu[(size_t)row * H + col] : Wg[(size_t)row * H + col];
    } else {
      const size_t l2 = local - gu_elems;
      const size_t tile = (size_t)nq * 1024;
      const int t = (int)(l2 / tile);
      const int rem = (int)(l2 % tile);
      const int q = rem / 1024, rem2 = rem % 1024;
      const int hg = rem2 / 64, r = (rem2 % 64) / 8, el = rem2 % 8;
      v = Wd[(size_t)(128 * t + 8 * hg + r) * I + 8 * (8 * m + q) + el];
    }
    blob[idx] = v;
  }
}

template <int H>
cudaError_t launch_wide(dx_ctx* ctx, const DxExpertParams& p, cudaStream_t st) {
  const size_t hdr = (sizeof(WideHeader) + 127) / 128 * 128;
  const size_t fixed = hdr + (size_t)32 * H + 2 * 2048;
  int n_stages = (int)(((size_t)ctx->smem_optin - fixed) / kStageBytes);
  if (n_stages > kMaxStages) n_stages = kMaxStages;
  if (n_stages < 3) return cudaErrorInvalidConfiguration;
  const size_t smem = fixed + (size_t)n_stages * kStageBytes;
  cudaError_t e = cudaFuncSetAttribute(dx_experts_wide_kernel<H>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = ctx->sm_count > 16 ? ctx->sm_count - DX_ROUTE_CLUSTER : ctx->sm_count;
  return dx_launch_pdl((ctx->pdl_mask & DX_PDL_EXPERTS) != 0, dx_experts_wide_kernel<H>, dim3(grid), dim3(kWideThreads),
                       smem, st, 1, p, n_stages);
}

}  // namespace

cudaError_t dx_launch_experts_wide(dx_ctx* ctx, const DxExpertParams& p, cudaStream_t st) {
  switch (p.H) {
    case 256: return launch_wide<256>(ctx, p, st);
    case 512: return launch_wide<512>(ctx, p, st);
    case 1024: return launch_wide<1024>(ctx, p, st);
    case 2048: return launch_wide<2048>(ctx, p, st);
    default: return cudaErrorInvalidConfiguration;
  }
}

cudaError_t dx_launch_pack_wide(int H, int I, const void* Wg, const void* Wu, const void* Wd, void* blob, cudaStream_t st) {
  const size_t n = (size_t)3 * H * I;
  int grid = (int)((n + 255) / 256);
  if (grid > 4096) grid = 4096;
  dx_pack_wide_kernel<<<grid, 256, 0, st>>>((const __nv_bfloat16*)Wg, (const __nv_bfloat16*)Wu, (const __nv_bfloat16*)Wd,
                                            (__nv_bfloat16*)blob, H, I);
  return cudaGetLastError();
}
