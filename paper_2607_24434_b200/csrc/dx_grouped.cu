// Grouped SwiGLU over the work list built by the routing kernel: for every
// group (an expert plus the block tokens routed to it)
//     y[tok] += w[tok] * W_d ( silu(W_g x[tok]) * (W_u x[tok]) )            (the summands of Eq. 4 / Eq. 5)
// with each expert's weights streamed from HBM exactly once per block.
//
// Work decomposition.  An expert is cut into I/8 "units": 8 rows of W_g, the
// same 8 rows of W_u and the matching 8 columns of W_d.  A unit is
// self-contained (its 8 activations feed only its own 8 columns of W_d), so the
// down projection is fused in and nothing intermediate ever reaches HBM.  The
// global unit list is split into equal contiguous ranges, one per CTA.  The MMA
// token slots are the block rows themselves for every group (a group's weight,
// zero for rows outside it, multiplies the activations), so a CTA keeps its
// partial y in registers across all its groups and adds it to y once, at the
// end, with fp32 reductions.
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
#include <cuda_fp16.h>

#include <type_traits>

#include "dx_internal.cuh"
#include "dx_stream.cuh"

namespace {

// ----------------------------------------------------- bf16 tensor-core path
// Streaming layout.  A unit (8 gate rows, 8 up rows, 8 down columns; 48*H bytes)
// is stored as eight equal "chunks", one per consumer warp: chunk w holds the
// gate/up fragments of contraction steps [w*H/128, (w+1)*H/128) followed by the
// down-projection fragments of output row tiles [w*H/128, (w+1)*H/128).  A chunk
// is one bulk copy, one ring slot, one full/empty mbarrier pair, and is read by
// exactly one warp, so slots recycle warp by warp and the producer can run
// more than two units ahead of the consumers.
//
// Overlap with routing.  The groups that do not depend on the router (the
// shared experts, and the draft expert in draft mode) are known from the layer
// description alone.  The kernel is launched with programmatic stream
// serialization behind the routing kernel, which lets it start before either
// kernel has its input: the producer streams those groups at once, the
// consumers begin when the routing kernel has published that the block is
// final, and the routed groups are polled out of the work list as the routing
// kernel writes it (fused entry points; otherwise the kernel simply waits for
// the routing kernel first).  Nothing is written to y before the routing
// kernel has completed (griddepcontrol.wait in front of the final reductions),
// because the routing kernel is what initialises y.
constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxSlots = 48;

struct SmemHeader {
  unsigned long long full[kMaxSlots];
  unsigned long long empty[kMaxSlots];
  int abort_flag;
  int r_e_lo, r_e_hi, r_u_lo;   // this CTA's routed entries and units, published by the producer warp
  int r_u_hi;
  float rstd[DX_MAX_K];
  float ssq[8][8];                   // sums of squares of the block rows, per consumer warp's slice
  int e_begin[DX_MAX_ENTRIES];       // first unit of each group (routing-independent groups first)
  int e_tiles[DX_MAX_ENTRIES];
  int e_gid[DX_MAX_ENTRIES];         // expert id of a routed group
  const unsigned char* e_blob[DX_MAX_ENTRIES];
  int kk;                            // selected experts per block row
  int n_pairs;                       // K * kk
  int pair_id[DX_MAX_PAIRS];         // [K,kk] selected expert ids and gate weights of the block
  float pair_w[DX_MAX_PAIRS];
};

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void cta_bar() { asm volatile("bar.sync 2, 288;" ::: "memory"); }

// TILES = 2: CTA pairs, one tile of eight block rows each (see below); only with NT = 1
// Eight 4-bit codes -> four bf16 pairs (a lane's A fragment of one contraction step).  Pair p sits in bits
// [4p, 4p+4) (first element) and [16+4p, 16+4p+4) (second): 0x4300 | code is the bf16 number 128 + code, and
// subtracting 136 leaves code - 8 exactly.
__device__ __forceinline__ uint32_t q4_pair(uint32_t w) {
  const uint32_t v = (w & 0x000F000Fu) | 0x43004300u;
  const __nv_bfloat162 r = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&v), __floats2bfloat162_rn(136.f, 136.f));
  return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ uint4 q4_fragment(uint32_t w) {
  return make_uint4(q4_pair(w), q4_pair(w >> 4), q4_pair(w >> 8), q4_pair(w >> 12));
}

// Q4: the units hold 4-bit codes with one fp16 scale per 32 weights along the contraction (see dx_pack_q4_kernel);
// the codes become bf16 fragments in registers and the scales multiply the accumulators of their block.
// SPLIT: the activations (block rows, then the SwiGLU products) enter the tensor cores as bf16 high part plus bf16
// residual, two products per fragment: results to ~1e-5 of the row maximum.  Without it they are plain bf16 (one
// rounding of at most 2^-9 relative each), which halves the tensor work -- on this part `mma.sync` is slow enough
// that the split's products take about as long as streaming the weights.
template <int H, int NT, int TILES, bool Q4 = false, bool SPLIT = true>
__global__ void __launch_bounds__(kThreads, 1) dx_experts_bf16_kernel(DxExpertParams p, int n_slots) {
  static_assert(!(Q4 && SPLIT), "4-bit units are evaluated with plain bf16 activations");
  constexpr int KW = H / 128;        // phase-1 contraction steps per consumer warp
  constexpr int PW = H / 256;        // phase-2 row-tile pairs per consumer warp
  constexpr int KSTEPS = H / 16;
  constexpr uint32_t CHUNK_A = Q4 ? KW * 144u : KW * 512u, CHUNK_D = Q4 ? PW * 192u : PW * 512u;
  constexpr uint32_t CHUNK = CHUNK_A + CHUNK_D;
  constexpr uint32_t UNIT_BYTES = 8u * CHUNK;
  constexpr bool kRegB = (NT == 1);  // token fragments live in registers (else in shared memory)

  extern __shared__ __align__(128) unsigned char smem[];
  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  constexpr size_t HDR = (sizeof(SmemHeader) + 127) / 128 * 128;
  float4* partial = reinterpret_cast<float4*>(smem + HDR);                         // [2][8][NT][32]
  constexpr size_t PART = (size_t)2 * 8 * NT * 32 * 16;
  // token fragments in shared memory if !kRegB: [NT][KSTEPS][32] of {hi, hi, lo, lo} (SPLIT) or {hi, hi}
  using FragT = typename std::conditional<SPLIT, uint4, uint2>::type;
  FragT* bfrag = reinterpret_cast<FragT*>(smem + HDR + PART);
  constexpr size_t BF = kRegB ? 0 : (size_t)NT * KSTEPS * 32 * sizeof(FragT);
  unsigned char* ring = smem + HDR + PART + BF;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const DxWork* W = p.work;
  // Blocks of more than eight rows whose second token tile does not fit next to the ring (H = 2048): the CTAs work
  // in pairs, both members stream the same share of the units (the second read of a unit comes out of L2, its
  // partner having just fetched it) and each multiplies it with one tile of eight block rows.
  constexpr int row_tiles = TILES;
  const int row_base = row_tiles == 2 ? 8 * (int)(blockIdx.x & 1) : 0;
  const int G = gridDim.x / row_tiles, cta = blockIdx.x / row_tiles;
  // groups that do not depend on routing: shared experts, then (draft mode) the draft expert
  const int n_static = p.n_shared + (p.draft_tiles > 0 ? 1 : 0);
  const int S0 = p.skip_shared ? p.n_shared * p.shared_tiles : 0;   // first routing-independent unit evaluated
  const int NS = p.do_static ? p.n_shared * p.shared_tiles + p.draft_tiles - S0 : 0;
  const int s_lo = S0 + (int)(((long long)NS * cta) / G), s_hi = S0 + (int)(((long long)NS * (cta + 1)) / G);
  volatile int* abort_flag = &hdr->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_slots; ++s) {
      mbar_init(smem_u32(&hdr->full[s]), 1);
      mbar_init(smem_u32(&hdr->empty[s]), 1);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < n_static) {
    const int i = threadIdx.x;
    const bool is_draft = i >= p.n_shared;
    hdr->e_begin[i] = is_draft ? p.n_shared * p.shared_tiles : i * p.shared_tiles;
    hdr->e_tiles[i] = is_draft ? p.draft_tiles : p.shared_tiles;
    hdr->e_blob[i] = DX_BOUNDS(i < p.table_len, p.dev_status) ? reinterpret_cast<const unsigned char*>(p.table[i]) : nullptr;
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------ producer
    uint32_t it = 0, slot = 0, phase = 0;   // chunk counter, its ring slot and that slot's phase bit
    const uint64_t l2pol = l2_evict_first_policy();
    auto issue = [&](int e0, int e1, int lo_u, int hi_u) {
      for (int e = e0; e < e1; ++e) {
        const int b = hdr->e_begin[e], nt = hdr->e_tiles[e];
        const int lo = max(b, lo_u), hi = min(b + nt, hi_u);
        const unsigned char* blob = hdr->e_blob[e];
        if (lo >= hi || blob == nullptr) continue;
        for (int u = lo; u < hi; ++u) {
          const unsigned char* src = blob + (size_t)(u - b) * UNIT_BYTES;
#pragma unroll 1
          for (int w = 0; w < kConsumerWarps; ++w, ++it) {
            // once anything has given up nothing more is copied (see mbar_wait)
            if (!mbar_wait(smem_u32(&hdr->empty[slot]), phase ^ 1u, abort_flag, p.wait_limit)) return;
            if (!DX_BOUNDS(slot < (uint32_t)n_slots && u - b >= 0 && u - b < nt, p.dev_status)) { *abort_flag = 1; return; }
            const uint32_t fb = smem_u32(&hdr->full[slot]);
            mbar_arrive_expect_tx(fb, CHUNK);
            bulk_g2s(smem_u32(ring + (size_t)slot * CHUNK), src + (size_t)w * CHUNK, CHUNK, fb, l2pol);
            if (++slot == (uint32_t)n_slots) { slot = 0; phase ^= 1u; }
          }
        }
      }
    };
    if (lane == 0) issue(0, n_static, s_lo, s_hi);
    __syncwarp();
    // The routed groups: the producer warp alone reads the work list, copies it into shared memory, signals the
    // consumers (bar.arrive: it does not wait for them, they may still be busy with their first reductions) and
    // goes straight on streaming.  With the hand-over the list is being written while this warp polls it; each
    // word says by itself when it is there.  Otherwise the routing kernel has completed once the wait returns,
    // and the first look succeeds.
    if (!p.handover) pdl_wait();
    constexpr int PER_LANE = DX_MAX_PAIRS / 32;
    unsigned long long gw[PER_LANE];
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) gw[i] = 0ull;
    int n_groups = 0, kk = 1, n_pairs = 0;
    bool have_list = false;
    for (uint32_t look = 0; look < p.wait_limit && !have_list; ++look) {
      const unsigned long long head = dx_word_load(&W->head);
      gw[0] = dx_word_load(&W->group[lane]);
      bool mine = false;
      if (head & DX_WORD_VALID) {
        n_groups = min((int)(head & 0xffffu), DX_MAX_PAIRS);
        kk = (int)((head >> 16) & 0xffu);
        n_pairs = min((int)((head >> 24) & 0xffu) * kk, DX_MAX_PAIRS);
        mine = lane >= n_groups || (gw[0] & DX_WORD_VALID);
      }
      have_list = __all_sync(0xffffffffu, mine);
    }
    // larger unions: the group words beyond the first 32
#pragma unroll
    for (int i = 1; i < PER_LANE; ++i) {
      const int idx = lane + 32 * i;
      bool mine = !have_list || idx >= n_groups;
      for (uint32_t look = 0; look < p.wait_limit; ++look) {
        if (!mine) {
          gw[i] = dx_word_load(&W->group[idx]);
          mine = (gw[i] & DX_WORD_VALID) != 0;
        }
        if (__all_sync(0xffffffffu, mine)) break;
        if (look + 1 == p.wait_limit) have_list = false;
      }
    }
    if (!have_list) {
      n_groups = 0;
      if (lane == 0) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
    }
    // groups left out by the subset mask drop out of the list here: the rest keeps its order and closes up
    int pos[PER_LANE];
    {
      int n_sel = 0;
#pragma unroll
      for (int i = 0; i < PER_LANE; ++i) {
        const int idx = lane + 32 * i, gid = dx_group_id(gw[i]);
        const bool in = idx < n_groups &&
                        (!p.use_subset || (gid < DX_MAX_E && ((p.subset[gid >> 6] >> (gid & 63)) & 1ull)));
        const unsigned int b = __ballot_sync(0xffffffffu, in);
        pos[i] = in ? n_sel + __popc(b & ((1u << lane) - 1u)) : -1;
        n_sel += __popc(b);
      }
      n_groups = n_sel;
    }
    int e_lo, e_hi, u_lo, u_hi;
    dx_routed_range(n_groups, p, n_static, NS, s_lo - S0, s_hi - S0, G, cta, e_lo, e_hi, u_lo, u_hi);
    const int unit_base = p.n_shared * p.shared_tiles + p.draft_tiles;
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) {
      const int idx = pos[i];
      if (idx >= 0) {
        const int gid = dx_group_id(gw[i]);
        const unsigned char* blob = reinterpret_cast<const unsigned char*>(dx_group_blob(gw[i]));
        // without the hand-over the table may have changed since the routing kernel ran (experts staged by the
        // cache in between): read it now
        if (!p.handover && gid < DX_MAX_E && DX_BOUNDS(p.n_shared + 1 + gid < p.table_len, p.dev_status))
          blob = reinterpret_cast<const unsigned char*>(p.table[p.n_shared + 1 + gid]);
        const int e = n_static + idx;
        if (!DX_BOUNDS(e < DX_MAX_ENTRIES, p.dev_status)) continue;
        hdr->e_begin[e] = unit_base + idx * p.routed_tiles;
        hdr->e_tiles[e] = p.routed_tiles;
        hdr->e_gid[e] = gid;
        hdr->e_blob[e] = blob;
        if (blob == nullptr && e >= e_lo && e < e_hi && !p.tolerate_missing) atomicExch(p.dev_status, DX_DEV_BAD_EXPERT_ID);
      }
    }
    if (lane == 0) {
      hdr->kk = kk;
      hdr->n_pairs = n_pairs;
      hdr->r_e_lo = e_lo; hdr->r_e_hi = e_hi; hdr->r_u_lo = u_lo; hdr->r_u_hi = u_hi;
    }
    __threadfence_block();   // bar.arrive alone does not order the shared-memory writes above
    __syncwarp();
    asm volatile("bar.arrive 2, 288;" ::: "memory");
    if (lane == 0) {
      issue(e_lo, e_hi, u_lo, u_hi);
      if (*abort_flag) {
        // something gave up: make sure no copy is still landing in this CTA's
        // shared memory before it is released (bounded, ignores the flag; the copies themselves take
        // microseconds, so this uses the library's default limit whatever the context's limit is)
        const uint32_t n_back = it < (uint32_t)n_slots ? it : (uint32_t)n_slots;
        for (uint32_t k = 1; k <= n_back; ++k) {
          const uint32_t j = it - k, s = j % (uint32_t)n_slots, ph = (j / (uint32_t)n_slots) & 1u;
          for (uint32_t spin = 0; spin < DX_WAIT_LIMIT_DEFAULT; ++spin)
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
  // register-resident token fragments: for contraction step i of this warp,
  // {hi(k0,k1), hi(k2,k3), lo(k0,k1), lo(k2,k3)} of token slot g
  uint32_t breg[kRegB ? KW : 1][4];

  // the producers are already streaming weights; the block itself may still be written by the kernel in front
  // of the routing kernel, which publishes its call number once that kernel has completed
  if (p.handover) {
    if (threadIdx.x == 0 && !flag_wait(p.handover, p.wait_limit)) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
    consumer_bar();   // one poller per CTA; the others pick the acquire up through the barrier
  } else {
    pdl_wait();
  }
  // 1/rms of every block row when the experts see RMSNorm(x) (fragments in shared memory: every warp takes rows;
  // fragments in registers: see below)
  if constexpr (!kRegB) {
    for (int r = warp; r < DX_MAX_K; r += kConsumerWarps) {
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
    consumer_bar();
  }

  // ---- token fragments: the MMA token slots are the block rows themselves, the same for every group (a group's
  // weight, zero for the rows outside it, multiplies the activations), so they are built once
  if constexpr (kRegB) {
    // one pass over the block: a lane loads exactly the values of its fragments (row g, this warp's slice of the
    // hidden dimension), the sum of squares of a row is put together from the eight warps' slices
    const int tk = row_base + g;
    const bool valid = tk < p.K;
    const float* xrow = p.x + (size_t)tk * H + 4 * c;
    float4 xv[KW];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < KW; ++i) {
      xv[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (valid) xv[i] = *reinterpret_cast<const float4*>(xrow + 16 * (warp * KW + i));
      ss += xv[i].x * xv[i].x + xv[i].y * xv[i].y + xv[i].z * xv[i].z + xv[i].w * xv[i].w;
    }
    float rs = 1.0f;
    if (p.rms_norm) {
      ss += __shfl_xor_sync(0xffffffffu, ss, 1);
      ss += __shfl_xor_sync(0xffffffffu, ss, 2);
      if (c == 0) hdr->ssq[warp][g] = ss;
      consumer_bar();
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) tot += hdr->ssq[w][g];
      rs = rsqrtf(tot / (float)H + 1e-6f);
    }
#pragma unroll
    for (int i = 0; i < KW; ++i) {
      const float4 v = xv[i];
      __nv_bfloat16 h0, h1, h2, h3, l0, l1, l2, l3;
      split_bf16(v.x * rs, h0, l0); split_bf16(v.y * rs, h1, l1);
      split_bf16(v.z * rs, h2, l2); split_bf16(v.w * rs, h3, l3);
      breg[i][0] = pack2(h0, h1); breg[i][1] = pack2(h2, h3);
      breg[i][2] = pack2(l0, l1); breg[i][3] = pack2(l2, l3);
    }
  } else {
    for (int idx = threadIdx.x; idx < NT * KSTEPS * 32; idx += kConsumerWarps * 32) {
      const int l = idx & 31, ks = (idx >> 5) % KSTEPS, nt = idx / (32 * KSTEPS);
      const int tk = nt * 8 + (l >> 2);
      uint4 o = make_uint4(0u, 0u, 0u, 0u);
      if (tk < p.K) {
        const float rs = hdr->rstd[tk];
        const float4 v = *reinterpret_cast<const float4*>(p.x + (size_t)tk * H + 16 * ks + 4 * (l & 3));
        __nv_bfloat16 h0, h1, h2, h3, l0, l1, l2, l3;
        split_bf16(v.x * rs, h0, l0); split_bf16(v.y * rs, h1, l1);
        split_bf16(v.z * rs, h2, l2); split_bf16(v.w * rs, h3, l3);
        o = make_uint4(pack2(h0, h1), pack2(h2, h3), pack2(l0, l1), pack2(l2, l3));
      }
      if constexpr (SPLIT) bfrag[idx] = o;
      else bfrag[idx] = make_uint2(o.x, o.y);
    }
    consumer_bar();
  }

  uint32_t cslot = (uint32_t)warp, cphase = 0;   // ring slot (and its phase bit) of this warp's chunk of the next unit
  int buf = 0;
  // partial-exchange source lanes: lane (g,c) ends up holding the sums of rows i = 2c and 2c+1 for token g
  const int src0 = (2 * c) * 4 + (g >> 1), src1 = src0 + 4;
  const bool odd = g & 1;

  // weight of group e's output in block row `row` (0 = the row does not belong to the group).  Token slots of
  // the MMAs are the block rows themselves, for every group alike, so the accumulators can stay in registers
  // across groups (the weight multiplies the activations) and y is touched once, at the very end.
  auto row_weight = [&](int e, int row) -> float {
    if (e < n_static) return row < p.K ? (e < p.n_shared ? 1.0f : p.gamma) : 0.0f;
    if (row >= p.K) return 0.0f;
    const int gid = hdr->e_gid[e], kk = hdr->kk;
    float w = 0.0f;
    for (int j = 0; j < kk; ++j)
      if (hdr->pair_id[row * kk + j] == gid) w = hdr->pair_w[row * kk + j];
    return w;
  };

  auto process = [&](int e0, int e1, int lo_u, int hi_u) {
    for (int e = e0; e < e1; ++e) {
      const int eb = hdr->e_begin[e], etiles = hdr->e_tiles[e];
      const int lo = max(eb, lo_u), hi = min(eb + etiles, hi_u);
      if (lo >= hi || hdr->e_blob[e] == nullptr) continue;
      // this lane's block rows (one per token tile) and their weights in this group
      float wrow[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) wrow[nt] = row_weight(e, row_base + nt * 8 + g);
      const bool need_hi = NT > 1 && __any_sync(0xffffffffu, wrow[NT - 1] != 0.0f);   // any of rows 8..15 routed here

      for (int u = lo; u < hi; ++u) {
        uint32_t s = cslot;
        const uint32_t ph = cphase;
        cslot += kConsumerWarps;   // (a ring has more slots than a unit has chunks: at most one wrap)
        if (cslot >= (uint32_t)n_slots) { cslot -= (uint32_t)n_slots; cphase ^= 1u; }
        // (a slot out of range is reported and replaced: every warp has to keep taking part in the barriers below)
        if (!DX_BOUNDS(s < (uint32_t)n_slots, p.dev_status)) { *abort_flag = 1; s = 0; }
        const uint4* A = reinterpret_cast<const uint4*>(ring + (size_t)s * CHUNK) + lane;
        mbar_wait(smem_u32(&hdr->full[s]), ph, abort_flag, p.wait_limit);

        // ---- phase 1: [8 gate rows ; 8 up rows] x tokens over this warp's slice of the contraction
        float ch[NT][2][4], cl[NT][2][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int r = 0; r < 4; ++r) ch[nt][0][r] = ch[nt][1][r] = cl[nt][0][r] = cl[nt][1][r] = 0.f;
        if constexpr (Q4) {
          // one 32-wide quantisation block = two contraction steps: codes -> exact bf16 fragments, the products of
          // the block go to fresh accumulators, and the rows' scales (gate row g, up row g) are applied to those
          const unsigned char* Cq = ring + (size_t)s * CHUNK;
          const uint2* Aq = reinterpret_cast<const uint2*>(Cq) + lane;
          const __half2* S1 = reinterpret_cast<const __half2*>(Cq + KW * 128) + g;
#pragma unroll
          for (int b = 0; b < KW / 2; ++b) {
            const uint2 cw = Aq[b * 32];
            const float2 sc = __half22float2(S1[b * 8]);
            const uint4 a0 = q4_fragment(cw.x), a1 = q4_fragment(cw.y);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              if (nt > 0 && !need_hi) continue;
              uint32_t b00, b01, b02, b03, b10, b11, b12, b13;
              if constexpr (kRegB) {
                b00 = breg[2 * b][0]; b01 = breg[2 * b][1]; b02 = breg[2 * b][2]; b03 = breg[2 * b][3];
                b10 = breg[2 * b + 1][0]; b11 = breg[2 * b + 1][1]; b12 = breg[2 * b + 1][2]; b13 = breg[2 * b + 1][3];
              } else {
                const FragT f0 = bfrag[(nt * KSTEPS + warp * KW + 2 * b) * 32 + lane];
                const FragT f1 = bfrag[(nt * KSTEPS + warp * KW + 2 * b + 1) * 32 + lane];
                b00 = f0.x; b01 = f0.y; b02 = 0u; b03 = 0u;
                b10 = f1.x; b11 = f1.y; b12 = 0u; b13 = 0u;
              }
              // (activations in bf16 without the low halves: with 4-bit weights the tensor pipe, not the stream,
              // sets the pace, and the rounding is far below the quantisation's own error)
              (void)b02; (void)b03; (void)b12; (void)b13;
              float t0[4] = {0.f, 0.f, 0.f, 0.f}, t1[4] = {0.f, 0.f, 0.f, 0.f};
              mma_k16(t0, a0, b00, b01);
              mma_k16(t1, a1, b10, b11);
              ch[nt][0][0] = fmaf(sc.x, t0[0] + t1[0], ch[nt][0][0]); ch[nt][0][1] = fmaf(sc.x, t0[1] + t1[1], ch[nt][0][1]);
              ch[nt][0][2] = fmaf(sc.y, t0[2] + t1[2], ch[nt][0][2]); ch[nt][0][3] = fmaf(sc.y, t0[3] + t1[3], ch[nt][0][3]);
            }
          }
        } else {
#pragma unroll
        for (int i = 0; i < KW; ++i) {
          const uint4 a = A[i * 32];
          if constexpr (kRegB) {
            mma_k16(ch[0][i & 1], a, breg[i][0], breg[i][1]);
            if constexpr (SPLIT) mma_k16(cl[0][i & 1], a, breg[i][2], breg[i][3]);
          } else {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              if (nt > 0 && !need_hi) continue;
              const FragT b = bfrag[(nt * KSTEPS + warp * KW + i) * 32 + lane];
              mma_k16(ch[nt][i & 1], a, b.x, b.y);
              if constexpr (SPLIT) mma_k16(cl[nt][i & 1], a, b.z, b.w);
            }
          }
        }
        }
        // re-fragment: C holds (gate|up row g, tokens 2c,2c+1); phase 2 wants rows (2c,2c+1) of token g
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float v[4];
#pragma unroll
          for (int r = 0; r < 4; ++r) v[r] = (ch[nt][0][r] + ch[nt][1][r]) + (cl[nt][0][r] + cl[nt][1][r]);
          const float a0 = __shfl_sync(0xffffffffu, v[0], src0), a1 = __shfl_sync(0xffffffffu, v[1], src0);
          const float a2 = __shfl_sync(0xffffffffu, v[2], src0), a3 = __shfl_sync(0xffffffffu, v[3], src0);
          const float b0 = __shfl_sync(0xffffffffu, v[0], src1), b1 = __shfl_sync(0xffffffffu, v[1], src1);
          const float b2 = __shfl_sync(0xffffffffu, v[2], src1), b3 = __shfl_sync(0xffffffffu, v[3], src1);
          partial[((buf * 8 + warp) * NT + nt) * 32 + lane] =
              make_float4(odd ? a1 : a0, odd ? a3 : a2, odd ? b1 : b0, odd ? b3 : b2);
        }
        consumer_bar();

        // ---- sum the eight slices, activation, phase-2 token fragment
        uint32_t bhi[NT], blo[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float4 q[8];
#pragma unroll
          for (int w = 0; w < 8; ++w) q[w] = partial[((buf * 8 + w) * NT + nt) * 32 + lane];
#pragma unroll
          for (int st = 1; st < 8; st <<= 1)
#pragma unroll
            for (int w = 0; w < 8; w += 2 * st) {
              q[w].x += q[w + st].x; q[w].y += q[w + st].y; q[w].z += q[w + st].z; q[w].w += q[w + st].w;
            }
          const float4 t = q[0];
          const float a0 = fast_silu(t.x) * t.y * wrow[nt], a1 = fast_silu(t.z) * t.w * wrow[nt];
          __nv_bfloat16 h0, l0, h1, l1;
          split_bf16(a0, h0, l0);
          split_bf16(a1, h1, l1);
          bhi[nt] = pack2(h0, h1);
          blo[nt] = pack2(l0, l1);
        }
        buf ^= 1;

        // ---- phase 2: 8 columns of W_d x activations for this warp's output rows
        if constexpr (Q4) {
          // the eight columns of a unit lie in one quantisation block of W_d: one scale per output row
          const unsigned char* Cq = ring + (size_t)s * CHUNK + CHUNK_A;
          const uint32_t* Dq = reinterpret_cast<const uint32_t*>(Cq) + lane;
          const uint2* S2 = reinterpret_cast<const uint2*>(Cq + PW * 128) + g;
#pragma unroll
          for (int q = 0; q < PW; ++q) {
            const uint4 a = q4_fragment(Dq[q * 32]);
            const uint2 sw = S2[q * 8];
            const float2 s01 = __half22float2(*reinterpret_cast<const __half2*>(&sw.x));   // tile 2q: rows g, g + 8
            const float2 s23 = __half22float2(*reinterpret_cast<const __half2*>(&sw.y));   // tile 2q + 1
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              if (nt > 0 && !need_hi) continue;
              float t0[4] = {0.f, 0.f, 0.f, 0.f}, t1[4] = {0.f, 0.f, 0.f, 0.f};
              mma_k8(t0, a.x, a.y, bhi[nt]);
              mma_k8(t1, a.z, a.w, bhi[nt]);
              acc[nt][2 * q][0] = fmaf(s01.x, t0[0], acc[nt][2 * q][0]);
              acc[nt][2 * q][1] = fmaf(s01.x, t0[1], acc[nt][2 * q][1]);
              acc[nt][2 * q][2] = fmaf(s01.y, t0[2], acc[nt][2 * q][2]);
              acc[nt][2 * q][3] = fmaf(s01.y, t0[3], acc[nt][2 * q][3]);
              acc[nt][2 * q + 1][0] = fmaf(s23.x, t1[0], acc[nt][2 * q + 1][0]);
              acc[nt][2 * q + 1][1] = fmaf(s23.x, t1[1], acc[nt][2 * q + 1][1]);
              acc[nt][2 * q + 1][2] = fmaf(s23.y, t1[2], acc[nt][2 * q + 1][2]);
              acc[nt][2 * q + 1][3] = fmaf(s23.y, t1[3], acc[nt][2 * q + 1][3]);
            }
          }
        } else {
        const uint4* D = A + KW * 32;
#pragma unroll
        for (int q = 0; q < PW; ++q) {
          const uint4 a = D[q * 32];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            if (nt > 0 && !need_hi) continue;
            mma_k8(acc[nt][2 * q], a.x, a.y, bhi[nt]);
            mma_k8(acc[nt][2 * q + 1], a.z, a.w, bhi[nt]);
            if constexpr (SPLIT) {
              mma_k8(acc[nt][2 * q], a.x, a.y, blo[nt]);
              mma_k8(acc[nt][2 * q + 1], a.z, a.w, blo[nt]);
            }
          }
        }
        }
        __syncwarp();
        if (lane == 0 && !*abort_flag) mbar_arrive(smem_u32(&hdr->empty[s]));   // (no slot is released after a give-up)
      }

    }
  };

  process(0, n_static, s_lo, s_hi);
  cta_bar();   // the producer warp has seen the routing call's work list and published its routed part
  // The (row, expert, gate) pairs come out of the gate arithmetic a little after the group list.  Every warp
  // fetches all of them for itself (same values from every warp, so no barrier is needed to use them).
  {
    const int n_pairs = hdr->n_pairs;
    bool ok = true;
    for (int idx = lane; idx < n_pairs; idx += 32) {
      unsigned long long w = 0ull;
      uint32_t look = 0;
      for (; look < p.wait_limit; ++look) {
        w = dx_word_load(&W->pair[idx]);
        if (w & DX_WORD_VALID) break;
      }
      ok = ok && look < p.wait_limit;
      if (!DX_BOUNDS(idx < DX_MAX_PAIRS, p.dev_status)) continue;
      hdr->pair_id[idx] = dx_pair_id(w);
      hdr->pair_w[idx] = dx_pair_weight(w);
    }
    if (!ok) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
    __syncwarp();
  }
  // Only now may the next kernel of the stream start: if it is a routing kernel it clears the hand-over words
  // (flag, group list, pairs) before its own wait, so every warp of this CTA has to be done with all of them.  (The
  // trigger used to sit in front of the pair fetch: a routing kernel that started in that window wiped pairs that
  // were still being polled -- rare, and seen as an expired wait on blocks of eight rows, whose gate arithmetic
  // takes longest.)
  consumer_bar();
  pdl_launch_dependents();
  process(hdr->r_e_lo, hdr->r_e_hi, hdr->r_u_lo, hdr->r_u_hi);
  pdl_wait();  // the routing kernel (which initialised y) has completed as a whole

  // ---- the CTA's partial output rows go to y (initialised by the routing kernel, which has completed).
  // A lane holds, per 16-row tile, rows g and g + 8 of block rows 2c and 2c + 1.  The four lanes g = 4q .. 4q+3 of a
  // column pair transpose their 4 x 4 values (two butterfly steps over lane bits 2 and 3), after which lane i of
  // the four holds four consecutive output rows of ONE (block row, half): one 16-byte reduction instead of four.
  {
    const int gi = g & 3;                       // this lane's place among the four, and the combination it ends up with:
    const int tok = 2 * c + (gi & 1);           //   block row 2c or 2c + 1 ...
    const int half = gi >> 1;                   //   ... rows g or g + 8 of the tile
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int row = row_base + nt * 8 + tok;
      float* yrow = p.y + (size_t)row * H + (g >> 2) * 4 + half * 8;
#pragma unroll
      for (int j = 0; j < 2 * PW; ++j) {
        // combination k of a lane: k = 0: (2c, g), 1: (2c+1, g), 2: (2c, g+8), 3: (2c+1, g+8)
        float v0 = acc[nt][j][0], v1 = acc[nt][j][1], v2 = acc[nt][j][2], v3 = acc[nt][j][3];
        // step 1 (partner differs in bit 0 of gi): keep combinations with my bit 0, get the partner's
        {
          const bool hi = gi & 1;
          const float s0 = hi ? v0 : v1, s1 = hi ? v2 : v3;          // what the partner wants from me
          const float r0 = __shfl_xor_sync(0xffffffffu, s0, 4), r1 = __shfl_xor_sync(0xffffffffu, s1, 4);
          if (hi) { v0 = r0; v2 = r1; } else { v1 = r0; v3 = r1; }
          // now (v0, v1) = combination (gi & 1) of lanes {gi & ~1, gi | 1}, rows g-pair order; (v2, v3) likewise + 2
        }
        // step 2 (partner differs in bit 1 of gi)
        {
          const bool hi = gi & 2;
          const float s0 = hi ? v0 : v2, s1 = hi ? v1 : v3;
          const float r0 = __shfl_xor_sync(0xffffffffu, s0, 8), r1 = __shfl_xor_sync(0xffffffffu, s1, 8);
          if (hi) { v0 = r0; v1 = r1; } else { v2 = r0; v3 = r1; }
        }
        // (v0, v1, v2, v3) = this lane's combination at rows 4q, 4q+1, 4q+2, 4q+3 of the tile's half
        if (row < p.K && DX_BOUNDS((g >> 2) * 4 + half * 8 + (warp * 2 * PW + j) * 16 + 3 < H, p.dev_status)) {
          float* dst = yrow + (warp * 2 * PW + j) * 16;
          asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                       :: "l"(dst), "f"(v0), "f"(v1), "f"(v2), "f"(v3) : "memory");
        }
      }
    }
  }
  if (*abort_flag && threadIdx.x == 0) atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------- fp32 path
// Plain CUDA-core version for fp32 weights (small layers): one CTA per unit,
// warp w owns gate/up row w, then every thread owns output columns.
__global__ void __launch_bounds__(256) dx_experts_fp32_kernel(DxExpertParams p) {
  __shared__ float s_act[DX_MAX_K][DX_TILE_I];
  __shared__ float s_rstd[DX_MAX_K];
  const DxWork* W = p.work;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // (no early trigger: the kernel reads the work list until its last unit, and a routing kernel that follows may
  // clear the list as soon as it starts)
  dx_pdl_wait();
  const unsigned long long head = W->head;
  const int n_groups = min((int)(head & 0xffffu), DX_MAX_PAIRS), kk = (int)((head >> 16) & 0xffu), H = p.H;
  for (int r = warp; r < DX_MAX_K; r += 8) {
    float rs = 1.0f;
    if (p.rms_norm && r < p.K) {
      float ss = 0.f;
      for (int j = lane; j < H; j += 32) { const float v = p.x[(size_t)r * H + j]; ss += v * v; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      rs = rsqrtf(ss / (float)H + 1e-6f);
    }
    if (lane == 0) s_rstd[r] = rs;
  }
  __syncthreads();
  // window of the routed groups covered by this launch (see routed_range) and the routing-independent units
  const int NS_all = p.n_shared * p.shared_tiles + p.draft_tiles;
  const int g_lo = min(n_groups, p.first_routed);
  const int g_hi = p.n_routed < 0 ? n_groups : min(n_groups, g_lo + p.n_routed);
  const int wu_lo = NS_all + g_lo * p.routed_tiles, wu_hi = NS_all + g_hi * p.routed_tiles;
  const int total = NS_all + n_groups * p.routed_tiles;
  __shared__ float s_roww[DX_MAX_K];
  for (int u = blockIdx.x; u < total; u += gridDim.x) {
    if (u < NS_all ? (!p.do_static || (p.skip_shared && u < p.n_shared * p.shared_tiles)) : (u < wu_lo || u >= wu_hi))
      continue;
    // the group of this unit, its blob and its weight in every block row (0 = the row is not in the group)
    int table_index, unit_begin, gid = -1;
    float w_static = 1.0f;
    if (u < p.n_shared * p.shared_tiles) {
      table_index = u / p.shared_tiles;
      unit_begin = table_index * p.shared_tiles;
    } else if (u < NS_all) {
      table_index = p.n_shared;
      unit_begin = p.n_shared * p.shared_tiles;
      w_static = p.gamma;
    } else {
      const int gi = (u - NS_all) / p.routed_tiles;
      gid = dx_group_id(W->group[gi]);
      if (p.use_subset && !(gid < DX_MAX_E && ((p.subset[gid >> 6] >> (gid & 63)) & 1ull))) continue;
      table_index = p.n_shared + 1 + gid;
      unit_begin = NS_all + gi * p.routed_tiles;
    }
    if (threadIdx.x < DX_MAX_K) {
      const int row = threadIdx.x;
      float w = 0.0f;
      if (row < p.K) {
        if (gid < 0) w = w_static;
        else
          for (int j = 0; j < kk; ++j)
            if (dx_pair_id(W->pair[row * kk + j]) == gid) w = dx_pair_weight(W->pair[row * kk + j]);
      }
      s_roww[row] = w;
    }
    __syncthreads();
    const float* blob = DX_BOUNDS(table_index >= 0 && table_index < p.table_len, p.dev_status)
                            ? reinterpret_cast<const float*>(p.table[table_index]) : nullptr;
    if (blob == nullptr) {
      if (threadIdx.x == 0) atomicExch(p.dev_status, DX_DEV_BAD_EXPERT_ID);
      __syncthreads();
      continue;
    }
    const float* unit = blob + (size_t)(u - unit_begin) * 24 * H;
    const float* gr = unit + (size_t)warp * H;
    const float* ur = unit + (size_t)(8 + warp) * H;
    for (int t = 0; t < p.K; ++t) {
      if (s_roww[t] == 0.0f) continue;
      const float* x = p.x + (size_t)t * H;
      const float rs = s_rstd[t];
      float ag = 0.f, au = 0.f;
      for (int j = lane; j < H; j += 32) {
        const float xv = x[j] * rs;
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
      for (int t = 0; t < p.K; ++t) {
        if (s_roww[t] == 0.0f) continue;
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) s = fmaf(s_act[t][i], d[i], s);
        atomicAdd(p.y + (size_t)t * H + hh, s_roww[t] * s);
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------ pack kernels
// bf16 blob, unit j (24*H elements) = 8 chunks of 3*H elements; chunk w:
//   gate/up part (2*H): step i < H/128, contraction step s = w*H/128 + i, lane l=(g,c): 8 elements
//       { Wg[8j+g][16s+4c+0..1], Wu[8j+g][16s+4c+0..1], Wg[8j+g][16s+4c+2..3], Wu[8j+g][16s+4c+2..3] }
//   down part (H): pair i < H/256, row-tile pair q = w*H/256 + i, lane l=(g,c): 8 elements
//       { Wd[32q+g][8j+2c..+1], Wd[32q+8+g][..], Wd[32q+16+g][..], Wd[32q+24+g][..] }
__global__ void dx_pack_bf16_kernel(const __nv_bfloat16* Wg, const __nv_bfloat16* Wu, const __nv_bfloat16* Wd,
                                    __nv_bfloat16* blob, int H, int I) {
  const size_t n = (size_t)3 * H * I;
  const int KW = H / 128, PW = H / 256;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(idx / (24 * (size_t)H));
    const int r = (int)(idx % (24 * (size_t)H));
    const int w = r / (3 * H), rr = r % (3 * H);
    __nv_bfloat16 v;
    if (rr < 2 * H) {
      const int i = rr / 256, l = (rr % 256) / 8, el = rr % 8;
      const int s = w * KW + i, g = l >> 2, c = l & 3;
      const int col = 16 * s + 4 * c + (el & 1) + ((el >> 2) << 1);
      const int row = 8 * j + g;
      v = ((el >> 1) & 1) ? Wu[(size_t)row * H + col] : Wg[(size_t)row * H + col];
    } else {
      const int r2 = rr - 2 * H;
      const int i = r2 / 256, l = (r2 % 256) / 8, el = r2 % 8;
      const int q = w * PW + i, g = l >> 2, c = l & 3;
      const int row = 32 * q + 8 * (el >> 1) + g;
      const int col = 8 * j + 2 * c + (el & 1);
      v = Wd[(size_t)row * I + col];
    }
    blob[idx] = v;
  }
}

// 4-bit block-quantised expert (three matrices of 18-byte blocks: fp16 scale, then 16 bytes of codes, low nibbles
// = weights 0..15 of the block, high nibbles = weights 16..31; weight = scale * (code - 8)) expanded straight
// into the bf16 streaming blob above, each value rounded to bf16 once.

// One thread writes one 16-byte fragment (eight values): the expansion sits between a host -> device copy and the
// first use of a cache slot, once per loaded expert, and an element-by-element version (index arithmetic and three
// byte loads per value) took as long as the copy itself.
//   first product: the fragment of lane (g, c), step s holds columns 16 s + 4 c .. + 3 of gate row 8 j + g and of up
//   row 8 j + g, as (g0 g1 u0 u1 g2 g3 u2 u3): four consecutive codes of one quantisation block per matrix;
//   second product: rows 32 q + g, + 8, + 16, + 24 of W_d at columns 8 j + 2 c, + 1: two consecutive codes of four
//   blocks.
__device__ __forceinline__ float q4_scale(const unsigned char* blk) {
  return __half2float(__ushort_as_half(*reinterpret_cast<const unsigned short*>(blk)));   // (blocks are 18 bytes: 2-byte aligned)
}
__device__ __forceinline__ uint32_t bf16_pair(float lo, float hi) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
}
__global__ void dx_expand_q4_kernel(const unsigned char* q4, __nv_bfloat16* blob, int H, int I) {
  const int KW = H / 128, PW = H / 256;
  const size_t mat_gu = (size_t)I * (H / 32) * 18;   // bytes of W_g (and of W_u)
  const unsigned char* Wg = q4;
  const unsigned char* Wu = q4 + mat_gu;
  const unsigned char* Wd = q4 + 2 * mat_gu;
  const int per_unit = 3 * H, per_chunk = 3 * H / 8, p1 = H / 4;   // 16-byte fragments per unit / per chunk / of the first product
  const size_t n = (size_t)(I / 8) * per_unit;
  uint4* out = reinterpret_cast<uint4*>(blob);
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(idx / per_unit);
    const int u4 = (int)(idx - (size_t)j * per_unit);
    const int w = u4 / per_chunk, r4 = u4 - w * per_chunk;
    uint4 v;
    if (r4 < p1) {
      const int i = r4 >> 5, l = r4 & 31, g = l >> 2, c = l & 3;
      const int col0 = 16 * (w * KW + i) + 4 * c, row = 8 * j + g;
      const size_t off = ((size_t)row * (H / 32) + col0 / 32) * 18;
      const int jj = col0 & 31, sh = (jj & 16) ? 4 : 0;
      float gv[4], uv[4];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        const unsigned char* blk = (m ? Wu : Wg) + off;
        const float d = q4_scale(blk);
        // four consecutive code bytes, 2-byte aligned
        const unsigned short b01 = *reinterpret_cast<const unsigned short*>(blk + 2 + (jj & 15));
        const unsigned short b23 = *reinterpret_cast<const unsigned short*>(blk + 4 + (jj & 15));
        float* dst = m ? uv : gv;
        dst[0] = d * (float)((int)((b01 >> sh) & 0xF) - 8);
        dst[1] = d * (float)((int)((b01 >> (8 + sh)) & 0xF) - 8);
        dst[2] = d * (float)((int)((b23 >> sh) & 0xF) - 8);
        dst[3] = d * (float)((int)((b23 >> (8 + sh)) & 0xF) - 8);
      }
      v = make_uint4(bf16_pair(gv[0], gv[1]), bf16_pair(uv[0], uv[1]), bf16_pair(gv[2], gv[3]), bf16_pair(uv[2], uv[3]));
    } else {
      const int r2 = r4 - p1;
      const int i = r2 >> 5, l = r2 & 31, g = l >> 2, c = l & 3;
      const int q = w * PW + i, col = 8 * j + 2 * c;
      const int jj = col & 31, sh = (jj & 16) ? 4 : 0;
      uint32_t o[4];
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        const int row = 32 * q + 8 * m + g;
        const unsigned char* blk = Wd + ((size_t)row * (I / 32) + col / 32) * 18;
        const float d = q4_scale(blk);
        const unsigned short b01 = *reinterpret_cast<const unsigned short*>(blk + 2 + (jj & 15));
        o[m] = bf16_pair(d * (float)((int)((b01 >> sh) & 0xF) - 8), d * (float)((int)((b01 >> (8 + sh)) & 0xF) - 8));
      }
      v = make_uint4(o[0], o[1], o[2], o[3]);
    }
    out[idx] = v;
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

template <int H, int NT, int TILES, bool Q4, bool SPLIT>
cudaError_t launch_bf16(dx_ctx* ctx, const DxExpertParams& p, cudaStream_t st) {
  const size_t hdr = (sizeof(SmemHeader) + 127) / 128 * 128;
  const size_t fixed = hdr + (size_t)2 * 8 * NT * 32 * 16 + (NT == 1 ? 0 : (size_t)NT * (H / 16) * 32 * (SPLIT ? 16 : 8));
  const size_t chunk = dx_chunk_bytes(H, Q4);
  int n_slots = (int)(((size_t)ctx->smem_optin - fixed) / chunk);
  if (n_slots > kMaxSlots) n_slots = kMaxSlots;
  if (n_slots < kConsumerWarps + 1) return cudaErrorInvalidConfiguration;   // a unit needs all its chunks at once
  const size_t smem = fixed + (size_t)n_slots * chunk;
  cudaError_t e = cudaFuncSetAttribute(dx_experts_bf16_kernel<H, NT, TILES, Q4, SPLIT>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // One CTA per SM, minus the SMs the routing cluster runs on at the same time: a CTA of this kernel
  // fills an SM, so a CTA that had to wait for a routing CTA's SM would start late and become the tail.
  int grid = ctx->sm_count > 16 ? ctx->sm_count - DX_ROUTE_CLUSTER : ctx->sm_count;
  if (TILES == 2) grid &= ~1;
  return dx_launch_pdl((ctx->pdl_mask & DX_PDL_EXPERTS) != 0, dx_experts_bf16_kernel<H, NT, TILES, Q4, SPLIT>, dim3(grid), dim3(kThreads), smem, st, 1,
                       p, n_slots);
}

template <int H, bool Q4, bool SPLIT>
cudaError_t launch_bf16_h(dx_ctx* ctx, const DxExpertParams& p_in, int K, cudaStream_t st) {
  DxExpertParams p = p_in;
  p.row_tiles = 1;
  if (K <= 8) return launch_bf16<H, 1, 1, Q4, SPLIT>(ctx, p, st);
  // two token tiles: fragments of both in shared memory where they fit next to a ring of at least one slot per
  // consumer warp and one to spare; otherwise CTA pairs with one tile each
  const size_t hdr = (sizeof(SmemHeader) + 127) / 128 * 128;
  const size_t fixed2 = hdr + (size_t)2 * 8 * 2 * 32 * 16 + (size_t)2 * (H / 16) * 32 * (SPLIT ? 16 : 8);
  if (fixed2 + (size_t)(kConsumerWarps + 1) * dx_chunk_bytes(H, Q4) <= (size_t)ctx->smem_optin)
    return launch_bf16<H, 2, 1, Q4, SPLIT>(ctx, p, st);
  p.row_tiles = 2;
  return launch_bf16<H, 1, 2, Q4, SPLIT>(ctx, p, st);
}

template <bool Q4, bool SPLIT>
cudaError_t launch_bf16_any(dx_ctx* ctx, const DxExpertParams& p, int K, cudaStream_t st) {
  switch (p.H) {
    case 256: return launch_bf16_h<256, Q4, SPLIT>(ctx, p, K, st);
    case 512: return launch_bf16_h<512, Q4, SPLIT>(ctx, p, K, st);
    case 1024: return launch_bf16_h<1024, Q4, SPLIT>(ctx, p, K, st);
    case 2048: return launch_bf16_h<2048, Q4, SPLIT>(ctx, p, K, st);
    default: return cudaErrorInvalidConfiguration;
  }
}

// Packed 4-bit units from the three matrices' Q4_0 blocks (18 bytes: fp16 scale d, then 16 bytes whose low /
// high nibbles are elements j / j + 16 of the block; value = d * (code - 8)).  One unit = the chunks of the eight
// consumer warps; a chunk holds, for warp w of unit j,
//   [KW/2][32 lanes] 8 bytes: the code words of contraction steps 2b and 2b+1 of the lane's gate / up fragment,
//   [KW/2][8 rows g] 2 halves: scales of gate row 8j+g and up row 8j+g in hidden block (w KW + 2b) / 2,
//   [PW][32 lanes]   4 bytes: the code word of the lane's W_d fragment for row-tile pair w PW + i,
//   [PW][8 rows g]   4 halves: scales of output rows 32q+g, +8, +16, +24 in intermediate block j / 4.
// A code word holds a fragment's four bf16 pairs as (first, second) = bits [4p, 4p+4), [16+4p, 16+4p+4).
__device__ __forceinline__ uint32_t q4_code(const unsigned char* m, int row, int col, int ncols) {
  const unsigned char* blk = m + ((size_t)row * (ncols / 32) + col / 32) * 18;
  const int j = col & 31;
  return j < 16 ? (blk[2 + j] & 0x0Fu) : (uint32_t)(blk[2 + j - 16] >> 4);
}
__device__ __forceinline__ unsigned short q4_scale_bits(const unsigned char* m, int row, int col, int ncols) {
  const unsigned char* blk = m + ((size_t)row * (ncols / 32) + col / 32) * 18;
  return (unsigned short)(blk[0] | (blk[1] << 8));
}

__global__ void dx_pack_q4_kernel(const unsigned char* Wg, const unsigned char* Wu, const unsigned char* Wd,
                                  unsigned char* blob, int H, int I) {
  const int KW = H / 128, PW = H / 256;
  const size_t chunk = (size_t)KW * 144 + (size_t)PW * 192, unit = 8 * chunk;
  const int per_chunk = KW * 32 + KW * 8 + PW * 32 + PW * 32;   // code words and scales of phase 1, then of phase 2
  const size_t n = (size_t)(I / 8) * 8 * per_chunk;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(idx / ((size_t)8 * per_chunk));
    const int r = (int)(idx % ((size_t)8 * per_chunk));
    const int w = r / per_chunk;
    int t = r % per_chunk;
    unsigned char* out = blob + (size_t)j * unit + (size_t)w * chunk;
    if (t < KW * 32) {                       // phase-1 code word of contraction step i, lane l
      const int i = t / 32, l = t % 32, g = l >> 2, c = l & 3;
      const int col = 16 * (w * KW + i) + 4 * c, row = 8 * j + g;
      uint32_t word = 0;
      // pairs: (gate col, col+1), (up col, col+1), (gate col+2, col+3), (up col+2, col+3)
#pragma unroll
      for (int pp = 0; pp < 4; ++pp) {
        const unsigned char* m = (pp & 1) ? Wu : Wg;
        const int cc = col + 2 * (pp >> 1);
        word |= q4_code(m, row, cc, H) << (4 * pp);
        word |= q4_code(m, row, cc + 1, H) << (16 + 4 * pp);
      }
      *reinterpret_cast<uint32_t*>(out + (size_t)(i / 2) * 256 + l * 8 + (i & 1) * 4) = word;
      continue;
    }
    t -= KW * 32;
    if (t < KW * 8) {                        // phase-1 scales of block pair b, row g, gate | up
      const int b = t / 16, g = (t % 16) / 2, which = t & 1;
      const int col = 16 * (w * KW + 2 * b);
      *reinterpret_cast<unsigned short*>(out + (size_t)KW * 128 + b * 32 + g * 4 + which * 2) =
          q4_scale_bits(which ? Wu : Wg, 8 * j + g, col, H);
      continue;
    }
    t -= KW * 8;
    if (t < PW * 32) {                       // phase-2 code word of row-tile pair i, lane l
      const int i = t / 32, l = t % 32, g = l >> 2, c = l & 3;
      const int q = w * PW + i, col = 8 * j + 2 * c;
      uint32_t word = 0;
#pragma unroll
      for (int pp = 0; pp < 4; ++pp) {
        const int row = 32 * q + 8 * pp + g;
        word |= q4_code(Wd, row, col, I) << (4 * pp);
        word |= q4_code(Wd, row, col + 1, I) << (16 + 4 * pp);
      }
      *reinterpret_cast<uint32_t*>(out + (size_t)KW * 144 + (size_t)i * 128 + l * 4) = word;
      continue;
    }
    t -= PW * 32;
    {                                        // phase-2 scales of row-tile pair i, row g, the four rows g + 8m
      const int i = t / 32, g = (t % 32) / 4, m = t & 3;
      const int q = w * PW + i;
      *reinterpret_cast<unsigned short*>(out + (size_t)KW * 144 + (size_t)PW * 128 + (size_t)i * 64 + g * 8 + m * 2) =
          q4_scale_bits(Wd, 32 * q + 8 * m + g, 8 * j, I);
    }
  }
}

}  // namespace

bool dx_bf16_hidden_supported(int H) { return H == 256 || H == 512 || H == 1024 || H == 2048; }

cudaError_t dx_launch_experts(dx_ctx* ctx, const DxExpertParams& p, int weight_dtype, int K, cudaStream_t st) {
  if (weight_dtype == DX_DTYPE_FP32) {
    return dx_launch_pdl((ctx->pdl_mask & DX_PDL_EXPERTS) != 0, dx_experts_fp32_kernel, dim3(ctx->sm_count * 4), dim3(256), 0, st, 1, p);
  }
  if (weight_dtype == DX_DTYPE_BF16_WIDE) return dx_launch_experts_wide(ctx, p, st);
  if (weight_dtype == DX_DTYPE_Q4) return launch_bf16_any<true, false>(ctx, p, K, st);
  return ctx->act_split ? launch_bf16_any<false, true>(ctx, p, K, st) : launch_bf16_any<false, false>(ctx, p, K, st);
}

cudaError_t dx_launch_pack_q4(int H, int I, const void* Wg, const void* Wu, const void* Wd, void* blob,
                              cudaStream_t st) {
  const size_t n = (size_t)I * ((size_t)(H / 128) * 40 + (size_t)(H / 256) * 64);
  int grid = (int)((n + 255) / 256);
  if (grid > 4096) grid = 4096;
  dx_pack_q4_kernel<<<grid, 256, 0, st>>>((const unsigned char*)Wg, (const unsigned char*)Wu, (const unsigned char*)Wd,
                                          (unsigned char*)blob, H, I);
  return cudaGetLastError();
}

cudaError_t dx_launch_expand_q4(int H, int I, const void* q4, void* blob, cudaStream_t st) {
  const size_t n = (size_t)3 * H * I / 8;   // 16-byte fragments
  int grid = (int)((n + 255) / 256);
  if (grid > 8192) grid = 8192;
  dx_expand_q4_kernel<<<grid, 256, 0, st>>>((const unsigned char*)q4, (__nv_bfloat16*)blob, H, I);
  return cudaGetLastError();
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
