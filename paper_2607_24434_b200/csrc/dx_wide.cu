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
// In either region the part of one unit in one stage is 2 KB of contiguous bytes, and the parts of consecutive units
// of an MU follow one another.
//
// Pieces.  The products cost the same whether a tile of 128 rows is full or not, so the CTA packs its units -- any
// units, of any experts -- eight at a time into "pieces": unit slot j of a piece is row groups 2 j, 2 j + 1 of the
// first product and contraction chunk j of the second (both operands of the block are the same for every expert; an
// expert's weight in a block row is folded into the activations).  A shared-memory stage is 16 KB = 8 unit slots of
// 2 KB; a run of consecutive units of one MU is one bulk copy per stage.
//
// Per piece: D1[128 x 16] = [gate rows; up rows] x block rows^T over H (accumulated in tensor memory over the
// H/64 stages), the epilogue warps read D1, form w * silu(g) * u in bf16 as the next operand in shared memory, and
// D2[T][128 x 16] += W_d tile x that, for every tile T of 128 output rows; D2 (H/128 tiles x 16 columns) stays in
// tensor memory across all pieces of the CTA and is added to y once, at the end.  Unit slots a piece does not use
// hold older weights or zeros (the ring is cleared once): their products are finite and meet zero activations.
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
constexpr int kMaxPieces = 40;
constexpr int kMaxRuns = 72;

struct WideHeader {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long d1_full[2];
  unsigned long long act_ready[2];
  unsigned long long d2_full;
  unsigned long long list_ready;   // the groups, pairs and pieces below are written
  unsigned long long static_ready; // (hand-over) the pieces of the routing-independent groups are written
  unsigned long long x_ready[4];   // quarters of the block-row operand, in the order the first product needs them
  uint32_t tmem_base;
  int abort_flag;
  int ph_e_lo[2], ph_e_hi[2], ph_u_lo[2], ph_u_hi[2];   // routing-independent groups, then routed groups
  int kk, n_pairs;
  float rstd[DX_MAX_K];
  int e_begin[DX_MAX_ENTRIES];
  short e_tiles[DX_MAX_ENTRIES];
  short e_gid[DX_MAX_ENTRIES];
  const unsigned char* e_blob[DX_MAX_ENTRIES];
  short pair_id[DX_MAX_PAIRS];
  float pair_w[DX_MAX_PAIRS];
  float roww[DX_MAX_ENTRIES][kTok];   // weight of every group in every block row (0: the row is not in the group)
  // the CTA's units packed into pieces of up to eight unit slots; a run = consecutive units of one macro-unit
  int n_pieces, n_runs;
  int n_pieces_a;                               // (hand-over) pieces that do not depend on routing: [0, n_pieces_a)
  short piece_run0[kMaxPieces + 1];             // runs of piece p: [piece_run0[p], piece_run0[p + 1])
  unsigned char piece_slots[kMaxPieces];        // unit slots piece p uses
  unsigned char piece_entry[kMaxPieces][8];     // group of every unit slot
  const unsigned char* run_src1[kMaxRuns];      // gate/up part of the run's first unit in stage 0
  const unsigned char* run_src2[kMaxRuns];      // down part of the run's first unit in tile 0
  unsigned int run_stride[kMaxRuns];            // bytes from one stage (tile) to the next in the blob
  unsigned char run_slot0[kMaxRuns], run_n[kMaxRuns];
};

// Shared-memory matrix descriptor (no swizzle, K-major) as two words: low = start address >> 4 | (lbo >> 4) << 16,
// high = sbo >> 4 | descriptor version; lbo = bytes between the two core matrices of a product along the
// contraction, sbo = bytes between groups of eight rows.  Only the start address changes from product to product,
// so the issuing thread adds to the low word and never rebuilds a descriptor: it is a single thread with nothing
// to hide its instruction latencies behind, and every instruction it executes between two products costs.
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo) { return ((addr & 0x3FFFFu) >> 4) | ((lbo >> 4) << 16); }
__device__ __forceinline__ constexpr uint32_t desc_hi(uint32_t sbo) { return (sbo >> 4) | (1u << 14); }
// D[128 x 16] (+)= A[128 x 16] B[16 x 16]^T, bf16 operands from shared memory, fp32 accumulator in tensor memory
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTok >> 3) << 17) | (8u << 24);
__device__ __forceinline__ void umma(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                     uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tmov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
               "setp.ne.b32 p, %6, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
               ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(kIdesc), "r"(accumulate) : "memory");
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

// Wait of the epilogue warps: lane 0 polls with a pause between looks and the warp takes the outcome from it.  The
// tensor-core thread and the copy thread share their scheduler partitions with these warps; 128 threads spinning on
// a barrier would take the issue slots (and the shared-memory cycles) those two need.
__device__ __forceinline__ bool epi_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit, int lane) {
  int ok = 1;
  if (lane == 0) {
    ok = 0;
    for (uint32_t it = 0; it < limit; ++it) {
      if (mbar_try_wait(bar, parity)) { ok = 1; break; }
      if ((it & 15u) == 15u && *abort_flag) break;
      __nanosleep(64);
    }
    if (!ok) *abort_flag = 1;
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

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
    for (int b = 0; b < 4; ++b) mbar_init(smem_u32(&hdr->x_ready[b]), 4);
    mbar_init(smem_u32(&hdr->list_ready), 1);
    mbar_init(smem_u32(&hdr->static_ready), 1);
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

  // Two ways to be launched.  Plain: the routing kernel in front has completed once the wait below returns (the work
  // list is final, y is initialised).  Hand-over (fused entry points): this kernel was made resident by the routing
  // kernel before either has its input; it streams and multiplies the routing-independent groups while the routing
  // kernel works, takes the block from memory once a word says it is final, and polls the routed groups and the
  // (row, expert, gate) pairs out of the work list as they are written (every word carries its own valid bit).
  const bool paired = p.handover != nullptr;
  if (!paired) dx_pdl_wait();

  if (warp == 4) {
    // ------------------------------------------------------------------------------------------ work list + copies
    if (lane < n_static) {
      const bool is_draft = lane >= p.n_shared;
      hdr->e_begin[lane] = is_draft ? p.n_shared * p.shared_tiles : lane * p.shared_tiles;
      hdr->e_tiles[lane] = is_draft ? p.draft_tiles : p.shared_tiles;
      hdr->e_gid[lane] = -1;
      hdr->e_blob[lane] = DX_BOUNDS(lane < p.table_len, p.dev_status)
                              ? reinterpret_cast<const unsigned char*>(p.table[lane]) : nullptr;
    }
    __syncwarp();
    // packing state and copy state (used by lane 0 only)
    int np = 0, nr = 0, pslot = 0;
    bool overflow = false;
    uint32_t it = 0, slot = 0, phase = 0;
    bool alive = true;
    const uint64_t l2pol = l2_evict_first_policy();
    if (lane == 0) hdr->piece_run0[0] = 0;
    // units [u_lo, u_hi) of the groups [e_lo, e_hi) into unit slots, eight to a piece
    auto pack = [&](int e_lo, int e_hi, int u_lo, int u_hi) {
      for (int e = e_lo; e < e_hi && !overflow; ++e) {
        const int b = hdr->e_begin[e], nt = hdr->e_tiles[e];
        const int lo = max(b, u_lo), hi = min(b + nt, u_hi);
        const unsigned char* blob = hdr->e_blob[e];
        if (lo >= hi || blob == nullptr) continue;
        for (int u = lo; u < hi && !overflow;) {
          const int m = (u - b) >> 3, end = min(hi, b + 8 * (m + 1)), nq = min(8, nt - 8 * m);
          const unsigned char* mu = blob + (size_t)m * 8 * UNIT_BYTES;
          int q = (u - b) & 7, left = end - u;
          while (left > 0) {
            if (nr >= kMaxRuns || np >= kMaxPieces) { overflow = true; break; }
            const int take = min(left, 8 - pslot);
            hdr->run_src1[nr] = mu + (size_t)q * 2048;
            hdr->run_src2[nr] = mu + (size_t)nq * 32 * H + (size_t)q * 2048;
            hdr->run_stride[nr] = (unsigned int)nq * 2048u;
            hdr->run_slot0[nr] = (unsigned char)pslot;
            hdr->run_n[nr] = (unsigned char)take;
            for (int i = 0; i < take; ++i) hdr->piece_entry[np][pslot + i] = (unsigned char)e;
            ++nr; pslot += take; q += take; left -= take;
            if (pslot == 8) { hdr->piece_slots[np] = 8; ++np; hdr->piece_run0[np] = (short)nr; pslot = 0; }
          }
          u = end;
        }
      }
    };
    auto close_piece = [&]() {   // a partly filled piece ends here
      if (!overflow && pslot > 0) {
        if (np >= kMaxPieces) overflow = true;
        else { hdr->piece_slots[np] = (unsigned char)pslot; ++np; hdr->piece_run0[np] = (short)nr; pslot = 0; }
      }
    };
    // one stage of piece pc: every run's part of it, completing on one barrier
    auto push = [&](int pc, bool second, uint32_t index) {
      if (!alive) return;
      if (!mbar_wait(smem_u32(&hdr->empty[slot]), phase ^ 1u, abort_flag, p.wait_limit)) { alive = false; return; }
      const uint32_t fb = smem_u32(&hdr->full[slot]);
      mbar_arrive_expect_tx(fb, (uint32_t)hdr->piece_slots[pc] * 2048u);
      const uint32_t dst = smem_u32(ring + (size_t)slot * kStageBytes);
      for (int r = hdr->piece_run0[pc]; r < hdr->piece_run0[pc + 1]; ++r) {
        const unsigned char* src = (second ? hdr->run_src2[r] : hdr->run_src1[r]) + (size_t)index * hdr->run_stride[r];
        bulk_g2s(dst + (uint32_t)hdr->run_slot0[r] * 2048u, src, (uint32_t)hdr->run_n[r] * 2048u, fb, l2pol);
      }
      ++it;
      if (++slot == (uint32_t)n_stages) { slot = 0; phase ^= 1u; }
    };
    // pieces [lo, hi): gate/up stages of a piece, then the down stages of the piece before it
    auto stream = [&](int lo, int hi) {
      for (int pc = lo; pc < hi; ++pc) {
        for (int st = 0; st < S1; ++st) push(pc, false, (uint32_t)st);
        if (pc > lo)
          for (int t = 0; t < S2; ++t) push(pc - 1, true, (uint32_t)t);
      }
      if (hi > lo)
        for (int t = 0; t < S2; ++t) push(hi - 1, true, (uint32_t)t);
    };
    // Hand-over: the routing-independent groups could be multiplied at once, but a CTA's share of them is a few
    // units -- a piece of their own costs a full piece's products and keeps this warp from polling the list -- so
    // they wait for the routed groups and are packed with them (measured: 30 us for 2.4 units in a dependent stack).
    // What overlaps with the routing kernel is this kernel's set-up and the conversion of the block rows.
    const int n_a = 0;
    if (lane == 0) {
      hdr->n_pieces_a = 0;
      if (paired) mbar_arrive(smem_u32(&hdr->static_ready));
    }
    // ---- the routed groups.  Plain launch: the whole list in one round trip (it is final, words past the valid
    // entries are merely ignored).  Hand-over: polled until the head and every group word it announces are valid.
    constexpr int PER_LANE = DX_MAX_PAIRS / 32;
    unsigned long long gw[PER_LANE], pw[PER_LANE];
    unsigned long long head = 0ull;
    // the routed part of the blob table goes to shared memory in the same round trip as the list (the loads are
    // issued here and consumed after the list has been looked at)
    const void* tab[DX_MAX_E / 32];
#pragma unroll
    for (int i = 0; i < DX_MAX_E / 32; ++i) {
      const int e = lane + 32 * i;
      tab[i] = (p.n_shared + 1 + e < p.table_len)
                   ? reinterpret_cast<const void*>((uintptr_t)__ldcg(
                         reinterpret_cast<const unsigned long long*>(p.table + p.n_shared + 1 + e)))
                   : nullptr;
    }
    if (!paired) {
      head = dx_word_load(&W->head);
#pragma unroll
      for (int i = 0; i < PER_LANE; ++i) gw[i] = dx_word_load(&W->group[lane + 32 * i]);
#pragma unroll
      for (int i = 0; i < PER_LANE; ++i) pw[i] = dx_word_load(&W->pair[lane + 32 * i]);
    } else {
      bool have = false;
      for (uint32_t look = 0; look < p.wait_limit && !have; ++look) {
        head = dx_word_load(&W->head);
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) gw[i] = dx_word_load(&W->group[lane + 32 * i]);
        bool mine = false;
        if (head & DX_WORD_VALID) {
          const int ng = min((int)(head & 0xffffu), DX_MAX_PAIRS);
          mine = true;
#pragma unroll
          for (int i = 0; i < PER_LANE; ++i) mine = mine && (lane + 32 * i >= ng || (gw[i] & DX_WORD_VALID));
        }
        have = __all_sync(0xffffffffu, mine);
      }
      if (!have) {
        head = 0ull;
        if (lane == 0) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
      }
#pragma unroll
      for (int i = 0; i < PER_LANE; ++i) pw[i] = 0ull;   // (the pairs are fetched by the epilogue warps)
    }
    int n_groups = 0, kk = 1, n_pairs = 0;
    if (head & DX_WORD_VALID) {
      n_groups = min((int)(head & 0xffffu), DX_MAX_PAIRS);
      kk = (int)((head >> 16) & 0xffu);
      n_pairs = min((int)((head >> 24) & 0xffu) * kk, DX_MAX_PAIRS);
    }
    int pos[PER_LANE];
    int n_sel = 0;
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) {
      const int idx = lane + 32 * i;
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
      const int gid = dx_group_id(gw[i]);
      // the blob of expert gid sits in lane gid % 32, register gid / 32 of the prefetched table
      unsigned long long got = 0ull;
#pragma unroll
      for (int j = 0; j < DX_MAX_E / 32; ++j) {
        const unsigned long long v = __shfl_sync(0xffffffffu, (unsigned long long)(uintptr_t)tab[j], gid & 31);
        if ((gid >> 5) == j) got = v;
      }
      if (idx < 0) continue;
      const unsigned char* blob = nullptr;
      if (gid < DX_MAX_E && DX_BOUNDS(p.n_shared + 1 + gid < p.table_len, p.dev_status))
        blob = reinterpret_cast<const unsigned char*>((uintptr_t)got);
      const int e = n_static + idx;
      if (!DX_BOUNDS(e < DX_MAX_ENTRIES, p.dev_status)) continue;
      hdr->e_begin[e] = unit_base + idx * p.routed_tiles;
      hdr->e_tiles[e] = p.routed_tiles;
      hdr->e_gid[e] = gid;
      hdr->e_blob[e] = blob;
      if (blob == nullptr && e >= e_lo && e < e_hi) atomicExch(p.dev_status, DX_DEV_BAD_EXPERT_ID);
    }
    if (!paired) {
#pragma unroll
      for (int i = 0; i < PER_LANE; ++i) {
        const int idx = lane + 32 * i;
        if (idx < n_pairs) {
          hdr->pair_id[idx] = dx_pair_id(pw[i]);
          hdr->pair_w[idx] = (pw[i] & DX_WORD_VALID) ? dx_pair_weight(pw[i]) : 0.0f;
        }
      }
    }
    __syncwarp();
    if (lane == 0) {
      hdr->kk = kk;
      hdr->n_pairs = n_pairs;
      hdr->ph_e_hi[0] = p.do_static ? n_static : 0;
      hdr->ph_e_hi[1] = e_hi;
      if (p.do_static) pack(0, n_static, s_lo, s_hi);
      // (the routed groups all have routed_tiles units: only the few whose units meet this CTA's range are walked)
      if (u_hi > u_lo && p.routed_tiles > 0) {
        const int first = n_static + max(0, u_lo - unit_base) / p.routed_tiles;
        const int last = n_static + max(0, u_hi - 1 - unit_base) / p.routed_tiles;
        pack(max(e_lo, first), min(e_hi, last + 1), u_lo, u_hi);
      }
      close_piece();
      if (overflow) { np = n_a; atomicExch(p.dev_status, DX_DEV_WORKLIST_OVERFLOW); }
      hdr->n_pieces = np;
      hdr->n_runs = nr;
      mbar_arrive(smem_u32(&hdr->list_ready));   // (release: everything written above is visible to who waits)
      if (!paired) dx_pdl_trigger();   // what follows on the stream may be scheduled (it waits for this grid to end)
      stream(n_a, np);
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
      bool alive = true;
      // quarters of the block-row operand known to be in shared memory; stage s of the first product reads the
      // hidden columns up to 64 s + 63, which lie in quarter ((8 s + 7) * padded rows) / 1024
      int x_have = 0;
      const int x_lg = p.K <= 1 ? 0 : p.K <= 2 ? 1 : p.K <= 4 ? 2 : p.K <= 8 ? 3 : 4;
      auto need_x = [&](int s) {
        const int want = min(3, ((8 * s + 7) << x_lg) >> 10);
        while (alive && x_have <= want) {
          if (!mbar_wait(smem_u32(&hdr->x_ready[x_have]), 0u, abort_flag, p.wait_limit)) alive = false;
          tc_fence_after();
          ++x_have;
        }
      };
      // low descriptor words of the operands at their base addresses (see desc_lo); a stage is 1024 sixteen-byte units
      const uint32_t ring_a1 = desc_lo(smem_u32(ring), 128), ring_a2 = desc_lo(smem_u32(ring), 2048);
      const uint32_t xs_lo = desc_lo(smem_u32(xs), 256), act_lo = desc_lo(smem_u32(acts), 256);
      constexpr uint32_t A1_HI = desc_hi(1024), A2_HI = desc_hi(128), B_HI = desc_hi(128);
      uint32_t d2_started = 0u;    // bit T: tile T of D2 has been written
      auto next_stage = [&]() -> bool {
        if (!alive) return false;
        // (the stage was written by a bulk copy, which completes on this barrier in the tensor core's own proxy: the
        // products may follow the wait directly; a tcgen05 fence here would drain the pipe once per stage)
        if (!mbar_wait(smem_u32(&hdr->full[slot]), phase, abort_flag, p.wait_limit)) { alive = false; return false; }
        return true;
      };
      auto release_stage = [&]() {
        umma_commit(smem_u32(&hdr->empty[slot]));     // the slot is free again once the products above have read it
        if (++slot == (uint32_t)n_stages) { slot = 0; phase ^= 1u; }
      };
      auto gate_up = [&](int pidx) {
        const uint32_t d1 = tm_d1 + (uint32_t)(pidx & 1) * kTok;
        uint32_t b_lo = xs_lo;                      // advances by 8 core-matrix pairs (8 x 256 bytes) per stage
        for (int s = 0; s < S1; ++s, b_lo += 128) {
          if (x_have < 4) need_x(s);
          if (!next_stage()) return;
          const uint32_t a_lo = ring_a1 + slot * 1024u;
          umma(d1, a_lo, A1_HI, b_lo, B_HI, s != 0 ? 1u : 0u);
          umma(d1, a_lo + 16, A1_HI, b_lo + 32, B_HI, 1u);
          umma(d1, a_lo + 32, A1_HI, b_lo + 64, B_HI, 1u);
          umma(d1, a_lo + 48, A1_HI, b_lo + 96, B_HI, 1u);
          release_stage();
        }
        umma_commit(smem_u32(&hdr->d1_full[pidx & 1]));
      };
      auto down = [&](int pidx) {
        // the SwiGLU products of this piece, written by the epilogue warps
        if (alive && !mbar_wait(smem_u32(&hdr->act_ready[pidx & 1]), (uint32_t)(pidx >> 1) & 1u, abort_flag, p.wait_limit))
          alive = false;
        tc_fence_after();
        const uint32_t b_lo = act_lo + (uint32_t)(pidx & 1) * 128u;
        // products whose two unit slots are both unused are left out (their activations are zero anyway)
        const int used = hdr->piece_slots[pidx];
        const bool use0 = true, use1 = used > 2, use2 = used > 4, use3 = used > 6;
        for (int t = 0; t < S2; ++t) {
          if (!next_stage()) return;
          const uint32_t a_lo = ring_a2 + slot * 1024u, d2 = tm_d2 + (uint32_t)t * kTok;
          uint32_t acc = (d2_started >> t) & 1u;
          if (use0) { umma(d2, a_lo, A2_HI, b_lo, B_HI, acc); acc = 1u; }
          if (use1) { umma(d2, a_lo + 256, A2_HI, b_lo + 32, B_HI, acc); acc = 1u; }
          if (use2) { umma(d2, a_lo + 512, A2_HI, b_lo + 64, B_HI, acc); acc = 1u; }
          if (use3) { umma(d2, a_lo + 768, A2_HI, b_lo + 96, B_HI, acc); acc = 1u; }
          release_stage();
        }
        d2_started = (S2 >= 32) ? 0xffffffffu : ((1u << S2) - 1u);
      };
      // pieces [lo, hi): first product of a piece, then the second product of the piece before it
      auto run = [&](int lo, int hi) {
        for (int pc = lo; pc < hi; ++pc) {
          gate_up(pc);
          if (pc > lo) down(pc - 1);
        }
        if (hi > lo) down(hi - 1);
      };
      int n_a = 0;
      if (paired) {   // the routing-independent pieces, while the routing kernel is still at work
        if (!mbar_wait(smem_u32(&hdr->static_ready), 0u, abort_flag, p.wait_limit)) alive = false;
        n_a = alive ? hdr->n_pieces_a : 0;
        run(0, n_a);
      }
      if (alive && !mbar_wait(smem_u32(&hdr->list_ready), 0u, abort_flag, p.wait_limit)) alive = false;
      run(n_a, alive ? hdr->n_pieces : n_a);
      umma_commit(smem_u32(&hdr->d2_full));   // (also what the epilogue waits for before it lets the memory go)
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    bool alive = true;
    if (paired) {
      // the block itself may still be written by the kernel in front of the routing kernel, which sets this word
      // once that kernel has completed
      if (threadIdx.x == 0 && !flag_wait(p.handover, p.wait_limit)) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
      epi_bar();   // one poller per CTA; the others pick the acquire up through the barrier
    }
    {
    // ---- the block rows as the bf16 operand [H/8][2][8 rows x 16 bytes], built while warp 4 reads the work list.
    // An item is 8 consecutive elements of one row; items are dealt to the 128 threads with the row index fastest
    // (rows padded to a power of two, so the index arithmetic is shifts) and fetched in batches of eight per thread:
    // sixteen 16-byte loads in flight instead of one round trip per item.  A batch covers a contiguous range of the
    // hidden dimension and is handed to the tensor-core thread as soon as it is stored, so the first products start
    // after one batch.  RMSNorm: the rows go in unscaled and the sums of squares are collected on the way; 1 / rms
    // of a row is a factor of its whole column of D1, applied by the epilogue.
    const int tid = threadIdx.x;   // 0..127 = tensor-memory lane
    constexpr int KG = H / 8, BATCH = 8;
    const int lg = p.K <= 1 ? 0 : p.K <= 2 ? 1 : p.K <= 4 ? 2 : p.K <= 8 ? 3 : 4, Kp = 1 << lg;
    const int n_items = Kp * KG;
    if (tid < kTok) hdr->rstd[tid] = 0.0f;
    for (int idx = tid; idx < (kTok - Kp) * KG; idx += kEpiThreads) {     // token columns beyond the padded block: zero
      const int kg = idx / (kTok - Kp), t = Kp + idx - kg * (kTok - Kp);
      *reinterpret_cast<uint4*>(xs + (size_t)kg * 256 + (t >> 3) * 128 + (t & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    epi_bar();
    int batch = 0;
    for (int base0 = 0; base0 < n_items; base0 += kEpiThreads * BATCH, ++batch) {   // (same trip count for every thread)
      const int base = base0 + tid;
      float4 a[BATCH], b[BATCH];
#pragma unroll
      for (int i = 0; i < BATCH; ++i) {
        const int idx = base + i * kEpiThreads, t = idx & (Kp - 1), kg = idx >> lg;
        a[i] = b[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (idx < n_items && t < p.K) {
          const float* src = p.x + (size_t)t * H + 8 * kg;
          a[i] = *reinterpret_cast<const float4*>(src);
          b[i] = *reinterpret_cast<const float4*>(src + 4);
        }
      }
      float ssq = 0.f;   // (all of a thread's items belong to one row: 128 is a multiple of the padded row count)
#pragma unroll
      for (int i = 0; i < BATCH; ++i) {
        const int idx = base + i * kEpiThreads, t = idx & (Kp - 1), kg = idx >> lg;
        if (idx < n_items) {
          uint4 o;
          __nv_bfloat162 c0 = __floats2bfloat162_rn(a[i].x, a[i].y), c1 = __floats2bfloat162_rn(a[i].z, a[i].w);
          __nv_bfloat162 c2 = __floats2bfloat162_rn(b[i].x, b[i].y), c3 = __floats2bfloat162_rn(b[i].z, b[i].w);
          o.x = *reinterpret_cast<uint32_t*>(&c0); o.y = *reinterpret_cast<uint32_t*>(&c1);
          o.z = *reinterpret_cast<uint32_t*>(&c2); o.w = *reinterpret_cast<uint32_t*>(&c3);
          *reinterpret_cast<uint4*>(xs + (size_t)kg * 256 + (t >> 3) * 128 + (t & 7) * 16) = o;
          ssq += a[i].x * a[i].x + a[i].y * a[i].y + a[i].z * a[i].z + a[i].w * a[i].w +
                 b[i].x * b[i].x + b[i].y * b[i].y + b[i].z * b[i].z + b[i].w * b[i].w;
        }
      }
      if (p.rms_norm) {
        // lanes that share a row (equal lane mod padded rows) fold their sums; one shared-memory addition per row
        // and warp (an addition per item made the rows' four to sixteen words a serial bottleneck: 11 us at K = 4)
        for (int off = 16; off >= Kp; off >>= 1) ssq += __shfl_xor_sync(0xffffffffu, ssq, off);
        if (lane < Kp && lane < p.K) atomicAdd(&hdr->rstd[lane], ssq);
      }
      proxy_fence();            // written with ordinary stores, read by the tensor core
      epi_bar();
      if (lane == 0 && batch < 4) mbar_arrive(smem_u32(&hdr->x_ready[batch]));
    }
    for (; batch < 4; ++batch)   // (short blocks need fewer batches)
      if (lane == 0) mbar_arrive(smem_u32(&hdr->x_ready[batch]));
    }
    const int tid = threadIdx.x;
    // lane of tensor memory = row of D1: row group rg = tid / 8 = 2 q + (0 gate | 1 up), row r of the unit
    const int q = tid >> 4, gu = (tid >> 3) & 1, r = tid & 7;
    const uint32_t lane_base = (uint32_t)(32 * warp) << 16;
    // weight of the groups [e_lo, e_hi) in every block row
    auto row_weights = [&](int e_lo, int e_hi) {
      const int kk = hdr->kk;
      for (int idx = tid + e_lo * kTok; idx < e_hi * kTok; idx += kEpiThreads) {
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
    };
    // pieces [lo, hi): D1 -> w * silu(gate) * up as the bf16 operand of the second product
    auto pieces = [&](int lo, int hi) {
      for (int pidx = lo; pidx < hi; ++pidx) {
        if (alive && !epi_wait(smem_u32(&hdr->d1_full[pidx & 1]), (uint32_t)(pidx >> 1) & 1u, abort_flag, p.wait_limit, lane))
          alive = false;
        tc_fence_after();
        float v[16];
        tmem_ld16(tm_d1 + lane_base + (uint32_t)(pidx & 1) * kTok, v);
        // a gate row takes block rows 0..7, its up row (8 lanes on) block rows 8..15: swap the halves each needs
        float other[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) other[i] = __shfl_xor_sync(0xffffffffu, gu ? v[i] : v[8 + i], 8);
        const bool mine = q < (int)hdr->piece_slots[pidx];
        unsigned char* dst = acts + (size_t)(pidx & 1) * 2048 + (size_t)q * 256 + gu * 128 + r * 2;
        const float* wrow = hdr->roww[mine ? hdr->piece_entry[pidx][q] : 0] + 8 * gu;
        const float* rsrow = hdr->rstd + 8 * gu;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float rs = rsrow[i];
          const float g = (gu ? other[i] : v[i]) * rs, u = (gu ? v[8 + i] : other[i]) * rs;
          const float a = mine ? fast_silu(g) * u * wrow[i] : 0.0f;
          *reinterpret_cast<__nv_bfloat16*>(dst + i * 16) = __float2bfloat16_rn(a);
        }
        proxy_fence();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->act_ready[pidx & 1]));
      }
    };
    if (tid < kTok) hdr->rstd[tid] = p.rms_norm ? rsqrtf(hdr->rstd[tid] / (float)H + 1e-6f) : 1.0f;
    int n_a = 0;
    if (paired) {
      if (!epi_wait(smem_u32(&hdr->static_ready), 0u, abort_flag, p.wait_limit, lane)) alive = false;
      n_a = alive ? hdr->n_pieces_a : 0;
      row_weights(0, n_static);
      epi_bar();
      pieces(0, n_a);
    }
    if (alive && !epi_wait(smem_u32(&hdr->list_ready), 0u, abort_flag, p.wait_limit, lane)) alive = false;
    const int n_pieces = alive ? hdr->n_pieces : n_a;
    if (paired) {
      // the (row, expert, gate) pairs come out of the gate arithmetic a little after the group list
      const int n_pairs = alive ? hdr->n_pairs : 0;
      bool ok = true;
      for (int idx = tid; idx < n_pairs; idx += kEpiThreads) {
        unsigned long long w = 0ull;
        uint32_t look = 0;
        for (; look < p.wait_limit; ++look) {
          w = dx_word_load(&W->pair[idx]);
          if (w & DX_WORD_VALID) break;
        }
        ok = ok && look < p.wait_limit;
        hdr->pair_id[idx] = dx_pair_id(w);
        hdr->pair_w[idx] = dx_pair_weight(w);
      }
      if (!ok) { *abort_flag = 1; atomicExch(p.dev_status, DX_DEV_WAIT_EXPIRED); }
      epi_bar();
      // Only now may the next kernel of the stream start: if it is a routing kernel it clears the hand-over words
      // before its own wait, so every thread of this CTA has to be done with all of them (warp 4 was done with the
      // group words before it signalled the list).
      dx_pdl_trigger();
      row_weights(n_static, hdr->ph_e_hi[1]);
    } else {
      row_weights(0, max(hdr->ph_e_hi[0], hdr->ph_e_hi[1]));
    }
    epi_bar();
    pieces(n_a, n_pieces);
    if (paired) dx_pdl_wait();   // the routing kernel (which initialised y) has completed as a whole
    // ---- this CTA's partial output rows: D2 tile T, lane = output row 128 T + tid, columns = block rows
    if (alive && !epi_wait(smem_u32(&hdr->d2_full), 0u, abort_flag, p.wait_limit, lane)) alive = false;
    tc_fence_after();
    if (n_pieces > 0 && alive && !*abort_flag) {
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
