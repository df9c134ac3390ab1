// Internal declarations shared by the translation units of libdraftexpert.
// Host-side handle structs, the device work list the routing kernel hands to
// the expert kernels, and small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "draftexpert.h"

#define DX_MAX_K 16
#define DX_MAX_E 256
#define DX_MAX_TOPK 8
#define DX_MAX_SHARED 8
#define DX_MAX_H 8192
#define DX_MAX_PAIRS (DX_MAX_K * DX_MAX_TOPK)
#define DX_MAX_ENTRIES (DX_MAX_SHARED + 1 + DX_MAX_PAIRS)
#define DX_TILE_I 8            // intermediate rows per streamed weight tile
#define DX_MAX_M 16            // accept rows
#define DX_ROUTE_CLUSTER 4     // CTAs (and SMs) of the routing kernel; the expert kernel leaves them free

// What the routing kernel hands to the expert kernels.  The routing-independent groups (shared experts, draft
// expert) follow from the launch parameters alone; the routed groups are listed here, one per expert that some
// block row selected, in the order in which their work units are numbered.  A group's weight in block row t is
// the gate weight of the pair (t, j) that selected its expert, or nothing if no pair of that row did.
//
// Every item is one 64-bit word that carries its own "valid" bit (bit 63), so a reader that runs concurrently
// with the routing kernel polls the words themselves: no flag, no fence, no second round trip.  The routing
// kernel of a fused pair zeroes all words before it lets its expert kernel start.
//   head : valid | K << 24 | k << 16 | number of routed groups
//   group: valid | expert id << 48 | (blob address >> 4), the blob as the layer's table had it at routing time
//   pair : valid | expert id << 32 | gate weight bits, index t * k + j
struct DxWork {
  unsigned long long head;
  unsigned long long group[DX_MAX_PAIRS];
  unsigned long long pair[DX_MAX_PAIRS];
};
#define DX_WORD_VALID (1ull << 63)
__host__ __device__ inline unsigned long long dx_head_word(int K, int k, int n_groups) {
  return DX_WORD_VALID | ((unsigned long long)K << 24) | ((unsigned long long)k << 16) | (unsigned long long)n_groups;
}
__host__ __device__ inline unsigned long long dx_group_word(int gid, const void* blob) {
  return DX_WORD_VALID | ((unsigned long long)gid << 48) | ((unsigned long long)(uintptr_t)blob >> 4);
}
__host__ __device__ inline int dx_group_id(unsigned long long w) { return (int)((w >> 48) & 0x7fff); }
__host__ __device__ inline const void* dx_group_blob(unsigned long long w) {
  return (const void*)(uintptr_t)((w & 0xffffffffffffull) << 4);
}
__device__ __forceinline__ unsigned long long dx_pair_word(int id, float w) {
  return DX_WORD_VALID | ((unsigned long long)id << 32) | (unsigned long long)__float_as_uint(w);
}
__device__ __forceinline__ int dx_pair_id(unsigned long long w) { return (int)((w >> 32) & 0x7fffffff); }
__device__ __forceinline__ float dx_pair_weight(unsigned long long w) { return __uint_as_float((unsigned int)w); }
// 8-byte accesses that go to the L2 (the point where concurrently running kernels meet)
__device__ __forceinline__ void dx_word_store(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long dx_word_load(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

struct dx_ctx {
  int device;
  int sm_count;
  int smem_optin;
  int act_split;              // 1: bf16 experts are evaluated with hi + residual activation fragments
  int pdl_mask;               // DX_PDL_* bits: kernels launched with programmatic stream serialization
  uint32_t wait_limit;        // polls after which a bounded wait inside a kernel gives up (dx_set_wait_limit)
  size_t accept_keep_bytes;   // leading bytes of the LM head the accept kernel asks L2 to retain (dx_set_accept_l2_keep)
  cudaError_t last_cuda;
  int64_t launches;
  // device scratch
  DxWork* work;        // work list
  unsigned int* ticket;        // last-CTA ticket of the accept kernels (second word)
  unsigned long long* keys;    // [DX_MAX_M] packed argmax keys
  int32_t* dev_status;
  unsigned int* handover;      // device word {block input final}: see DxExpertParams
  float2* conf_part;           // [8 * sm_count][DX_MAX_M] per-CTA online-softmax pairs of the confidence variant
  int32_t* scratch_i32;        // two ints the draft-token entry point parks unused outputs in
  int32_t* union_dev;          // [DX_MAX_E] union ids, [1] union count, [DX_MAX_TOPK] draft selection: what the
  int32_t* union_host;         //   cached entry points read on the host (page-locked and mapped; the routing kernel writes it)
  int32_t* union_host_dev;     //   ... and its device mapping, which the routing kernel writes
};

// a CUDA runtime call inside an entry point: the error goes to the context, the entry point returns DX_ERR_CUDA
#define DX_CUDA(ctx, call)                 \
  do {                                     \
    cudaError_t e__ = (call);              \
    if (e__ != cudaSuccess) {              \
      if (ctx) (ctx)->last_cuda = e__;     \
      return DX_ERR_CUDA;                  \
    }                                      \
  } while (0)

struct dx_cache;
// (cached layer calls) the compute stream waits for the layer's copies that are still in flight and the layer's blob
// table is brought up to date: after this the table names exactly the experts the cache holds
dx_status dx_cache_prepare_layer(dx_cache* c, int layer, cudaStream_t st);
// true if none of the layer's copies is still in flight
bool dx_cache_layer_quiet(dx_cache* c, int layer);

struct dx_layer {
  dx_ctx* ctx;
  dx_layer_desc desc;
  const void* W_r;
  const float* bias;
  // blob table: [0,n_shared) shared, [n_shared] draft, [n_shared+1, n_shared+1+E) routed
  const void** table_host;
  const void** table_dev;
  int table_len;
  bool dirty;
  dx_cache* cache;
  int cache_layer;
};

struct DxRouteParams {
  const float* h;
  int K, H, E, k;
  int score_fn, norm_topk;
  float scale, gamma;
  const void* W_r;
  const float* bias;
  const void* const* table;   // layer blob table (device)
  int n_shared, shared_tiles, routed_tiles, draft_tiles;
  int draft_mode;   // 0: verify block, 1: drafter (shared + draft expert + top_r routed)
  int top_r;        // drafter: routed groups taken from the top of the selection (0 = none)
  int skip_top1;    // verify: leave every row's first selected expert out (the missing residual of Eq. 6)
  int rms_norm;     // 1: route and experts see RMSNorm(h)
  int residual;     // 0: y starts at zero, 1: y starts as a copy of h (pre-norm residual form)
  unsigned int* handover; // not null: the expert kernel of this call runs concurrently (fused entry points): zero
                          // the hand-over words first, and set this word once everything in front of this
                          // kernel in the stream has completed
  float* y;
  DxWork* work;
  int32_t* dev_status;
  int32_t* topk_ids;
  float* topk_w;
  unsigned long long* union_mask;
  int32_t* union_ids;
  int32_t* union_count;
  int32_t* offsets;
  int32_t* perm;
  // not null: page-locked host memory (through its device mapping) that gets a copy of what the host needs to go on
  // after this kernel -- [0, DX_MAX_E) the union's expert ids, [DX_MAX_E] their count, [DX_MAX_E + 1, + k) the
  // selection of block row 0 -- so that no device -> host copy has to follow the kernel
  int32_t* host_mirror;
};

struct DxExpertParams {
  const float* x;            // [K,H] block input (never written while the kernel runs)
  float* y;                  // [K,H] accumulated into; initialised by the routing kernel
  const void* const* table;  // layer blob table (device)
  int table_len;             // entries of the table (bounds of the checked build)
  const DxWork* work;
  int32_t* dev_status;
  int H, K;
  int rms_norm;              // 1: the experts see RMSNorm(x) (unit gain, eps 1e-6)
  // groups known without routing: shared experts (all K rows, weight 1) and, in draft mode, the draft expert
  int n_shared, shared_tiles, draft_tiles, routed_tiles;
  float gamma;
  // window of the routed entries this launch covers (position among them, count or -1 = all) and whether
  // the routing-independent groups are part of it; a cache-staged union is processed in several windows
  int first_routed, n_routed, do_static;
  int skip_shared;           // 1: of the routing-independent groups only the draft expert is evaluated
  // of the routed groups (inside the window above) only those whose expert id has its bit set are evaluated: a wave
  // of a cache-staged union need not be a contiguous run of the ascending id list
  int use_subset;
  unsigned long long subset[DX_MAX_E / 64];
  // 1: a routed group whose blob-table entry is null is left out without a word in the status (the caller launched
  // this kernel before it knew which expert the router would select, and evaluates the group afterwards if it was
  // not resident); 0: such a group is reported as DX_DEV_BAD_EXPERT_ID
  int tolerate_missing;
  int row_tiles;             // set by the launcher: 2 = CTA pairs, one tile of eight block rows each (K > 8)
  // Hand-over from the routing kernel launched right before this one (fused entry points only; null otherwise,
  // and then the kernel simply waits for everything in front of it).  With the hand-over this kernel may be running
  // before its inputs are final: consumers read the block only once this word is set, and the routed groups are
  // polled out of the work list.  The routing kernel of the next pair clears the word and the list before it lets
  // its own expert kernel start; this kernel in turn lets that routing kernel start only when it is past both.
  unsigned int* handover;
  uint32_t wait_limit;       // polls after which a bounded wait gives up (sets DX_DEV_WAIT_EXPIRED)
};

// Persistent draft stack (dx_draft_stack.cu): one descriptor per layer in device memory ...
struct DxStackLayer {
  const void* const* table;   // the layer's device blob table
  const void* W_r;            // [E,H] bf16
  const float* bias;          // [E] or null
  float gamma;
  int pad;
};
// ... and the launch parameters
// Partial sums a layer's contributions to the hidden row are spread over (CTA c adds into copy c mod this): every
// word of a single row would take one addition from every CTA, and additions to one address are carried out one
// after the other in L2 -- with 148 CTAs the last CTA's release waited 2.5 us for them.
#define DX_STACK_COPIES 4
struct DxStackParams {
  const DxStackLayer* layers;
  int n_layers;
  const float* h_in;          // [H]
  float* h_out;               // [H]
  // all zero at launch:
  float* delta;               // [n_layers][DX_STACK_COPIES][H] what layer l adds to the hidden row, in partial sums
  unsigned long long* zword;  // [n_layers][E] router logits exchanged between the CTAs, (1 << 32 | float bits)
  unsigned int* sync;         // [n_layers] CTAs that have added all of their share of layer l
  int32_t* topk_ids;          // [n_layers][k] or null
  float* topk_w;              // [n_layers][k] or null
  int32_t* dev_status;
  int H, E, k, score_fn, norm_topk;
  float scale;
  int n_shared, shared_tiles, draft_tiles, routed_tiles;
  int q4;                     // 1: the units are 4-bit codes with block scales
  uint32_t wait_limit;        // polls after which a bounded wait gives up
};
struct dx_stack {
  dx_ctx* ctx;
  int n_layers;
  dx_layer** layers;          // host copy of the handles
  DxStackLayer* desc_host;    // what desc_dev holds (all zero at first)
  DxStackLayer* desc_dev;
  unsigned char* scratch;     // delta rows, logit words, arrival counters (cleared before every launch)
  size_t scratch_bytes, zword_off, sync_off;
};
cudaError_t dx_launch_draft_stack(dx_ctx* ctx, const DxStackParams& p, cudaStream_t st);

// launchers (each returns the cudaError_t of the launch)
cudaError_t dx_launch_route(dx_ctx* ctx, const DxRouteParams& p, int weight_dtype, cudaStream_t st);
cudaError_t dx_launch_experts(dx_ctx* ctx, const DxExpertParams& p, int weight_dtype, int K, cudaStream_t st);
cudaError_t dx_launch_pack(int weight_dtype, int H, int I, const void* Wg, const void* Wu, const void* Wd,
                           void* blob, cudaStream_t st);
// bytes of one consumer warp's chunk of a unit (a unit = 8 chunks = 8 intermediate rows of an expert)
inline size_t dx_chunk_bytes(int H, bool q4) {
  return q4 ? (size_t)(H / 128) * 144 + (size_t)(H / 256) * 192 : (size_t)6 * H;
}
cudaError_t dx_launch_experts_wide(dx_ctx* ctx, const DxExpertParams& p, cudaStream_t st);
cudaError_t dx_launch_pack_wide(int H, int I, const void* Wg, const void* Wu, const void* Wd, void* blob,
                                cudaStream_t st);
cudaError_t dx_launch_pack_q4(int H, int I, const void* Wg, const void* Wu, const void* Wd, void* blob,
                              cudaStream_t st);
cudaError_t dx_launch_expand_q4(int H, int I, const void* q4, void* blob, cudaStream_t st);
cudaError_t dx_launch_accept(dx_ctx* ctx, const float* h, int M, const void* W_lm, int V, int H, int w_dtype,
                             const int32_t* draft, int K, int rms_norm, int32_t* target, int32_t* n_accept,
                             int32_t* next_token, float* conf, cudaStream_t st);
cudaError_t dx_launch_router_agreement(const dx_layer* L, const float* h_star, const float* h_draft, int K, float* kl,
                                       int32_t* agree, cudaStream_t st);
cudaError_t dx_launch_squared_error(const float* a, const float* b, long long n, float* out, cudaStream_t st);
cudaError_t dx_experts_prepare(dx_ctx* ctx);   // opt-in shared memory attributes, once per context

// cache hooks used by the layer code
void dx_cache_note_use(dx_cache* c, int layer, cudaStream_t st);

// Programmatic dependent launch: wait for the preceding kernel of the stream / let the next one start early.
__device__ __forceinline__ void dx_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dx_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Which kernels are launched with programmatic stream serialization (dx_ctx::pdl_mask, dx_set_launch_overlap):
// bit 0 routing, bit 1 experts, bit 2 greedy accept.
enum { DX_PDL_ROUTE = 1, DX_PDL_EXPERTS = 2, DX_PDL_ACCEPT = 4 };
#define DX_WAIT_LIMIT_DEFAULT (1u << 22)

// Launch with programmatic stream serialization so that the kernel may begin while its predecessor drains.
template <typename... KArgs, typename... Args>
inline cudaError_t dx_launch_pdl(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, int cluster, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (cluster > 1) {   // the grid is made of thread-block clusters of this many CTAs
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// This CTA's share of the routed groups.  The launch may be restricted to a window of the routed entries
// (a "wave" of union experts when the experts are staged through a cache); the units of the window, together
// with the routing-independent units handled before (NSe of them, [s_lo,s_hi) on this CTA), are split evenly.
__device__ __forceinline__ void dx_routed_range(int n_groups, const DxExpertParams& p, int n_static, int NSe, int s_lo,
                                             int s_hi, int G, int cta, int& e_lo, int& e_hi, int& u_lo, int& u_hi) {
  const int g_lo = min(n_groups, p.first_routed);
  const int g_hi = p.n_routed < 0 ? n_groups : min(n_groups, g_lo + p.n_routed);
  e_lo = n_static + g_lo;
  e_hi = n_static + g_hi;
  if (g_lo >= g_hi) { u_lo = u_hi = 0; return; }
  // (unit counts are a few ten thousand at most, grids a few hundred CTAs: the products fit 32 bits)
  const unsigned int base = (unsigned int)(p.n_shared * p.shared_tiles + p.draft_tiles);
  const unsigned int R0 = base + (unsigned int)(g_lo * p.routed_tiles);
  const unsigned int NR = (unsigned int)((g_hi - g_lo) * p.routed_tiles), T = (unsigned int)NSe + NR;
  const unsigned int uG = (unsigned int)G, ucta = (unsigned int)cta;
  int a, b;
  if (T / uG >= ((unsigned int)NSe + uG - 1u) / uG) {   // keep routing-independent + routed units balanced together
    a = (int)((T * ucta) / uG) - s_lo; b = (int)((T * (ucta + 1u)) / uG) - s_hi;
  } else {
    a = (int)((NR * ucta) / uG); b = (int)((NR * (ucta + 1u)) / uG);
  }
  u_lo = (int)R0 + a;
  u_hi = (int)R0 + b;
}

// Bounds checks of the checked build (-DDX_CHECKED, the stand-in for a memory checker): `if (DX_BOUNDS(i < n, status))`
// guards an indexed access; a violated bound records DX_DEV_BOUNDS in the status word and skips the access.  In the
// normal build the condition is not evaluated.
#ifdef DX_CHECKED
#define DX_BOUNDS(cond, status) ((cond) ? true : (atomicExch((status), (int32_t)DX_DEV_BOUNDS), false))
#else
#define DX_BOUNDS(cond, status) (true)
#endif

__device__ __forceinline__ float dx_silu(float x) { return x / (1.0f + expf(-x)); }

// Monotone map from float to uint32 (larger float -> larger unsigned).
__device__ __forceinline__ unsigned int dx_orderable(float f) {
  unsigned int u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
