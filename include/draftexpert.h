/*
 * draftexpert.h -- C ABI of the B200 (sm_100a) draft / verify MoE hot path of
 * DraftExpert, expansion-aware self-speculative decoding for MoE models.
 *
 * What the library computes (paper notation):
 *   - drafter,  Eq. 5 (Sec. 3.2):  y^d = S(h) + g_{e1} E_{e1}(h) + gamma E^d(h),  e1 = argmax_e R(h)_e
 *   - verifier, Eq. 4 (Sec. 3.2):  y*_t = S(h_t) + sum_{e in TopK(h_t)} g_{t,e} E_e(h_t)   for a K-token block,
 *     evaluated grouped by the block's expert set U(D) = union_t TopK(h_t) (Eq. 2, Eq. 3) so that each
 *     expert's weights are read from HBM once per block
 *   - exact greedy verification, Algorithm 1 last two steps: target tokens = vocabulary argmax, accepted
 *     length = longest draft prefix that equals them
 *   - the accelerator expert cache C and in-flight set P of Sec. 3.5 / Algorithm 1 (prefetch, wait, on-demand)
 *
 * Conventions
 *   - Every function returns a dx_status; nothing throws, aborts or prints.
 *   - "device pointer" = memory of the context's GPU, "host pointer" = ordinary host memory, "pinned host
 *     pointer" = page-locked host memory.  All tensor pointers are BORROWED: the caller allocates and frees
 *     them and keeps them alive until the stream work that uses them has finished.
 *   - Handles (dx_ctx, dx_layer, dx_cache) are owned by the library; release them with the matching destroy.
 *   - Compute calls only enqueue work on the caller's stream (a cudaStream_t passed as void*; NULL is the
 *     default stream).  They do not synchronise the host, except where a function says so.
 *   - A context carries one set of device scratch buffers; calls that share a context must be issued on one
 *     stream (or otherwise ordered).  Use one context per concurrent stream.
 *   - Matrices are row-major.  Hidden states, outputs, gate weights and logits are fp32; weights are fp32 or
 *     bf16 as stated by weight_dtype; all accumulation is fp32.  DX_DTYPE_Q4: the expert weights (shared, draft,
 *     routed) are 4-bit block-quantised, the format of the paper's mobile runs (Sec. 4): every row of W_g, W_u
 *     [inter, hidden] and W_d [hidden, inter] in blocks of 32 weights, 18 bytes each -- an fp16 scale d, then 16
 *     bytes whose low / high nibbles are the codes of weights j / j + 16; weight = d * (code - 8), evaluated
 *     exactly (no rounding of the product).  The router of such a layer is bf16.  The experts stay 4-bit in HBM
 *     and are de-quantised inside the streaming loop of the expert kernel, so a Q4 expert costs 0.94 bytes per
 *     weight of HBM traffic instead of 2.  Every intermediate size must then be a multiple of 32.
 *     DX_DTYPE_BF16_WIDE: bf16 weights whose expert blobs are packed for the kernel that runs the grouped SwiGLU on
 *     the 5th-generation tensor cores (tcgen05, accumulators in tensor memory) with the block rows as the 16-column
 *     operand: its time does not depend on the block length, so it is the layout to choose when blocks of 9..16 rows
 *     matter (Eq. 4 over longer verification blocks); the streaming layout of DX_DTYPE_BF16 is a little faster for
 *     blocks of up to 8 rows.  Same blob size, same entry points; activations enter the tensor cores as plain bf16
 *     (dx_set_activation_split does not apply); dx_stack_create and the 4-bit host pool refuse such layers.
 *   - Limits: block length K <= 16, experts E <= 256, top-k <= 8, shared experts <= 8, every intermediate size
 *     a multiple of 8; hidden a multiple of 256 up to 8192 for fp32 weights and one of 256, 512, 1024, 2048
 *     for bf16 weights.  Outside them: DX_ERR_UNSUPPORTED.
 *   - Device-side anomalies (an id out of range, a bounded wait that expired) never trap: the kernel records
 *     a code in the context's device status word, readable with dx_last_device_status.
 */
#ifndef DRAFTEXPERT_H_
#define DRAFTEXPERT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t dx_status;
enum {
  DX_OK = 0,
  DX_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, misaligned blob, index out of range */
  DX_ERR_SHAPE = 2,         /* sizes inconsistent with the layer description */
  DX_ERR_CUDA = 3,          /* a CUDA runtime call failed; see dx_last_cuda_error */
  DX_ERR_OOM = 4,
  DX_ERR_NOT_RESIDENT = 5,  /* an expert needed by the call has no weights attached / registered */
  DX_ERR_TIMEOUT = 6,
  DX_ERR_CACHE_FULL = 7,
  DX_ERR_UNSUPPORTED = 8
};

enum { DX_SCORE_SOFTMAX = 0, DX_SCORE_SIGMOID = 1 };
enum {
  DX_DTYPE_FP32 = 0,
  DX_DTYPE_BF16 = 1,
  DX_DTYPE_Q4 = 2,        /* experts 4-bit, router bf16 */
  DX_DTYPE_BF16_WIDE = 3  /* bf16 router and experts, the experts packed for the tcgen05 kernel (see below) */
};

/* Codes a kernel may leave in the device status word (0 = clean). */
enum {
  DX_DEV_OK = 0,
  DX_DEV_BAD_EXPERT_ID = 1,     /* a routed expert has no weight blob attached */
  DX_DEV_WAIT_EXPIRED = 2,      /* a bounded wait inside a kernel gave up */
  DX_DEV_WORKLIST_OVERFLOW = 3,
  DX_DEV_BOUNDS = 4             /* checked build only (-DDX_CHECKED): an index left its range; the access was skipped */
};

typedef struct dx_ctx dx_ctx;
typedef struct dx_layer dx_layer;
typedef struct dx_cache dx_cache;

/* One MoE layer.  score_fn / norm_topk / routed_scale define R(h) and g_{l,e} of Eq. 4 (the paper leaves
 * them to the model: softmax or sigmoid scores, top-k weights renormalised or not, times a routed scaling
 * factor that multiplies the routed sum only).  draft_gamma is gamma_l of Eq. 5. */
typedef struct {
  int32_t hidden;        /* H */
  int32_t n_experts;     /* N_l (E) */
  int32_t top_k;         /* k_l */
  int32_t inter;         /* I of the routed experts */
  int32_t n_shared;      /* number of shared experts making up S_l */
  int32_t shared_inter;  /* I of each shared expert */
  int32_t draft_inter;   /* I of the draft expert E^d_l (0 = none) */
  int32_t score_fn;      /* DX_SCORE_* */
  int32_t norm_topk;     /* 1: gate weights renormalised over the selected k */
  int32_t weight_dtype;  /* DX_DTYPE_* of router and expert weights */
  float routed_scale;
  float draft_gamma;
} dx_layer_desc;

const char* dx_status_string(dx_status s);

/* ---- context -------------------------------------------------------------------------------------------
 * dx_create binds to CUDA device `device`, allocates the context's small device scratch (a few MB: work
 * list, normalised block, router logits, argmax keys, status word) and returns the handle in *out.
 * Synchronises the host.  dx_destroy frees it (device must be idle with respect to this context). */
dx_status dx_create(int device, dx_ctx** out);
dx_status dx_destroy(dx_ctx* ctx);
/* Reads (and clears) the device status word.  Synchronises `stream` first. */
dx_status dx_last_device_status(dx_ctx* ctx, void* stream, int32_t* dev_status_out);
/* How bf16 experts are evaluated (DX_DTYPE_BF16 layers; set before the calls it should affect).  Off (the
 * default): the activations -- the block rows, then the SwiGLU products -- enter the tensor cores as bf16, one
 * rounding of at most 2^-9 relative each, as a bf16 model does; layer outputs are then within ~5e-3 of the row
 * maximum of exact arithmetic on the same weights (the stated tolerance is 2e-2).  On: every activation is fed
 * as a bf16 high part plus a bf16 residual (two products per fragment), which brings the outputs to ~1e-5 at
 * twice the tensor work (a few percent of the expert kernel's time for blocks of up to 8 rows, about twice the
 * time above).  fp32 layers and the single-token stack kernel always use fp32 activations; 4-bit layers always
 * plain bf16. */
dx_status dx_set_activation_split(dx_ctx* ctx, int32_t on);
/* Which kernels are launched so that they may begin while the kernel in front of them on the stream drains
 * (programmatic stream serialization): bit 0 the routing kernel, bit 1 the expert kernels, bit 2 the greedy-accept
 * kernels.  Default 3.  0 gives plain stream order everywhere; results never depend on the mask. */
dx_status dx_set_launch_overlap(dx_ctx* ctx, int32_t mask);
/* Every wait inside a kernel (for a word another kernel publishes, for a copy into shared memory, for the other CTAs
 * of a cooperative launch) polls at most `polls` times, then records DX_DEV_WAIT_EXPIRED in the device status word and
 * lets the kernel run to its end; the outputs of that call are then undefined, the context stays usable.  Default
 * 2^22 polls (seconds); 0 restores it. */
dx_status dx_set_wait_limit(dx_ctx* ctx, uint32_t polls);
/* spec_accept / spec_draft_token with a bf16 head: the leading `bytes` of W_lm are read with an L2 evict-last hint and
 * the rest with evict-first, so that the head of the matrix (the same in every decode step, and larger than L2 as a
 * whole) is still in L2 at the next call and only the rest comes from HBM again.  0 (the default) reads the whole
 * matrix as a plain stream.  Results do not depend on it. */
dx_status dx_set_accept_l2_keep(dx_ctx* ctx, size_t bytes);
/* Host -> device transfer of a step's inputs (a block of hidden rows, draft tokens): dst (device, any alignment) <-
 * src_host (page-locked host memory; DX_ERR_INVALID_ARG otherwise), in stream order.  Up to 1 MB with both addresses
 * 16-byte aligned is moved by a kernel that reads the host buffer through its device mapping (no copy-engine set-up;
 * the host may rewrite the buffer once the call's work has completed); anything else goes through cudaMemcpyAsync.
 * The result pointers of spec_accept / spec_draft_token may point into page-locked host memory as well: the kernel
 * then writes the few result words straight to the host and no device -> host copy is needed. */
dx_status dx_stage_block(dx_ctx* ctx, void* dst, const void* src_host, size_t bytes, void* stream);
/* Exercises that give-up path without a fault: clears the hand-over words and launches the expert half of a verify
 * block alone, as if the routing kernel it expects beside it never ran.  The kernel's waits run out, it returns, and
 * dx_last_device_status reads DX_DEV_WAIT_EXPIRED; y is undefined afterwards.  Refused (DX_ERR_INVALID_ARG) unless the
 * wait limit has been set to at most 2^16 polls, so that the kernel gives up within milliseconds; bf16 / 4-bit layers
 * only.  h [K,H], y [K,H] device pointers as for moe_verify_block. */
dx_status dx_selftest_wait_expiry(dx_layer* layer, const float* h, int32_t K, float* y, void* stream);
/* Last cudaError_t seen by this context as an int (0 = none). */
int32_t dx_last_cuda_error(dx_ctx* ctx);
/* Number of kernels this context has launched so far (for launch accounting by a caller). */
int64_t dx_kernel_launches(dx_ctx* ctx);

/* ---- expert weights ---------------------------------------------------------------------------------------
 * An expert is a SwiGLU feed-forward E(h) = W_d ( silu(W_g h) * (W_u h) ), W_g,W_u [I,H], W_d [H,I]
 * (the expert form the paper's parameter count in Sec. 2.1 implies: 3*H*I per expert).
 * The kernels stream each expert from ONE contiguous "blob" in a tile-major layout of the library's choosing
 * (the same number of bytes as the three matrices).  dx_expert_blob_bytes gives its size;
 * dx_pack_expert fills a blob from the three canonical row-major matrices (all device pointers; the blob must
 * be 128-byte aligned; runs on `stream`).  Blobs can be copied around freely (host pool, cache slots).
 * DX_DTYPE_Q4: Wg, Wu, Wd point to the matrices' 4-bit blocks (uint8 [rows][cols/32][18], device, 2-byte aligned)
 * and the blob keeps the codes 4-bit (inter * (hidden/128*144 + hidden/256*192) bytes: the codes in the order the
 * kernel's fragments want them, each 32-weight block's scale next to them). */
dx_status dx_expert_blob_bytes(const dx_layer_desc* desc, int32_t inter, size_t* bytes_out);
dx_status dx_pack_expert(dx_ctx* ctx, const dx_layer_desc* desc, int32_t inter,
                         const void* Wg, const void* Wu, const void* Wd, void* blob_out, void* stream);

/* ---- 4-bit block-quantised experts (the paper's mobile runs use Q4_0 weights, Sec. 4) ----------------------
 * Format of a quantised expert: the Q4_0 blocks of W_g [inter,hidden], W_u [inter,hidden] and W_d [hidden,inter],
 * row-major, one matrix after the other; a block covers 32 consecutive weights of a row and is 18 bytes: the fp16
 * scale d (little endian), then 16 bytes whose low nibbles are the codes of weights 0..15 and whose high nibbles
 * those of weights 16..31; weight = d * (code - 8).  inter must be a multiple of 32; bf16 layers only.
 * On this hardware the quantised form is the *transport and storage* form: 180 GB of HBM hold expanded slots
 * easily, the scarce link is host -> device.  dx_expand_q4_expert (device pointers, asynchronous on `stream`)
 * writes the bf16 streaming blob of dx_expert_blob_bytes bytes (128-byte aligned), each weight rounded to bf16
 * once: out = bf16(d * (code - 8)); the compute kernels are the bf16 ones, unchanged.  A cache switched with
 * expert_cache_set_q4 takes quantised blobs in expert_cache_register and expands each copy on its copy stream
 * (see the cache section). */
dx_status dx_q4_expert_bytes(const dx_layer_desc* desc, int32_t inter, size_t* bytes_out);
dx_status dx_expand_q4_expert(dx_ctx* ctx, const dx_layer_desc* desc, int32_t inter, const void* q4_blob,
                              void* blob_out, void* stream);

/* ---- layer ------------------------------------------------------------------------------------------------
 * dx_layer_create copies the description and allocates the layer's device pointer table.
 * set_router: W_r [E,H] in weight_dtype, optional fp32 bias[E] added to the router logits (NULL = none).
 * set_shared / set_draft / set_expert attach packed blobs (device pointers, 128-byte aligned, borrowed).
 * set_expert with blob == NULL detaches expert e (a block that then routes to it reports
 * DX_DEV_BAD_EXPERT_ID in the device status word and skips that expert).
 * The table is uploaded on the next compute call's stream, so set_* calls must not be interleaved with
 * compute calls that are still being captured into a CUDA graph. */
dx_status dx_layer_create(dx_ctx* ctx, const dx_layer_desc* desc, dx_layer** out);
/* (A layer attached to a cache may be destroyed before or after the cache: each side forgets the other.) */
dx_status dx_layer_destroy(dx_layer* layer);
dx_status dx_layer_set_router(dx_layer* layer, const void* W_r, const float* bias);
dx_status dx_layer_set_shared(dx_layer* layer, int32_t s, const void* blob);
dx_status dx_layer_set_draft(dx_layer* layer, const void* blob);
dx_status dx_layer_set_expert(dx_layer* layer, int32_t e, const void* blob);
/* Routed experts of this layer are looked up in cache slots of `cache` (layer index `layer_index` there)
 * instead of the table filled by set_expert. */
dx_status dx_layer_attach_cache(dx_layer* layer, dx_cache* cache, int32_t layer_index);

/* ---- drafter: Eq. 5 -----------------------------------------------------------------------------------------
 * One token.  h [H] fp32 in, y [H] fp32 out (overwritten), topk_ids [k] int32 and topk_w [k] fp32 out:
 * the router's full top-k in descending score (ties: lower id first) with the gate weights of Eq. 4;
 * e1 = topk_ids[0], and the k ids are the predicted verifier experts \hat{E}_{l,i} of Sec. 3.4.
 * All device pointers. */
dx_status moe_draft_step(dx_layer* layer, const float* h, float* y, int32_t* topk_ids, float* topk_w,
                         void* stream);

/* The training-free shared + top-r self-drafter of Sec. 2.2 / Sec. 4 (r = 1, 2, 3 in the paper), and mixtures:
 * y = S(h) + sum_{j<top_r} g_{e_j} E_{e_j}(h) (+ gamma E^d(h) iff use_draft_expert != 0), gate weights as in Eq. 4.
 * top_r = 1 with the draft expert is moe_draft_step; 1 <= top_r <= k. */
dx_status moe_draft_step_topr(dx_layer* layer, const float* h, float* y, int32_t top_r, int32_t use_draft_expert,
                              int32_t* topk_ids, float* topk_w, void* stream);

/* ---- verifier: Eq. 4 over a block, grouped by the union of Eq. 2 / Eq. 3 -----------------------------------
 * h [K,H] in, y [K,H] out (overwritten; must not overlap h).  Routing outputs (device pointers, each may be NULL if unwanted):
 *   topk_ids [K,k] int32, topk_w [K,k] fp32;
 *   union_mask [ceil(E/64)] uint64 (bit e set iff e in U); union_ids [min(E,K*k)] int32 ascending;
 *   union_count [1] int32 = |U|;
 *   offsets [E+1] int32 and perm [K*k] int32: the token-expert pairs p = t*k + j sorted by (expert, p);
 *   expert e owns perm[offsets[e] .. offsets[e+1]).
 * moe_verify_block gives the results of moe_verify_route followed by moe_verify_experts on the same stream; the
 * two halves are exported so that a caller with offloaded experts can make them resident in between.  The fused
 * call (and moe_draft_step, the *_residual forms) overlaps the two kernels: the expert kernel is made resident by
 * the routing kernel before either has its input, streams the shared experts, and picks the block and the routed
 * groups up from device memory as the routing kernel publishes them.  Every wait in it is bounded: if the routing
 * kernel never runs, the expert kernel gives up, records DX_DEV_WAIT_EXPIRED and returns.  The fused calls are safe
 * to capture into CUDA graphs and to replay. */
dx_status moe_verify_block(dx_layer* layer, const float* h, int32_t K, float* y,
                           int32_t* topk_ids, float* topk_w, uint64_t* union_mask, int32_t* union_ids,
                           int32_t* union_count, int32_t* offsets, int32_t* perm, void* stream);
dx_status moe_verify_route(dx_layer* layer, const float* h, int32_t K, float* y,
                           int32_t* topk_ids, float* topk_w, uint64_t* union_mask, int32_t* union_ids,
                           int32_t* union_count, int32_t* offsets, int32_t* perm, void* stream);
dx_status moe_verify_experts(dx_layer* layer, const float* h, int32_t K, float* y, void* stream);
/* The expert half restricted to a window of the union: union positions [first_union, first_union + n_union)
 * of the ascending union_ids list, plus the shared experts iff include_shared != 0.  y is added to (the route
 * half initialised it), so a union that does not fit the cache slots is evaluated in several windows ("waves"),
 * each after staging its experts; exactly one window must include the shared experts. */
dx_status moe_verify_experts_range(dx_layer* layer, const float* h, int32_t K, float* y, int32_t first_union,
                                   int32_t n_union, int32_t include_shared, void* stream);
/* The two halves of moe_draft_step, for layers whose routed experts are staged through a cache: after
 * moe_draft_route the caller reads topk_ids[0] (= e1), makes that expert resident, then runs the experts. */
dx_status moe_draft_route(dx_layer* layer, const float* h, float* y, int32_t* topk_ids, float* topk_w,
                          void* stream);
dx_status moe_draft_experts(dx_layer* layer, const float* h, float* y, void* stream);

/* ---- the same two calls on a layer whose routed experts come through an expert cache (Sec. 3.5, Algorithm 1:
 * "wait for useful in-flight prefetches", "any missed expert is still loaded on demand") ---------------------------
 * The layer must be attached to a cache (dx_layer_attach_cache; DX_ERR_INVALID_ARG otherwise).  Both calls
 * synchronise the host with `stream` once: the routing decision is made on the device, the copies are issued by
 * the host.  residual != 0 selects the pre-norm residual form (h_out = h + MoE(RMSNorm(h))) of the next section.
 *   moe_verify_block_cached: routes the block, reads the union back, and evaluates it in waves of at most
 *     slots_per_layer experts -- first the experts the cache already holds (landed or in flight, so that no load
 *     of this block evicts them before use), then the missing ones by ascending id -- each wave staged with
 *     expert_cache_stage and evaluated by one launch of the expert kernel (shared experts with the first wave).
 *     Routing outputs as for moe_verify_block (device, each may be NULL); host_union_ids [min(E,K*k)] /
 *     host_union_count [1] (HOST pointers, may be NULL) receive the union the host read.
 *   moe_draft_step_cached: routes the token, reads the k selected ids back (host_topk_ids [k], HOST pointer, may be
 *     NULL: the predicted verifier experts to hand to dx_controller_propose / expert_cache_prefetch), stages e1 and
 *     evaluates Eq. 5.  (bf16 / 4-bit units: the expert kernel is launched with the routing kernel, on the blob table
 *     as the cache has it; if e1 turns out not to be held it is loaded and evaluated by a second launch.  The cache
 *     sees one expert_cache_stage(e1) per call either way.) */
dx_status moe_verify_block_cached(dx_layer* layer, const float* h, int32_t K, float* y, int32_t residual,
                                  int32_t* topk_ids, float* topk_w, uint64_t* union_mask, int32_t* union_ids,
                                  int32_t* union_count, int32_t* offsets, int32_t* perm, int32_t* host_union_ids,
                                  int32_t* host_union_count, void* stream);
dx_status moe_draft_step_cached(dx_layer* layer, const float* h, float* y, int32_t residual, int32_t* topk_ids,
                                float* topk_w, int32_t* host_topk_ids, void* stream);

/* ---- pre-norm residual forms for layer stacks (synthetic stacks stub attention out) --------------------------
 * h_out = h_in + MoE(RMSNorm(h_in)) with unit gain and eps 1e-6, MoE = Eq. 4 (verify, [K,H]) or Eq. 5 (draft,
 * K = 1).  h_in and h_out must not overlap (a stack alternates two buffers).  Routing outputs as above. */
dx_status moe_verify_block_residual(dx_layer* layer, const float* h_in, float* h_out, int32_t K,
                                    int32_t* topk_ids, float* topk_w, uint64_t* union_mask,
                                    int32_t* union_ids, int32_t* union_count, int32_t* offsets,
                                    int32_t* perm, void* stream);
dx_status moe_draft_step_residual(dx_layer* layer, const float* h_in, float* h_out, int32_t* topk_ids,
                                  float* topk_w, void* stream);
/* moe_draft_step_topr (the shared + top-r self-drafter of Sec. 2.2) in the same residual form. */
dx_status moe_draft_step_topr_residual(dx_layer* layer, const float* h_in, float* h_out, int32_t top_r,
                                       int32_t use_draft_expert, int32_t* topk_ids, float* topk_w, void* stream);

/* ---- the drafter through a whole stack in one launch --------------------------------------------------------
 * The chain  h_{l+1} = moe_draft_step_residual(layer_l, h_l),  l = 0 .. n_layers-1  (Eq. 5 per layer, one
 * token), run by ONE persistent kernel: a draft step reads so few bytes per layer that the gaps between
 * per-layer launches are a visible share of its time, and the weights of layer l+1 can stream while layer l is
 * still being reduced.  dx_stack_create records the layer handles (host array of n_layers handles, all of one
 * context and one shape, bf16 or 4-bit experts (one kind per stack), no expert cache attached; DX_ERR_SHAPE /
 * DX_ERR_UNSUPPORTED otherwise)
 * and owns the scratch rows; the layers must outlive the stack.  moe_draft_stack: h_in, h_out [H] fp32 device,
 * 16-byte aligned, distinct; topk_ids [n_layers, k] int32 and topk_w [n_layers, k] fp32 device or NULL (the
 * selection of every layer, gates as in Eq. 4).  Every expert of every layer must be resident
 * (DX_ERR_NOT_RESIDENT).  The kernel is launched cooperatively (one CTA per SM, all resident at once): a
 * device that cannot place the grid fails the launch with DX_ERR_CUDA.  Its CTAs wait on one another with
 * bounded polls; a wait that runs out sets DX_DEV_WAIT_EXPIRED in dx_device_status and the call's outputs are
 * then undefined.  One call at a time per stack. */
typedef struct dx_stack dx_stack;
dx_status dx_stack_create(dx_ctx* ctx, dx_layer* const* layers, int32_t n_layers, dx_stack** out);
dx_status dx_stack_destroy(dx_stack* stack);
dx_status moe_draft_stack(dx_stack* stack, const float* h_in, float* h_out, int32_t* topk_ids, float* topk_w,
                          void* stream);

/* ---- exact greedy verification: Algorithm 1, "verify" and "accept the target-consistent prefix" -------------
 * h [M,H] fp32: row i is the hidden state that predicts draft token i (M = K, or K+1 to also get the token
 * after a fully accepted block).  W_lm [V,H] in w_dtype.  draft [K] int32.  Outputs (device):
 *   target [M] int32 = argmax_v <W_lm[v], h_i> (lowest v on ties);
 *   n_accept [1] = length of the longest prefix with target[i] == draft[i];
 *   next_token [1] = target[n_accept] if n_accept < M else -1.
 * rms_norm != 0 applies RMSNorm (unit gain, eps 1e-6) to each row of h first.  M <= 16, H <= 8192. */
dx_status spec_accept(dx_ctx* ctx, const float* h, int32_t M, const void* W_lm, int32_t V, int32_t H,
                      int32_t w_dtype, const int32_t* draft, int32_t K, int32_t rms_norm,
                      int32_t* target, int32_t* n_accept, int32_t* next_token, void* stream);

/* ---- drafting one token: Algorithm 1 "Draft v_i" (its LM-head step) and "Compute confidence q_i" -------------------
 * For each of the M rows of h: token[i] = argmax_v <W_lm[v], h_i> and confidence[i] = the softmax probability of
 * that token, q = 1 / sum_v exp(l_v - l_max) (the paper asks only for "a confidence score from the draft logits";
 * the maximum softmax probability is the reading taken).  Same kernels and limits as spec_accept, with an online
 * (max, sum-of-exp) pair carried next to the running argmax.  token [M] int32 and confidence [M] fp32 are device
 * pointers. */
dx_status spec_draft_token(dx_ctx* ctx, const float* h, int32_t M, const void* W_lm, int32_t V, int32_t H,
                           int32_t w_dtype, int32_t rms_norm, int32_t* token, float* confidence, void* stream);

/* ---- confidence-expansion truncation: Sec. 3.4, Eq. 12-14, Algorithm 1 loop body ------------------------------------
 * Host-only.  The controller keeps the predicted block-level verifier set U_hat (Eq. 12) as one bitmask per layer.
 *   reset:   U_hat <- empty (start of a decode step, Algorithm 1 line 1).
 *   propose: candidate token i with confidence q and draft-router predictions predicted[l*k + j] (host ints: the
 *            topk_ids moe_draft_step returned in layer l).  Computes Delta_i = |U_hat_i| - |U_hat| (Eq. 13, counted
 *            in (layer, expert) pairs).  If q < tau and Delta_i > budget (Eq. 14) the candidate is dropped:
 *            *stop_out = 1, U_hat unchanged.  Otherwise *stop_out = 0, U_hat <- U_hat_i, and the new pairs -- the
 *            ones to prefetch -- are listed in new_layers_out / new_experts_out (each sized L*k, may be NULL). */
typedef struct dx_controller dx_controller;
dx_status dx_controller_create(int32_t n_layers, int32_t n_experts, dx_controller** out);
dx_status dx_controller_destroy(dx_controller* c);
dx_status dx_controller_reset(dx_controller* c);
dx_status dx_controller_size(dx_controller* c, int32_t* size_out);
dx_status dx_controller_propose(dx_controller* c, const int32_t* predicted, int32_t k, float q, float tau,
                                int32_t budget, int32_t* delta_out, int32_t* stop_out, int32_t* new_layers_out,
                                int32_t* new_experts_out, int32_t* n_new_out);

/* ---- one decode step of Algorithm 1 over an offloaded stack, as a host loop inside the library -------------------
 * dx_decoder_create: layers[l] must be attached to `cache` as cache layer l (bf16 layers of one shape; shared and
 *   draft experts resident, routed experts registered with the cache).  emb [V,H] bf16 token embeddings (device,
 *   16-byte aligned), W_lm [V,H] bf16 LM head (device); k_max <= 16 tokens drafted per step; tau and budget are the
 *   threshold and the layer-expert budget B_i of Eq. 14 (budget < 0: what is left of the cache's n_layers * slots
 *   pairs once the predictions accepted so far are counted).  Attention is not part of the path: a token's hidden
 *   states depend on its own embedding alone.
 * dx_decoder_step: from the last emitted token t0 -- draft candidates one by one through the drafter's stack (Eq. 5,
 *   moe_draft_step_cached in the residual form; spec_draft_token on RMSNorm of the final row), apply the stop rule
 *   (dx_controller_propose), prefetch the newly predicted experts (expert_cache_prefetch), verify the block through
 *   the target stack (moe_verify_block_cached, residual form) and accept greedily (spec_accept on RMSNorm of the
 *   final rows).  Exactly the calls, in the order, a caller of those entry points would make; the host waits for
 *   `stream` after every routing decision and token.  HOST outputs: drafted [k_max] / n_drafted, n_accept (the
 *   comparison's, or min(scripted_accept, n_drafted) if scripted_accept >= 0 -- for untrained draft experts),
 *   emitted [k_max + 1] / n_emitted (d_1 .. d_n, then the target's token for position n + 1 if a row is left for it),
 *   target [max(1, n_drafted)] (may be NULL), union_sizes [n_layers] (may be NULL). */
typedef struct dx_decoder dx_decoder;
dx_status dx_decoder_create(dx_ctx* ctx, dx_layer* const* layers, int32_t n_layers, dx_cache* cache, const void* emb,
                            const void* W_lm, int32_t V, int32_t k_max, float tau, int32_t budget, dx_decoder** out);
dx_status dx_decoder_destroy(dx_decoder* d);
dx_status dx_decoder_step(dx_decoder* d, int32_t t0, int32_t scripted_accept, int32_t* drafted, int32_t* n_drafted,
                          int32_t* n_accept, int32_t* emitted, int32_t* n_emitted, int32_t* target,
                          int32_t* union_sizes, void* stream);

/* ---- evaluation terms of the self-distillation section (Sec. 3.3); forward only, nothing is trained ---------
 * All pointers are device pointers; K block rows, 1 <= K <= 16; asynchronous on `stream`.
 *
 * moe_missing_residual: Eq. 6 for a block, m[t] = y*_t - S(h_t) - g_{t,e1} E_{e1}(h_t), evaluated as what it is
 *   equal to: the routed sum of Eq. 4 over each row's selected experts except the first, with the gate weights
 *   of the full top-k.  h [K,H] in, m [K,H] out (overwritten); topk_ids [K,k] / topk_w [K,k] optional outputs
 *   (NULL to skip) as in moe_verify_block.  Every routed expert of the layer must be resident.
 * moe_draft_expert_term: gamma * E^d(h_t) for every row, the left operand of Eq. 7.  out [K,H] overwritten.
 *   DX_ERR_UNSUPPORTED for a layer without a draft expert.
 * moe_router_agreement: per row t, kl[t] = KL( R(h*_t) || R(h^d_t) ) -- the summand of Eq. 10 -- and
 *   agree[t] = | TopK(h*_t) & TopK(h^d_t) |, the top-k set agreement tracked beside it.  R is the router's softmax;
 *   for sigmoid routers the scores are divided by their sum first (they are not a distribution otherwise).
 *   h_star, h_draft [K,H]; kl [K] fp32 and agree [K] int32, either may be NULL.  Any K >= 1.
 * dx_squared_error: out[0] = sum_i (a[i] - b[i])^2 over n floats in a fixed order -- with the two calls above,
 *   one layer's term of Eq. 7. */
dx_status moe_missing_residual(dx_layer* layer, const float* h, int32_t K, float* m, int32_t* topk_ids, float* topk_w,
                               void* stream);
dx_status moe_draft_expert_term(dx_layer* layer, const float* h, int32_t K, float* out, void* stream);
dx_status moe_router_agreement(dx_layer* layer, const float* h_star, const float* h_draft, int32_t K, float* kl,
                               int32_t* agree, void* stream);
dx_status dx_squared_error(dx_ctx* ctx, const float* a, const float* b, int64_t n, float* out, void* stream);

/* ---- greedy verification without any allocation ----------------------------------------------------------------
 * (No counterpart in the paper: an addition for callers of this library that cannot allocate device memory --
 * a serving thread whose memory pool was sized once at start-up and where a late cudaMalloc is forbidden or
 * would stall every stream, a plugin that is handed buffers and a stream but no allocator.  dx_create
 * allocates, so such callers cannot use a context.)  Same inputs, outputs and results as spec_accept, but without a context handle: the kernels' scratch
 * (one packed 64-bit argmax key per row and a ticket) is a static device array inside the library, 256-byte
 * aligned and sized for at most 16 rows, which every GPU that loads the library keeps until the process exits.
 * The call performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *   - M > 16 (or any size spec_accept rejects) returns DX_ERR_UNSUPPORTED; nothing is truncated.
 *   - The first call on a device resolves the array's device address (cudaGetSymbolAddress, with that device
 *     current) and reads two device attributes; make that first call before any stream capture.  Host threads
 *     that make the first call on a device at the same time are serialised inside (one does the set-up).
 *   - All calls share the one array, which keeps the previous call's contents; each call clears it on `stream`
 *     first.  Calls that overlap on the GPU (different streams, no ordering between them) race on it and give
 *     undefined results: keep calls to this entry point on one stream or order them yourself.
 * All tensor pointers are device pointers, as for spec_accept. */
dx_status spec_accept_noalloc(const float* h, int32_t M, const void* W_lm, int32_t V, int32_t H, int32_t w_dtype,
                              const int32_t* draft, int32_t K, int32_t rms_norm, int32_t* target,
                              int32_t* n_accept, int32_t* next_token, void* stream);

/* ---- accelerator expert cache: C and P of Algorithm 1, Sec. 3.5 ----------------------------------------------
 * A cache owns n_layers * slots_per_layer HBM slots of blob_bytes each (allocated in create), a side stream
 * for transfers and one event per slot.  With ctx == NULL, create builds a bookkeeping-only cache (no device
 * memory, no copies, streams ignored) that runs the same policy on the host, e.g. to plan or to test it.  Routed experts live in a host pool the caller registers blob by
 * blob (pinned host pointers, borrowed).  All id arrays are HOST pointers.
 *   prefetch: for each id not cached and not in flight, take a free slot, else the least-recently-used slot
 *             that is neither protected (prefetched this step and not used yet) nor pinned, and start a
 *             non-blocking copy on the side stream (Algorithm 1: prefetch U_hat \ (C u P)); never blocks; a
 *             hint that finds no slot is dropped.
 *   stage:    make ids resident now: cached ones are hits; in-flight ones are waited for; the rest are copied
 *             on demand.  `stream` is made to wait (cudaStreamWaitEvent) for exactly the copies it needs.
 *             n must not exceed slots_per_layer (DX_ERR_CACHE_FULL); larger unions are staged in waves.
 *   wait:     like stage but never starts a copy: ids that are neither cached nor in flight give
 *             DX_ERR_NOT_RESIDENT; host-polls outstanding copies up to timeout_s (DX_ERR_TIMEOUT).
 * Results never depend on the cache: it only decides where a blob sits and when it moves. */
typedef struct {
  int64_t lookups;          /* ids asked for by stage / wait */
  int64_t hits;             /* of those, already cached or in flight (no on-demand copy) */
  int64_t on_demand;        /* copies started by stage */
  int64_t prefetch_issued;  /* copies started by prefetch */
  int64_t prefetch_used;    /* prefetched experts later asked for by stage / wait */
  int64_t prefetch_wasted;  /* prefetched experts evicted before any use */
  int64_t evictions;
  int64_t bytes_h2d;
  int64_t waited_copies;    /* copies that had not landed yet when a call needed them -- or, for the drafter's layer
                             * call, which runs its kernels before the selection is known, might need them (the
                             * stream or the host waited) */
  int64_t stall_ns;         /* host time spent polling for such copies in expert_cache_wait */
  int64_t stream_stall_ns;  /* time the compute stream spent waiting for such copies, measured on the device (an event
                             * in front of the waits and one behind them; counted once both have completed, so a
                             * call's waits show up in the statistics read after its work has run) */
} dx_cache_stats;

dx_status expert_cache_create(dx_ctx* ctx, int32_t n_layers, int32_t n_experts, int32_t slots_per_layer,
                              size_t blob_bytes, dx_cache** out);
dx_status expert_cache_destroy(dx_cache* cache);
/* Switch the host pool to 4-bit block-quantised blobs (dx_q4_expert_bytes each; see above): must be called before
 * the first expert_cache_register; DX_ERR_SHAPE if desc/inter do not give the slot size the cache was created
 * with.  bytes_h2d then counts the quantised bytes that actually cross the link. */
dx_status expert_cache_set_q4(dx_cache* cache, const dx_layer_desc* desc, int32_t inter);
dx_status expert_cache_register(dx_cache* cache, int32_t layer, int32_t expert, const void* pinned_host_blob);
/* Start of a decode step (Algorithm 1, line 1: P <- empty): experts prefetched earlier and never used since
 * are counted as wasted and stop being protected from eviction. */
dx_status expert_cache_begin_step(dx_cache* cache);
dx_status expert_cache_prefetch(dx_cache* cache, int32_t layer, const int32_t* host_ids, int32_t n);
dx_status expert_cache_stage(dx_cache* cache, int32_t layer, const int32_t* host_ids, int32_t n, void* stream);
dx_status expert_cache_wait(dx_cache* cache, int32_t layer, const int32_t* host_ids, int32_t n, void* stream,
                            double timeout_s);
dx_status expert_cache_stats(dx_cache* cache, dx_cache_stats* out);
/* Failure-detection aid: queues a host callback that sleeps `milliseconds` (at most 1000) on the cache's copy stream,
 * so that copies issued after it complete that much later -- a slow link made on the host, with which the
 * DX_ERR_TIMEOUT path of expert_cache_wait can be exercised.  Nothing on the GPU waits or spins meanwhile. */
dx_status expert_cache_inject_transfer_delay(dx_cache* cache, int32_t milliseconds);
/* Slot currently holding `expert` of `layer` (-1 if none) and whether its copy is still in flight. */
dx_status expert_cache_query(dx_cache* cache, int32_t layer, int32_t expert, int32_t* slot_out,
                             int32_t* in_flight_out);

#ifdef __cplusplus
}
#endif
#endif /* DRAFTEXPERT_H_ */
