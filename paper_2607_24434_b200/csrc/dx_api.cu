// C-ABI entry points: context and layer handles, argument checking, and the
// launch sequences of the draft step (Eq. 5), the verify block (Eq. 4 grouped
// by the union of Eq. 2 / Eq. 3) and greedy acceptance (Algorithm 1).
#include <new>

#include "dx_internal.cuh"

bool dx_bf16_hidden_supported(int H);
void dx_cache_forget_layer(dx_cache* c, dx_layer* L);

extern "C" const char* dx_status_string(dx_status s) {
  switch (s) {
    case DX_OK: return "ok";
    case DX_ERR_INVALID_ARG: return "invalid argument";
    case DX_ERR_SHAPE: return "shape mismatch";
    case DX_ERR_CUDA: return "CUDA runtime error";
    case DX_ERR_OOM: return "out of memory";
    case DX_ERR_NOT_RESIDENT: return "expert not resident";
    case DX_ERR_TIMEOUT: return "timed out";
    case DX_ERR_CACHE_FULL: return "expert cache full";
    case DX_ERR_UNSUPPORTED: return "unsupported configuration";
    default: return "unknown status";
  }
}

extern "C" dx_status dx_create(int device, dx_ctx** out) {
  if (!out) return DX_ERR_INVALID_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return DX_ERR_CUDA;
  dx_ctx* ctx = new (std::nothrow) dx_ctx();
  if (!ctx) return DX_ERR_OOM;
  ctx->device = device;
  ctx->last_cuda = cudaSuccess;
  ctx->launches = 0;
  ctx->pdl_mask = DX_PDL_ROUTE | DX_PDL_EXPERTS;
  ctx->accept_keep_bytes = 0;
  ctx->wait_limit = DX_WAIT_LIMIT_DEFAULT;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->work, sizeof(DxWork));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->ticket, sizeof(unsigned int) * 4);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->keys, sizeof(unsigned long long) * DX_MAX_M);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->dev_status, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->handover, 4 * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(ctx->handover, 0, 4 * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->conf_part, sizeof(float2) * 8 * ctx->sm_count * DX_MAX_M);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->scratch_i32, sizeof(int32_t) * 2);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->union_dev, sizeof(int32_t) * (DX_MAX_E + 1 + DX_MAX_TOPK));
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&ctx->union_host, sizeof(int32_t) * (DX_MAX_E + 1 + DX_MAX_TOPK),
                                          cudaHostAllocMapped);
  if (e == cudaSuccess) e = cudaHostGetDevicePointer((void**)&ctx->union_host_dev, ctx->union_host, 0);
  if (e == cudaSuccess) e = cudaMemset(ctx->work, 0, sizeof(DxWork));
  if (e == cudaSuccess) e = cudaMemset(ctx->ticket, 0, sizeof(unsigned int) * 4);
  if (e == cudaSuccess) e = cudaMemset(ctx->keys, 0, sizeof(unsigned long long) * DX_MAX_M);
  if (e == cudaSuccess) e = cudaMemset(ctx->dev_status, 0, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    dx_destroy(ctx);
    return e == cudaErrorMemoryAllocation ? DX_ERR_OOM : DX_ERR_CUDA;
  }
  *out = ctx;
  return DX_OK;
}

extern "C" dx_status dx_destroy(dx_ctx* ctx) {
  if (!ctx) return DX_ERR_INVALID_ARG;
  cudaFree(ctx->work);
  cudaFree(ctx->ticket);
  cudaFree(ctx->keys);
  cudaFree(ctx->dev_status);
  cudaFree(ctx->handover);
  cudaFree(ctx->conf_part);
  cudaFree(ctx->scratch_i32);
  cudaFree(ctx->union_dev);
  if (ctx->union_host) cudaFreeHost(ctx->union_host);
  delete ctx;
  return DX_OK;
}

extern "C" dx_status dx_last_device_status(dx_ctx* ctx, void* stream, int32_t* out) {
  if (!ctx || !out) return DX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  DX_CUDA(ctx, cudaMemcpyAsync(out, ctx->dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  DX_CUDA(ctx, cudaMemsetAsync(ctx->dev_status, 0, sizeof(int32_t), st));
  DX_CUDA(ctx, cudaStreamSynchronize(st));
  return DX_OK;
}

extern "C" dx_status dx_set_activation_split(dx_ctx* ctx, int32_t on) {
  if (!ctx) return DX_ERR_INVALID_ARG;
  ctx->act_split = on ? 1 : 0;
  return DX_OK;
}

extern "C" dx_status dx_set_launch_overlap(dx_ctx* ctx, int32_t mask) {
  if (!ctx || mask < 0 || mask > (DX_PDL_ROUTE | DX_PDL_EXPERTS | DX_PDL_ACCEPT)) return DX_ERR_INVALID_ARG;
  ctx->pdl_mask = mask;
  return DX_OK;
}

extern "C" dx_status dx_set_wait_limit(dx_ctx* ctx, uint32_t polls) {
  if (!ctx) return DX_ERR_INVALID_ARG;
  ctx->wait_limit = polls ? polls : DX_WAIT_LIMIT_DEFAULT;
  return DX_OK;
}

extern "C" dx_status dx_set_accept_l2_keep(dx_ctx* ctx, size_t bytes) {
  if (!ctx) return DX_ERR_INVALID_ARG;
  ctx->accept_keep_bytes = bytes;
  return DX_OK;
}

// Small host -> device transfers by a kernel that reads the pinned buffer through its device mapping: a copy-engine
// transfer of a few ten KB costs more in set-up than in time on the link (measured: a 32 KB memcpy node in front of a
// decode step adds 13 us to it, this kernel 4 us).
namespace {
__global__ void dx_stage_block_kernel(uint4* dst, const uint4* src, size_t n16, unsigned char* dst_tail,
                                      const unsigned char* src_tail, int n_tail) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  // a routing kernel behind this one may become resident and fetch its router rows while the link is read; it waits
  // for this grid's completion before it touches the block
  dx_pdl_trigger();
  if (i < n16) {
    uint4 v;   // (a volatile load: the host rewrites the buffer between two calls, nothing may be served from a cache)
    asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(src + i));
    dst[i] = v;
  }
  if (i < (size_t)n_tail) dst_tail[i] = *reinterpret_cast<const volatile unsigned char*>(src_tail + i);
}
}  // namespace

extern "C" dx_status dx_stage_block(dx_ctx* ctx, void* dst, const void* src_host, size_t bytes, void* stream) {
  if (!ctx || !dst || !src_host) return DX_ERR_INVALID_ARG;
  if (bytes == 0) return DX_OK;
  cudaStream_t st = (cudaStream_t)stream;
  void* src_dev = nullptr;
  if (cudaHostGetDevicePointer(&src_dev, const_cast<void*>(src_host), 0) != cudaSuccess) {
    (void)cudaGetLastError();
    return DX_ERR_INVALID_ARG;   // not page-locked (or not mapped): the kernel could not read it
  }
  if (bytes > ((size_t)1 << 20) || ((uintptr_t)dst) % 16 || ((uintptr_t)src_dev) % 16) {
    DX_CUDA(ctx, cudaMemcpyAsync(dst, src_host, bytes, cudaMemcpyHostToDevice, st));   // large or unaligned: the copy engine
    return DX_OK;
  }
  const size_t n16 = bytes / 16;
  const int n_tail = (int)(bytes % 16);
  const size_t threads = n16 > (size_t)n_tail ? n16 : (size_t)n_tail;
  const int grid = (int)((threads + 255) / 256);
  dx_stage_block_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<uint4*>(dst), reinterpret_cast<const uint4*>(src_dev), n16,
                                              reinterpret_cast<unsigned char*>(dst) + n16 * 16,
                                              reinterpret_cast<const unsigned char*>(src_dev) + n16 * 16, n_tail);
  DX_CUDA(ctx, cudaGetLastError());
  ctx->launches++;
  return DX_OK;
}

extern "C" int32_t dx_last_cuda_error(dx_ctx* ctx) { return ctx ? (int32_t)ctx->last_cuda : 0; }
extern "C" int64_t dx_kernel_launches(dx_ctx* ctx) { return ctx ? ctx->launches : 0; }

static dx_status check_desc(const dx_layer_desc* d) {
  if (!d) return DX_ERR_INVALID_ARG;
  if (d->hidden <= 0 || d->n_experts <= 0 || d->top_k <= 0 || d->inter <= 0 || d->n_shared < 0) return DX_ERR_SHAPE;
  if (d->top_k > d->n_experts) return DX_ERR_SHAPE;
  if (d->weight_dtype != DX_DTYPE_FP32 && d->weight_dtype != DX_DTYPE_BF16 && d->weight_dtype != DX_DTYPE_Q4 &&
      d->weight_dtype != DX_DTYPE_BF16_WIDE)
    return DX_ERR_INVALID_ARG;
  if (d->score_fn != DX_SCORE_SOFTMAX && d->score_fn != DX_SCORE_SIGMOID) return DX_ERR_INVALID_ARG;
  if (d->hidden > DX_MAX_H || d->hidden % 256 || d->n_experts > DX_MAX_E || d->top_k > DX_MAX_TOPK ||
      d->n_shared > DX_MAX_SHARED)
    return DX_ERR_UNSUPPORTED;
  if (d->inter % DX_TILE_I || (d->n_shared && (d->shared_inter <= 0 || d->shared_inter % DX_TILE_I)) ||
      d->draft_inter < 0 || d->draft_inter % DX_TILE_I)
    return DX_ERR_UNSUPPORTED;
  if (d->weight_dtype != DX_DTYPE_FP32 && !dx_bf16_hidden_supported(d->hidden)) return DX_ERR_UNSUPPORTED;
  // 4-bit experts: quantisation blocks of 32 along the rows of W_d [hidden, inter]
  if (d->weight_dtype == DX_DTYPE_Q4 &&
      (d->inter % 32 || (d->n_shared && d->shared_inter % 32) || d->draft_inter % 32))
    return DX_ERR_UNSUPPORTED;
  return DX_OK;
}

extern "C" dx_status dx_expert_blob_bytes(const dx_layer_desc* desc, int32_t inter, size_t* bytes_out) {
  if (!desc || !bytes_out) return DX_ERR_INVALID_ARG;
  if (inter <= 0 || inter % DX_TILE_I || desc->hidden <= 0 || desc->hidden % 256) return DX_ERR_UNSUPPORTED;
  if (desc->weight_dtype == DX_DTYPE_Q4) {
    if (inter % 32 || !dx_bf16_hidden_supported(desc->hidden)) return DX_ERR_UNSUPPORTED;
    *bytes_out = (size_t)inter * dx_chunk_bytes(desc->hidden, true);   // inter / 8 units of 8 chunks
    return DX_OK;
  }
  if (desc->weight_dtype == DX_DTYPE_BF16_WIDE && !dx_bf16_hidden_supported(desc->hidden)) return DX_ERR_UNSUPPORTED;
  *bytes_out = (size_t)3 * desc->hidden * inter * (desc->weight_dtype == DX_DTYPE_FP32 ? 4 : 2);
  return DX_OK;
}

extern "C" dx_status dx_pack_expert(dx_ctx* ctx, const dx_layer_desc* desc, int32_t inter, const void* Wg,
                                    const void* Wu, const void* Wd, void* blob_out, void* stream) {
  if (!ctx || !desc || !Wg || !Wu || !Wd || !blob_out) return DX_ERR_INVALID_ARG;
  if (inter <= 0 || inter % DX_TILE_I || desc->hidden <= 0 || desc->hidden % 256) return DX_ERR_UNSUPPORTED;
  if (((uintptr_t)blob_out) % 128) return DX_ERR_INVALID_ARG;
  if (desc->weight_dtype == DX_DTYPE_Q4) {
    if (inter % 32 || !dx_bf16_hidden_supported(desc->hidden)) return DX_ERR_UNSUPPORTED;
    if (((uintptr_t)Wg) % 2 || ((uintptr_t)Wu) % 2 || ((uintptr_t)Wd) % 2) return DX_ERR_INVALID_ARG;
    DX_CUDA(ctx, dx_launch_pack_q4(desc->hidden, inter, Wg, Wu, Wd, blob_out, (cudaStream_t)stream));
  } else if (desc->weight_dtype == DX_DTYPE_BF16_WIDE) {
    if (!dx_bf16_hidden_supported(desc->hidden)) return DX_ERR_UNSUPPORTED;
    DX_CUDA(ctx, dx_launch_pack_wide(desc->hidden, inter, Wg, Wu, Wd, blob_out, (cudaStream_t)stream));
  } else {
    DX_CUDA(ctx, dx_launch_pack(desc->weight_dtype, desc->hidden, inter, Wg, Wu, Wd, blob_out, (cudaStream_t)stream));
  }
  ctx->launches++;
  return DX_OK;
}

extern "C" dx_status dx_q4_expert_bytes(const dx_layer_desc* desc, int32_t inter, size_t* bytes_out) {
  if (!desc || !bytes_out) return DX_ERR_INVALID_ARG;
  if (desc->weight_dtype != DX_DTYPE_BF16 && desc->weight_dtype != DX_DTYPE_Q4) return DX_ERR_UNSUPPORTED;
  // blocks of 32 along the rows of W_g, W_u [inter, hidden] and of W_d [hidden, inter]
  if (inter <= 0 || inter % 32 || desc->hidden <= 0 || desc->hidden % 256) return DX_ERR_UNSUPPORTED;
  *bytes_out = (size_t)3 * desc->hidden * inter / 32 * 18;
  return DX_OK;
}

extern "C" dx_status dx_expand_q4_expert(dx_ctx* ctx, const dx_layer_desc* desc, int32_t inter, const void* q4_blob,
                                         void* blob_out, void* stream) {
  if (!ctx || !desc || !q4_blob || !blob_out) return DX_ERR_INVALID_ARG;
  if (desc->weight_dtype != DX_DTYPE_BF16) return DX_ERR_UNSUPPORTED;   // the result is a bf16 blob
  size_t need = 0;
  dx_status s = dx_q4_expert_bytes(desc, inter, &need);
  if (s != DX_OK) return s;
  if (((uintptr_t)blob_out) % 128 || ((uintptr_t)q4_blob) % 2) return DX_ERR_INVALID_ARG;
  DX_CUDA(ctx, dx_launch_expand_q4(desc->hidden, inter, q4_blob, blob_out, (cudaStream_t)stream));
  ctx->launches++;
  return DX_OK;
}

extern "C" dx_status dx_layer_create(dx_ctx* ctx, const dx_layer_desc* desc, dx_layer** out) {
  if (!ctx || !out) return DX_ERR_INVALID_ARG;
  *out = nullptr;
  dx_status s = check_desc(desc);
  if (s != DX_OK) return s;
  dx_layer* L = new (std::nothrow) dx_layer();
  if (!L) return DX_ERR_OOM;
  L->ctx = ctx;
  L->desc = *desc;
  L->W_r = nullptr;
  L->bias = nullptr;
  L->table_len = desc->n_shared + 1 + desc->n_experts;
  L->table_host = new (std::nothrow) const void*[L->table_len]();
  L->table_dev = nullptr;
  L->dirty = true;
  L->cache = nullptr;
  L->cache_layer = -1;
  if (!L->table_host) { delete L; return DX_ERR_OOM; }
  cudaError_t e = cudaMalloc((void**)&L->table_dev, sizeof(void*) * L->table_len);
  if (e != cudaSuccess) {
    ctx->last_cuda = e;
    delete[] L->table_host;
    delete L;
    return DX_ERR_OOM;
  }
  *out = L;
  return DX_OK;
}

extern "C" dx_status dx_layer_destroy(dx_layer* L) {
  if (!L) return DX_ERR_INVALID_ARG;
  if (L->cache) dx_cache_forget_layer(L->cache, L);   // the cache must not patch a table that is gone
  cudaFree((void*)L->table_dev);
  delete[] L->table_host;
  delete L;
  return DX_OK;
}

extern "C" dx_status dx_layer_set_router(dx_layer* L, const void* W_r, const float* bias) {
  if (!L || !W_r) return DX_ERR_INVALID_ARG;
  if (((uintptr_t)W_r) % 16 || ((uintptr_t)bias) % 4) return DX_ERR_INVALID_ARG;
  L->W_r = W_r;
  L->bias = bias;
  return DX_OK;
}

static dx_status set_slot(dx_layer* L, int idx, const void* blob, bool allow_null) {
  if (!blob && !allow_null) return DX_ERR_INVALID_ARG;
  if (((uintptr_t)blob) % 128) return DX_ERR_INVALID_ARG;
  L->table_host[idx] = blob;
  L->dirty = true;
  return DX_OK;
}
extern "C" dx_status dx_layer_set_shared(dx_layer* L, int32_t s, const void* blob) {
  if (!L || s < 0 || s >= L->desc.n_shared) return DX_ERR_INVALID_ARG;
  return set_slot(L, s, blob, false);
}
extern "C" dx_status dx_layer_set_draft(dx_layer* L, const void* blob) {
  if (!L || L->desc.draft_inter <= 0) return DX_ERR_INVALID_ARG;
  return set_slot(L, L->desc.n_shared, blob, false);
}
extern "C" dx_status dx_layer_set_expert(dx_layer* L, int32_t e, const void* blob) {
  if (!L || e < 0 || e >= L->desc.n_experts) return DX_ERR_INVALID_ARG;
  return set_slot(L, L->desc.n_shared + 1 + e, blob, true);
}

static dx_status upload_table(dx_layer* L, cudaStream_t st) {
  if (!L->dirty) return DX_OK;
  // pageable source: the runtime stages the bytes before returning, the copy itself is stream-ordered
  DX_CUDA(L->ctx, cudaMemcpyAsync((void*)L->table_dev, L->table_host, sizeof(void*) * L->table_len,
                                  cudaMemcpyHostToDevice, st));
  L->dirty = false;
  return DX_OK;
}

struct RouteOut {
  int32_t* topk_ids;
  float* topk_w;
  uint64_t* union_mask;
  int32_t* union_ids;
  int32_t* union_count;
  int32_t* offsets;
  int32_t* perm;
};

static dx_status do_route(dx_layer* L, const float* h, int K, float* y, const RouteOut& o, bool draft, bool residual,
                          cudaStream_t st, int top_r = 1, bool use_draft_expert = true, bool paired = false,
                          bool skip_top1 = false, bool mirror_to_host = false) {
  dx_ctx* ctx = L->ctx;
  const dx_layer_desc& d = L->desc;
  if (!h || !y || h == y) return DX_ERR_INVALID_ARG;
  if (K < 1 || K > DX_MAX_K) return DX_ERR_UNSUPPORTED;
  if (!L->W_r) return DX_ERR_NOT_RESIDENT;
  for (int s = 0; s < d.n_shared; ++s)
    if (!L->table_host[s]) return DX_ERR_NOT_RESIDENT;
  if (draft && use_draft_expert && d.draft_inter > 0 && !L->table_host[d.n_shared]) return DX_ERR_NOT_RESIDENT;
  if (top_r < 0 || top_r > d.top_k) return DX_ERR_INVALID_ARG;
  if (((uintptr_t)h) % 16 || ((uintptr_t)y) % 16) return DX_ERR_INVALID_ARG;
  dx_status s = upload_table(L, st);
  if (s != DX_OK) return s;
  DxRouteParams p{};
  p.h = h; p.K = K; p.H = d.hidden; p.E = d.n_experts; p.k = d.top_k;
  p.score_fn = d.score_fn; p.norm_topk = d.norm_topk; p.scale = d.routed_scale; p.gamma = d.draft_gamma;
  p.W_r = L->W_r; p.bias = L->bias; p.table = L->table_dev;
  p.n_shared = d.n_shared;
  p.shared_tiles = d.n_shared ? d.shared_inter / DX_TILE_I : 0;
  p.routed_tiles = d.inter / DX_TILE_I;
  p.draft_tiles = draft && use_draft_expert ? d.draft_inter / DX_TILE_I : 0;
  p.draft_mode = draft ? 1 : 0;
  p.top_r = top_r;
  p.skip_top1 = skip_top1 ? 1 : 0;
  p.rms_norm = residual ? 1 : 0;
  p.residual = residual ? 1 : 0;
  p.y = y; p.work = ctx->work; p.dev_status = ctx->dev_status;
  p.handover = paired ? ctx->handover : nullptr;
  p.topk_ids = o.topk_ids; p.topk_w = o.topk_w;
  p.union_mask = (unsigned long long*)o.union_mask; p.union_ids = o.union_ids; p.union_count = o.union_count;
  p.offsets = o.offsets; p.perm = o.perm;
  p.host_mirror = mirror_to_host ? ctx->union_host_dev : nullptr;
  // (the router of a layer with 4-bit experts, or with experts in the wide layout, is bf16)
  DX_CUDA(ctx, dx_launch_route(ctx, p, d.weight_dtype == DX_DTYPE_FP32 ? DX_DTYPE_FP32 : DX_DTYPE_BF16, st));
  ctx->launches++;
  return DX_OK;
}

static dx_status do_experts(dx_layer* L, const float* h, int K, float* y, bool draft, bool residual,
                            cudaStream_t st, int first_routed = 0, int n_routed = -1, bool do_static = true,
                            bool paired = false, bool skip_shared = false,
                            const unsigned long long* subset = nullptr, bool tolerate_missing = false) {
  dx_ctx* ctx = L->ctx;
  const dx_layer_desc& d = L->desc;
  if (!h || !y || h == y) return DX_ERR_INVALID_ARG;
  if (K < 1 || K > DX_MAX_K) return DX_ERR_UNSUPPORTED;
  if (((uintptr_t)h) % 16 || ((uintptr_t)y) % 16) return DX_ERR_INVALID_ARG;   // 16-byte loads and reductions
  dx_status s = upload_table(L, st);
  if (s != DX_OK) return s;
  DxExpertParams p{};
  p.x = h;
  p.y = y;
  p.table = L->table_dev;
  p.table_len = L->table_len;
  p.work = ctx->work;
  p.dev_status = ctx->dev_status;
  p.H = d.hidden;
  p.K = K;
  p.rms_norm = residual ? 1 : 0;
  p.n_shared = d.n_shared;
  p.shared_tiles = d.n_shared ? d.shared_inter / DX_TILE_I : 0;
  p.draft_tiles = draft ? d.draft_inter / DX_TILE_I : 0;
  p.routed_tiles = d.inter / DX_TILE_I;
  p.gamma = d.draft_gamma;
  p.handover = paired ? ctx->handover : nullptr;
  p.wait_limit = ctx->wait_limit;
  p.first_routed = first_routed;
  p.n_routed = n_routed;
  p.do_static = do_static ? 1 : 0;
  p.skip_shared = skip_shared ? 1 : 0;
  p.use_subset = subset ? 1 : 0;
  p.tolerate_missing = tolerate_missing ? 1 : 0;
  for (int i = 0; i < DX_MAX_E / 64; ++i) p.subset[i] = subset ? subset[i] : 0ull;
  DX_CUDA(ctx, dx_launch_experts(ctx, p, L->desc.weight_dtype, K, st));
  ctx->launches++;
  if (L->cache) dx_cache_note_use(L->cache, L->cache_layer, st);
  return DX_OK;
}

// Routing kernel and expert kernel of one layer call, launched back to back.  Only here the two kernels use the
// device-side hand-over (bf16 blobs): the routing kernel sets the words, the expert kernel that is certain to
// follow consumes and clears them.
static dx_status do_pair(dx_layer* L, const float* h, int K, float* y, const RouteOut& o, bool draft, bool residual,
                         cudaStream_t st, int top_r = 1, bool use_draft_expert = true) {
  const bool paired = L->desc.weight_dtype != DX_DTYPE_FP32;
  dx_status s = do_route(L, h, K, y, o, draft, residual, st, top_r, use_draft_expert, paired);
  if (s != DX_OK) return s;
  s = do_experts(L, h, K, y, draft && use_draft_expert, residual, st, 0, -1, true, paired);
  if (s != DX_OK && paired) cudaMemsetAsync(L->ctx->handover, 0, 4 * sizeof(unsigned int), st);
  return s;
}

extern "C" dx_status moe_draft_step(dx_layer* L, const float* h, float* y, int32_t* topk_ids, float* topk_w,
                                    void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  RouteOut o{topk_ids, topk_w, nullptr, nullptr, nullptr, nullptr, nullptr};
  return do_pair(L, h, 1, y, o, true, false, st);
}

extern "C" dx_status moe_draft_step_residual(dx_layer* L, const float* h_in, float* h_out, int32_t* topk_ids,
                                             float* topk_w, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  RouteOut o{topk_ids, topk_w, nullptr, nullptr, nullptr, nullptr, nullptr};
  return do_pair(L, h_in, 1, h_out, o, true, true, st);
}

extern "C" dx_status moe_verify_route(dx_layer* L, const float* h, int32_t K, float* y, int32_t* topk_ids,
                                      float* topk_w, uint64_t* union_mask, int32_t* union_ids, int32_t* union_count,
                                      int32_t* offsets, int32_t* perm, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  RouteOut o{topk_ids, topk_w, union_mask, union_ids, union_count, offsets, perm};
  return do_route(L, h, K, y, o, false, false, (cudaStream_t)stream);
}

extern "C" dx_status moe_verify_experts(dx_layer* L, const float* h, int32_t K, float* y, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  return do_experts(L, h, K, y, false, false, (cudaStream_t)stream);
}

extern "C" dx_status moe_verify_experts_range(dx_layer* L, const float* h, int32_t K, float* y, int32_t first_union,
                                              int32_t n_union, int32_t include_shared, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  if (first_union < 0 || n_union < 0) return DX_ERR_INVALID_ARG;
  return do_experts(L, h, K, y, false, false, (cudaStream_t)stream, first_union, n_union, include_shared != 0);
}

extern "C" dx_status moe_draft_step_topr(dx_layer* L, const float* h, float* y, int32_t top_r,
                                         int32_t use_draft_expert, int32_t* topk_ids, float* topk_w, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  RouteOut o{topk_ids, topk_w, nullptr, nullptr, nullptr, nullptr, nullptr};
  if (top_r < 1) return DX_ERR_INVALID_ARG;
  return do_pair(L, h, 1, y, o, true, false, st, top_r, use_draft_expert != 0);
}

extern "C" dx_status moe_draft_step_topr_residual(dx_layer* L, const float* h_in, float* h_out, int32_t top_r,
                                                  int32_t use_draft_expert, int32_t* topk_ids, float* topk_w,
                                                  void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  RouteOut o{topk_ids, topk_w, nullptr, nullptr, nullptr, nullptr, nullptr};
  if (top_r < 1) return DX_ERR_INVALID_ARG;
  return do_pair(L, h_in, 1, h_out, o, true, true, (cudaStream_t)stream, top_r, use_draft_expert != 0);
}

extern "C" dx_status moe_draft_route(dx_layer* L, const float* h, float* y, int32_t* topk_ids, float* topk_w,
                                     void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  RouteOut o{topk_ids, topk_w, nullptr, nullptr, nullptr, nullptr, nullptr};
  return do_route(L, h, 1, y, o, true, false, (cudaStream_t)stream);
}

extern "C" dx_status moe_draft_experts(dx_layer* L, const float* h, float* y, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  return do_experts(L, h, 1, y, true, false, (cudaStream_t)stream);
}

extern "C" dx_status moe_verify_block(dx_layer* L, const float* h, int32_t K, float* y, int32_t* topk_ids,
                                      float* topk_w, uint64_t* union_mask, int32_t* union_ids, int32_t* union_count,
                                      int32_t* offsets, int32_t* perm, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  RouteOut o{topk_ids, topk_w, union_mask, union_ids, union_count, offsets, perm};
  return do_pair(L, h, K, y, o, false, false, (cudaStream_t)stream);
}

extern "C" dx_status moe_verify_block_residual(dx_layer* L, const float* h_in, float* h_out, int32_t K,
                                               int32_t* topk_ids, float* topk_w, uint64_t* union_mask,
                                               int32_t* union_ids, int32_t* union_count, int32_t* offsets,
                                               int32_t* perm, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  RouteOut o{topk_ids, topk_w, union_mask, union_ids, union_count, offsets, perm};
  return do_pair(L, h_in, K, h_out, o, false, true, st);
}

// ---- layers whose routed experts come through an expert cache (Sec. 3.5, Algorithm 1) ------------------------
int dx_cache_slot_of(const dx_cache* c, int layer, int expert);
int dx_cache_slots(const dx_cache* c);

// The one round trip on-demand loading needs (the routing decision is made on the device, the copies are issued by
// the host): the routing kernel itself writes what the host needs into page-locked host memory (a device -> host copy
// behind it costs ~10 us of copy-engine set-up for a few ten bytes), and the host waits for the stream.
static dx_status wait_for_routing(dx_ctx* ctx, cudaStream_t st) {
  DX_CUDA(ctx, cudaStreamSynchronize(st));
  return DX_OK;
}

extern "C" dx_status moe_verify_block_cached(dx_layer* L, const float* h, int32_t K, float* y, int32_t residual,
                                             int32_t* topk_ids, float* topk_w, uint64_t* union_mask,
                                             int32_t* union_ids, int32_t* union_count, int32_t* offsets,
                                             int32_t* perm, int32_t* host_union_ids, int32_t* host_union_count,
                                             void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  if (!L->cache) return DX_ERR_INVALID_ARG;
  dx_ctx* ctx = L->ctx;
  dx_cache* c = L->cache;
  cudaStream_t st = (cudaStream_t)stream;
  const int E = L->desc.n_experts;
  // the union goes to the context's scratch if the caller does not want it, and from there to the host
  int32_t* uid = union_ids ? union_ids : ctx->union_dev;
  int32_t* ucnt = union_count ? union_count : ctx->union_dev + DX_MAX_E;
  RouteOut o{topk_ids, topk_w, union_mask, uid, ucnt, offsets, perm};
  dx_status s = do_route(L, h, K, y, o, false, residual != 0, st, 1, true, false, false, true);
  if (s != DX_OK) return s;
  const int cap = E < K * L->desc.top_k ? E : K * L->desc.top_k;
  s = wait_for_routing(ctx, st);
  if (s != DX_OK) return s;
  const int n = ctx->union_host[DX_MAX_E];
  if (n < 0 || n > cap) return DX_ERR_CUDA;
  if (host_union_count) *host_union_count = n;
  if (host_union_ids)
    for (int i = 0; i < n; ++i) host_union_ids[i] = ctx->union_host[i];
  // Waves of at most S experts: the ones the cache already holds (landed or in flight) first, so that no load of
  // this block can evict them before they are used, then the missing ones in ascending id order.
  const int S = dx_cache_slots(c);
  int32_t order[DX_MAX_E];
  int m = 0;
  for (int i = 0; i < n; ++i)
    if (dx_cache_slot_of(c, L->cache_layer, ctx->union_host[i]) >= 0) order[m++] = ctx->union_host[i];
  for (int i = 0; i < n; ++i)
    if (dx_cache_slot_of(c, L->cache_layer, ctx->union_host[i]) < 0) order[m++] = ctx->union_host[i];
  int first = 0;
  do {
    const int cnt = n - first < S ? n - first : S;
    unsigned long long subset[DX_MAX_E / 64] = {};
    for (int i = 0; i < cnt; ++i) subset[order[first + i] >> 6] |= 1ull << (order[first + i] & 63);
    s = expert_cache_stage(c, L->cache_layer, order + first, cnt, stream);
    if (s != DX_OK) return s;
    s = do_experts(L, h, K, y, false, residual != 0, st, 0, -1, first == 0, false, false, subset);
    if (s != DX_OK) return s;
    first += cnt;
  } while (first < n);
  return DX_OK;
}

extern "C" dx_status moe_draft_step_cached(dx_layer* L, const float* h, float* y, int32_t residual,
                                           int32_t* topk_ids, float* topk_w, int32_t* host_topk_ids, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  if (!L->cache) return DX_ERR_INVALID_ARG;
  dx_ctx* ctx = L->ctx;
  cudaStream_t st = (cudaStream_t)stream;
  const int k = L->desc.top_k;
  int32_t* ids = topk_ids ? topk_ids : ctx->union_dev + DX_MAX_E + 1;
  RouteOut o{ids, topk_w, nullptr, nullptr, nullptr, nullptr, nullptr};
  int32_t* host = ctx->union_host + DX_MAX_E + 1;
  dx_status s;
  const int dt = L->desc.weight_dtype;
  if ((dt == DX_DTYPE_BF16 || dt == DX_DTYPE_Q4) && dx_cache_layer_quiet(L->cache, L->cache_layer)) {
    // Most selections are of experts the cache already holds, so -- while none of the layer's copies is in flight:
    // otherwise the stream would have to wait for all of them, not just for the one it may need -- the expert kernel
    // is launched beside the routing kernel, as for a resident layer, before the host knows the selection: the blob
    // table is first brought up to date (it then names exactly what the cache holds), the kernel leaves a routed
    // expert out if the table has no blob for it, and only in that case the expert is loaded and evaluated by a
    // second launch.  The cache sees the same calls in the same order either way.
    s = dx_cache_prepare_layer(L->cache, L->cache_layer, st);
    if (s != DX_OK) return s;
    s = do_route(L, h, 1, y, o, true, residual != 0, st, 1, true, true, false, true);
    if (s != DX_OK) return s;
    s = do_experts(L, h, 1, y, true, residual != 0, st, 0, -1, true, true, false, nullptr, true);
    if (s != DX_OK) { cudaMemsetAsync(ctx->handover, 0, 4 * sizeof(unsigned int), st); return s; }
    s = wait_for_routing(ctx, st);
    if (s != DX_OK) return s;
    if (host_topk_ids)
      for (int j = 0; j < k; ++j) host_topk_ids[j] = host[j];
    const int32_t e1 = host[0];
    if (e1 < 0 || e1 >= L->desc.n_experts) return DX_ERR_CUDA;
    const bool was_resident = dx_cache_slot_of(L->cache, L->cache_layer, e1) >= 0;
    s = expert_cache_stage(L->cache, L->cache_layer, &e1, 1, stream);   // the bookkeeping of a hit, or the load
    if (s != DX_OK || was_resident) return s;
    return do_experts(L, h, 1, y, true, residual != 0, st, 0, -1, false);   // the routed expert alone, now that it is there
  }
  s = do_route(L, h, 1, y, o, true, residual != 0, st, 1, true, false, false, true);
  if (s != DX_OK) return s;
  s = wait_for_routing(ctx, st);
  if (s != DX_OK) return s;
  if (host_topk_ids)
    for (int j = 0; j < k; ++j) host_topk_ids[j] = host[j];
  const int32_t e1 = host[0];
  s = expert_cache_stage(L->cache, L->cache_layer, &e1, 1, stream);   // hit, in flight (waited for) or on demand
  if (s != DX_OK) return s;
  return do_experts(L, h, 1, y, true, residual != 0, st);
}

// ---- exercising the bounded waits without a fault -------------------------------------------------------------
extern "C" dx_status dx_selftest_wait_expiry(dx_layer* L, const float* h, int32_t K, float* y, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  dx_ctx* ctx = L->ctx;
  if (L->desc.weight_dtype == DX_DTYPE_FP32) return DX_ERR_UNSUPPORTED;   // the fp32 kernels have no hand-over
  if (ctx->wait_limit > (1u << 16)) return DX_ERR_INVALID_ARG;            // keep the give-up short: set a limit first
  cudaStream_t st = (cudaStream_t)stream;
  // hand-over words as a routing kernel leaves them before it publishes anything, and then no routing kernel
  DX_CUDA(ctx, cudaMemsetAsync(ctx->handover, 0, 4 * sizeof(unsigned int), st));
  DX_CUDA(ctx, cudaMemsetAsync(ctx->work, 0, sizeof(DxWork), st));
  return do_experts(L, h, K, y, false, false, st, 0, -1, true, true);
}

// ---- draft stack: Eq. 5 through a whole stack of layers in one persistent kernel -----------------------------
extern "C" dx_status dx_stack_create(dx_ctx* ctx, dx_layer* const* layers, int32_t n_layers, dx_stack** out) {
  if (!ctx || !layers || !out) return DX_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_layers < 1 || n_layers > 1024) return DX_ERR_UNSUPPORTED;
  for (int l = 0; l < n_layers; ++l) {
    dx_layer* L = layers[l];
    if (!L || L->ctx != ctx) return DX_ERR_INVALID_ARG;
    const dx_layer_desc &d = L->desc, &d0 = layers[0]->desc;
    if ((d.weight_dtype != DX_DTYPE_BF16 && d.weight_dtype != DX_DTYPE_Q4) || L->cache)
      return DX_ERR_UNSUPPORTED;   // resident bf16 / 4-bit experts in the streaming layout only
    if (d.weight_dtype != d0.weight_dtype) return DX_ERR_SHAPE;
    if (d.hidden != d0.hidden || d.n_experts != d0.n_experts || d.top_k != d0.top_k || d.inter != d0.inter ||
        d.n_shared != d0.n_shared || d.shared_inter != d0.shared_inter || d.draft_inter != d0.draft_inter ||
        d.score_fn != d0.score_fn || d.norm_topk != d0.norm_topk || d.routed_scale != d0.routed_scale)
      return DX_ERR_SHAPE;
    if (!L->W_r) return DX_ERR_NOT_RESIDENT;
  }
  dx_stack* s = new (std::nothrow) dx_stack();
  if (!s) return DX_ERR_OOM;
  s->ctx = ctx;
  s->n_layers = n_layers;
  s->layers = new (std::nothrow) dx_layer*[n_layers];
  s->desc_host = new (std::nothrow) DxStackLayer[n_layers]();
  s->desc_dev = nullptr; s->scratch = nullptr;
  if (!s->layers || !s->desc_host) { delete[] s->layers; delete[] s->desc_host; delete s; return DX_ERR_OOM; }
  for (int l = 0; l < n_layers; ++l) s->layers[l] = layers[l];
  const dx_layer_desc& d = layers[0]->desc;
  cudaError_t e = cudaMalloc(&s->desc_dev, sizeof(DxStackLayer) * n_layers);
  s->zword_off = sizeof(float) * (size_t)n_layers * DX_STACK_COPIES * d.hidden;
  s->sync_off = s->zword_off + sizeof(unsigned long long) * (size_t)n_layers * d.n_experts;
  s->scratch_bytes = s->sync_off + sizeof(unsigned int) * n_layers;
  if (e == cudaSuccess) e = cudaMalloc(&s->scratch, s->scratch_bytes);
  if (e != cudaSuccess) {
    ctx->last_cuda = e;
    dx_stack_destroy(s);
    return e == cudaErrorMemoryAllocation ? DX_ERR_OOM : DX_ERR_CUDA;
  }
  *out = s;
  return DX_OK;
}

extern "C" dx_status dx_stack_destroy(dx_stack* s) {
  if (!s) return DX_ERR_INVALID_ARG;
  cudaFree(s->desc_dev);
  cudaFree(s->scratch);
  delete[] s->layers;
  delete[] s->desc_host;
  delete s;
  return DX_OK;
}

extern "C" dx_status moe_draft_stack(dx_stack* s, const float* h_in, float* h_out, int32_t* topk_ids, float* topk_w,
                                     void* stream) {
  if (!s || !h_in || !h_out || h_in == h_out) return DX_ERR_INVALID_ARG;
  if (((uintptr_t)h_in) % 16 || ((uintptr_t)h_out) % 16) return DX_ERR_INVALID_ARG;
  dx_ctx* ctx = s->ctx;
  cudaStream_t st = (cudaStream_t)stream;
  const dx_layer_desc& d = s->layers[0]->desc;
  // every expert of every layer has to be resident, and the layers' tables and the descriptors up to date
  bool changed = false;
  for (int l = 0; l < s->n_layers; ++l) {
    dx_layer* L = s->layers[l];
    for (int i = 0; i < L->table_len; ++i)
      if (!L->table_host[i] && !(i == d.n_shared && d.draft_inter == 0)) return DX_ERR_NOT_RESIDENT;
    dx_status u = upload_table(L, st);
    if (u != DX_OK) return u;
    DxStackLayer now{};
    now.table = L->table_dev;
    now.W_r = L->W_r;
    now.bias = L->bias;
    now.gamma = L->desc.draft_gamma;
    DxStackLayer& have = s->desc_host[l];
    if (have.table != now.table || have.W_r != now.W_r || have.bias != now.bias || have.gamma != now.gamma) {
      have = now;
      changed = true;
    }
  }
  // (the source outlives the copy: it belongs to the stack)
  cudaError_t e = cudaSuccess;
  if (changed)
    e = cudaMemcpyAsync(s->desc_dev, s->desc_host, sizeof(DxStackLayer) * s->n_layers, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(s->scratch, 0, s->scratch_bytes, st);
  DX_CUDA(ctx, e);
  DxStackParams p{};
  p.layers = s->desc_dev;
  p.n_layers = s->n_layers;
  p.h_in = h_in;
  p.h_out = h_out;
  p.delta = reinterpret_cast<float*>(s->scratch);
  p.zword = reinterpret_cast<unsigned long long*>(s->scratch + s->zword_off);
  p.sync = reinterpret_cast<unsigned int*>(s->scratch + s->sync_off);
  p.topk_ids = topk_ids;
  p.topk_w = topk_w;
  p.dev_status = ctx->dev_status;
  p.H = d.hidden; p.E = d.n_experts; p.k = d.top_k; p.score_fn = d.score_fn; p.norm_topk = d.norm_topk;
  p.scale = d.routed_scale;
  p.n_shared = d.n_shared;
  p.shared_tiles = d.n_shared ? d.shared_inter / DX_TILE_I : 0;
  p.draft_tiles = d.draft_inter / DX_TILE_I;
  p.routed_tiles = d.inter / DX_TILE_I;
  p.q4 = d.weight_dtype == DX_DTYPE_Q4 ? 1 : 0;
  p.wait_limit = ctx->wait_limit;
  DX_CUDA(ctx, dx_launch_draft_stack(ctx, p, st));
  ctx->launches++;
  return DX_OK;
}

// ---- evaluation terms of Sec. 3.3 (no training involved) -----------------------------------------------------
extern "C" dx_status moe_missing_residual(dx_layer* L, const float* h, int32_t K, float* m, int32_t* topk_ids,
                                          float* topk_w, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  RouteOut o{topk_ids, topk_w, nullptr, nullptr, nullptr, nullptr, nullptr};
  // Eq. 6 is the routed sum of Eq. 4 without each row's first selected expert: same kernels, that pair's weight
  // set to zero (and its expert left out of the union unless another pair selects it), shared experts skipped
  dx_status s = do_route(L, h, K, m, o, false, false, st, 1, true, false, true);
  if (s != DX_OK) return s;
  return do_experts(L, h, K, m, false, false, st, 0, -1, false);
}

extern "C" dx_status moe_draft_expert_term(dx_layer* L, const float* h, int32_t K, float* out, void* stream) {
  if (!L) return DX_ERR_INVALID_ARG;
  if (L->desc.draft_inter <= 0) return DX_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  RouteOut o{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  // gamma * E^d(h_t) for K rows: the drafter's kernels with no routed group and the shared experts skipped
  dx_status s = do_route(L, h, K, out, o, true, false, st, 0, true);
  if (s != DX_OK) return s;
  return do_experts(L, h, K, out, true, false, st, 0, -1, true, false, true);
}

extern "C" dx_status moe_router_agreement(dx_layer* L, const float* h_star, const float* h_draft, int32_t K, float* kl,
                                          int32_t* agree, void* stream) {
  if (!L || !h_star || !h_draft || (!kl && !agree)) return DX_ERR_INVALID_ARG;
  if (K < 1) return DX_ERR_SHAPE;
  if (!L->W_r) return DX_ERR_NOT_RESIDENT;
  DX_CUDA(L->ctx, dx_launch_router_agreement(L, h_star, h_draft, K, kl, agree, (cudaStream_t)stream));
  L->ctx->launches++;
  return DX_OK;
}

extern "C" dx_status dx_squared_error(dx_ctx* ctx, const float* a, const float* b, int64_t n, float* out,
                                      void* stream) {
  if (!ctx || !a || !b || !out) return DX_ERR_INVALID_ARG;
  if (n < 0) return DX_ERR_SHAPE;
  DX_CUDA(ctx, dx_launch_squared_error(a, b, (long long)n, out, (cudaStream_t)stream));
  ctx->launches++;
  return DX_OK;
}

extern "C" dx_status spec_accept(dx_ctx* ctx, const float* h, int32_t M, const void* W_lm, int32_t V, int32_t H,
                                 int32_t w_dtype, const int32_t* draft, int32_t K, int32_t rms_norm, int32_t* target,
                                 int32_t* n_accept, int32_t* next_token, void* stream) {
  if (!ctx || !h || !W_lm || !target || !n_accept || !next_token) return DX_ERR_INVALID_ARG;
  if (K > 0 && !draft) return DX_ERR_INVALID_ARG;
  if (M < 1 || V < 1 || K < 0) return DX_ERR_SHAPE;
  if (w_dtype != DX_DTYPE_FP32 && w_dtype != DX_DTYPE_BF16) return DX_ERR_INVALID_ARG;
  if (M > DX_MAX_M || K > DX_MAX_K || H <= 0 || H > DX_MAX_H || H % 256) return DX_ERR_UNSUPPORTED;
  if (((uintptr_t)h) % 16 || ((uintptr_t)W_lm) % 16) return DX_ERR_INVALID_ARG;
  if (w_dtype == DX_DTYPE_BF16) {
    const size_t smem = (size_t)((M + 7) / 8) * H * 32;
    if (smem > (size_t)ctx->smem_optin) return DX_ERR_UNSUPPORTED;
  }
  DX_CUDA(ctx, dx_launch_accept(ctx, h, M, W_lm, V, H, w_dtype, draft, K, rms_norm, target, n_accept, next_token,
                                nullptr, (cudaStream_t)stream));
  ctx->launches++;
  return DX_OK;
}

extern "C" dx_status spec_draft_token(dx_ctx* ctx, const float* h, int32_t M, const void* W_lm, int32_t V, int32_t H,
                                      int32_t w_dtype, int32_t rms_norm, int32_t* token, float* confidence,
                                      void* stream) {
  if (!ctx || !h || !W_lm || !token || !confidence) return DX_ERR_INVALID_ARG;
  if (M < 1 || V < 1) return DX_ERR_SHAPE;
  if (w_dtype != DX_DTYPE_FP32 && w_dtype != DX_DTYPE_BF16) return DX_ERR_INVALID_ARG;
  if (M > DX_MAX_M || H <= 0 || H > DX_MAX_H || H % 256) return DX_ERR_UNSUPPORTED;
  if (((uintptr_t)h) % 16 || ((uintptr_t)W_lm) % 16) return DX_ERR_INVALID_ARG;
  if (w_dtype == DX_DTYPE_BF16 && (size_t)((M + 7) / 8) * H * 32 > (size_t)ctx->smem_optin) return DX_ERR_UNSUPPORTED;
  DX_CUDA(ctx, dx_launch_accept(ctx, h, M, W_lm, V, H, w_dtype, nullptr, 0, rms_norm, token, ctx->scratch_i32,
                                ctx->scratch_i32 + 1, confidence, (cudaStream_t)stream));
  ctx->launches++;
  return DX_OK;
}
