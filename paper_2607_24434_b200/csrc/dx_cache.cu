// Accelerator expert cache (Sec. 3.5 and Algorithm 1: cache C, in-flight set P).
//
// Host-side state machine plus the transfers it drives.  Per layer there are S
// HBM slots of one expert blob each.  Routed experts live in pinned host memory
// (registered blob by blob) and are copied into slots with cudaMemcpyAsync on
// one side stream, so transfers are ordered among themselves and overlap with
// compute; one event per slot lets the compute stream wait for exactly the
// copies it needs.  The layer's device blob table is patched on the compute
// stream (tiny kernel, entries passed by value) right before the kernels that
// read it.  Policy (deterministic given the call sequence):
//   - stamp = global access counter; a hit, a prefetch and an on-demand load set stamp = now;
//   - P = slots prefetched since the last begin_step and not used yet: they are "protected";
//   - prefetch victim: free slot (lowest index), else least-recently-used unprotected slot, else drop the hint;
//   - stage victim:    free slot, else LRU unprotected slot not pinned by this call, else LRU protected
//                      slot not pinned by this call (counted as a wasted prefetch), else DX_ERR_CACHE_FULL;
//   - an id already cached (landed or in flight) is never copied again.
// With ctx == NULL the cache is bookkeeping only: the same policy without device memory or copies.
#include <chrono>
#include <new>
#include <thread>
#include <vector>

#include "dx_internal.cuh"

struct DxSlot {
  int expert = -1;
  unsigned long long stamp = 0;
  bool prefetched = false;   // member of P: prefetched this step, not used yet
  bool copy_pending = false; // a copy was issued and not yet seen complete
  bool ev_valid = false;     // the event has been recorded at least once
  cudaEvent_t ev = nullptr;
};

struct DxTablePatch {
  int n;
  int idx[32];
  const void* ptr[32];
};

struct dx_cache {
  dx_ctx* ctx;
  int L, E, S;
  size_t blob_bytes;
  unsigned char* slab;
  // quantised host pool: registered blobs are 4-bit block-quantised (q4_bytes each); a copy lands in the slot's
  // staging area and is expanded into the slot on a stream of its own, so that the link goes on with the next copy
  size_t q4_bytes;
  int q4_hidden, q4_inter;
  unsigned char* staging;
  cudaStream_t copy_stream;
  cudaStream_t expand_stream;           // (quantised pool) staging area -> slot
  cudaEvent_t staged_ev;                // (quantised pool) the copy in front of an expansion has landed
  unsigned long long clock;
  dx_cache_stats stats;
  std::vector<const void*> host_blob;   // [L*E]
  std::vector<DxSlot> slots;            // [L*S]
  std::vector<int> slot_of;             // [L*E] -> slot or -1
  std::vector<dx_layer*> layer;         // attached layer per cache layer
  std::vector<cudaEvent_t> used_ev;     // last compute use of the layer's slots
  std::vector<char> used_valid;
  std::vector<std::vector<std::pair<int, const void*>>> pending;   // table patches not yet applied, per layer
  // the compute stream's waits for copies, timed on the device: (event in front, event behind) pairs not yet read,
  // and events free for reuse
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> stall_open;
  std::vector<cudaEvent_t> stall_free;
};

namespace {

__global__ void dx_table_patch_kernel(const void** table, int table_len, int32_t* dev_status, DxTablePatch patch) {
  dx_pdl_wait();
  if ((int)threadIdx.x < patch.n &&
      DX_BOUNDS(patch.idx[threadIdx.x] >= 0 && patch.idx[threadIdx.x] < table_len, dev_status))
    table[patch.idx[threadIdx.x]] = patch.ptr[threadIdx.x];
}

inline DxSlot& slot_ref(dx_cache* c, int layer, int s) { return c->slots[(size_t)layer * c->S + s]; }
inline void* slot_ptr(dx_cache* c, int layer, int s) {
  return c->slab ? c->slab + ((size_t)layer * c->S + s) * c->blob_bytes : nullptr;
}
inline void* staging_ptr(dx_cache* c, int layer, int s) {
  return c->staging + ((size_t)layer * c->S + s) * ((c->q4_bytes + 255) / 256 * 256);
}

// victim search; protected_ok: may take a slot of P; pinned: slots of the call in progress
int find_victim(dx_cache* c, int layer, const std::vector<char>& pinned, bool protected_ok, bool* was_protected) {
  *was_protected = false;
  for (int s = 0; s < c->S; ++s)
    if (slot_ref(c, layer, s).expert < 0 && !pinned[s]) return s;
  int best = -1;
  for (int s = 0; s < c->S; ++s) {
    const DxSlot& sl = slot_ref(c, layer, s);
    if (pinned[s] || sl.prefetched) continue;
    if (best < 0 || sl.stamp < slot_ref(c, layer, best).stamp) best = s;
  }
  if (best >= 0 || !protected_ok) return best;
  for (int s = 0; s < c->S; ++s) {
    const DxSlot& sl = slot_ref(c, layer, s);
    if (pinned[s]) continue;
    if (best < 0 || sl.stamp < slot_ref(c, layer, best).stamp) best = s;
  }
  if (best >= 0) *was_protected = true;
  return best;
}

// puts expert e of `layer` into slot s (evicting what is there) and starts the copy
dx_status load_into(dx_cache* c, int layer, int s, int e, bool as_prefetch) {
  DxSlot& sl = slot_ref(c, layer, s);
  if (sl.expert >= 0) {
    c->stats.evictions++;
    c->slot_of[(size_t)layer * c->E + sl.expert] = -1;
    c->pending[layer].push_back({sl.expert, nullptr});
  }
  sl.expert = e;
  sl.prefetched = as_prefetch;
  sl.stamp = ++c->clock;
  c->slot_of[(size_t)layer * c->E + e] = s;
  c->pending[layer].push_back({e, slot_ptr(c, layer, s)});
  c->stats.bytes_h2d += (int64_t)(c->q4_bytes ? c->q4_bytes : c->blob_bytes);
  if (c->ctx) {
    // the slot may still be read by kernels already enqueued on the compute stream
    if (c->used_valid[layer]) {
      cudaError_t e0 = cudaStreamWaitEvent(c->copy_stream, c->used_ev[layer], 0);
      if (e0 != cudaSuccess) { c->ctx->last_cuda = e0; return DX_ERR_CUDA; }
    }
    cudaError_t e1;
    if (c->q4_bytes) {
      // a quarter of the bytes cross the host link; the expansion to the streaming layout runs at HBM speed, behind
      // the copy but on the expansion stream (the staging area of a slot is overwritten by the copy stream only
      // after the slot's previous expansion, which the slot's event marks, has run)
      e1 = sl.ev_valid ? cudaStreamWaitEvent(c->copy_stream, sl.ev, 0) : cudaSuccess;
      if (e1 == cudaSuccess)
        e1 = cudaMemcpyAsync(staging_ptr(c, layer, s), c->host_blob[(size_t)layer * c->E + e], c->q4_bytes,
                             cudaMemcpyHostToDevice, c->copy_stream);
      if (e1 == cudaSuccess) e1 = cudaEventRecord(c->staged_ev, c->copy_stream);
      if (e1 == cudaSuccess) e1 = cudaStreamWaitEvent(c->expand_stream, c->staged_ev, 0);
      if (e1 == cudaSuccess)
        e1 = dx_launch_expand_q4(c->q4_hidden, c->q4_inter, staging_ptr(c, layer, s), slot_ptr(c, layer, s),
                                 c->expand_stream);
      if (e1 == cudaSuccess) c->ctx->launches++;
      if (e1 == cudaSuccess) e1 = cudaEventRecord(sl.ev, c->expand_stream);
      if (e1 != cudaSuccess) { c->ctx->last_cuda = e1; return DX_ERR_CUDA; }
      sl.ev_valid = true;
      sl.copy_pending = true;
      return DX_OK;
    } else {
      e1 = cudaMemcpyAsync(slot_ptr(c, layer, s), c->host_blob[(size_t)layer * c->E + e], c->blob_bytes,
                           cudaMemcpyHostToDevice, c->copy_stream);
    }
    if (e1 == cudaSuccess) e1 = cudaEventRecord(sl.ev, c->copy_stream);
    if (e1 != cudaSuccess) { c->ctx->last_cuda = e1; return DX_ERR_CUDA; }
    sl.copy_pending = true;
  }
  return DX_OK;
}

bool copy_done(dx_cache* c, DxSlot& sl) {
  if (!sl.copy_pending) return true;
  if (!c->ctx) { sl.copy_pending = false; return true; }
  if (cudaEventQuery(sl.ev) == cudaSuccess) { sl.copy_pending = false; return true; }
  return false;
}

// A timed event (from the free list, or a new one); null if none can be had (the wait is then simply not timed).
cudaEvent_t stall_event(dx_cache* c) {
  if (!c->stall_free.empty()) { cudaEvent_t e = c->stall_free.back(); c->stall_free.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
  return e;
}
// Makes `st` wait for the copies of the slots `want` marks that are still in flight, with an event in front of the
// waits and one behind them.  Returns how many copies were waited for.
int wait_for_copies(dx_cache* c, int layer, const std::vector<char>* want, cudaStream_t st, cudaError_t* err) {
  *err = cudaSuccess;
  int n = 0;
  cudaEvent_t a = nullptr;
  for (int s = 0; s < c->S; ++s) {
    if (want && !(*want)[s]) continue;
    DxSlot& sl = slot_ref(c, layer, s);
    if (sl.expert < 0 || copy_done(c, sl)) continue;
    if (n == 0) {
      a = stall_event(c);
      if (a && cudaEventRecord(a, st) != cudaSuccess) { (void)cudaGetLastError(); c->stall_free.push_back(a); a = nullptr; }
    }
    *err = cudaStreamWaitEvent(st, sl.ev, 0);
    if (*err != cudaSuccess) break;
    ++n;
  }
  if (a) {
    cudaEvent_t b = stall_event(c);
    if (b && cudaEventRecord(b, st) == cudaSuccess) c->stall_open.push_back({a, b});
    else { (void)cudaGetLastError(); c->stall_free.push_back(a); if (b) c->stall_free.push_back(b); }
  }
  return n;
}
// Adds the waits that have run to the statistics.
void harvest_stalls(dx_cache* c) {
  size_t keep = 0;
  for (size_t i = 0; i < c->stall_open.size(); ++i) {
    auto pr = c->stall_open[i];
    if (cudaEventQuery(pr.second) == cudaSuccess) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, pr.first, pr.second) == cudaSuccess) c->stats.stream_stall_ns += (int64_t)(ms * 1e6f);
      c->stall_free.push_back(pr.first);
      c->stall_free.push_back(pr.second);
    } else {
      (void)cudaGetLastError();
      c->stall_open[keep++] = pr;
    }
  }
  c->stall_open.resize(keep);
}

// applies the layer's pending table patches on `st`
dx_status flush_patches(dx_cache* c, int layer, cudaStream_t st) {
  auto& pend = c->pending[layer];
  dx_layer* L = c->layer[layer];
  if (!c->ctx || !L) { pend.clear(); return DX_OK; }
  const int base = L->desc.n_shared + 1;
  // several patches may name the same expert (evicted, then loaded again): only the last one counts, and one
  // launch must not carry two writes to the same table entry
  {
    std::vector<std::pair<int, const void*>> last;
    for (size_t a = 0; a < pend.size(); ++a) {
      bool later = false;
      for (size_t b = a + 1; b < pend.size(); ++b)
        if (pend[b].first == pend[a].first) { later = true; break; }
      if (!later) last.push_back(pend[a]);
    }
    pend.swap(last);
  }
  size_t i = 0;
  while (i < pend.size()) {
    DxTablePatch patch;
    patch.n = 0;
    while (i < pend.size() && patch.n < 32) {
      patch.idx[patch.n] = base + pend[i].first;
      patch.ptr[patch.n] = pend[i].second;
      L->table_host[base + pend[i].first] = pend[i].second;
      ++patch.n;
      ++i;
    }
    dx_table_patch_kernel<<<1, 32, 0, st>>>(L->table_dev, L->table_len, c->ctx->dev_status, patch);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { c->ctx->last_cuda = e; return DX_ERR_CUDA; }
    c->ctx->launches++;
  }
  pend.clear();
  return DX_OK;
}

dx_status check_ids(dx_cache* c, int layer, const int32_t* ids, int n) {
  if (!c || (n > 0 && !ids) || n < 0) return DX_ERR_INVALID_ARG;
  if (layer < 0 || layer >= c->L) return DX_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i)
    if (ids[i] < 0 || ids[i] >= c->E) return DX_ERR_INVALID_ARG;
  return DX_OK;
}

}  // namespace

// A layer that is destroyed before its cache: drop the back pointer and the table patches queued for it.
void dx_cache_forget_layer(dx_cache* c, dx_layer* L) {
  if (!c || !L) return;
  for (int l = 0; l < c->L; ++l)
    if (c->layer[l] == L) { c->layer[l] = nullptr; c->pending[l].clear(); }
}

// Slot of `expert` in `layer` (-1: neither cached nor in flight); no statistics are touched.
int dx_cache_slot_of(const dx_cache* c, int layer, int expert) {
  if (!c || layer < 0 || layer >= c->L || expert < 0 || expert >= c->E) return -1;
  return c->slot_of[(size_t)layer * c->E + expert];
}
int dx_cache_slots(const dx_cache* c) { return c ? c->S : 0; }

bool dx_cache_layer_quiet(dx_cache* c, int layer) {
  if (!c || layer < 0 || layer >= c->L) return false;
  if (!c->ctx) return true;
  for (int s = 0; s < c->S; ++s) {
    DxSlot& sl = slot_ref(c, layer, s);
    if (sl.expert >= 0 && !copy_done(c, sl)) return false;
  }
  return true;
}

dx_status dx_cache_prepare_layer(dx_cache* c, int layer, cudaStream_t st) {
  if (!c || layer < 0 || layer >= c->L) return DX_ERR_INVALID_ARG;
  if (!c->ctx) return DX_OK;
  cudaError_t e;
  c->stats.waited_copies += wait_for_copies(c, layer, nullptr, st, &e);
  if (e != cudaSuccess) { c->ctx->last_cuda = e; return DX_ERR_CUDA; }
  return flush_patches(c, layer, st);
}

void dx_cache_note_use(dx_cache* c, int layer, cudaStream_t st) {
  if (!c || !c->ctx || layer < 0 || layer >= c->L) return;
  if (cudaEventRecord(c->used_ev[layer], st) == cudaSuccess) c->used_valid[layer] = 1;
}

extern "C" dx_status expert_cache_create(dx_ctx* ctx, int32_t n_layers, int32_t n_experts, int32_t slots_per_layer,
                                         size_t blob_bytes, dx_cache** out) {
  if (!out) return DX_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_layers < 1 || n_experts < 1 || slots_per_layer < 1 || blob_bytes == 0 || blob_bytes % 128)
    return DX_ERR_INVALID_ARG;
  if (n_experts > DX_MAX_E) return DX_ERR_UNSUPPORTED;
  dx_cache* c = new (std::nothrow) dx_cache();
  if (!c) return DX_ERR_OOM;
  c->ctx = ctx;
  c->L = n_layers; c->E = n_experts; c->S = slots_per_layer;
  c->blob_bytes = blob_bytes;
  c->slab = nullptr;
  c->q4_bytes = 0;
  c->q4_hidden = c->q4_inter = 0;
  c->staging = nullptr;
  c->copy_stream = nullptr;
  c->expand_stream = nullptr;
  c->staged_ev = nullptr;
  c->clock = 0;
  c->stats = dx_cache_stats{};
  c->host_blob.assign((size_t)n_layers * n_experts, nullptr);
  c->slots.assign((size_t)n_layers * slots_per_layer, DxSlot());
  c->slot_of.assign((size_t)n_layers * n_experts, -1);
  c->layer.assign(n_layers, nullptr);
  c->used_ev.assign(n_layers, nullptr);
  c->used_valid.assign(n_layers, 0);
  c->pending.resize(n_layers);
  if (ctx) {
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e == cudaSuccess) e = cudaMalloc(&c->slab, (size_t)n_layers * slots_per_layer * blob_bytes);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->expand_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->staged_ev, cudaEventDisableTiming);
    for (size_t i = 0; e == cudaSuccess && i < c->slots.size(); ++i)
      e = cudaEventCreateWithFlags(&c->slots[i].ev, cudaEventDisableTiming);
    for (int l = 0; e == cudaSuccess && l < n_layers; ++l)
      e = cudaEventCreateWithFlags(&c->used_ev[l], cudaEventDisableTiming);
    if (e != cudaSuccess) {
      ctx->last_cuda = e;
      expert_cache_destroy(c);
      return e == cudaErrorMemoryAllocation ? DX_ERR_OOM : DX_ERR_CUDA;
    }
  }
  *out = c;
  return DX_OK;
}

extern "C" dx_status expert_cache_destroy(dx_cache* c) {
  if (!c) return DX_ERR_INVALID_ARG;
  if (c->ctx) {
    if (c->copy_stream) cudaStreamSynchronize(c->copy_stream);
    if (c->expand_stream) cudaStreamSynchronize(c->expand_stream);
    if (c->staged_ev) cudaEventDestroy(c->staged_ev);
    for (auto& pr : c->stall_open) { cudaEventDestroy(pr.first); cudaEventDestroy(pr.second); }
    for (auto& ev : c->stall_free) cudaEventDestroy(ev);
    if (c->expand_stream) cudaStreamDestroy(c->expand_stream);
    for (auto& s : c->slots)
      if (s.ev) cudaEventDestroy(s.ev);
    for (auto& e : c->used_ev)
      if (e) cudaEventDestroy(e);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    cudaFree(c->slab);
    cudaFree(c->staging);
  }
  for (auto* L : c->layer)
    if (L) { L->cache = nullptr; L->cache_layer = -1; }
  delete c;
  return DX_OK;
}

extern "C" dx_status dx_layer_attach_cache(dx_layer* L, dx_cache* c, int32_t layer_index) {
  if (!L || !c || layer_index < 0 || layer_index >= c->L) return DX_ERR_INVALID_ARG;
  if (L->desc.n_experts != c->E) return DX_ERR_SHAPE;
  size_t need = 0;
  if (dx_expert_blob_bytes(&L->desc, L->desc.inter, &need) != DX_OK || need != c->blob_bytes) return DX_ERR_SHAPE;
  L->cache = c;
  L->cache_layer = layer_index;
  c->layer[layer_index] = L;
  // routed entries now follow the slots: nothing is resident until it is staged
  const int base = L->desc.n_shared + 1;
  for (int e = 0; e < c->E; ++e) {
    const int s = c->slot_of[(size_t)layer_index * c->E + e];
    L->table_host[base + e] = s >= 0 ? slot_ptr(c, layer_index, s) : nullptr;
  }
  L->dirty = true;
  return DX_OK;
}

extern "C" dx_status expert_cache_set_q4(dx_cache* c, const dx_layer_desc* desc, int32_t inter) {
  if (!c || !desc) return DX_ERR_INVALID_ARG;
  if (desc->weight_dtype != DX_DTYPE_BF16) return DX_ERR_UNSUPPORTED;   // the slots hold expanded bf16 blobs
  size_t q4 = 0, full = 0;
  dx_status s = dx_q4_expert_bytes(desc, inter, &q4);
  if (s != DX_OK) return s;
  if (dx_expert_blob_bytes(desc, inter, &full) != DX_OK || full != c->blob_bytes) return DX_ERR_SHAPE;
  // only before anything is registered or resident: the pool's format is one for all experts
  for (const void* b : c->host_blob)
    if (b) return DX_ERR_INVALID_ARG;
  if (c->q4_bytes) return DX_ERR_INVALID_ARG;
  if (c->ctx) {
    cudaError_t e = cudaSetDevice(c->ctx->device);
    if (e == cudaSuccess) e = cudaMalloc(&c->staging, (size_t)c->L * c->S * ((q4 + 255) / 256 * 256));
    if (e != cudaSuccess) {
      c->ctx->last_cuda = e;
      return e == cudaErrorMemoryAllocation ? DX_ERR_OOM : DX_ERR_CUDA;
    }
  }
  c->q4_bytes = q4;
  c->q4_hidden = desc->hidden;
  c->q4_inter = inter;
  return DX_OK;
}

extern "C" dx_status expert_cache_register(dx_cache* c, int32_t layer, int32_t expert, const void* blob) {
  if (!c || !blob || layer < 0 || layer >= c->L || expert < 0 || expert >= c->E) return DX_ERR_INVALID_ARG;
  if (((uintptr_t)blob) % 16) return DX_ERR_INVALID_ARG;
  c->host_blob[(size_t)layer * c->E + expert] = blob;
  return DX_OK;
}

extern "C" dx_status expert_cache_begin_step(dx_cache* c) {
  if (!c) return DX_ERR_INVALID_ARG;
  for (auto& s : c->slots)
    if (s.prefetched) { s.prefetched = false; c->stats.prefetch_wasted++; }
  if (c->ctx) harvest_stalls(c);   // (keeps the list of timed waits short)
  return DX_OK;
}

extern "C" dx_status expert_cache_prefetch(dx_cache* c, int32_t layer, const int32_t* ids, int32_t n) {
  dx_status st = check_ids(c, layer, ids, n);
  if (st != DX_OK) return st;
  std::vector<char> pinned(c->S, 0);
  for (int i = 0; i < n; ++i) {
    const int e = ids[i];
    if (c->slot_of[(size_t)layer * c->E + e] >= 0) continue;   // cached or in flight already
    if (!c->host_blob[(size_t)layer * c->E + e]) return DX_ERR_NOT_RESIDENT;
    bool was_protected;
    const int s = find_victim(c, layer, pinned, false, &was_protected);
    if (s < 0) continue;   // every slot is protected: drop the hint
    st = load_into(c, layer, s, e, true);
    if (st != DX_OK) return st;
    c->stats.prefetch_issued++;
  }
  return DX_OK;
}

static dx_status resolve(dx_cache* c, int layer, const int32_t* ids, int n, cudaStream_t stream, bool may_load,
                         double timeout_s) {
  dx_status st = check_ids(c, layer, ids, n);
  if (st != DX_OK) return st;
  if (n > c->S) return DX_ERR_CACHE_FULL;
  std::vector<char> pinned(c->S, 0);
  // hits first (they pin their slots), then the misses in the order given
  for (int i = 0; i < n; ++i) {
    const int s = c->slot_of[(size_t)layer * c->E + ids[i]];
    if (s < 0) continue;
    DxSlot& sl = slot_ref(c, layer, s);
    if (!pinned[s]) {
      c->stats.lookups++;
      c->stats.hits++;
      if (sl.prefetched) { sl.prefetched = false; c->stats.prefetch_used++; }
      sl.stamp = ++c->clock;
      pinned[s] = 1;
    }
  }
  for (int i = 0; i < n; ++i) {
    const int e = ids[i];
    if (c->slot_of[(size_t)layer * c->E + e] >= 0) continue;
    if (!may_load) return DX_ERR_NOT_RESIDENT;
    if (!c->host_blob[(size_t)layer * c->E + e]) return DX_ERR_NOT_RESIDENT;
    bool was_protected;
    const int s = find_victim(c, layer, pinned, true, &was_protected);
    if (s < 0) return DX_ERR_CACHE_FULL;
    if (was_protected) { c->stats.prefetch_wasted++; slot_ref(c, layer, s).prefetched = false; }
    c->stats.lookups++;
    c->stats.on_demand++;
    st = load_into(c, layer, s, e, false);
    if (st != DX_OK) return st;
    pinned[s] = 1;
  }
  if (!c->ctx) { c->pending[layer].clear(); return DX_OK; }
  // the compute stream waits for exactly the copies it needs that are not known to be complete
  if (timeout_s > 0.0) {
    // bounded host wait (expert_cache_wait): poll the copies' events up to the deadline (counted from the call's start)
    const auto t0 = std::chrono::steady_clock::now();
    for (int s = 0; s < c->S; ++s) {
      if (!pinned[s]) continue;
      DxSlot& sl = slot_ref(c, layer, s);
      if (copy_done(c, sl)) continue;
      c->stats.waited_copies++;
      const auto ts = std::chrono::steady_clock::now();
      bool late = false;
      while (!late && !copy_done(c, sl))
        late = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count() > timeout_s;
      c->stats.stall_ns += (int64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(
                               std::chrono::steady_clock::now() - ts).count();
      if (late) return DX_ERR_TIMEOUT;
    }
  } else {
    cudaError_t e;
    c->stats.waited_copies += wait_for_copies(c, layer, &pinned, stream, &e);
    if (e != cudaSuccess) { c->ctx->last_cuda = e; return DX_ERR_CUDA; }
  }
  return flush_patches(c, layer, stream);
}

extern "C" dx_status expert_cache_stage(dx_cache* c, int32_t layer, const int32_t* ids, int32_t n, void* stream) {
  return resolve(c, layer, ids, n, (cudaStream_t)stream, true, 0.0);
}

extern "C" dx_status expert_cache_wait(dx_cache* c, int32_t layer, const int32_t* ids, int32_t n, void* stream,
                                       double timeout_s) {
  return resolve(c, layer, ids, n, (cudaStream_t)stream, false, timeout_s);
}

namespace {
void CUDART_CB sleep_on_host(void* ms) {
  std::this_thread::sleep_for(std::chrono::milliseconds((long long)(intptr_t)ms));
}
}  // namespace

extern "C" dx_status expert_cache_inject_transfer_delay(dx_cache* c, int32_t milliseconds) {
  if (!c || milliseconds < 0 || milliseconds > 1000) return DX_ERR_INVALID_ARG;
  if (!c->ctx) return DX_OK;
  cudaError_t e = cudaLaunchHostFunc(c->copy_stream, sleep_on_host, (void*)(intptr_t)milliseconds);
  if (e != cudaSuccess) { c->ctx->last_cuda = e; return DX_ERR_CUDA; }
  return DX_OK;
}

extern "C" dx_status expert_cache_stats(dx_cache* c, dx_cache_stats* out) {
  if (!c || !out) return DX_ERR_INVALID_ARG;
  if (c->ctx) harvest_stalls(c);
  *out = c->stats;
  return DX_OK;
}

extern "C" dx_status expert_cache_query(dx_cache* c, int32_t layer, int32_t expert, int32_t* slot_out,
                                        int32_t* in_flight_out) {
  if (!c || layer < 0 || layer >= c->L || expert < 0 || expert >= c->E) return DX_ERR_INVALID_ARG;
  const int s = c->slot_of[(size_t)layer * c->E + expert];
  if (slot_out) *slot_out = s;
  if (in_flight_out) *in_flight_out = s >= 0 ? (copy_done(c, slot_ref(c, layer, s)) ? 0 : 1) : 0;
  return DX_OK;
}
