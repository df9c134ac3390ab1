"""Thin ctypes binding over ``libdraftexpert.so`` (the C ABI in ``include/draftexpert.h``).

Argument marshalling only: PyTorch supplies device memory and the current
stream, every step of the path (routing, union, grouped SwiGLU, argmax/accept,
weight packing, cache transfers) runs inside the library.  Function names match
the C entry points.  There is no fallback: if the shared library is missing or
a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

import torch

from .synth import DTYPE_BF16, LayerShape

_HERE = os.path.dirname(os.path.abspath(__file__))
# DX_LIB_PATH in the environment points the binding at another build of the library (e.g. a debug build)
LIB_PATH = os.environ.get("DX_LIB_PATH") or os.path.join(_HERE, "libdraftexpert.so")

DX_OK = 0
STATUS_NAMES = {0: "DX_OK", 1: "DX_ERR_INVALID_ARG", 2: "DX_ERR_SHAPE", 3: "DX_ERR_CUDA", 4: "DX_ERR_OOM",
                5: "DX_ERR_NOT_RESIDENT", 6: "DX_ERR_TIMEOUT", 7: "DX_ERR_CACHE_FULL", 8: "DX_ERR_UNSUPPORTED"}


class DxError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)}")
        self.status = status


class LayerDesc(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_experts", C.c_int32), ("top_k", C.c_int32), ("inter", C.c_int32),
                ("n_shared", C.c_int32), ("shared_inter", C.c_int32), ("draft_inter", C.c_int32),
                ("score_fn", C.c_int32), ("norm_topk", C.c_int32), ("weight_dtype", C.c_int32),
                ("routed_scale", C.c_float), ("draft_gamma", C.c_float)]


class CacheStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("lookups", "hits", "on_demand", "prefetch_issued", "prefetch_used",
                                         "prefetch_wasted", "evictions", "bytes_h2d", "waited_copies", "stall_ns",
                                         "stream_stall_ns")]


_P = C.c_void_p
_I = C.c_int32
# name -> (restype, argtypes): one line per declaration in include/draftexpert.h
SIGNATURES = {
    "dx_status_string": (C.c_char_p, [_I]),
    "dx_create": (_I, [C.c_int, C.POINTER(_P)]),
    "dx_destroy": (_I, [_P]),
    "dx_last_device_status": (_I, [_P, _P, C.POINTER(_I)]),
    "dx_set_activation_split": (_I, [_P, _I]),
    "dx_set_launch_overlap": (_I, [_P, _I]),
    "dx_set_wait_limit": (_I, [_P, C.c_uint32]),
    "dx_set_accept_l2_keep": (_I, [_P, C.c_size_t]),
    "dx_stage_block": (_I, [_P, _P, _P, C.c_size_t, _P]),
    "dx_selftest_wait_expiry": (_I, [_P, _P, _I, _P, _P]),
    "dx_last_cuda_error": (_I, [_P]),
    "dx_kernel_launches": (C.c_int64, [_P]),
    "dx_expert_blob_bytes": (_I, [C.POINTER(LayerDesc), _I, C.POINTER(C.c_size_t)]),
    "dx_pack_expert": (_I, [_P, C.POINTER(LayerDesc), _I, _P, _P, _P, _P, _P]),
    "dx_q4_expert_bytes": (_I, [C.POINTER(LayerDesc), _I, C.POINTER(C.c_size_t)]),
    "dx_expand_q4_expert": (_I, [_P, C.POINTER(LayerDesc), _I, _P, _P, _P]),
    "dx_layer_create": (_I, [_P, C.POINTER(LayerDesc), C.POINTER(_P)]),
    "dx_layer_destroy": (_I, [_P]),
    "dx_layer_set_router": (_I, [_P, _P, _P]),
    "dx_layer_set_shared": (_I, [_P, _I, _P]),
    "dx_layer_set_draft": (_I, [_P, _P]),
    "dx_layer_set_expert": (_I, [_P, _I, _P]),
    "dx_layer_attach_cache": (_I, [_P, _P, _I]),
    "moe_draft_step": (_I, [_P, _P, _P, _P, _P, _P]),
    "moe_draft_step_topr": (_I, [_P, _P, _P, _I, _I, _P, _P, _P]),
    "moe_draft_step_residual": (_I, [_P, _P, _P, _P, _P, _P]),
    "moe_draft_step_topr_residual": (_I, [_P, _P, _P, _I, _I, _P, _P, _P]),
    "dx_stack_create": (_I, [_P, C.POINTER(_P), C.c_int32, C.POINTER(_P)]),
    "dx_stack_destroy": (_I, [_P]),
    "moe_draft_stack": (_I, [_P, _P, _P, _P, _P, _P]),
    "moe_verify_block": (_I, [_P, _P, _I, _P, _P, _P, _P, _P, _P, _P, _P, _P]),
    "moe_verify_route": (_I, [_P, _P, _I, _P, _P, _P, _P, _P, _P, _P, _P, _P]),
    "moe_verify_experts": (_I, [_P, _P, _I, _P, _P]),
    "moe_verify_experts_range": (_I, [_P, _P, _I, _P, _I, _I, _I, _P]),
    "moe_draft_route": (_I, [_P, _P, _P, _P, _P, _P]),
    "moe_draft_experts": (_I, [_P, _P, _P, _P]),
    "moe_verify_block_cached": (_I, [_P, _P, _I, _P, _I, _P, _P, _P, _P, _P, _P, _P, _P, C.POINTER(_I), _P]),
    "moe_draft_step_cached": (_I, [_P, _P, _P, _I, _P, _P, _P, _P]),
    "moe_verify_block_residual": (_I, [_P, _P, _P, _I, _P, _P, _P, _P, _P, _P, _P, _P]),
    "spec_accept": (_I, [_P, _P, _I, _P, _I, _I, _I, _P, _I, _I, _P, _P, _P, _P]),
    "spec_draft_token": (_I, [_P, _P, _I, _P, _I, _I, _I, _I, _P, _P, _P]),
    "dx_controller_create": (_I, [_I, _I, C.POINTER(_P)]),
    "dx_controller_destroy": (_I, [_P]),
    "dx_controller_reset": (_I, [_P]),
    "dx_controller_size": (_I, [_P, C.POINTER(_I)]),
    "dx_controller_propose": (_I, [_P, _P, _I, C.c_float, C.c_float, _I, C.POINTER(_I), C.POINTER(_I), _P, _P,
                                   C.POINTER(_I)]),
    "dx_decoder_create": (_I, [_P, _P, _I, _P, _P, _P, _I, _I, C.c_float, _I, C.POINTER(_P)]),
    "dx_decoder_destroy": (_I, [_P]),
    "dx_decoder_step": (_I, [_P, _I, _I, _P, C.POINTER(_I), C.POINTER(_I), _P, C.POINTER(_I), _P, _P, _P]),
    "spec_accept_noalloc": (_I, [_P, _I, _P, _I, _I, _I, _P, _I, _I, _P, _P, _P, _P]),
    "moe_missing_residual": (_I, [_P, _P, _I, _P, _P, _P, _P]),
    "moe_draft_expert_term": (_I, [_P, _P, _I, _P, _P]),
    "moe_router_agreement": (_I, [_P, _P, _P, _I, _P, _P, _P]),
    "dx_squared_error": (_I, [_P, _P, _P, C.c_int64, _P, _P]),
    "expert_cache_create": (_I, [_P, _I, _I, _I, C.c_size_t, C.POINTER(_P)]),
    "expert_cache_set_q4": (_I, [_P, C.POINTER(LayerDesc), _I]),
    "expert_cache_destroy": (_I, [_P]),
    "expert_cache_register": (_I, [_P, _I, _I, _P]),
    "expert_cache_begin_step": (_I, [_P]),
    "expert_cache_prefetch": (_I, [_P, _I, _P, _I]),
    "expert_cache_stage": (_I, [_P, _I, _P, _I, _P]),
    "expert_cache_wait": (_I, [_P, _I, _P, _I, _P, C.c_double]),
    "expert_cache_stats": (_I, [_P, C.POINTER(CacheStats)]),
    "expert_cache_inject_transfer_delay": (_I, [_P, _I]),
    "expert_cache_query": (_I, [_P, _I, _I, C.POINTER(_I), C.POINTER(_I)]),
}

_lib = None


def load() -> C.CDLL:
    """Loads the shared library (built by ``paper_2607_24434_b200/build.py``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} not built: run `python -m paper_2607_24434_b200.build`")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _check(status: int, what: str) -> None:
    if status != DX_OK:
        raise DxError(status, what)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _desc(shape: LayerShape) -> LayerDesc:
    return LayerDesc(shape.hidden, shape.n_experts, shape.top_k, shape.inter, shape.n_shared, shape.shared_inter,
                     shape.draft_inter, shape.score_fn, shape.norm_topk, shape.weight_dtype, shape.routed_scale,
                     shape.draft_gamma)


class Context:
    def __init__(self, device: int = 0, act_split: bool = False):
        """``act_split``: evaluate bf16 experts with high + residual activation fragments (see
        ``dx_set_activation_split``); the default feeds plain bf16 activations to the tensor cores."""
        self.lib = load()
        self.device = device
        h = _P()
        _check(self.lib.dx_create(device, C.byref(h)), "dx_create")
        self.handle = h
        if act_split:
            self.set_activation_split(True)

    def set_activation_split(self, on: bool) -> None:
        _check(self.lib.dx_set_activation_split(self.handle, 1 if on else 0), "dx_set_activation_split")

    def set_launch_overlap(self, mask: int) -> None:
        _check(self.lib.dx_set_launch_overlap(self.handle, mask), "dx_set_launch_overlap")

    def set_wait_limit(self, polls: int) -> None:
        _check(self.lib.dx_set_wait_limit(self.handle, polls), "dx_set_wait_limit")

    def set_accept_l2_keep(self, nbytes: int) -> None:
        """Leading bytes of a bf16 LM head that spec_accept asks L2 to retain between calls (0: plain stream)."""
        _check(self.lib.dx_set_accept_l2_keep(self.handle, nbytes), "dx_set_accept_l2_keep")

    def close(self) -> None:
        if self.handle:
            self.lib.dx_destroy(self.handle)
            self.handle = None

    def device_status(self) -> int:
        out = _I(0)
        _check(self.lib.dx_last_device_status(self.handle, _stream(), C.byref(out)), "dx_last_device_status")
        return out.value

    def kernel_launches(self) -> int:
        return int(self.lib.dx_kernel_launches(self.handle))

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def expert_blob_bytes(shape: LayerShape, inter: int) -> int:
    n = C.c_size_t(0)
    d = _desc(shape)
    _check(load().dx_expert_blob_bytes(C.byref(d), inter, C.byref(n)), "dx_expert_blob_bytes")
    return n.value


def pack_expert(ctx: Context, shape: LayerShape, Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dx_pack_expert: canonical W_g [I,H], W_u [I,H], W_d [H,I] -> one streaming blob (uint8 tensor)."""
    inter = Wg.shape[0]
    nbytes = expert_blob_bytes(shape, inter)
    if out is None:
        out = torch.empty(nbytes, dtype=torch.uint8, device=Wg.device)
    d = _desc(shape)
    _check(ctx.lib.dx_pack_expert(ctx.handle, C.byref(d), inter, _ptr(Wg.contiguous()), _ptr(Wu.contiguous()),
                                  _ptr(Wd.contiguous()), _ptr(out), _stream()), "dx_pack_expert")
    return out


def q4_expert_bytes(shape: LayerShape, inter: int) -> int:
    n = C.c_size_t(0)
    d = _desc(shape)
    _check(load().dx_q4_expert_bytes(C.byref(d), inter, C.byref(n)), "dx_q4_expert_bytes")
    return n.value


def expand_q4_expert(ctx: Context, shape: LayerShape, inter: int, q4_blob: torch.Tensor,
                     out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dx_expand_q4_expert: a 4-bit block-quantised expert (uint8 device tensor) -> the bf16 streaming blob."""
    if q4_blob.numel() != q4_expert_bytes(shape, inter):
        raise ValueError("quantised blob has the wrong size")
    if out is None:
        out = torch.empty(expert_blob_bytes(shape, inter), dtype=torch.uint8, device=q4_blob.device)
    d = _desc(shape)
    _check(ctx.lib.dx_expand_q4_expert(ctx.handle, C.byref(d), inter, _ptr(q4_blob), _ptr(out), _stream()),
           "dx_expand_q4_expert")
    return out


class Layer:
    """Handle of one MoE layer plus the tensors it borrows (kept alive here)."""

    def __init__(self, ctx: Context, shape: LayerShape):
        self.ctx, self.shape, self.lib = ctx, shape, ctx.lib
        d = _desc(shape)
        h = _P()
        _check(self.lib.dx_layer_create(ctx.handle, C.byref(d), C.byref(h)), "dx_layer_create")
        self.handle = h
        self._keep: Dict[str, object] = {}

    def close(self) -> None:
        if self.handle:
            self.lib.dx_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_router(self, W_r: torch.Tensor, bias: Optional[torch.Tensor]) -> None:
        self._keep["router"] = (W_r, bias)
        _check(self.lib.dx_layer_set_router(self.handle, _ptr(W_r), _ptr(bias)), "dx_layer_set_router")

    def set_shared(self, s: int, blob: torch.Tensor) -> None:
        self._keep[f"shared{s}"] = blob
        _check(self.lib.dx_layer_set_shared(self.handle, s, _ptr(blob)), "dx_layer_set_shared")

    def set_draft(self, blob: torch.Tensor) -> None:
        self._keep["draft"] = blob
        _check(self.lib.dx_layer_set_draft(self.handle, _ptr(blob)), "dx_layer_set_draft")

    def set_expert(self, e: int, blob: Optional[torch.Tensor]) -> None:
        self._keep[f"expert{e}"] = blob
        _check(self.lib.dx_layer_set_expert(self.handle, e, _ptr(blob)), "dx_layer_set_expert")

    def share(self, ctx: "Context") -> "Layer":
        """A second handle on the same weights under another context (its own scratch and work list), so that the
        layer can be used from another stream, or several routed layers can be in flight at once."""
        other = Layer(ctx, self.shape)
        W_r, bias = self._keep["router"]
        other.set_router(W_r, bias)
        for name, blob in self._keep.items():
            if name.startswith("shared"):
                other.set_shared(int(name[6:]), blob)
            elif name == "draft":
                other.set_draft(blob)
            elif name.startswith("expert") and blob is not None:
                other.set_expert(int(name[6:]), blob)
        other.blobs = getattr(self, "blobs", None)
        return other

    @classmethod
    def from_weights(cls, ctx: Context, layer: Dict[str, object], routed_resident: bool = True) -> "Layer":
        """Packs a canonical-layout layer (see ``synth.make_layer``) that already sits on the GPU and
        attaches everything.  The routed experts share one [E, blob_bytes] allocation."""
        shape: LayerShape = layer["shape"]
        L = cls(ctx, shape)
        L.set_router(layer["router"].contiguous(), None if layer["bias"] is None else layer["bias"].contiguous())
        for s, (g, u, d) in enumerate(layer["shared"]):
            L.set_shared(s, pack_expert(ctx, shape, g, u, d))
        if layer["draft"] is not None:
            L.set_draft(pack_expert(ctx, shape, *layer["draft"]))
        Wg, Wu, Wd = layer["experts"]
        nbytes = expert_blob_bytes(shape, shape.inter)
        blobs = torch.empty((shape.n_experts, nbytes), dtype=torch.uint8, device=Wg.device)
        for e in range(shape.n_experts):
            pack_expert(ctx, shape, Wg[e], Wu[e], Wd[e], out=blobs[e])
            if routed_resident:
                L.set_expert(e, blobs[e])
        L.blobs = blobs
        return L


def _routing_buffers(shape: LayerShape, K: int, device) -> Dict[str, torch.Tensor]:
    E, k = shape.n_experts, shape.top_k
    i32 = dict(dtype=torch.int32, device=device)
    return {
        "topk_ids": torch.empty((K, k), **i32),
        "topk_w": torch.empty((K, k), dtype=torch.float32, device=device),
        "union_mask": torch.empty(((E + 63) // 64,), dtype=torch.int64, device=device),
        "union_ids": torch.full((min(E, K * k),), -1, **i32),
        "union_count": torch.empty((1,), **i32),
        "offsets": torch.empty((E + 1,), **i32),
        "perm": torch.empty((K * k,), **i32),
    }


def moe_draft_step(layer: Layer, h: torch.Tensor, y: Optional[torch.Tensor] = None,
                   out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """Eq. 5 for one token: h [H] (or [1,H]) fp32 -> y, topk_ids [k], topk_w [k]."""
    sh = layer.shape
    if out is None:
        out = {"topk_ids": torch.empty((sh.top_k,), dtype=torch.int32, device=h.device),
               "topk_w": torch.empty((sh.top_k,), dtype=torch.float32, device=h.device)}
    if y is None:
        y = torch.empty_like(h)
    _check(layer.lib.moe_draft_step(layer.handle, _ptr(h), _ptr(y), _ptr(out["topk_ids"]), _ptr(out["topk_w"]),
                                    _stream()), "moe_draft_step")
    out["y"] = y
    return out


def moe_draft_step_residual(layer: Layer, h_in: torch.Tensor, h_out: Optional[torch.Tensor] = None,
                            out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """h_out = h_in + Eq. 5 applied to RMSNorm(h_in), one token."""
    sh = layer.shape
    if out is None:
        out = {"topk_ids": torch.empty((sh.top_k,), dtype=torch.int32, device=h_in.device),
               "topk_w": torch.empty((sh.top_k,), dtype=torch.float32, device=h_in.device)}
    if h_out is None:
        h_out = torch.empty_like(h_in)
    _check(layer.lib.moe_draft_step_residual(layer.handle, _ptr(h_in), _ptr(h_out), _ptr(out["topk_ids"]),
                                             _ptr(out["topk_w"]), _stream()), "moe_draft_step_residual")
    out["h"] = h_out
    return out


class DraftStack:
    """A stack of layers the drafter runs through in one persistent launch (Eq. 5 per layer, one token)."""

    def __init__(self, ctx: Context, layers: Sequence[Layer]):
        self.lib, self.ctx, self.layers = ctx.lib, ctx, list(layers)
        arr = (_P * len(self.layers))(*[l.handle for l in self.layers])
        h = _P()
        _check(self.lib.dx_stack_create(ctx.handle, arr, len(self.layers), C.byref(h)), "dx_stack_create")
        self.handle = h

    def close(self) -> None:
        if self.handle:
            self.lib.dx_stack_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def moe_draft_stack(stack: DraftStack, h_in: torch.Tensor, h_out: Optional[torch.Tensor] = None,
                    out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """h_out = the drafter's hidden row after every layer of the stack; topk_ids / topk_w [n_layers, k]."""
    sh, n = stack.layers[0].shape, len(stack.layers)
    if out is None:
        out = {"topk_ids": torch.empty((n, sh.top_k), dtype=torch.int32, device=h_in.device),
               "topk_w": torch.empty((n, sh.top_k), dtype=torch.float32, device=h_in.device)}
    if h_out is None:
        h_out = torch.empty_like(h_in)
    _check(stack.lib.moe_draft_stack(stack.handle, _ptr(h_in), _ptr(h_out), _ptr(out["topk_ids"]),
                                     _ptr(out["topk_w"]), _stream()), "moe_draft_stack")
    out["h"] = h_out
    return out


def moe_verify_block(layer: Layer, h: torch.Tensor, y: Optional[torch.Tensor] = None,
                     out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """Eq. 4 for a block h [K,H] fp32, grouped by the union of Eq. 2/3.  Returns y and the routing outputs."""
    K = h.shape[0]
    if out is None:
        out = _routing_buffers(layer.shape, K, h.device)
    if y is None:
        y = torch.empty_like(h)
    _check(layer.lib.moe_verify_block(layer.handle, _ptr(h), K, _ptr(y), _ptr(out["topk_ids"]), _ptr(out["topk_w"]),
                                      _ptr(out["union_mask"]), _ptr(out["union_ids"]), _ptr(out["union_count"]),
                                      _ptr(out["offsets"]), _ptr(out["perm"]), _stream()), "moe_verify_block")
    out["y"] = y
    return out


def moe_verify_route(layer: Layer, h: torch.Tensor, y: torch.Tensor, out: Dict[str, torch.Tensor]) -> None:
    _check(layer.lib.moe_verify_route(layer.handle, _ptr(h), h.shape[0], _ptr(y), _ptr(out["topk_ids"]),
                                      _ptr(out["topk_w"]), _ptr(out["union_mask"]), _ptr(out["union_ids"]),
                                      _ptr(out["union_count"]), _ptr(out["offsets"]), _ptr(out["perm"]), _stream()),
           "moe_verify_route")


def moe_verify_experts(layer: Layer, h: torch.Tensor, y: torch.Tensor) -> None:
    _check(layer.lib.moe_verify_experts(layer.handle, _ptr(h), h.shape[0], _ptr(y), _stream()), "moe_verify_experts")


def moe_verify_block_residual(layer: Layer, h_in: torch.Tensor, h_out: Optional[torch.Tensor] = None,
                              out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """h_out = h_in + MoE(RMSNorm(h_in)) for the block (h_in and h_out distinct buffers)."""
    K = h_in.shape[0]
    if out is None:
        out = _routing_buffers(layer.shape, K, h_in.device)
    if h_out is None:
        h_out = torch.empty_like(h_in)
    _check(layer.lib.moe_verify_block_residual(layer.handle, _ptr(h_in), _ptr(h_out), K, _ptr(out["topk_ids"]),
                                               _ptr(out["topk_w"]), _ptr(out["union_mask"]), _ptr(out["union_ids"]),
                                               _ptr(out["union_count"]), _ptr(out["offsets"]), _ptr(out["perm"]),
                                               _stream()), "moe_verify_block_residual")
    out["h"] = h_out
    return out


def stage_block(ctx: Context, dst: torch.Tensor, src_pinned: torch.Tensor) -> None:
    """dst (device) <- src_pinned (page-locked host tensor of the same byte size), in stream order."""
    nbytes = src_pinned.numel() * src_pinned.element_size()
    if nbytes != dst.numel() * dst.element_size():
        raise ValueError("stage_block: sizes differ")
    _check(ctx.lib.dx_stage_block(ctx.handle, _ptr(dst), _ptr(src_pinned), nbytes, _stream()), "dx_stage_block")


def spec_accept(ctx: Context, h: torch.Tensor, W_lm: torch.Tensor, draft: torch.Tensor, rms_norm: bool = False,
                out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """Greedy exact verification: target [M], n_accept [1], next_token [1] (all int32, on the device)."""
    M, H = h.shape
    V = W_lm.shape[0]
    if out is None:
        out = {"target": torch.empty((M,), dtype=torch.int32, device=h.device),
               "n_accept": torch.empty((1,), dtype=torch.int32, device=h.device),
               "next_token": torch.empty((1,), dtype=torch.int32, device=h.device)}
    wd = 1 if W_lm.dtype == torch.bfloat16 else 0
    _check(ctx.lib.spec_accept(ctx.handle, _ptr(h), M, _ptr(W_lm), V, H, wd, _ptr(draft), int(draft.shape[0]),
                               1 if rms_norm else 0, _ptr(out["target"]), _ptr(out["n_accept"]),
                               _ptr(out["next_token"]), _stream()), "spec_accept")
    return out


def spec_accept_noalloc(h: torch.Tensor, W_lm: torch.Tensor, draft: torch.Tensor, out: Dict[str, torch.Tensor],
                        rms_norm: bool = False) -> Dict[str, torch.Tensor]:
    """Greedy verification through the entry point that allocates nothing: no context, and the caller passes
    the output tensors (``target`` [M], ``n_accept`` [1], ``next_token`` [1], int32, on the device) because
    this wrapper does not allocate either.  For callers that cannot allocate device memory (a memory pool fixed
    at start-up, or no allocator at hand).  At most 16 rows; calls must not overlap on the GPU."""
    M, H = h.shape
    wd = 1 if W_lm.dtype == torch.bfloat16 else 0
    _check(load().spec_accept_noalloc(_ptr(h), M, _ptr(W_lm), W_lm.shape[0], H, wd, _ptr(draft), int(draft.shape[0]),
                                      1 if rms_norm else 0, _ptr(out["target"]), _ptr(out["n_accept"]),
                                      _ptr(out["next_token"]), _stream()), "spec_accept_noalloc")
    return out


class ExpertCache:
    """Handle of an accelerator expert cache (Sec. 3.5).  ``ctx=None`` gives the bookkeeping-only cache."""

    def __init__(self, ctx: Optional[Context], n_layers: int, n_experts: int, slots: int, blob_bytes: int):
        self.lib = load()
        self.ctx = ctx
        self.n_layers, self.n_experts, self.slots, self.blob_bytes = n_layers, n_experts, slots, blob_bytes
        h = _P()
        _check(self.lib.expert_cache_create(ctx.handle if ctx else None, n_layers, n_experts, slots, blob_bytes,
                                            C.byref(h)), "expert_cache_create")
        self.handle = h
        self._keep: List[object] = []

    def close(self) -> None:
        if self.handle:
            self.lib.expert_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _ids(ids: Sequence[int]):
        arr = (C.c_int32 * len(ids))(*[int(i) for i in ids])
        return arr, len(ids)

    def set_q4(self, shape: LayerShape) -> None:
        """The host pool holds 4-bit block-quantised blobs from now on (before the first register)."""
        d = _desc(shape)
        _check(self.lib.expert_cache_set_q4(self.handle, C.byref(d), shape.inter), "expert_cache_set_q4")

    def register(self, layer: int, expert: int, pinned_blob: torch.Tensor) -> None:
        self._keep.append(pinned_blob)
        _check(self.lib.expert_cache_register(self.handle, layer, expert, _ptr(pinned_blob)), "expert_cache_register")

    def register_fake(self, layer: int, expert: int) -> None:
        """Bookkeeping-only caches never read the blob; any non-null 16-byte-aligned address will do."""
        _check(self.lib.expert_cache_register(self.handle, layer, expert, 4096), "expert_cache_register")

    def attach(self, layer_handle: "Layer", layer: int) -> None:
        _check(self.lib.dx_layer_attach_cache(layer_handle.handle, self.handle, layer), "dx_layer_attach_cache")

    def begin_step(self) -> None:
        _check(self.lib.expert_cache_begin_step(self.handle), "expert_cache_begin_step")

    def prefetch(self, layer: int, ids: Sequence[int]) -> None:
        arr, n = self._ids(ids)
        _check(self.lib.expert_cache_prefetch(self.handle, layer, arr, n), "expert_cache_prefetch")

    def stage(self, layer: int, ids: Sequence[int]) -> None:
        arr, n = self._ids(ids)
        st = _stream() if self.ctx else None
        _check(self.lib.expert_cache_stage(self.handle, layer, arr, n, st), "expert_cache_stage")

    def wait(self, layer: int, ids: Sequence[int], timeout_s: float = 0.0) -> None:
        arr, n = self._ids(ids)
        st = _stream() if self.ctx else None
        _check(self.lib.expert_cache_wait(self.handle, layer, arr, n, st, timeout_s), "expert_cache_wait")

    def inject_transfer_delay(self, milliseconds: int) -> None:
        _check(self.lib.expert_cache_inject_transfer_delay(self.handle, milliseconds),
               "expert_cache_inject_transfer_delay")

    def stats(self) -> Dict[str, int]:
        s = CacheStats()
        _check(self.lib.expert_cache_stats(self.handle, C.byref(s)), "expert_cache_stats")
        return {name: int(getattr(s, name)) for name, _ in CacheStats._fields_}

    def query(self, layer: int, expert: int) -> Tuple[int, int]:
        slot, infl = _I(0), _I(0)
        _check(self.lib.expert_cache_query(self.handle, layer, expert, C.byref(slot), C.byref(infl)),
               "expert_cache_query")
        return slot.value, infl.value


def moe_verify_experts_range(layer: Layer, h: torch.Tensor, y: torch.Tensor, first_union: int, n_union: int,
                             include_shared: bool) -> None:
    _check(layer.lib.moe_verify_experts_range(layer.handle, _ptr(h), h.shape[0], _ptr(y), first_union, n_union,
                                              1 if include_shared else 0, _stream()), "moe_verify_experts_range")


def moe_draft_route(layer: Layer, h: torch.Tensor, y: torch.Tensor, out: Dict[str, torch.Tensor]) -> None:
    _check(layer.lib.moe_draft_route(layer.handle, _ptr(h), _ptr(y), _ptr(out["topk_ids"]), _ptr(out["topk_w"]),
                                     _stream()), "moe_draft_route")


def moe_draft_experts(layer: Layer, h: torch.Tensor, y: torch.Tensor) -> None:
    _check(layer.lib.moe_draft_experts(layer.handle, _ptr(h), _ptr(y), _stream()), "moe_draft_experts")


def moe_verify_block_cached(layer: Layer, cache: ExpertCache, layer_index: int, h: torch.Tensor,
                            y: Optional[torch.Tensor] = None, out: Optional[Dict[str, torch.Tensor]] = None,
                            residual: bool = False):
    """Verify block on a layer whose routed experts come through ``cache`` (``moe_verify_block_cached`` of the
    library: route, one read of the union on the host, waves of at most ``cache.slots`` experts -- cached ones
    first, then misses by ascending id).  ``cache`` / ``layer_index`` are what the layer was attached with."""
    K = h.shape[0]
    if out is None:
        out = _routing_buffers(layer.shape, K, h.device)
    if y is None:
        y = torch.empty_like(h)
    cap = min(layer.shape.n_experts, K * layer.shape.top_k)
    host_ids = (C.c_int32 * cap)()
    host_n = _I(0)
    _check(layer.lib.moe_verify_block_cached(layer.handle, _ptr(h), K, _ptr(y), 1 if residual else 0,
                                             _ptr(out["topk_ids"]), _ptr(out["topk_w"]), _ptr(out["union_mask"]),
                                             _ptr(out["union_ids"]), _ptr(out["union_count"]), _ptr(out["offsets"]),
                                             _ptr(out["perm"]), host_ids, C.byref(host_n), _stream()),
           "moe_verify_block_cached")
    out["h" if residual else "y"] = y
    out["union_list"] = [int(host_ids[i]) for i in range(host_n.value)]
    return out


def moe_draft_step_cached(layer: Layer, h: torch.Tensor, y: Optional[torch.Tensor] = None,
                          out: Optional[Dict[str, torch.Tensor]] = None, residual: bool = False):
    """Draft step (Eq. 5) on a cache-attached layer: route, read the selection on the host, stage e1, experts.
    ``out["host_ids"]`` is the router's top-k as a Python list (the predicted verifier experts)."""
    sh = layer.shape
    if out is None:
        out = {"topk_ids": torch.empty((sh.top_k,), dtype=torch.int32, device=h.device),
               "topk_w": torch.empty((sh.top_k,), dtype=torch.float32, device=h.device)}
    if y is None:
        y = torch.empty_like(h)
    host_ids = (C.c_int32 * sh.top_k)()
    _check(layer.lib.moe_draft_step_cached(layer.handle, _ptr(h), _ptr(y), 1 if residual else 0, _ptr(out["topk_ids"]),
                                           _ptr(out["topk_w"]), host_ids, _stream()), "moe_draft_step_cached")
    out["h" if residual else "y"] = y
    out["host_ids"] = [int(host_ids[j]) for j in range(sh.top_k)]
    return out


def selftest_wait_expiry(layer: Layer, h: torch.Tensor, y: torch.Tensor) -> None:
    _check(layer.lib.dx_selftest_wait_expiry(layer.handle, _ptr(h), h.shape[0], _ptr(y), _stream()),
           "dx_selftest_wait_expiry")


def moe_draft_step_topr(layer: Layer, h: torch.Tensor, top_r: int, use_draft_expert: bool,
                        y: Optional[torch.Tensor] = None) -> Dict[str, torch.Tensor]:
    """Shared + top-r drafter (Sec. 2.2), optionally with the draft expert."""
    sh = layer.shape
    out = {"topk_ids": torch.empty((sh.top_k,), dtype=torch.int32, device=h.device),
           "topk_w": torch.empty((sh.top_k,), dtype=torch.float32, device=h.device)}
    if y is None:
        y = torch.empty_like(h)
    _check(layer.lib.moe_draft_step_topr(layer.handle, _ptr(h), _ptr(y), top_r, 1 if use_draft_expert else 0,
                                         _ptr(out["topk_ids"]), _ptr(out["topk_w"]), _stream()),
           "moe_draft_step_topr")
    out["y"] = y
    return out


def moe_draft_step_topr_residual(layer: Layer, h_in: torch.Tensor, h_out: torch.Tensor, top_r: int,
                                 use_draft_expert: bool, out: Dict[str, torch.Tensor]) -> None:
    """h_out = h_in + (shared + top-r drafter, optionally with the draft expert) applied to RMSNorm(h_in)."""
    _check(layer.lib.moe_draft_step_topr_residual(layer.handle, _ptr(h_in), _ptr(h_out), top_r,
                                                  1 if use_draft_expert else 0, _ptr(out["topk_ids"]),
                                                  _ptr(out["topk_w"]), _stream()), "moe_draft_step_topr_residual")


def spec_draft_token(ctx: Context, h: torch.Tensor, W_lm: torch.Tensor, rms_norm: bool = False):
    """Draft-side LM head: token [M] = argmax and confidence [M] = its softmax probability (Algorithm 1, q_i)."""
    M, H = h.shape
    token = torch.empty((M,), dtype=torch.int32, device=h.device)
    conf = torch.empty((M,), dtype=torch.float32, device=h.device)
    wd = 1 if W_lm.dtype == torch.bfloat16 else 0
    _check(ctx.lib.spec_draft_token(ctx.handle, _ptr(h), M, _ptr(W_lm), W_lm.shape[0], H, wd, 1 if rms_norm else 0,
                                    _ptr(token), _ptr(conf), _stream()), "spec_draft_token")
    return token, conf


def moe_missing_residual(layer: Layer, h: torch.Tensor) -> Dict[str, torch.Tensor]:
    """Eq. 6 for a block: m[t] = y*_t - S(h_t) - g_{t,e1} E_{e1}(h_t).  Returns m and the routing it used."""
    K, sh = h.shape[0], layer.shape
    out = {"m": torch.empty_like(h),
           "topk_ids": torch.empty((K, sh.top_k), dtype=torch.int32, device=h.device),
           "topk_w": torch.empty((K, sh.top_k), dtype=torch.float32, device=h.device)}
    _check(layer.lib.moe_missing_residual(layer.handle, _ptr(h), K, _ptr(out["m"]), _ptr(out["topk_ids"]),
                                          _ptr(out["topk_w"]), _stream()), "moe_missing_residual")
    return out


def moe_draft_expert_term(layer: Layer, h: torch.Tensor) -> torch.Tensor:
    """gamma * E^d(h_t) for every row (left operand of Eq. 7)."""
    out = torch.empty_like(h)
    _check(layer.lib.moe_draft_expert_term(layer.handle, _ptr(h), h.shape[0], _ptr(out), _stream()),
           "moe_draft_expert_term")
    return out


def moe_router_agreement(layer: Layer, h_star: torch.Tensor, h_draft: torch.Tensor):
    """Per row: KL(R(h*) || R(h^d)) (summand of Eq. 10) and the size of the top-k sets' intersection."""
    K = h_star.shape[0]
    kl = torch.empty((K,), dtype=torch.float32, device=h_star.device)
    agree = torch.empty((K,), dtype=torch.int32, device=h_star.device)
    _check(layer.lib.moe_router_agreement(layer.handle, _ptr(h_star), _ptr(h_draft), K, _ptr(kl), _ptr(agree),
                                          _stream()), "moe_router_agreement")
    return kl, agree


def squared_error(ctx: Context, a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """sum (a - b)^2 (with moe_draft_expert_term and moe_missing_residual: one layer's term of Eq. 7)."""
    out = torch.empty((1,), dtype=torch.float32, device=a.device)
    _check(ctx.lib.dx_squared_error(ctx.handle, _ptr(a), _ptr(b), a.numel(), _ptr(out), _stream()), "dx_squared_error")
    return out


class Decoder:
    """One decode step of Algorithm 1 over an offloaded stack as a host loop inside the library (``dx_decoder_step``).
    ``layers[l]`` must be attached to ``cache`` as cache layer l; ``emb`` / ``W_lm`` are bf16 device tensors [V, H];
    ``budget`` < 0 derives B_i of Eq. 14 from the cache's free pairs."""

    def __init__(self, ctx: "Context", layers: Sequence["Layer"], cache: "ExpertCache", emb: torch.Tensor,
                 W_lm: torch.Tensor, k_max: int = 8, tau: float = 1.0, budget: int = -1):
        if emb.dtype != torch.bfloat16 or W_lm.dtype != torch.bfloat16:
            raise ValueError("Decoder: emb and W_lm must be bf16")
        self.lib, self.ctx, self.k_max, self.n_layers = ctx.lib, ctx, k_max, len(layers)
        self._keep = (list(layers), cache, emb, W_lm)        # (the library keeps raw pointers to all of them)
        arr = (_P * len(layers))(*[l.handle for l in layers])
        h = _P()
        _check(self.lib.dx_decoder_create(ctx.handle, arr, len(layers), cache.handle, _ptr(emb), _ptr(W_lm),
                                          int(W_lm.shape[0]), k_max, float(tau), int(budget), C.byref(h)),
               "dx_decoder_create")
        self.handle = h
        self._drafted = (C.c_int32 * k_max)()
        self._emitted = (C.c_int32 * (k_max + 1))()
        self._target = (C.c_int32 * k_max)()
        self._unions = (C.c_int32 * self.n_layers)()

    def close(self) -> None:
        if self.handle:
            self.lib.dx_decoder_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def step(self, t0: int, scripted_accept: Optional[int] = None) -> Dict[str, object]:
        nd, na, ne = _I(0), _I(0), _I(0)
        _check(self.lib.dx_decoder_step(self.handle, int(t0), -1 if scripted_accept is None else int(scripted_accept),
                                        self._drafted, C.byref(nd), C.byref(na), self._emitted, C.byref(ne),
                                        self._target, self._unions, _stream()), "dx_decoder_step")
        drafted = [int(self._drafted[i]) for i in range(nd.value)]
        emitted = [int(self._emitted[i]) for i in range(ne.value)]
        K = max(1, nd.value)
        return {"drafted": drafted, "n_accept": na.value, "emitted": emitted, "next": emitted[-1],
                "target": [int(self._target[i]) for i in range(K)], "block_rows": K,
                "union_sizes": [int(self._unions[l]) for l in range(self.n_layers)]}


class Controller:
    """Confidence-expansion truncation (Sec. 3.4): host-side predicted verifier set and stop rule."""

    def __init__(self, n_layers: int, n_experts: int):
        self.lib = load()
        self.n_layers = n_layers
        h = _P()
        _check(self.lib.dx_controller_create(n_layers, n_experts, C.byref(h)), "dx_controller_create")
        self.handle = h

    def close(self) -> None:
        if self.handle:
            self.lib.dx_controller_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self) -> None:
        _check(self.lib.dx_controller_reset(self.handle), "dx_controller_reset")

    def size(self) -> int:
        n = _I(0)
        _check(self.lib.dx_controller_size(self.handle, C.byref(n)), "dx_controller_size")
        return n.value

    def propose(self, predicted: Sequence[Sequence[int]], q: float, tau: float, budget: int):
        """predicted[l] = the draft router's top-k ids in layer l.  Returns (stop, delta, new (layer, expert) pairs)."""
        k = len(predicted[0])
        flat = [int(e) for row in predicted for e in row]
        arr = (C.c_int32 * len(flat))(*flat)
        nl = (C.c_int32 * len(flat))()
        ne = (C.c_int32 * len(flat))()
        delta, stop, n_new = _I(0), _I(0), _I(0)
        _check(self.lib.dx_controller_propose(self.handle, arr, k, q, tau, budget, C.byref(delta), C.byref(stop), nl,
                                              ne, C.byref(n_new)), "dx_controller_propose")
        return bool(stop.value), delta.value, [(nl[i], ne[i]) for i in range(n_new.value)]
