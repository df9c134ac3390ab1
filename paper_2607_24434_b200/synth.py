"""Seeded synthetic inputs for the draft / verify MoE hot path.

This module only *produces data*: random weights, hidden-state blocks, router
biases and draft-token sequences with the shapes and statistics of the
workloads in Sec. 4 (Table 1: 64 routed + 2 shared experts, top-6, and the
DeepSeek-V2-Lite parameter split of Sec. 2.1).  None of the method's
arithmetic (routing, SwiGLU, union, accept) lives here, so both the CUDA path
and the CPU checker can consume the same buffers without sharing code.

Every tensor is drawn once from a ``torch.Generator`` seeded with
``(seed, tag)``; bf16 tensors are rounded to nearest-even from the fp32 draw
before anyone sees them.  A tensor generated on one device is copied to the
other side, so parity is parity of bytes, not of two random generators.
"""
from __future__ import annotations

import dataclasses
import hashlib
import math
from typing import Dict, List, Optional

import numpy as np
import torch

SCORE_SOFTMAX = 0
SCORE_SIGMOID = 1
DTYPE_FP32 = 0
DTYPE_BF16 = 1
DTYPE_Q4 = 2      # experts 4-bit block-quantised (18-byte blocks of 32 weights), router bf16
DTYPE_BF16_WIDE = 3   # bf16 weights, expert blobs packed for the tcgen05 kernel


@dataclasses.dataclass(frozen=True)
class LayerShape:
    """Static description of one MoE layer (mirrors ``dx_layer_desc``)."""

    hidden: int
    n_experts: int
    top_k: int
    inter: int
    n_shared: int
    shared_inter: int
    draft_inter: int
    score_fn: int = SCORE_SOFTMAX
    norm_topk: int = 1
    weight_dtype: int = DTYPE_BF16
    routed_scale: float = 1.0
    draft_gamma: float = 1.0

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.weight_dtype == DTYPE_FP32 else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.weight_dtype == DTYPE_FP32 else 2

    def expert_bytes(self, inter: Optional[int] = None) -> int:
        return 3 * self.hidden * (self.inter if inter is None else inter) * self.elem_bytes


def shape_tiny() -> LayerShape:
    """Tiny fp32 layer: hidden 256, 8 experts of intermediate 128, softmax top-2."""
    return LayerShape(hidden=256, n_experts=8, top_k=2, inter=128, n_shared=1,
                      shared_inter=128, draft_inter=128, score_fn=SCORE_SOFTMAX,
                      norm_topk=1, weight_dtype=DTYPE_FP32)


def shape_v2lite() -> LayerShape:
    """DeepSeek-V2-Lite-shaped layer (Sec. 2.1, Table 1): 64 x (2048 -> 1408), top-6, 2 shared."""
    return LayerShape(hidden=2048, n_experts=64, top_k=6, inter=1408, n_shared=2,
                      shared_inter=1408, draft_inter=1408, score_fn=SCORE_SOFTMAX,
                      norm_topk=1, weight_dtype=DTYPE_BF16)


def shape_moonlight() -> LayerShape:
    """Moonlight-16B-A3B-shaped layer (Table 1): sigmoid scores, routed scale 2.446."""
    return dataclasses.replace(shape_v2lite(), score_fn=SCORE_SIGMOID, routed_scale=2.446)


def _seed_for(seed: int, tag: str) -> int:
    digest = hashlib.sha256(f"{seed}:{tag}".encode()).digest()
    return int.from_bytes(digest[:8], "little") & ((1 << 63) - 1)


def _gen(seed: int, tag: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed_for(seed, tag))
    return g


def normal(shape, std: float, seed: int, tag: str, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """N(0, std^2) tensor drawn in fp32 then rounded (nearest-even) to ``dtype``."""
    x = torch.randn(shape, generator=_gen(seed, tag, device), device=device, dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    return x.to(dtype)


def zipf_bias(n_experts: int, seed: int, tag: str = "zipf", s: float = 1.1) -> torch.Tensor:
    """Per-expert additive router bias ``-s * ln(rank)`` with a seeded rank permutation.

    Added to the router logits it skews expert popularity like a Zipf(s) law,
    which is how block tokens come to reuse experts.
    """
    rng = np.random.default_rng(_seed_for(seed, tag))
    rank = rng.permutation(n_experts).astype(np.float64) + 1.0
    return torch.from_numpy((-s * np.log(rank)).astype(np.float32))


def make_layer(shape: LayerShape, seed: int, device="cpu", std: float = 0.02,
               zipf: bool = False) -> Dict[str, object]:
    """Random layer weights in the canonical row-major layouts.

    Returns a dict with ``router`` [E,H], ``bias`` [E] fp32 or None, ``shared``
    (list of (Wg[I,H], Wu[I,H], Wd[H,I])), ``draft`` (same triple) and
    ``experts`` = (Wg[E,I,H], Wu[E,I,H], Wd[E,H,I]).
    """
    dt = shape.torch_dtype
    H, E, I = shape.hidden, shape.n_experts, shape.inter

    def triple(inter: int, tag: str):
        return (normal((inter, H), std, seed, tag + ".g", dt, device),
                normal((inter, H), std, seed, tag + ".u", dt, device),
                normal((H, inter), std, seed, tag + ".d", dt, device))

    layer: Dict[str, object] = {"shape": shape, "seed": seed}
    layer["router"] = normal((E, H), std, seed, "router", dt, device)
    layer["bias"] = zipf_bias(E, seed).to(device) if zipf else None
    layer["shared"] = [triple(shape.shared_inter, f"shared{s}") for s in range(shape.n_shared)]
    layer["draft"] = triple(shape.draft_inter, "draft") if shape.draft_inter > 0 else None
    layer["experts"] = (normal((E, I, H), std, seed, "experts.g", dt, device),
                        normal((E, I, H), std, seed, "experts.u", dt, device),
                        normal((E, H, I), std, seed, "experts.d", dt, device))
    return layer


def hidden_block(K: int, H: int, seed: int, rho: float = 0.0, device="cpu",
                 tag: str = "hidden") -> torch.Tensor:
    """K hidden-state rows ~ N(0,1); rho > 0 chains them as an AR(1) process so
    neighbouring block tokens route alike and expert unions grow sublinearly."""
    eps = normal((K, H), 1.0, seed, tag, torch.float32, device)
    if rho == 0.0 or K == 1:
        return eps
    out = torch.empty_like(eps)
    out[0] = eps[0]
    c = math.sqrt(1.0 - rho * rho)
    for t in range(1, K):
        out[t] = rho * out[t - 1] + c * eps[t]
    return out


def lm_head(V: int, H: int, seed: int, dtype: torch.dtype, device="cpu", std: float = 0.02) -> torch.Tensor:
    return normal((V, H), std, seed, "lm_head", dtype, device)


def embedding_table(V: int, H: int, seed: int, device="cpu") -> torch.Tensor:
    """Token embeddings for the closed-loop token chain of the offloaded-stack workload: bf16, N(0, 1) entries."""
    return normal((V, H), 1.0, seed, "embedding", torch.bfloat16, device)


def draft_tokens_from_target(target: np.ndarray, V: int, seed: int, p_accept: float = 0.85) -> np.ndarray:
    """Draft tokens that agree with ``target`` for a geometric(p) prefix.

    Positions match while a Bernoulli(p) draw succeeds; the first failure gets
    ``(t + 1) mod V`` and later positions are uniform random tokens.
    """
    rng = np.random.default_rng(_seed_for(seed, "draft_tokens"))
    K = int(target.shape[0])
    out = np.empty(K, dtype=np.int32)
    failed = False
    for i in range(K):
        if not failed and rng.random() < p_accept:
            out[i] = target[i]
        elif not failed:
            out[i] = (int(target[i]) + 1) % V
            failed = True
        else:
            out[i] = rng.integers(0, V)
    return out


# --------------------------------------------------------------------------
# 4-bit block-quantised routed experts (the mobile workload of Sec. 4 runs Q4_0 weights).  Quantising is input
# preparation, like the bf16 rounding above: it is done once, here, and both sides consume the resulting bytes.
# Format (the published Q4_0 block): 32 consecutive weights of a matrix row share one fp16 scale d; each weight is
# stored as a 4-bit code q with value d * (q - 8); a block is 18 bytes, the scale first, then 16 bytes whose low
# nibbles hold codes 0..15 and whose high nibbles hold codes 16..31.
# --------------------------------------------------------------------------
Q4_BLOCK = 32
Q4_BLOCK_BYTES = 18


def quantize_q4_0(w: torch.Tensor, device=None) -> torch.Tensor:
    """[R, C] float weights (C a multiple of 32) -> uint8 [R, C/32, 18] of Q4_0 blocks.  Per block: d = m / -8
    with m the entry of largest magnitude (the first one on ties), code = min(15, floor(x / d + 8.5)), and d is
    stored rounded to fp16."""
    R, Ccols = w.shape
    assert Ccols % Q4_BLOCK == 0
    x = w.detach().to(torch.float32).to(device if device is not None else "cpu").reshape(
        R, Ccols // Q4_BLOCK, Q4_BLOCK)
    idx = x.abs().argmax(dim=2, keepdim=True)
    m = torch.gather(x, 2, idx)
    d = m / -8.0
    inv = torch.where(d != 0, 1.0 / d, torch.zeros_like(d))
    q = torch.clamp(torch.floor(x * inv + 8.5), max=15.0).to(torch.uint8)
    d16 = d.to(torch.float16)
    out = torch.empty((R, Ccols // Q4_BLOCK, Q4_BLOCK_BYTES), dtype=torch.uint8, device=x.device)
    out[:, :, 0:2] = d16.view(torch.uint8).reshape(R, Ccols // Q4_BLOCK, 2)
    out[:, :, 2:] = q[:, :, :16] | (q[:, :, 16:] << 4)
    return out


def q4_expert_blob(Wg: torch.Tensor, Wu: torch.Tensor, Wd: torch.Tensor) -> torch.Tensor:
    """One routed expert as the host pool stores it when quantised: the Q4_0 blocks of W_g [I,H], W_u [I,H] and
    W_d [H,I], row-major, one matrix after the other (uint8, 3*H*I*18/32 bytes)."""
    return torch.cat([quantize_q4_0(Wg).reshape(-1), quantize_q4_0(Wu).reshape(-1), quantize_q4_0(Wd).reshape(-1)])


def quantize_layer(layer: Dict[str, object]) -> Dict[str, object]:
    """The layer with every expert matrix (shared, draft, routed) replaced by its Q4_0 blocks (uint8
    [rows, cols/32, 18], on the layer's device); router and bias unchanged; ``shape.weight_dtype`` = DTYPE_Q4."""
    sh: LayerShape = layer["shape"]
    dev = layer["router"].device

    def q(w: torch.Tensor) -> torch.Tensor:
        return quantize_q4_0(w, dev)

    def q_stack(w: torch.Tensor) -> torch.Tensor:
        return torch.stack([q(w[e]) for e in range(w.shape[0])])

    out: Dict[str, object] = {"shape": dataclasses.replace(sh, weight_dtype=DTYPE_Q4), "router": layer["router"],
                              "bias": layer["bias"]}
    out["shared"] = [tuple(q(w) for w in tr) for tr in layer["shared"]]
    out["draft"] = None if layer["draft"] is None else tuple(q(w) for w in layer["draft"])
    out["experts"] = tuple(q_stack(w) for w in layer["experts"])
    return out


def to_numpy_f32(t: torch.Tensor) -> np.ndarray:
    """Exact fp32 view of a (possibly bf16, possibly CUDA) tensor as a numpy array."""
    return t.detach().to("cpu", torch.float32).numpy()


def layer_to_numpy(layer: Dict[str, object]) -> Dict[str, object]:
    """Canonical-layout fp32 numpy copy of a layer for a host-side consumer."""
    out: Dict[str, object] = {"shape": layer["shape"]}
    out["router"] = to_numpy_f32(layer["router"])
    out["bias"] = None if layer["bias"] is None else to_numpy_f32(layer["bias"])
    out["shared"] = [tuple(to_numpy_f32(w) for w in tr) for tr in layer["shared"]]
    out["draft"] = None if layer["draft"] is None else tuple(to_numpy_f32(w) for w in layer["draft"])
    out["experts"] = tuple(to_numpy_f32(w) for w in layer["experts"])
    return out
