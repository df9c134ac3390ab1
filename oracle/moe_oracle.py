"""CPU checker for the DraftExpert MoE draft / verify hot path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the hot path computes, written
from the paper's equations.  It exists so that the tests, the smoke check and
the benchmark's CPU-baseline leg have something independent to compare the
CUDA library against.  Nothing in the product path may import it, and it
shares no code, tables or helpers with the CUDA sources.

All arithmetic is numpy in ``float64`` by default (pass ``dtype=np.float32``
for single precision); inputs are the already-rounded weight values, widened
exactly.  There is no blocking, grouping or reordering: each token is pushed
through each of its experts one at a time, exactly as the equations read.

Pinned by the host-only tests in ``tests/test_oracle_pins.py`` (closed forms, dense evaluation,
enumeration, library routines, the paper's parameter arithmetic).  Two
quantities of the paper cannot be pinned here because they need its trained
draft experts and prompt suites: draft acceptance rate and prefetch hit rate
-- "parity unpinned" for those; they are not computed by this file.

Notation follows the paper: h hidden state, R_l(h) router distribution,
TopK_l(h), g_{l,e} gate weights, S_l shared path, E_{l,e} routed experts,
E^d_l draft expert, gamma_l its scale, U_l(D) the block's expert union.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

SCORE_SOFTMAX = 0
SCORE_SIGMOID = 1


# --------------------------------------------------------------------------
# Router: R_l(h), TopK_l(h) (Eq. 1) and the gate weights g_{l,e} of Eq. 4.
# --------------------------------------------------------------------------
def router_logits(h: np.ndarray, W_r: np.ndarray, bias: Optional[np.ndarray], dtype=np.float64) -> np.ndarray:
    """z[t, e] = sum_j W_r[e, j] h[t, j] (+ b[e]) -- the pre-activation of R_l(h) (Sec. 3.2)."""
    z = np.asarray(h, dtype) @ np.asarray(W_r, dtype).T
    if bias is not None:
        z = z + np.asarray(bias, dtype)[None, :]
    return z


def router_probs(z: np.ndarray, score_fn: int) -> np.ndarray:
    """R_l(h): softmax over all experts, or an element-wise sigmoid."""
    if score_fn == SCORE_SOFTMAX:
        e = np.exp(z - z.max(axis=-1, keepdims=True))
        return e / e.sum(axis=-1, keepdims=True)
    if score_fn == SCORE_SIGMOID:
        return 1.0 / (1.0 + np.exp(-z))
    raise ValueError("score_fn")


def topk_select(p: np.ndarray, k: int) -> np.ndarray:
    """TopK_l(h) of Eq. 1: ids of the k largest scores per row, listed in
    descending score; equal scores are ordered by ascending expert id."""
    T, E = p.shape
    ids = np.empty((T, k), dtype=np.int32)
    for t in range(T):
        order = sorted(range(E), key=lambda e: (-p[t, e], e))
        ids[t] = order[:k]
    return ids


def gate_weights(p: np.ndarray, ids: np.ndarray, norm_topk: int, routed_scale: float) -> np.ndarray:
    """g_{l,e} of Eq. 4: the selected scores, optionally renormalised to sum to
    one over the selected set, times the routed scaling factor."""
    sel = np.take_along_axis(p, ids.astype(np.int64), axis=1)
    if norm_topk:
        sel = sel / sel.sum(axis=1, keepdims=True)
    return sel * routed_scale


def route(h, W_r, bias, k, score_fn, norm_topk, routed_scale, dtype=np.float64,
          forced_ids: Optional[np.ndarray] = None):
    """Router end to end: logits z, scores p, TopK ids (or ``forced_ids`` when
    a near-tied selection is being replayed) and gate weights."""
    z = router_logits(h, W_r, bias, dtype)
    p = router_probs(z, score_fn)
    ids = topk_select(p, k) if forced_ids is None else np.asarray(forced_ids, np.int32)
    g = gate_weights(p, ids, norm_topk, routed_scale)
    return z, p, ids, g


def selection_gaps(z: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """Per row: the smallest gap between adjacent logits among the first k+1 in
    sorted order (order gap) -- a row whose gap is below the parity threshold
    is "near-tied" and may legitimately resolve either way in fp32."""
    zs = -np.sort(-z, axis=1)
    upto = min(k + 1, z.shape[1])
    d = zs[:, : upto - 1] - zs[:, 1:upto]
    set_gap = d[:, k - 1] if upto > k else np.full(z.shape[0], np.inf)
    return d.min(axis=1) if d.shape[1] else np.full(z.shape[0], np.inf), set_gap


# --------------------------------------------------------------------------
# Experts: the SwiGLU feed-forward used for S_l, E_{l,e} and E^d_l.
# --------------------------------------------------------------------------
def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def swiglu_expert(h_t: np.ndarray, Wg: np.ndarray, Wu: np.ndarray, Wd: np.ndarray, dtype=np.float64) -> np.ndarray:
    """E(h) = W_d ( silu(W_g h) * (W_u h) ) for one token; W_g, W_u are [I, H], W_d is [H, I]."""
    x = np.asarray(h_t, dtype)
    a = silu(np.asarray(Wg, dtype) @ x) * (np.asarray(Wu, dtype) @ x)
    return np.asarray(Wd, dtype) @ a


def shared_path(h_t: np.ndarray, shared: Sequence[Tuple[np.ndarray, np.ndarray, np.ndarray]], dtype=np.float64):
    """S_l(h): the always-on shared experts, summed with unit weight."""
    y = np.zeros(np.asarray(h_t).shape[-1], dtype)
    for (Wg, Wu, Wd) in shared:
        y = y + swiglu_expert(h_t, Wg, Wu, Wd, dtype)
    return y


# --------------------------------------------------------------------------
# Eq. 4: the frozen target MoE layer, token by token, expert by expert.
# --------------------------------------------------------------------------
def moe_target(h: np.ndarray, layer: Dict[str, object], dtype=np.float64,
               forced_ids: Optional[np.ndarray] = None):
    """y*_t = S(h_t) + sum_{e in TopK(h_t)} g_{t,e} E_e(h_t)  (Eq. 4).

    Returns (y [K,H], ids [K,k], g [K,k], z [K,E])."""
    sh = layer["shape"]
    h = np.asarray(h, dtype)
    z, p, ids, g = route(h, layer["router"], layer["bias"], sh.top_k, sh.score_fn, sh.norm_topk,
                         sh.routed_scale, dtype, forced_ids)
    Wg, Wu, Wd = layer["experts"]
    y = np.zeros_like(h)
    for t in range(h.shape[0]):
        acc = shared_path(h[t], layer["shared"], dtype)
        for j in range(sh.top_k):
            e = int(ids[t, j])
            acc = acc + g[t, j] * swiglu_expert(h[t], Wg[e], Wu[e], Wd[e], dtype)
        y[t] = acc
    return y, ids, g, z


# --------------------------------------------------------------------------
# Eq. 5: the fixed-footprint drafter (shared + router top-1 + draft expert).
# --------------------------------------------------------------------------
def moe_draft(h: np.ndarray, layer: Dict[str, object], dtype=np.float64,
              forced_ids: Optional[np.ndarray] = None, top_r: int = 1, gamma: Optional[float] = None):
    """y^d = S(h) + g_{e1} E_{e1}(h) + gamma E^d(h), e1 = argmax_e R(h)_e  (Eq. 5).

    g_{e1} is the same gate weight the target layer gives e1 (Eq. 6 removes
    exactly that term from y*), so the router still runs its full top-k; the
    k ids it returns are the predicted verifier experts of Sec. 3.4.
    ``top_r`` > 1 gives the training-free shared+top-r drafter of Sec. 2.2.
    """
    sh = layer["shape"]
    h = np.asarray(h, dtype)
    gam = sh.draft_gamma if gamma is None else gamma
    z, p, ids, g = route(h, layer["router"], layer["bias"], sh.top_k, sh.score_fn, sh.norm_topk,
                         sh.routed_scale, dtype, forced_ids)
    Wg, Wu, Wd = layer["experts"]
    y = np.zeros_like(h)
    for t in range(h.shape[0]):
        acc = shared_path(h[t], layer["shared"], dtype)
        for j in range(top_r):
            e = int(ids[t, j])
            acc = acc + g[t, j] * swiglu_expert(h[t], Wg[e], Wu[e], Wd[e], dtype)
        if layer["draft"] is not None and gam != 0.0:
            dg, du, dd = layer["draft"]
            acc = acc + gam * swiglu_expert(h[t], dg, du, dd, dtype)
        y[t] = acc
    return y, ids, g, z


def missing_residual(h: np.ndarray, layer: Dict[str, object], dtype=np.float64) -> np.ndarray:
    """m* = y* - S(h) - g_{e1} E_{e1}(h)  (Eq. 6), the part the draft expert stands in for."""
    y_star, ids, g, _ = moe_target(h, layer, dtype)
    y_top1, _, _, _ = moe_draft(h, layer, dtype, gamma=0.0)
    return y_star - y_top1


def dequantize_q4_0(blocks: np.ndarray, dtype=np.float64) -> np.ndarray:
    """Values of 4-bit block-quantised weights (the format of the paper's mobile runs, Sec. 4): ``blocks`` is
    uint8 [R, C/32, 18]; bytes 0..1 of a block are the fp16 scale d (little endian), byte 2 + j holds the code of
    weight j in its low nibble and of weight 16 + j in its high nibble; the weight is d * (code - 8).  Plain
    loops over the block structure; returns [R, C]."""
    blocks = np.asarray(blocks, np.uint8)
    R, nb, nbytes = blocks.shape
    assert nbytes == 18
    out = np.zeros((R, nb * 32), dtype)
    for r in range(R):
        for b in range(nb):
            blk = blocks[r, b]
            d = dtype(np.frombuffer(blk[0:2].tobytes(), dtype="<f2")[0])
            for j in range(16):
                out[r, 32 * b + j] = d * (int(blk[2 + j] & 0x0F) - 8)
                out[r, 32 * b + 16 + j] = d * (int(blk[2 + j] >> 4) - 8)
    return out


def draft_expert_term(h: np.ndarray, layer: Dict[str, object], dtype=np.float64, gamma: Optional[float] = None):
    """gamma_l * E^d_l(h_t) for every row -- the left operand of Eq. 7."""
    sh = layer["shape"]
    gam = sh.draft_gamma if gamma is None else gamma
    h = np.asarray(h, dtype)
    Wg, Wu, Wd = layer["draft"]
    return np.stack([gam * swiglu_expert(h[t], Wg, Wu, Wd, dtype) for t in range(h.shape[0])])


def residual_loss(h_draft: np.ndarray, h_star: np.ndarray, layer: Dict[str, object], dtype=np.float64) -> float:
    """One layer's term of L_res (Eq. 7): sum_t || gamma E^d(h^d_t) - m*_t ||_2^2, the draft expert evaluated on
    the drafter's hidden states and the missing residual (Eq. 6) on the teacher-forced ones."""
    d = draft_expert_term(h_draft, layer, dtype) - missing_residual(h_star, layer, dtype)
    return float((d * d).sum())


def router_distribution(z: np.ndarray, score_fn: int) -> np.ndarray:
    """R_l(h) as a distribution over the experts: the softmax itself, or -- for sigmoid routers, whose scores do
    not sum to one -- the scores divided by their sum (a reading: Eq. 10 takes a KL between two R_l)."""
    p = router_probs(z, score_fn)
    if score_fn == SCORE_SIGMOID:
        p = p / p.sum(axis=-1, keepdims=True)
    return p


def router_agreement(h_star: np.ndarray, h_draft: np.ndarray, layer: Dict[str, object], dtype=np.float64):
    """Per row: KL( R_l(h*_t) || R_l(h^d_t) ), whose sum over rows and layers is L_router (Eq. 10), and the
    number of experts that TopK_l(h*_t) and TopK_l(h^d_t) have in common (the top-k set agreement that Sec. 3.3
    tracks as a validation metric).  Also returns the two selections."""
    sh = layer["shape"]
    zs = router_logits(h_star, layer["router"], layer["bias"], dtype)
    zd = router_logits(h_draft, layer["router"], layer["bias"], dtype)
    ps, pd = router_distribution(zs, sh.score_fn), router_distribution(zd, sh.score_fn)
    kl = np.zeros(zs.shape[0], dtype)
    for t in range(zs.shape[0]):
        for e in range(zs.shape[1]):
            if ps[t, e] > 0.0:
                kl[t] += ps[t, e] * (np.log(ps[t, e]) - np.log(pd[t, e]))
    ids_s = topk_select(router_probs(zs, sh.score_fn), sh.top_k)
    ids_d = topk_select(router_probs(zd, sh.score_fn), sh.top_k)
    agree = np.array([len(set(ids_s[t].tolist()) & set(ids_d[t].tolist())) for t in range(zs.shape[0])], np.int32)
    return kl, agree, ids_s, ids_d


# --------------------------------------------------------------------------
# Eq. 2 / Eq. 3: the block's expert set and the pair permutation grouped by expert.
# --------------------------------------------------------------------------
def block_union(ids: np.ndarray, n_experts: int):
    """U_l(D) = union over block tokens of TopK_l(h_t)  (Eq. 2, Eq. 3).

    Returns (mask words u64 [ceil(E/64)], union_ids ascending, offsets[E+1],
    perm[K*k]).  ``perm`` lists the pair indices p = t*k + j ordered by
    (expert id, p); ``offsets[e] .. offsets[e+1]`` is expert e's segment, so
    ``offsets[e+1]-offsets[e]`` is the number of block tokens routed to e.
    """
    K, k = ids.shape
    members = [e for e in range(n_experts) if any(int(ids[t, j]) == e for t in range(K) for j in range(k))]
    mask = np.zeros((n_experts + 63) // 64, dtype=np.uint64)
    for e in members:
        mask[e // 64] |= np.uint64(1) << np.uint64(e % 64)
    pairs = sorted(range(K * k), key=lambda p: (int(ids[p // k, p % k]), p))
    offsets = np.zeros(n_experts + 1, dtype=np.int32)
    for e in range(n_experts):
        offsets[e + 1] = offsets[e] + sum(1 for p in pairs if int(ids[p // k, p % k]) == e)
    return mask, np.asarray(members, np.int32), offsets, np.asarray(pairs, np.int32)


def block_cost(union_sizes: Sequence[int], cost_per_expert: float = 1.0) -> float:
    """C(B) = sum_l sum_{e in U_l(B)} c_{l,e} with a uniform per-expert cost (Eq. 2)."""
    return float(sum(union_sizes)) * cost_per_expert


# --------------------------------------------------------------------------
# Algorithm 1, last two lines: exact greedy verification.
# --------------------------------------------------------------------------
def lm_logits(h: np.ndarray, W_lm: np.ndarray, dtype=np.float64) -> np.ndarray:
    return np.asarray(h, dtype) @ np.asarray(W_lm, dtype).T


def greedy_accept(h: np.ndarray, W_lm: np.ndarray, draft: np.ndarray, dtype=np.float64,
                  logits: Optional[np.ndarray] = None):
    """Target tokens t_i = argmax_v (W_lm h_i)_v (lowest v on ties); accepted
    length n = longest prefix with t_i == d_i; ``next`` = t_n, the target's own
    token after the accepted prefix, or -1 when no row is left for it."""
    lg = lm_logits(h, W_lm, dtype) if logits is None else logits
    M = lg.shape[0]
    target = np.empty(M, dtype=np.int32)
    for i in range(M):
        best = 0
        for v in range(1, lg.shape[1]):
            if lg[i, v] > lg[i, best]:
                best = v
        target[i] = best
    K = len(draft)
    n = 0
    while n < K and n < M and int(draft[n]) == int(target[n]):
        n += 1
    nxt = int(target[n]) if n < M else -1
    return target, n, nxt, lg


def greedy_accept_fast(h, W_lm, draft, dtype=np.float64):
    """Same result as :func:`greedy_accept`, with numpy's argmax (first
    maximum) in place of the explicit scan -- for full-size vocabularies."""
    lg = lm_logits(h, W_lm, dtype)
    target = lg.argmax(axis=1).astype(np.int32)
    K, M = len(draft), lg.shape[0]
    n = 0
    while n < K and n < M and int(draft[n]) == int(target[n]):
        n += 1
    nxt = int(target[n]) if n < M else -1
    return target, n, nxt, lg


# --------------------------------------------------------------------------
# Layer stack with the attention sub-layer stubbed out (synthetic workloads).
# --------------------------------------------------------------------------
def rmsnorm(h: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    return h / np.sqrt((h * h).mean(axis=-1, keepdims=True) + eps)


def stack_layer_target(h: np.ndarray, layer, dtype=np.float64, norm: bool = True, forced_ids=None):
    """One pre-norm residual MoE sub-layer: h + MoE(RMSNorm(h))."""
    h = np.asarray(h, dtype)
    x = rmsnorm(h) if norm else h
    y, ids, g, z = moe_target(x, layer, dtype, forced_ids)
    return h + y, ids, g, z


def stack_layer_draft(h: np.ndarray, layer, dtype=np.float64, norm: bool = True, forced_ids=None):
    h = np.asarray(h, dtype)
    x = rmsnorm(h) if norm else h
    y, ids, g, z = moe_draft(x, layer, dtype, forced_ids)
    return h + y, ids, g, z


# --------------------------------------------------------------------------
# Sec. 3.4: confidence of a draft token and confidence-expansion truncation.
# --------------------------------------------------------------------------
def draft_confidence(h: np.ndarray, W_lm: np.ndarray, dtype=np.float64):
    """Draft token = argmax of the draft logits; q = its softmax probability (the reading taken for
    "a confidence score from the draft logits")."""
    lg = lm_logits(h, W_lm, dtype)
    e = np.exp(lg - lg.max(axis=1, keepdims=True))
    prob = e / e.sum(axis=1, keepdims=True)
    tok = lg.argmax(axis=1).astype(np.int32)
    return tok, prob[np.arange(lg.shape[0]), tok], lg


class TruncationController:
    """U_hat_i = union_{j<=i} union_l E_hat_{l,j} (Eq. 12) as a set of (layer, expert) pairs;
    Delta_i = |U_hat_i| - |U_hat_{i-1}| (Eq. 13); stop before appending token i when q_i < tau and
    Delta_i > B_i (Eq. 14); a stopped candidate leaves U_hat as it was (Algorithm 1)."""

    def __init__(self):
        self.u_hat = set()

    def reset(self):
        self.u_hat = set()

    def propose(self, predicted, q, tau, budget):
        cand = self.u_hat | {(l, int(e)) for l, row in enumerate(predicted) for e in row}
        delta = len(cand) - len(self.u_hat)
        stop = (q < tau) and (delta > budget)
        new = sorted(cand - self.u_hat)
        if not stop:
            self.u_hat = cand
        return stop, delta, ([] if stop else new)
