"""Pins for the CPU checker: each test ties one of its functions to something
other than itself -- the paper's printed numbers, a closed form, a library
routine written differently, a dense / brute-force evaluation or an invariant
-- so that a dropped term, a wrong sign or index, or a transposed operand in
``oracle/moe_oracle.py`` fails at least one of them."""
import dataclasses
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _layer(shape=None, seed=0, zipf=False, std=0.02):
    shape = shape or synth.shape_tiny()
    return synth.layer_to_numpy(synth.make_layer(shape, seed, "cpu", std=std, zipf=zipf))


def _h(K, H, seed=1, rho=0.0):
    return synth.hidden_block(K, H, seed, rho).numpy().astype(np.float64)


# ---------------------------------------------------------------- shapes ----
def test_parameter_split_matches_paper_numbers():
    """Sec. 2.1: 14.4 B routed parameters = 26.8 GiB in BF16; top-6 of 64 = 9.4 %."""
    gold = {}
    for line in open(os.path.join(GOLDEN, "v2lite_parameter_split.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            gold[k] = float(v)
    sh = synth.shape_v2lite()
    moe_layers = int(gold["layers"]) - 1          # the first transformer layer is dense
    n = moe_layers * sh.n_experts * 3 * sh.hidden * sh.inter
    assert sh.n_experts == gold["routed_experts"] and sh.top_k == gold["top_k"]
    assert round(n / 1e9, 1) == gold["routed_params_billion"]
    assert round(n * 2 / 2**30, 1) == gold["routed_bf16_gib"]
    assert round(100.0 * sh.top_k / sh.n_experts, 1) == gold["topk_fraction_percent"]
    assert sh.expert_bytes() == 17301504


# ---------------------------------------------------------------- router ----
def test_router_logits_orientation_and_bias():
    """z[t,e] = <W_r[e,:], h[t,:]> + b[e]: one-hot probes catch a transposed operand."""
    E, H = 5, 7
    W = np.arange(E * H, dtype=np.float64).reshape(E, H)
    b = np.array([10., 20., 30., 40., 50.])
    h = np.zeros((2, H)); h[0, 3] = 1.0; h[1, 6] = 2.0
    z = O.router_logits(h, W, b)
    assert z.shape == (2, E)
    assert np.array_equal(z[0], W[:, 3] + b)
    assert np.array_equal(z[1], 2 * W[:, 6] + b)


def test_router_probs_against_torch_and_closed_forms():
    rng = np.random.default_rng(0)
    z = rng.normal(size=(6, 16)) * 3
    p = O.router_probs(z, O.SCORE_SOFTMAX)
    assert np.allclose(p.sum(1), 1.0, atol=1e-14)
    assert np.allclose(p, torch.softmax(torch.from_numpy(z), dim=1).numpy(), atol=1e-15)
    # shift invariance and the two-class closed form softmax([a,b])[0] = sigmoid(a-b)
    assert np.allclose(O.router_probs(z + 100.0, O.SCORE_SOFTMAX), p, atol=1e-13)
    two = O.router_probs(np.array([[1.5, -0.5]]), O.SCORE_SOFTMAX)
    assert abs(two[0, 0] - 1 / (1 + math.exp(-2.0))) < 1e-15
    s = O.router_probs(z, O.SCORE_SIGMOID)
    assert np.allclose(s, torch.sigmoid(torch.from_numpy(z)).numpy(), atol=1e-15)
    assert abs(O.router_probs(np.zeros((1, 1)), O.SCORE_SIGMOID)[0, 0] - 0.5) < 1e-16


def test_topk_select_bruteforce_ties_and_order():
    rng = np.random.default_rng(1)
    p = rng.random((20, 12))
    ids = O.topk_select(p, 4)
    tk = torch.topk(torch.from_numpy(p), 4, dim=1).indices.numpy()
    assert np.array_equal(ids, tk)                       # distinct values: unique answer
    for t in range(20):                                  # brute force over all 4-subsets
        best = max(itertools.combinations(range(12), 4), key=lambda c: sum(p[t, list(c)]))
        assert set(best) == set(ids[t])
        assert list(p[t, ids[t]]) == sorted(p[t, ids[t]], reverse=True)
    tie = np.array([[0.2, 0.5, 0.5, 0.1, 0.5, 0.2]])
    assert list(O.topk_select(tie, 4)[0]) == [1, 2, 4, 0]  # equal scores -> ascending id


def test_gate_weights_normalisation_scale_and_dense_limit():
    rng = np.random.default_rng(2)
    z = rng.normal(size=(5, 8))
    p = O.router_probs(z, O.SCORE_SOFTMAX)
    ids = O.topk_select(p, 3)
    g = O.gate_weights(p, ids, 1, 2.5)
    assert np.allclose(g.sum(1), 2.5)
    assert np.allclose(g[:, 0] / g[:, 1], p[np.arange(5), ids[:, 0]] / p[np.arange(5), ids[:, 1]])
    g_raw = O.gate_weights(p, ids, 0, 1.0)
    assert np.array_equal(g_raw, p[np.arange(5)[:, None], ids])
    # k = E: the selection is everything, normalised gates are s * softmax (dense MoE)
    ids_all = O.topk_select(p, 8)
    g_all = O.gate_weights(p, ids_all, 1, 1.7)
    dense = np.zeros_like(p)
    dense[np.arange(5)[:, None], ids_all] = g_all
    assert np.allclose(dense, 1.7 * p, atol=1e-15)
    # monotone score functions select the same set as the raw logits
    for fn in (O.SCORE_SOFTMAX, O.SCORE_SIGMOID):
        sel = O.topk_select(O.router_probs(z, fn), 3)
        assert np.array_equal(sel, np.argsort(-z, axis=1, kind="stable")[:, :3])


# --------------------------------------------------------------- experts ----
def test_silu_against_library_and_values():
    x = np.linspace(-8, 8, 41)
    assert np.allclose(O.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy(), atol=1e-15)
    assert O.silu(np.array([0.0]))[0] == 0.0
    assert abs(O.silu(np.array([1.0]))[0] - 1 / (1 + math.exp(-1))) < 1e-16
    assert abs(O.silu(np.array([-1.0]))[0] + 1 / (1 + math.e)) < 1e-16


def test_swiglu_closed_form_and_operand_roles():
    """Hand-built 2->3->2 expert: every matrix has a distinct role and shape, so
    swapping gate/up, transposing W_d or dropping the activation changes the result."""
    Wg = np.array([[1., 0.], [0., 1.], [1., 1.]])        # [I=3, H=2]
    Wu = np.array([[2., 0.], [0., 3.], [1., -1.]])
    Wd = np.array([[1., 0., 2.], [0., 1., -1.]])          # [H=2, I=3]
    h = np.array([0.5, -2.0])
    sig = lambda v: 1 / (1 + math.exp(-v))
    a = [0.5 * sig(0.5) * 1.0, -2.0 * sig(-2.0) * -6.0, -1.5 * sig(-1.5) * 2.5]
    want = np.array([a[0] + 2 * a[2], a[1] - a[2]])
    got = O.swiglu_expert(h, Wg, Wu, Wd)
    assert np.allclose(got, want, atol=1e-15)
    # library formulation in torch, batched and written differently
    rng = np.random.default_rng(3)
    Wg, Wu, Wd = rng.normal(size=(6, 4)), rng.normal(size=(6, 4)), rng.normal(size=(4, 6))
    hb = rng.normal(size=(3, 4))
    T = torch.from_numpy
    ref = (torch.nn.functional.silu(T(hb) @ T(Wg).T) * (T(hb) @ T(Wu).T)) @ T(Wd).T
    for t in range(3):
        assert np.allclose(O.swiglu_expert(hb[t], Wg, Wu, Wd), ref[t].numpy(), atol=1e-13)
    assert np.array_equal(O.swiglu_expert(np.zeros(4), Wg, Wu, Wd), np.zeros(4))
    assert np.array_equal(O.swiglu_expert(hb[0], np.zeros_like(Wg), Wu, Wd), np.zeros(4))


# ------------------------------------------------------- target layer (Eq. 4)
def test_target_equals_dense_gate_matrix_evaluation():
    """Evaluate ALL experts for every token, then contract with a dense gate
    matrix that is zero off the top-k: must equal the routed sum of Eq. 4."""
    L = _layer(std=0.3)
    sh = L["shape"]
    h = _h(5, sh.hidden)
    y, ids, g, z = O.moe_target(h, L)
    T = torch.from_numpy
    Wg, Wu, Wd = (T(w.astype(np.float64)) for w in L["experts"])
    hb = T(h)
    allexp = torch.einsum("ehi,tei->teh", Wd,
                          torch.nn.functional.silu(torch.einsum("eih,th->tei", Wg, hb))
                          * torch.einsum("eih,th->tei", Wu, hb))
    G = torch.zeros(5, sh.n_experts, dtype=torch.float64)
    probs = torch.softmax(hb @ T(L["router"].astype(np.float64)).T, dim=1)
    top = torch.topk(probs, sh.top_k, dim=1)
    G.scatter_(1, top.indices, top.values / top.values.sum(1, keepdim=True))
    sg, su, sd = (T(w.astype(np.float64)) for w in L["shared"][0])
    shared = (torch.nn.functional.silu(hb @ sg.T) * (hb @ su.T)) @ sd.T
    dense = shared + torch.einsum("te,teh->th", G, allexp)
    assert np.array_equal(ids, top.indices.numpy())
    assert np.allclose(y, dense.numpy(), rtol=1e-12, atol=1e-14)


def test_target_special_cases():
    L = _layer(std=0.3)
    sh = L["shape"]
    h = _h(3, sh.hidden, seed=4)
    # identical routed experts: routing no longer matters, y = S(h) + s * E(h)
    Wg, Wu, Wd = L["experts"]
    same = dict(L)
    same["experts"] = (np.repeat(Wg[:1], sh.n_experts, 0), np.repeat(Wu[:1], sh.n_experts, 0),
                       np.repeat(Wd[:1], sh.n_experts, 0))
    same["shape"] = dataclasses.replace(sh, routed_scale=1.7)
    y, _, g, _ = O.moe_target(h, same)
    for t in range(3):
        want = O.shared_path(h[t], L["shared"]) + 1.7 * O.swiglu_expert(h[t], Wg[0], Wu[0], Wd[0])
        assert np.allclose(y[t], want, rtol=1e-12)
    # h = 0 -> y = 0 ; duplicated rows -> identical outputs
    assert np.array_equal(O.moe_target(np.zeros((2, sh.hidden)), L)[0], np.zeros((2, sh.hidden)))
    hd = np.stack([h[0], h[1], h[0]])
    yd = O.moe_target(hd, L)[0]
    assert np.array_equal(yd[0], yd[2])
    # two shared experts add (unit weight each)
    two = dict(L)
    two["shared"] = [L["shared"][0], L["draft"]]
    y2 = O.moe_target(h, two)[0]
    y1 = O.moe_target(h, L)[0]
    for t in range(3):
        assert np.allclose(y2[t] - y1[t], O.swiglu_expert(h[t], *L["draft"]), rtol=1e-10, atol=1e-14)


# -------------------------------------------------------- drafter (Eq. 5, 6)
def test_draft_identities():
    L = _layer(std=0.3)
    sh = L["shape"]
    h = _h(4, sh.hidden, seed=5)
    y_star, ids, g, _ = O.moe_target(h, L)
    y_d0, ids_d, g_d, _ = O.moe_draft(h, L, gamma=0.0)
    assert np.array_equal(ids, ids_d) and np.array_equal(g, g_d)   # same router, same gates
    Wg, Wu, Wd = L["experts"]
    m_star = O.missing_residual(h, L)
    for t in range(4):
        # Eq. 6: what is missing from the top-1 path is exactly the other k-1 routed terms
        rest = sum(g[t, j] * O.swiglu_expert(h[t], Wg[ids[t, j]], Wu[ids[t, j]], Wd[ids[t, j]])
                   for j in range(1, sh.top_k))
        assert np.allclose(y_star[t] - y_d0[t], rest, rtol=1e-10, atol=1e-14)
        assert np.allclose(m_star[t], rest, rtol=1e-10, atol=1e-14)
        # e1 is the router's argmax
        z = O.router_logits(h[t:t + 1], L["router"], L["bias"])
        assert ids_d[t, 0] == int(np.argmax(z[0]))
    # linear in gamma, and the draft term is gamma * E^d(h)
    y_g = O.moe_draft(h, L, gamma=0.75)[0]
    for t in range(4):
        assert np.allclose(y_g[t] - y_d0[t], 0.75 * O.swiglu_expert(h[t], *L["draft"]), rtol=1e-10, atol=1e-14)
    # k = 1 and gamma = 0: the drafter IS the target layer
    L1 = dict(L); L1["shape"] = dataclasses.replace(sh, top_k=1)
    assert np.allclose(O.moe_draft(h, L1, gamma=0.0)[0], O.moe_target(h, L1)[0], rtol=1e-13)
    # shared + top-r with r = k and gamma = 0 is the target layer too
    assert np.allclose(O.moe_draft(h, L, gamma=0.0, top_r=sh.top_k)[0], y_star, rtol=1e-13)


# ------------------------------------------------------ Sec. 3.3: evaluation terms (Eq. 6, 7, 10)
def test_router_agreement_closed_forms():
    TINY = synth.shape_tiny()
    sh = dataclasses.replace(TINY, n_experts=2, top_k=1)
    L = synth.layer_to_numpy(synth.make_layer(sh, 21, "cpu"))
    # two experts, softmax: R = (s, 1 - s) with s = sigmoid(z0 - z1); KL of two Bernoullis in closed form
    rng = np.random.default_rng(22)
    hs, hd = rng.standard_normal((3, sh.hidden)), rng.standard_normal((3, sh.hidden))
    kl, agree, ids_s, ids_d = O.router_agreement(hs, hd, L)
    zs, zd = O.router_logits(hs, L["router"], L["bias"]), O.router_logits(hd, L["router"], L["bias"])
    for t in range(3):
        a = 1.0 / (1.0 + math.exp(-(zs[t, 0] - zs[t, 1])))
        b = 1.0 / (1.0 + math.exp(-(zd[t, 0] - zd[t, 1])))
        want = a * math.log(a / b) + (1 - a) * math.log((1 - a) / (1 - b))
        assert abs(kl[t] - want) <= 1e-12 * max(1.0, abs(want))
        assert agree[t] == int((zs[t, 0] >= zs[t, 1]) == (zd[t, 0] >= zd[t, 1]))
    # identical hidden states: zero divergence, full agreement; KL is never negative and is not symmetric
    sh6 = TINY
    L6 = synth.layer_to_numpy(synth.make_layer(sh6, 23, "cpu"))
    h = rng.standard_normal((4, sh6.hidden))
    kl0, ag0, _, _ = O.router_agreement(h, h, L6)
    assert np.all(np.abs(kl0) <= 1e-15) and np.all(ag0 == sh6.top_k)
    h2 = h + 0.5 * rng.standard_normal(h.shape)
    kl_ab, ag_ab, ia, ib = O.router_agreement(h, h2, L6)
    kl_ba, ag_ba, _, _ = O.router_agreement(h2, h, L6)
    assert np.all(kl_ab >= 0) and np.all(kl_ba >= 0) and not np.allclose(kl_ab, kl_ba)
    assert np.array_equal(ag_ab, ag_ba) and np.all(ag_ab <= sh6.top_k)
    for t in range(4):
        assert ag_ab[t] == len(np.intersect1d(ia[t], ib[t]))
    # against the library routine on the same distributions
    from scipy.special import rel_entr, softmax
    za = O.router_logits(h, L6["router"], L6["bias"]); zb = O.router_logits(h2, L6["router"], L6["bias"])
    assert np.allclose(kl_ab, rel_entr(softmax(za, axis=1), softmax(zb, axis=1)).sum(axis=1), rtol=1e-10, atol=1e-14)
    # sigmoid routers: scores normalised to a distribution first (the reading), so scaling has no effect
    Ls = dict(L6); Ls["shape"] = dataclasses.replace(sh6, score_fn=synth.SCORE_SIGMOID)
    kls, _, _, _ = O.router_agreement(h, h2, Ls)
    pa = 1 / (1 + np.exp(-za)); pb = 1 / (1 + np.exp(-zb))
    assert np.allclose(kls, rel_entr(pa / pa.sum(1, keepdims=True), pb / pb.sum(1, keepdims=True)).sum(axis=1),
                       rtol=1e-10, atol=1e-14)


def test_residual_loss_identities():
    TINY = synth.shape_tiny()
    sh = TINY
    L = synth.layer_to_numpy(synth.make_layer(sh, 24, "cpu"))
    rng = np.random.default_rng(25)
    h = rng.standard_normal((3, sh.hidden))
    # Eq. 7 with gamma = 0 is the squared norm of the missing residual; it is quadratic in gamma in general
    m = O.missing_residual(h, L)
    L0 = dict(L); L0["shape"] = dataclasses.replace(sh, draft_gamma=0.0)
    assert abs(O.residual_loss(h, h, L0) - float((m * m).sum())) <= 1e-12 * float((m * m).sum())
    d = np.stack([O.swiglu_expert(h[t], *L["draft"]) for t in range(3)])
    for gam in (0.5, 1.0, -2.0):
        Lg = dict(L); Lg["shape"] = dataclasses.replace(sh, draft_gamma=gam)
        want = float(((gam * d - m) ** 2).sum())
        assert abs(O.residual_loss(h, h, Lg) - want) <= 1e-12 * want
        assert np.allclose(O.draft_expert_term(h, Lg), gam * d, rtol=1e-13)
    # a draft expert that reproduces the residual exactly has zero loss: y_d == y* then (Eq. 5 vs Eq. 4)
    y_star = O.moe_target(h, L)[0]
    y_top1 = O.moe_draft(h, L, gamma=0.0)[0]
    assert np.allclose(y_top1 + m, y_star, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------ 4-bit block-quantised experts (Sec. 4, mobile runs)
def test_q4_blocks_round_trip_and_error_bound():
    rng = np.random.default_rng(30)
    w = torch.from_numpy(rng.standard_normal((5, 96)).astype(np.float32) * 0.02)
    w[0, :32] = 0.0                                  # an all-zero block: scale 0, every weight 0
    w[1, 7] = -0.2                                   # a block whose extreme is negative: d > 0, code 0 is the extreme
    w[2, 40] = 0.3                                   # ... and one whose extreme is positive: d < 0
    blocks = synth.quantize_q4_0(w).numpy()
    assert blocks.shape == (5, 3, 18)
    deq = O.dequantize_q4_0(blocks)
    x = w.numpy().astype(np.float64)
    for r in range(5):
        for b in range(3):
            seg, got = x[r, 32 * b:32 * b + 32], deq[r, 32 * b:32 * b + 32]
            d = float(np.frombuffer(blocks[r, b, :2].tobytes(), dtype="<f2")[0])
            i_ext = int(np.argmax(np.abs(seg)))
            if seg[i_ext] == 0.0:
                assert d == 0.0 and np.all(got == 0.0)
                continue
            # the scale is the extreme over -8, rounded to fp16, and the extreme gets code 0
            assert d == float(np.float16(seg[i_ext] / -8.0))
            assert got[i_ext] == -8.0 * d
            # every weight lies on the grid d * {-8..7}; the error is at most half a step, except where a value
            # of the sign opposite to the extreme would need code 16 and is clipped to 15 (at most one step);
            # rounding the scale to fp16 moves the grid by at most 8 * |d| * 2^-11
            codes = got / d
            assert np.all(codes == np.round(codes)) and codes.min() >= -8 and codes.max() <= 7
            slack = 8 * abs(d) * 2.0 ** -11 + 1e-12
            clipped = (seg / (seg[i_ext] / -8.0)) > 7.5
            assert np.all(np.abs(got - seg)[~clipped] <= 0.5 * abs(d) + slack)
            assert np.all(np.abs(got - seg)[clipped] <= 1.0 * abs(d) + slack)
    # values already on a block's grid are reproduced exactly; blocks do not influence each other
    d0 = float(np.float16(0.0123))
    grid = torch.tensor([[d0 * (c - 8) for c in range(16)] * 2], dtype=torch.float32)
    assert np.array_equal(O.dequantize_q4_0(synth.quantize_q4_0(grid).numpy())[0], grid.numpy()[0].astype(np.float64))
    w2 = w.clone(); w2[3, 64:] *= 5.0
    b2 = synth.quantize_q4_0(w2).numpy()
    assert np.array_equal(b2[3, :2], blocks[3, :2]) and not np.array_equal(b2[3, 2], blocks[3, 2])
    # nibble order: low nibbles are weights 0..15 of the block, high nibbles weights 16..31
    ramp = torch.tensor([[-8.0 + (j % 16) for j in range(32)]], dtype=torch.float32)   # extreme -8 -> d = 1
    rb = synth.quantize_q4_0(ramp).numpy()[0, 0]
    assert float(np.frombuffer(rb[:2].tobytes(), dtype="<f2")[0]) == 1.0
    assert [int(v & 15) for v in rb[2:]] == list(range(16)) and [int(v >> 4) for v in rb[2:]] == list(range(16))
    # expert blob: three matrices one after the other, 18 bytes per 32 weights
    Wg = torch.from_numpy(rng.standard_normal((8, 64)).astype(np.float32))
    Wd = torch.from_numpy(rng.standard_normal((64, 32)).astype(np.float32))
    blob = synth.q4_expert_blob(Wg, Wg * 2, Wd)
    assert blob.numel() == (8 * 64 * 2 + 64 * 32) * 18 // 32
    assert np.array_equal(blob[:8 * 2 * 18].numpy().reshape(8, 2, 18), synth.quantize_q4_0(Wg).numpy())


# ------------------------------------------------------ union (Eq. 2, Eq. 3)
def test_block_union_enumeration_and_invariants():
    rng = np.random.default_rng(6)
    for K, k, E in [(1, 6, 64), (4, 6, 64), (8, 2, 8), (16, 6, 64), (5, 3, 130)]:
        ids = np.stack([rng.choice(E, size=k, replace=False) for _ in range(K)]).astype(np.int32)
        mask, uids, offsets, perm = O.block_union(ids, E)
        want = sorted(set(ids.flatten().tolist()))
        assert uids.tolist() == want
        bits = [e for e in range(E) if (int(mask[e // 64]) >> (e % 64)) & 1]
        assert bits == want
        assert k <= len(want) <= min(E, K * k)
        if K == 1:
            assert len(want) == k
        assert sorted(perm.tolist()) == list(range(K * k))            # bijection
        assert offsets[0] == 0 and offsets[-1] == K * k and np.all(np.diff(offsets) >= 0)
        for e in range(E):
            seg = perm[offsets[e]:offsets[e + 1]]
            toks = [int(p) // k for p in seg]
            assert toks == sorted(t for t in range(K) if e in ids[t])  # exactly e's tokens, ascending
            assert all(ids[p // k, p % k] == e for p in seg)
    # duplicate rows: the union does not grow
    ids = np.array([[3, 1, 2], [3, 1, 2]], np.int32)
    assert O.block_union(ids, 8)[1].tolist() == [1, 2, 3]


def test_union_size_closed_form_under_uniform_routing():
    """Unbiased i.i.d. routing: E|U| = E (1 - (1 - k/E)^K)."""
    rng = np.random.default_rng(7)
    E, k = 64, 6
    for K in (2, 4, 8):
        sizes = []
        for _ in range(400):
            ids = np.stack([rng.choice(E, size=k, replace=False) for _ in range(K)]).astype(np.int32)
            sizes.append(len(O.block_union(ids, E)[1]))
        want = E * (1 - (1 - k / E) ** K)
        assert abs(np.mean(sizes) - want) < 0.35
    assert O.block_cost([3, 4, 5], 2.0) == 24.0


# ------------------------------------------------- greedy verification (Alg. 1)
def test_greedy_accept_invariants():
    H, V = 16, 16
    eye = np.eye(V, H)
    rng = np.random.default_rng(8)
    h = rng.normal(size=(5, H))
    target, n, nxt, lg = O.greedy_accept(h, eye, np.argmax(h[:4], axis=1))
    assert np.array_equal(target, np.argmax(h, axis=1))      # identity head: argmax of h itself
    assert n == 4 and nxt == target[4]                        # draft == target accepts all, bonus row 5
    d = target[:4].copy()
    assert O.greedy_accept(h[:4], eye, d)[1:3] == (4, -1)     # no spare row: nothing after the prefix
    d0 = d.copy(); d0[0] = (d0[0] + 1) % V
    assert O.greedy_accept(h, eye, d0)[1:3] == (0, int(target[0]))
    for j in range(4):                                        # first mismatch at j -> n = j
        dj = d.copy(); dj[j] = (dj[j] + 1) % V
        t2, n2, nx2, _ = O.greedy_accept(h, eye, dj)
        assert (n2, nx2) == (j, int(target[j]))
        dj[j + 1:] = rng.integers(0, V, size=3 - j)           # the tail never matters
        assert O.greedy_accept(h, eye, dj)[1] == j
    # ties resolve to the lowest vocabulary id
    W = np.zeros((6, 3)); W[2, 0] = W[4, 0] = 1.0
    assert O.greedy_accept(np.array([[2.0, 0, 0]]), W, np.array([2]))[0][0] == 2
    # orientation of the head: logits[i, v] = <W_lm[v], h_i>
    Wr = rng.normal(size=(7, H))
    assert np.allclose(O.lm_logits(h, Wr), np.einsum("vh,ih->iv", Wr, h))
    a = O.greedy_accept(h, Wr, np.array([1, 2, 3]))
    b = O.greedy_accept_fast(h, Wr, np.array([1, 2, 3]))
    assert np.array_equal(a[0], b[0]) and a[1:3] == b[1:3]


def test_exactness_of_speculation_on_a_toy_chain():
    """Whatever the drafter proposes, emitting the accepted prefix plus the
    target's own next token reproduces plain greedy decoding of the target."""
    L = _layer(std=0.3)
    sh = L["shape"]
    V = 32
    emb = synth.normal((V, sh.hidden), 1.0, 11, "emb", torch.float32).numpy().astype(np.float64)
    head = synth.normal((V, sh.hidden), 0.3, 11, "head", torch.float32).numpy().astype(np.float64)

    def target_next(tok):
        hid = O.stack_layer_target(emb[tok][None], L)[0]
        return int(np.argmax(O.lm_logits(O.rmsnorm(hid), head)[0]))

    def draft_next(tok):
        hid = O.stack_layer_draft(emb[tok][None], L)[0]
        return int(np.argmax(O.lm_logits(O.rmsnorm(hid), head)[0]))

    ar = [3]
    while len(ar) < 20:
        ar.append(target_next(ar[-1]))
    out = [3]
    while len(out) < 20:
        drafts, cur = [], out[-1]
        for _ in range(4):
            cur = draft_next(cur); drafts.append(cur)
        rows = np.stack([O.stack_layer_target(emb[t][None], L)[0][0] for t in [out[-1]] + drafts])
        target, n, nxt, _ = O.greedy_accept(O.rmsnorm(rows), head, np.array(drafts))
        out.extend(drafts[:n]); out.append(nxt)
    assert out[:20] == ar


def test_rmsnorm_and_precision_option():
    x = np.array([[3.0, 4.0]])
    assert np.allclose(O.rmsnorm(x, eps=0.0), x / math.sqrt(12.5))
    L = _layer()
    h = _h(2, L["shape"].hidden, seed=9)
    y64 = O.moe_target(h, L)[0]
    y32 = O.moe_target(h, L, dtype=np.float32)[0]
    assert y32.dtype == np.float32
    assert np.max(np.abs(y32 - y64)) <= 1e-5 * np.max(np.abs(y64))


def test_selection_gaps():
    z = np.array([[5.0, 1.0, 4.0, 3.9995, 0.0]])
    order_gap, set_gap = O.selection_gaps(z, 2)
    assert abs(set_gap[0] - 0.0005) < 1e-12 and abs(order_gap[0] - 0.0005) < 1e-12
    order_gap, set_gap = O.selection_gaps(z, 3)
    assert abs(order_gap[0] - 0.0005) < 1e-12 and abs(set_gap[0] - 2.9995) < 1e-12
