"""Confidence-expansion truncation (Sec. 3.4, Eq. 12-14): pins of the checker's controller and parity of the
library's host-side controller with it.  No GPU needed."""
import numpy as np
import torch

from oracle import moe_oracle as O


def test_controller_model_pins():
    c = O.TruncationController()
    # Eq. 12/13 by hand: two layers, k = 2
    stop, d, new = c.propose([[1, 2], [1, 3]], q=0.9, tau=0.5, budget=0)
    assert (stop, d) == (False, 4) and new == [(0, 1), (0, 2), (1, 1), (1, 3)]      # same id in two layers counts twice
    stop, d, new = c.propose([[2, 5], [3, 1]], q=0.9, tau=0.5, budget=0)
    assert (stop, d, new) == (False, 1, [(0, 5)])
    # Eq. 14 truth table: stop only when BOTH unlikely (q < tau) and expensive (delta > budget)
    for q, budget, want in [(0.4, 0, True), (0.4, 2, False), (0.6, 0, False), (0.6, 2, False)]:
        c2 = O.TruncationController(); c2.u_hat = set(c.u_hat)
        stop, d, new = c2.propose([[7, 8], [3, 1]], q=q, tau=0.5, budget=budget)
        assert d == 2 and stop == want
        assert (c2.u_hat == c.u_hat) == want            # a stopped candidate leaves the set unchanged
    assert c.propose([[1, 2], [1, 3]], 0.0, 1.0, 0)[:2] == (False, 0)               # nothing new is never "expensive"
    c.reset()
    assert c.propose([[1, 1], [1, 1]], 0.9, 0.5, 0)[1] == 2


def test_confidence_is_max_softmax_probability():
    rng = np.random.default_rng(0)
    h, W = rng.normal(size=(3, 16)), rng.normal(size=(50, 16))
    tok, q, lg = O.draft_confidence(h, W)
    prob = torch.softmax(torch.from_numpy(lg), dim=1).numpy()
    assert np.array_equal(tok, prob.argmax(1)) and np.allclose(q, prob.max(1), atol=1e-15)
    assert np.all(q > 1 / 50) and np.all(q <= 1)
    # uniform logits: q = 1/V
    assert abs(O.draft_confidence(np.zeros((1, 16)), W)[1][0] - 1 / 50) < 1e-15


def test_library_controller_matches_model():
    from paper_2607_24434_b200 import binding
    L, E, k = 5, 70, 6
    rng = np.random.default_rng(3)
    lib, ref = binding.Controller(L, E), O.TruncationController()
    for step in range(200):
        if rng.random() < 0.15:
            lib.reset(); ref.reset()
        pred = [rng.choice(E, size=k, replace=False).tolist() for _ in range(L)]
        q, tau, budget = float(rng.random()), 0.5, int(rng.integers(0, 20))
        a, b = lib.propose(pred, q, tau, budget), ref.propose(pred, q, tau, budget)
        assert a[0] == b[0] and a[1] == b[1] and sorted(a[2]) == b[2]
        assert lib.size() == len(ref.u_hat)
    lib.close()
