"""Pins of the oracle router (Eq. 1): closed forms, invariants, brute force, and a library routine."""
import itertools

import numpy as np
import torch

from oracle import router as orouter


def test_closed_form_probabilities_and_order():
    # logits ln 1..ln 4 -> probabilities 0.1, 0.2, 0.3, 0.4; identity router so z = h
    h = np.log(np.array([1.0, 2.0, 3.0, 4.0]))
    ids, p, z = orouter.route_token(h, np.eye(4), 2)
    assert ids.tolist() == [3, 2]
    np.testing.assert_allclose(p, [0.4, 0.3], rtol=1e-14)
    np.testing.assert_allclose(orouter.softmax(z), [0.1, 0.2, 0.3, 0.4], rtol=1e-14)
    # weights are NOT renormalised over the selected k (Section 3.4)
    assert abs(p.sum() - 0.7) < 1e-14


def test_logits_are_the_matrix_vector_product_with_bias():
    rng = np.random.default_rng(0)
    w = rng.standard_normal((5, 7))
    h = rng.standard_normal(7)
    b = rng.standard_normal(5)
    _, _, z = orouter.route_token(h, w, 2, bias=b)
    for e in range(5):                                   # the definition, term by term
        assert abs(z[e] - (sum(w[e, j] * h[j] for j in range(7)) + b[e])) < 1e-12
    # transposed operand or dropped bias would fail:
    assert not np.allclose(z, w @ h)


def test_ties_go_to_the_lower_expert_id():
    w = np.zeros((6, 3))
    w[1] = w[4] = [1.0, 0.0, 0.0]                         # experts 1 and 4 tie at the top
    w[2] = w[5] = [0.5, 0.0, 0.0]                         # experts 2 and 5 tie next
    ids, p, _ = orouter.route_token(np.array([2.0, 0.0, 0.0]), w, 3)
    assert ids.tolist() == [1, 4, 2]
    assert p[0] == p[1] > p[2]


def test_shift_invariance_and_normalisation():
    rng = np.random.default_rng(1)
    w = rng.standard_normal((16, 8))
    h = rng.standard_normal((5, 8))
    ids, p, z = orouter.route(h, w, 4)
    ids2, p2, _ = orouter.route(h, w, 4, bias=np.full(16, 123.456))      # a constant added to every logit
    assert np.array_equal(ids, ids2)
    np.testing.assert_allclose(p, p2, rtol=1e-9)
    for t in range(5):
        full = orouter.softmax(z[t])
        assert abs(full.sum() - 1.0) < 1e-12 and (full > 0).all()
        assert p[t].sum() <= 1.0 + 1e-12
        assert np.all(np.diff(p[t]) <= 0)                 # descending


def test_selected_set_is_the_brute_force_maximiser():
    rng = np.random.default_rng(2)
    for trial in range(20):
        E, k = 7, 3
        z = rng.standard_normal(E).round(1)               # coarse values: ties happen
        ids, _, _ = orouter.route_token(z, np.eye(E), k)
        best = max(itertools.combinations(range(E), k), key=lambda s: (sum(z[list(s)]), [-e for e in s]))
        assert sorted(ids.tolist()) == sorted(best), (z, ids, best)


def test_against_library_softmax_and_topk():
    g = torch.Generator().manual_seed(3)
    w = torch.randn(32, 64, generator=g, dtype=torch.float64)
    h = torch.randn(9, 64, generator=g, dtype=torch.float64)
    ids, p, _ = orouter.route(h.numpy(), w.numpy(), 5)
    probs = torch.softmax(h @ w.t(), dim=-1)
    tp, ti = torch.topk(probs, 5, dim=-1)                 # random reals: no ties
    assert np.array_equal(ids, ti.numpy().astype(np.int32))
    np.testing.assert_allclose(p, tp.numpy(), rtol=1e-12)
