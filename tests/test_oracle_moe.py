"""Pins for the oracle's layer output (Eq. 2) against restatements and library routines (no GPU)."""
import numpy as np
import pytest
import torch

from oracle import moe, quant
from paper_2608_15383_b200 import synth

import helpers

SHAPE = synth.Shape(d_model=256, d_ff=128, num_experts=8, top_k=2)


@pytest.fixture(scope="module")
def layer():
    wg, wu, wd = synth.expert_weights(SHAPE, seed=0)
    deq = []
    for e in range(SHAPE.num_experts):
        mats = []
        for w in (wg[e], wu[e], wd[e]):
            q, s = quant.quantize_g128(w.float().numpy())
            mats.append(quant.dequantize_g128(q, s))
        deq.append(tuple(mats))
    hidden = synth.hidden_states(SHAPE, 16, seed=1)
    ids, p = helpers.route(hidden, synth.router_weights(SHAPE, seed=2), SHAPE.top_k)
    return deq, hidden.float().numpy(), ids.numpy(), p.numpy()


def run(layer, hidden=None, ids=None, p=None):
    deq, h0, i0, p0 = layer
    hidden = h0 if hidden is None else hidden
    ids = i0 if ids is None else ids
    p = p0 if p is None else p
    return moe.moe_layer_forward(hidden, ids, p, lambda e: deq[e], SHAPE.num_experts)


def test_dense_restatement(layer):
    """Eq. 2 as a dense sum over ALL experts with p~ = 0 off the top-k, batched with einsum."""
    deq, hidden, ids, p = layer
    T, E = hidden.shape[0], SHAPE.num_experts
    ptilde = np.zeros((T, E))
    for t in range(T):
        for j in range(ids.shape[1]):
            ptilde[t, ids[t, j]] += p[t, j]
    Wg = torch.tensor(np.stack([d[0] for d in deq]))
    Wu = torch.tensor(np.stack([d[1] for d in deq]))
    Wd = torch.tensor(np.stack([d[2] for d in deq]))
    x = torch.tensor(hidden, dtype=torch.float64)
    g = torch.einsum("eih,th->tei", Wg, x)
    u = torch.einsum("eih,th->tei", Wu, x)
    a = torch.nn.functional.silu(g) * u
    y = torch.einsum("ehi,tei->teh", Wd, a)
    dense = torch.einsum("te,teh->th", torch.tensor(ptilde), y).numpy()
    got, _ = run(layer)
    assert np.allclose(got, dense, rtol=1e-12, atol=1e-15)
    assert np.abs(got).max() > 1e-4


def test_single_expert_is_a_swiglu_mlp(layer):
    deq, hidden, _, _ = layer
    ids = np.full((hidden.shape[0], 1), 3, dtype=np.int32)
    p = np.ones((hidden.shape[0], 1), dtype=np.float32)
    got, _ = run(layer, ids=ids, p=p)
    x = torch.tensor(hidden, dtype=torch.float64)
    wg, wu, wd = (torch.tensor(m) for m in deq[3])
    ref = (torch.nn.functional.silu(x @ wg.t()) * (x @ wu.t())) @ wd.t()
    assert np.allclose(got, ref.numpy(), rtol=1e-12, atol=1e-15)


def test_gate_and_up_are_not_interchangeable(layer):
    deq, hidden, _, _ = layer
    wg, wu, wd = deq[0]
    a = moe.expert_ffn(hidden[0], wg, wu, wd)
    b = moe.expert_ffn(hidden[0], wu, wg, wd)
    assert np.abs(a - b).max() > 1e-3 * np.abs(a).max()


def test_linear_in_mixture_weights_and_zero_weight(layer):
    _, hidden, ids, p = layer
    y1, _ = run(layer)
    y2, _ = run(layer, p=2.5 * p)
    assert np.allclose(y2, 2.5 * y1, rtol=1e-12)
    p0 = p.copy()
    p0[:, 1] = 0.0
    y0, _ = run(layer, p=p0)
    only0, _ = run(layer, ids=ids[:, :1], p=p[:, :1])
    assert np.allclose(y0, only0, rtol=1e-12, atol=1e-18)
    only1, _ = run(layer, ids=ids[:, 1:], p=p[:, 1:])
    assert np.allclose(only0 + only1, y1, rtol=1e-12, atol=1e-18)      # disjoint contributions add up


def test_token_permutation_and_duplicates(layer):
    _, hidden, ids, p = layer
    perm = np.random.default_rng(0).permutation(hidden.shape[0])
    y, out = run(layer)
    yp, outp = run(layer, hidden=hidden[perm], ids=ids[perm], p=p[perm])
    assert np.array_equal(yp, y[perm]) and np.array_equal(outp, out[perm])
    h2 = np.concatenate([hidden[:1], hidden[:1]])
    yd, _ = run(layer, hidden=h2, ids=np.concatenate([ids[:1], ids[:1]]), p=np.concatenate([p[:1], p[:1]]))
    assert np.array_equal(yd[0], yd[1])


def test_invalid_id_contributes_nothing(layer):
    _, hidden, ids, p = layer
    bad = ids.copy()
    bad[:, 1] = SHAPE.num_experts + 3
    yb, _ = run(layer, ids=bad)
    only0, _ = run(layer, ids=ids[:, :1], p=p[:, :1])
    assert np.array_equal(yb, only0)


def test_output_is_bf16_rounding_of_sum(layer):
    y, out = run(layer)
    lib = torch.tensor(y).to(torch.float32).to(torch.bfloat16).double().numpy()
    # the double rounding of the library path differs at most in rare ties; values must be BF16
    assert np.array_equal(torch.tensor(out).to(torch.bfloat16).double().numpy(), out)
    assert (out != lib).mean() < 1e-3
    assert np.abs(out - y).max() <= np.abs(y).max() * 2.0 ** -8


def test_w4_error_against_unquantised_weights_is_the_quantiser_noise(layer):
    """Sanity on magnitude: W4 vs the BF16 weights differs by roughly the int4 noise level."""
    deq, hidden, ids, p = layer
    wg, wu, wd = synth.expert_weights(SHAPE, seed=0)
    full = lambda e: (wg[e].double().numpy(), wu[e].double().numpy(), wd[e].double().numpy())
    yq, _ = run(layer)
    yf, _ = moe.moe_layer_forward(hidden, ids, p, full, SHAPE.num_experts)
    rel = np.linalg.norm(yq - yf) / np.linalg.norm(yf)
    assert 0.02 < rel < 0.5


def test_rounding_matched_mode_differs_only_by_the_activation_rounding():
    """The second oracle mode rounds phi(g)*u to BF16 before the down projection: its distance to the definition is
    bounded by that rounding (relative 2^-9 per activation), and with an activation that is BF16-exact it is zero."""
    from oracle import moe as omoe
    from oracle.bf16 import round_to_bf16
    rng = np.random.default_rng(11)
    H, I = 16, 8
    wg, wu, wd = rng.standard_normal((I, H)), rng.standard_normal((I, H)), rng.standard_normal((H, I))
    x = round_to_bf16(rng.standard_normal(H))
    plain = omoe.expert_ffn(x, wg, wu, wd)
    matched = omoe.expert_ffn(x, wg, wu, wd, round_activation=True)
    a = omoe.silu(wg @ x) * (wu @ x)
    bound = np.abs(wd) @ (np.abs(a) * 2.0 ** -9)
    assert np.all(np.abs(plain - matched) <= bound + 1e-15) and np.any(plain != matched)
    # gate = 0 rows make a = 0 exactly: both modes agree bit for bit
    assert np.array_equal(omoe.expert_ffn(x, np.zeros((I, H)), wu, wd), omoe.expert_ffn(x, np.zeros((I, H)), wu, wd, True))
