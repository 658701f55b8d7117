"""GPU parity of the fused router (Eq. 1) against the oracle router, through the C ABI.

The top-k choice is an integer decided by floating point: the kernel decides in binary32 (its own precision),
the oracle in binary64.  So the comparison is: identical ids wherever the oracle's logits separate the experts
by more than the binary32 rounding of a 2048-term sum; where the kernel's choice differs, the two experts must
be such a near-tie in the oracle (the choice is then valid either way); weights within binary32 rounding.
"""
import numpy as np
import pytest
import torch

from oracle import router as orouter
from paper_2608_15383_b200 import synth

import helpers

pytestmark = pytest.mark.gpu

NEAR_TIE = 2e-5          # logit gap below which binary32 and binary64 may order two experts differently


@pytest.fixture(scope="module")
def B():
    from paper_2608_15383_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def check(shape, hidden, w_router, bias, ids_gpu, w_gpu):
    ids_ref, p_ref, z = orouter.route(hidden.float().numpy(), w_router.float().numpy(), shape.top_k,
                                      None if bias is None else bias.double().numpy())
    ids_gpu, w_gpu = ids_gpu.cpu().numpy(), w_gpu.cpu().numpy()
    assert ids_gpu.dtype == np.int32 and ids_gpu.shape == ids_ref.shape
    n_diff = 0
    for t in range(ids_ref.shape[0]):
        assert len(set(ids_gpu[t].tolist())) == shape.top_k                      # k distinct, valid experts
        assert ((ids_gpu[t] >= 0) & (ids_gpu[t] < shape.num_experts)).all()
        full = orouter.softmax(z[t])
        np.testing.assert_allclose(w_gpu[t], full[ids_gpu[t]], rtol=2e-5, atol=1e-9)   # weights of what it chose
        assert np.all(np.diff(w_gpu[t]) <= 1e-9)                                 # descending
        if np.array_equal(ids_gpu[t], ids_ref[t]):
            continue
        n_diff += 1
        for j in range(shape.top_k):                                             # any difference is a near-tie
            if ids_gpu[t, j] != ids_ref[t, j]:
                assert abs(z[t, ids_gpu[t, j]] - z[t, ids_ref[t, j]]) < NEAR_TIE, (t, j)
    return n_diff


@pytest.mark.parametrize("shape,T,alpha", [(synth.TINY, 16, 0.0), (synth.MID, 33, 1.0), (synth.OLMOE, 1, 0.0),
                                           (synth.OLMOE, 64, 1.0), (synth.OLMOE, 300, 0.5)])
def test_router_matches_oracle(B, shape, T, alpha):
    hidden = synth.hidden_states(shape, T, seed=11 + T)
    w_router = synth.router_weights(shape, seed=5)
    bias = synth.zipf_bias(shape.num_experts, alpha, seed=9) if alpha else None
    ids, w = B.exmoe_route(shape, hidden.cuda(), w_router.cuda(), None if bias is None else bias.cuda())
    torch.cuda.synchronize()
    n_diff = check(shape, hidden, w_router, bias, ids, w)
    assert n_diff <= max(1, T // 50)                      # near-ties are rare with random inputs
    # the harness router (torch, binary32) makes the same choices up to the same near-ties
    ids_t, w_t = helpers.route(hidden.cuda(), w_router.cuda(), shape.top_k, None if bias is None else bias.cuda())
    same = (ids_t == ids).all(dim=1).float().mean().item()
    assert same >= 0.95


def test_router_ties_and_edge_cases(B):
    shape = synth.Shape(d_model=128, d_ff=128, num_experts=8, top_k=3)
    w_router = torch.zeros((8, 128), dtype=torch.bfloat16)
    w_router[2, 0] = w_router[5, 0] = 1.0                 # experts 2 and 5 tie at the top, the rest tie at zero
    hidden = torch.zeros((2, 128), dtype=torch.bfloat16)
    hidden[0, 0] = 3.0
    ids, w = B.exmoe_route(shape, hidden.cuda(), w_router.cuda())
    assert ids[0].tolist() == [2, 5, 0]                   # ties to the lower id
    assert ids[1].tolist() == [0, 1, 2]                   # all logits equal
    np.testing.assert_allclose(w[1].cpu().numpy(), [1 / 8] * 3, rtol=1e-6)
    ids_ref, p_ref, _ = orouter.route(hidden.float().numpy(), w_router.float().numpy(), 3)
    assert np.array_equal(ids.cpu().numpy(), ids_ref)
    np.testing.assert_allclose(w.cpu().numpy(), p_ref, rtol=1e-6)
    # T = 0 is a no-op; bad shapes are refused
    B.exmoe_route(shape, torch.empty((0, 128), dtype=torch.bfloat16, device="cuda"), w_router.cuda())
    with pytest.raises(B.ExmoeError) as ei:
        B.exmoe_route(synth.Shape(d_model=100, d_ff=128, num_experts=8, top_k=3), hidden.cuda(), w_router.cuda())
    assert ei.value.code == B.EXMOE_ERR_SHAPE


def test_router_feeds_the_layer(B):
    """Router output goes straight into exmoe_moe_forward: the layer result equals the one on the harness router's
    ids wherever the two routers agree (they do on these inputs)."""
    import helpers
    shape = synth.MID
    ora, bank = helpers.make_layer(shape, seed=77)
    hidden = synth.hidden_states(shape, 12, seed=3)
    w_router = synth.router_weights(shape, seed=4)
    ids, w = B.exmoe_route(shape, hidden.cuda(), w_router.cuda())
    cache = B.Cache(shape, [bank], shape.num_experts, max_tokens=16)
    out = cache.forward(0, hidden.cuda(), ids, w)
    y, ref = ora.forward(hidden, ids.cpu(), w.cpu())
    helpers.check_output(out, y, ref, "router-fed layer")
    cache.close()
