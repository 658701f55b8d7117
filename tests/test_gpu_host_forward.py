"""exmoe_moe_forward_host: the layer call with host tensors in and out.

It must give the bits of exmoe_moe_forward on the same inputs: for pageable and page-locked tensors, for tiny batches
on their first call (plain launches) and on later ones (replay of the recorded graph), for small results (written
straight into pinned host memory) and large ones, with all experts resident and with a 16-slot cache, where the slot
map and counters must also stay the oracle's.
"""
import numpy as np
import pytest
import torch

from oracle import cache as ocache
from paper_2608_15383_b200 import synth

import helpers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2608_15383_b200 import binding, build
    build.build()
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def olmoe_layer(B):
    return helpers.make_layer(synth.OLMOE, seed=2000)


@pytest.mark.parametrize("C", [64, 16])
def test_host_forward_matches_device_forward(B, olmoe_layer, C):
    ora, bank = olmoe_layer
    s = synth.OLMOE
    full = B.Cache(s, [bank], 64, max_tokens=200)
    host = B.Cache(s, [bank], C, max_tokens=200)
    sc = ocache.SlotCache(64, C, 0, bytes_per_expert=host.bytes_per_expert)
    stream = torch.cuda.Stream()
    order = [1, 16, 1, 3, 16, 64, 1, 200, 64, 3, 200, 16]              # every size comes back
    for step, T in enumerate(order):
        hidden, ids, p = helpers.routed_inputs(s, T, seed=26000 + step, alpha=0.5)
        want = full.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).cpu()
        out = torch.full((T, s.d_model), 7.0, dtype=torch.bfloat16)
        if step % 2:                                                   # page-locked tensors: large calls skip the staging buffer
            hidden, ids, p, out = hidden.pin_memory(), ids.pin_memory(), p.pin_memory(), out.pin_memory()
        got = host.forward_host(0, hidden, ids, p, out=out, stream=stream)
        assert got is out and torch.equal(got.view(torch.int16), want.view(torch.int16)), (step, T)
        if C < 64:
            helpers.compare_plan(host, sc, ids)
        if step in (0, 4):
            y, ref = ora.forward(hidden, ids, p)
            helpers.check_output(got.cuda(), y, ref, f"host forward step {step}")
    assert host.status() == 0
    # the legacy default stream cannot be captured: the call still works, as plain launches
    hidden, ids, p = helpers.routed_inputs(s, 5, seed=26100, alpha=0.0)
    want = full.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).cpu()
    for _ in range(2):
        got = host.forward_host(0, hidden, ids, p)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
        if C < 64:
            helpers.compare_plan(host, sc, ids)
    with pytest.raises(ValueError):
        host.forward_host(0, hidden.cuda(), ids, p)
    with pytest.raises(B.ExmoeError):
        host.forward_host(3, hidden, ids, p)
    full.close(); host.close()


def test_host_forward_follows_a_miss_path_switch(B, olmoe_layer):
    """Recorded graphs belong to one miss path: after a switch the call runs the other path's sequence."""
    _, bank = olmoe_layer
    s = synth.OLMOE
    full = B.Cache(s, [bank], 64, max_tokens=16)
    host = B.Cache(s, [bank], 16, max_tokens=16)
    sc = ocache.SlotCache(64, 16, 0, bytes_per_expert=host.bytes_per_expert)
    stream = torch.cuda.Stream()
    for step in range(9):
        T = 2 if step % 3 else 16                                      # T = 2 replays a graph, T = 16 is plain launches
        if step == 3:
            host.set_miss_path(B.MISS_HOST_COPIES)
        if step == 6:
            host.set_miss_path(B.MISS_DEVICE_FETCH)
        hidden, ids, p = helpers.routed_inputs(s, T, seed=26200 + step, alpha=1.0)
        want = full.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).cpu()
        got = host.forward_host(0, hidden, ids, p, stream=stream)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), step
        helpers.compare_plan(host, sc, ids)
    assert host.status() == 0
    full.close(); host.close()
