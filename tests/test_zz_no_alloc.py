"""exmoe_moe_forward_static: the allocation-free tiny-batch forward, checked against exmoe_moe_forward.

The entry point serves callers that cannot allocate device memory when they need the layer (a serving loop
whose memory was handed to a pool at start-up, a plug-in under a framework that owns the allocator, code that
must avoid the device-wide synchronisation of cudaMalloc/cudaFree): its scratch is a fixed `__device__` array
inside the library.  Up to 24 token-expert pairs it runs the same kernels as the cache-based entry point, so the
outputs must agree bit for bit; above that the cache-based entry point takes its streaming kernels and the two
agree within the oracle-derived tolerance used everywhere else, which the test holds both to in every case.  Two calls in a row check that the
contents the shared scratch keeps from the first call do not leak into the second.
Collected last (file name) so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2608_15383_b200 import synth

import helpers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2608_15383_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def close(a, b):
    a = a.float().cpu().numpy().astype(np.float64)
    b = b.float().cpu().numpy().astype(np.float64)
    err = a - b
    assert np.abs(err).max() <= helpers.MAX_ERR_FRAC * max(np.abs(b).max(), 1e-30)
    assert np.linalg.norm(err) <= helpers.REL_FRO * max(np.linalg.norm(b), 1e-30)


@pytest.mark.parametrize("shape,T", [(synth.TINY, 3), (synth.OLMOE, 1), (synth.OLMOE, 3), (synth.OLMOE, 4)])
def test_static_forward_matches_cache_forward_twice(B, shape, T):
    ora, bank = helpers.make_layer(shape, seed=4242)
    experts = bank.cuda()                                  # fully resident layer: expert e at e * bytes_per_expert
    cache = B.Cache(shape, [bank], shape.num_experts, max_tokens=8)
    out = torch.empty((T, shape.d_model), dtype=torch.bfloat16, device="cuda")
    for call in range(2):                                  # second call reuses the scratch the first one dirtied
        hidden, ids, p = helpers.routed_inputs(shape, T, seed=7000 + 10 * T + call)
        if call == 1:
            ids[0, 0] = shape.num_experts + 5              # an invalid id contributes nothing in both entry points
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        ref = cache.forward(0, h, i, w).clone()
        out.fill_(7.0)
        got = B.exmoe_moe_forward_static(shape, experts, h, i, w, out)
        torch.cuda.synchronize()
        close(got, ref)
        if T * shape.top_k <= 24:                          # same kernels, same order: same bits
            assert torch.equal(got.view(torch.int16), ref.view(torch.int16))
        if shape is synth.TINY or call == 0:
            y, o = ora.forward(hidden, ids, p)
            helpers.check_output(got, y, o, f"static T={T} call={call}")
    cache.status()
    cache.close()


def test_static_forward_rejects_oversize_and_bad_arguments(B):
    shape = synth.TINY
    _, bank = helpers.make_layer(shape, seed=1)
    experts = bank.cuda()
    T = 17                                                 # 17 * top_k(2) = 34 pairs > 32
    hidden, ids, p = helpers.routed_inputs(shape, T, seed=3)
    out = torch.empty((T, shape.d_model), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.ExmoeError) as ei:
        B.exmoe_moe_forward_static(shape, experts, hidden.cuda(), ids.cuda(), p.cuda(), out)
    assert ei.value.code == B.EXMOE_ERR_SHAPE
    wide = synth.Shape(d_model=256, d_ff=4096 + 128, num_experts=2, top_k=1)     # d_ff beyond the scratch
    with pytest.raises(B.ExmoeError) as ei:
        B.exmoe_moe_forward_static(wide, experts, hidden[:1].cuda(), ids[:1, :1].contiguous().cuda(),
                                   p[:1, :1].contiguous().cuda(), out[:1])
    assert ei.value.code == B.EXMOE_ERR_SHAPE
    empty = torch.empty((0, shape.d_model), dtype=torch.bfloat16, device="cuda")
    B.exmoe_moe_forward_static(shape, experts, empty, torch.empty((0, 2), dtype=torch.int32, device="cuda"),
                               torch.empty((0, 2), dtype=torch.float32, device="cuda"), empty)   # T = 0: no-op
