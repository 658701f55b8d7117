"""GPU parity of the one-launch tiny-batch layers: Eq. 2 through Sec. 3.4's two grouped GEMMs and the fixed-order
sum, all inside one kernel.  Two forms: the cooperative kernel (all CTAs resident, one device-wide barrier between
the projections) and the cluster kernel (a thread-block cluster per token-expert pair and K range, activations
exchanged through distributed shared memory).

Against the CPU oracle at the benchmark spec's tolerance, and bit for bit against the other decode kernels of the
library (per-pair kernels through the allocation-free entry point, in-CTA-grouping kernels through a multi-wave
cache): the layer output may not depend on which kernel family, slot count or wave partition served the call.
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


@pytest.fixture(scope="module")
def layers(B):
    return {"tiny": (synth.TINY, *helpers.make_layer(synth.TINY, seed=0)),
            "mid": (synth.MID, *helpers.make_layer(synth.MID, seed=5)),
            "olmoe": (synth.OLMOE, *helpers.make_layer(synth.OLMOE, seed=2000))}


def bits(t):
    return t.view(torch.int16).cpu().numpy()


@pytest.mark.parametrize("name,T", [("tiny", 1), ("tiny", 7), ("tiny", 12), ("mid", 1), ("mid", 3), ("mid", 6),
                                    ("olmoe", 1), ("olmoe", 2), ("olmoe", 3)])
def test_one_launch_kernels_match_oracle_and_the_other_decode_kernels(B, layers, name, T):
    s, ora, bank = layers[name]
    hidden, ids, p = helpers.routed_inputs(s, T, seed=900 + T, alpha=0.5)
    y_ref, out_ref = ora.forward(hidden, ids, p)
    h, i, w = hidden.cuda(), ids.cuda(), p.cuda()

    full = B.Cache(s, [bank], s.num_experts, max_tokens=16)
    out = full.forward(0, h, i, w)
    # the cooperative kernel wherever all of its CTAs fit the GPU at once (OLMoE shape: one token), else the per-pair kernels
    assert full.last_path() == (B.PATH_PAIR if name == "olmoe" and T > 1 else B.PATH_COOP)
    helpers.check_output(out, y_ref, out_ref, f"{name} T={T}")
    again = full.forward(0, h, i, w)                     # the arrival counters clean themselves
    assert np.array_equal(bits(out), bits(again))
    # the cluster kernel at every cluster size the shape fits: the exchange through distributed shared memory changes nothing
    try:
        for cs in (1, 2, 4, 8):
            B.exmoe_debug_force_cluster_size(cs)
            forced = full.forward(0, h, i, w)
            if full.last_path() == B.PATH_CLUSTER:
                assert np.array_equal(bits(out), bits(forced)), cs
            else:
                assert name == "olmoe" and cs in (1, 2)  # 540 KB / 270 KB of weights per CTA do not fit
    finally:
        B.exmoe_debug_force_cluster_size(0)
    assert full.status() == 0

    # per-pair gate/up + by-token down kernels (the allocation-free entry point runs them)
    old = torch.empty_like(out)
    B.exmoe_moe_forward_static(s, bank.cuda().reshape(-1), h, i, w, old)
    assert np.array_equal(bits(out), bits(old))

    # several waves: grouping rebuilt inside the GEMM CTAs, fused last-arriver combine
    C = max(s.top_k, 3)
    multi = B.Cache(s, [bank], C, max_tokens=16, wave_cap=max(1, C // 2))
    out_m = multi.forward(0, h, i, w)
    if T * s.top_k > C // 2:
        assert multi.last_path() == B.PATH_SMALL
    assert np.array_equal(bits(out), bits(out_m))
    assert multi.status() == 0
    full.close()
    multi.close()


def test_one_launch_kernels_read_slots_through_the_map(B, layers):
    """C < E, one wave: the kernel finds its weights through slot_of; same bits as the resident run, miss after miss."""
    s, ora, bank = layers["olmoe"]
    full = B.Cache(s, [bank], s.num_experts, max_tokens=4)
    part = B.Cache(s, [bank], 16, max_tokens=4)
    for step in range(6):
        hidden, ids, p = helpers.routed_inputs(s, 1 + step % 2, seed=950 + step, alpha=1.0)
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        B.exmoe_debug_force_cluster_size(4)
        try:
            cl = part.forward(0, h, i, w) if step == 0 else None      # the cluster kernel, through the map, on a cold cache
            assert cl is None or part.last_path() == B.PATH_CLUSTER
        finally:
            B.exmoe_debug_force_cluster_size(0)
        a = full.forward(0, h, i, w)
        b = part.forward(0, h, i, w)
        assert cl is None or np.array_equal(bits(a), bits(cl))
        want = B.PATH_COOP if h.shape[0] == 1 else B.PATH_PAIR
        assert full.last_path() == want and part.last_path() == want
        assert np.array_equal(bits(a), bits(b))
    y_ref, out_ref = ora.forward(hidden, ids, p)
    helpers.check_output(b, y_ref, out_ref, "olmoe C=16")
    assert part.stats(0)["misses"] > 0 and part.status() == 0
    full.close()
    part.close()


@pytest.mark.parametrize("kernel", ["coop", "cluster"])
def test_one_launch_kernels_invalid_ids(B, layers, kernel):
    """An id outside [0, E) adds nothing and is reported; a token with no valid id gets a zero row."""
    s, ora, bank = layers["mid"]
    hidden, ids, p = helpers.routed_inputs(s, 3, seed=977)
    ids = ids.clone()
    ids[0, 1] = s.num_experts            # one bad pair
    ids[2, :] = -1                       # a token without any valid id
    y_ref, out_ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=4)
    want = B.PATH_COOP if kernel == "coop" else B.PATH_CLUSTER
    B.exmoe_debug_force_cluster_size(0 if kernel == "coop" else 2)
    try:
        out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
        assert cache.last_path() == want
        assert cache.status() == B.EXMOE_ERR_BAD_EXPERT_ID
        helpers.check_output(out, y_ref, out_ref, "bad ids")
        assert not out[2].float().abs().any()
        hidden2, ids2, p2 = helpers.routed_inputs(s, 3, seed=978)     # counters and barrier words are clean afterwards
        y2, o2 = ora.forward(hidden2, ids2, p2)
        helpers.check_output(cache.forward(0, hidden2.cuda(), ids2.cuda(), p2.cuda()), y2, o2, "after bad ids")
        assert cache.last_path() == want and cache.status() == 0
    finally:
        B.exmoe_debug_force_cluster_size(0)
    cache.close()


def test_cooperative_kernel_replays_from_a_graph(B, layers):
    s, ora, bank = layers["olmoe"]
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=1)
    sets = [tuple(x.cuda() for x in helpers.routed_inputs(s, 1, seed=990 + n)) for n in range(4)]
    eager = [cache.forward(0, *x).clone() for x in sets]
    outs = [torch.empty_like(eager[0]) for _ in sets]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        cache.forward(0, *sets[0], out=outs[0], stream=stream)
    stream.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for x, o in zip(sets, outs):
            cache.forward(0, *x, out=o, stream=stream)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    for e, o in zip(eager, outs):
        assert np.array_equal(bits(e), bits(o))
    assert cache.status() == 0
    cache.close()
