"""Device-initiated miss path (exmoe_cache_set_miss_path, Section 3.4 step 3 without the host in the loop).

What must hold: the slot map, LRU state, waves, miss list and counters are the oracle's bit for bit, every occupied
slot holds the host bank's bytes, and the layer output equals the fully resident output bit for bit (Section 3.4's
last sentence), on every kernel path; and the call, being a fixed launch sequence, replays from a CUDA graph with
misses inside it.
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


@pytest.mark.parametrize("C,Cw", [(16, 0), (16, 8), (24, 10), (8, 0)])
def test_state_slots_and_output_match_oracle_and_resident_run(B, olmoe_layer, C, Cw):
    ora, bank = olmoe_layer
    s = synth.OLMOE
    full = B.Cache(s, [bank], 64, max_tokens=300)
    dev = B.Cache(s, [bank], C, max_tokens=300, wave_cap=Cw)            # device-initiated fetch is the default
    sc = ocache.SlotCache(64, C, Cw, bytes_per_expert=dev.bytes_per_expert)
    waves = set()
    # pairwise (1, 2, 3), grouped small with several waves, streaming (16..56), tensor-core small-N and large-N
    for step, (T, alpha) in enumerate([(1, 0.0), (2, 1.0), (3, 2.0), (1, 0.0), (16, 0.5), (33, 0.0), (16, 2.0), (64, 1.0),
                                       (129, 0.0), (300, 1.0), (1, 1.0), (5, 0.0)]):
        hidden, ids, p = helpers.routed_inputs(s, T, seed=21000 + step, alpha=alpha)
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        a = full.forward(0, h, i, w).clone()
        b = dev.forward(0, h, i, w).clone()
        plan = helpers.compare_plan(dev, sc, ids)
        waves.add(plan.n_waves)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16)), (step, T, alpha)
        if step in (0, 4, 8):
            y, ref = ora.forward(hidden, ids, p)
            helpers.check_output(b, y, ref, f"device fetch step {step}")
    assert len(waves) >= 2
    _, slot_expert, _, _ = dev.state(0)
    for slot in (0, C // 2, C - 1):
        assert np.array_equal(dev.read_slot(0, slot), bank[int(slot_expert[slot])].numpy())
    for c in (full, dev):
        assert c.status() == 0
        c.close()


def test_switching_modes_keeps_one_history(B, olmoe_layer):
    """Host copies, device fetch and host copies again on one cache: the LRU history runs through."""
    _, bank = olmoe_layer
    s = synth.OLMOE
    full = B.Cache(s, [bank], 64, max_tokens=16)
    cache = B.Cache(s, [bank], 16, max_tokens=16)
    sc = ocache.SlotCache(64, 16, 0, bytes_per_expert=cache.bytes_per_expert)
    for step in range(9):
        if step % 3 == 0:
            cache.set_miss_path(B.MISS_DEVICE_FETCH if (step // 3) % 2 else B.MISS_HOST_COPIES)
        hidden, ids, p = helpers.routed_inputs(s, 16 if step % 2 else 1, seed=22000 + step, alpha=0.5)
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        a = full.forward(0, h, i, w).clone()
        b = cache.forward(0, h, i, w).clone()
        helpers.compare_plan(cache, sc, ids)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16)), step
    with pytest.raises(B.ExmoeError):
        cache.set_miss_path(7)
    assert cache.status() == 0
    full.close(); cache.close()


@pytest.mark.parametrize("T", [1, 16])
def test_offloaded_layer_replays_from_a_cuda_graph(B, olmoe_layer, T):
    """C < E inside a CUDA graph: resolution, miss fetch and GEMMs of six calls are captured once; every replay
    starts from the state the previous one left, so the replayed calls keep missing and keep being right."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    cache = B.Cache(s, [bank], 16, max_tokens=16)
    cache.set_miss_path(B.MISS_DEVICE_FETCH)
    full = B.Cache(s, [bank], 64, max_tokens=16)
    inputs = [tuple(x.cuda() for x in helpers.routed_inputs(s, T, seed=23000 + i, alpha=0.5)) for i in range(6)]
    outs = [torch.empty_like(inputs[0][0]) for _ in inputs]
    want = [full.forward(0, *inp).clone() for inp in inputs]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        cache.forward(0, *inputs[0], out=outs[0], stream=stream)            # first call outside capture
    stream.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for (h, i, w), o in zip(inputs, outs):
            cache.forward(0, h, i, w, out=o, stream=stream)
    before = cache.stats(0)
    for rep in range(2):
        for o in outs:
            o.zero_()
        with torch.cuda.stream(stream):
            g.replay()
        stream.synchronize()
        for o, ref in zip(outs, want):
            assert torch.equal(o.view(torch.int16), ref.view(torch.int16)), rep
    after = cache.stats(0)
    assert after["forwards"] == before["forwards"] + 12 and after["misses"] > before["misses"]
    h, i, w = inputs[3]
    y, ref = ora.forward(h.cpu(), i.cpu(), w.cpu())
    helpers.check_output(outs[3], y, ref, "graph, offloaded")
    assert cache.status() == 0
    cache.close(); full.close()


def check_state(cache, sc, layer=0):
    es, se, stamp, tick = cache.state(layer)
    assert np.array_equal(es, sc.expert_slot) and np.array_equal(se, sc.slot_expert)
    assert np.array_equal(stamp, sc.slot_stamp) and tick == sc.tick
    st = cache.stats(layer)
    assert st == {"lookups": sc.stats.lookups, "hits": sc.stats.hits, "misses": sc.stats.misses,
                  "waves": sc.stats.waves, "h2d_bytes": sc.stats.h2d_bytes, "forwards": sc.stats.forwards}


def test_prefetch_is_a_layer_call_without_tokens(B, olmoe_layer):
    """exmoe_cache_prefetch advances slot map, LRU stamps and counters exactly as the oracle's resolution of the same
    ids (Section 3.3 / 3.4 steps 1-3), leaves the slots holding the bank's bytes, and a forward that selects the
    prefetched experts then misses nothing and still equals the resident run bit for bit."""
    _, bank = olmoe_layer
    s = synth.OLMOE
    cache = B.Cache(s, [bank], 16, max_tokens=16)
    full = B.Cache(s, [bank], 64, max_tokens=16)
    sc = ocache.SlotCache(64, 16, 0, bytes_per_expert=cache.bytes_per_expert)
    rng = np.random.default_rng(5)
    for step in range(8):
        T = (1, 2, 16, 1)[step % 4]
        hidden, ids, p = helpers.routed_inputs(s, T, seed=24000 + step, alpha=0.5)
        if step % 2 == 0:
            guess = ids.reshape(-1).clone()                       # a perfect guess (repeats and all)
        else:
            guess = torch.from_numpy(rng.integers(0, 64, size=11).astype(np.int32))   # an unrelated one
        cache.prefetch(0, guess.cuda())
        sc.resolve(guess.numpy())
        check_state(cache, sc)
        before = cache.stats(0)["misses"]
        a = full.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).clone()
        b = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).clone()
        helpers.compare_plan(cache, sc, ids)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16)), step
        if step % 2 == 0 and len(set(guess.tolist())) <= 16:
            assert cache.stats(0)["misses"] == before             # everything selected was already there
    _, slot_expert, _, _ = cache.state(0)
    for slot in (0, 9, 15):
        assert np.array_equal(cache.read_slot(0, slot), bank[int(slot_expert[slot])].numpy())
    cache.prefetch(0, torch.tensor([3, 99, -1], dtype=torch.int32).cuda())            # invalid ids are ignored, and reported
    assert cache.status() == B.EXMOE_ERR_BAD_EXPERT_ID
    cache.set_miss_path(B.MISS_HOST_COPIES)
    with pytest.raises(B.ExmoeError) as ei:
        cache.prefetch(0, torch.tensor([1], dtype=torch.int32).cuda())
    assert ei.value.code == B.EXMOE_ERR_STATE
    full.prefetch(0, torch.tensor([1], dtype=torch.int32).cuda())                     # C = E: no-op
    cache.close(); full.close()


def test_prefetch_of_the_next_layer_overlaps_a_forward(B):
    """Two layers, two streams: while layer 0 computes on the main stream, layer 1's experts are prefetched on a side
    stream (own resolution buffers); layer 1's forward, ordered after the prefetch by an event, finds them resident."""
    s = synth.MID
    layers = [helpers.make_layer(s, seed=70 + l) for l in range(2)]
    cache = B.Cache(s, [b for _, b in layers], 6, max_tokens=32)
    full = B.Cache(s, [b for _, b in layers], s.num_experts, max_tokens=32)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    for step in range(6):
        ins = [tuple(x.cuda() for x in helpers.routed_inputs(s, 20, seed=25000 + 10 * step + l, alpha=0.5)) for l in range(2)]
        want = [full.forward(l, *ins[l]).clone() for l in range(2)]
        torch.cuda.synchronize()
        guess = ins[1][1].reshape(-1)[:6].contiguous()            # six of layer 1's ids: they fit the six slots
        done = torch.cuda.Event()
        with torch.cuda.stream(side):
            cache.prefetch(1, guess, stream=side)
            done.record(side)
        with torch.cuda.stream(main):
            out0 = cache.forward(0, *ins[0], stream=main).clone()
            main.wait_event(done)
            out1 = cache.forward(1, *ins[1], stream=main).clone()
        torch.cuda.synchronize()
        assert torch.equal(out0.view(torch.int16), want[0].view(torch.int16)), step
        assert torch.equal(out1.view(torch.int16), want[1].view(torch.int16)), step
    assert cache.status() == 0
    cache.close(); full.close()


def test_miss_fetch_overlaps_the_resident_groups_kernels(B, olmoe_layer):
    """Config 3's path (16 tokens, 16 slots): the wave's fetch kernel runs on the side stream while the GEMM kernels run
    over the groups whose experts were resident.  Device timestamps show fetch time inside GEMM intervals; the output
    stays bit-identical to the resident run and the plan, state and counters to the oracle."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    full = B.Cache(s, [bank], 64, max_tokens=16)
    part = B.Cache(s, [bank], 16, max_tokens=16)
    sc = ocache.SlotCache(64, 16, 0, bytes_per_expert=part.bytes_per_expert)
    part.profile_enable(True)
    for step in range(8):
        hidden, ids, p = helpers.routed_inputs(s, 16, seed=8800 + step, alpha=2.0)     # strong skew: many hits per step
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        a = full.forward(0, h, i, w)
        b = part.forward(0, h, i, w)
        assert part.last_path() == B.PATH_STREAM
        helpers.compare_plan(part, sc, ids)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16)), step
    fetch_ms, both_ms = part.profile_overlap()
    part.profile_enable(False)
    st = part.stats(0)
    assert st["hits"] > 0 and st["misses"] > 0
    assert fetch_ms > 0 and 0 < both_ms <= fetch_ms
    assert part.status() == 0 and full.status() == 0
    full.close()
    part.close()
