"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle on the same seeded inputs.

Bit-exact: packed bytes, slot maps, waves, miss lists, counters, token grouping, slot contents.
Toleranced (spec bound): BF16 layer output, max|err| <= 2e-2*max|ref| and rel. Frobenius <= 5e-3.
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
def tiny_layer(B):
    return helpers.make_layer(synth.TINY, seed=0)


@pytest.fixture(scope="module")
def mid_layer(B):
    return helpers.make_layer(synth.MID, seed=5)


@pytest.fixture(scope="module")
def olmoe_layer(B):
    return helpers.make_layer(synth.OLMOE, seed=2000)


# ------------------------------------------------------------------------------------ a0: pack
def test_pack_bytes_tiny_all_experts(B, tiny_layer):
    ora, bank = tiny_layer
    assert B.exmoe_packed_bytes(synth.TINY) == 50688 == bank.shape[1]
    for e in range(synth.TINY.num_experts):
        assert np.array_equal(bank[e].numpy(), ora.packed(e)), e


def test_pack_bytes_olmoe_shape(B, olmoe_layer):
    ora, bank = olmoe_layer
    assert B.exmoe_packed_bytes(synth.OLMOE) == 3244032
    for e in (0, 37):
        assert np.array_equal(bank[e].numpy(), ora.packed(e)), e


def test_pack_special_groups_and_errors(B):
    s = synth.Shape(d_model=256, d_ff=128, num_experts=1, top_k=1)
    wg, wu, wd = synth.expert_weights(s, seed=3)
    wg[0, 3, 128:] = 0                               # zero group
    wg[0, 5, :128] = 0
    wg[0, 5, 17] = 0.0123                            # one-nonzero group
    wu[0, 2, :128] = 2.0 ** -30                      # FP16-underflowing scale
    wd[0, 0, :128] = 0
    wd[0, 0, :8] = torch.tensor([1.5, 0.5, -0.5, 2.5, -2.5, 3.5, 7, -7]) * 2.0 ** -6   # s = 2^-6: exact ties
    ora = helpers.OracleLayer(s, wg, wu, wd)
    got = B.exmoe_pack(s, wg[0].cuda(), wu[0].cuda(), wd[0].cuda()).cpu().numpy()
    assert np.array_equal(got, ora.packed(0))
    bad = wg[0].clone()
    bad[1, 1] = float("nan")
    with pytest.raises(B.ExmoeError) as ei:
        B.exmoe_pack(s, bad.cuda(), wu[0].cuda(), wd[0].cuda())
    assert ei.value.code == B.EXMOE_ERR_NONFINITE
    bad = wg[0].clone()
    bad[1, 1] = 3e38                                 # absmax/7 overflows FP16
    with pytest.raises(B.ExmoeError) as ei:
        B.exmoe_pack(s, bad.cuda(), wu[0].cuda(), wd[0].cuda())
    assert ei.value.code == B.EXMOE_ERR_NONFINITE
    with pytest.raises(B.ExmoeError) as ei:
        B.exmoe_packed_bytes(synth.Shape(d_model=200, d_ff=128, num_experts=4, top_k=2))
    assert ei.value.code == B.EXMOE_ERR_SHAPE


# ------------------------------------------------------------------------------------ a1/a2: plan
compare_plan = helpers.compare_plan


@pytest.mark.parametrize("miss_path", ["device", "host"])
@pytest.mark.parametrize("C,Cw,T,alpha", [(8, 0, 16, 0.0), (2, 0, 5, 0.0), (4, 2, 16, 1.0), (3, 0, 1, 0.0), (5, 3, 40, 0.5)])
def test_plan_bit_exact_tiny(B, tiny_layer, C, Cw, T, alpha, miss_path):
    ora, bank = tiny_layer
    s = synth.TINY
    cache = B.Cache(s, [bank], C, max_tokens=64, wave_cap=Cw)
    cache.set_miss_path(B.MISS_DEVICE_FETCH if miss_path == "device" else B.MISS_HOST_COPIES)
    sc = ocache.SlotCache(s.num_experts, C, Cw, bytes_per_expert=cache.bytes_per_expert)
    for step in range(12):
        hidden, ids, p = helpers.routed_inputs(s, T, seed=100 + step, alpha=alpha)
        cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
        compare_plan(cache, sc, ids)
    assert cache.status() == 0
    cache.close()


@pytest.mark.parametrize("C,Cw,T,alpha", [(16, 0, 16, 1.0), (16, 8, 16, 0.5), (32, 0, 4, 1.0), (8, 0, 1, 0.0),
                                          (64, 0, 16, 1.0), (16, 0, 200, 0.0), (64, 0, 300, 1.0)])
def test_plan_bit_exact_olmoe(B, olmoe_layer, C, Cw, T, alpha):
    """Resolution, LRU, waves and grouping on OLMoE geometry, incl. the multi-CTA grouping path (T*k > 1024);
    host-issued miss copies here, the device-initiated path (the default) has the same test in its own file."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    cache = B.Cache(s, [bank], C, max_tokens=max(T, 16), wave_cap=Cw)
    cache.set_miss_path(B.MISS_HOST_COPIES)
    sc = ocache.SlotCache(s.num_experts, C, Cw, bytes_per_expert=cache.bytes_per_expert)
    for step in range(4 if T > 64 else 10):
        hidden, ids, p = helpers.routed_inputs(s, T, seed=300 + step, alpha=alpha)
        cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
        compare_plan(cache, sc, ids)
    cache.close()


@pytest.mark.parametrize("miss_path", ["device", "host"])
def test_slot_bytes_after_miss_copies(B, olmoe_layer, miss_path):
    """After misses, every occupied slot holds exactly the host bank's bytes of its expert (Section 3.3)."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    cache = B.Cache(s, [bank], 16, max_tokens=16)
    cache.set_miss_path(B.MISS_DEVICE_FETCH if miss_path == "device" else B.MISS_HOST_COPIES)
    for step in range(3):
        hidden, ids, p = helpers.routed_inputs(s, 16, seed=400 + step, alpha=0.5)
        cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    _, slot_expert, _, _ = cache.state(0)
    assert (slot_expert >= 0).all()
    for slot in (0, 7, 15):
        assert np.array_equal(cache.read_slot(0, slot), bank[int(slot_expert[slot])].numpy())
    cache.close()


# ------------------------------------------------------------------------------------ a4-a6: output
def test_config1_tiny_output(B, tiny_layer):
    """Config 1: d_model 256, d_ff 128, 8 experts, top-2, 16 tokens, all resident, seed 0."""
    ora, bank = tiny_layer
    s = synth.TINY
    hidden, ids, p = helpers.routed_inputs(s, 16, seed=0)
    y, ref = ora.forward(hidden, ids, p)
    outs = {}
    for C, Cw in [(8, 0), (2, 0), (4, 2), (5, 3)]:
        cache = B.Cache(s, [bank], C, max_tokens=16, wave_cap=Cw)
        out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
        helpers.check_output(out, y, ref, f"C={C}")
        outs[(C, Cw)] = out.cpu()
        assert cache.status() == 0
        cache.close()
    base = outs[(8, 0)]
    for key, o in outs.items():                      # independent of slot count and wave partition, bit for bit
        assert torch.equal(o.view(torch.int16), base.view(torch.int16)), key


@pytest.mark.parametrize("T", [1, 3, 8, 9, 33, 100])
def test_mid_shape_ragged_groups(B, mid_layer, T):
    ora, bank = mid_layer
    s = synth.MID
    hidden, ids, p = helpers.routed_inputs(s, T, seed=50 + T, alpha=1.0)
    y, ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=128)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    helpers.check_output(out, y, ref, f"T={T}")
    cache2 = B.Cache(s, [bank], 6, max_tokens=128, wave_cap=3)
    out2 = cache2.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
    cache.close()
    cache2.close()


@pytest.mark.parametrize("T", [1, 7, 16, 30, 90, 250, 400])
def test_odd_block_counts(B, T):
    """d_model = 3 * 128 and d_ff = 5 * 128: block counts that are not powers of two take the generic kernel
    bodies (no K split, one block per step) on every path; 3 experts per token, ragged groups.  On the tensor-core
    path (T = 250: 64-row tiles, T = 400: 256-row tiles) 6 and 10 ring stages per tile are no multiple of the ring
    depth, so the MMA issue loop is the plain one, not the unrolled one."""
    s = synth.Shape(d_model=384, d_ff=640, num_experts=8, top_k=3)
    if not hasattr(test_odd_block_counts, "layer"):
        test_odd_block_counts.layer = helpers.make_layer(s, seed=123)
    ora, bank = test_odd_block_counts.layer
    hidden, ids, p = helpers.routed_inputs(s, T, seed=4100 + T, alpha=1.0)
    y, ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=400)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    helpers.check_output(out, y, ref, f"T={T}")
    if T >= 250:
        assert cache.last_path() == (B.PATH_TENSOR_SMALL_N if T == 250 else B.PATH_TENSOR)
    cache2 = B.Cache(s, [bank], 4, max_tokens=400, wave_cap=3)          # several waves, misses
    sc = ocache.SlotCache(s.num_experts, 4, 3, bytes_per_expert=cache2.bytes_per_expert)
    out2 = cache2.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    compare_plan(cache2, sc, ids)
    helpers.check_output(out2, y, ref, f"T={T} offloaded")
    assert cache.status() == 0 and cache2.status() == 0
    cache.close()
    cache2.close()


@pytest.mark.parametrize("T", [7, 100, 300])
def test_many_experts_small_dims(B, T):
    """256 experts of 128 x 128: more active groups than the streaming kernel's scan keeps in registers, one tile per
    group, several groups per CTA; fully resident and with 64 slots (several waves)."""
    s = synth.Shape(d_model=128, d_ff=128, num_experts=256, top_k=4)
    if not hasattr(test_many_experts_small_dims, "layer"):
        test_many_experts_small_dims.layer = helpers.make_layer(s, seed=321)
    ora, bank = test_many_experts_small_dims.layer
    hidden, ids, p = helpers.routed_inputs(s, T, seed=5200 + T, alpha=0.3)
    y, ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=300)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    helpers.check_output(out, y, ref, f"T={T}")
    cache2 = B.Cache(s, [bank], 64, max_tokens=300, wave_cap=48)
    sc = ocache.SlotCache(s.num_experts, 64, 48, bytes_per_expert=cache2.bytes_per_expert)
    out2 = cache2.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    compare_plan(cache2, sc, ids)
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
    assert cache.status() == 0 and cache2.status() == 0
    cache.close()
    cache2.close()


def test_config2_decode_olmoe(B, olmoe_layer):
    """Config 2: OLMoE shape, 1 token per step, 64 slots, fresh hidden state per step."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    cache = B.Cache(s, [bank], 64, max_tokens=16)
    for step in range(4):
        hidden, ids, p = helpers.routed_inputs(s, 1, seed=2000 + step)
        y, ref = ora.forward(hidden, ids, p)
        out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
        helpers.check_output(out, y, ref, f"step {step}")
    st = cache.stats(0)
    assert all(v == 0 for v in st.values())          # full residency bypasses the accounting
    cache.close()


def test_config3_offload_matches_resident(B, olmoe_layer):
    """Config 3: 16 slots over the 64-expert host bank, 16 tokens per step, Zipf-biased routing:
    1-4 waves with LRU misses; output equals the 64-slot run bit for bit and the oracle within tolerance."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    full = B.Cache(s, [bank], 64, max_tokens=16)
    small = B.Cache(s, [bank], 16, max_tokens=16)
    half = B.Cache(s, [bank], 16, max_tokens=16, wave_cap=8)
    half.set_miss_path(B.MISS_HOST_COPIES)               # `small` takes the default, the device-initiated miss path
    sc = ocache.SlotCache(64, 16, 0, bytes_per_expert=small.bytes_per_expert)
    waves = set()
    for step, alpha in enumerate([2.0, 1.0, 0.5, 0.0, 2.0, 0.0]):
        hidden, ids, p = helpers.routed_inputs(s, 16, seed=3000 + step, alpha=alpha)
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        o_full = full.forward(0, h, i, w)
        o_small = small.forward(0, h, i, w)
        o_half = half.forward(0, h, i, w)
        plan = compare_plan(small, sc, ids)
        waves.add(plan.n_waves)
        assert torch.equal(o_small.view(torch.int16), o_full.view(torch.int16)), step
        assert torch.equal(o_half.view(torch.int16), o_full.view(torch.int16)), step
        if step in (1, 3):
            y, ref = ora.forward(hidden, ids, p)
            helpers.check_output(o_small, y, ref, f"step {step}")
    assert len(waves) >= 3 and max(waves) == 4
    for c in (full, small, half):
        assert c.status() == 0
        c.close()


@pytest.mark.parametrize("M", [1, 2, 3, 4, 7, 8, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128])
def test_group_size_sweep_single_expert(B, M):
    """Kernel check in the paper's style (Section 5.3): token-group sizes 1..128 on one expert of OLMoE's
    gate/up and down shapes, against the dequantised reference."""
    s = synth.Shape(d_model=2048, d_ff=1024, num_experts=2, top_k=1)
    if not hasattr(test_group_size_sweep_single_expert, "layer"):
        test_group_size_sweep_single_expert.layer = helpers.make_layer(s, seed=77)
    ora, bank = test_group_size_sweep_single_expert.layer
    hidden = synth.hidden_states(s, M, seed=900 + M)
    ids = torch.ones((M, 1), dtype=torch.int32)
    p = torch.rand((M, 1), generator=torch.Generator().manual_seed(M)) + 0.5
    y, ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], 2, max_tokens=128)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    helpers.check_output(out, y, ref, f"M={M}")
    cache.close()


# ------------------------------------------------------------------------------------ tensor-core path
@pytest.mark.parametrize("T,alpha", [(170, 0.0), (200, 1.0), (513, 0.5)])
def test_prefill_path_mid_shape(B, mid_layer, T, alpha):
    """T*k > 640 routes through the tcgen05/TMEM kernels: ragged groups, several n-tiles, all tokens checked."""
    ora, bank = mid_layer
    s = synth.MID
    hidden, ids, p = helpers.routed_inputs(s, T, seed=600 + T, alpha=alpha)
    y, ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=600)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    helpers.check_output(out, y, ref, f"T={T}")
    assert cache.status() == 0
    cache2 = B.Cache(s, [bank], 6, max_tokens=600, wave_cap=3)       # multi-wave with misses, same kernels
    sc = ocache.SlotCache(s.num_experts, 6, 3, bytes_per_expert=cache2.bytes_per_expert)
    out2 = cache2.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    compare_plan(cache2, sc, ids)
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
    assert cache2.status() == 0
    cache.close()
    cache2.close()


@pytest.mark.parametrize("alpha", [0.0, 1.0])
def test_config4_prefill_olmoe_sampled(B, olmoe_layer, alpha):
    """Config 4: 2048 tokens x top-8 = 16384 rows over 64 experts (uniform and Zipf-skewed), 64 slots.
    The plan is compared in full; the output on sampled tokens the oracle computes one by one."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    T = 2048
    hidden, ids, p = helpers.routed_inputs(s, T, seed=4000, alpha=alpha)
    cache = B.Cache(s, [bank], 64, max_tokens=T)
    sc = ocache.SlotCache(64, 64, 0, bytes_per_expert=cache.bytes_per_expert)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    plan = compare_plan(cache, sc, ids)
    rows = np.bincount(ids.numpy().reshape(-1), minlength=64)
    assert rows.sum() == 16384 and (rows.max() > 1500 if alpha else rows.max() < 400)
    sample = [0, 1, 777, 1023, 1024, 2047] + list(range(300, 306))
    y, ref = ora.forward(hidden[sample], ids[sample], p[sample])
    helpers.check_output(out[sample], y, ref, f"alpha={alpha}")
    assert cache.status() == 0
    again = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())      # deterministic
    assert torch.equal(again.view(torch.int16), out.view(torch.int16))
    cache.close()


def test_config5_stack_teacher_forced(B):
    """Config 5 in small: a 4-layer stack with per-layer routers and the identity-plus-noise residual, slots < experts.
    The stack runs free on the GPU; every layer is then checked on its own (the oracle gets the GPU's layer input
    and routing), because near-ties in the router would let two free-running stacks pick different experts."""
    s = synth.MID
    L = 4
    layers = [helpers.make_layer(s, seed=900 + l) for l in range(L)]
    cache = B.Cache(s, [bank for _, bank in layers], 6, max_tokens=16)
    models = [ocache.SlotCache(s.num_experts, 6, 0, bytes_per_expert=cache.bytes_per_expert) for _ in range(L)]
    stack = synth.SyntheticStack(s, L, seed=31, alpha=1.0, device="cuda")
    h = synth.hidden_states(s, 5, seed=3).cuda()
    for step in range(3):
        rec = []
        h = stack.step(lambda l, x, ids, w: cache.forward(l, x, ids, w).clone(), h,
                       lambda l, x: helpers.route(x, stack.routers[l], s.top_k, stack.bias[l]), record=rec)
        for (l, x, ids, w, out) in rec:
            y, ref = layers[l][0].forward(x.cpu(), ids.cpu(), w.cpu())
            helpers.check_output(out, y, ref, f"step {step} layer {l}")
            models[l].resolve(ids.cpu().numpy())
    for l in range(L):
        st = cache.stats(l)
        assert (st["hits"], st["misses"], st["waves"]) == (models[l].stats.hits, models[l].stats.misses, models[l].stats.waves)
        assert st["h2d_bytes"] == st["misses"] * cache.bytes_per_expert
    assert cache.status() == 0
    cache.close()


# ------------------------------------------------------------------------------------ edge cases
def test_edge_cases(B, tiny_layer):
    ora, bank = tiny_layer
    s = synth.TINY
    cache = B.Cache(s, [bank], 4, max_tokens=16)
    # T = 0 is a no-op
    empty = torch.empty((0, s.d_model), dtype=torch.bfloat16, device="cuda")
    cache.forward(0, empty, torch.empty((0, 2), dtype=torch.int32, device="cuda"),
                  torch.empty((0, 2), dtype=torch.float32, device="cuda"))
    # invalid ids contribute nothing and raise the sticky status
    hidden, ids, p = helpers.routed_inputs(s, 6, seed=9)
    bad = ids.clone()
    bad[2, 1] = 99
    bad[4, 0] = -1
    y, ref = ora.forward(hidden, bad, p)
    out = cache.forward(0, hidden.cuda(), bad.cuda(), p.cuda())
    helpers.check_output(out, y, ref, "bad ids")
    assert cache.status() == B.EXMOE_ERR_BAD_EXPERT_ID
    assert cache.status() == 0                       # cleared by the read
    # too many tokens, bad layer
    big = synth.hidden_states(s, 17, seed=1).cuda()
    with pytest.raises(B.ExmoeError):
        cache.forward(0, big, torch.zeros((17, 2), dtype=torch.int32, device="cuda"),
                      torch.zeros((17, 2), dtype=torch.float32, device="cuda"))
    with pytest.raises(B.ExmoeError):
        cache.forward(3, hidden.cuda(), ids.cuda(), p.cuda())
    # same input twice -> identical bits; zero weights -> zero output
    o1 = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).clone()
    o2 = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    oz = cache.forward(0, hidden.cuda(), ids.cuda(), torch.zeros_like(p).cuda())
    assert not oz.float().abs().max().item()
    cache.close()


def test_bounded_wait_expires_and_reports(B, tiny_layer):
    """Failure detection without a fault: a wait that can never succeed runs out of its (short) budget, the kernel
    returns, the sticky status says EXMOE_ERR_TIMEOUT and the context keeps working."""
    ora, bank = tiny_layer
    s = synth.TINY
    cache = B.Cache(s, [bank], 8, max_tokens=16)
    assert cache.status() == 0
    assert cache.wait_timeout_selftest(budget_cycles=2_000_000) == 3          # ~1 ms at 1.9 GHz
    assert cache.status() == B.EXMOE_ERR_TIMEOUT
    assert cache.status() == 0
    hidden, ids, p = helpers.routed_inputs(s, 4, seed=12)
    y, ref = ora.forward(hidden, ids, p)
    helpers.check_output(cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda()), y, ref, "after timeout")
    cache.close()


@pytest.mark.parametrize("T", [1, 8])
def test_graph_replay_matches_oracle(B, olmoe_layer, T):
    """The launch configuration bench.py times: fully resident decode steps captured in a CUDA graph and replayed
    (T = 1: pairwise kernels; T = 8: grouping + streaming kernels + combine, chained by programmatic dependent
    launches inside the graph)."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    cache = B.Cache(s, [bank], 64, max_tokens=8)
    inputs = [tuple(x.cuda() for x in helpers.routed_inputs(s, T, seed=8100 + i, alpha=1.0)) for i in range(6)]
    outs = [torch.empty_like(inputs[0][0]) for _ in inputs]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        cache.forward(0, *inputs[0], out=outs[0], stream=stream)            # first call outside capture
    stream.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for (h, i, w), o in zip(inputs, outs):
            cache.forward(0, h, i, w, out=o, stream=stream)
    for o in outs:
        o.zero_()
    with torch.cuda.stream(stream):
        g.replay()
    stream.synchronize()
    for idx in (0, 3, 5):
        h, i, w = inputs[idx]
        y, ref = ora.forward(h.cpu(), i.cpu(), w.cpu())
        helpers.check_output(outs[idx], y, ref, f"graph step {idx}")
    cache.close()


@pytest.mark.parametrize("T", [1, 3, 8, 33, 100])
def test_rounding_matched_oracle_mode_is_nearly_bit_exact(B, mid_layer, T):
    """Against the oracle's second mode (SwiGLU output rounded to BF16 before the down projection, the one rounding
    the BF16 activation buffer forces) the register-dequantisation paths (T*k <= 640: codes and activations enter the
    MMA exactly, scales are applied in binary32) agree almost bit for bit: what is left is binary32 summation order
    meeting a BF16 rounding boundary."""
    ora, bank = mid_layer
    s = synth.MID
    hidden, ids, p = helpers.routed_inputs(s, T, seed=700 + T, alpha=0.5)
    _, ref = ora.forward(hidden, ids, p, round_activation=True)
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=128)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).float().cpu().numpy().astype(np.float64)
    err = out - ref
    assert np.linalg.norm(err) <= 1e-3 * np.linalg.norm(ref)
    assert np.mean(err == 0) >= 0.90
    cache.close()


def test_random_sizes_are_invariant_to_slots_and_waves(B, olmoe_layer):
    """Section 3.4, last sentence, over every kernel path: for random batch sizes and routing skews the output of a
    16-slot cache and of a 24-slot cache with 10-expert waves equals the fully resident output bit for bit, and a
    repeated call reproduces it."""
    _, bank = olmoe_layer
    s = synth.OLMOE
    full = B.Cache(s, [bank], 64, max_tokens=300)
    part = B.Cache(s, [bank], 16, max_tokens=300)
    half = B.Cache(s, [bank], 24, max_tokens=300, wave_cap=10)
    part.set_miss_path(B.MISS_HOST_COPIES)               # one cache per miss path (`half`: device-initiated, the default)
    rng = np.random.default_rng(7)
    sizes = [1, 2, 3, 4, 5, 8, 16, 33, 56, 57, 64, 128, 129, 300]
    for it in range(24):
        T = int(sizes[it % len(sizes)])
        alpha = float(rng.choice([0.0, 0.5, 1.0, 2.0]))
        hidden, ids, p = helpers.routed_inputs(s, T, seed=12000 + it, alpha=alpha)
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        a = full.forward(0, h, i, w).clone()
        b = part.forward(0, h, i, w).clone()
        c = half.forward(0, h, i, w).clone()
        a2 = full.forward(0, h, i, w).clone()
        assert bool(torch.isfinite(a.float()).all()), (T, alpha)
        for other, what in ((b, "16 slots"), (c, "24 slots, waves of 10"), (a2, "repeat")):
            assert torch.equal(a.view(torch.int16), other.view(torch.int16)), (T, alpha, what)
    for c_ in (full, part, half):
        assert c_.status() == 0
        c_.close()


def test_create_rejects_bad_arguments(B, tiny_layer):
    ora, bank = tiny_layer
    s = synth.TINY
    with pytest.raises(B.ExmoeError) as ei:
        B.Cache(s, [bank], 1, max_tokens=4)           # C < k
    assert ei.value.code == B.EXMOE_ERR_SHAPE
    with pytest.raises(B.ExmoeError) as ei:
        B.Cache(s, [bank], 9, max_tokens=4)           # C > E
    assert ei.value.code == B.EXMOE_ERR_SHAPE
    unpinned = bank.clone()                           # pageable copy
    with pytest.raises(B.ExmoeError) as ei:
        B.Cache(s, [unpinned], 4, max_tokens=4)
    assert ei.value.code == B.EXMOE_ERR_NOT_PINNED


def test_multi_layer_caches_are_independent(B, tiny_layer):
    ora, bank = tiny_layer
    s = synth.TINY
    ora2, bank2 = helpers.make_layer(s, seed=1)
    cache = B.Cache(s, [bank, bank2], 3, max_tokens=16)
    hidden, ids, p = helpers.routed_inputs(s, 8, seed=21)
    for layer, o in ((0, ora), (1, ora2), (0, ora)):
        out = cache.forward(layer, hidden.cuda(), ids.cuda(), p.cuda())
        y, ref = o.forward(hidden, ids, p)
        helpers.check_output(out, y, ref, f"layer {layer}")
    assert cache.stats(0)["forwards"] == 2 and cache.stats(1)["forwards"] == 1
    cache.reset(0)
    assert cache.stats(0)["forwards"] == 0 and (cache.state(0)[0] == -1).all()
    cache.close()


@pytest.mark.parametrize("T", [1, 5, 40, 160])
def test_shared_expert_geometry(B, T):
    """A Qwen-MoE-like block: routed experts with d_ff = 1408 (11 blocks of 128) chosen 4 at a time, plus a shared
    expert of d_ff = 5632 (44 blocks) that every token uses with weight 1.  The shared expert is a second bank with
    one expert and top_k = 1; the block output is the sum of the two layer outputs.  Both run on every kernel path
    (pairwise, grouped small, streaming, tensor-core small-N) as T grows."""
    routed = synth.Shape(d_model=2048, d_ff=1408, num_experts=12, top_k=4)
    shared = synth.Shape(d_model=2048, d_ff=5632, num_experts=1, top_k=1)
    if not hasattr(test_shared_expert_geometry, "layers"):
        test_shared_expert_geometry.layers = (helpers.make_layer(routed, seed=611), helpers.make_layer(shared, seed=612))
    (ora_r, bank_r), (ora_s, bank_s) = test_shared_expert_geometry.layers
    hidden, ids, p = helpers.routed_inputs(routed, T, seed=6100 + T, alpha=0.5)
    ids_s = torch.zeros((T, 1), dtype=torch.int32)
    w_s = torch.ones((T, 1), dtype=torch.float32)
    y_r, ref_r = ora_r.forward(hidden, ids, p)
    y_s, ref_s = ora_s.forward(hidden, ids_s, w_s)
    cr = B.Cache(routed, [bank_r], 6, max_tokens=160)                       # half of the routed experts resident
    cs = B.Cache(shared, [bank_s], 1, max_tokens=160)
    out_r = cr.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).clone()
    out_s = cs.forward(0, hidden.cuda(), ids_s.cuda(), w_s.cuda()).clone()
    helpers.check_output(out_r, y_r, ref_r, f"routed T={T}")
    helpers.check_output(out_s, y_s, ref_s, f"shared T={T}")
    block = out_r.float() + out_s.float()                                    # the caller's sum, as for the residual
    want = ref_r.astype(np.float64) + ref_s.astype(np.float64)
    err = block.cpu().numpy().astype(np.float64) - want
    assert np.linalg.norm(err) <= 2 * helpers.REL_FRO * np.linalg.norm(want)
    full = B.Cache(routed, [bank_r], 12, max_tokens=160)
    assert torch.equal(full.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).view(torch.int16), out_r.view(torch.int16))
    for c in (cr, cs, full):
        assert c.status() == 0
        c.close()


def test_padding_of_dims_that_are_not_multiples_of_128(B):
    """Section 7 leaves shapes that are not multiples of the group size to padding.  d_model = 200, d_ff = 300 padded with zeros to 256 / 384:
    the padded layer matches the oracle on the padded weights, its extra output columns are exactly zero, and the
    first 200 columns agree, up to int4 quantisation noise, with the unquantised layer (Eq. 2) on the unpadded weights."""
    raw = synth.Shape(d_model=200, d_ff=300, num_experts=4, top_k=2)
    g = torch.Generator().manual_seed(99)
    wg = (torch.randn((4, 300, 200), generator=g) * 0.05).bfloat16()
    wu = (torch.randn((4, 300, 200), generator=g) * 0.05).bfloat16()
    wd = (torch.randn((4, 200, 300), generator=g) * 0.05).bfloat16()
    Hp, Ip = B.padded_dims(200, 300)
    assert (Hp, Ip) == (256, 384)
    pg, pu, pd = B.pad_expert_weights(wg, wu, wd)
    assert pg.shape == (4, 384, 256) and pd.shape == (4, 256, 384)
    assert torch.equal(pg[:, :300, :200], wg) and float(pg[:, 300:, :].abs().max()) == 0 and float(pd[:, 200:, :].abs().max()) == 0
    s = synth.Shape(d_model=Hp, d_ff=Ip, num_experts=4, top_k=2)
    ora = helpers.OracleLayer(s, pg, pu, pd)
    bank = B.pack_bank(s, pg, pu, pd)
    T = 9
    hidden = torch.randn((T, 200), generator=g).bfloat16()
    ids = torch.stack([torch.randperm(4, generator=g)[:2] for _ in range(T)]).int()
    p = torch.rand((T, 2), generator=g).float()
    hp = B.pad_hidden(hidden, Hp)
    cache = B.Cache(s, [bank], 4, max_tokens=16)
    out = cache.forward(0, hp.cuda(), ids.cuda(), p.cuda())
    y, ref = ora.forward(hp, ids, p)
    helpers.check_output(out, y, ref, "padded")
    assert float(out[:, 200:].float().abs().max()) == 0.0
    # the unpadded, unquantised layer in fp64: Eq. 2 on the original tensors
    x = hidden.double().numpy()
    want = np.zeros((T, 200))
    for t in range(T):
        for j in range(2):
            e = int(ids[t, j])
            a, b = wg[e].double().numpy() @ x[t], wu[e].double().numpy() @ x[t]
            want[t] += float(p[t, j]) * (wd[e].double().numpy() @ (a / (1 + np.exp(-a)) * b))
    got = out[:, :200].float().cpu().numpy().astype(np.float64)
    # int4 group quantisation noise of three matrices is ~0.2 of the signal; a misplaced column or slice gives ~1.4
    assert np.linalg.norm(got - want) <= 0.35 * np.linalg.norm(want)
    assert cache.status() == 0
    cache.close()
