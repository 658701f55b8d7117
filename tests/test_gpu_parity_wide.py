"""GPU parity, the wider cases: config 4 sampled from the plan (group ends and token-tile edges), the tensor-core kernels
at OLMoE shape in the batched-decode range and on single-expert group sizes (the kernel-level gate of Sec. 5.3), the
global-histogram grouping path, config 5 at its real size (16 OLMoE layers, teacher-forced), and guard bands around
every buffer the kernels write (the stand-in for a memory checker: no byte outside a buffer may change).
"""
import numpy as np
import pytest
import torch

from oracle import cache as ocache
from paper_2608_15383_b200 import synth

import helpers

pytestmark = pytest.mark.gpu
compare_plan = helpers.compare_plan


@pytest.fixture(scope="module")
def B():
    from paper_2608_15383_b200 import binding, build
    build.build()
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def olmoe_layer(B):
    ora, bank = helpers.make_layer(synth.OLMOE, seed=2000)
    ora.max_cached = 64                                   # every expert stays dequantised (3.2 GB of host memory)
    return ora, bank


def tile_rows(cnt, bn):
    """First rows of the token tiles a group of `cnt` rows is cut into: ceil(cnt / bn) pieces of equal size rounded up
    to 16 rows (the rule of the tensor-core kernels' tile list; restated here only to CHOOSE which rows to sample)."""
    pieces = -(-cnt // bn)
    per = (-(-cnt // pieces) + 15) // 16 * 16
    return list(range(0, cnt, per))


@pytest.mark.parametrize("alpha", [0.0, 1.0])
def test_config4_prefill_olmoe_sampled_from_the_plan(B, olmoe_layer, alpha):
    """Config 4 (2048 tokens x top-8 over 64 experts, uniform and Zipf): the tokens behind the first and the last
    grouped row of every active expert and behind the rows on both sides of every token-tile edge are checked against
    the oracle, plus one row from the middle of every group."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    T = 2048
    hidden, ids, p = helpers.routed_inputs(s, T, seed=4000, alpha=alpha)
    cache = B.Cache(s, [bank], 64, max_tokens=T)
    sc = ocache.SlotCache(64, 64, 0, bytes_per_expert=cache.bytes_per_expert)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    assert cache.last_path() == B.PATH_TENSOR
    compare_plan(cache, sc, ids)
    plan = cache.last_plan(0, ids.numel())
    tokens = set()
    for e in range(64):
        cnt, off = int(plan["counts"][e]), int(plan["offsets"][e])
        if cnt == 0:
            continue
        rows = {0, cnt // 2, cnt - 1}
        for n0 in tile_rows(cnt, 256)[1:]:
            rows.update((n0 - 1, n0))
        tokens.update(int(plan["perm"][off + r]) // s.top_k for r in rows)
    sample = sorted(tokens)
    assert 100 <= len(sample) <= 700                      # group ends of different experts often share a token
    y, ref = ora.forward(hidden[sample], ids[sample], p[sample])
    helpers.check_output(out[sample], y, ref, f"alpha={alpha}, {len(sample)} tokens")
    assert cache.status() == 0
    cache.close()


@pytest.mark.parametrize("T", [96, 128])
def test_small_n_tensor_core_kernels_at_olmoe_shape(B, olmoe_layer, T):
    """Batched decode with 768 and 1024 pairs at OLMoE shape: the 64-row, eight-stage tensor-core kernel shape, every
    token against the oracle."""
    ora, bank = olmoe_layer
    s = synth.OLMOE
    hidden, ids, p = helpers.routed_inputs(s, T, seed=7100 + T, alpha=1.0)
    y, ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], 64, max_tokens=T)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    assert cache.last_path() == B.PATH_TENSOR_SMALL_N
    helpers.check_output(out, y, ref, f"T={T}")
    assert cache.status() == 0
    cache.close()


@pytest.mark.parametrize("M", [641, 800, 1025, 1300])
def test_group_size_sweep_reaches_the_tensor_core_kernels(B, M):
    """One expert, k = 1, group sizes past the streaming kernels' range: both tensor-core kernel shapes on a single
    group with ragged tiles (641 = 10 tiles of 64 rows + 1 row; 1300 = 6 tiles of 224 rows, the last one short),
    every row against the dequantised reference (Sec. 5.3 checks group sizes against such a reference)."""
    s = synth.Shape(d_model=2048, d_ff=1024, num_experts=2, top_k=1)
    if not hasattr(test_group_size_sweep_reaches_the_tensor_core_kernels, "layer"):
        test_group_size_sweep_reaches_the_tensor_core_kernels.layer = helpers.make_layer(s, seed=77)
    ora, bank = test_group_size_sweep_reaches_the_tensor_core_kernels.layer
    hidden = synth.hidden_states(s, M, seed=900 + M)
    ids = torch.ones((M, 1), dtype=torch.int32)
    p = torch.rand((M, 1), generator=torch.Generator().manual_seed(M)) + 0.5
    y, ref = ora.forward(hidden, ids, p)
    cache = B.Cache(s, [bank], 2, max_tokens=M)
    out = cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda())
    assert cache.last_path() == (B.PATH_TENSOR_SMALL_N if M <= 1024 else B.PATH_TENSOR)
    helpers.check_output(out, y, ref, f"M={M}")
    assert cache.status() == 0
    cache.close()


def test_global_histogram_grouping_path(B):
    """A key space of 8192 (256 experts, 128 slots, waves of 4) with more than 2048 pairs: grouping by global histogram
    and one CTA per key (the scheme behind the single-CTA and the chunked ones).  Plan, state and counters bit for
    bit against the oracle over several calls; output against the oracle and against the resident run."""
    s = synth.Shape(d_model=128, d_ff=128, num_experts=256, top_k=4)
    ora, bank = helpers.make_layer(s, seed=321)
    T = 600
    cache = B.Cache(s, [bank], 128, max_tokens=T, wave_cap=4)
    assert cache.n_keys == 8192
    full = B.Cache(s, [bank], s.num_experts, max_tokens=T)
    sc = ocache.SlotCache(s.num_experts, 128, 4, bytes_per_expert=cache.bytes_per_expert)
    for step in range(3):
        hidden, ids, p = helpers.routed_inputs(s, T, seed=8100 + step, alpha=0.3)
        h, i, w = hidden.cuda(), ids.cuda(), p.cuda()
        out = cache.forward(0, h, i, w)
        compare_plan(cache, sc, ids)
        ref_out = full.forward(0, h, i, w)
        assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16)), step
    y, ref = ora.forward(hidden, ids, p)
    helpers.check_output(out, y, ref, "key space 8192")
    assert cache.status() == 0 and full.status() == 0
    cache.close()
    full.close()


def test_config5_real_size_teacher_forced(B):
    """Config 5 at the paper's geometry (Sec. 4.1: 16 sparse layers, 64 experts, top-8, 2048 / 1024), 16 slots, 16
    tokens, one step: per layer the plan, state and counters bit for bit against the oracle's cache model, and the
    output of sampled tokens against the oracle fed with the GPU's layer input and routing (teacher forcing)."""
    s, L, T, C = synth.OLMOE, 16, 16, 16
    layers = []
    for l in range(L):
        wg, wu, wd = synth.expert_weights(s, 6000 + l, device="cuda")
        layers.append((helpers.OracleLayer(s, wg, wu, wd), B.pack_bank(s, wg, wu, wd)))
    cache = B.Cache(s, [bank for _, bank in layers], C, max_tokens=T)
    models = [ocache.SlotCache(s.num_experts, C, 0, bytes_per_expert=cache.bytes_per_expert) for _ in range(L)]
    stack = synth.SyntheticStack(s, L, seed=41, alpha=0.5, device="cuda")
    h = synth.hidden_states(s, T, seed=4).cuda()
    waves = []
    for l in range(L):
        bias = None if stack.bias[l] is None else stack.bias[l].float().contiguous()
        ids, w = B.exmoe_route(s, h, stack.routers[l], bias)
        out = cache.forward(l, h, ids, w).clone()
        plan = compare_plan(cache, models[l], ids.cpu(), layer=l)
        waves.append(plan.n_waves)
        sample = [0, 5, 10, T - 1]                           # four tokens per layer: up to 32 experts to dequantise
        y, ref = layers[l][0].forward(h[sample].cpu(), ids[sample].cpu(), w[sample].cpu())
        helpers.check_output(out[sample], y, ref, f"layer {l}")
        layers[l][0]._deq.clear()
        h = (h.float() + out.float() + stack.draw_noise(T)[0]).to(torch.bfloat16)
    assert max(waves) >= 2 and cache.status() == 0
    assert bool(torch.isfinite(h.float()).all())
    cache.close()


def guarded_out(T, H):
    """An output tensor inside a larger one filled with a pattern; returns (view, whole, first, last)."""
    pad = 4096
    whole = torch.full((T * H + 2 * pad,), -1.0, dtype=torch.bfloat16, device="cuda")      # 0xBF80 everywhere
    return whole[pad:pad + T * H].view(T, H), whole, pad, pad + T * H


def out_guards_intact(whole, first, last):
    torch.cuda.synchronize()
    return bool((whole[:first] == -1.0).all()) and bool((whole[last:] == -1.0).all())


@pytest.mark.parametrize("case", ["pairwise", "in-CTA grouping, several waves", "streaming", "tensor small-N", "tensor large-N",
                                  "chunked grouping", "host copies", "prefetch"])
def test_no_kernel_writes_outside_its_buffers(B, case):
    """Slot memory, workspace and the output each sit between margins filled with a pattern; one call per kernel path,
    both miss paths and the prefetch; afterwards every margin byte is unchanged (and the result is still right)."""
    s = synth.MID
    if not hasattr(test_no_kernel_writes_outside_its_buffers, "layer"):
        test_no_kernel_writes_outside_its_buffers.layer = helpers.make_layer(s, seed=5)
    ora, bank = test_no_kernel_writes_outside_its_buffers.layer
    T, C, Cw, want = {"pairwise": (2, 16, 0, B.PATH_PAIR), "in-CTA grouping, several waves": (5, 6, 3, B.PATH_SMALL),
                      "streaming": (40, 6, 0, B.PATH_STREAM), "tensor small-N": (200, 6, 3, B.PATH_TENSOR_SMALL_N),
                      "tensor large-N": (300, 16, 0, B.PATH_TENSOR), "chunked grouping": (700, 6, 0, B.PATH_TENSOR),
                      "host copies": (40, 5, 2, B.PATH_STREAM), "prefetch": (3, 8, 0, None)}[case]
    cache = B.Cache(s, [bank], C, max_tokens=T, wave_cap=Cw, guard_bytes=1 << 16)
    if case == "host copies":
        cache.set_miss_path(B.MISS_HOST_COPIES)
    hidden, ids, p = helpers.routed_inputs(s, T, seed=9300 + T, alpha=0.5)
    y, ref = ora.forward(hidden, ids, p)
    out, whole, first, last = guarded_out(T, s.d_model)
    if case == "prefetch":
        cache.prefetch(0, ids.cuda().reshape(-1)[:8].contiguous())
    for _ in range(2):                                       # a cold cache, then hits and LRU replacement
        cache.forward(0, hidden.cuda(), ids.cuda(), p.cuda(), out=out)
    if want is not None:
        assert cache.last_path() == want
    assert cache.guards_intact() and out_guards_intact(whole, first, last)
    helpers.check_output(out, y, ref, case)
    assert cache.status() == 0
    cache.close()


def test_static_entry_point_writes_only_its_output(B):
    s = synth.MID
    ora, bank = test_no_kernel_writes_outside_its_buffers.layer if hasattr(test_no_kernel_writes_outside_its_buffers, "layer") \
        else helpers.make_layer(s, seed=5)
    T = 4
    hidden, ids, p = helpers.routed_inputs(s, T, seed=9400)
    y, ref = ora.forward(hidden, ids, p)
    out, whole, first, last = guarded_out(T, s.d_model)
    stream = torch.cuda.Stream()                             # not the default stream
    stream.wait_stream(torch.cuda.current_stream())
    B.exmoe_moe_forward_static_status()                      # the word is sticky: drop what an earlier caller left
    B.exmoe_moe_forward_static(s, bank.cuda().reshape(-1), hidden.cuda(), ids.cuda(), p.cuda(), out, stream=stream)
    stream.synchronize()
    assert out_guards_intact(whole, first, last)
    helpers.check_output(out, y, ref, "static, side stream")
    assert B.exmoe_moe_forward_static_status() == 0
    bad = ids.clone()
    bad[1, 0] = -3
    B.exmoe_moe_forward_static(s, bank.cuda().reshape(-1), hidden.cuda(), bad.cuda(), p.cuda(), out, stream=stream)
    assert B.exmoe_moe_forward_static_status() == B.EXMOE_ERR_BAD_EXPERT_ID      # reported, then cleared
    assert B.exmoe_moe_forward_static_status() == 0
    # a shape whose down kernel would need 264 KB of shared memory is refused before anything is queued
    big = synth.Shape(d_model=256, d_ff=4096, num_experts=32, top_k=32)
    with pytest.raises(B.ExmoeError) as ei:
        B.exmoe_moe_forward_static(big, bank.cuda().reshape(-1), torch.zeros((1, 256), dtype=torch.bfloat16, device="cuda"),
                                   torch.zeros((1, 32), dtype=torch.int32, device="cuda"),
                                   torch.zeros((1, 32), dtype=torch.float32, device="cuda"),
                                   torch.zeros((1, 256), dtype=torch.bfloat16, device="cuda"))
    assert ei.value.code == B.EXMOE_ERR_SHAPE


def test_zero_tokens_through_the_abi_and_host_copy_bytes(B):
    """T = 0 reaches the C entry points (no early return in the binding); the host-buffer call copies what T needs,
    not what max_tokens would."""
    s = synth.MID
    ora, bank = helpers.make_layer(s, seed=5)
    cache = B.Cache(s, [bank], s.num_experts, max_tokens=2048)
    empty_h = torch.empty((0, s.d_model), dtype=torch.bfloat16, device="cuda")
    empty_i = torch.empty((0, s.top_k), dtype=torch.int32, device="cuda")
    empty_w = torch.empty((0, s.top_k), dtype=torch.float32, device="cuda")
    assert cache.forward(0, empty_h, empty_i, empty_w).shape == (0, s.d_model)
    assert cache.forward_host(0, empty_h.cpu(), empty_i.cpu(), empty_w.cpu()).shape == (0, s.d_model)
    B.exmoe_moe_forward_static(s, bank.cuda().reshape(-1), empty_h, empty_i, empty_w, torch.empty_like(empty_h))
    hidden, ids, p = helpers.routed_inputs(s, 1, seed=9500)
    y, ref = ora.forward(hidden, ids, p)
    out = cache.forward_host(0, hidden, ids, p)
    helpers.check_output(out, y, ref, "host call, T = 1 of max_tokens = 2048")
    assert cache.last_host_copy_bytes() == s.d_model * 2 + 2 * s.top_k * 4       # 1056 bytes, not 2 MB
    assert cache.status() == 0
    cache.close()


@pytest.mark.parametrize("T", [16, 128, 2048])
def test_graph_replay_of_the_larger_paths_is_bit_identical_to_plain_launches(B, olmoe_layer, T):
    """bench.py times every leg as a CUDA-graph replay: the streaming kernels (T = 16), the 64-row tensor-core shape
    (T = 128) and the 256-row one (T = 2048, config 4) must give, replayed from a graph over two rotating input sets,
    the very bits of their plain launches (which the other tests hold to the oracle)."""
    _, bank = olmoe_layer
    s = synth.OLMOE
    cache = B.Cache(s, [bank], 64, max_tokens=T)
    inputs = [tuple(x.cuda() for x in helpers.routed_inputs(s, T, seed=8800 + T + i, alpha=0.5)) for i in range(2)]
    plain = [cache.forward(0, h, i, w).clone() for h, i, w in inputs]
    want = {16: B.PATH_STREAM, 128: B.PATH_TENSOR_SMALL_N, 2048: B.PATH_TENSOR}[T]
    assert cache.last_path() == want
    outs = [torch.zeros_like(plain[0]) for _ in inputs]
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for (h, i, w), o in zip(inputs, outs):
            cache.forward(0, h, i, w, out=o, stream=stream)
    for rep in range(2):
        for o in outs:
            o.zero_()
        with torch.cuda.stream(stream):
            g.replay()
        stream.synchronize()
        for o, p in zip(outs, plain):
            assert torch.equal(o.view(torch.int16), p.view(torch.int16)), f"T={T} replay {rep}"
    assert cache.status() == 0
    cache.close()
