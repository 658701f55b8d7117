"""Shared test scaffolding: builds a synthetic layer for both sides (CUDA library and CPU oracle).

The oracle side quantises the BF16 weights itself (oracle.quant); nothing it consumes comes from
the GPU.  The GPU side packs the same BF16 weights with exmoe_pack.
"""
import numpy as np
import torch

from oracle import cache as ocache
from oracle import layout as olayout
from oracle import moe as omoe
from oracle import quant as oquant
from paper_2608_15383_b200 import synth

# spec tolerance for the BF16 layer output
MAX_ERR_FRAC = 2e-2      # max |err| <= 2e-2 * max |ref|
REL_FRO = 5e-3           # ||err||_F / ||ref||_F <= 5e-3


class OracleLayer:
    """Dequantised experts of one layer, computed lazily by the oracle's own quantiser."""

    def __init__(self, shape, wg, wu, wd):
        self.shape, self.wg, self.wu, self.wd = shape, wg, wu, wd
        self._deq = {}
        self.max_cached = 40

    def expert(self, e):
        if e not in self._deq:
            mats = []
            for w in (self.wg[e], self.wu[e], self.wd[e]):
                q, s = oquant.quantize_g128(w.float().cpu().numpy())
                mats.append(oquant.dequantize_g128(q, s))
            if len(self._deq) >= self.max_cached:               # bound host memory (150 MB per OLMoE expert)
                self._deq.pop(next(iter(self._deq)))
            self._deq[e] = tuple(mats)
        return self._deq[e]

    def packed(self, e):
        return olayout.pack_expert(self.wg[e].float().cpu().numpy(), self.wu[e].float().cpu().numpy(),
                                   self.wd[e].float().cpu().numpy())

    def forward(self, hidden, ids, w, round_activation=False):
        return omoe.moe_layer_forward(hidden.float().cpu().numpy(), ids.cpu().numpy(), w.cpu().numpy(),
                                      self.expert, self.shape.num_experts, round_activation=round_activation)


def check_output(out_gpu, y_ref, out_ref, what=""):
    """out_gpu: BF16 tensor; y_ref unrounded float64; out_ref BF16-rounded float64."""
    got = out_gpu.float().cpu().numpy().astype(np.float64)
    err = got - out_ref
    max_ref = np.abs(out_ref).max()
    fro = np.linalg.norm(err) / max(np.linalg.norm(out_ref), 1e-30)
    assert np.isfinite(got).all(), what
    assert np.abs(err).max() <= MAX_ERR_FRAC * max_ref, (what, np.abs(err).max(), max_ref)
    assert fro <= REL_FRO, (what, fro)
    return fro


def make_layer(shape, seed, device="cuda"):
    from paper_2608_15383_b200 import binding
    wg, wu, wd = synth.expert_weights(shape, seed)
    bank = binding.pack_bank(shape, wg, wu, wd, device=device)
    return OracleLayer(shape, wg, wu, wd), bank


def route(hidden, w_router, top_k, bias=None):
    """Harness router, Eq. 1 restated with torch ops in binary32: logits -> softmax over all experts -> top-k, ties
    to the lower id, no renormalisation.  Returns (ids int32 [T,k], p fp32 [T,k]).  It only makes layer INPUTS for
    the tests (the product's router is exmoe_route, the oracle's is oracle/router.py)."""
    logits = hidden.float() @ w_router.float().t()
    if bias is not None:
        logits = logits + bias.to(logits.device)
    p = torch.softmax(logits, dim=-1)
    order = torch.sort(-p, dim=-1, stable=True).indices[:, :top_k]
    w = torch.gather(p, 1, order)
    return order.to(torch.int32).contiguous(), w.contiguous()


def routed_inputs(shape, T, seed, alpha=0.0, device="cuda"):
    hidden = synth.hidden_states(shape, T, seed)
    wr = synth.router_weights(shape, seed + 7919)
    bias = synth.zipf_bias(shape.num_experts, alpha, seed + 31) if alpha else None
    ids, p = route(hidden, wr, shape.top_k, bias)
    return hidden, ids, p


def oracle_plan(sc: ocache.SlotCache, ids):
    plan = sc.resolve(ids)
    counts, offsets, perm = ocache.group_pairs(ids, plan, sc.C, sc.max_waves)
    return plan, counts, offsets, perm


def compare_plan(cache, sc, ids, layer=0):
    """Advance the oracle's slot cache by this call and compare plan, grouping, state and counters bit for bit."""
    plan, counts, offsets, perm = oracle_plan(sc, ids.numpy())
    got = cache.last_plan(layer, ids.numel())
    assert got["n_active"] == plan.n_active and got["n_waves"] == plan.n_waves
    assert np.array_equal(got["wave_of"], plan.wave_of)
    assert np.array_equal(got["slot_of"], plan.slot_of)
    assert got["misses"] == plan.misses
    assert np.array_equal(got["counts"], counts)
    assert np.array_equal(got["offsets"], offsets)
    assert np.array_equal(got["perm"], perm)
    if sc.C < sc.E:
        es, se, stamp, tick = cache.state(layer)
        assert np.array_equal(es, sc.expert_slot) and np.array_equal(se, sc.slot_expert)
        assert np.array_equal(stamp, sc.slot_stamp) and tick == sc.tick
    st = cache.stats(layer)
    assert st == {"lookups": sc.stats.lookups, "hits": sc.stats.hits, "misses": sc.stats.misses,
                  "waves": sc.stats.waves, "h2d_bytes": sc.stats.h2d_bytes, "forwards": sc.stats.forwards}
    return plan
