"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module only draws random tensors.  It holds none of the method's arithmetic (no quantiser,
no expert MLP, no cache logic, no router: Eq. 1 is `exmoe_route` in the library, `oracle/router.py`
in the oracle and a torch restatement in the test helpers), so both the CUDA path and the CPU
oracle can be fed from it without sharing code.

Recipe (stand-in for the OLMoE checkpoint and prompts the paper measures on):
  expert weights  N(0, 0.02) rounded to BF16          W_g, W_u: [E, I, H]   W_d: [E, H, I]
  hidden states   N(0, 1)    rounded to BF16          [T, H]
  router          N(0, 0.02) rounded to BF16          [E, H]
  routing         (by the caller's router) logits + optional per-expert bias, softmax over all
                  E experts, top-k, ties to the lower expert id, weights NOT renormalised.
  Zipf skew       bias_e = alpha * (-1.1 * ln rank_e), rank a seeded permutation of 1..E.
"""
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Shape:
    d_model: int
    d_ff: int
    num_experts: int
    top_k: int
    group_size: int = 128


TINY = Shape(d_model=256, d_ff=128, num_experts=8, top_k=2)        # config 1
OLMOE = Shape(d_model=2048, d_ff=1024, num_experts=64, top_k=8)    # configs 2-5
MID = Shape(d_model=512, d_ff=256, num_experts=16, top_k=4)        # parity size between the two


def _gen(seed, device="cpu"):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal_bf16(shape, std, seed, device="cpu"):
    x = torch.randn(*shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return (x * std).to(torch.bfloat16)


def expert_weights(shape: Shape, seed, device="cpu", std=0.02):
    """(W_g [E,I,H], W_u [E,I,H], W_d [E,H,I]) in BF16."""
    E, I, H = shape.num_experts, shape.d_ff, shape.d_model
    wg = normal_bf16((E, I, H), std, 3 * seed + 0, device)
    wu = normal_bf16((E, I, H), std, 3 * seed + 1, device)
    wd = normal_bf16((E, H, I), std, 3 * seed + 2, device)
    return wg, wu, wd


def hidden_states(shape: Shape, T, seed, device="cpu"):
    return normal_bf16((T, shape.d_model), 1.0, seed, device)


def router_weights(shape: Shape, seed, device="cpu"):
    return normal_bf16((shape.num_experts, shape.d_model), 0.02, seed, device)


def zipf_bias(num_experts, alpha, seed):
    """alpha * (-1.1 * ln rank_e) with rank a seeded permutation of 1..E (fp32, CPU)."""
    perm = torch.randperm(num_experts, generator=_gen(seed))
    rank = torch.empty(num_experts, dtype=torch.float32)
    rank[perm] = torch.arange(1, num_experts + 1, dtype=torch.float32)
    return alpha * (-1.1 * torch.log(rank))


class SyntheticStack:
    """Stand-in for a 16-layer sparse model around the MoE layers (config 5): per layer BF16 router weights and an
    optional Zipf bias, and between layers the dense parts abstracted to h <- bf16(h + moe_out + N(0, 0.1)).
    Only input generation: the MoE layer is `layer_fn`, the router (Eq. 1) is `route_fn`, both the caller's."""

    def __init__(self, shape: Shape, num_layers, seed, alpha=1.0, device="cpu"):
        self.shape, self.L, self.device = shape, int(num_layers), device
        self.routers = [router_weights(shape, seed + 17 * l, device=device) for l in range(self.L)]
        self.bias = [zipf_bias(shape.num_experts, alpha, seed + 1000 + l).to(device) if alpha else None
                     for l in range(self.L)]
        self.gen = _gen(seed + 5, device)

    def draw_noise(self, T):
        """One N(0, 0.1) residual per layer, for callers that need fixed tensors (CUDA-graph capture)."""
        return [torch.randn((T, self.shape.d_model), generator=self.gen, device=self.device, dtype=torch.float32) * 0.1
                for _ in range(self.L)]

    def step(self, layer_fn, hidden, route_fn, record=None, noise=None, lookahead_fn=None):
        """layer_fn(layer, hidden, ids, weights) -> moe output.  Returns the hidden state after all layers.
        `noise`: per-layer residual tensors to use instead of drawing fresh ones.
        `route_fn(layer, hidden) -> (ids, weights)`: the router (Eq. 1), applied by the caller to this stack's
        `routers[layer]` and `bias[layer]`.
        `lookahead_fn(next_layer, hidden)`: called before layer l runs, with layer l's input and l + 1 (a prefetch
        policy can guess layer l + 1's experts from it); its result is ignored."""
        h = hidden
        for l in range(self.L):
            ids, w = route_fn(l, h)
            if lookahead_fn is not None and l + 1 < self.L:
                lookahead_fn(l + 1, h)
            out = layer_fn(l, h, ids, w)
            if record is not None:
                record.append((l, h, ids, w, out))
            eps = noise[l] if noise is not None else \
                torch.randn(h.shape, generator=self.gen, device=h.device, dtype=torch.float32) * 0.1
            h = (h.float() + out.float() + eps).to(torch.bfloat16)
        return h
