"""Sparse block output with dequantised int4 experts (oracle; test infrastructure).

Eq. 2 of the paper (Section 3.1):

    y_t = sum_{e in S_t} p_{t,e} * W_d,e [ phi(W_g,e h_t) (.) W_u,e h_t ],

with W_g, W_u, W_d replaced by their dequantised values W^ = s*q, which "define
the corresponding mathematical operations" (Section 3.1, Section 3.2).  Router weights are
used as given and never renormalised (Section 3.4).  phi is SiLU (the experts are
SwiGLU MLPs).  Everything is binary64; the layer result is rounded once to BF16
because the block hands BF16 activations to the rest of the model.

The loop below is the definition written out: for every token, for every one of
its k selected experts in the order given, three matrix-vector products.  Waves,
slots and token grouping are execution details that do not appear here, which is
the point: the result must not depend on them (Section 3.4, last sentence).
"""
import numpy as np

from .bf16 import round_to_bf16


def silu(g):
    """phi(g) = g * sigmoid(g) = g / (1 + exp(-g))."""
    g = np.asarray(g, dtype=np.float64)
    with np.errstate(over="ignore"):
        return g / (1.0 + np.exp(-g))


def expert_ffn(x, w_gate, w_up, w_down, round_activation=False):
    """One expert on one token: W_d [ phi(W_g x) (.) W_u x ]  (the bracket of Eq. 2).

    round_activation: round the bracket's left factor a = phi(g) (.) u to BF16 before the down projection.  This is
    NOT the definition; it is the one rounding every implementation with BF16 activations between the two
    projections must make, kept as a second mode so that a test can see how much of the distance to the
    definition that single rounding explains."""
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(w_gate, dtype=np.float64) @ x
    u = np.asarray(w_up, dtype=np.float64) @ x
    a = silu(g) * u
    if round_activation:
        a = round_to_bf16(a)
    return np.asarray(w_down, dtype=np.float64) @ a


def moe_layer_forward(hidden, topk_ids, topk_weights, expert_weights, num_experts, round_activation=False):
    """Eq. 2 for every token.

    hidden        float [T, H]  (BF16-valued)
    topk_ids      int   [T, k]  selected experts, in the router's order
    topk_weights  float [T, k]  mixture weights p, used as given
    expert_weights(e) -> (W^_g [I,H], W^_u [I,H], W^_d [H,I]) dequantised, float64
    An id outside [0, num_experts) selects nothing and contributes nothing.

    Returns (y float64 [T, H] unrounded, out float64 [T, H] rounded to BF16).
    """
    hidden = np.asarray(hidden, dtype=np.float64)
    topk_ids = np.asarray(topk_ids)
    topk_weights = np.asarray(topk_weights, dtype=np.float64)
    T, H = hidden.shape
    y = np.zeros((T, H), dtype=np.float64)
    for t in range(T):
        acc = np.zeros(H, dtype=np.float64)
        for j in range(topk_ids.shape[1]):
            e = int(topk_ids[t, j])
            if e < 0 or e >= num_experts:
                continue
            wg, wu, wd = expert_weights(e)
            acc += topk_weights[t, j] * expert_ffn(hidden[t], wg, wu, wd, round_activation)
        y[t] = acc
    return y, round_to_bf16(y)
