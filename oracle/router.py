"""Router of a sparse block (oracle; test infrastructure).

Eq. 1 of the paper (Section 3.1):  z_t = W_r h_t,  S_t = TopK(z_t, k),  "with router-derived mixture
weights p_{t,e}".  The paper keeps the model's own router unchanged; for the OLMoE geometry it evaluates
(Section 4.1) that router is: softmax of the logits over all E experts, the k largest, the mixture weights
are the selected probabilities as they are (never renormalised over the selected k, Section 3.4).

Reading taken where the paper is silent: equal logits are ordered by ascending expert id; an optional
per-expert additive bias on the logits (used by the synthetic Zipf-skewed workloads) enters before the softmax.

Everything is binary64 on the exact values of the BF16 inputs: the definition written out, one token at a time.
"""
import numpy as np


def softmax(z):
    """p_e = exp(z_e) / sum_j exp(z_j), evaluated after subtracting max(z) (the value is unchanged)."""
    z = np.asarray(z, dtype=np.float64)
    e = np.exp(z - np.max(z))
    return e / np.sum(e)


def route_token(h, w_router, top_k, bias=None):
    """One token.  Returns (ids int32 [k] in descending-logit order, p float64 [k], z float64 [E])."""
    z = np.asarray(w_router, dtype=np.float64) @ np.asarray(h, dtype=np.float64)
    if bias is not None:
        z = z + np.asarray(bias, dtype=np.float64)
    p = softmax(z)
    order = sorted(range(len(z)), key=lambda e: (-z[e], e))[:top_k]     # largest logit first, ties to the lower id
    ids = np.asarray(order, dtype=np.int32)
    return ids, p[ids], z


def route(hidden, w_router, top_k, bias=None):
    """Eq. 1 for every token: (ids int32 [T, k], p float64 [T, k], logits float64 [T, E])."""
    hidden = np.asarray(hidden, dtype=np.float64)
    T, E = hidden.shape[0], np.asarray(w_router).shape[0]
    ids = np.zeros((T, top_k), dtype=np.int32)
    p = np.zeros((T, top_k), dtype=np.float64)
    z = np.zeros((T, E), dtype=np.float64)
    for t in range(T):
        ids[t], p[t], z[t] = route_token(hidden[t], w_router, top_k, bias)
    return ids, p, z
