"""Symmetric group-128 int4 quantiser of one expert matrix (oracle; test infrastructure).

Follows Eq. 3 of the paper (Section 3.2): for W in R^{N x K}, the input dimension K
is cut into groups of 128; for row i and group g

    s = max_j |W_ij| / 7,   q_ij = clip(round(W_ij / s), -8, 7),   W^_ij = s * q_ij,

and an all-zero group is defined as s = 0, q = 0 with no division.  Scales are
stored as FP16 (Section 3.2, "pack q and FP16 scales").

Readings where the paper is silent (each one is listed in the design notes):
  * "round" is round-half-to-even.
  * absmax, the division by 7 and the division W/s are single IEEE binary32 operations.
  * the divisor is the STORED scale, i.e. the FP16-rounded value widened back to
    binary32, so that q and W^ are consistent with what a kernel later reads.
  * a scale that rounds to FP16 zero makes the group a zero group; a scale that
    is not finite in FP16, or a non-finite weight, is an error.
"""
import numpy as np

GROUP = 128


class NonFiniteError(ValueError):
    pass


def quantize_g128(W):
    """W: float32 [N, K] (K % 128 == 0) -> (q int8 [N, K], s float16 [N, K/128])."""
    W = np.asarray(W, dtype=np.float32)
    N, K = W.shape
    if K % GROUP:
        raise ValueError("K must be a multiple of 128")
    if not np.isfinite(W).all():
        raise NonFiniteError("non-finite weight")
    Wg = W.reshape(N, K // GROUP, GROUP)
    amax = np.abs(Wg).max(axis=2)                       # binary32
    s32 = amax / np.float32(7.0)                        # one binary32 division
    with np.errstate(over="ignore"):
        s16 = s32.astype(np.float16)                    # stored scale, RN-even
    if not np.isfinite(s16).all():
        raise NonFiniteError("scale overflows FP16")
    s = s16.astype(np.float32)                          # the value that divides
    zero = s == 0                                       # all-zero group, or FP16 underflow
    divisor = np.where(zero, np.float32(1.0), s)
    r = np.rint(Wg / divisor[:, :, None])               # binary32 divide, half-to-even
    q = np.clip(r, -8, 7).astype(np.int8)
    q[zero] = 0
    s16 = np.where(zero, np.float16(0), s16)
    return q.reshape(N, K), s16


def dequantize_g128(q, s, dtype=np.float64):
    """W^ = s * q (Eq. 3), exact in binary32 and binary64 (11-bit x 4-bit product)."""
    q = np.asarray(q)
    N, K = q.shape
    sw = np.asarray(s).astype(dtype)
    return (q.reshape(N, K // GROUP, GROUP).astype(dtype) * sw[:, :, None]).reshape(N, K)
