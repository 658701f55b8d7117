"""Packed byte layout of one expert (oracle; test infrastructure).

The paper stores one representation of an expert everywhere: packed int4 codes
plus FP16 scales, gate and up concatenated, down separate (Section 3.2), the same
bytes in the pinned host pool and in a GPU slot (Section 3.3), with the size
model of Eq. 4: bytes = params * (4/8 + 16/(128*8)).  The paper's byte order is
that of a library kernel for other hardware; this build defines its own order,
written out below.  This file is the independent statement of that order that
the GPU packer is compared against byte for byte.

Layout of a matrix W[N, K] (N % 16 == 0, K % 128 == 0)
------------------------------------------------------
  * rows are cut into PANELS of 16 rows, K into BLOCKS of 128 (one scale group);
    block (p, kb) starts at byte ((p * K/128) + kb) * 1056.
  * a block is 1024 bytes of codes followed by 32 bytes of scales.
  * codes: 64 CHUNKS of 16 bytes, chunk index = 32*h + 4*q + c with
        h in {0,1}  the 64-wide half of the block,
        q in 0..7   row within the half-panel,
        c in 0..3   octet selector.
    A chunk is four little-endian 32-bit words:
        word 0: row q,   k = 64h + 8c + t        (t = 0..7)
        word 1: row q+8, k = 64h + 8c + t
        word 2: row q,   k = 64h + 32 + 8c + t
        word 3: row q+8, k = 64h + 32 + 8c + t
    Inside a word the code for offset t sits in nibble (t >> 1) + 4*(t & 1)
    (nibble n = bits 4n..4n+3).  A code is stored offset-binary: u = q + 8.
  * scales: 16 FP16 values, index 2*q + r for row q + 8*r  (r in {0,1}).

Layout of an expert
-------------------
  [ W13 | W2 ] with W13 the 2I x H matrix whose 16-row panels alternate
  gate panel 0, up panel 0, gate panel 1, up panel 1, ... and W2 the H x I down
  projection.  Total = 3*I*H * 0.515625 bytes (Eq. 4).
"""
import numpy as np

from .quant import quantize_g128

BLOCK_BYTES = 1056
CODE_BYTES = 1024


def packed_bytes(d_model, d_ff):
    """Bytes of one packed expert; Eq. 4 with P_expert = 3 * d_ff * d_model."""
    params = 3 * d_ff * d_model
    assert (params * 33) % 64 == 0
    return params * 33 // 64          # 4/8 + 16/(128*8) = 33/64


def _index_tables():
    """(row, k, shift) of every code inside a block, in stored order [h][q][c][word][t]."""
    row = np.zeros((2, 8, 4, 4, 8), dtype=np.int64)
    col = np.zeros((2, 8, 4, 4, 8), dtype=np.int64)
    shift = np.zeros((2, 8, 4, 4, 8), dtype=np.uint32)
    for h in range(2):
        for qq in range(8):
            for c in range(4):
                for w in range(4):
                    for t in range(8):
                        row[h, qq, c, w, t] = qq + 8 * (w & 1)
                        col[h, qq, c, w, t] = 64 * h + 32 * (w >> 1) + 8 * c + t
                        shift[h, qq, c, w, t] = 4 * ((t >> 1) + 4 * (t & 1))
    return row, col, shift


_ROW, _COL, _SHIFT = _index_tables()
_SROW = np.array([qq + 8 * r for qq in range(8) for r in range(2)])   # scale index 2q+r -> row


def pack_matrix(q, s):
    """q int8 [N, K] in [-8, 7], s float16 [N, K/128] -> uint8 [N/16 * K/128 * 1056]."""
    q = np.asarray(q, dtype=np.int8)
    s = np.asarray(s, dtype=np.float16)
    N, K = q.shape
    assert N % 16 == 0 and K % 128 == 0
    P, KB = N // 16, K // 128
    u = (q.astype(np.int32) + 8).astype(np.uint32)              # offset-binary code
    blocks = u.reshape(P, 16, KB, 128).transpose(0, 2, 1, 3)    # [p][kb][row][k]
    codes = blocks[:, :, _ROW, _COL]                            # [p][kb][h][q][c][word][t]
    words = np.bitwise_or.reduce(codes << _SHIFT, axis=-1)      # [p][kb][h][q][c][word]
    out = np.zeros((P, KB, BLOCK_BYTES), dtype=np.uint8)
    out[:, :, :CODE_BYTES] = np.ascontiguousarray(words.reshape(P, KB, 256).astype("<u4")).view(np.uint8)
    sc = s.reshape(P, 16, KB).transpose(0, 2, 1)[:, :, _SROW]   # [p][kb][2q+r]
    out[:, :, CODE_BYTES:] = np.ascontiguousarray(sc.astype("<f2")).view(np.uint8)
    return out.reshape(-1)


def interleave_gate_up(gate, up):
    """Rows of W13: 16-row panels alternating gate, up (first axis of any array)."""
    I = gate.shape[0]
    assert I % 16 == 0 and gate.shape == up.shape
    g = gate.reshape(I // 16, 16, *gate.shape[1:])
    u = up.reshape(I // 16, 16, *up.shape[1:])
    return np.stack([g, u], axis=1).reshape(2 * I, *gate.shape[1:])


def pack_expert(w_gate, w_up, w_down):
    """float32 BF16-valued W_g[I,H], W_u[I,H], W_d[H,I] -> packed uint8 blob.

    Quantises each matrix with Eq. 3 and lays the codes and scales out as above.
    """
    qg, sg = quantize_g128(w_gate)
    qu, su = quantize_g128(w_up)
    qd, sd = quantize_g128(w_down)
    w13 = pack_matrix(interleave_gate_up(qg, qu), interleave_gate_up(sg, su))
    w2 = pack_matrix(qd, sd)
    return np.concatenate([w13, w2])


def unpack_matrix(blob, N, K):
    """Inverse of pack_matrix (used by tests to read a packed blob or a GPU slot back)."""
    P, KB = N // 16, K // 128
    b = np.asarray(blob, dtype=np.uint8).reshape(P, KB, BLOCK_BYTES)
    words = np.ascontiguousarray(b[:, :, :CODE_BYTES]).view("<u4").reshape(P, KB, 2, 8, 4, 4)
    codes = (words[..., None] >> _SHIFT) & np.uint32(0xF)        # [p][kb][h][q][c][word][t]
    blocks = np.zeros((P, KB, 16, 128), dtype=np.int8)
    blocks[:, :, _ROW, _COL] = codes.astype(np.int8) - 8
    q = blocks.transpose(0, 2, 1, 3).reshape(N, K)
    sc = np.ascontiguousarray(b[:, :, CODE_BYTES:]).view("<f2").reshape(P, KB, 16)
    rows = np.zeros((P, KB, 16), dtype=np.float16)
    rows[:, :, _SROW] = sc
    s = rows.transpose(0, 2, 1).reshape(N, KB)
    return q, s
