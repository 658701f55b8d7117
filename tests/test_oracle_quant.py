"""Pins for the oracle's quantiser, packer and BF16 helpers (no GPU)."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import bf16, layout, quant

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bf16_weights(shape, seed, std=0.02):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * std).to(torch.bfloat16).float().numpy()


def read_golden(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append(line.split())
    return rows


# ---------------------------------------------------------------- Eq. 3: worked example
def test_hand_placed_ties_and_zero_group():
    rows = read_golden("quant_ties.txt")
    W = np.zeros((1, 256), dtype=np.float32)
    s = 2.0 ** -6
    for k, w_over_s, _ in rows:
        W[0, int(k)] = float(w_over_s) * s
    q, sc = quant.quantize_g128(W)
    assert float(sc[0, 0]) == s and float(sc[0, 1]) == 0.0
    for k, _, expect in rows:
        assert int(q[0, int(k)]) == int(expect), k
    assert not q[0, 128:].any()                      # zero group: q = 0, s = 0


def test_brute_force_exact_rational():
    """Eq. 3 in exact rational arithmetic on groups whose scale is exactly representable."""
    rng = np.random.default_rng(5)
    W = np.zeros((2, 256), dtype=np.float32)
    for r in range(2):
        for g in range(2):
            e = -3 - 2 * r - g
            vals = rng.integers(-28, 29, size=128) * 2.0 ** (e - 2)   # multiples of s/4: many ties
            vals[rng.integers(128)] = 7 * 2.0 ** e                    # absmax = 7 * 2^e -> s = 2^e
            W[r, 128 * g:128 * g + 128] = vals
    assert np.array_equal(bf16.bits_to_float(bf16.float_to_bits(W)), W)   # inputs are BF16 values
    q, sc = quant.quantize_g128(W)
    for r in range(2):
        for g in range(2):
            grp = [Fraction(float(x)) for x in W[r, 128 * g:128 * g + 128]]
            s = max(abs(x) for x in grp) / 7
            assert Fraction(float(sc[r, g])) == s
            for j, x in enumerate(grp):
                expect = max(-8, min(7, round(x / s)))                 # round(Fraction) is half-even
                assert int(q[r, 128 * g + j]) == expect


# ---------------------------------------------------------------- Eq. 3: invariants
@pytest.fixture(scope="module")
def wq():
    W = bf16_weights((64, 512), 11)
    W[3, 128:256] = 0.0
    W[5, :128] = 0.0
    W[5, 7] = 0.0123
    W = torch.tensor(W).to(torch.bfloat16).float().numpy()
    q, s = quant.quantize_g128(W)
    return W, q, s


def test_code_range_and_extreme(wq):
    W, q, s = wq
    assert q.min() >= -7 and q.max() <= 7            # clip to -8 never fires with s = absmax/7
    qa = np.abs(q.reshape(64, 4, 128)).max(axis=2)
    nz = s.astype(np.float32) != 0
    assert (qa[nz] == 7).all() and (qa[~nz] == 0).all()
    assert s[3, 1] == 0 and not q[3, 128:256].any()
    assert abs(int(q[5, 7])) == 7 and np.count_nonzero(q[5, :128]) == 1   # one-nonzero group


def test_round_trip_bound(wq):
    W, q, s = wq
    What = quant.dequantize_g128(q, s)
    bound = 0.5 * np.repeat(s.astype(np.float64), 128, axis=1)
    assert (np.abs(W.astype(np.float64) - What) <= bound * (1 + 1e-6)).all()


def test_idempotent_sign_and_scale(wq):
    W, q, s = wq
    What = quant.dequantize_g128(q, s, dtype=np.float32)
    q2, s2 = quant.quantize_g128(What)
    assert np.array_equal(q2, q) and np.array_equal(s2, s)
    qn, sn = quant.quantize_g128(-W)
    assert np.array_equal(qn, -q) and np.array_equal(sn, s)
    qd, sd = quant.quantize_g128(2 * W)
    assert np.array_equal(qd, q) and np.array_equal(sd.astype(np.float32), 2 * s.astype(np.float32))


def test_dequant_matches_library_product(wq):
    _, q, s = wq
    a = quant.dequantize_g128(q, s)
    b = (torch.tensor(q.astype(np.float64)).reshape(64, 4, 128)
         * torch.tensor(s.astype(np.float64))[:, :, None]).reshape(64, 512).numpy()
    assert np.array_equal(a, b)


def test_rejects_non_finite_and_bad_shape():
    W = np.zeros((16, 128), dtype=np.float32)
    W[0, 0] = np.inf
    with pytest.raises(quant.NonFiniteError):
        quant.quantize_g128(W)
    W[0, 0] = 3e38                                   # absmax/7 overflows FP16
    with pytest.raises(quant.NonFiniteError):
        quant.quantize_g128(W)
    with pytest.raises(ValueError):
        quant.quantize_g128(np.zeros((16, 100), dtype=np.float32))


def test_fp16_underflow_is_zero_group():
    W = np.zeros((16, 128), dtype=np.float32)
    W[0, 0] = 2.0 ** -30                             # absmax/7 rounds to FP16 zero
    q, s = quant.quantize_g128(W)
    assert s[0, 0] == 0 and not q.any()


# ---------------------------------------------------------------- Eq. 4 and the paper's sizes
def test_packed_size_against_paper():
    gold = {r[0]: r[1:] for r in read_golden("paper_numbers.txt") if r[0] != "table1"}
    H, I = int(gold["d_model"][0]), int(gold["d_ff"][0])
    E, L = int(gold["experts"][0]), int(gold["layers"][0])
    per_expert = layout.packed_bytes(H, I)
    assert per_expert == 3244032
    assert per_expert == 3 * I * H * (4 / 8 + 16 / (128 * 8))            # Eq. 4
    assert round(3 * I * H * E * L / 1e9, 2) == float(gold["routed_expert_params_billion"][0])
    assert round(per_expert * E * L / 2 ** 30, 2) == float(gold["packed_pool_gib"][0])
    assert layout.packed_bytes(256, 128) == 50688


def test_table1_traffic_is_one_packed_expert_per_miss():
    """Table 1: H2D per request ~= lookups * (1 - hit rate) * bytes of one packed expert."""
    rows = [r for r in read_golden("paper_numbers.txt") if r[0] == "table1"]
    per_expert = layout.packed_bytes(2048, 1024)
    for _, slots, hit, gib in rows:
        lookups = 8 * 16 * 128                       # top-k * layers * decoded tokens
        est = lookups * (1 - float(hit) / 100) * per_expert / 2 ** 30
        assert abs(est - float(gib)) / float(gib) < 0.02, slots


# ---------------------------------------------------------------- layout
def test_pack_unpack_round_trip_and_size():
    W = bf16_weights((32, 256), 3)
    q, s = quant.quantize_g128(W)
    blob = layout.pack_matrix(q, s)
    assert blob.size == 32 * 256 * 33 // 64
    q2, s2 = layout.unpack_matrix(blob, 32, 256)
    assert np.array_equal(q2, q) and np.array_equal(s2, s)


def test_layout_by_hand_single_code():
    """One non-zero code: find its byte and nibble from the written layout rule."""
    q = np.zeros((32, 256), dtype=np.int8)
    s = np.zeros((32, 2), dtype=np.float16)
    row, k = 16 + 11, 128 + 64 + 32 + 8 * 2 + 5      # panel 1, block 1, h=1, word 2|1, c=2, t=5
    q[row, k] = -3
    s[row, 1] = 0.5
    blob = layout.pack_matrix(q, s)
    base = (1 * 2 + 1) * 1056                        # block (p=1, kb=1)
    qq, r = 11 % 8, 11 // 8
    chunk = 32 * 1 + 4 * qq + 2
    word = 2 * 1 + r                                 # second 32-wide set, row q+8
    nib = (5 >> 1) + 4 * (5 & 1)
    byte = base + 16 * chunk + 4 * word + nib // 2
    expect = np.full(blob.size, 0x88, dtype=np.uint8)    # code 0 is stored as 8
    for b in range(blob.size // 1056):
        expect[b * 1056 + 1024:(b + 1) * 1056] = 0
    val = (-3 + 8)
    expect[byte] = (0x80 | val) if nib % 2 == 0 else ((val << 4) | 0x08)
    sb = np.array([0.5], dtype="<f2").view(np.uint8)
    off = base + 1024 + 2 * (2 * qq + r)
    expect[off:off + 2] = sb
    assert np.array_equal(blob, expect)


def test_layout_by_hand_second_code_first_half_word_zero_even_t():
    """A second hand-placed code on the other branch of every rule: first half (h = 0), word 0 (first 32-wide set,
    row q), an even t (low nibbles 0-3), panel 0, block 0, plus a neighbour with odd t in the same word: the byte
    offsets and nibbles below are worked out from the written layout, not from the index tables."""
    q = np.zeros((16, 128), dtype=np.int8)
    s = np.zeros((16, 1), dtype=np.float16)
    # row 5 (q = 5, r = 0), k = 8*3 + 4: h = 0, set 0, c = 3, t = 4 -> chunk 4*5 + 3 = 23, word 0, nibble (4 >> 1) = 2
    q[5, 28] = 7
    # same word, t = 1 (k = 25): nibble (1 >> 1) + 4 = 4
    q[5, 25] = -8
    s[5, 0] = 2.0
    blob = layout.pack_matrix(q, s)
    expect = np.full(1056, 0x88, dtype=np.uint8)
    expect[1024:] = 0
    word_off = 16 * 23 + 4 * 0
    expect[word_off + 1] = 0x80 | (7 + 8)            # nibble 2 = low nibble of byte 1; its high nibble keeps code 0
    expect[word_off + 2] = 0x80 | (-8 + 8)           # nibble 4 = low nibble of byte 2
    expect[1024 + 2 * (2 * 5 + 0):1024 + 2 * (2 * 5 + 0) + 2] = np.array([2.0], dtype="<f2").view(np.uint8)
    assert np.array_equal(blob, expect)
    # and the whole word as the kernels read it: eight codes at shifts 0, 16, 4, 20, 8, 24, 12, 28 for t = 0..7
    word = int(blob[word_off:word_off + 4].view("<u4")[0])
    codes = [((word >> (4 * ((t >> 1) + 4 * (t & 1)))) & 0xF) - 8 for t in range(8)]
    assert codes == [0, -8, 0, 0, 7, 0, 0, 0]


def test_expert_blob_order_and_determinism():
    wg, wu, wd = bf16_weights((128, 256), 1), bf16_weights((128, 256), 2), bf16_weights((256, 128), 3)
    blob = layout.pack_expert(wg, wu, wd)
    assert blob.size == layout.packed_bytes(256, 128)
    assert np.array_equal(blob, layout.pack_expert(wg, wu, wd))
    n13 = 2 * 128 * 256 * 33 // 64
    q13, s13 = layout.unpack_matrix(blob[:n13], 256, 256)
    qg, sg = quant.quantize_g128(wg)
    qu, su = quant.quantize_g128(wu)
    for p in range(8):                                # panels alternate gate, up
        assert np.array_equal(q13[32 * p:32 * p + 16], qg[16 * p:16 * p + 16])
        assert np.array_equal(q13[32 * p + 16:32 * p + 32], qu[16 * p:16 * p + 16])
        assert np.array_equal(s13[32 * p + 16:32 * p + 32], su[16 * p:16 * p + 16])
    qd, sd = layout.unpack_matrix(blob[n13:], 256, 128)
    qd0, sd0 = quant.quantize_g128(wd)
    assert np.array_equal(qd, qd0) and np.array_equal(sd, sd0)


# ---------------------------------------------------------------- BF16 helpers vs the library cast
def test_bf16_rounding_matches_library_cast():
    g = torch.Generator().manual_seed(9)
    x = torch.randn(20000, generator=g, dtype=torch.float32) * 37.0
    ties = torch.tensor([1.00390625, 1.01171875, -1.00390625, 3.0e-39, 65280.0 * 2.0 ** 112])
    x = torch.cat([x, ties])
    lib = x.to(torch.bfloat16).float().numpy().astype(np.float64)
    mine = bf16.round_to_bf16(x.numpy().astype(np.float64))
    assert np.array_equal(mine, lib)
    bits = bf16.float_to_bits(lib.astype(np.float32))
    assert np.array_equal(bf16.bits_to_float(bits), lib.astype(np.float32))
    assert np.array_equal(bits.view(np.int16), x.to(torch.bfloat16).view(torch.int16).numpy())
