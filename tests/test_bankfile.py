"""Flat bank file: what is written is the packed byte image, what is read back is identical (no GPU needed: the
bank of this test comes from the oracle's packer)."""
import numpy as np
import pytest
import torch

from oracle import layout as olayout
from paper_2608_15383_b200 import bankfile, synth


def make_bank(shape, seed):
    wg, wu, wd = synth.expert_weights(shape, seed)
    rows = [olayout.pack_expert(wg[e].float().numpy(), wu[e].float().numpy(), wd[e].float().numpy())
            for e in range(shape.num_experts)]
    return np.stack(rows)


def test_round_trip_and_header(tmp_path):
    s = synth.TINY
    bank = make_bank(s, seed=3)
    assert bank.shape == (8, 50688)
    path = tmp_path / "layer0.bank"
    bankfile.save_bank(path, s, bank)
    assert path.stat().st_size == 64 + 8 * 50688                      # header + Eq. 4 bytes, nothing else
    h, got = bankfile.load_bank(path, shape=s, pin=False)
    assert h == {"d_model": 256, "d_ff": 128, "num_experts": 8, "top_k": 2, "group_size": 128, "bytes_per_expert": 50688}
    assert got.dtype == torch.uint8 and np.array_equal(got.numpy(), bank)
    raw = path.read_bytes()
    assert raw[:8] == b"EXMOEBNK" and raw[64:64 + 50688] == bank[0].tobytes()   # payload = the byte image itself


def test_rejects_wrong_geometry_truncation_and_foreign_files(tmp_path):
    s = synth.TINY
    path = tmp_path / "layer0.bank"
    bankfile.save_bank(path, s, make_bank(s, seed=4))
    with pytest.raises(bankfile.BankFileError):
        bankfile.load_bank(path, shape=synth.MID, pin=False)
    data = path.read_bytes()
    (tmp_path / "short.bank").write_bytes(data[:-100])
    with pytest.raises(bankfile.BankFileError):
        bankfile.load_bank(tmp_path / "short.bank", pin=False)
    (tmp_path / "other.bin").write_bytes(b"not a bank" * 20)
    with pytest.raises(bankfile.BankFileError):
        bankfile.read_header(tmp_path / "other.bin")
    with pytest.raises(bankfile.BankFileError):
        bankfile.save_bank(tmp_path / "bad.bank", s, np.zeros((3, 10), dtype=np.uint8))


@pytest.mark.gpu
def test_gpu_packed_bank_survives_the_file_and_serves_the_layer(tmp_path):
    from paper_2608_15383_b200 import binding, build
    import helpers
    build.build()
    s = synth.MID
    ora, bank = helpers.make_layer(s, seed=77)
    path = tmp_path / "mid.bank"
    bankfile.save_bank(path, s, bank)
    h, back = bankfile.load_bank(path, shape=s)
    assert back.is_pinned() and torch.equal(back, bank)
    assert np.array_equal(back[5].numpy(), ora.packed(5))              # the file holds the oracle's byte image too
    hidden, ids, p = helpers.routed_inputs(s, 9, seed=123)
    a = binding.Cache(s, [bank], 8, max_tokens=16)
    b = binding.Cache(s, [back], 8, max_tokens=16)
    ya = a.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).clone()
    yb = b.forward(0, hidden.cuda(), ids.cuda(), p.cuda()).clone()
    torch.cuda.synchronize()
    assert torch.equal(ya.view(torch.int16), yb.view(torch.int16))
    y, o = ora.forward(hidden, ids, p)
    helpers.check_output(yb, y, o, "bank file")
    a.status(); b.status()
