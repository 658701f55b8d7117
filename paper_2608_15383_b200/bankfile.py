"""Flat file format of a packed expert bank (Section 3.2: "quantization and packing happen offline once per
checkpoint conversion"; Section 3.3: the host pool and the GPU slots hold the same representation).

One file per sparse layer:

    offset  size  field
    0       8     magic  b"EXMOEBNK"
    8       4     format version (little-endian uint32) = 1
    12      20    d_model, d_ff, num_experts, top_k, group_size (five little-endian int32)
    32      8     bytes_per_expert (little-endian uint64; Eq. 4: 3,244,032 for the OLMoE geometry)
    40      24    reserved, zero
    64      E * bytes_per_expert   the packed experts, expert e at 64 + e * bytes_per_expert, exactly as
                                   exmoe_pack wrote them

The payload is the byte image the library reads, so loading is one read into pinned memory: no conversion.
"""
import struct

import numpy as np
import torch

MAGIC = b"EXMOEBNK"
VERSION = 1
HEADER_BYTES = 64


class BankFileError(ValueError):
    pass


def save_bank(path, shape, bank):
    """bank: uint8 tensor or array [E, bytes_per_expert] (e.g. from binding.pack_bank)."""
    arr = bank.cpu().numpy() if isinstance(bank, torch.Tensor) else np.asarray(bank)
    if arr.dtype != np.uint8 or arr.ndim != 2 or arr.shape[0] != shape.num_experts:
        raise BankFileError("bank must be uint8 [num_experts, bytes_per_expert]")
    hdr = MAGIC + struct.pack("<I5iQ", VERSION, shape.d_model, shape.d_ff, shape.num_experts, shape.top_k,
                              getattr(shape, "group_size", 128), arr.shape[1])
    hdr += b"\0" * (HEADER_BYTES - len(hdr))
    with open(path, "wb") as f:
        f.write(hdr)
        f.write(np.ascontiguousarray(arr).tobytes())


def read_header(path):
    with open(path, "rb") as f:
        hdr = f.read(HEADER_BYTES)
    if len(hdr) != HEADER_BYTES or hdr[:8] != MAGIC:
        raise BankFileError(f"{path}: not an expert bank file")
    version, d_model, d_ff, E, k, g, bpe = struct.unpack("<I5iQ", hdr[8:40])
    if version != VERSION:
        raise BankFileError(f"{path}: format version {version}, this reader knows {VERSION}")
    return {"d_model": d_model, "d_ff": d_ff, "num_experts": E, "top_k": k, "group_size": g, "bytes_per_expert": bpe}


def load_bank(path, shape=None, pin=True):
    """Returns (header dict, uint8 tensor [E, bytes_per_expert], pinned when a CUDA runtime is present and pin=True).
    If `shape` is given the file must have been written for the same geometry."""
    h = read_header(path)
    if shape is not None:
        want = (shape.d_model, shape.d_ff, shape.num_experts, getattr(shape, "group_size", 128))
        got = (h["d_model"], h["d_ff"], h["num_experts"], h["group_size"])
        if want != got:
            raise BankFileError(f"{path}: geometry {got} does not match {want}")
    E, bpe = h["num_experts"], h["bytes_per_expert"]
    bank = torch.empty((E, bpe), dtype=torch.uint8)
    if pin and torch.cuda.is_available():
        bank = bank.pin_memory()
    with open(path, "rb") as f:
        f.seek(HEADER_BYTES)
        n = f.readinto(memoryview(bank.numpy()).cast("B"))
    if n != E * bpe:
        raise BankFileError(f"{path}: truncated ({n} of {E * bpe} payload bytes)")
    return h, bank
