"""The C-ABI library builds for sm_100a, loads without a GPU and exports every declared symbol."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2608_15383_b200 import build
    return build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "exmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(exmoe_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_symbols()
    for must in ("exmoe_pack", "exmoe_packed_bytes", "exmoe_cache_create", "exmoe_moe_forward",
                 "exmoe_cache_workspace_bytes", "exmoe_cache_destroy", "exmoe_status", "exmoe_strerror"):
        assert must in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_covers_every_declared_symbol(libpath):
    from paper_2608_15383_b200 import binding
    assert sorted(binding._SIGNATURES) == declared_symbols()
    binding.lib()


def test_host_only_calls(libpath):
    """Entry points that touch no device: size model (Eq. 4), argument checks, error strings."""
    from paper_2608_15383_b200 import binding, synth
    assert binding.exmoe_packed_bytes(synth.OLMOE) == 3244032
    assert binding.exmoe_packed_bytes(synth.TINY) == 50688
    slot_total, ws = binding.exmoe_cache_workspace_bytes(synth.OLMOE, 16, 16, 64)
    assert slot_total == 16 * 16 * 3244032
    assert ws >= 64 * 8 * (1024 * 2 + 2048 * 4)
    for bad in (synth.Shape(200, 128, 4, 2), synth.Shape(256, 128, 4, 8), synth.Shape(256, 128, 4, 2, group_size=64)):
        with pytest.raises(binding.ExmoeError) as ei:
            binding.exmoe_packed_bytes(bad)
        assert ei.value.code == binding.EXMOE_ERR_SHAPE
    with pytest.raises(binding.ExmoeError):
        binding.exmoe_cache_workspace_bytes(synth.OLMOE, 1, 4, 16)      # C < k
    assert "pinned" in binding.strerror(binding.EXMOE_ERR_NOT_PINNED)
    assert binding.exmoe_launch_count() == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2608_15383_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        binding.lib()
