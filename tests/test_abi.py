"""The C-ABI library loads and exports every symbol the headers under include/ declare.

No kernel is launched here; the host-side pure functions are compared with the
oracle's own statement of the same formulas.
"""
import ctypes
import os
import re

import pytest

import oracle
from paper_1805_08768_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared_functions():
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not header.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(sbc_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert "sbc_encode" in names and "sbc_decode_accumulate" in names and "sbc_stream_bytes" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared under include/ but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_library_is_in_tree_and_has_no_oracle_dependency():
    assert os.path.dirname(binding.LIB_PATH) == os.path.join(ROOT, "paper_1805_08768_b200")
    blob = open(binding.LIB_PATH, "rb").read()
    assert b"sbc_oracle" not in blob


@pytest.mark.parametrize("p", [0.3, 0.1, 0.05, 0.01, 0.003, 0.001, 3e-4, 1e-4, 1e-5])
def test_host_scalars_agree_with_the_oracle(lib, p):
    assert binding.sbc_golomb_b(p) == oracle.golomb_b(p)
    for n in (1, 64, 1000, 4097, 2**20, 25557032, 2**30, 2**31 - 1):
        assert binding.sbc_kept_count(n, p) == oracle.kept_count(n, p)
        assert binding.sbc_stream_bytes(n, p) == oracle.stream_bytes(n, p)
        assert binding.sbc_workspace_bytes(n, p) > 0
    b = binding.sbc_golomb_b(p)
    assert binding.sbc_mean_position_bits(p, b) == pytest.approx(oracle.mean_position_bits(p, b), rel=1e-14)


def test_host_functions_reject_bad_arguments(lib):
    assert binding.sbc_kept_count(0, 0.01) == 0
    assert binding.sbc_kept_count(10, 0.0) == 0
    assert binding.sbc_golomb_b(1.0) == -1
    assert binding.sbc_stream_bytes(2**31, 0.01) == 0
    assert binding.sbc_stream_bytes(100, 1e-12) == 0          # b* above 30
    assert binding.sbc_workspace_bytes(-5, 0.01) == 0
    # pointer checks happen before any CUDA call
    rc = lib.sbc_encode(None, None, 10, 0.1, None, 0, None, None, 0, None)
    assert rc == binding.SBC_EINVAL
    rc = lib.sbc_decode_accumulate(None, 1, None, 10, None, None)
    assert rc == binding.SBC_EINVAL


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.sbc_golomb_b(0.01)
