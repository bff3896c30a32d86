"""The C-ABI library builds, loads without a GPU and exports every function include/surelock.h declares."""
import ctypes
import os
import re

import pytest

from paper_2602_06412_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "surelock.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(surelock_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    lib_path = B.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in surelock.h but not exported"


def test_host_side_argument_checks_need_no_gpu():
    lib = ctypes.CDLL(B.build())
    lib.surelock_strerror.restype = ctypes.c_char_p
    assert lib.surelock_strerror(0) == b"ok"
    assert b"invalid" in lib.surelock_strerror(-1)
    # null pointers and bad sizes are rejected before any CUDA call
    assert lib.surelock_init(None, None, None, 4, 1, None) == -1
    assert lib.surelock_reset(None) == -1
    assert lib.surelock_step(None, None, None, None, ctypes.c_float(1e-3), None) == -1
    assert lib.surelock_compact(None, 1, 1, None, None, None, None, None, None, None) == -1
    lib.surelock_compact_scratch_bytes.restype = ctypes.c_size_t
    lib.surelock_compact_scratch_bytes.argtypes = [ctypes.c_int64]
    assert lib.surelock_compact_scratch_bytes(1) >= 24
    assert lib.surelock_compact_scratch_bytes(1 << 26) >= 8 * ((1 << 26) // 4096)


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2602_06412_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(binding.SurelockError):
        binding.lib()
