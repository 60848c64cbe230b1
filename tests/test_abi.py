"""The C-ABI library loads and exports every symbol the header declares (no compute, no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sfs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sfs_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_10848_b200 import binding
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 10
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, f"declared in include/sfs.h but not exported: {missing}"


def test_status_strings_and_host_side_validation():
    from paper_2506_10848_b200 import binding as sfs
    assert sfs.sfs_status_string(0) == "ok"
    assert "missing" in sfs.sfs_status_string(sfs.ERR_MISSING_ROW)
    # argument errors are caught on the host before any CUDA call
    p = sfs.Params.default(w_hist=99)
    rc = sfs.lib().sfs_state_init(ctypes.c_void_p(16), 1, 4, ctypes.byref(p), None)
    assert rc == sfs.ERR_INVALID_ARG and "w_hist" in sfs.sfs_last_error()
    rc = sfs.lib().sfs_row_stats(None, 0, 8, ctypes.c_int64(8), None, 1, None, None, None, None)
    assert rc == sfs.ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2506_10848_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libsfs.so"))
    with pytest.raises(FileNotFoundError):
        binding.lib()
