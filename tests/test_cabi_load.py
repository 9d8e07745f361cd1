"""The C-ABI library builds, loads without a GPU, and exports every symbol
that include/shareprefill.h declares.  No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2505_19578_b200 import binding, build
    build.build()
    return binding.load()


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            txt = open(os.path.join(inc, f)).read()
            txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
            names |= set(re.findall(r"\b(sp_[a-z0-9_]+)\s*\(", txt))
    return names


def test_every_declared_symbol_is_exported(lib):
    from paper_2505_19578_b200 import binding
    names = _declared()
    assert {"sp_prefill_attn", "sp_dense_pivot_attn", "sp_block_mask_from_importance",
            "sp_block_sparse_attn"} <= names
    assert names == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_host_only_calls(lib):
    from paper_2505_19578_b200 import binding
    assert binding.error_string(0) == "ok"
    assert "timed out" in binding.error_string(binding.SP_ERR_TIMEOUT)
    b = binding.workspace_bytes(131072, 32, 8, 128, 128, 4)
    nb = 1024
    # importance + mask + counts + lists, and per-tile statistics: one region of 2 * nb * 128 floats per
    # persistent CTA (at most one per SM) instead of one float per row of every causal tile of every pivot
    assert b >= 4 * nb * nb * (4 + 1 + 4) + 2 * nb * 128 * 4
    assert b < 256 << 20
    # the one-row-block kernel (other shapes) keeps the per-tile layout
    b64 = binding.workspace_bytes(8192, 8, 8, 64, 64, 2)
    assert b64 >= 2 * 128 * 129 // 2 * 64 * 4
    wa, wl = binding.workspace_bytes_patterns(131072, 32, 8, 128, 128, 6)
    assert wa > 32 * nb * nb * 5 and wl > 0            # masks and lists of every head's own pattern
    assert binding.workspace_bytes_patterns(131072, 32, 8, 128, 128, 6, True)[0] > wa - (200 << 20)
    out = ctypes.c_size_t()
    assert lib.sp_workspace_bytes(1000, 32, 8, 128, 128, 4, ctypes.byref(out)) == binding.SP_ERR_UNSUPPORTED
    assert lib.sp_workspace_bytes(4096, 32, 8, 96, 128, 4, ctypes.byref(out)) == binding.SP_ERR_UNSUPPORTED
    assert lib.sp_workspace_bytes(4096, 32, 8, 128, 128, 4, None) == binding.SP_ERR_INVALID_ARG


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2505_19578_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()
