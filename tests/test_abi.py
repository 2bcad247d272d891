"""The C-ABI library builds, loads and exports every symbol the header declares
(no compute calls: this runs without a GPU)."""
import ctypes
import os
import re

import pytest

import paper_2607_18002_b200 as moe
from paper_2607_18002_b200 import build as moe_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    return moe_build.build()


def test_header_symbols_are_exported(built):
    text = open(os.path.join(ROOT, "include", "moe_apk.h")).read()
    declared = set(re.findall(r"\b(moe_[a-z_]+)\s*\(", text))
    assert declared == set(moe.EXPORTS)
    lib = ctypes.CDLL(built)
    for name in declared:
        assert hasattr(lib, name), name


def test_host_side_validation_needs_no_gpu(built):
    cfg = moe.moe_config_t(256, 8, 3072, 1536, moe.MOE_DTYPE_BF16, 8192, 2, 0, 0, 0)
    n = moe.moe_workspace_bytes(cfg)
    rows = 8192 * 8
    assert n > rows * (3072 + 1536) * 2 * 2                      # A and D scratch of both slots
    assert moe.strerror(moe.MOE_ETIMEOUT) == "a device-side wait ran out"
    for bad in (dict(hidden=3000), dict(inter=100), dict(n_experts=0), dict(top_k=0),
                dict(max_ops=99), dict(max_tokens_per_op=0)):
        c = moe.moe_config_t(256, 8, 3072, 1536, 0, 8192, 2, 0, 0, 0)
        for k, v in bad.items():
            setattr(c, k, v)
        with pytest.raises(moe.MoeError) as ei:
            moe.moe_workspace_bytes(c)
        assert ei.value.code == moe.MOE_EINVAL


def test_struct_layouts_match_the_header(built):
    assert ctypes.sizeof(moe.moe_config_t) == 40
    assert ctypes.sizeof(moe.moe_op_t) == 8 + 15 * 8 + 8
    assert ctypes.sizeof(moe.moe_tile_rec_t) == 32 and moe.TILE_REC_DTYPE.itemsize == 32


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(moe, "_lib", None)
    monkeypatch.setattr(moe, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        moe.lib()
