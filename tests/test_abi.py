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
    # after_op and notify_after share a word; decode_sms + layout, slab_rows + padding
    assert ctypes.sizeof(moe.moe_op_t) == 8 + 15 * 8 + 8 + 8 + 8 + 8
    assert moe.moe_op_t.notify.offset == 8 + 15 * 8 + 8 and moe.moe_op_t.notify_after.offset == 8 + 15 * 8 + 4
    assert ctypes.sizeof(moe.moe_tile_rec_t) == 32 and moe.TILE_REC_DTYPE.itemsize == 32


def test_binding_structs_match_what_a_c_compiler_makes_of_the_header(tmp_path):
    """The ctypes structs are laid out as gcc lays out the header's (sizes and a few offsets)."""
    import os, shutil, subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    src = tmp_path / "layout.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "moe_apk.h"\n'
        'int main(void) { printf("%zu %zu %zu %zu %zu %zu %zu %zu\\n", sizeof(moe_config_t), sizeof(moe_op_t),\n'
        '  offsetof(moe_op_t, y), offsetof(moe_op_t, ready), offsetof(moe_op_t, after_op),\n'
        '  offsetof(moe_op_t, notify_after), offsetof(moe_op_t, notify), sizeof(moe_tile_rec_t));\n'
        '  printf("%zu %zu %zu\\n", offsetof(moe_op_t, decode_sms), offsetof(moe_op_t, layout), offsetof(moe_op_t, slab_rows));\n'
        '  return 0; }\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", inc, "-o", str(exe), str(src)], check=True)
    got = [int(v) for v in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    o = moe.moe_op_t
    assert got == [ctypes.sizeof(moe.moe_config_t), ctypes.sizeof(o), o.y.offset, o.ready.offset, o.after_op.offset,
                   o.notify_after.offset, o.notify.offset, ctypes.sizeof(moe.moe_tile_rec_t), o.decode_sms.offset,
                   o.layout.offset, o.slab_rows.offset]


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(moe, "_lib", None)
    monkeypatch.setattr(moe, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        moe.lib()
