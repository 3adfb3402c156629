"""The C-ABI library loads on a machine without a GPU and exports every symbol that
include/moe_b200.h declares; argument errors come back as status codes.  No compute call."""

import ctypes
import os
import re
import shutil
import subprocess

import pytest

from paper_2609_07536_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "moe_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"^(?:int32_t|const char \*)\s*(\w+)\s*\(", text, flags=re.M)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert len(names) >= 14
    L = B.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(B.EXPORTS) == names


def test_structs_match_header_sizes():
    assert ctypes.sizeof(B.moe_shape) == 32
    assert ctypes.sizeof(B.moe_occupancy) == 28
    assert ctypes.sizeof(B.moe_sm_limits) == 44
    assert ctypes.sizeof(B.moe_rho) == 80
    assert ctypes.sizeof(B.moe_plan) == 56
    assert ctypes.sizeof(B.moe_status) == 16


def test_struct_layouts_match_the_compiled_header(tmp_path):
    # sizes and the offsets of the last fields as a C compiler lays the header's structs out, against the
    # ctypes mirrors the binding passes across the boundary
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    header = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "moe_b200.h")
    structs = {"moe_shape": "L", "moe_occupancy": "comp_slot_sms", "moe_sm_limits": "co_min_waves", "moe_rho": "co_order",
               "moe_plan": "co_warps", "moe_routing": "max_mtiles", "moe_status": "count"}
    src = tmp_path / "layout.c"
    lines = ['#include <stdio.h>', '#include <stddef.h>', f'#include "{header}"', 'int main(void) {']
    for name, last in structs.items():
        lines.append(f'  printf("{name} %zu %zu\\n", sizeof({name}), offsetof({name}, {last}));')
    lines += ['  return 0;', '}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run([gcc, "-std=c99", "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    seen = 0
    for line in out:
        if not line.strip():
            continue
        name, size, off = line.split()
        cls = getattr(B, name)
        assert ctypes.sizeof(cls) == int(size), name
        assert getattr(cls, structs[name]).offset == int(off), name
        seen += 1
    assert seen == len(structs)


def test_workspace_sizes_and_argument_errors():
    s = B.make_shape(256, 256, 128, 8, 2, 1, 2, 1)
    rb, yb, fb, sb = B.moe_workspace_bytes(s, 64, 64)
    max_mtiles = 512 // 64 + 8
    assert yb >= 256 * 1 * 2 * 1 * 256 * 2 and sb == 16      # token-major partials: T x L x k_tot x TP x H/L
    assert fb >= (64 + 1 * 1 * max_mtiles * 4) * 4
    assert rb >= 3 * 512 * 4 + 3 * max_mtiles * 4
    with pytest.raises(B.MoeError) as e:
        B.moe_workspace_bytes(B.make_shape(256, 250, 128, 8, 2, 1, 2, 1), 64, 64)   # H % 8
    assert e.value.code == B.MOE_ERR_SHAPE
    with pytest.raises(B.MoeError) as e:
        B.moe_workspace_bytes(B.make_shape(256, 256, 100, 8, 2, 1, 2, 1), 64, 64)   # K % 16
    assert e.value.code == B.MOE_ERR_SHAPE
    with pytest.raises(B.MoeError) as e:
        B.moe_workspace_bytes(s, 96, 64)
    assert e.value.code == B.MOE_ERR_UNSUPPORTED
    assert B.lib().moe_workspace_bytes(None, 64, 64, None, None, None, None) == B.MOE_ERR_NULL
    assert B.lib().moe_destroy(None) == B.MOE_OK
    assert B.moe_host_arena_bytes(s, 64, 64) > rb + yb + fb


def test_header_is_plain_c():
    # the boundary is a C ABI: the header has to compile as C99 on its own (no C++-isms, no torch types)
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler here")
    header = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "moe_b200.h")
    res = subprocess.run([gcc, "-std=c99", "-Wall", "-Werror", "-fsyntax-only", "-x", "c", header],
                         capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
