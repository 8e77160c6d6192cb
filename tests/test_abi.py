"""The C-ABI library builds, loads without a GPU and exports every entry point
that include/pquant.h declares; host-side argument logic is exercised (no
kernel is launched here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2602_22592_b200 import build
    build.build()
    from paper_2602_22592_b200 import binding
    return binding


def declared_symbols():
    src = open(os.path.join(ROOT, "include", "pquant.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(pq_[a-z0-9_]+)\s*\(", src)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "pq_pack_weights" in names and "pq_linear_forward" in names and "pq_linear_backward" in names
    L = lib.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in pquant.h but not exported"
    assert set(lib.EXPORTS) <= set(names)


def test_struct_layout_matches_header(lib):
    assert ctypes.sizeof(lib.pq_desc) == 32
    d = lib.make_desc(256, 512, 512, 32, 1, scale_vector=True)
    assert d.size == 32 and d.flags == lib.PQ_SCALE_VECTOR


def test_every_struct_of_the_header_has_the_same_layout_in_the_binding(lib, tmp_path):
    # the header compiled as plain C (it has to be: the boundary is a C ABI) prints size and field offsets of each struct;
    # the ctypes mirrors must agree field by field
    structs = {"pq_desc": lib.pq_desc, "pq_decode_item": lib.pq_decode_item, "pq_decode_view": lib.pq_decode_view,
               "pq_ffn_desc": lib.pq_ffn_desc, "pq_ffn_view": lib.pq_ffn_view, "pq_bwd_view": lib.pq_bwd_view}
    lines = ["#include <stdio.h>", "#include <stddef.h>", '#include "pquant.h"', "int main(void) {"]
    for name, cls in structs.items():
        lines.append(f'  printf("{name} sizeof %zu\\n", sizeof({name}));')
        for field, _ in cls._fields_:
            lines.append(f'  printf("{name} {field} %zu\\n", offsetof({name}, {field}));')
    lines += ["  return 0;", "}"]
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    import subprocess
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    seen = 0
    for line in out:
        if not line:
            continue
        name, field, value = line.split()
        cls = structs[name]
        if field == "sizeof":
            assert ctypes.sizeof(cls) == int(value), name
        else:
            assert getattr(cls, field).offset == int(value), f"{name}.{field}"
        seen += 1
    assert seen == sum(1 + len(c._fields_) for c in structs.values())


def test_status_strings(lib):
    assert lib.pq_status_string(0) == "ok"
    for s in range(-7, 0):
        assert lib.pq_status_string(s) not in ("ok", "unknown status")


def test_sizes_and_shape_checks(lib):
    d = lib.make_desc(8192, 2048, 5632, 128, 8)
    sv = lib.pq_saved_bytes(d)
    # q (int8) + xt (bf16) + xs (bf16) dominate: 5 bytes per activation element
    assert 5 * 8192 * 2048 <= sv <= 5 * 8192 * 2048 * 1.2
    assert lib.pq_workspace_bytes(d, lib.PQ_PHASE_FWD) >= sv
    assert lib.pq_workspace_bytes(d, lib.PQ_PHASE_PACK) > 0
    assert lib.pq_workspace_bytes(d, lib.PQ_PHASE_BWD) > 2 * 8192 * 5632
    for bad in (lib.make_desc(0, 64, 64), lib.make_desc(8, 100, 64), lib.make_desc(8, 64, 48),
                lib.make_desc(8, 64, 64, 12, 1), lib.make_desc(8, 64, 64, 32, 0), lib.make_desc(8, 64, 64, 32, 17)):
        assert lib.pq_saved_bytes(bad) == 0
    # the paper's gating is top-1; anything else is refused, not approximated
    assert lib.pq_saved_bytes(lib.make_desc(8, 64, 64, 32, 4, top_k=2)) == 0
    # pure 1-bit layer (attention projections): E is ignored
    assert lib.pq_saved_bytes(lib.make_desc(8, 64, 64, 0, 0)) > 0


def test_null_arguments_rejected_before_any_launch(lib):
    d = lib.make_desc(128, 64, 64)
    L = lib.lib()
    assert L.pq_pack_weights(ctypes.byref(d), None, None, None, None, None, 0, None) == lib.PQ_ERR_NULL
    assert L.pq_debug_gemm(0, 128, 128, 128, None, None, None, None) == lib.PQ_ERR_NULL


def test_launch_options_are_host_state(lib):
    # options only set process-wide switches: no device is touched, unknown ids are refused
    L = lib.lib()
    for opt in (lib.PQ_OPT_DECODE_PDL, lib.PQ_OPT_SIDE_STREAM):
        assert L.pq_set_option(opt, 0) == lib.PQ_OK
        assert L.pq_set_option(opt, 1) == lib.PQ_OK
    assert L.pq_set_option(99, 1) == lib.PQ_ERR_UNSUPPORTED
    hdr = open(os.path.join(ROOT, "include", "pquant.h")).read()
    assert re.search(r"PQ_OPT_DECODE_PDL\s*=\s*%d\b" % lib.PQ_OPT_DECODE_PDL, hdr)
    assert re.search(r"PQ_OPT_SIDE_STREAM\s*=\s*%d\b" % lib.PQ_OPT_SIDE_STREAM, hdr)
