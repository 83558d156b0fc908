"""The C-ABI library builds, loads and exports every symbol include/flop.h declares
(no compute: these run without a GPU), and host-side argument checks answer with
return codes before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_1910_04732_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    from paper_1910_04732_b200 import binding
    return binding.load_library()


def test_header_symbols_are_exported(lib):
    text = open(os.path.join(ROOT, "include", "flop.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(flop_[a-z0-9_]+)\s*\(", text)))
    assert "flop_gate_sample" in declared and "flop_compact_fwd" in declared and len(declared) >= 9
    for name in declared:
        assert hasattr(lib, name), name
    from paper_1910_04732_b200 import binding
    assert sorted(binding.EXPORTS) == declared


def test_status_strings(lib):
    from paper_1910_04732_b200 import binding as b
    assert b.status_string(b.OK) == "ok"
    assert "workspace" in b.status_string(b.ERR_WORKSPACE)
    assert "timed out" in b.status_string(b.ERR_TIMEOUT)
    assert b.status_string(99) == "unknown status"


def test_workspace_query_and_argument_checks(lib):
    from paper_1910_04732_b200 import binding as b
    # forward scratch holds H'[T, r] with r padded to 8 elements
    assert b.workspace_bytes(b.OP_FWD, 100, 64, 64, 30, b.BF16) >= 100 * 32 * 2
    assert b.workspace_bytes(b.OP_FWD, 100, 64, 64, 30, b.F32) >= 100 * 32 * 4
    assert b.workspace_bytes(b.OP_BWD, 4096, 768, 768, 768, b.BF16) > 4096 * 768 * 2
    assert b.workspace_bytes(b.OP_L0, 55296, 0, 0, 72, b.F32) >= 8 * (54 + 72)
    assert b.workspace_bytes(b.OP_COMPACT, 0, 1024, 4096, 1024, b.BF16) == 0
    out = ctypes.c_size_t(0)
    assert lib.flop_workspace_bytes(99, 1, 1, 1, 1, 0, ctypes.byref(out)) == b.ERR_INVALID_ARG
    assert lib.flop_workspace_bytes(b.OP_FWD, -1, 1, 1, 1, 0, ctypes.byref(out)) == b.ERR_INVALID_ARG
    assert lib.flop_workspace_bytes(b.OP_FWD, 1, 1, 1, 1, 7, ctypes.byref(out)) == b.ERR_INVALID_ARG
    # invalid hard-concrete constants and null pointers are refused on the host
    bad = b.HcParams(0.0, -0.1, 1.1)
    assert lib.flop_gate_sample(None, 8, bad, 0, 0, None, None, None, None) == b.ERR_INVALID_ARG
    good = b.HcParams(2 / 3, -0.1, 1.1)
    assert lib.flop_gate_sample(None, 8, good, 0, 0, None, None, None, None) == b.ERR_INVALID_ARG
    assert lib.flop_gate_sample(None, 0, good, 0, 0, None, None, None, None) == b.OK       # n = 0: nothing to do
    assert lib.flop_gate_sample(None, -1, good, 0, 0, None, None, None, None) == b.ERR_INVALID_ARG
    assert lib.flop_gated_lowrank_fwd(None, 8, None, 8, None, 8, None, None, 8, None, 8, 4, 8, 8, 8, b.BF16,
                                      None, 0, None) == b.ERR_INVALID_ARG
    assert lib.flop_gated_lowrank_fwd(None, 8, None, 8, None, 8, None, None, 8, None, 8, 0, 8, 8, 8, b.BF16,
                                      None, 0, None) == b.OK                              # T = 0
    assert lib.flop_compact_ranks(None, 2, good, 8, None, 0, None, 0, 0, 0, 0, None, None, None, None, 0, None, 0,
                                  None, 0, None) == b.ERR_INVALID_ARG


def test_struct_layouts_match_the_header(tmp_path):
    """Every argument struct of include/flop.h, compiled as plain C, has the size and the field offsets of its
    ctypes mirror in the binding (a field added on one side only would shift every pointer after it)."""
    import shutil
    import subprocess
    from paper_1910_04732_b200 import binding as b
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    pairs = {"flop_hc_params_t": b.HcParams, "flop_fwd_problem_t": b.FwdProblem, "flop_bwd_problem_t": b.BwdProblem,
             "flop_scale_rows_t": b.ScaleRows, "flop_active_gather_t": b.ActiveGather,
             "flop_active_scatter_t": b.ActiveScatter}
    text = open(os.path.join(ROOT, "include", "flop.h")).read()
    structs = set(re.findall(r"}\s*(flop_[a-z0-9_]+_t)\s*;", re.sub(r"/\*.*?\*/", "", text, flags=re.S)))
    structs -= {"flop_status_t", "flop_op_t", "flop_dtype_t"}      # enums
    assert structs == set(pairs), structs ^ set(pairs)
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "flop.h"', 'int main(void) {']
    for cname, cls in pairs.items():
        lines.append(f'  printf("{cname} size %zu\\n", sizeof({cname}));')
        for fname, _ in cls._fields_:
            lines.append(f'  printf("{cname} {fname} %zu\\n", offsetof({cname}, {fname}));')
    lines += ['  return 0;', '}']
    src, exe = tmp_path / "layout.c", tmp_path / "layout"
    src.write_text("\n".join(lines))
    subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)])
    out = subprocess.check_output([str(exe)], text=True).split("\n")
    want = {}
    for ln in out:
        if ln.strip():
            c, f, v = ln.split()
            want[(c, f)] = int(v)
    for cname, cls in pairs.items():
        assert ctypes.sizeof(cls) == want[(cname, "size")], cname
        for fname, _ in cls._fields_:
            assert getattr(cls, fname).offset == want[(cname, fname)], (cname, fname)
        # and no field of the C struct is missing from the mirror: the sizes agree and the last field ends the struct
        last = cls._fields_[-1][0]
        assert getattr(cls, last).offset + getattr(cls, last).size <= ctypes.sizeof(cls)
