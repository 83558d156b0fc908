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
