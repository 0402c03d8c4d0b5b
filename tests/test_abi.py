"""The C-ABI library loads and exports every symbol the header declares; host-side checks that need no GPU."""
import ctypes
import os
import re

import pytest

from paper_2508_12594_b200 import build, flare

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return flare.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "flare.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(flare_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"flare_encode", "flare_decode", "flare_forward", "flare_backward"} <= set(names)
    raw = ctypes.CDLL(flare.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
    assert sorted(flare.exported_symbols()) == names


def test_binding_argument_counts_match_the_header():
    """Every prototype in the header has as many parameters as the binding's ctypes signature."""
    text = open(os.path.join(ROOT, "include", "flare.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    protos = dict(re.findall(r"\b(flare_[a-z_]+)\s*\(([^)]*)\)\s*;", text))
    assert set(protos) == set(flare._SIGNATURES)
    for name, params in protos.items():
        n = 0 if params.strip() in ("", "void") else params.count(",") + 1
        assert n == len(flare._SIGNATURES[name][1]), name


def test_status_strings(lib):
    assert lib.flare_status_string(0) == b"ok"
    for s in range(1, 7):
        assert len(lib.flare_status_string(s)) > 0
    assert lib.flare_version() >= 100


def test_descriptor_validation_needs_no_device(lib):
    ok = flare.FlareDesc(1, 2, 1024, 16, 16, flare.DTYPE_F32, 1.0)
    assert flare.flare_workspace_bytes(ok, flare.OP_FORWARD) > 0
    assert flare.flare_encode_partials(ok) >= 1
    for bad in (flare.FlareDesc(0, 2, 8, 16, 16, 0, 1.0), flare.FlareDesc(1, 2, 8, 16, 12, 0, 1.0),
                flare.FlareDesc(1, 2, 8, 17, 16, flare.DTYPE_BF16, 1.0), flare.FlareDesc(1, 2, 8, 4096, 16, 1, 1.0),
                flare.FlareDesc(1, 2, 8, 16, 16, 7, 1.0), flare.FlareDesc(1, 2, 8, 16, 16, 0, float("nan"))):
        assert flare.flare_workspace_bytes(bad, flare.OP_FORWARD) == 0
    # null pointers are rejected before anything touches a device
    rc = lib.flare_encode(ctypes.byref(ok), None, None, None, None, None, None, None, 0, None)
    assert rc == flare.ERR_INVALID_ARG
    rc = lib.flare_decode(ctypes.byref(flare.FlareDesc(1, 2, 8, 16, 12, 0, 1.0)), None, None, None, None, None, None, 0, None)
    assert rc == flare.ERR_UNSUPPORTED


def test_every_head_width_of_the_paper_is_accepted(lib):
    """D = 4 and 8 (the paper's PDE models: C = 64 with 16 or 8 heads) up to 64, both dtypes, all operations."""
    for D in (4, 8, 16, 32, 64):
        for dtype in (flare.DTYPE_F32, flare.DTYPE_BF16):
            desc = flare.FlareDesc(2, 64 // D if D <= 16 else 2, 1000, 64, D, dtype, 1.0)
            for op in (flare.OP_ENCODE, flare.OP_FORWARD, flare.OP_BACKWARD):
                assert flare.flare_workspace_bytes(desc, op) > 0, (D, dtype, op)
    assert flare.flare_workspace_bytes(flare.FlareDesc(2, 4, 1000, 64, 2, flare.DTYPE_BF16, 1.0), flare.OP_FORWARD) == 0


def test_workspace_never_scales_with_n_times_m(lib):
    """Scratch is O(partials * B*H*M*(D+2)): growing N a thousandfold must not grow it by the same factor."""
    small = flare.FlareDesc(1, 8, 4096, 256, 16, flare.DTYPE_BF16, 1.0)
    big = flare.FlareDesc(1, 8, 1048576, 256, 16, flare.DTYPE_BF16, 1.0)
    ws, wb = flare.flare_workspace_bytes(small, 2), flare.flare_workspace_bytes(big, 2)
    assert wb < 1048576 * 256 * 2 / 8          # far below one N x M bf16 matrix of a single head
    rows = 8 * 256
    assert wb <= 256 + 4096 + flare.flare_encode_partials(big) * rows * (16 + 2) * 4 + rows * 16 * 4 + 4 * 256
    assert ws <= wb
