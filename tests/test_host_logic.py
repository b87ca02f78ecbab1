"""CPU-only checks: the C-ABI library loads, exports every declared symbol, sizes
workspaces and rejects bad arguments before touching a GPU."""
import ctypes
import os
import re

import pytest

from paper_2410_17765_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "cpmtp.h")).read()
    declared = set(re.findall(r"\b(cpmtp_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_checked_build_exports_the_same_symbols():
    """The checked build (index checks in every epilogue) is the same library plus the checks."""
    dbg = ctypes.CDLL(build.build(debug=True))
    for name in binding.EXPORTS:
        assert getattr(dbg, name) is not None
    dbg.cpmtp_debug_status.restype = ctypes.c_int
    # without a device the status word cannot be read: an error code, never "clean"
    import torch

    if not torch.cuda.is_available():
        assert dbg.cpmtp_debug_status() < 0


def test_release_build_reports_that_it_has_no_index_checks(lib):
    if os.environ.get("CPMTP_LIBRARY"):
        pytest.skip("another library was selected")
    assert binding.debug_status() == -1


def test_version_and_status_strings(lib):
    assert lib.cpmtp_version() >= 100
    assert lib.cpmtp_status_string(0) == b"ok"
    for code in range(-7, 0):
        assert lib.cpmtp_status_string(code) not in (b"ok", b"unknown status")


def test_workspace_sizes(lib):
    s = binding.make_shape(64, 256, 1024, 3, 4)
    fwd = binding.workspace_bytes(s, binding.OP_FORWARD)
    bwd = binding.workspace_bytes(s, binding.OP_BACKWARD)
    # forward holds at least z (bf16) ; backward at least dz and one 128-row chunk of logit gradients
    assert fwd >= 2 * 64 * 12 * 256
    assert bwd >= 2 * 64 * 12 * 256 + 2 * 128 * 1024
    assert binding.workspace_bytes(s, binding.OP_SCORE) > 0
    assert binding.workspace_bytes(s, 99) == 0
    assert binding.host_staging_bytes(s) >= 2 * 64 * 256 + 4 * 64 * 3 + 4 * 64


@pytest.mark.parametrize("bad", [dict(N=0), dict(d=100), dict(d=32), dict(V=1), dict(n=0), dict(n=9), dict(r=0), dict(r=33)])
def test_invalid_shapes_are_rejected(lib, bad):
    args = dict(N=8, d=128, V=100, n=2, r=2)
    args.update(bad)
    s = binding.make_shape(**args)
    assert binding.workspace_bytes(s, binding.OP_FORWARD) == 0
    buf = (ctypes.c_char * 4096)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    rc = lib.cpmtp_forward(ctypes.byref(s), p, p, p, p, p, p, None, None, None, p, 4096, None, None)
    assert rc == -2


def test_null_and_misaligned_pointers_are_rejected(lib):
    s = binding.make_shape(8, 128, 100, 2, 2)
    buf = (ctypes.c_char * 8192)()
    base = ctypes.addressof(buf)
    base += (-base) % 256
    p = ctypes.c_void_p(base)
    odd = ctypes.c_void_p(base + 2)
    assert lib.cpmtp_forward(ctypes.byref(s), None, p, p, p, p, p, None, None, None, p, 4096, None, None) == -1
    assert lib.cpmtp_forward(ctypes.byref(s), odd, p, p, p, p, p, None, None, None, p, 4096, None, None) == -3
    assert lib.cpmtp_backward(ctypes.byref(s), p, p, p, p, p, None, None, p, p, p, p, p, 4096, None, None) in (-1, -5, -6)
    assert lib.cpmtp_forward(None, p, p, p, p, p, p, None, None, None, p, 4096, None, None) == -1


def test_distill_workspace_and_argument_checks(lib):
    s = binding.make_shape(64, 256, 1024, 3, 3)
    fwd = binding.workspace_bytes(s, binding.OP_FORWARD)
    dfwd = binding.workspace_bytes(s, binding.OP_DISTILL_FORWARD)
    dbwd = binding.workspace_bytes(s, binding.OP_DISTILL_BACKWARD)
    assert dfwd > fwd                                   # the plain forward plus the KL partials
    # backward: dz, one chunk of logit gradients of whole padded tiles (32 groups of 3 rows), weights per (i, k)
    assert dbwd >= 2 * 64 * 9 * 256 + 2 * 96 * 1024 + 4 * 64 * 3
    buf = (ctypes.c_char * 8192)()
    base = ctypes.addressof(buf)
    base += (-base) % 256
    p = ctypes.c_void_p(base)
    f = ctypes.c_float
    # shape errors come first, then missing pointers
    bad = binding.make_shape(64, 100, 1024, 3, 3)
    assert lib.cpmtp_distill_forward(ctypes.byref(bad), p, p, p, p, p, p, f(0.9), f(1.0), p, p, None, None, None,
                                     p, 4096, None, None) == -2
    assert lib.cpmtp_distill_forward(ctypes.byref(s), p, p, p, p, p, None, f(0.9), f(1.0), p, p, None, None, None,
                                     p, 4096, None, None) in (-1, -5, -6)
    assert lib.cpmtp_distill_backward(ctypes.byref(s), p, p, p, p, p, None, None, None, f(0.9), f(1.0), None, None,
                                      p, p, p, p, p, 4096, None, None) == -1


def test_product_and_oracle_do_not_import_each_other():
    """The package never imports the oracle (no CPU fallback can hide behind it) and the oracle never imports the
    package's CUDA side; only the seeded input generators are shared."""
    import ast
    import pathlib

    root = pathlib.Path(__file__).resolve().parents[1]

    def imported(path):
        names = set()
        for node in ast.walk(ast.parse(path.read_text())):
            if isinstance(node, ast.Import):
                names.update(a.name for a in node.names)
            elif isinstance(node, ast.ImportFrom):
                names.add(("." * node.level) + (node.module or ""))
                names.update(f"{node.module or ''}.{a.name}" for a in node.names)
        return names

    for f in (root / "paper_2410_17765_b200").glob("*.py"):
        assert not any(n.split(".")[0] == "oracle" or ".oracle" in n for n in imported(f)), f
    for f in (root / "oracle").glob("*.py"):
        assert not any("binding" in n or "build" in n or "dist_util" in n for n in imported(f)), f
