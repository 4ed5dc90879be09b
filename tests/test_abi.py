"""The C-ABI library loads, exports every symbol the header declares, and rejects bad
arguments on the host (no GPU needed: argument checks come before any CUDA call)."""
import ctypes
import os
import re
from fractions import Fraction

import pytest

import paper_2410_18311_b200 as ci
from paper_2410_18311_b200 import _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    _build.build()
    return ci.binding.load()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "coreinfer.h")).read()
    declared = set(re.findall(r"\b(coreinfer_[a-z0-9_]+)\s*\(", header))
    assert declared == set(ci.binding.SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None, name


def test_count_rule_matches_exact_rational(lib):
    for frac in ("0.1", "0.2", "0.25", "0.4", "1.0"):
        fr, fl = Fraction(frac), float(frac)
        for n in list(range(0, 3000)) + [11008, 16384, 20480, 36864]:
            v = fr * n
            exact = min(n, -((-v.numerator) // v.denominator))
            assert ci.coreinfer_count(fl, n) == exact, (frac, n)


def test_argument_errors_are_reported_without_a_device(lib):
    null = ctypes.c_void_p(None)
    buf = (ctypes.c_char * 1024)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    # selection: NULL activations, bad fraction, bad dtype
    assert lib.coreinfer_select_core(null, ci.F32, 4, 8, 8, 0.4, 0.2, p, null, p, 1024, null) == ci.ERR_INVALID_ARG
    assert b"NULL" in lib.coreinfer_last_error()
    assert lib.coreinfer_select_core(p, ci.F32, 4, 8, 8, 1.5, 0.2, p, null, p, 1024, null) == ci.ERR_INVALID_ARG
    assert lib.coreinfer_select_core(p, 7, 4, 8, 8, 0.4, 0.2, p, null, p, 1024, null) == ci.ERR_UNSUPPORTED
    # 16-bit rows must start on 16-byte boundaries: a row stride of 12 entries does for fp32, not for bf16
    assert lib.coreinfer_select_core(p, ci.F32, 4, 8, 12, 0.4, 0.2, p, null, p, 16, null) == ci.ERR_WORKSPACE
    assert lib.coreinfer_select_core(p, ci.BF16, 4, 8, 12, 0.4, 0.2, p, null, p, 1024, null) == ci.ERR_INVALID_ARG
    # a fraction inside (0, 1] that still rounds to an empty set
    assert lib.coreinfer_select_core(p, ci.F32, 4, 8, 8, 0.4, 1e-9, p, null, p, 1024, null) == ci.ERR_INVALID_ARG
    assert b"no neuron" in lib.coreinfer_last_error()
    assert lib.coreinfer_select_core(p, ci.F32, 4, 8, 8, 0.4, 0.2, p, null, p, 16, null) == ci.ERR_WORKSPACE
    # compaction: K out of range, gate given without its output
    assert lib.coreinfer_compact(p, null, p, null, ci.F32, 8, 16, p, 17, p, null, p, null, null) == ci.ERR_INVALID_ARG
    assert lib.coreinfer_compact(p, p, p, null, ci.F32, 8, 16, p, 4, p, null, p, null, null) == ci.ERR_INVALID_ARG
    # decode: batch out of range, row not a multiple of 16 bytes, missing gate
    assert lib.coreinfer_ffn_decode(p, 9, ci.BF16, ci.FFN_RELU, 64, 4, p, null, p, null, null, p, p, 1024, null) == ci.ERR_UNSUPPORTED
    assert lib.coreinfer_ffn_decode(p, 1, ci.BF16, ci.FFN_RELU, 60, 4, p, null, p, null, null, p, p, 1024, null) == ci.ERR_INVALID_ARG
    assert lib.coreinfer_ffn_decode(p, 1, ci.BF16, ci.FFN_RELU_GATED, 64, 4, p, null, p, null, null, p, p, 1024, null) == ci.ERR_INVALID_ARG
    # stack: batch beyond COREINFER_MAX_BATCH, L out of range
    layers = ci.binding.Layer * 1
    assert lib.coreinfer_ffn_decode_stack(layers(), 1, p, 9, ci.BF16, ci.FFN_RELU, 64, p, null, null, p, 1024, null) == ci.ERR_UNSUPPORTED
    assert lib.coreinfer_ffn_decode_stack(layers(), 0, p, 1, ci.BF16, ci.FFN_RELU, 64, p, null, null, p, 1024, null) == ci.ERR_INVALID_ARG
    # dense: y without h
    assert lib.coreinfer_ffn_dense_ref(p, 4, ci.F32, ci.FFN_RELU, 8, 16, p, null, p, null, null, null, p, null) == ci.ERR_INVALID_ARG


def test_workspace_sizes(lib):
    assert ci.coreinfer_select_workspace_bytes(0, 8) == 0
    assert ci.coreinfer_select_workspace_bytes(64, 3072) >= 64 * 3072 * 2 + 3072 * 4
    assert ci.coreinfer_ffn_decode_workspace_bytes(1, 4096, 3277) >= 4
    assert ci.coreinfer_ffn_decode_workspace_bytes(8, 4096, 2752) >= 8 * 2752 * 4
    assert ci.coreinfer_ffn_decode_stack_workspace_bytes(32, 1, 4096, 3277) >= 256 + 3 * 4096 * 4
    assert ci.coreinfer_ffn_decode_stack_workspace_bytes(32, 8, 4096, 2752) >= 8 * 2752 * 4 + 3 * 8 * 4096 * 4
