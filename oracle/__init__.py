"""CPU oracle for the CoreInfer hot path -- TEST INFRASTRUCTURE ONLY.

A thin numpy/ctypes front for ``coreinfer_oracle.c`` (plain C, double
accumulators, full sorts).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg use it; the CUDA library and its Python binding
never import this package, and this package imports nothing of theirs.

Passages followed: Definition 1 / Eq. 1 (token-wise core neurons), Eq. 3
(membership counts), Definition 2 / Eq. 2 (sentence-wise core neurons),
Section 4.2 (decode through the fixed set), Section 5 "Models" (fp32
intermediates).  Nothing here is "parity unpinned": each function is checked
in ``tests/test_oracle_*.py`` against values it did not produce itself.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "coreinfer_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libcoreinfer_oracle.so")
_LIB_F32 = os.path.join(_HERE, "_build", "libcoreinfer_oracle_f32acc.so")   # -DORACLE_F32_ACC, not the oracle
_lock = threading.Lock()
_lib = None


def build(force: bool = False, f32_acc: bool = False) -> str:
    """Compile the oracle with gcc (C11, -O2, OpenMP, no fast-math, no contraction) and
    return the library path.  f32_acc builds the fp32-accumulator variant of the FFN loops."""
    lib = _LIB_F32 if f32_acc else _LIB
    os.makedirs(os.path.dirname(lib), exist_ok=True)
    if (not force and os.path.exists(lib)
            and os.path.getmtime(lib) >= os.path.getmtime(_SRC)):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
           "-fno-fast-math", "-ffp-contract=off"] + (["-DORACLE_F32_ACC"] if f32_acc else []) + ["-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i32, i64, f64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
            lib.oracle_num_threads.restype = ctypes.c_int
            lib.oracle_count.restype = i32
            lib.oracle_count.argtypes = [f64, i32]
            lib.oracle_token_core.restype = i32
            lib.oracle_token_core.argtypes = [vp, i32, f64, vp]
            lib.oracle_select.restype = i32
            lib.oracle_select.argtypes = [vp, i32, i32, i64, f64, f64, vp, vp]
            lib.oracle_compact.restype = None
            lib.oracle_compact.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, i32, vp, vp, vp, vp]
            lib.oracle_ffn.restype = None
            lib.oracle_ffn.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
            lib.oracle_ffn_dense.restype = None
            lib.oracle_ffn_dense.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
            lib.oracle_glue.restype = None
            lib.oracle_glue.argtypes = [vp, vp, i32, vp]
            lib.oracle_top_by_count.restype = None
            lib.oracle_top_by_count.argtypes = [vp, i32, i32, vp]
            lib.oracle_counts_add_set.restype = None
            lib.oracle_counts_add_set.argtypes = [vp, vp, i32]
            lib.oracle_core_similarity.restype = None
            lib.oracle_core_similarity.argtypes = [vp, i32, vp, i32, vp]
            lib.oracle_nearest_centroid.restype = i32
            lib.oracle_nearest_centroid.argtypes = [vp, i32, i32, vp, vp]
            lib.oracle_set_delta.restype = i32
            lib.oracle_set_delta.argtypes = [vp, i32, vp, vp, vp]
            _lib = lib
    return _lib


RELU = 0
RELU_GATED = 1
SILU_GATED = 2      # h = silu(w_gate.x) * (w_up.x); Definition 1 is applied to h unchanged


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def count(frac: float, n: int) -> int:
    """Size of a "top fraction": ceil(frac * n) clamped to [0, n]."""
    return int(_load().oracle_count(float(frac), int(n)))


def token_core(a, alpha: float) -> np.ndarray:
    """Definition 1 / Eq. 1: indices of one token's core neurons, in rank order
    (largest activation first, equal values by lower index)."""
    a = _f32(a)
    assert a.ndim == 1
    members = np.empty(max(a.shape[0], 1), dtype=np.int32)
    k = _load().oracle_token_core(_ptr(a), a.shape[0], float(alpha), _ptr(members))
    return members[:k].copy()


def select(A, alpha: float, beta: float):
    """Definition 2 / Eq. 2-3: (S, f) with S the ascending int32 list of the
    ceil(beta*N) sentence-wise core neurons of A [T, N] and f [N] the counts."""
    A = _f32(A)
    assert A.ndim == 2
    T, N = A.shape
    K = count(beta, N)
    S = np.empty(max(K, 1), dtype=np.int32)
    f = np.empty(max(N, 1), dtype=np.int32)
    k = _load().oracle_select(_ptr(A), T, N, N, float(alpha), float(beta), _ptr(S), _ptr(f))
    assert k == K
    return S[:K].copy(), f[:N].copy()


def compact(w_up, w_gate, w_down, b_up, S):
    """Element-copy compaction.  Arrays may have any fixed-size dtype (bf16
    payloads are passed as uint16 views); returns (w_up_c, w_gate_c, w_downT_c,
    b_up_c) of the same dtype with shapes [K, d], [K, d] | None, [K, d], [K] | None."""
    w_up = np.ascontiguousarray(w_up)
    w_down = np.ascontiguousarray(w_down)
    N, d = w_up.shape
    assert w_down.shape == (d, N)
    dt = w_up.dtype
    S = np.ascontiguousarray(S, dtype=np.int32)
    K = S.shape[0]
    w_gate = None if w_gate is None else np.ascontiguousarray(w_gate, dtype=dt)
    b_up = None if b_up is None else np.ascontiguousarray(b_up, dtype=dt)
    up_c = np.empty((K, d), dtype=dt)
    gate_c = None if w_gate is None else np.empty((K, d), dtype=dt)
    down_c = np.empty((K, d), dtype=dt)
    bup_c = None if b_up is None else np.empty((K,), dtype=dt)
    _load().oracle_compact(_ptr(w_up), _ptr(w_gate), _ptr(w_down), _ptr(b_up),
                           dt.itemsize, d, N, _ptr(S), K,
                           _ptr(up_c), _ptr(gate_c), _ptr(down_c), _ptr(bup_c))
    return up_c, gate_c, down_c, bup_c


_lib_f32 = None


def ffn_f32_accumulators(x, kind, w_up_c, w_gate_c, w_downT_c, b_up_c=None, b_down=None):
    """The FFN loops of ffn() with fp32 running sums (the -DORACLE_F32_ACC build).  Not the
    oracle: it exists to report the distance between fp32 and double accumulation."""
    global _lib_f32
    with _lock:
        if _lib_f32 is None:
            _lib_f32 = ctypes.CDLL(build(f32_acc=True))
            vp, i32 = ctypes.c_void_p, ctypes.c_int32
            _lib_f32.oracle_ffn.restype = None
            _lib_f32.oracle_ffn.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    x = _f32(x)
    if x.ndim == 1:
        x = x[None, :]
    B, d = x.shape
    w_up_c, w_gate_c, w_downT_c = _f32(w_up_c), _f32(w_gate_c), _f32(w_downT_c)
    b_up_c, b_down = _f32(b_up_c), _f32(b_down)
    K = w_up_c.shape[0]
    y = np.empty((B, d), dtype=np.float32)
    _lib_f32.oracle_ffn(_ptr(x), B, int(kind), d, K, _ptr(w_up_c), _ptr(w_gate_c), _ptr(w_downT_c),
                        _ptr(b_up_c), _ptr(b_down), _ptr(y), None)
    return y


def ffn(x, kind, w_up_c, w_gate_c, w_downT_c, b_up_c=None, b_down=None, return_h=False):
    """Decode FFN over compacted weights; x [B, d] -> y [B, d] fp32."""
    x = _f32(x)
    if x.ndim == 1:
        x = x[None, :]
    B, d = x.shape
    w_up_c, w_gate_c, w_downT_c = _f32(w_up_c), _f32(w_gate_c), _f32(w_downT_c)
    b_up_c, b_down = _f32(b_up_c), _f32(b_down)
    K = w_up_c.shape[0]
    assert w_up_c.shape == (K, d) and w_downT_c.shape == (K, d)
    assert (kind in (RELU_GATED, SILU_GATED)) == (w_gate_c is not None)
    y = np.empty((B, d), dtype=np.float32)
    h = np.empty((B, max(K, 1)), dtype=np.float32) if return_h else None
    _load().oracle_ffn(_ptr(x), B, int(kind), d, K, _ptr(w_up_c), _ptr(w_gate_c),
                       _ptr(w_downT_c), _ptr(b_up_c), _ptr(b_down), _ptr(y), _ptr(h))
    return (y, h[:, :K]) if return_h else y


def ffn_dense(x, kind, w_up, w_gate, w_down, b_up=None, b_down=None, want_h=True, want_y=True):
    """Dense FFN on the uncompacted weights; returns (H [T, N] | None, Y [T, d] | None)."""
    x = _f32(x)
    if x.ndim == 1:
        x = x[None, :]
    T, d = x.shape
    w_up, w_gate, w_down = _f32(w_up), _f32(w_gate), _f32(w_down)
    b_up, b_down = _f32(b_up), _f32(b_down)
    N = w_up.shape[0]
    assert w_up.shape == (N, d) and w_down.shape == (d, N)
    assert (kind in (RELU_GATED, SILU_GATED)) == (w_gate is not None)
    H = np.empty((T, N), dtype=np.float32) if want_h else None
    Y = np.empty((T, d), dtype=np.float32) if want_y else None
    _load().oracle_ffn_dense(_ptr(x), T, int(kind), d, N, _ptr(w_up), _ptr(w_gate),
                             _ptr(w_down), _ptr(b_up), _ptr(b_down), _ptr(H), _ptr(Y))
    return H, Y


def glue(x, y) -> np.ndarray:
    """Stack glue (not from the paper): (x + y) / rms(x + y), fp32 result."""
    x, y = _f32(x).reshape(-1), _f32(y).reshape(-1)
    out = np.empty_like(x)
    _load().oracle_glue(_ptr(x), _ptr(y), x.shape[0], _ptr(out))
    return out


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def top_by_count(counts, frac: float) -> np.ndarray:
    """The ceil(frac * N) neurons with the largest counts (equal counts: lower index first),
    ascending: Definition 2's rule applied to any count vector (summed token counts of a prompt
    that arrived in pieces; per-group membership counts of similarity-guided prediction)."""
    counts = _i32(counts)
    N = counts.shape[0]
    K = count(frac, N)
    S = np.empty(max(K, 1), dtype=np.int32)
    _load().oracle_top_by_count(_ptr(counts), N, K, _ptr(S))
    return S[:K].copy()


def group_counts(sets, N: int) -> np.ndarray:
    """counts[n] = number of the given core sets that hold neuron n (Section 4.1, similarity-guided)."""
    c = np.zeros(N, dtype=np.int32)
    for S in sets:
        S = _i32(S)
        _load().oracle_counts_add_set(_ptr(c), _ptr(S), S.shape[0])
    return c


def core_similarity(A, B):
    """(shared, involved) = (|A and B|, |A or B|); Insight-2's similarity is shared / involved."""
    A, B = _i32(A), _i32(B)
    out = np.zeros(2, dtype=np.int32)
    _load().oracle_core_similarity(_ptr(A), A.shape[0], _ptr(B), B.shape[0], _ptr(out))
    return int(out[0]), int(out[1])


def nearest_centroid(centroids, v):
    """(group, squared distances in double) of the centroid nearest to v; ties go to the lower group."""
    centroids, v = _f32(centroids), _f32(v).reshape(-1)
    G, D = centroids.shape
    d2 = np.empty(G, dtype=np.float64)
    g = _load().oracle_nearest_centroid(_ptr(centroids), G, D, _ptr(v), _ptr(d2))
    return int(g), d2


def set_delta(slot_neuron, S_new):
    """Rows to rewrite when the deployed set changes to S_new: (slots, neurons, new slot_neuron)."""
    slot_neuron = _i32(slot_neuron).copy()
    S_new = _i32(S_new)
    K = slot_neuron.shape[0]
    assert S_new.shape[0] == K
    slots = np.empty(max(K, 1), dtype=np.int32)
    neurons = np.empty(max(K, 1), dtype=np.int32)
    n = _load().oracle_set_delta(_ptr(slot_neuron), K, _ptr(S_new), _ptr(slots), _ptr(neurons))
    return slots[:n].copy(), neurons[:n].copy(), slot_neuron
