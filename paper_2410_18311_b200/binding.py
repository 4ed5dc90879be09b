"""ctypes binding of libcoreinfer.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/coreinfer.h)
and takes torch CUDA tensors for the device buffers; all arithmetic runs in the CUDA
kernels.  There is no CPU fallback: if the library is missing or a call fails, a
CoreInferError is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import _build

F32, BF16, F16 = 0, 1, 2
FFN_RELU, FFN_RELU_GATED, FFN_SILU_GATED = 0, 1, 2
MAX_BATCH, MAX_LAYERS = 8, 128
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)

# every symbol include/coreinfer.h declares
SYMBOLS = (
    "coreinfer_count", "coreinfer_last_error",
    "coreinfer_select_workspace_bytes", "coreinfer_select_core",
    "coreinfer_compact", "coreinfer_verify_core_idx",
    "coreinfer_ffn_decode_workspace_bytes", "coreinfer_ffn_decode",
    "coreinfer_ffn_decode_stack_workspace_bytes", "coreinfer_ffn_decode_stack",
    "coreinfer_ffn_decode_stack_noalloc",
    "coreinfer_workspace_status",
    "coreinfer_debug_stamps",
    "coreinfer_ffn_dense_ref",
    "coreinfer_prefill_activations_workspace_bytes", "coreinfer_prefill_activations",
    "coreinfer_counts_add", "coreinfer_counts_add_set", "coreinfer_top_by_count", "coreinfer_core_similarity",
    "coreinfer_nearest_centroid_workspace_bytes", "coreinfer_nearest_centroid",
    "coreinfer_update_core_set_workspace_bytes", "coreinfer_update_core_set",
)
STAMP_SLOTS = 16


class CoreInferError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("coreinfer status %d: %s" % (status, message))
        self.status = status


class Layer(ctypes.Structure):
    """coreinfer_layer"""
    _fields_ = [("w_up_c", ctypes.c_void_p), ("w_gate_c", ctypes.c_void_p),
                ("w_downT_c", ctypes.c_void_p), ("b_up_c", ctypes.c_void_p),
                ("b_down", ctypes.c_void_p), ("K", ctypes.c_int32), ("reserved", ctypes.c_int32)]


_lib = None
_lib_path = None


def library_path() -> str:
    return _lib_path or _build.LIB_PATH


def use_library(path: str) -> None:
    """Make every later call go to another build of the library (the phase-timing variant)."""
    global _lib, _lib_path
    _lib, _lib_path = None, path


def load() -> ctypes.CDLL:
    """Load libcoreinfer.so; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise CoreInferError(ERR_CUDA, "%s not found: build it with "
                             "`python -m paper_2410_18311_b200._build`" % path)
    lib = ctypes.CDLL(path)
    i32, i64, f64, vp, sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_size_t
    lib.coreinfer_count.restype = i32
    lib.coreinfer_count.argtypes = [f64, i32]
    lib.coreinfer_last_error.restype = ctypes.c_char_p
    lib.coreinfer_last_error.argtypes = []
    lib.coreinfer_select_workspace_bytes.restype = sz
    lib.coreinfer_select_workspace_bytes.argtypes = [i32, i32]
    lib.coreinfer_select_core.restype = ctypes.c_int
    lib.coreinfer_select_core.argtypes = [vp, ctypes.c_int, i32, i32, i64, f64, f64, vp, vp, vp, sz, vp]
    lib.coreinfer_compact.restype = ctypes.c_int
    lib.coreinfer_compact.argtypes = [vp, vp, vp, vp, ctypes.c_int, i32, i32, vp, i32, vp, vp, vp, vp, vp]
    lib.coreinfer_verify_core_idx.restype = ctypes.c_int
    lib.coreinfer_verify_core_idx.argtypes = [vp, i32, i32, vp, vp]
    lib.coreinfer_ffn_decode_workspace_bytes.restype = sz
    lib.coreinfer_ffn_decode_workspace_bytes.argtypes = [i32, i32, i32]
    lib.coreinfer_ffn_decode.restype = ctypes.c_int
    lib.coreinfer_ffn_decode.argtypes = [vp, i32, ctypes.c_int, ctypes.c_int, i32, i32, vp, vp, vp, vp, vp,
                                         vp, vp, sz, vp]
    lib.coreinfer_ffn_decode_stack_workspace_bytes.restype = sz
    lib.coreinfer_ffn_decode_stack_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.coreinfer_ffn_decode_stack.restype = ctypes.c_int
    lib.coreinfer_ffn_decode_stack.argtypes = [ctypes.POINTER(Layer), i32, vp, i32, ctypes.c_int, ctypes.c_int,
                                               i32, vp, vp, vp, vp, sz, vp]
    lib.coreinfer_ffn_decode_stack_noalloc.restype = ctypes.c_int
    lib.coreinfer_ffn_decode_stack_noalloc.argtypes = [ctypes.POINTER(Layer), i32, vp, i32, ctypes.c_int,
                                                       ctypes.c_int, i32, vp, vp, vp, vp]
    lib.coreinfer_workspace_status.restype = ctypes.c_int
    lib.coreinfer_workspace_status.argtypes = [vp, vp]
    lib.coreinfer_debug_stamps.restype = ctypes.c_int
    lib.coreinfer_debug_stamps.argtypes = [vp, sz]
    lib.coreinfer_ffn_dense_ref.restype = ctypes.c_int
    lib.coreinfer_ffn_dense_ref.argtypes = [vp, i32, ctypes.c_int, ctypes.c_int, i32, i32, vp, vp, vp, vp, vp,
                                            vp, vp, vp]
    lib.coreinfer_prefill_activations_workspace_bytes.restype = sz
    lib.coreinfer_prefill_activations_workspace_bytes.argtypes = []
    lib.coreinfer_prefill_activations.restype = ctypes.c_int
    lib.coreinfer_prefill_activations.argtypes = [vp, i32, ctypes.c_int, ctypes.c_int, i32, i32, vp, vp, vp, vp, ctypes.c_int, i64,
                                                  vp, sz, vp]
    lib.coreinfer_counts_add.restype = ctypes.c_int
    lib.coreinfer_counts_add.argtypes = [vp, vp, i32, vp]
    lib.coreinfer_counts_add_set.restype = ctypes.c_int
    lib.coreinfer_counts_add_set.argtypes = [vp, vp, i32, i32, vp]
    lib.coreinfer_top_by_count.restype = ctypes.c_int
    lib.coreinfer_top_by_count.argtypes = [vp, i32, i32, f64, vp, vp]
    lib.coreinfer_core_similarity.restype = ctypes.c_int
    lib.coreinfer_core_similarity.argtypes = [vp, i32, vp, i32, vp, vp]
    lib.coreinfer_nearest_centroid_workspace_bytes.restype = sz
    lib.coreinfer_nearest_centroid_workspace_bytes.argtypes = [i32]
    lib.coreinfer_nearest_centroid.restype = ctypes.c_int
    lib.coreinfer_nearest_centroid.argtypes = [vp, i32, i32, vp, vp, vp, sz, vp]
    lib.coreinfer_update_core_set_workspace_bytes.restype = sz
    lib.coreinfer_update_core_set_workspace_bytes.argtypes = [i32, i32]
    lib.coreinfer_update_core_set.restype = ctypes.c_int
    lib.coreinfer_update_core_set.argtypes = [vp, vp, vp, vp, ctypes.c_int, i32, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp,
                                              sz, vp]
    _lib = lib
    return lib


def _check(status: int) -> None:
    if status != OK:
        raise CoreInferError(status, load().coreinfer_last_error().decode())


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float16:
        return F16
    raise CoreInferError(ERR_UNSUPPORTED, "unsupported torch dtype %s" % t.dtype)


def coreinfer_count(frac: float, n: int) -> int:
    return int(load().coreinfer_count(float(frac), int(n)))


def coreinfer_last_error() -> str:
    return load().coreinfer_last_error().decode()


def coreinfer_select_workspace_bytes(T: int, d_ff: int) -> int:
    return int(load().coreinfer_select_workspace_bytes(T, d_ff))


def coreinfer_select_core(act, alpha, beta, core_idx, counts_out, workspace, stream=None,
                          T=None, d_ff=None, ld_act=None, act_dtype=None):
    """act [T, d_ff] fp32, bf16 or fp16 (row stride ld_act) -> core_idx [K] int32 ascending, counts_out [d_ff] | None."""
    T = act.shape[0] if T is None else T
    d_ff = act.shape[1] if d_ff is None else d_ff
    ld_act = act.stride(0) if ld_act is None else ld_act
    _check(load().coreinfer_select_core(_p(act), dtype_code(act) if act_dtype is None else act_dtype,
                                        T, d_ff, ld_act, float(alpha), float(beta), _p(core_idx),
                                        _p(counts_out), _p(workspace),
                                        0 if workspace is None else workspace.numel() * workspace.element_size(),
                                        _stream(stream)))


def coreinfer_compact(w_up, w_gate, w_down, b_up, core_idx, K, w_up_c, w_gate_c, w_downT_c, b_up_c,
                      stream=None):
    d_ff, d_model = w_up.shape
    _check(load().coreinfer_compact(_p(w_up), _p(w_gate), _p(w_down), _p(b_up), dtype_code(w_up), d_model,
                                    d_ff, _p(core_idx), int(K), _p(w_up_c), _p(w_gate_c), _p(w_downT_c),
                                    _p(b_up_c), _stream(stream)))


def coreinfer_verify_core_idx(core_idx, d_ff, report, stream=None, K=None):
    """report: CUDA int32 [2] <- (number of bad positions, first bad position or INT32_MAX)."""
    _check(load().coreinfer_verify_core_idx(_p(core_idx), core_idx.numel() if K is None else int(K), int(d_ff),
                                            _p(report), _stream(stream)))


def coreinfer_ffn_decode_workspace_bytes(batch: int, d_model: int, K: int) -> int:
    return int(load().coreinfer_ffn_decode_workspace_bytes(batch, d_model, K))


def coreinfer_ffn_decode(x, kind, w_up_c, w_gate_c, w_downT_c, b_up_c, b_down, y, workspace, stream=None):
    """x [batch, d_model] -> y [batch, d_model] fp32 over compacted [K, d_model] weights."""
    batch, d_model = x.shape
    K = w_up_c.shape[0]
    _check(load().coreinfer_ffn_decode(_p(x), batch, dtype_code(x), int(kind), d_model, K, _p(w_up_c),
                                       _p(w_gate_c), _p(w_downT_c), _p(b_up_c), _p(b_down), _p(y),
                                       _p(workspace),
                                       0 if workspace is None else workspace.numel() * workspace.element_size(),
                                       _stream(stream)))


def coreinfer_ffn_decode_stack_workspace_bytes(L: int, batch: int, d_model: int, K_max: int) -> int:
    return int(load().coreinfer_ffn_decode_stack_workspace_bytes(L, batch, d_model, K_max))


def make_layers(layers):
    """[(w_up_c, w_gate_c | None, w_downT_c, b_up_c | None, b_down | None), ...] -> coreinfer_layer[L]."""
    arr = (Layer * len(layers))()
    for i, (up, gate, down, bup, bdown) in enumerate(layers):
        arr[i].w_up_c = up.data_ptr()
        arr[i].w_gate_c = None if gate is None else gate.data_ptr()
        arr[i].w_downT_c = down.data_ptr()
        arr[i].b_up_c = None if bup is None else bup.data_ptr()
        arr[i].b_down = None if bdown is None else bdown.data_ptr()
        arr[i].K = up.shape[0]
        arr[i].reserved = 0
    return arr


def coreinfer_ffn_decode_stack(layers, x0, kind, y_last, y_layers, x_layers, workspace, stream=None):
    """layers: a coreinfer_layer array from make_layers(); x0 [batch, d_model], batch 1..8."""
    batch, d_model = x0.shape
    _check(load().coreinfer_ffn_decode_stack(layers, len(layers), _p(x0), batch, dtype_code(x0), int(kind),
                                             d_model, _p(y_last), _p(y_layers), _p(x_layers), _p(workspace),
                                             workspace.numel() * workspace.element_size(), _stream(stream)))


def coreinfer_ffn_decode_stack_noalloc(layers, x0, kind, y_last, y_layers, x_layers, stream=None):
    """coreinfer_ffn_decode_stack for callers that cannot allocate: no workspace argument, the
    scratch is a fixed 128 KiB array inside the library (d_model beyond 10901 raises ERR_UNSUPPORTED).
    Calls that may overlap on the GPU must not share it; make the first call on a device
    outside stream capture."""
    batch, d_model = x0.shape
    _check(load().coreinfer_ffn_decode_stack_noalloc(layers, len(layers), _p(x0), batch, dtype_code(x0),
                                                     int(kind), d_model, _p(y_last), _p(y_layers),
                                                     _p(x_layers), _stream(stream)))


def coreinfer_workspace_status(workspace, stream=None) -> None:
    """Synchronises the stream; raises CoreInferError(ERR_TIMEOUT) if a device-side wait gave up."""
    _check(load().coreinfer_workspace_status(_p(workspace), _stream(stream)))


def coreinfer_debug_stamps(stamps) -> None:
    """stamps: CUDA int64 tensor [CTAs, L, STAMP_SLOTS] that later stack launches fill with cycle
    counts, or None to stop recording.  Raises ERR_UNSUPPORTED unless the phase-timing build is loaded."""
    _check(load().coreinfer_debug_stamps(_p(stamps), 0 if stamps is None else stamps.numel() * stamps.element_size()))


def coreinfer_ffn_dense_ref(x, kind, w_up, w_gate, w_down, b_up, b_down, h_out, y_out, stream=None):
    T, d_model = x.shape
    d_ff = w_up.shape[0]
    _check(load().coreinfer_ffn_dense_ref(_p(x), T, dtype_code(x), int(kind), d_model, d_ff, _p(w_up),
                                          _p(w_gate), _p(w_down), _p(b_up), _p(b_down), _p(h_out), _p(y_out),
                                          _stream(stream)))


def coreinfer_prefill_activations_workspace_bytes() -> int:
    return int(load().coreinfer_prefill_activations_workspace_bytes())


def coreinfer_prefill_activations(x, kind, w_up, w_gate, b_up, act_out, workspace, stream=None):
    """x [T, d], w_up / w_gate [d_ff, d] bf16 or fp16 -> act_out [T, d_ff] fp32, bf16 or fp16 (tensor cores)."""
    T, d_model = x.shape
    d_ff = w_up.shape[0]
    _check(load().coreinfer_prefill_activations(_p(x), T, dtype_code(x), int(kind), d_model, d_ff, _p(w_up), _p(w_gate),
                                                _p(b_up), _p(act_out), dtype_code(act_out), act_out.stride(0), _p(workspace),
                                                workspace.numel() * workspace.element_size(), _stream(stream)))


def coreinfer_counts_add(counts, f, stream=None):
    _check(load().coreinfer_counts_add(_p(counts), _p(f), counts.numel(), _stream(stream)))


def coreinfer_counts_add_set(counts, core_idx, stream=None):
    _check(load().coreinfer_counts_add_set(_p(counts), _p(core_idx), core_idx.numel(), counts.numel(), _stream(stream)))


def coreinfer_top_by_count(counts, max_count, frac, core_idx, stream=None):
    _check(load().coreinfer_top_by_count(_p(counts), counts.numel(), int(max_count), float(frac), _p(core_idx),
                                         _stream(stream)))


def coreinfer_core_similarity(set_a, set_b, shared_involved, stream=None):
    """set_a ascending; shared_involved: CUDA int32 [2] <- (|A and B|, |A or B|)."""
    _check(load().coreinfer_core_similarity(_p(set_a), set_a.numel(), _p(set_b), set_b.numel(), _p(shared_involved),
                                            _stream(stream)))


def coreinfer_nearest_centroid_workspace_bytes(G: int) -> int:
    return int(load().coreinfer_nearest_centroid_workspace_bytes(G))


def coreinfer_nearest_centroid(centroids, v, group_out, workspace, stream=None):
    G, D = centroids.shape
    _check(load().coreinfer_nearest_centroid(_p(centroids), G, D, _p(v), _p(group_out), _p(workspace),
                                             workspace.numel() * workspace.element_size(), _stream(stream)))


def coreinfer_update_core_set_workspace_bytes(d_ff: int, K: int) -> int:
    return int(load().coreinfer_update_core_set_workspace_bytes(d_ff, K))


def coreinfer_update_core_set(w_up, w_gate, w_down, b_up, slot_neuron, core_idx_new, w_up_c, w_gate_c, w_downT_c, b_up_c,
                              n_changed_out, workspace, stream=None):
    d_ff, d_model = w_up.shape
    _check(load().coreinfer_update_core_set(_p(w_up), _p(w_gate), _p(w_down), _p(b_up), dtype_code(w_up), d_model, d_ff,
                                            _p(slot_neuron), _p(core_idx_new), slot_neuron.numel(), _p(w_up_c),
                                            _p(w_gate_c), _p(w_downT_c), _p(b_up_c), _p(n_changed_out), _p(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream)))
