"""Shared helpers of the GPU parity tests (no arithmetic of the method lives here)."""
import numpy as np
import pytest
import torch

import paper_2410_18311_b200 as ci


def require_gpu():
    """The GPU tests never fall back: without the device or the built library they fail/skip loudly."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    ci.binding.load()


def to_f32_np(t):
    """torch tensor (fp32 or bf16, any device) -> float32 numpy, exact."""
    return None if t is None else t.detach().float().cpu().numpy()


def raw_np(t):
    """torch tensor -> numpy array of its bytes (bf16 as uint16)."""
    if t is None:
        return None
    t = t.detach().cpu().contiguous()
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()


def rel_err_fp32(y, y_ref):
    """max_j |y_j - ref_j| / max(|ref_j|, rms(ref)) per row; the fp32 gate is 1e-4."""
    y, y_ref = np.asarray(y, np.float64), np.asarray(y_ref, np.float64)
    rms = np.sqrt(np.mean(y_ref ** 2, axis=-1, keepdims=True))
    return float(np.max(np.abs(y - y_ref) / np.maximum(np.abs(y_ref), np.maximum(rms, 1e-30))))


def rel_err_rms(y, y_ref):
    """max_j |y_j - ref_j| / rms(ref) per row; the bf16 gate is 1e-2."""
    y, y_ref = np.asarray(y, np.float64), np.asarray(y_ref, np.float64)
    rms = np.sqrt(np.mean(y_ref ** 2, axis=-1, keepdims=True))
    return float(np.max(np.abs(y - y_ref) / np.maximum(rms, 1e-30)))


def assert_ffn_close(y, y_ref, dtype):
    if dtype == torch.float32:
        e = rel_err_fp32(y, y_ref)
        assert e <= 1e-4, "fp32 FFN error %.3g > 1e-4" % e
    else:
        e = rel_err_rms(y, y_ref)
        assert e <= 1e-2, "bf16 FFN error %.3g > 1e-2 of the output RMS" % e


def gpu_select(A, alpha, beta, want_counts=True):
    """Run coreinfer_select_core on a CUDA fp32 tensor; returns (S, f) as numpy."""
    T, N = A.shape
    K = ci.coreinfer_count(beta, N)
    S = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    f = torch.full((N,), -1, dtype=torch.int32, device="cuda") if want_counts else None
    ws = torch.empty(ci.coreinfer_select_workspace_bytes(T, N), dtype=torch.uint8, device="cuda")
    ci.coreinfer_select_core(A, alpha, beta, S, f, ws)
    ci.coreinfer_workspace_status(ws)
    return S.cpu().numpy(), (None if f is None else f.cpu().numpy())


def gpu_compact(w_up, w_gate, w_down, b_up, S):
    K = S.shape[0]
    d = w_up.shape[1]
    mk = lambda: torch.empty((K, d), dtype=w_up.dtype, device="cuda")
    up_c, down_c = mk(), mk()
    gate_c = mk() if w_gate is not None else None
    bup_c = torch.empty((K,), dtype=w_up.dtype, device="cuda") if b_up is not None else None
    ci.coreinfer_compact(w_up, w_gate, w_down, b_up, S, K, up_c, gate_c, down_c, bup_c)
    torch.cuda.synchronize()
    return up_c, gate_c, down_c, bup_c


def gpu_decode(x, kind, up_c, gate_c, down_c, bup_c=None, bdown=None):
    B, d = x.shape
    K = up_c.shape[0]
    y = torch.full((B, d), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(ci.coreinfer_ffn_decode_workspace_bytes(B, d, K), dtype=torch.uint8, device="cuda")
    ci.coreinfer_ffn_decode(x, kind, up_c, gate_c, down_c, bup_c, bdown, y, ws)
    ci.coreinfer_workspace_status(ws)
    return y.cpu().numpy()


def check_stack_teacher_forced(layers_gpu, x0, kind, dtype, layers_to_check=None, noalloc=False):
    """One coreinfer_ffn_decode_stack call with per-layer dumps; every checked layer's output is
    compared with the oracle on the very input that layer consumed (Section 4.2), and the step
    between layers with the oracle's residual + RMS glue.  layers_gpu: [(up, gate | None, down,
    b_up | None, b_down | None)] CUDA tensors; x0 [B, d] CUDA.  Returns (y_last, y_layers, x_layers)."""
    import oracle
    L, (B, d) = len(layers_gpu), x0.shape
    Kmax = max(ly[0].shape[0] for ly in layers_gpu)
    arr = ci.binding.make_layers(layers_gpu)
    y_last = torch.full((B, d), float("nan"), device="cuda")
    y_layers = torch.full((L, B, d), float("nan"), device="cuda")
    x_layers = torch.zeros((L, B, d), dtype=dtype, device="cuda")
    if noalloc:
        ci.coreinfer_ffn_decode_stack_noalloc(arr, x0, kind, y_last, y_layers, x_layers)
        torch.cuda.synchronize()
    else:
        ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(L, B, d, Kmax), dtype=torch.uint8, device="cuda")
        ci.coreinfer_ffn_decode_stack(arr, x0, kind, y_last, y_layers, x_layers, ws)
        ci.coreinfer_workspace_status(ws)
    yl, xl = y_layers.cpu().numpy(), to_f32_np(x_layers)
    assert np.isfinite(yl).all()
    np.testing.assert_array_equal(xl[0], to_f32_np(x0))
    np.testing.assert_allclose(y_last.cpu().numpy(), yl[L - 1], rtol=1e-4, atol=1e-5)
    tol = 1e-5 if dtype == torch.float32 else 2 ** -7     # one rounding step of the layer-input type
    for l in (range(L) if layers_to_check is None else layers_to_check):
        up, gate, down, bup, bdown = (to_f32_np(t) for t in layers_gpu[l])
        y_o = oracle.ffn(xl[l], kind, up, gate, down, bup, bdown)
        assert_ffn_close(yl[l], y_o, dtype)
        if l + 1 < L:
            for b in range(B):
                x_next = torch.from_numpy(oracle.glue(xl[l][b], yl[l][b])).to(dtype).float().numpy()
                np.testing.assert_allclose(xl[l + 1][b], x_next.reshape(-1), rtol=tol, atol=tol)
    return y_last, y_layers, x_layers
