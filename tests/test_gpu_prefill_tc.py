"""The tensor-core pre-fill (tcgen05.mma) against the oracle's dense FFN intermediate: fp32 gate
(1e-4 relative), ragged and full-size shapes, and selection on its output (Definition 1-2 are
exact on whichever tensor they are given)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from paper_2410_18311_b200 import workloads as wl
from helpers import require_gpu, to_f32_np, assert_ffn_close, gpu_select

pytestmark = pytest.mark.gpu


def _tc(X, kind, w_up, w_gate, b_up):
    T, N = X.shape[0], w_up.shape[0]
    A = torch.full((T, N), float("nan"), device="cuda")
    ws = torch.empty(ci.coreinfer_prefill_activations_workspace_bytes(), dtype=torch.uint8, device="cuda")
    ci.coreinfer_prefill_activations(X, kind, w_up, w_gate, b_up, A, ws)
    ci.coreinfer_workspace_status(ws)
    return A


@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("T,d,N", [(1, 64, 8), (37, 328, 1000), (128, 512, 128), (200, 1024, 3072), (300, 264, 652)])
def test_small_and_ragged_shapes(gated, T, d, N):
    require_gpu()
    g = torch.Generator().manual_seed(T + d + N)
    mk = lambda *s, std=1.0: (torch.randn(*s, generator=g) * std).to(torch.bfloat16).cuda()
    X, w_up = mk(T, d), mk(N, d, std=0.05)
    w_gate = mk(N, d, std=0.05) if gated else None
    b_up = None if gated else mk(N, std=0.5)
    kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
    A = _tc(X, kind, w_up, w_gate, b_up).cpu().numpy()
    assert np.isfinite(A).all()
    w_down = np.zeros((d, N), np.float32)
    H_o, _ = oracle.ffn_dense(to_f32_np(X), kind, to_f32_np(w_up), to_f32_np(w_gate), w_down, to_f32_np(b_up), None,
                              want_y=False)
    assert_ffn_close(A, H_o, torch.float32)


def test_integer_inputs_are_bit_exact():
    """Small integers: every product and every partial sum is exact in fp32 in any order."""
    require_gpu()
    rng = np.random.default_rng(5)
    T, d, N = 150, 256, 300
    mk = lambda *s: torch.from_numpy(rng.integers(-4, 5, size=s).astype(np.float32)).to(torch.bfloat16).cuda()
    X, w_up, w_gate = mk(T, d), mk(N, d), mk(N, d)
    for kind, gate in ((ci.FFN_RELU, None), (ci.FFN_RELU_GATED, w_gate)):
        A = _tc(X, kind, w_up, gate, None).cpu().numpy()
        H_o, _ = oracle.ffn_dense(to_f32_np(X), kind, to_f32_np(w_up), to_f32_np(gate), np.zeros((d, N), np.float32),
                                  want_y=False)
        np.testing.assert_array_equal(A, H_o)


@pytest.mark.parametrize("name", ["opt6.7b", "relu-llama2-7b"])
def test_full_size_layer_and_selection_on_its_output(name):
    require_gpu()
    cfg = wl.CONFIGS[name]
    X = wl.prompt_hidden(cfg, device="cuda")
    w_up, w_gate, _ = wl.layer_weights(cfg, 2, device="cuda")
    kind = ci.FFN_RELU_GATED if cfg.gated else ci.FFN_RELU
    A = _tc(X, kind, w_up, w_gate, None)
    rows = [0, 77, cfg.T - 1]
    H_o, _ = oracle.ffn_dense(to_f32_np(X[rows]), kind, to_f32_np(w_up), to_f32_np(w_gate),
                              np.zeros((cfg.d_model, cfg.d_ff), np.float32), want_y=False)
    assert_ffn_close(A[rows].cpu().numpy(), H_o, torch.float32)
    # against the plain GPU reference on all rows (another summation order)
    A_ref = torch.empty_like(A)
    ci.coreinfer_ffn_dense_ref(X, kind, w_up, w_gate, wl.layer_weights(cfg, 2, device="cuda")[2], None, None, A_ref, None)
    torch.cuda.synchronize()
    assert_ffn_close(A.cpu().numpy(), A_ref.cpu().numpy(), torch.float32)
    S, f = gpu_select(A, cfg.alpha, cfg.beta)
    S_o, f_o = oracle.select(A.cpu().numpy(), cfg.alpha, cfg.beta)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)


@pytest.mark.parametrize("gated,width", [(False, 256), (False, 224), (False, 192), (False, 160), (True, 96), (True, 64)])
def test_every_tile_width_the_host_can_pick(gated, width):
    """The tile width is picked per call so that the tiles fill whole waves of the GPU's SMs:
    with one row tile and d_ff = (SM count) x width - 4 exactly that width wins (every wider one
    needs as many waves for wider tiles, the next narrower one a second wave), and the last tile
    of the ragged d_ff is cut.  Integer inputs: bit-exact against the oracle on all rows."""
    require_gpu()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    T, d, N = 100, 192, sms * width - 4
    rng = np.random.default_rng(width)
    mk = lambda *s: torch.from_numpy(rng.integers(-3, 4, size=s).astype(np.float32)).to(torch.bfloat16).cuda()
    X, w_up = mk(T, d), mk(N, d)
    w_gate = mk(N, d) if gated else None
    b_up = None if gated else mk(N)
    kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
    A = _tc(X, kind, w_up, w_gate, b_up).cpu().numpy()
    H_o, _ = oracle.ffn_dense(to_f32_np(X), kind, to_f32_np(w_up), to_f32_np(w_gate), np.zeros((d, N), np.float32),
                              to_f32_np(b_up), None, want_y=False)
    np.testing.assert_array_equal(A, H_o)


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("gated", [False, True])
def test_sixteen_bit_output_and_selection_on_it(out_dtype, gated):
    """The activations written as bf16 / fp16 (one rounding after the activation; half the bytes):
    integer inputs give the exactly rounded tensor; a full-width ragged layer stays within the
    16-bit tolerance of the oracle and the selection on the stored values is bit-exact."""
    require_gpu()
    rng = np.random.default_rng(11)
    T, d, N = 150, 256, 1004
    mk = lambda *s: torch.from_numpy(rng.integers(-4, 5, size=s).astype(np.float32)).to(torch.bfloat16).cuda()
    X, w_up = mk(T, d), mk(N, d)
    w_gate = mk(N, d) if gated else None
    kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
    ld = (N + 7) // 8 * 8
    buf = torch.full((T, ld), float("nan"), dtype=out_dtype, device="cuda")
    A = buf[:, :N]
    ws = torch.empty(ci.coreinfer_prefill_activations_workspace_bytes(), dtype=torch.uint8, device="cuda")
    ci.coreinfer_prefill_activations(X, kind, w_up, w_gate, None, A, ws)
    ci.coreinfer_workspace_status(ws)
    H_o, _ = oracle.ffn_dense(to_f32_np(X), kind, to_f32_np(w_up), to_f32_np(w_gate), np.zeros((d, N), np.float32),
                              want_y=False)
    expect = torch.from_numpy(H_o).to(out_dtype).to(torch.float32).numpy()     # round to nearest even, once
    got = A.to(torch.float32).cpu().numpy()
    np.testing.assert_array_equal(got, expect)
    assert torch.isnan(buf[:, N:].float()).all()                              # the padding is not written

    g = torch.Generator().manual_seed(5)
    mkr = lambda *s, std=1.0: (torch.randn(*s, generator=g) * std).to(torch.bfloat16).cuda()
    T, d, N = 260, 512, 3000
    X, w_up = mkr(T, d), mkr(N, d, std=0.05)
    w_gate = mkr(N, d, std=0.05) if gated else None
    A = torch.empty((T, N), dtype=out_dtype, device="cuda")
    ci.coreinfer_prefill_activations(X, kind, w_up, w_gate, None, A, ws)
    ci.coreinfer_workspace_status(ws)
    H_o, _ = oracle.ffn_dense(to_f32_np(X), kind, to_f32_np(w_up), to_f32_np(w_gate), np.zeros((d, N), np.float32),
                              want_y=False)
    A32 = A.to(torch.float32).cpu().numpy()
    # one rounding of an fp32 result that itself is within 1e-4 (relative to the RMS) of the oracle's
    rms = float(np.sqrt(np.mean(H_o.astype(np.float64) ** 2)))
    bound = 0.5 * torch.finfo(out_dtype).eps * np.abs(H_o) * 1.001 + 2e-4 * rms
    assert (np.abs(A32 - H_o) <= bound).all()
    S, f = gpu_select(A, 0.4, 0.2)
    S_o, f_o = oracle.select(A32, 0.4, 0.2)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)
