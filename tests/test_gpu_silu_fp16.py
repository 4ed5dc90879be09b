"""The second workload family: SiLU-gated FFN (the paper's LLaMA runs) and fp16 storage (the
paper's weight type).  Every entry point against the oracle; Definition 1 is applied to
h = silu(W_gate x) * (W_up x) as it stands, so entries of h that are not positive never count."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from helpers import (require_gpu, gpu_select, gpu_compact, gpu_decode, to_f32_np, raw_np, assert_ffn_close,
                     check_stack_teacher_forced)

pytestmark = pytest.mark.gpu
KINDS = {"relu": ci.FFN_RELU, "relu_gated": ci.FFN_RELU_GATED, "silu_gated": ci.FFN_SILU_GATED}


def _layer(d, K, gated, dtype, seed, std=0.05):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: (torch.randn(*s, generator=g) * std).to(dtype).cuda()
    return mk(K, d), (mk(K, d) if gated else None), mk(K, d)


@pytest.mark.parametrize("dtype,kind", [(torch.float16, "relu"), (torch.float16, "relu_gated"), (torch.float16, "silu_gated"),
                                        (torch.bfloat16, "silu_gated"), (torch.float32, "silu_gated")])
@pytest.mark.parametrize("B,d,K", [(1, 64, 7), (1, 1032, 150), (1, 4096, 333), (1, 5120, 301), (3, 1024, 333), (8, 4096, 611),
                                   (8, 360, 77)])
def test_decode_layer(dtype, kind, B, d, K):
    require_gpu()
    gated = kind != "relu"
    up, gate, down = _layer(d, K, gated, dtype, d + K)
    x = torch.randn(B, d, generator=torch.Generator().manual_seed(B)).to(dtype).cuda()
    y = gpu_decode(x, KINDS[kind], up, gate, down)
    y_o = oracle.ffn(to_f32_np(x), KINDS[kind], to_f32_np(up), to_f32_np(gate), to_f32_np(down))
    assert np.isfinite(y).all()
    assert_ffn_close(y, y_o, dtype)


@pytest.mark.parametrize("dtype,kind,B", [(torch.float16, "silu_gated", 1), (torch.bfloat16, "silu_gated", 1),
                                          (torch.float16, "relu", 1), (torch.bfloat16, "silu_gated", 8),
                                          (torch.float16, "silu_gated", 4)])
def test_stack_teacher_forced(dtype, kind, B):
    require_gpu()
    gated = kind != "relu"
    d, L = 2048, 4
    layers = []
    for l in range(L):
        up, gate, down = _layer(d, 300 + 11 * l, gated, dtype, 50 + l)
        layers.append((up, gate, down, None, None))
    x0 = torch.randn(B, d, generator=torch.Generator().manual_seed(3)).to(dtype).cuda()
    check_stack_teacher_forced(layers, x0, KINDS[kind], dtype)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16, torch.float32])
def test_dense_reference_and_selection_on_silu_activations(dtype):
    """The dense pass with the SiLU gate, selection on its intermediate (which has negative
    entries: they are simply not positive), compaction of the selected rows, decode."""
    require_gpu()
    T, d, N = 48, 256, 1024
    g = torch.Generator().manual_seed(7)
    mk = lambda *s, std=0.05: (torch.randn(*s, generator=g) * std).to(dtype).cuda()
    X, w_up, w_gate, w_down = mk(T, d, std=1.0), mk(N, d), mk(N, d), mk(d, N)
    H = torch.empty((T, N), device="cuda")
    Y = torch.empty((T, d), device="cuda")
    ci.coreinfer_ffn_dense_ref(X, ci.FFN_SILU_GATED, w_up, w_gate, w_down, None, None, H, Y)
    torch.cuda.synchronize()
    H_o, Y_o = oracle.ffn_dense(to_f32_np(X), oracle.SILU_GATED, to_f32_np(w_up), to_f32_np(w_gate), to_f32_np(w_down))
    assert_ffn_close(H.cpu().numpy(), H_o, torch.float32)
    assert_ffn_close(Y.cpu().numpy(), Y_o, torch.float32)
    assert (H < 0).any()
    S, f = gpu_select(H, 0.4, 0.25)
    S_o, f_o = oracle.select(H.cpu().numpy(), 0.4, 0.25)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)
    up_c, gate_c, down_c, _ = gpu_compact(w_up, w_gate, w_down, None, torch.from_numpy(S).cuda())
    o_up, o_gate, o_down, _ = oracle.compact(raw_np(w_up), raw_np(w_gate), raw_np(w_down), None, S_o)
    assert raw_np(up_c).tobytes() == o_up.tobytes() and raw_np(gate_c).tobytes() == o_gate.tobytes()
    assert raw_np(down_c).tobytes() == o_down.tobytes()
    x = mk(1, d, std=1.0)
    y = gpu_decode(x, ci.FFN_SILU_GATED, up_c, gate_c, down_c)
    y_o = oracle.ffn(to_f32_np(x), oracle.SILU_GATED, to_f32_np(up_c), to_f32_np(gate_c), to_f32_np(down_c))
    assert_ffn_close(y, y_o, dtype)


@pytest.mark.parametrize("dtype,kind", [(torch.float16, "relu"), (torch.float16, "silu_gated"), (torch.bfloat16, "silu_gated")])
def test_tensor_core_prefill(dtype, kind):
    require_gpu()
    gated = kind != "relu"
    T, d, N = 200, 520, 1300
    g = torch.Generator().manual_seed(9)
    mk = lambda *s, std=0.05: (torch.randn(*s, generator=g) * std).to(dtype).cuda()
    X, w_up = mk(T, d, std=1.0), mk(N, d)
    w_gate = mk(N, d) if gated else None
    b_up = None if gated else mk(N, std=0.5)
    A = torch.full((T, N), float("nan"), device="cuda")
    ws = torch.empty(ci.coreinfer_prefill_activations_workspace_bytes(), dtype=torch.uint8, device="cuda")
    ci.coreinfer_prefill_activations(X, KINDS[kind], w_up, w_gate, b_up, A, ws)
    ci.coreinfer_workspace_status(ws)
    H_o, _ = oracle.ffn_dense(to_f32_np(X), KINDS[kind], to_f32_np(w_up), to_f32_np(w_gate), np.zeros((d, N), np.float32),
                              to_f32_np(b_up), None, want_y=False)
    assert_ffn_close(A.cpu().numpy(), H_o, torch.float32)
