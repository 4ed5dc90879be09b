"""Decode FFN kernels vs the oracle (Section 4.2): within 1e-4 (fp32, relative) and 1e-2 of
the output RMS (bf16); bit-exact where the arithmetic is exact in any order."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from paper_2410_18311_b200 import workloads as wl
from helpers import require_gpu, gpu_decode, to_f32_np, assert_ffn_close, rel_err_rms

pytestmark = pytest.mark.gpu


def _rand_layer(d, K, gated, dtype, seed, bias):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s, std=0.05: (torch.randn(*s, generator=g) * std).to(dtype)
    up, down = mk(K, d), mk(K, d)
    gate = mk(K, d) if gated else None
    bup = mk(K, std=0.5) if (bias and not gated) else None
    bdown = mk(d, std=0.5) if bias else None
    return up, gate, down, bup, bdown


def _run_case(B, d, K, gated, dtype, seed=0, bias=True):
    require_gpu()
    up, gate, down, bup, bdown = _rand_layer(d, K, gated, dtype, seed, bias)
    x = torch.randn(B, d, generator=torch.Generator().manual_seed(seed + 1)).to(dtype)
    kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
    cu = lambda t: None if t is None else t.cuda()
    y = gpu_decode(cu(x), kind, cu(up), cu(gate), cu(down), cu(bup), cu(bdown))
    y_o = oracle.ffn(to_f32_np(x), kind, to_f32_np(up), to_f32_np(gate), to_f32_np(down),
                     to_f32_np(bup), to_f32_np(bdown))
    assert np.isfinite(y).all()
    assert_ffn_close(y, y_o, dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("d,K", [(8, 1), (64, 7), (768, 615), (1032, 150), (4096, 333), (5120, 301), (9216, 160),
                                 (256, 5000)])
def test_batch1(dtype, gated, d, K):
    if dtype == torch.float32 and d * 4 > 32768:
        pytest.skip("rows wider than 32 KiB are not built (no fp32 configuration needs them)")
    _run_case(1, d, K, gated, dtype, seed=d + K)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("B", [2, 3, 8])
def test_small_batches(dtype, gated, B):
    _run_case(B, 1024, 333, gated, dtype, seed=B)
    _run_case(B, 72 * (2 if dtype == torch.float32 else 1), 65, gated, dtype, seed=B + 10)


@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("B,d,K", [(5, 2048, 20), (8, 4096, 611), (2, 256, 1), (7, 3072, 150), (8, 4096 + 256, 40)])
def test_batches_on_the_tensor_core_path_and_beside_it(gated, B, d, K):
    """bf16 rows that are a multiple of 256 columns up to 4096 take the mma kernel (K smaller than
    the SM count, ragged K, every batch size); 4352 columns fall back to the plain kernels."""
    _run_case(B, d, K, gated, torch.bfloat16, seed=B * 1000 + K)


def test_no_bias_pointers():
    _run_case(1, 512, 100, False, torch.bfloat16, bias=False)
    _run_case(4, 512, 100, True, torch.bfloat16, bias=False)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("B", [1, 8])
def test_integer_valued_case_is_bit_exact(dtype, gated, B):
    """|values| <= 4 integers: every product and partial sum is exact in fp32 in any order."""
    require_gpu()
    rng = np.random.default_rng(3)
    d, K = 256, 200
    mk = lambda *s: torch.from_numpy(rng.integers(-4, 5, size=s).astype(np.float32)).to(dtype)
    up, down, x = mk(K, d), mk(K, d), mk(B, d)
    gate = mk(K, d) if gated else None
    bup = None if gated else mk(K)
    bdown = mk(d)
    kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
    cu = lambda t: None if t is None else t.cuda()
    y = gpu_decode(cu(x), kind, cu(up), cu(gate), cu(down), cu(bup), cu(bdown))
    y_o = oracle.ffn(to_f32_np(x), kind, to_f32_np(up), to_f32_np(gate), to_f32_np(down),
                     to_f32_np(bup), to_f32_np(bdown))
    np.testing.assert_array_equal(y, y_o)


def test_stack_layers_teacher_forced():
    """The persistent multi-layer launch: every layer's output is checked against the oracle on
    the very input that layer consumed, and the glue between layers against the oracle's."""
    require_gpu()
    for dtype, gated, d, K, L in [(torch.bfloat16, False, 1024, 301, 5), (torch.bfloat16, True, 512, 77, 3),
                                  (torch.float32, False, 768, 615, 4), (torch.bfloat16, False, 4096, 700, 6)]:
        layers_cpu = [_rand_layer(d, K + 3 * l, gated, dtype, 100 + l, bias=not gated) for l in range(L)]
        layers_gpu = [tuple(None if t is None else t.cuda() for t in ly) for ly in layers_cpu]
        x0 = torch.randn(1, d, generator=torch.Generator().manual_seed(9)).to(dtype)
        kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
        y_last = torch.full((1, d), float("nan"), device="cuda")
        y_layers = torch.full((L, 1, d), float("nan"), device="cuda")
        x_layers = torch.zeros((L, 1, d), dtype=dtype, device="cuda")
        ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(L, 1, d, K + 3 * L), dtype=torch.uint8,
                         device="cuda")
        arr = ci.binding.make_layers(layers_gpu)
        for _ in range(2):          # a second call on the same workspace must give the same answer
            ci.coreinfer_ffn_decode_stack(arr, x0.cuda(), kind, y_last, y_layers, x_layers, ws)
            ci.coreinfer_workspace_status(ws)
            yl, xl = y_layers.cpu().numpy(), to_f32_np(x_layers)
            np.testing.assert_array_equal(xl[0], to_f32_np(x0))
            # same partial sums, added in two different orders
            np.testing.assert_allclose(y_last.cpu().numpy(), yl[L - 1], rtol=1e-4, atol=1e-5)
            for l in range(L):
                up, gate, down, bup, bdown = (to_f32_np(t) for t in layers_cpu[l])
                y_o = oracle.ffn(xl[l], kind, up, gate, down, bup, bdown)
                assert_ffn_close(yl[l], y_o, dtype)
                if l + 1 < L:
                    x_next = torch.from_numpy(oracle.glue(xl[l], yl[l])).to(dtype).float().numpy()
                    # identical up to one rounding step of the layer-input type
                    tol = 1e-5 if dtype == torch.float32 else 2 ** -7
                    np.testing.assert_allclose(xl[l + 1][0], x_next, rtol=tol, atol=tol)


@pytest.mark.parametrize("B", [2, 5, 8])
def test_stack_of_small_batches_teacher_forced(B):
    """The stack for 2..8 sequences that share the core sets (one batched FFN and one glue launch
    per layer): every layer's output for every sequence against the oracle on the input that layer
    consumed, and the glue per sequence against the oracle's.  Covers the tensor-core kernel
    (bf16, d_model a multiple of 256) and the plain batched kernels (fp32; bf16 d_model 384)."""
    require_gpu()
    for dtype, gated, d, K, L in [(torch.bfloat16, True, 512, 300, 3), (torch.bfloat16, False, 1024, 257, 4),
                                  (torch.float32, False, 768, 200, 3), (torch.bfloat16, False, 384, 100, 2)]:
        layers_cpu = [_rand_layer(d, K + 3 * l, gated, dtype, 300 + l, bias=not gated) for l in range(L)]
        layers_gpu = [tuple(None if t is None else t.cuda() for t in ly) for ly in layers_cpu]
        x0 = torch.randn(B, d, generator=torch.Generator().manual_seed(19)).to(dtype)
        kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
        arr = ci.binding.make_layers(layers_gpu)
        ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(L, B, d, K + 3 * L), dtype=torch.uint8,
                         device="cuda")
        y_last = torch.full((B, d), float("nan"), device="cuda")
        y_layers = torch.full((L, B, d), float("nan"), device="cuda")
        x_layers = torch.zeros((L, B, d), dtype=dtype, device="cuda")
        ci.coreinfer_ffn_decode_stack(arr, x0.cuda(), kind, y_last, y_layers, x_layers, ws)
        ci.coreinfer_workspace_status(ws)
        yl, xl = y_layers.cpu().numpy(), to_f32_np(x_layers)
        np.testing.assert_array_equal(xl[0], to_f32_np(x0))
        np.testing.assert_array_equal(y_last.cpu().numpy(), yl[L - 1])
        for l in range(L):
            up, gate, down, bup, bdown = (to_f32_np(t) for t in layers_cpu[l])
            y_o = oracle.ffn(xl[l], kind, up, gate, down, bup, bdown)
            assert_ffn_close(yl[l], y_o, dtype)
            if l + 1 < L:
                tol = 1e-5 if dtype == torch.float32 else 2 ** -7
                for b in range(B):
                    x_next = torch.from_numpy(oracle.glue(xl[l][b], yl[l][b])).to(dtype).float().numpy()
                    np.testing.assert_allclose(xl[l + 1][b], x_next, rtol=tol, atol=tol)
        # without the per-layer dumps the result is the same up to the order of the sums
        y2 = torch.empty((B, d), device="cuda")
        ws.fill_(0xFF)      # NaN patterns: a y buffer of the workspace that nobody cleared would show
        ci.coreinfer_ffn_decode_stack(arr, x0.cuda(), kind, y2, None, None, ws)
        ci.coreinfer_workspace_status(ws)
        from helpers import rel_err_rms
        assert rel_err_rms(y2.cpu().numpy(), y_last.cpu().numpy()) < 0.05      # rounding flips of x may amplify over layers


def test_stack_matches_layer_by_layer_calls():
    require_gpu()
    cfg = wl.CONFIGS["opt6.7b"].with_(L=3)
    K = 410
    layers = [wl.compacted_weights_random(cfg, l, K, device="cuda") for l in range(cfg.L)]
    arr = ci.binding.make_layers([(u, g, dn, None, None) for (u, g, dn) in layers])
    x0 = wl.decode_input(cfg, 0, device="cuda")
    d = cfg.d_model
    y_last = torch.empty((1, d), device="cuda")
    x_layers = torch.empty((cfg.L, 1, d), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(cfg.L, 1, d, K), dtype=torch.uint8, device="cuda")
    ci.coreinfer_ffn_decode_stack(arr, x0, ci.FFN_RELU, y_last, None, x_layers, ws)
    ci.coreinfer_workspace_status(ws)
    u, g, dn = layers[-1]
    y_single = gpu_decode(x_layers[-1], ci.FFN_RELU, u, None, dn)
    assert rel_err_rms(y_last.cpu().numpy(), y_single) < 1e-4
