"""Parity at the shapes of the five workload configurations that the smaller tests do not reach:
the one-group instantiations of the batch-1 stack kernel (rows wider than 8 KB) across layers,
the beta sweep of the OPT-13B-shaped layer, the long-prompt selection of the OPT-66B-shaped
layer, and the full gated stack at batch 1.  Everything is compared with the oracle on
identical inputs: sets and counts bit-exact, compacted bytes identical, FFN outputs within
1e-2 of the output RMS (bf16), per layer on the input that layer consumed."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from paper_2410_18311_b200 import workloads as wl
from helpers import (require_gpu, gpu_select, gpu_compact, gpu_decode, to_f32_np, raw_np, assert_ffn_close,
                     check_stack_teacher_forced)

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rand_layers(d, Ks, gated, dtype, seed, bias):
    out = []
    for l, K in enumerate(Ks):
        g = torch.Generator().manual_seed(seed + l)
        mk = lambda *s, std=0.05: (torch.randn(*s, generator=g) * std).to(dtype).cuda()
        up, down = mk(K, d), mk(K, d)
        gate = mk(K, d) if gated else None
        bup = mk(K, std=0.5) if (bias and not gated) else None
        bdown = mk(d, std=0.5) if bias else None
        out.append((up, gate, down, bup, bdown))
    return out


@pytest.mark.parametrize("d,gated", [(5120, False), (5120, True), (9216, False), (9216, True), (6144, False)])
def test_wide_rows_across_layers_teacher_forced(d, gated):
    """Rows of 10, 12 and 18 KB run one consumer group (three or five 16-byte vectors per thread):
    five layers with ragged slabs of two to four neurons per CTA, so that the rotating reduction
    targets, the producer's run-ahead into the next layer and the step between layers of these
    instantiations all run, with biases."""
    require_gpu()
    Ks = [2 * 148 + 11 + 37 * l for l in range(5)]
    layers = _rand_layers(d, Ks, gated, torch.bfloat16, 7000 + d, bias=True)
    x0 = torch.randn(1, d, generator=torch.Generator().manual_seed(d)).to(torch.bfloat16).cuda()
    kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
    for _ in range(2):
        check_stack_teacher_forced(layers, x0, kind, torch.bfloat16)


def test_opt66b_shaped_six_layer_cut_at_full_k():
    """Six layers of the OPT-66B-shaped stack at the full K = 7373 (49 or 50 rows of 18 KB per
    CTA and layer): every layer against the oracle on the input it consumed."""
    require_gpu()
    cfg = wl.CONFIGS["opt66b"].with_(L=6)
    K = ci.coreinfer_count(cfg.beta, cfg.d_ff)
    assert K == 7373
    layers = [wl.compacted_weights_random(cfg, l, K, device="cuda") for l in range(cfg.L)]
    layers = [(u, g, dn, None, None) for (u, g, dn) in layers]
    x0 = wl.decode_input(cfg, 0, device="cuda")
    check_stack_teacher_forced(layers, x0, ci.FFN_RELU, torch.bfloat16)


def test_opt13b_shaped_eight_layer_cut_at_full_k():
    """Eight layers of the OPT-13B-shaped stack at K = 4096 (27 or 28 rows of 10 KB per CTA)."""
    require_gpu()
    cfg = wl.CONFIGS["opt13b"].with_(L=8)
    K = ci.coreinfer_count(cfg.beta, cfg.d_ff)
    assert K == 4096
    layers = [wl.compacted_weights_random(cfg, l, K, device="cuda") for l in range(cfg.L)]
    layers = [(u, g, dn, None, None) for (u, g, dn) in layers]
    x0 = wl.decode_input(cfg, 0, device="cuda")
    check_stack_teacher_forced(layers, x0, ci.FFN_RELU, torch.bfloat16)


@pytest.mark.parametrize("beta,K", [(0.1, 2048), (0.4, 8192), (1.0, 20480)])
def test_opt13b_shaped_layer_beta_sweep(beta, K):
    """One full-size OPT-13B-shaped layer (d_model 5120, d_ff 20480, T 512) at the other points
    of the beta sweep: set and counts bit-exact on the kernel's own activations, compacted bytes
    identical, decode within tolerance; beta = 1 is also the dense FFN."""
    require_gpu()
    cfg = wl.CONFIGS["opt13b"]
    layer = 11
    X = wl.prompt_hidden(cfg, device="cuda")
    w_up, _, w_down = wl.layer_weights(cfg, layer, device="cuda")
    H = torch.empty((cfg.T, cfg.d_ff), device="cuda")
    ci.coreinfer_ffn_dense_ref(X, ci.FFN_RELU, w_up, None, w_down, None, None, H, None)
    S, f = gpu_select(H, cfg.alpha, beta)
    S_o, f_o = oracle.select(H.cpu().numpy(), cfg.alpha, beta)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)
    assert len(S) == K == ci.coreinfer_count(beta, cfg.d_ff)
    up_c, _, down_c, _ = gpu_compact(w_up, None, w_down, None, torch.from_numpy(S).cuda())
    o_up, _, o_down, _ = oracle.compact(raw_np(w_up), None, raw_np(w_down), None, S_o)
    assert raw_np(up_c).tobytes() == o_up.tobytes() and raw_np(down_c).tobytes() == o_down.tobytes()
    x = wl.decode_input(cfg, layer, device="cuda")
    y = gpu_decode(x, ci.FFN_RELU, up_c, None, down_c)
    y_o = oracle.ffn(to_f32_np(x), ci.FFN_RELU, to_f32_np(up_c), None, to_f32_np(down_c))
    assert_ffn_close(y, y_o, torch.bfloat16)
    if beta == 1.0:
        np.testing.assert_array_equal(S, np.arange(cfg.d_ff))
        _, Y_o = oracle.ffn_dense(to_f32_np(x), ci.FFN_RELU, to_f32_np(w_up), None, to_f32_np(w_down), want_h=False)
        assert_ffn_close(y, Y_o, torch.bfloat16)


@pytest.mark.parametrize("T", [2048, 4096])
def test_opt66b_shaped_selection_long_prompts(T):
    """d_ff = 36864 with 14 or 28 rows per CTA (byte counters, the row's entries held in
    registers): set and counts bit-exact, planted subset inside the set."""
    require_gpu()
    cfg = wl.CONFIGS["opt66b"]
    A, core = wl.planted_activations(cfg, 1, T, device="cuda")
    S, f = gpu_select(A, cfg.alpha, cfg.beta)
    S_o, f_o = oracle.select(A.cpu().numpy(), cfg.alpha, cfg.beta)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)
    assert len(S) == 7373 and np.isin(core.cpu().numpy(), S).all()


def test_full_size_gated_stack_at_batch_one():
    """The ReLU-Llama-2-7B-shaped stack (32 gated layers, K = 2752) at batch 1 in one launch:
    sampled layers against the oracle on the inputs they consumed."""
    require_gpu()
    cfg = wl.CONFIGS["relu-llama2-7b"]
    K = ci.coreinfer_count(cfg.beta, cfg.d_ff)
    assert K == 2752
    layers = [wl.compacted_weights_random(cfg, l, K, device="cuda") for l in range(cfg.L)]
    layers = [(u, g, dn, None, None) for (u, g, dn) in layers]
    x0 = wl.decode_input(cfg, 0, device="cuda")
    check_stack_teacher_forced(layers, x0, ci.FFN_RELU_GATED, torch.bfloat16, layers_to_check=(0, 1, 9, 22, 30, 31))


@pytest.mark.parametrize("slots", [8, 16])
def test_stacks_on_a_ring_of_a_few_slots(slots):
    """With the ring capped at a few slots it wraps several times per layer and, since slab
    sizes are not multiples of the batch, a phase rarely ends on a batch boundary: the cases in
    which consumer groups would trade slots if batches were not pinned to ring positions.  The
    cap is read from the environment when the library is first used, hence the child process."""
    require_gpu()
    env = dict(os.environ, COREINFER_RING_SLOTS=str(slots))
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_decode.py") + "::test_stack_layers_teacher_forced",
           os.path.join(ROOT, "tests", "test_gpu_configs.py") + "::test_wide_rows_across_layers_teacher_forced",
           os.path.join(ROOT, "tests", "test_gpu_configs.py") + "::test_two_group_stack_with_odd_slabs"]
    res = subprocess.run(cmd, env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]


def test_two_group_stack_with_odd_slabs():
    """Rows of 2 to 8 KB (two consumer groups) with 22 or 23 neurons per CTA, gated and not,
    six layers: slab sizes that are no multiple of the batch of 4, so every phase ends in a
    batch that is partly empty."""
    require_gpu()
    for d, gated in [(4096, False), (4096, True), (2048, False), (1024, True)]:
        Ks = [22 * 148 + 21 + 13 * l for l in range(6)]
        layers = _rand_layers(d, Ks, gated, torch.bfloat16, 9000 + d, bias=not gated)
        x0 = torch.randn(1, d, generator=torch.Generator().manual_seed(d + 1)).to(torch.bfloat16).cuda()
        check_stack_teacher_forced(layers, x0, ci.FFN_RELU_GATED if gated else ci.FFN_RELU, torch.bfloat16)


@pytest.mark.parametrize("dtype,kind", [(torch.float16, "silu"), (torch.bfloat16, "silu"), (torch.float16, "relu_gated")])
def test_llama_shaped_layer_with_silu_gate_and_fp16(dtype, kind):
    """One full-size Llama-2-7B-shaped layer (d_model 4096, d_ff 11008, T 1024) of the second
    workload family: tensor-core activations with the SiLU gate, selection on them (they carry
    negative entries), compaction, decode at 1 and 8 sequences; and eight layers of the stack."""
    require_gpu()
    cfg = wl.CONFIGS["relu-llama2-7b"]
    k = ci.FFN_SILU_GATED if kind == "silu" else ci.FFN_RELU_GATED
    X = wl.prompt_hidden(cfg, device="cuda").to(dtype)
    w_up, w_gate, w_down = (t.to(dtype) for t in wl.layer_weights(cfg, 5, device="cuda"))
    A = torch.empty((cfg.T, cfg.d_ff), device="cuda")
    tws = torch.empty(ci.coreinfer_prefill_activations_workspace_bytes(), dtype=torch.uint8, device="cuda")
    ci.coreinfer_prefill_activations(X, k, w_up, w_gate, None, A, tws)
    ci.coreinfer_workspace_status(tws)
    rows = [0, 500, cfg.T - 1]
    H_o, _ = oracle.ffn_dense(to_f32_np(X[rows]), k, to_f32_np(w_up), to_f32_np(w_gate),
                              np.zeros((cfg.d_model, cfg.d_ff), np.float32), want_y=False)
    assert_ffn_close(A[rows].cpu().numpy(), H_o, torch.float32)
    S, f = gpu_select(A, cfg.alpha, cfg.beta)
    S_o, f_o = oracle.select(A.cpu().numpy(), cfg.alpha, cfg.beta)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)
    up_c, gate_c, down_c, _ = gpu_compact(w_up, w_gate, w_down, None, torch.from_numpy(S).cuda())
    o_up, o_gate, o_down, _ = oracle.compact(raw_np(w_up), raw_np(w_gate), raw_np(w_down), None, S_o)
    assert raw_np(up_c).tobytes() == o_up.tobytes() and raw_np(gate_c).tobytes() == o_gate.tobytes()
    assert raw_np(down_c).tobytes() == o_down.tobytes()
    for B in (1, 8):
        x = wl.decode_input(cfg, 3, device="cuda", batch=B).to(dtype)
        y = gpu_decode(x, k, up_c, gate_c, down_c)
        y_o = oracle.ffn(to_f32_np(x), k, to_f32_np(up_c), to_f32_np(gate_c), to_f32_np(down_c))
        assert_ffn_close(y, y_o, dtype)
    K = len(S)
    layers = [tuple(t if t is None else t.to(dtype) for t in wl.compacted_weights_random(cfg.with_(L=8), l, K, device="cuda")) + (None, None)
              for l in range(8)]
    check_stack_teacher_forced(layers, wl.decode_input(cfg, 0, device="cuda").to(dtype), k, dtype, layers_to_check=(0, 3, 7))
