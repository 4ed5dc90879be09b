"""The workspace-free stack entry point (for callers that cannot allocate device memory while
decoding) must give what the workspace variant gives, and what the oracle gives.  Collected last
on purpose: a run that stops at the first failure has then already exercised every other test."""
import numpy as np
import pytest
import torch

import paper_2410_18311_b200 as ci
from paper_2410_18311_b200 import workloads as wl
from helpers import require_gpu, assert_ffn_close, check_stack_teacher_forced

pytestmark = pytest.mark.gpu


def _stack(cfg, K):
    layers = [wl.compacted_weights_random(cfg, l, K, device="cuda") for l in range(cfg.L)]
    return layers, ci.binding.make_layers([(u, g, dn, None, None) for (u, g, dn) in layers])


def test_noalloc_matches_workspace_variant_twice_in_a_row():
    require_gpu()
    cfg = wl.CONFIGS["opt6.7b"].with_(L=4, d_model=2048)
    K, d, L = 333, cfg.d_model, cfg.L
    keep, arr = _stack(cfg, K)
    ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(L, 1, d, K), dtype=torch.uint8, device="cuda")
    for call in range(2):                      # the second call finds the first one's leftovers in the scratch
        x0 = wl.decode_input(cfg, call, device="cuda")
        y_ref = torch.full((1, d), float("nan"), device="cuda")
        yl_ref = torch.full((L, 1, d), float("nan"), device="cuda")
        ci.coreinfer_ffn_decode_stack(arr, x0, ci.FFN_RELU, y_ref, yl_ref, None, ws)
        ci.coreinfer_workspace_status(ws)
        y = torch.full((1, d), float("nan"), device="cuda")
        yl = torch.full((L, 1, d), float("nan"), device="cuda")
        xl = torch.zeros((L, 1, d), dtype=torch.bfloat16, device="cuda")
        ci.coreinfer_ffn_decode_stack_noalloc(arr, x0, ci.FFN_RELU, y, yl, xl)
        torch.cuda.synchronize()
        assert torch.isfinite(y).all() and torch.isfinite(yl).all()
        assert torch.equal(xl[0], x0)
        assert_ffn_close(y.cpu().numpy(), y_ref.cpu().numpy(), torch.bfloat16)
        for l in range(L):
            assert_ffn_close(yl[l].cpu().numpy(), yl_ref[l].cpu().numpy(), torch.bfloat16)
        # and against the oracle, layer by layer on the inputs the layers consumed (its private
        # status word cannot be read back, so a wait that gave up would show here as a mismatch)
        check_stack_teacher_forced([(u, g, dn, None, None) for (u, g, dn) in keep], x0, ci.FFN_RELU,
                                   torch.bfloat16, noalloc=True)
    del keep


def test_noalloc_rejects_shapes_beyond_its_scratch():
    require_gpu()
    cfg = wl.CONFIGS["opt6.7b"].with_(L=2, d_model=16384)        # 256 + 12 * 16384 B = 192 KiB > 128 KiB
    up, _, down = wl.compacted_weights_random(cfg, 0, 8, device="cuda")
    arr = ci.binding.make_layers([(up, None, down, None, None)] * cfg.L)
    x0 = wl.decode_input(cfg, 0, device="cuda")
    y = torch.zeros((1, cfg.d_model), device="cuda")
    with pytest.raises(ci.CoreInferError) as err:
        ci.coreinfer_ffn_decode_stack_noalloc(arr, x0, ci.FFN_RELU, y, None, None)
    assert err.value.status == ci.ERR_UNSUPPORTED and "scratch" in str(err.value)
    torch.cuda.synchronize()
    assert float(y.abs().sum()) == 0.0         # nothing was enqueued
