"""Dense reference FFN kernels vs the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from helpers import require_gpu, to_f32_np, assert_ffn_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("T,d,N", [(1, 8, 16), (5, 72, 130), (64, 768, 3072), (130, 256, 515)])
def test_dense_ffn(dtype, gated, T, d, N):
    require_gpu()
    g = torch.Generator().manual_seed(T + d + N)
    mk = lambda *s, std=0.05: (torch.randn(*s, generator=g) * std).to(dtype)
    w_up, w_down = mk(N, d), mk(d, N)
    w_gate = mk(N, d) if gated else None
    b_up = None if gated else mk(N, std=0.3)
    b_down = mk(d, std=0.3)
    x = mk(T, d, std=1.0)
    kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
    cu = lambda t: None if t is None else t.cuda()
    H = torch.full((T, N), float("nan"), device="cuda")
    Y = torch.full((T, d), float("nan"), device="cuda")
    ci.coreinfer_ffn_dense_ref(cu(x), kind, cu(w_up), cu(w_gate), cu(w_down), cu(b_up), cu(b_down), H, Y)
    torch.cuda.synchronize()
    H_o, Y_o = oracle.ffn_dense(to_f32_np(x), kind, to_f32_np(w_up), to_f32_np(w_gate), to_f32_np(w_down),
                                to_f32_np(b_up), to_f32_np(b_down))
    # the intermediate is an fp32 quantity for both input types
    assert_ffn_close(H.cpu().numpy(), H_o, torch.float32)
    assert_ffn_close(Y.cpu().numpy(), Y_o, dtype)
    # h only
    H2 = torch.empty((T, N), device="cuda")
    ci.coreinfer_ffn_dense_ref(cu(x), kind, cu(w_up), cu(w_gate), cu(w_down), cu(b_up), cu(b_down), H2, None)
    torch.cuda.synchronize()
    assert torch.equal(H, H2)
