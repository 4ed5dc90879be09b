"""Compaction kernels vs the oracle: byte-identical buffers."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from helpers import require_gpu, gpu_compact, raw_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("gated,bias", [(False, True), (True, False), (False, False)])
@pytest.mark.parametrize("d,N,K", [(8, 16, 16), (64, 200, 1), (72, 333, 41), (768, 3072, 615), (1024, 4100, 1025)])
def test_compact_bytes(dtype, gated, bias, d, N, K):
    require_gpu()
    if dtype == torch.float32 and d % 4 or dtype == torch.bfloat16 and d % 8:
        pytest.skip("row not a multiple of 16 bytes")
    g = torch.Generator().manual_seed(d * N + K)
    mk = lambda *s: torch.randn(*s, generator=g).to(dtype)
    w_up, w_down = mk(N, d), mk(d, N)
    w_gate = mk(N, d) if gated else None
    b_up = mk(N) if bias else None
    S_np = np.sort(np.random.default_rng(K).permutation(N)[:K]).astype(np.int32)
    cu = lambda t: None if t is None else t.cuda()
    up_c, gate_c, down_c, bup_c = gpu_compact(cu(w_up), cu(w_gate), cu(w_down), cu(b_up),
                                              torch.from_numpy(S_np).cuda())
    o_up, o_gate, o_down, o_bup = oracle.compact(raw_np(w_up), raw_np(w_gate), raw_np(w_down), raw_np(b_up), S_np)
    assert raw_np(up_c).tobytes() == o_up.tobytes()
    assert raw_np(down_c).tobytes() == o_down.tobytes()
    if gated:
        assert raw_np(gate_c).tobytes() == o_gate.tobytes()
    if bias:
        assert raw_np(bup_c).tobytes() == o_bup.tobytes()


def test_verify_core_idx_reports_the_first_bad_position():
    """The index check that guards coreinfer_compact (which trusts its list): a valid list passes,
    and every kind of defect -- out of range, negative, repeated, descending -- is counted and
    located.  Only the list itself is read, so bad lists are safe to test."""
    require_gpu()
    d_ff = 1000
    good = torch.arange(0, 900, 3, dtype=torch.int32, device="cuda")
    report = torch.empty(2, dtype=torch.int32, device="cuda")
    ci.coreinfer_verify_core_idx(good, d_ff, report)
    assert report.cpu().tolist() == [0, 2 ** 31 - 1]
    S_o, _ = oracle.select(np.abs(np.random.default_rng(0).standard_normal((7, d_ff))).astype(np.float32), 0.4, 0.2)
    ci.coreinfer_verify_core_idx(torch.from_numpy(S_o).cuda(), d_ff, report)      # a set as the oracle emits it
    assert report.cpu().tolist() == [0, 2 ** 31 - 1]
    for pos, val, nbad in [(17, 1000, 2), (0, -1, 1), (40, 40 * 3 - 3, 1), (299, 5, 1), (120, 2 ** 31 - 1, 2)]:
        bad = good.clone()
        bad[pos] = val
        ci.coreinfer_verify_core_idx(bad, d_ff, report)
        n, first = report.cpu().tolist()
        assert first == pos and n == nbad, (pos, val, n, first)
