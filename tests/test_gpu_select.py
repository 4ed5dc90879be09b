"""Selection kernels vs the oracle: index sets and counts bit-exact (Definition 1 / Eq. 1,
Eq. 3, Definition 2 / Eq. 2)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from paper_2410_18311_b200 import workloads as wl
from conftest import load_hand_example
from helpers import require_gpu, gpu_select

pytestmark = pytest.mark.gpu


def _check(A_np, alpha, beta):
    S_o, f_o = oracle.select(A_np, alpha, beta)
    S, f = gpu_select(torch.from_numpy(np.ascontiguousarray(A_np)).cuda(), alpha, beta)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)


def _pad_rows(A, mult=4):
    """rows must have a stride that is a multiple of 4 elements"""
    T, N = A.shape
    ld = (N + mult - 1) // mult * mult
    buf = np.full((T, ld), 7.0, dtype=np.float32)      # positive garbage in the padding must be ignored
    buf[:, :N] = A
    return buf


def test_hand_worked_example():
    require_gpu()
    A, cases = load_hand_example()
    for alpha, beta, f_exp, S_exp in cases:
        S, f = gpu_select(torch.from_numpy(A).cuda(), alpha, beta)
        np.testing.assert_array_equal(f, f_exp)
        np.testing.assert_array_equal(S, S_exp)


@pytest.mark.parametrize("T,N,alpha,beta", [
    (1, 4, 0.4, 0.2), (3, 8, 0.5, 0.5), (7, 260, 0.4, 0.2), (33, 1000, 0.4, 0.25),
    (64, 3072, 0.4, 0.2), (5, 4100, 0.1, 0.4), (300, 4096 + 8, 0.4, 0.2), (16, 512, 1.0, 1.0),
    (20, 11008, 0.4, 0.25), (9, 20480, 0.4, 0.1), (6, 36864, 0.4, 0.2), (4, 24580, 0.4, 0.2),
])
def test_random_rows(T, N, alpha, beta):
    require_gpu()
    rng = np.random.default_rng(T * 7919 + N)
    A = rng.standard_normal((T, N)).astype(np.float32)
    A[rng.random((T, N)) < 0.2] = 0.0
    _check(A, alpha, beta)


@pytest.mark.parametrize("T,N", [(5, 64), (40, 1024), (17, 5000), (12, 16384), (3, 36864)])
def test_quantised_rows_heavy_ties(T, N):
    """Values on a coarse grid: the token threshold falls inside a group of equal values,
    so the lower-index rule decides."""
    require_gpu()
    rng = np.random.default_rng(N + T)
    A = (rng.integers(-3, 6, size=(T, N)) * 0.25).astype(np.float32)
    _check(A, 0.4, 0.2)
    _check(A, 0.5, 0.5)


def test_row_stride_and_ragged_width():
    require_gpu()
    rng = np.random.default_rng(5)
    for N in (1, 2, 3, 5, 257, 1001, 4099):
        A = rng.standard_normal((6, N)).astype(np.float32)
        buf = _pad_rows(A)
        dev = torch.from_numpy(buf).cuda()
        K = ci.coreinfer_count(0.3, N)
        S = torch.empty(K, dtype=torch.int32, device="cuda")
        f = torch.empty(N, dtype=torch.int32, device="cuda")
        ws = torch.empty(ci.coreinfer_select_workspace_bytes(6, N), dtype=torch.uint8, device="cuda")
        ci.coreinfer_select_core(dev, 0.4, 0.3, S, f, ws, T=6, d_ff=N, ld_act=buf.shape[1])
        ci.coreinfer_workspace_status(ws)
        S_o, f_o = oracle.select(A, 0.4, 0.3)
        np.testing.assert_array_equal(f.cpu().numpy(), f_o)
        np.testing.assert_array_equal(S.cpu().numpy(), S_o)


def test_special_floats_and_degenerate_rows():
    require_gpu()
    sub = np.float32(1e-45)
    A = np.zeros((5, 16), dtype=np.float32)
    A[0, :8] = [np.nan, np.inf, -np.inf, 0.0, -0.0, sub, 1.0, -sub]
    A[1] = -1.0                                   # no positive entry
    A[2] = 2.5                                    # all equal
    A[3, 3] = np.float32(3e-39)                   # a single subnormal
    A[4] = np.linspace(-1, 1, 16, dtype=np.float32)
    for alpha, beta in [(0.4, 0.2), (1.0, 1.0), (0.34, 0.5)]:
        _check(A, alpha, beta)
    _check(-np.abs(A), 0.4, 0.25)                 # nothing positive anywhere: f = 0, S = lowest K


def test_many_rows_per_cta_and_alpha_beta_extremes():
    require_gpu()
    rng = np.random.default_rng(11)
    A = rng.standard_normal((700, 2048)).astype(np.float32)      # > 4 rows per CTA
    _check(A, 0.4, 0.2)
    _check(A[:50], 1.0, 0.001)                                   # K = ceil(2.048) = 3
    _check(A[:50], 0.0001, 1.0)                                  # k_t = 1


@pytest.mark.parametrize("T", [40000, 66000])
def test_more_rows_than_one_cta_counts_in_bytes(T):
    """The row kernel counts memberships in bytes (at most 255 rows per CTA): T = 40000 needs more
    CTAs than there are SMs for that, T = 66000 is beyond it and takes the kernel with wide
    counters; both also exercise the two-pass search of the top-K kernel (counts above 4095)."""
    require_gpu()
    rng = np.random.default_rng(T)
    A = rng.standard_normal((T, 64)).astype(np.float32)
    A[:, :7] = np.abs(A[:, :7]) + 3.0                            # a stable subset, so counts reach T
    _check(A, 0.4, 0.2)


def test_device_count_rule_for_every_P():
    """Row t has exactly t positives, all distinct: membership count of row t is ceil(alpha t),
    so f summed over neurons must equal the host rule for every P in 0..N."""
    require_gpu()
    N = 1200
    for alpha in (0.4, 0.1, 0.25):
        A = np.full((N + 1, N), -1.0, dtype=np.float32)
        for t in range(N + 1):
            A[t, :t] = np.arange(t, 0, -1, dtype=np.float32)      # descending: members are the lowest indices
        S, f = gpu_select(torch.from_numpy(A).cuda(), alpha, 0.2)
        k = np.array([ci.coreinfer_count(alpha, t) for t in range(N + 1)])
        f_exp = np.array([(k > n).sum() for n in range(N)])
        np.testing.assert_array_equal(f, f_exp)
        assert f.sum() == sum(oracle.count(alpha, t) for t in range(N + 1))


def test_planted_structure_config():
    """Stability structure (Section 3.2): planted subset inside the set, bit-exact vs oracle."""
    require_gpu()
    cfg = wl.CONFIGS["opt66b"].with_(d_ff=9216)
    A, core = wl.planted_activations(cfg, 0, 160, device="cuda")
    S, f = gpu_select(A, cfg.alpha, cfg.beta)
    S_o, f_o = oracle.select(A.cpu().numpy(), cfg.alpha, cfg.beta)
    np.testing.assert_array_equal(f, f_o)
    np.testing.assert_array_equal(S, S_o)
    assert np.isin(core.cpu().numpy(), S).all()


def test_same_input_same_output_twice():
    require_gpu()
    rng = np.random.default_rng(2)
    A = torch.from_numpy(rng.standard_normal((100, 3072)).astype(np.float32)).cuda()
    S1, f1 = gpu_select(A, 0.4, 0.2)
    S2, f2 = gpu_select(A, 0.4, 0.2)
    np.testing.assert_array_equal(S1, S2)
    np.testing.assert_array_equal(f1, f2)


def _sixteen_bit(A32, dtype, ld_mult=8, fill=7.0):
    """A [T, N] tensor of a 16-bit type inside a buffer whose rows are padded (with positive
    garbage) to a multiple of 8 entries; returns the CUDA view and the values widened to fp32."""
    T, N = A32.shape
    ld = (N + ld_mult - 1) // ld_mult * ld_mult
    buf = torch.full((T, ld), fill, dtype=dtype)
    buf[:, :N] = torch.from_numpy(A32).to(dtype)
    dev = buf.cuda()
    return dev[:, :N], buf[:, :N].to(torch.float32).numpy()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("T,N,alpha,beta", [
    (1, 4, 0.4, 0.2), (3, 9, 0.5, 0.5), (7, 261, 0.4, 0.2), (33, 1003, 0.4, 0.25), (64, 3072, 0.4, 0.2),
    (300, 4096 + 6, 0.4, 0.2), (20, 11008, 0.4, 0.25), (6, 36864, 0.4, 0.2), (4, 24581, 0.4, 0.2),
])
def test_sixteen_bit_activations(dtype, T, N, alpha, beta):
    """bf16 / fp16 activations are ranked as the values they store: the sets and counts equal the
    oracle's on the same values widened to fp32.  Sixteen-bit values tie often (a few hundred
    distinct values per row), so the lower-index rule decides most thresholds."""
    require_gpu()
    rng = np.random.default_rng(T * 31 + N)
    A = rng.standard_normal((T, N)).astype(np.float32)
    A[rng.random((T, N)) < 0.2] = 0.0
    view, A16 = _sixteen_bit(A, dtype)
    S_o, f_o = oracle.select(A16, alpha, beta)
    K = ci.coreinfer_count(beta, N)
    S = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    f = torch.full((N,), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty(ci.coreinfer_select_workspace_bytes(T, N), dtype=torch.uint8, device="cuda")
    ci.coreinfer_select_core(view, alpha, beta, S, f, ws, T=T, d_ff=N, ld_act=view.stride(0))
    ci.coreinfer_workspace_status(ws)
    np.testing.assert_array_equal(f.cpu().numpy(), f_o)
    np.testing.assert_array_equal(S.cpu().numpy(), S_o)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_sixteen_bit_special_values_and_many_rows(dtype):
    """Negative zero, infinities, NaN, the smallest subnormal and the largest finite value of the
    16-bit type; and enough rows (66000) that the general row kernel with 16-bit counters runs."""
    require_gpu()
    fi = torch.finfo(dtype)
    tiny_sub = float(torch.tensor(2.0 ** -133 if dtype == torch.bfloat16 else 2.0 ** -24).to(dtype))
    assert tiny_sub > 0.0
    specials = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, tiny_sub, -tiny_sub, fi.max, -fi.max, fi.tiny, 1.0, 1.0,
                         0.5, 2.0, -1.0, 3.0, 1.0], dtype=np.float32)
    rng = np.random.default_rng(3)
    A = np.stack([rng.permutation(specials) for _ in range(40)])
    for alpha, beta in ((0.4, 0.3), (1.0, 1.0), (0.1, 0.1)):
        view, A16 = _sixteen_bit(A, dtype)
        S_o, f_o = oracle.select(A16, alpha, beta)
        K = ci.coreinfer_count(beta, A.shape[1])
        S = torch.full((K,), -1, dtype=torch.int32, device="cuda")
        f = torch.full((A.shape[1],), -1, dtype=torch.int32, device="cuda")
        ws = torch.empty(ci.coreinfer_select_workspace_bytes(*A.shape), dtype=torch.uint8, device="cuda")
        ci.coreinfer_select_core(view, alpha, beta, S, f, ws, T=A.shape[0], d_ff=A.shape[1], ld_act=view.stride(0))
        ci.coreinfer_workspace_status(ws)
        np.testing.assert_array_equal(f.cpu().numpy(), f_o)
        np.testing.assert_array_equal(S.cpu().numpy(), S_o)
    T, N = 66000, 40
    A = (rng.integers(-2, 5, size=(T, N)) * 0.5).astype(np.float32)
    view, A16 = _sixteen_bit(A, dtype)
    S_o, f_o = oracle.select(A16, 0.4, 0.2)
    S = torch.full((ci.coreinfer_count(0.2, N),), -1, dtype=torch.int32, device="cuda")
    f = torch.full((N,), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty(ci.coreinfer_select_workspace_bytes(T, N), dtype=torch.uint8, device="cuda")
    ci.coreinfer_select_core(view, 0.4, 0.2, S, f, ws, T=T, d_ff=N, ld_act=view.stride(0))
    ci.coreinfer_workspace_status(ws)
    np.testing.assert_array_equal(f.cpu().numpy(), f_o)
    np.testing.assert_array_equal(S.cpu().numpy(), S_o)
