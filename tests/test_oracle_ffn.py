"""Pins for the oracle's compaction, decode FFN, dense FFN and stack glue.

Expected values come from numpy indexing / float64 matmul, exact-arithmetic
integer cases, one-hot inputs worked by hand, and the identities that tie the
compacted FFN to the dense one (Section 4.2: decoding uses the dense FFN's
neurons restricted to the fixed set).
"""
import numpy as np
import pytest

import oracle


def _weights(rng, d, N, gated, scale=0.02):
    w_up = (rng.standard_normal((N, d)) * scale).astype(np.float32)
    w_gate = (rng.standard_normal((N, d)) * scale).astype(np.float32) if gated else None
    w_down = (rng.standard_normal((d, N)) * scale).astype(np.float32)
    return w_up, w_gate, w_down


def _np_ffn_dense(x, w_up, w_gate, w_down, b_up=None, b_down=None):
    """float64 library-matmul restatement, with fp32 rounding of the intermediates."""
    x64 = x.astype(np.float64)
    u = x64 @ w_up.astype(np.float64).T
    if w_gate is None:
        if b_up is not None:
            u = u + b_up.astype(np.float64)
        h = np.maximum(u.astype(np.float32), 0)
    else:
        g = (x64 @ w_gate.astype(np.float64).T).astype(np.float32)
        h = np.maximum(g, 0) * u.astype(np.float32)
    y = h.astype(np.float64) @ w_down.astype(np.float64).T
    if b_down is not None:
        y = y + b_down.astype(np.float64)
    return h, y.astype(np.float32)


# -------------------------------------------------------------- compaction --
@pytest.mark.parametrize("dt", [np.float32, np.uint16])
@pytest.mark.parametrize("gated", [False, True])
def test_compact_is_fancy_indexing(dt, gated):
    rng = np.random.default_rng(0)
    d, N = 24, 50
    mk = (lambda *s: rng.integers(0, 65535, size=s).astype(np.uint16)) if dt == np.uint16 \
        else (lambda *s: rng.standard_normal(s).astype(np.float32))
    w_up, w_down, b_up = mk(N, d), mk(d, N), mk(N)
    w_gate = mk(N, d) if gated else None
    S = np.sort(rng.permutation(N)[:13]).astype(np.int32)
    up_c, gate_c, down_c, bup_c = oracle.compact(w_up, w_gate, w_down, b_up, S)
    assert up_c.tobytes() == w_up[S].tobytes()
    assert down_c.tobytes() == np.ascontiguousarray(w_down[:, S].T).tobytes()
    assert bup_c.tobytes() == b_up[S].tobytes()
    if gated:
        assert gate_c.tobytes() == w_gate[S].tobytes()
    else:
        assert gate_c is None


# -------------------------------------------------------------- dense FFN ---
@pytest.mark.parametrize("gated", [False, True])
def test_dense_matches_float64_matmul(gated):
    rng = np.random.default_rng(1)
    d, N, T = 96, 320, 5
    w_up, w_gate, w_down = _weights(rng, d, N, gated, scale=0.1)
    b_up = None if gated else (rng.standard_normal(N) * 0.1).astype(np.float32)
    b_down = (rng.standard_normal(d) * 0.1).astype(np.float32)
    x = rng.standard_normal((T, d)).astype(np.float32)
    kind = oracle.RELU_GATED if gated else oracle.RELU
    H, Y = oracle.ffn_dense(x, kind, w_up, w_gate, w_down, b_up, b_down)
    h_np, y_np = _np_ffn_dense(x, w_up, w_gate, w_down, b_up, b_down)
    # matmul may sum in another order, in double: agreement to a few fp32 ulps
    np.testing.assert_allclose(H, h_np, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(Y, y_np, rtol=1e-5, atol=1e-6)


# ------------------------------------------- compacted FFN vs dense FFN -----
@pytest.mark.parametrize("gated", [False, True])
def test_compacted_equals_dense_restricted_to_the_set(gated):
    rng = np.random.default_rng(2)
    d, N, B = 64, 200, 3
    w_up, w_gate, w_down = _weights(rng, d, N, gated, scale=0.1)
    b_up = None if gated else (rng.standard_normal(N) * 0.1).astype(np.float32)
    x = rng.standard_normal((B, d)).astype(np.float32)
    kind = oracle.RELU_GATED if gated else oracle.RELU
    S = np.sort(rng.permutation(N)[:41]).astype(np.int32)
    up_c, gate_c, down_c, bup_c = oracle.compact(w_up, w_gate, w_down, b_up, S)
    y, h = oracle.ffn(x, kind, up_c, gate_c, down_c, bup_c, None, return_h=True)
    # dense with every neuron outside S switched off (its W_down column zeroed)
    w_down_masked = np.zeros_like(w_down)
    w_down_masked[:, S] = w_down[:, S]
    H, Y = oracle.ffn_dense(x, kind, w_up, w_gate, w_down_masked, b_up, None)
    np.testing.assert_array_equal(h, H[:, S])
    np.testing.assert_allclose(y, Y, rtol=1e-6, atol=1e-7)
    # and against the float64 matmul on the sliced weights
    _, y_np = _np_ffn_dense(x, w_up[S], None if w_gate is None else w_gate[S], w_down[:, S],
                            None if b_up is None else b_up[S], None)
    np.testing.assert_allclose(y, y_np, rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("gated", [False, True])
def test_alpha_beta_one_reproduces_dense_exactly(gated):
    """alpha = beta = 1 selects every neuron, and the compacted FFN is then the
    dense FFN bit for bit (same terms added in the same order)."""
    rng = np.random.default_rng(3)
    d, N, T = 32, 100, 6
    w_up, w_gate, w_down = _weights(rng, d, N, gated, scale=0.2)
    x = rng.standard_normal((T, d)).astype(np.float32)
    kind = oracle.RELU_GATED if gated else oracle.RELU
    H, Y = oracle.ffn_dense(x, kind, w_up, w_gate, w_down)
    S, _ = oracle.select(H, 1.0, 1.0)
    np.testing.assert_array_equal(S, np.arange(N))
    up_c, gate_c, down_c, _ = oracle.compact(w_up, w_gate, w_down, None, S)
    y = oracle.ffn(x, kind, up_c, gate_c, down_c)
    assert y.tobytes() == Y.tobytes()


# --------------------------------------------------- exact arithmetic case --
@pytest.mark.parametrize("gated", [False, True])
def test_integer_valued_case_is_exact(gated):
    """Small integers: every product and partial sum is an exact integer in any
    order, so the result must equal int64 arithmetic bit for bit."""
    rng = np.random.default_rng(4)
    d, K, B = 128, 96, 2
    up = rng.integers(-4, 5, size=(K, d))
    gate = rng.integers(-4, 5, size=(K, d)) if gated else None
    down = rng.integers(-4, 5, size=(K, d))
    x = rng.integers(-4, 5, size=(B, d))
    bup = None if gated else rng.integers(-4, 5, size=K)
    bdown = rng.integers(-4, 5, size=d)
    u = x @ up.T
    if gated:
        h = np.maximum(x @ gate.T, 0) * u
    else:
        h = np.maximum(u + bup, 0)
    y_int = h @ down + bdown
    assert np.abs(y_int).max() < 2 ** 24 and np.abs(h).max() < 2 ** 24
    kind = oracle.RELU_GATED if gated else oracle.RELU
    f = lambda a: None if a is None else a.astype(np.float32)
    y, hh = oracle.ffn(f(x), kind, f(up), f(gate), f(down), f(bup), f(bdown), return_h=True)
    np.testing.assert_array_equal(hh, h.astype(np.float32))
    np.testing.assert_array_equal(y, y_int.astype(np.float32))


# ----------------------------------------------------------- one-hot input --
def test_one_hot_input_by_hand():
    """x = e_1 picks column 1 of the up weights:
    h = relu([0.5, -1, 2] + [0, 0, -0.5]) = [0.5, 0, 1.5];
    y = 0.5*[1, 2] + 1.5*[-1, 4] + [10, 20] = [9, 27]."""
    up = np.array([[9.0, 0.5], [9.0, -1.0], [9.0, 2.0]], dtype=np.float32)
    down = np.array([[1.0, 2.0], [100.0, 100.0], [-1.0, 4.0]], dtype=np.float32)
    bup = np.array([0.0, 0.0, -0.5], dtype=np.float32)
    bdown = np.array([10.0, 20.0], dtype=np.float32)
    x = np.array([[0.0, 1.0]], dtype=np.float32)
    y = oracle.ffn(x, oracle.RELU, up, None, down, bup, bdown)
    np.testing.assert_array_equal(y, np.array([[9.0, 27.0]], dtype=np.float32))
    # gated: gate column [1, -1, 2] -> relu -> [1, 0, 2]; times up column [0.5, -1, 2]
    # h = [0.5, 0, 4]; y = 0.5*[1, 2] + 4*[-1, 4] = [-3.5, 17]
    gate = np.array([[7.0, 1.0], [7.0, -1.0], [7.0, 2.0]], dtype=np.float32)
    y = oracle.ffn(x, oracle.RELU_GATED, up, gate, down)
    np.testing.assert_array_equal(y, np.array([[-3.5, 17.0]], dtype=np.float32))


def test_gated_negative_product_is_kept_in_h():
    """gate > 0 with up < 0 gives a negative h: it is not "positive" for the
    selection, but the FFN still carries it."""
    up = np.array([[-2.0]], dtype=np.float32)
    gate = np.array([[3.0]], dtype=np.float32)
    down = np.array([[1.0]], dtype=np.float32)
    x = np.array([[1.0]], dtype=np.float32)
    y, h = oracle.ffn(x, oracle.RELU_GATED, up, gate, down, return_h=True)
    assert h[0, 0] == -6.0 and y[0, 0] == -6.0
    assert oracle.token_core(h[0], 1.0).tolist() == []


# -------------------------------------------------------------------- glue --
def test_glue_closed_forms():
    x = np.array([3.0, 0.0, -4.0, 0.0], dtype=np.float32)
    y = np.zeros(4, dtype=np.float32)
    # rms = sqrt((9 + 16) / 4) = 2.5
    np.testing.assert_allclose(oracle.glue(x, y), x / 2.5, rtol=1e-7)
    rng = np.random.default_rng(6)
    a, b = rng.standard_normal(300).astype(np.float32), rng.standard_normal(300).astype(np.float32)
    out = oracle.glue(a, b)
    np.testing.assert_allclose(np.sqrt(np.mean(out.astype(np.float64) ** 2)), 1.0, rtol=1e-6)
    s = (a.astype(np.float64) + b)
    np.testing.assert_allclose(out, s / np.sqrt(np.mean(s * s)), rtol=1e-6)
    np.testing.assert_allclose(oracle.glue(4 * a, 4 * b), out, rtol=1e-6)    # scale-free


def test_fp32_accumulators_stay_close_to_the_double_oracle():
    """The oracle keeps double running sums (a sequential fp32 sum over thousands of terms would
    spend part of the 1e-4 budget by itself).  The fp32-accumulator build of the same loops is
    reported against it: its distance must stay far below the bf16 gate and is printed."""
    rng = np.random.default_rng(11)
    d, K = 4096, 700
    x = rng.standard_normal((2, d)).astype(np.float32)
    up = (rng.standard_normal((K, d)) * 0.02).astype(np.float32)
    down = (rng.standard_normal((K, d)) * 0.02).astype(np.float32)
    y64 = oracle.ffn(x, oracle.RELU, up, None, down)
    y32 = oracle.ffn_f32_accumulators(x, oracle.RELU, up, None, down)
    rms = np.sqrt(np.mean(y64.astype(np.float64) ** 2, axis=-1, keepdims=True))
    dist = float(np.max(np.abs(y32.astype(np.float64) - y64) / rms))
    print("fp32-accumulator FFN vs double-accumulator oracle: %.3g of the output RMS (d=%d, K=%d)" % (dist, d, K))
    assert 0.0 < dist < 1e-4


# ---- SiLU-gated kind (h = silu(w_gate.x) * (w_up.x)) --------------------------------------
def _silu_case(seed=21, B=3, d=96, K=50):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, d)).astype(np.float32)
    up = (rng.standard_normal((K, d)) * 0.3).astype(np.float32)
    gate = (rng.standard_normal((K, d)) * 0.3).astype(np.float32)
    down = (rng.standard_normal((K, d)) * 0.3).astype(np.float32)
    return x, up, gate, down


def test_silu_gated_matches_library_sigmoid_and_matmul():
    """Library routines: float64 matmul and scipy's expit (silu(g) = g * expit(g))."""
    from scipy.special import expit
    x, up, gate, down = _silu_case()
    y, h = oracle.ffn(x, oracle.SILU_GATED, up, gate, down, return_h=True)
    g = (x.astype(np.float64) @ gate.astype(np.float64).T).astype(np.float32).astype(np.float64)
    u = (x.astype(np.float64) @ up.astype(np.float64).T).astype(np.float32).astype(np.float64)
    h_ref = ((g * expit(g)).astype(np.float32).astype(np.float64) * u).astype(np.float32)
    np.testing.assert_allclose(h, h_ref, rtol=2e-7, atol=1e-30)
    y_ref = h_ref.astype(np.float64) @ down.astype(np.float64)
    np.testing.assert_allclose(y, y_ref, rtol=1e-6, atol=1e-6)


def test_silu_identities():
    """silu(a) - silu(-a) = a, silu(0) = 0, silu(a) -> a and silu(-a) -> 0 for large a: a wrong
    sign or a dropped term breaks one of them.  The layer is built so that h_k = silu(a_k):
    gate row k picks coordinate k of x, every up row picks the last coordinate (= 1)."""
    K = 6
    d = K + 2                                                      # one spare coordinate, d even
    a = np.array([0.0, 0.5, -1.25, 3.0, 30.0, -30.0], np.float32)
    gate = np.zeros((K, d), np.float32); gate[np.arange(K), np.arange(K)] = 1.0
    up = np.zeros((K, d), np.float32); up[:, K] = 1.0
    down = np.zeros((K, d), np.float32); down[np.arange(K), np.arange(K)] = 1.0
    x = np.zeros((2, d), np.float32); x[0, :K] = a; x[1, :K] = -a; x[:, K] = 1.0
    y = oracle.ffn(x, oracle.SILU_GATED, up, gate, down).astype(np.float64)
    hp, hm = y[0, :K], y[1, :K]
    np.testing.assert_allclose(hp - hm, a.astype(np.float64), rtol=1e-6, atol=1e-7)
    assert hp[0] == 0.0 and hm[0] == 0.0
    np.testing.assert_allclose(hp[4], 30.0, rtol=1e-6)
    assert abs(hm[4]) < 1e-10 and abs(hp[5]) < 1e-10
    np.testing.assert_allclose(hp[1], 0.5 / (1.0 + np.exp(-0.5)), rtol=1e-6)   # 0.3112296656...
    assert abs(hp[1] - 0.31122966560092726) < 1e-7


def test_silu_gated_compacted_equals_dense_restricted():
    x, up, gate, down = _silu_case(seed=5, B=2, d=64, K=40)
    N = 40
    w_down = np.ascontiguousarray(down.T)
    H, Y = oracle.ffn_dense(x, oracle.SILU_GATED, up, gate, w_down)
    y_all = oracle.ffn(x, oracle.SILU_GATED, up, gate, down)
    np.testing.assert_array_equal(Y, y_all)                       # same loops over all neurons
    S = np.array([1, 4, 9, 16, 25, 36], np.int32)
    y_S = oracle.ffn(x, oracle.SILU_GATED, up[S], gate[S], down[S])
    mask = np.zeros(N, bool); mask[S] = True
    y_ref = (np.where(mask, H, 0).astype(np.float64) @ down.astype(np.float64))
    np.testing.assert_allclose(y_S, y_ref, rtol=1e-6, atol=1e-6)
    # negative intermediates exist and are never selected by Definition 1
    assert (H < 0).any()
    Ssel, f = oracle.select(H, 1.0, 1.0)
    assert f[(H <= 0).all(axis=0)].sum() == 0
