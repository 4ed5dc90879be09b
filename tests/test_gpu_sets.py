"""Core sets over several sentences (prompts in pieces, semantic groups, set similarity, nearest
centroid, in-place set update) against the oracle: integer results bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_18311_b200 as ci
from paper_2410_18311_b200 import workloads as wl
from helpers import require_gpu, gpu_select, gpu_compact, gpu_decode, to_f32_np, raw_np, assert_ffn_close

pytestmark = pytest.mark.gpu


def _top(counts, max_count, frac):
    K = ci.coreinfer_count(frac, counts.numel())
    S = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    ci.coreinfer_top_by_count(counts, max_count, frac, S)
    torch.cuda.synchronize()
    return S.cpu().numpy()


@pytest.mark.parametrize("N,maxc", [(8, 4), (1000, 5), (16384, 300), (36864, 5000), (5000, 70000)])
def test_top_by_count(N, maxc):
    require_gpu()
    rng = np.random.default_rng(N)
    for frac in (0.1, 0.25, 1.0):
        c = rng.integers(0, maxc + 1, size=N).astype(np.int32)
        np.testing.assert_array_equal(_top(torch.from_numpy(c).cuda(), maxc, frac), oracle.top_by_count(c, frac))


def test_prompt_in_pieces():
    """Selection over a prompt that arrives in three pieces: the pieces' counts are added and the
    set follows from the sum; identical to selecting over the whole prompt at once."""
    require_gpu()
    cfg = wl.CONFIGS["opt6.7b"].with_(d_ff=4096)
    A, _ = wl.planted_activations(cfg, 0, 200, device="cuda")
    S_all, f_all = gpu_select(A, cfg.alpha, cfg.beta)
    acc = torch.zeros(cfg.d_ff, dtype=torch.int32, device="cuda")
    for a, b in ((0, 64), (64, 65), (65, 200)):
        _, f = gpu_select(A[a:b].contiguous(), cfg.alpha, cfg.beta)
        ci.coreinfer_counts_add(acc, torch.from_numpy(f).cuda())
    torch.cuda.synchronize()
    np.testing.assert_array_equal(acc.cpu().numpy(), f_all)
    np.testing.assert_array_equal(_top(acc, 200, cfg.beta), S_all)
    S_o, f_o = oracle.select(A.cpu().numpy(), cfg.alpha, cfg.beta)
    np.testing.assert_array_equal(S_all, S_o)


def test_semantic_group_table_and_assignment():
    """Similarity-guided prediction on synthetic groups: sentences of a group share a planted
    neuron subset; the group's set is the top gamma by the number of sentences whose core set holds
    a neuron; an input is assigned to the nearest centroid."""
    require_gpu()
    N, G, n_sent, gamma = 4096, 4, 12, 0.2
    cfg = wl.CONFIGS["opt6.7b"].with_(d_ff=N)
    group_sets, group_sets_o = [], []
    for g in range(G):
        counts = torch.zeros(N, dtype=torch.int32, device="cuda")
        sets = []
        for s in range(n_sent):
            A, _ = wl.planted_activations(cfg, 10 * g, 40, device="cuda")          # same planted subset per group
            A = A[torch.randperm(40, generator=torch.Generator().manual_seed(100 * g + s))[:24].cuda()].contiguous()
            S, _ = gpu_select(A, 0.4, 0.2)
            S_o, _ = oracle.select(A.cpu().numpy(), 0.4, 0.2)
            np.testing.assert_array_equal(S, S_o)
            sets.append(S_o)
            ci.coreinfer_counts_add_set(counts, torch.from_numpy(S).cuda())
        torch.cuda.synchronize()
        c_o = oracle.group_counts(sets, N)
        np.testing.assert_array_equal(counts.cpu().numpy(), c_o)
        got, ref = _top(counts, n_sent, gamma), oracle.top_by_count(c_o, gamma)
        np.testing.assert_array_equal(got, ref)
        group_sets.append(got)
    # different groups, different sets (planted subsets differ)
    sh, inv = oracle.core_similarity(group_sets[0], group_sets[1])
    assert sh / inv < 0.5
    # assignment
    D = 300
    rng = np.random.default_rng(0)
    C = rng.standard_normal((G, D)).astype(np.float32)
    ws = torch.empty(ci.coreinfer_nearest_centroid_workspace_bytes(G), dtype=torch.uint8, device="cuda")
    out = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for g in range(G):
        v = C[g] + 0.05 * rng.standard_normal(D).astype(np.float32)
        ci.coreinfer_nearest_centroid(torch.from_numpy(C).cuda(), torch.from_numpy(v).cuda(), out, ws)
        torch.cuda.synchronize()
        g_o, d2_o = oracle.nearest_centroid(C, v)
        assert int(out.item()) == g_o == g
        np.testing.assert_allclose(ws.view(torch.float64).cpu().numpy(), d2_o, rtol=1e-12)
    # a tie goes to the lower group
    C2 = np.array([[0, 0, 0, 0], [2, 0, 0, 0], [0, 2, 0, 0]], np.float32)
    ci.coreinfer_nearest_centroid(torch.from_numpy(C2).cuda(), torch.tensor([1.0, 1.0, 0, 0]).cuda(), out,
                                  torch.empty(ci.coreinfer_nearest_centroid_workspace_bytes(3), dtype=torch.uint8, device="cuda"))
    assert int(out.item()) == oracle.nearest_centroid(C2, np.array([1, 1, 0, 0], np.float32))[0] == 0


def test_core_similarity():
    require_gpu()
    rng = np.random.default_rng(1)
    out = torch.empty(2, dtype=torch.int32, device="cuda")
    for KA, KB, N in [(1, 1, 5), (100, 37, 300), (3277, 3277, 16384), (7373, 5000, 36864)]:
        A = np.sort(rng.choice(N, size=KA, replace=False)).astype(np.int32)
        B = rng.permutation(rng.choice(N, size=KB, replace=False)).astype(np.int32)
        ci.coreinfer_core_similarity(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), out)
        assert tuple(out.cpu().tolist()) == oracle.core_similarity(A, B)


@pytest.mark.parametrize("dtype,gated", [(torch.bfloat16, False), (torch.float32, True), (torch.float16, True)])
def test_update_core_set_in_place(dtype, gated):
    """The deployed set moves from S0 to S1 and on to S2: only the rows whose neuron left are
    rewritten (pairs as the oracle lists them), the buffers then hold exactly the new set's rows
    in slot order, and decoding through them matches the oracle on those rows."""
    require_gpu()
    d, N, K = 256, 2000, 400
    g = torch.Generator().manual_seed(3)
    mk = lambda *s: (torch.randn(*s, generator=g) * 0.05).to(dtype).cuda()
    w_up, w_down = mk(N, d), mk(d, N)
    w_gate = mk(N, d) if gated else None
    b_up = None if gated else mk(N)
    rng = np.random.default_rng(4)
    S0 = np.sort(rng.choice(N, size=K, replace=False)).astype(np.int32)
    up_c, gate_c, down_c, bup_c = gpu_compact(w_up, w_gate, w_down, b_up, torch.from_numpy(S0).cuda())
    slot_neuron = torch.from_numpy(S0.copy()).cuda()
    slot_o = S0.copy()
    ws = torch.empty(ci.coreinfer_update_core_set_workspace_bytes(N, K), dtype=torch.uint8, device="cuda")
    nch = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for step in range(2):
        keep = rng.choice(slot_o, size=K - 37 * (step + 1), replace=False)
        fresh = rng.choice(np.setdiff1d(np.arange(N), slot_o), size=K - len(keep), replace=False)
        S1 = np.sort(np.concatenate([keep, fresh])).astype(np.int32)
        before = (raw_np(up_c).copy(), raw_np(down_c).copy())
        ci.coreinfer_update_core_set(w_up, w_gate, w_down, b_up, slot_neuron, torch.from_numpy(S1).cuda(), up_c, gate_c,
                                     down_c, bup_c, nch, ws)
        torch.cuda.synchronize()
        slots_o, neurons_o, slot_o = oracle.set_delta(slot_o, S1)
        assert int(nch.item()) == len(slots_o) == K - len(keep)
        np.testing.assert_array_equal(slot_neuron.cpu().numpy(), slot_o)
        order = torch.from_numpy(slot_o.astype(np.int64)).cuda()
        assert torch.equal(up_c, w_up[order]) and torch.equal(down_c, w_down[:, order].t().contiguous())
        if gated:
            assert torch.equal(gate_c, w_gate[order])
        else:
            assert torch.equal(bup_c, b_up[order])
        untouched = np.setdiff1d(np.arange(K), slots_o)
        assert (raw_np(up_c)[untouched] == before[0][untouched]).all() and (raw_np(down_c)[untouched] == before[1][untouched]).all()
        # same bytes as a fresh compaction of the new set, row for row after sorting the slots
        o_up, _, o_down, _ = oracle.compact(raw_np(w_up), raw_np(w_gate), raw_np(w_down), raw_np(b_up), S1)
        perm = np.argsort(slot_o, kind="stable")
        assert raw_np(up_c)[perm].tobytes() == o_up.tobytes() and raw_np(down_c)[perm].tobytes() == o_down.tobytes()
        x = mk(1, d) * 20
        kind = ci.FFN_RELU_GATED if gated else ci.FFN_RELU
        y = gpu_decode(x, kind, up_c, gate_c, down_c, bup_c)
        y_o = oracle.ffn(to_f32_np(x), kind, to_f32_np(up_c), to_f32_np(gate_c), to_f32_np(down_c), to_f32_np(bup_c))
        assert_ffn_close(y, y_o, dtype)


def test_update_core_set_at_the_opt67b_shape():
    """A deployed OPT-6.7B-shaped layer (d_model 4096, d_ff 16384, K 3277) whose set changes by 5 %:
    pairs as the oracle lists them, buffers equal to a fresh compaction of the new set row for row."""
    require_gpu()
    cfg = wl.CONFIGS["opt6.7b"]
    w_up, _, w_down = wl.layer_weights(cfg, 1, device="cuda")
    N, K = cfg.d_ff, ci.coreinfer_count(cfg.beta, cfg.d_ff)
    rng = np.random.default_rng(8)
    S0 = np.sort(rng.choice(N, size=K, replace=False)).astype(np.int32)
    up_c, _, down_c, _ = gpu_compact(w_up, None, w_down, None, torch.from_numpy(S0).cuda())
    keep = rng.choice(S0, size=K - K // 20, replace=False)
    S1 = np.sort(np.concatenate([keep, rng.choice(np.setdiff1d(np.arange(N), S0), size=K - len(keep), replace=False)])).astype(np.int32)
    slot_neuron = torch.from_numpy(S0.copy()).cuda()
    ws = torch.empty(ci.coreinfer_update_core_set_workspace_bytes(N, K), dtype=torch.uint8, device="cuda")
    nch = torch.zeros(1, dtype=torch.int32, device="cuda")
    sim = torch.zeros(2, dtype=torch.int32, device="cuda")
    ci.coreinfer_core_similarity(torch.from_numpy(S0).cuda(), torch.from_numpy(S1).cuda(), sim)
    ci.coreinfer_update_core_set(w_up, None, w_down, None, slot_neuron, torch.from_numpy(S1).cuda(), up_c, None, down_c, None, nch, ws)
    torch.cuda.synchronize()
    assert tuple(sim.cpu().tolist()) == oracle.core_similarity(S0, S1) == (len(keep), 2 * K - len(keep))
    slots_o, neurons_o, slot_o = oracle.set_delta(S0, S1)
    assert int(nch.item()) == len(slots_o) == K // 20
    np.testing.assert_array_equal(slot_neuron.cpu().numpy(), slot_o)
    o_up, _, o_down, _ = oracle.compact(raw_np(w_up), None, raw_np(w_down), None, S1)
    perm = np.argsort(slot_o, kind="stable")
    assert raw_np(up_c)[perm].tobytes() == o_up.tobytes() and raw_np(down_c)[perm].tobytes() == o_down.tobytes()
