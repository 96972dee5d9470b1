"""Pins for the CPU oracle: what the paper and the mathematics fix, independent
of the oracle's own code paths (brute force, closed forms, invariants, library
routines).  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import brute, hsa_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rnd(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


def all_blocks(H, N, groups=1):
    return [[np.arange(O.n_blocks(N), dtype=np.int32) for _ in range(groups)] for _ in range(H)]


# ---------------------------------------------------------------- sizes the paper prints
def test_golden_active_kv_tokens():
    rows = [l.split() for l in open(os.path.join(GOLD, "hkv_active_kv_tokens.txt")) if l[0] != "#"]
    kp, frames, tpf, total = map(int, rows[0])
    assert kp * frames * tpf == total == 49920
    assert O.n_blocks(total) == 780          # blocks of 64
    assert O.block_count(779, total) == 64 and O.block_count(780, total) == 0


def test_golden_block_sizes():
    for l in open(os.path.join(GOLD, "hsa_block_sizes.txt")):
        if l[0] == "#":
            continue
        name, B, ct, ch, cw = l.split()
        assert int(B) == int(ct) * int(ch) * int(cw)
        if name == "intra":
            assert int(B) == O.BLOCK


def test_block_counts_of_configs():
    # one continuous token stream; a single partial tail block
    for N, nb, tail in [(46800, 732, 16), (280800, 4388, 32), (140400, 2194, 48), (2048, 32, 64)]:
        assert O.n_blocks(N) == nb
        assert O.block_count(nb - 1, N) == tail


# ---------------------------------------------------------------- dense equivalence
@pytest.mark.parametrize("causal,q_pos0,N", [(False, 150, 150), (True, 150 - 24, 150), (True, 10, 150)])
def test_all_selected_no_linear_equals_dense_brute(causal, q_pos0, N):
    H, d, Lq = 2, 8, 24
    q, K, V = rnd((Lq, H, d), 1), rnd((N, H, d), 2), rnd((N, H, d), 3)
    r = O.hsa_forward(q, K, V, q_pos0, causal, all_blocks(H, N), no_linear=True)
    keysets = [[list(range(N)) for _ in range(Lq)] for _ in range(H)]
    ref = np.array(brute.attention_rows(q, K, V, N, H, d, Lq, q_pos0, causal, keysets))
    assert np.abs(r["out"] - ref).max() < 1e-12
    assert np.abs(r["out"] - O.dense_attention(q, K, V, q_pos0, causal)).max() < 1e-12


@pytest.mark.parametrize("causal", [False, True])
def test_all_selected_equals_torch_sdpa(causal):
    H, d, Lq, N = 3, 16, 40, 200
    q, K, V = rnd((Lq, H, d), 4), rnd((N, H, d), 5), rnd((N, H, d), 6)
    q_pos0 = N - Lq if causal else N
    r = O.hsa_forward(q, K, V, q_pos0, causal, all_blocks(H, N), no_linear=True)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(K).permute(1, 0, 2)[None]
    tv = torch.from_numpy(V).permute(1, 0, 2)[None]
    mask = None
    if causal:
        mask = (torch.arange(N)[None, :] <= (q_pos0 + torch.arange(Lq))[:, None])
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.abs(r["out"] - ref).max() < 1e-12


# ---------------------------------------------------------------- linear branch identities
@pytest.mark.parametrize("causal,q_pos0", [(False, 300), (True, 300 - 37), (True, 5)])
def test_linear_recurrent_equals_parallel(causal, q_pos0):
    H, d, Lq, N = 2, 16, 37, 300
    q, K, V = rnd((Lq, H, d), 7), rnd((N, H, d), 8), rnd((N, H, d), 9)
    a = O.linear_parallel(q, K, V, q_pos0, causal)
    b = O.linear_recurrent(q, K, V, q_pos0, causal)
    assert np.abs(a - b).max() <= 1e-10 * max(1.0, np.abs(a).max())


@pytest.mark.parametrize("causal", [False, True])
def test_linear_chunked_equals_parallel(causal):
    H, d, Lq, N = 2, 16, 50, 260
    q, K, V = rnd((Lq, H, d), 10), rnd((N, H, d), 11), rnd((N, H, d), 12)
    q_pos0 = N - Lq if causal else N
    a = O.linear_parallel(q, K, V, q_pos0, causal)
    c = O.linear_chunked(q, K, V, q_pos0, causal, boundary=N - Lq)
    assert np.abs(a - c).max() <= 1e-10
    if not causal:
        S, z = O.linear_state(K, V)
        s = O.linear_from_state(q, S, z)
        assert np.abs(a - s).max() <= 1e-10


def test_linear_brute_force():
    H, d, Lq, N = 2, 4, 6, 70
    q, K, V = rnd((Lq, H, d), 13), rnd((N, H, d), 14), rnd((N, H, d), 15)
    for causal, q_pos0 in [(False, N), (True, N - Lq), (True, 3)]:
        a = O.linear_parallel(q, K, V, q_pos0, causal)
        b = np.array(brute.linear_rows(q, K, V, N, H, d, Lq, q_pos0, causal))
        assert np.abs(a - b).max() < 1e-12


def test_phi_is_elu_plus_one():
    x = np.array([-30.0, -1.0, -1e-9, 0.0, 1e-9, 2.5])
    ref = torch.nn.functional.elu(torch.from_numpy(x)).numpy() + 1.0
    assert np.allclose(O.phi(x), ref, rtol=0, atol=1e-15)
    assert (O.phi(x) > 0).all()


# ---------------------------------------------------------------- the relu feature map
def test_relu_feature_map_is_torch_relu():
    x = np.array([-30.0, -1.0, -1e-9, 0.0, 1e-9, 2.5])
    assert np.array_equal(O.phi(x, "relu"), torch.relu(torch.from_numpy(x)).numpy())
    with pytest.raises(ValueError):
        O.phi(x, "gelu")


@pytest.mark.parametrize("causal,q_pos0", [(False, 300), (True, 300 - 37), (True, 5)])
def test_relu_recurrent_equals_parallel_equals_chunked(causal, q_pos0):
    """The algebraic identities of the running-state form hold for any feature map."""
    H, d, Lq, N = 2, 16, 37, 300
    q, K, V = rnd((Lq, H, d), 7), rnd((N, H, d), 8), rnd((N, H, d), 9)
    a = O.linear_parallel(q, K, V, q_pos0, causal, fmap="relu")
    b = O.linear_recurrent(q, K, V, q_pos0, causal, fmap="relu")
    assert np.abs(a - b).max() <= 1e-10 * max(1.0, np.abs(a).max())
    if q_pos0 >= N - Lq - 1:
        c = O.linear_chunked(q, K, V, q_pos0, causal, boundary=N - Lq, fmap="relu")
        assert np.abs(a - c).max() <= 1e-10
    if not causal:
        S, z = O.linear_state(K, V, fmap="relu")
        assert np.abs(a - O.linear_from_state(q, S, z, "relu")).max() <= 1e-10
    # and the map matters: the two forms differ on the same inputs
    assert np.abs(a - O.linear_parallel(q, K, V, q_pos0, causal)).max() > 1e-3


def test_relu_brute_force_and_closed_forms():
    H, d, Lq, N = 2, 4, 6, 70
    q, K, V = rnd((Lq, H, d), 13), rnd((N, H, d), 14), rnd((N, H, d), 15)
    for causal, q_pos0 in [(False, N), (True, N - Lq), (True, 3)]:
        a = O.linear_parallel(q, K, V, q_pos0, causal, fmap="relu")
        b = np.array(brute.linear_rows(q, K, V, N, H, d, Lq, q_pos0, causal, relu=True))
        assert np.abs(a - b).max() < 1e-12
    # keys without a positive component carry no weight: the state is zero and the branch is 0 / eps = 0
    Kn = -np.abs(K)
    S, z = O.linear_state(Kn, V, fmap="relu")
    assert not S.any() and not z.any()
    assert not O.linear_parallel(q, Kn, V, N, False, fmap="relu").any()
    # one key e_0, queries with a positive first component w: weight w, so O_lin = w v / (w + eps)
    K1 = np.zeros((1, H, d)); K1[0, :, 0] = 1.0
    q1 = np.abs(q) + 0.5
    out = O.linear_parallel(q1, K1, V[:1], 1, False, fmap="relu")
    w = q1[:, :, :1]
    assert np.allclose(out, w * V[0][None] / (w + O.RELU_EPS), atol=1e-14)
    # V = 1 everywhere: every row with weight returns 1 up to eps / (den + eps)
    ones = np.ones_like(V)
    o1 = O.linear_parallel(q, np.abs(K) + 0.1, ones, N, False, fmap="relu")
    den = (O.phi(q, "relu").reshape(Lq, H, 1, d) * (np.abs(K) + 0.1).transpose(1, 0, 2)[None]).sum(axis=(2, 3))
    has = den > 0
    assert np.allclose(o1[has], (den / (den + O.RELU_EPS))[has][:, None] * np.ones(d), atol=1e-14)
    assert not o1[~has].any()


def test_forward_with_relu_uses_it_in_the_linear_branch_only():
    H, d, Lq, N = 2, 8, 16, 192
    q, K, V = rnd((Lq, H, d), 31), rnd((N, H, d), 32), rnd((N, H, d), 33)
    sel = O.select_blocks(q, K, N, False, [2] * H)[0]
    a = O.hsa_forward(q, K, V, N, False, sel, fmap="relu")
    b = O.hsa_forward(q, K, V, N, False, sel)
    assert np.array_equal(a["O_sp"], b["O_sp"])
    assert np.allclose(a["O_lin"], O.linear_parallel(q, K, V, N, False, fmap="relu"), atol=0)
    assert np.allclose(a["out"], a["O_lin"] + a["O_sp"], atol=1e-15)
    s = O.hsa_forward(q, K, V, N, False, sel, fmap="relu", linear_form="state")
    assert np.abs(s["O_lin"] - a["O_lin"]).max() <= 1e-10


def test_single_token_history():
    H, d, Lq = 2, 8, 5
    q, K, V = rnd((Lq, H, d), 16), rnd((1, H, d), 17), rnd((1, H, d), 18)
    r = O.hsa_forward(q, K, V, 1, False, all_blocks(H, 1))
    for i in range(Lq):
        assert np.allclose(r["O_sp"][i], V[0], atol=1e-14)
        assert np.allclose(r["O_lin"][i], V[0], atol=1e-14)
        assert np.allclose(r["out"][i], 2 * V[0], atol=1e-14)


# ---------------------------------------------------------------- sparse branch vs brute force
@pytest.mark.parametrize("seed", range(6))
def test_sparse_brute_force_tiny(seed):
    rng = np.random.default_rng(100 + seed)
    H = int(rng.integers(1, 3))
    d = int(rng.choice([2, 4, 8]))
    N = int(rng.integers(1, 193))
    Lq = int(rng.integers(1, 17))
    causal = bool(rng.integers(0, 2))
    q_pos0 = int(rng.integers(0, N + 1)) if causal else N
    q, K, V = rnd((Lq, H, d), seed), rnd((N, H, d), seed + 50), rnd((N, H, d), seed + 99)
    budgets = [int(rng.choice([0, 1, 2, -1])) for _ in range(H)]
    sel, s = O.select_blocks(q, K, q_pos0, causal, budgets)
    # selection against the pure-Python scorer + selector
    bs = brute.block_scores(q, K, N, H, d, Lq)
    nb = O.n_blocks(N)
    for h in range(H):
        assert np.allclose(s[h, 0], bs[h], atol=1e-13)
        cand = [(64 * b < N) and (not causal or 64 * b <= q_pos0 + Lq - 1) for b in range(nb)]
        assert list(sel[h][0]) == brute.topk_blocks(bs[h], cand, budgets[h])
    # sparse output against the pure-Python attention over the selected blocks' keys
    keysets = [[[j for b in sel[h][0] for j in range(64 * b, min(N, 64 * b + 64))]
                for _ in range(Lq)] for h in range(H)]
    ref = np.array(brute.attention_rows(q, K, V, N, H, d, Lq, q_pos0, causal, keysets))
    out = O.sparse_branch(q, K, V, sel, q_pos0, causal)
    assert np.abs(out - ref).max() < 1e-12


def test_partition_of_unity():
    H, d, Lq, N = 2, 8, 20, 200
    q, K = rnd((Lq, H, d), 20), rnd((N, H, d), 21)
    V = np.ones((N, H, d))
    sel, _ = O.select_blocks(q, K, N, False, [2, 1])
    r = O.hsa_forward(q, K, V, N, False, sel)
    assert np.allclose(r["O_sp"], 1.0, atol=1e-14)
    assert np.allclose(r["O_lin"], 1.0, atol=1e-14)
    assert np.allclose(r["out"], 2.0, atol=1e-13)


def test_identical_keys_give_mean_of_values():
    H, d, Lq, N = 1, 8, 7, 64 * 3
    q, V = rnd((Lq, H, d), 22), rnd((N, H, d), 23)
    K = rnd((N, H, d), 24)
    K[64:128] = K[64]                       # block 1: identical keys
    out = O.sparse_branch(q, K, V, [[np.array([1])]], N, False)
    assert np.allclose(out[:, 0], V[64:128, 0].mean(axis=0)[None], atol=1e-13)
    # causal, query in the middle of the block sees only the prefix
    out = O.sparse_branch(q[:1], K, V, [[np.array([1])]], 64 + 9, True)
    assert np.allclose(out[0, 0], V[64:64 + 10, 0].mean(axis=0), atol=1e-13)


def test_zero_budget_gives_linear_only_and_empty_rows_zero():
    H, d, Lq, N = 2, 8, 9, 130
    q, K, V = rnd((Lq, H, d), 25), rnd((N, H, d), 26), rnd((N, H, d), 27)
    sel, _ = O.select_blocks(q, K, N, False, [0, 0])
    r = O.hsa_forward(q, K, V, N, False, sel)
    assert np.array_equal(r["O_sp"], np.zeros_like(r["O_sp"]))
    assert np.array_equal(r["out"], r["O_lin"])
    # causal: a selected block lying wholly after a query contributes nothing to that row
    out = O.sparse_branch(q, K, V, [[np.array([1])], [np.array([1])]], 0, True)
    assert np.array_equal(out, np.zeros_like(out))      # positions 0..8 < 64
    lin = O.linear_parallel(q, K, V, -5, True)
    assert np.array_equal(lin[:5], np.zeros_like(lin[:5]))   # positions < 0 see nothing


# ---------------------------------------------------------------- selection
def test_selection_properties_and_planted_block():
    H, d, Lq, N = 3, 16, 32, 64 * 20 + 13
    q, K = rnd((Lq, H, d), 30), rnd((N, H, d), 31, 0.2)
    qbar = q.mean(axis=0)
    for h in range(H):
        K[64 * 7:64 * 8, h] += 3.0 * qbar[h] / np.linalg.norm(qbar[h])   # planted block 7
    budgets = [1, 5, 40]
    sel, s = O.select_blocks(q, K, N, False, budgets)
    nb = O.n_blocks(N)
    assert nb == 21
    for h in range(H):
        ids = sel[h][0]
        assert len(ids) == min(budgets[h], nb)
        assert list(ids) == sorted(ids)
        assert 7 in ids
        assert int(np.argmax(s[h, 0])) == 7
        rest = np.setdiff1d(np.arange(nb), ids)
        if len(rest) and len(ids):
            assert s[h, 0, ids].min() >= s[h, 0, rest].max()
        # full fp64 sort done independently
        ref = sorted(sorted(range(nb), key=lambda b: (-s[h, 0, b], b))[:budgets[h]])
        assert list(ids) == ref


def test_selection_ties_and_budget_edge_cases():
    sc = np.array([1.0, 3.0, 3.0, 3.0, 0.5, 3.0])
    cand = np.ones(6, bool)
    assert list(O.select_topk(sc, cand, 2)) == [1, 2]          # lower index wins
    assert list(O.select_topk(sc, cand, 4)) == [1, 2, 3, 5]
    assert list(O.select_topk(sc, cand, 0)) == []
    assert list(O.select_topk(sc, cand, -1)) == [0, 1, 2, 3, 4, 5]
    assert list(O.select_topk(sc, cand, 99)) == [0, 1, 2, 3, 4, 5]
    cand[1] = False
    assert list(O.select_topk(sc, cand, 2)) == [2, 3]


def test_candidates_under_causal_mask():
    N = 64 * 5 + 3
    assert O.candidate_mask(N, N, 10, False).sum() == 6
    # last query position 130 -> blocks starting at 0, 64, 128
    assert list(np.nonzero(O.candidate_mask(N, 100, 31, True))[0]) == [0, 1, 2]


def test_scores_use_means_of_partial_block():
    H, d, Lq, N = 1, 4, 3, 64 + 5
    q, K = rnd((Lq, H, d), 32), rnd((N, H, d), 33)
    s = O.block_scores(q, K)
    ref = q.mean(axis=0)[0] @ K[64:, 0].mean(axis=0) / math.sqrt(d)
    assert abs(s[0, 0, 1] - ref) < 1e-14


def test_per_group_selection_layout():
    H, d, Lq, N = 1, 8, 40, 64 * 6
    q, K = rnd((Lq, H, d), 34), rnd((N, H, d), 35)
    sel, s = O.select_blocks(q, K, N, False, [2], group_tokens=16)
    assert s.shape == (1, 3, 6) and len(sel[0]) == 3
    s0 = O.block_scores(q[16:32], K)
    assert np.allclose(s[0, 1], s0[0, 0], atol=1e-14)


# ---------------------------------------------------------------- merge
def test_merge_linear_in_gates_and_single_branch_modes():
    H, d, Lq = 2, 4, 6
    a, b = rnd((Lq, H, d), 40), rnd((Lq, H, d), 41)
    one, zero = np.ones((Lq, H)), np.zeros((Lq, H))
    assert np.array_equal(O.merge(a, b, one, zero), a)
    assert np.array_equal(O.merge(a, b, zero, one), b)
    assert np.array_equal(O.merge(a, b), a + b)
    g1, g2 = rnd((Lq, H), 42), rnd((Lq, H, d), 43)
    assert np.allclose(O.merge(a, b, 2 * g1, g2), 2 * g1[..., None] * a + g2 * b)
    sg = 1 / (1 + np.exp(-g1))
    assert np.allclose(O.merge(a, b, g1, None, gate_act=1), sg[..., None] * a + b)


# ---------------------------------------------------------------- Linformer form
def test_linformer_identity_projection_is_dense_attention():
    H, d, Lq, L_seg = 2, 8, 10, 32
    N = 3 * L_seg
    q, K, V = rnd((Lq, H, d), 50), rnd((N, H, d), 51), rnd((N, H, d), 52)
    E = np.broadcast_to(np.eye(L_seg), (H, L_seg, L_seg))
    Kt, Vt = O.linformer_compress(K, V, E, E, L_seg)
    assert np.array_equal(Kt, K) and np.array_equal(Vt, V)
    out = O.linformer_branch(q, Kt, Vt)
    keysets = [[list(range(N)) for _ in range(Lq)] for _ in range(H)]
    ref = np.array(brute.attention_rows(q, K, V, N, H, d, Lq, N, False, keysets))
    assert np.abs(out - ref).max() < 1e-12


def test_linformer_mean_projection_and_incremental():
    H, d, L_seg, r = 2, 4, 16, 3
    N = 2 * L_seg + 5                        # trailing incomplete segment is ignored
    K, V = rnd((N, H, d), 53), rnd((N, H, d), 54)
    E = np.full((H, L_seg, r), 1.0 / L_seg)
    Kt, Vt = O.linformer_compress(K, V, E, E, L_seg)
    assert Kt.shape == (2 * r, H, d)
    assert np.allclose(Kt[0], K[:L_seg].mean(axis=0)) and np.allclose(Vt[r], V[L_seg:2 * L_seg].mean(axis=0))
    E2 = rnd((H, L_seg, r), 55)
    a, _ = O.linformer_compress(K, V, E2, E2, L_seg)
    b, _ = O.linformer_compress(K[:L_seg], V[:L_seg], E2, E2, L_seg)
    assert np.array_equal(a[:r], b)


# ---------------------------------------------------------------- float32 carriers are widened
def test_float32_inputs_are_computed_in_float64():
    H, d, Lq, N = 2, 8, 12, 150
    q = torch.randn(Lq, H, d).bfloat16().float().numpy()
    K = torch.randn(N, H, d).bfloat16().float().numpy()
    V = torch.randn(N, H, d).bfloat16().float().numpy()
    sel32, s32 = O.select_blocks(q, K, N, False, [1, 2])
    sel64, s64 = O.select_blocks(q.astype(np.float64), K.astype(np.float64), N, False, [1, 2])
    assert np.array_equal(s32, s64)
    a = O.hsa_forward(q, K, V, N, False, sel32)["out"]
    b = O.hsa_forward(q.astype(np.float64), K.astype(np.float64), V.astype(np.float64), N, False, sel64)["out"]
    assert a.dtype == np.float64 and np.array_equal(a, b)


# ---------------------------------------------------------------- head-adaptive budgets (Gini / tau rule)
def test_gini_closed_forms():
    N = 37
    assert abs(O.gini_of_weights(np.full(N, 1.0 / N))) < 1e-15               # uniform -> 0
    onehot = np.zeros(N)
    onehot[0] = 1.0
    assert abs(O.gini_of_weights(onehot) - (N - 1) / N) < 1e-15              # one-hot -> (N-1)/N
    # two equal masses: (1/N) * ((N-1) + (N-3)) / 2
    two = np.zeros(N)
    two[:2] = 0.5
    assert abs(O.gini_of_weights(two) - (N - 2) / N) < 1e-15
    assert O.gini_of_weights(np.zeros(0)) == 0.0


def test_block_weights_are_a_softmax_over_candidates():
    s = np.array([0.3, -1.0, 2.0, 0.0, 5.0])
    cand = np.array([True, True, True, False, True])
    p = O.block_weights(s, cand)
    ref = torch.softmax(torch.tensor(s[cand]), 0).numpy()
    assert np.allclose(p[cand], ref, atol=1e-15) and p[3] == 0.0 and abs(p.sum() - 1) < 1e-15


def test_adaptive_selection_minimal_prefix_and_threshold_map():
    H, d, Lq, N = 3, 16, 40, 64 * 23 + 7
    q, K = rnd((Lq, H, d), 60, 3.0), rnd((N, H, d), 61)
    for tmin, tmax in [(0.35, 1.0), (0.5, 0.5), (0.0, 0.9)]:
        sel, gini, tau = O.adaptive_selection(q, K, N, False, tmin, tmax)
        s = O.block_scores(q, K)
        for h in range(H):
            p = O.block_weights(s[h, 0], np.ones(s.shape[2], bool))
            # brute force: sort pairs in Python, walk the prefix
            order = sorted(range(p.size), key=lambda b: (-s[h, 0, b], b))
            g_ref = sum((p.size - 2 * (m + 1) + 1) * p[b] for m, b in enumerate(order)) / p.size
            assert abs(gini[h] - g_ref) < 1e-14
            assert abs(tau[h] - (tmin + g_ref * (tmax - tmin))) < 1e-14
            acc, k = 0.0, 0
            for b in order:
                acc += p[b]
                k += 1
                if acc >= tau[h]:
                    break
            assert sorted(order[:k]) == list(sel[h][0])
            if k > 1:                                   # minimal: one block fewer falls short
                assert sum(p[b] for b in order[:k - 1]) < tau[h]
    # monotone in the threshold; tau = 0 keeps exactly one block; peaked head keeps fewer blocks
    a, _, _ = O.adaptive_selection(q, K, N, False, 0.3, 0.3)
    b, _, _ = O.adaptive_selection(q, K, N, False, 0.8, 0.8)
    z, _, _ = O.adaptive_selection(q, K, N, False, 0.0, 0.0)
    for h in range(H):
        assert set(a[h][0]) <= set(b[h][0]) and len(z[h][0]) == 1


def test_adaptive_selection_per_group_gini_is_averaged():
    H, d, Lq, N = 1, 8, 48, 64 * 9
    q, K = rnd((Lq, H, d), 62, 2.0), rnd((N, H, d), 63)
    sel, gini, tau = O.adaptive_selection(q, K, N, False, 0.2, 0.9, group_tokens=16)
    s = O.block_scores(q, K, 16)
    gs = []
    for g in range(3):
        p = O.block_weights(s[0, g], np.ones(9, bool))
        gs.append(O.gini_of_weights(np.sort(p)[::-1]))
    assert abs(gini[0] - np.mean(gs)) < 1e-14 and len(sel[0]) == 3


# ---------------------------------------------------------------- inter- / intra-chunk granularity
def test_mixed_selection_reduces_to_plain_selection():
    """One page per inter-chunk block and no intra-chunk region is the plain per-page selection."""
    q, K = rnd((12, 2, 8), 70), rnd((300, 2, 8), 71)
    for causal, q_pos0 in ((False, 300), (True, 200)):
        ref, s_ref = O.select_blocks(q, K, q_pos0, causal, [2, 3])
        got, s_got = O.select_blocks_mixed(q, K, q_pos0, causal, [2, 3], inter_pages=1, intra_first_page=-1)
        assert all(np.array_equal(got[h][0], ref[h][0]) for h in range(2))
        assert np.allclose(s_got, s_ref, rtol=0, atol=1e-14)


def test_coarse_block_score_is_token_weighted_mean_of_its_pages():
    """mean over a 128-token block = (c0 mean0 + c1 mean1) / (c0 + c1): the coarse score follows from
    the per-page scores and the page token counts (here the last block is one and a bit pages)."""
    N = 64 * 4 + 64 + 10
    q, K = rnd((7, 1, 8), 72), rnd((N, 1, 8), 73)
    page = O.block_scores(q, K)[0, 0]
    _, s = O.select_blocks_mixed(q, K, N, False, [1], inter_pages=2, intra_first_page=-1)
    cnt = [O.block_count(b, N) for b in range(O.n_blocks(N))]
    for c in range(3):
        b0, b1 = 2 * c, 2 * c + 1
        want = (cnt[b0] * page[b0] + cnt[b1] * page[b1]) / (cnt[b0] + cnt[b1])
        assert abs(s[0, 0, c] - want) < 1e-12


def test_mixed_selection_brute_force_and_intra_always_on():
    """Pure-Python loops over tokens: coarse blocks ranked by their own mean key, chunk pages always kept."""
    N, H, d, Lq = 64 * 5 + 20, 2, 4, 5
    q, K = rnd((Lq, H, d), 74), rnd((N, H, d), 75)
    p0 = 4                                    # pages 4 and 5 belong to the current chunk
    got, _ = O.select_blocks_mixed(q, K, N, False, [1, 2], inter_pages=2, intra_first_page=p0)
    for h in range(H):
        qbar = [sum(float(q[i, h, c]) for i in range(Lq)) / Lq for c in range(d)]
        sc = []
        for c in range(2):                    # coarse blocks = pages (0,1) and (2,3)
            toks = range(128 * c, 128 * c + 128)
            kbar = [sum(float(K[j, h, e]) for j in toks) / 128 for e in range(d)]
            sc.append(sum(a * b for a, b in zip(qbar, kbar)) / math.sqrt(d))
        keep = brute.topk_blocks(sc, [True, True], [1, 2][h])
        pages = sorted(sum(([2 * c, 2 * c + 1] for c in keep), [])) + [4, 5]
        assert got[h][0].tolist() == pages
    # an intra-chunk budget selects among the chunk's own pages only, by their own scores
    got2, s2 = O.select_blocks_mixed(q, K, N, False, [0, 0], inter_pages=2, intra_first_page=p0, intra_budgets=[1, 1])
    for h in range(H):
        assert got2[h][0].tolist() == [4 + int(np.argmax(s2[h, 0, 2:]))]


def test_mixed_selection_causal_candidates_and_ragged_inter_region():
    N = 64 * 7
    q, K = rnd((4, 1, 4), 76), rnd((N, 1, 4), 77)
    ranges, n_inter = O.mixed_candidates(N, 2, 5)      # 5 history pages -> blocks (0,1), (2,3), (4)
    assert n_inter == 3 and ranges[:3] == [(0, 128), (128, 256), (256, 320)] and ranges[3:] == [(320, 384), (384, 448)]
    # last query position 200: candidates are the blocks that start at or before it
    got, _ = O.select_blocks_mixed(q, K, 197, True, [-1], inter_pages=2, intra_first_page=5)
    assert got[0][0].tolist() == [0, 1, 2, 3]


# ---------------------------------------------------------------- HKV Stage 2 retrieval as a candidate mask
def test_kv_page_size_from_the_paper():
    """8 frames of 1560 tokens per KV page (Sec. 3.2) = 195 blocks of 64; 4 pages = 49,920 tokens."""
    rows = [l.split() for l in open(os.path.join(GOLD, "hkv_active_kv_tokens.txt")) if l[0] != "#"]
    kp, frames, tpf, total = map(int, rows[0])
    assert frames * tpf == 195 * O.BLOCK and kp * 195 == O.n_blocks(total)


def test_kv_page_retrieval_brute_force_and_reduction():
    N, H, d, Lq = 64 * 7 + 30, 2, 4, 6
    q, K = rnd((Lq, H, d), 80), rnd((N, H, d), 81)
    got, alpha = O.retrieve_kv_pages(q, K, kv_page_blocks=2, top_kp=2)
    sc = []
    for j in range(4):                                       # pages of 128 tokens, the last one short
        toks = range(128 * j, min(N, 128 * j + 128))
        tot = 0.0
        for h in range(H):
            qbar = [sum(float(q[i, h, c]) for i in range(Lq)) / Lq for c in range(d)]
            kbar = [sum(float(K[t, h, c]) for t in toks) / len(toks) for c in range(d)]
            tot += sum(a * b for a, b in zip(qbar, kbar))
        sc.append(tot / H / math.sqrt(d))
    assert np.allclose(alpha, sc, rtol=0, atol=1e-13)
    assert got.tolist() == brute.topk_blocks(sc, [True] * 4, 2)
    # one head, one block per page: the page score is the block score of the plain selection
    q1, K1 = q[:, :1], K[:, :1]
    a1 = O.kv_page_scores(q1, K1, 1)
    assert np.allclose(a1, O.block_scores(q1, K1)[0, 0], rtol=0, atol=1e-14)
    sel, _ = O.select_blocks(q1, K1, N, False, [3])
    assert O.retrieve_kv_pages(q1, K1, 1, 3)[0].tolist() == sel[0][0].tolist()


def test_retrieved_pages_mask_the_selection():
    N = 64 * 12
    q, K = rnd((5, 2, 4), 82), rnd((N, 2, 4), 83)
    full, _ = O.select_blocks_mixed(q, K, N, False, [3, 3], inter_pages=1)
    same, _ = O.select_blocks_mixed(q, K, N, False, [3, 3], inter_pages=1, kv_pages=[0, 1, 2, 3], kv_page_blocks=3)
    assert all(same[h][0].tolist() == full[h][0].tolist() for h in range(2))      # every page retrieved: no mask
    got, s = O.select_blocks_mixed(q, K, N, False, [3, 5], inter_pages=1, kv_pages=[1, 3], kv_page_blocks=3)
    allowed = [3, 4, 5, 9, 10, 11]
    for h in range(2):
        assert set(got[h][0].tolist()) <= set(allowed)
        best = sorted(allowed, key=lambda b: (-s[h, 0, b], b))[:[3, 5][h]]
        assert got[h][0].tolist() == sorted(best)
    # a budget beyond the retrieved pages takes all of them and nothing else; the chunk's own pages are never masked
    got2, _ = O.select_blocks_mixed(q, K, N, False, [-1, 99], inter_pages=2, intra_first_page=10,
                                    kv_pages=[0], kv_page_blocks=3)
    assert all(got2[h][0].tolist() == [0, 1, 10, 11] for h in range(2))   # block (2, 3) straddles the page end


# ---------------------------------------------------------------- row subsets and the state form
@pytest.mark.parametrize("causal,group_tokens", [(False, 0), (True, 0), (False, 128), (True, 128)])
def test_row_subset_and_state_form_match_brute_force_on_those_rows(causal, group_tokens):
    """The full-size GPU parity cases evaluate the oracle on a subset of query rows
    (rows=...) and, for non-causal cases, with the linear branch in its state form.
    Both must give, on the chosen rows, what the pure-Python brute force gives for them,
    and exact zeros on every other row."""
    H, d, Lq, N = 2, 8, 300, 330                    # 6 blocks (tail 10), 3 query groups of 128
    q, K, V = rnd((Lq, H, d), 40), rnd((N, H, d), 41), rnd((N, H, d), 42)
    q_pos0 = N - Lq if causal else N
    sel, _ = O.select_blocks(q, K, q_pos0, causal, [2, 3], group_tokens)
    rows = np.array([0, 1, 127, 128, 131, 255, 256, 299])
    groups = O.group_bounds(Lq, group_tokens)
    g_of = lambda i: next(g for g, (a, e) in enumerate(groups) if a <= i < e)
    keysets = [[[j for b in sel[h][g_of(i)] for j in range(64 * int(b), min(N, 64 * int(b) + 64))]
                if i in rows else [] for i in range(Lq)] for h in range(H)]
    sp_ref = np.array(brute.attention_rows(q, K, V, N, H, d, Lq, q_pos0, causal, keysets))
    lin_ref = np.array(brute.linear_rows(q, K, V, N, H, d, Lq, q_pos0, causal))
    other = np.setdiff1d(np.arange(Lq), rows)
    lin_ref[other] = 0.0
    sp = O.sparse_branch(q, K, V, sel, q_pos0, causal, group_tokens, rows=rows)
    lp = O.linear_parallel(q, K, V, q_pos0, causal, rows=rows)
    assert np.abs(sp - sp_ref).max() < 1e-12 and np.abs(sp[other]).max() == 0.0
    assert np.abs(lp - lin_ref).max() < 1e-12 and np.abs(lp[other]).max() == 0.0
    for form in ("parallel", "state"):
        r = O.hsa_forward(q, K, V, q_pos0, causal, sel, group_tokens, rows=rows, linear_form=form)
        assert np.abs(r["O_sp"] - sp_ref).max() < 1e-12
        assert np.abs(r["O_lin"] - lin_ref).max() < 1e-11
        assert np.abs(r["out"] - (sp_ref + lin_ref)).max() < 1e-11
        assert np.abs(r["out"][other]).max() == 0.0
        full = O.hsa_forward(q, K, V, q_pos0, causal, sel, group_tokens, linear_form=form)
        assert np.abs(full["out"][rows] - r["out"][rows]).max() < 1e-11
    # the same with gates: rows outside the subset stay exactly zero
    g1, g2 = rnd((Lq, H), 43), rnd((Lq, H, d), 44)
    r = O.hsa_forward(q, K, V, q_pos0, causal, sel, group_tokens, g1, g2, 1, rows=rows, linear_form="state")
    sig = lambda x: 1.0 / (1.0 + np.exp(-x))
    assert np.abs(r["out"] - (sig(g1)[:, :, None] * lin_ref + sig(g2) * sp_ref)).max() < 1e-11
