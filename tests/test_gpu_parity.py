"""GPU parity: the C-ABI path against the CPU fp64 oracle on identical seeded bf16 inputs.
Selection must match bit-exactly (ties within 1e-6 forgiven); outputs within max-abs 2e-2 and
mean-abs 2e-3 (bf16 inputs, fp32 accumulation) plus a 1e-2 relative Frobenius bound."""
import numpy as np
import pytest
import torch

import hsa_harness as Hn
from oracle import hsa_oracle as O
from paper_2609_34606_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["cfg1a", "cfg1b", "cfg1_sharp", "mid_d64", "mid_d128", "mid_mix",
                                  "mid_causal", "mid_shuffle"])
def test_small_workloads_full_parity(name, cuda_device):
    Hn.run_case(W.WORKLOADS[name], cuda_device)


@pytest.mark.parametrize("name", ["mid_d128", "mid_mix", "mid_causal", "mid_d64", "cfg1b"])
def test_relu_feature_map(name, cuda_device):
    """phi(x) = max(x, 0) in every kernel that applies the feature map (fused and SIMT append, the
    forward epilogue, the stand-alone linear kernel, the causal intra-chunk part), with 1e-6 in the
    denominator: state, both branches and the merged output against the oracle's relu form."""
    res = Hn.run_case(W.WORKLOADS[name], cuda_device, fmap="relu")
    assert res["S_rel"] <= 1e-5 and res["z_rel"] <= 1e-5


def test_relu_rows_without_any_weight_are_zero(cuda_device):
    """Queries with no positive component have weight zero on every key: the linear branch of those
    rows is 0 / 1e-6 = 0 (no division by zero, no NaN), in the fused epilogue and in the stand-alone
    linear kernel; the other rows match the oracle."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_d128"]
    ctx = Hn.build_context(w, cuda_device, feature_map=1)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w).float()
    q[::3] = -q[::3].abs()            # every third row: all components negative
    q = q.to(torch.bfloat16)
    qd = q.to(cuda_device)
    si, sc = ctx.select_blocks(qd, W.gen_budgets(w).to(cuda_device))
    o_lin = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_SPARSE))
    out = Hn.f64(ctx.forward(qd, si, sc))
    o_sp = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_LINEAR))
    assert ctx.device_status() == 0
    assert np.isfinite(o_lin).all() and np.isfinite(out).all()
    assert not o_lin[::3].any()
    assert np.abs(out[::3] - o_sp[::3]).max() == 0.0
    ref = O.linear_parallel(Hn.f32(q), Hn.f32(K), Hn.f32(V), w.q_pos0, False, fmap="relu")
    Hn.assert_close(o_lin, ref, "O_lin (relu)")
    ctx.destroy()


@pytest.mark.parametrize("gates,act", [("head", 0), ("dim", 1), ("head", 1)])
def test_gated_merge(gates, act, cuda_device):
    Hn.run_case(W.WORKLOADS["mid_d128"], cuda_device, gates=gates, gate_act=act, check_state=False)


def test_per_tile_query_groups(cuda_device):
    Hn.run_case(W.WORKLOADS["mid_d128"], cuda_device, group_tokens=128, check_state=False)
    Hn.run_case(W.WORKLOADS["mid_causal"], cuda_device, group_tokens=128, check_state=False)


@pytest.mark.parametrize("name", ["cfg1a", "cfg1b", "mid_d128"])
def test_all_blocks_no_linear_equals_dense_attention(name, cuda_device):
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS[name]
    ctx = Hn.build_context(w, cuda_device)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    allsel = [[np.arange(w.n_blocks, dtype=np.int32)] for _ in range(w.H)]
    si, sc = Hn.selection_to_device(allsel, ctx.max_topk, cuda_device)
    out = ctx.forward(q.to(cuda_device), si, sc, q_pos0=w.q_pos0, causal=w.causal,
                      flags=hsa.HSA_FWD_NO_LINEAR)
    ref = O.dense_attention(Hn.f32(q), Hn.f32(K), Hn.f32(V), w.q_pos0, w.causal)
    Hn.assert_close(Hn.f64(out), ref, "dense")
    assert ctx.device_status() == 0


def test_page_table_permutation_invariance_and_determinism(cuda_device):
    w = W.WORKLOADS["mid_shuffle"]
    import dataclasses
    w_id = dataclasses.replace(w, shuffle_pages=False)
    outs = []
    for wl in (w, w_id, w):
        ctx = Hn.build_context(wl, cuda_device)
        Hn.append_history(ctx, wl, cuda_device)
        q = W.gen_query(wl).to(cuda_device)
        si, sc = ctx.select_blocks(q, W.gen_budgets(wl).to(cuda_device))
        outs.append((ctx.forward(q, si, sc).cpu(), si.cpu(), sc.cpu()))
        ctx.destroy()
    for a, b in [(0, 1), (0, 2)]:
        assert torch.equal(outs[a][0], outs[b][0])           # same bits
        assert torch.equal(outs[a][2], outs[b][2])
        for h in range(w.H):
            n = int(outs[a][2][h, 0])
            assert torch.equal(outs[a][1][h, 0, :n], outs[b][1][h, 0, :n])


def test_incremental_append_matches_any_chunking(cuda_device):
    """Appending the same tokens in ragged pieces (partial tail pages continued) gives the same pool,
    key sums and selection; the state agrees to fp32 rounding."""
    w = W.WORKLOADS["mid_d128"]
    K, V = W.gen_history(w)
    res = []
    for pieces in ([333] * 7, [1, 63, 64, 65, 200, 300, 333, 333, 333, 333, 306], [200] * 11 + [131]):
        ctx = Hn.build_context(w, cuda_device)
        off = 0
        for n in pieces:
            ctx.append_kv(K[off:off + n].to(cuda_device), V[off:off + n].to(cuda_device))
            off += n
        assert off == w.N and ctx.n_tokens == w.N
        q = W.gen_query(w).to(cuda_device)
        si, sc = ctx.select_blocks(q, W.gen_budgets(w).to(cuda_device))
        out = ctx.forward(q, si, sc)
        res.append((ctx.k_pool.clone().cpu(), Hn.f64(ctx.ksum[:, :w.n_blocks]), Hn.f64(ctx.S),
                    Hn.selection_lists(si, sc), Hn.f64(out)))
        ctx.destroy()
    # rows of the partial tail page beyond N are never written, so compare only valid rows
    valid_rows = w.N
    for r in res[1:]:
        a = res[0][0].view(torch.bfloat16).view(-1, w.H, 64, w.d)
        b = r[0].view(torch.bfloat16).view(-1, w.H, 64, w.d)
        full = valid_rows // 64
        assert torch.equal(a[:full], b[:full])
        assert torch.equal(a[full, :, :valid_rows % 64], b[full, :, :valid_rows % 64])
        assert np.allclose(r[1], res[0][1], rtol=1e-6, atol=1e-6)
        assert np.linalg.norm(r[2] - res[0][2]) <= 1e-5 * np.linalg.norm(res[0][2])
        assert all(list(x[0]) == list(y[0]) for x, y in zip(r[3], res[0][3]))
        assert np.abs(r[4] - res[0][4]).max() <= 4e-3


def test_rewind_undoes_the_last_append_without_restoring_anything(cuda_device):
    """Appending a chunk, taking it back with hsa_rewind and appending another one (here twice, and
    with a history that ends inside a block, so that the tail block's key sum is involved) must
    leave exactly what a context that never saw the dropped chunks holds: state, key sums, selection
    and output bit for bit -- with no copy of the state by the caller."""
    w = W.WORKLOADS["mid_d128"]            # chunks of 333 tokens: every chunk starts inside a block
    ks = [W.gen_kv_chunk(w, c) for c in range(w.n_chunks + 2)]
    q = W.gen_query(w).to(cuda_device)
    budgets = W.gen_budgets(w).to(cuda_device)

    def finish(ctx):
        si, sc = ctx.select_blocks(q, budgets)
        out = ctx.forward(q, si, sc)
        assert ctx.device_status() == 0
        return (ctx.S.clone(), ctx.z.clone(), ctx.ksum[:, :ctx.n_blocks].clone(), sc.clone(), si.clone(), out.clone())

    ref_ctx = Hn.build_context(w, cuda_device, extra_pages=8)
    for c in range(w.n_chunks):
        ref_ctx.append_kv(ks[c][0].to(cuda_device), ks[c][1].to(cuda_device))
    ref = finish(ref_ctx)

    ctx = Hn.build_context(w, cuda_device, extra_pages=8)
    for c in range(w.n_chunks - 1):
        ctx.append_kv(ks[c][0].to(cuda_device), ks[c][1].to(cuda_device))
    n0 = ctx.n_tokens
    assert n0 % 64 != 0
    for dropped in (w.n_chunks, w.n_chunks + 1):          # two chunks that are taken back again
        ctx.append_kv(ks[dropped][0].to(cuda_device), ks[dropped][1].to(cuda_device))
        assert ctx.n_tokens == n0 + w.chunk
        ctx.rewind(n0)
        assert ctx.n_tokens == n0
    ctx.append_kv(ks[w.n_chunks - 1][0].to(cuda_device), ks[w.n_chunks - 1][1].to(cuda_device))
    got = finish(ctx)
    for a, b in zip(got, ref):
        assert torch.equal(a, b)
    ctx.destroy()
    ref_ctx.destroy()


def test_edge_cases(cuda_device):
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_d64"]
    ctx = Hn.build_context(w, cuda_device, extra_pages=1)
    q = W.gen_query(w).to(cuda_device)
    budgets = W.gen_budgets(w).to(cuda_device)
    # empty history: nothing to select, output exactly zero
    si, sc = ctx.select_blocks(q, budgets)
    out = ctx.forward(q, si, sc)
    assert int(sc.sum()) == 0 and float(out.float().abs().max()) == 0.0
    # single token history: both branches return v_0 (closed form), out = 2 v_0
    k, v = W.gen_kv_chunk(w, 0)
    ctx.append_kv(k[:1].to(cuda_device), v[:1].to(cuda_device))
    si, sc = ctx.select_blocks(q, budgets)
    out = ctx.forward(q, si, sc)
    assert sc.tolist() == [[1]] * w.H
    ref = 2.0 * v[:1].float().expand(w.Lq, -1, -1)
    assert float((out.float().cpu() - ref).abs().max()) <= 2e-2
    # zero budget: out == linear branch alone; both branches off: zeros
    zero = torch.zeros_like(budgets)
    si0, sc0 = ctx.select_blocks(q, zero)
    a = ctx.forward(q, si0, sc0)
    b = ctx.forward(q, si, sc, flags=hsa.HSA_FWD_NO_SPARSE)
    assert int(sc0.sum()) == 0 and torch.equal(a, b)
    c = ctx.forward(q, si, sc, flags=hsa.HSA_FWD_NO_SPARSE | hsa.HSA_FWD_NO_LINEAR)
    assert float(c.float().abs().max()) == 0.0
    # out of pages, oversize chunk
    kk, vv = W.gen_kv_chunk(w, 1)
    for _ in range(w.n_chunks + 2):
        try:
            ctx.append_kv(kk.to(cuda_device), vv.to(cuda_device))
        except hsa.HSAError as e:
            assert e.code == hsa.HSA_ERR_OUT_OF_PAGES
            break
    else:
        raise AssertionError("pool never filled")
    with pytest.raises(hsa.HSAError):
        ctx.append_kv(torch.cat([kk, kk]).to(cuda_device), torch.cat([vv, vv]).to(cuda_device))
    assert ctx.device_status() == 0
    ctx.destroy()


def test_tiles_without_work_write_exact_zeros(cuda_device):
    """A tile with no selected block and no linear branch never looks at its queries; its output
    must still be exact zeros (the output tile is staged where the query tile lands), every time."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["cfg2"]
    ctx = Hn.build_context(w, cuda_device, max_topk=w.topk)
    k, v = W.gen_kv_chunk(w, 0)
    ctx.append_kv(k.to(cuda_device), v.to(cuda_device))
    q = (W.gen_query(w) + 3.0).to(cuda_device)   # nowhere near zero, so stale queries would show
    si, sc = ctx.select_blocks(q, torch.zeros(w.H, dtype=torch.int32, device=cuda_device))
    assert int(sc.sum()) == 0
    for _ in range(25):
        out = ctx.forward(q, si, sc, flags=hsa.HSA_FWD_NO_LINEAR)
        assert int(torch.count_nonzero(out.view(torch.int16) & 0x7FFF)) == 0
    assert ctx.device_status() == 0
    ctx.destroy()


def test_bad_selection_index_is_flagged_not_followed(cuda_device):
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_d64"]
    ctx = Hn.build_context(w, cuda_device)
    Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w).to(cuda_device)
    sel = [[np.array([1, 10_000_000], dtype=np.int32)] for _ in range(w.H)]
    si, sc = Hn.selection_to_device(sel, ctx.max_topk, cuda_device)
    ctx.forward(q, si, sc)
    assert ctx.device_status() == hsa.HSA_ERR_DEVICE_BOUNDS
    assert ctx.device_status() == 0          # the status word is cleared by the read
    # causal forward with the linear branch needs the query chunk to be the last append
    with pytest.raises(hsa.HSAError) as e:
        ctx.forward(q, si, sc, q_pos0=0, causal=True)
    assert e.value.code == hsa.HSA_ERR_UNSUPPORTED
    ctx.destroy()


def test_selection_kcap_clamp_and_large_candidate_sets(cuda_device):
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_mix"]
    ctx = Hn.build_context(w, cuda_device, max_topk=7)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    budgets = torch.full((w.H,), -1, dtype=torch.int32)
    si, sc = ctx.select_blocks(q.to(cuda_device), budgets.to(cuda_device))
    assert sc.flatten().tolist() == [7] * w.H
    assert si[:, 0, :7].cpu().tolist() == [list(range(7))] * w.H
    assert ctx.device_status() == hsa.HSA_ERR_DEVICE_BOUNDS
    ctx.destroy()


@pytest.mark.parametrize("name,fmap", [("cfg2", "elu1"), ("cfg2", "relu")])
def test_full_size_sampled_parity(name, fmap, cuda_device):
    """Full-size workload in the launch configuration the benchmark times (and the same with the relu
    feature map): selection checked in full, outputs on the first and last query tile plus seeded
    random rows (rows are independent given the selection), state and key sums in full."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS[name]
    ctx = Hn.build_context(w, cuda_device, max_topk=max(w.topk, 1), feature_map=1 if fmap == "relu" else 0)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    qd = q.to(cuda_device)
    budgets = W.gen_budgets(w)
    qn, Kn, Vn = Hn.f32(q), Hn.f32(K), Hn.f32(V)
    S_ref, z_ref = O.linear_state(Kn, Vn, fmap=fmap)
    assert np.linalg.norm(Hn.f64(ctx.S) - S_ref) <= 1e-5 * np.linalg.norm(S_ref)
    assert np.linalg.norm(Hn.f64(ctx.z) - z_ref) <= 1e-5 * np.linalg.norm(z_ref)
    si, sc = ctx.select_blocks(qd, budgets.to(cuda_device))
    sel_gpu = Hn.selection_lists(si, sc)
    sel_ref, scores = O.select_blocks(qn, Kn, w.q_pos0, w.causal, budgets.tolist())
    Hn.check_selection(sel_gpu, sel_ref, scores)
    rows = W.sample_rows(w, n_random=256).numpy()
    ref = O.hsa_forward(qn, Kn, Vn, w.q_pos0, w.causal, sel_gpu, rows=rows, linear_form="state", fmap=fmap)
    out = Hn.f64(ctx.forward(qd, si, sc))
    o_sp = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_LINEAR))
    o_lin = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_SPARSE))
    assert ctx.device_status() == 0
    Hn.assert_close(o_sp[rows], ref["O_sp"][rows], "O_sp")
    Hn.assert_close(o_lin[rows], ref["O_lin"][rows], "O_lin")
    Hn.assert_close(out[rows], ref["out"][rows], "out")
    # properties that hold at any size: finite everywhere; V == const would give const (checked small)
    assert np.isfinite(out).all()
    ctx.destroy()


def test_full_size_per_tile_selection_sampled(cuda_device):
    """cfg2 with one selection per 128-row query tile (37 groups x 12 heads, the granularity the
    sparse branch is defined at): every list against the oracle, outputs on sampled rows."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["cfg2"]
    gt = 128
    ctx = Hn.build_context(w, cuda_device, max_topk=w.topk)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    qd = q.to(cuda_device)
    budgets = W.gen_budgets(w)
    qn, Kn, Vn = Hn.f32(q), Hn.f32(K), Hn.f32(V)
    si, sc = ctx.select_blocks(qd, budgets.to(cuda_device), group_tokens=gt)
    assert tuple(sc.shape) == (w.H, 37)
    sel_gpu = Hn.selection_lists(si, sc)
    sel_ref, scores = O.select_blocks(qn, Kn, w.q_pos0, False, budgets.tolist(), gt)
    Hn.check_selection(sel_gpu, sel_ref, scores)
    assert len({tuple(x) for x in sel_gpu[0]}) > 1, "the groups of a head must not all pick the same blocks"
    rows = W.sample_rows(w, n_random=256).numpy()
    ref = O.hsa_forward(qn, Kn, Vn, w.q_pos0, False, sel_gpu, gt, rows=rows, linear_form="state")
    out = Hn.f64(ctx.forward(qd, si, sc, group_tokens=gt))
    o_sp = Hn.f64(ctx.forward(qd, si, sc, group_tokens=gt, flags=hsa.HSA_FWD_NO_LINEAR))
    assert ctx.device_status() == 0
    Hn.assert_close(o_sp[rows], ref["O_sp"][rows], "O_sp")
    Hn.assert_close(out[rows], ref["out"][rows], "out")
    assert np.isfinite(out).all()
    ctx.destroy()


def test_linformer_full_size_segments_sampled(cuda_device):
    """The Linformer form at the layer's own sizes: rank 256, segments of one 4680-token chunk,
    three segments, 12 heads; outputs on sampled rows (rows are independent)."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["cfg2_linformer"]
    rank, seg = 256, w.chunk
    ek, ev = W.gen_linformer_weights(w, rank, seg)
    ctx = hsa.HSAContext(w.H, w.d, max_pages=w.n_blocks, max_q_tokens=w.Lq, max_topk=w.topk,
                         lin_mode=hsa.HSA_LIN_LINFORMER, lin_rank=rank, lin_seg_tokens=seg,
                         e_k=ek.to(cuda_device), e_v=ev.to(cuda_device), device=cuda_device)
    for pool in (ctx.k_pool, ctx.v_pool, ctx.kc_pool, ctx.vc_pool):
        pool.fill_(0xFF)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    qd = q.to(cuda_device)
    budgets = W.gen_budgets(w)
    qn, Kn, Vn = Hn.f32(q), Hn.f32(K), Hn.f32(V)
    si, sc = ctx.select_blocks(qd, budgets.to(cuda_device))
    sel_gpu = Hn.selection_lists(si, sc)
    sel_ref, scores = O.select_blocks(qn, Kn, w.N, False, budgets.tolist())
    Hn.check_selection(sel_gpu, sel_ref, scores)
    rows = W.sample_rows(w, n_random=256).numpy()
    Kt, Vt = O.linformer_compress(Kn, Vn, Hn.f32(ek), Hn.f32(ev), seg)
    assert Kt.shape[0] == w.n_chunks * rank
    o_lin_ref = O.linformer_branch(qn[rows], Kt, Vt)
    o_sp_ref = O.sparse_branch(qn, Kn, Vn, sel_gpu, w.N, False, rows=rows)[rows]
    out = Hn.f64(ctx.forward(qd, si, sc))
    o_lin = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_SPARSE))
    assert ctx.device_status() == 0
    Hn.assert_close(o_lin[rows], o_lin_ref, "O_lin (Linformer)")
    Hn.assert_close(out[rows], o_lin_ref + o_sp_ref, "out")
    assert np.isfinite(out).all()
    ctx.destroy()


def test_safe_pass_when_later_blocks_dominate(cuda_device):
    """Scores of later blocks exceed the first block's row maximum by far more than the fixed
    exponent reference of the normal pass allows: the tile must be redone with a running maximum
    and still match the oracle (and ordinary inputs must never take that path)."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_d128"]
    ctx = Hn.build_context(w, cuda_device)
    K, V = W.gen_history(w)
    K = K.float()
    K[:128] *= 0.05          # the first step (blocks 0 and 1) barely scores
    K[128:] *= 12.0          # everything later scores tens of nats higher
    K = K.to(torch.bfloat16)
    off = 0
    while off < w.N:
        ctx.append_kv(K[off:off + w.chunk].to(cuda_device), V[off:off + w.chunk].to(cuda_device))
        off += w.chunk
    q = W.gen_query(w)
    allsel = [[np.arange(w.n_blocks, dtype=np.int32)] for _ in range(w.H)]
    si, sc = Hn.selection_to_device(allsel, ctx.max_topk, cuda_device)
    assert ctx.safe_pass_tiles() == 0
    out = ctx.forward(q.to(cuda_device), si, sc, flags=hsa.HSA_FWD_NO_LINEAR)
    assert ctx.device_status() == 0
    assert ctx.safe_pass_tiles() > 0
    ref = O.dense_attention(Hn.f32(q), Hn.f32(K), Hn.f32(V), w.q_pos0, False)
    s = Hn.err_stats(Hn.f64(out), ref)
    assert s["rel_fro"] <= 1e-2 and s["max_abs"] <= 4e-2, s
    # ordinary N(0,1) inputs stay on the normal pass
    ctx2 = Hn.build_context(w, cuda_device)
    Hn.append_history(ctx2, w, cuda_device)
    out2 = ctx2.forward(q.to(cuda_device), si, sc)
    assert ctx2.safe_pass_tiles() == 0 and ctx2.device_status() == 0
    ctx.destroy()
    ctx2.destroy()


def _sampled_forward_check(w, ctx, K, V, q, device, n_random=192):
    """Selection in full, outputs on sampled rows, for a context whose history is (K, V)."""
    from paper_2609_34606_b200 import hsa
    qd = q.to(device)
    budgets = W.gen_budgets(w)
    qn = Hn.f32(q)
    si, sc = ctx.select_blocks(qd, budgets.to(device))
    sel_gpu = Hn.selection_lists(si, sc)
    sel_ref, scores = O.select_blocks(qn, K, K.shape[0], False, budgets.tolist())
    Hn.check_selection(sel_gpu, sel_ref, scores)
    rows = W.sample_rows(w, n_random=n_random).numpy()
    ref = O.hsa_forward(qn, K, V, K.shape[0], False, sel_gpu, rows=rows, linear_form="state")
    out = Hn.f64(ctx.forward(qd, si, sc))
    o_sp = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_LINEAR))
    o_lin = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_SPARSE))
    assert ctx.device_status() == 0
    Hn.assert_close(o_sp[rows], ref["O_sp"][rows], "O_sp")
    # the linear branch on its own: inside `out` it is an order of magnitude below the sparse branch
    Hn.assert_close(o_lin[rows], ref["O_lin"][rows], "O_lin")
    Hn.assert_close(out[rows], ref["out"][rows], "out")
    assert np.isfinite(out).all() and np.isfinite(o_lin).all()
    return sel_gpu


@pytest.mark.parametrize("name", ["cfg3", "cfg4"])
def test_long_history_and_head_adaptive_budgets_sampled(name, cuda_device):
    """cfg3: 280,800-token history behind a shuffled page table, top-128; cfg4: scene-segment
    mixture with per-head budgets from {0,16,32,64,128,all}.  Selection is checked in full, the
    state in full, outputs on the first / last query tile plus seeded rows."""
    w = W.WORKLOADS[name]
    ctx = Hn.build_context(w, cuda_device, max_topk=w.n_blocks if w.budget_set else w.topk)
    Ks, Vs = [], []
    for c in range(w.n_chunks):
        k, v = W.gen_kv_chunk(w, c)
        ctx.append_kv(k.to(cuda_device), v.to(cuda_device))
        Ks.append(k.float().numpy())
        Vs.append(v.float().numpy())
    K, V = np.concatenate(Ks), np.concatenate(Vs)
    del Ks, Vs
    S_ref, z_ref = O.linear_state(K, V)
    assert np.linalg.norm(Hn.f64(ctx.S) - S_ref) <= 1e-5 * np.linalg.norm(S_ref)
    assert np.linalg.norm(Hn.f64(ctx.z) - z_ref) <= 1e-5 * np.linalg.norm(z_ref)
    sel = _sampled_forward_check(w, ctx, K, V, W.gen_query(w), cuda_device)
    if w.mixture:
        # structure of the mixture: every head with a budget <= 128 selects inside the queries' segment
        seg = W.query_segment(w)
        lo, hi = seg * w.seg_chunks * w.chunk // 64, ((seg + 1) * w.seg_chunks * w.chunk + 63) // 64
        budgets = W.gen_budgets(w).tolist()
        for h, b in enumerate(budgets):
            if 0 < b <= 128:
                assert all(lo <= x <= hi for x in sel[h][0]), (h, b)
    ctx.destroy()


@pytest.mark.parametrize("layer", [0, 29])
def test_rollout_steps_sampled(layer, cuda_device):
    """cfg5 shape: append a chunk, select, forward, 80 times on one layer's context (the first and
    the last layer of the stack); the oracle checks the steps at chunks 0, 1, 39 and 79 (its linear
    state is carried along in fp64)."""
    w = W.WORKLOADS["cfg5"]
    ctx = Hn.build_context(w, cuda_device, max_topk=w.topk)
    Ks, Vs = [], []
    S = np.zeros((w.H, w.d, w.d))
    z = np.zeros((w.H, w.d))
    budgets = W.gen_budgets(w)
    bd = budgets.to(cuda_device)
    sel = ctx.alloc_selection(w.Lq)
    for c in range(w.n_chunks):
        k, v = W.gen_kv_chunk(w, c, layer=layer)
        ctx.append_kv(k.to(cuda_device), v.to(cuda_device))
        kn, vn = k.float().numpy(), v.float().numpy()
        Ks.append(kn)
        Vs.append(vn)
        dS, dz = O.linear_state(kn, vn)
        S += dS
        z += dz
        q = W.gen_query(w, step=c, layer=layer)
        qd = q.to(cuda_device)
        ctx.select_blocks(qd, bd, sel=sel)
        out = ctx.forward(qd, sel[0], sel[1])
        if c in (0, 1, 39, 79):
            K, V = np.concatenate(Ks), np.concatenate(Vs)
            qn = Hn.f32(q)
            sel_gpu = Hn.selection_lists(sel[0], sel[1])
            sel_ref, scores = O.select_blocks(qn, K, K.shape[0], False, budgets.tolist())
            Hn.check_selection(sel_gpu, sel_ref, scores)
            rows = W.sample_rows(w, n_random=64).numpy()
            o_sp = O.sparse_branch(qn, K, V, sel_gpu, K.shape[0], False, rows=rows)
            o_lin = O.linear_from_state(qn, S, z)
            ref = (o_sp + o_lin)[rows]
            Hn.assert_close(Hn.f64(out)[rows], ref, f"out@chunk{c}")
            assert np.linalg.norm(Hn.f64(ctx.S) - S) <= 1e-5 * np.linalg.norm(S)
            del K, V
    assert ctx.device_status() == 0 and ctx.n_tokens == w.N
    ctx.destroy()


def test_linformer_linear_branch(cuda_device):
    """The paper's own linear branch: per appended segment K~ = E_K^T K, V~ = E_V^T V (rank rows),
    softmax attention over all compressed rows, merged with the sparse branch."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_linformer"]
    rank, seg = 128, w.chunk
    ek, ev = W.gen_linformer_weights(w, rank, seg)
    ctx = hsa.HSAContext(w.H, w.d, max_pages=w.n_blocks, max_q_tokens=max(w.Lq, w.chunk), max_topk=w.n_blocks,
                         lin_mode=hsa.HSA_LIN_LINFORMER, lin_rank=rank, lin_seg_tokens=seg,
                         e_k=ek.to(cuda_device), e_v=ev.to(cuda_device), device=cuda_device)
    ctx.k_pool.fill_(0xFF)
    ctx.v_pool.fill_(0xFF)
    ctx.kc_pool.fill_(0xFF)
    ctx.vc_pool.fill_(0xFF)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    qd = q.to(cuda_device)
    budgets = W.gen_budgets(w)
    qn, Kn, Vn = Hn.f32(q), Hn.f32(K), Hn.f32(V)
    si, sc = ctx.select_blocks(qd, budgets.to(cuda_device))
    sel_gpu = Hn.selection_lists(si, sc)
    sel_ref, scores = O.select_blocks(qn, Kn, w.N, False, budgets.tolist())
    Hn.check_selection(sel_gpu, sel_ref, scores)
    Kt, Vt = O.linformer_compress(Kn, Vn, Hn.f32(ek), Hn.f32(ev), seg)
    assert Kt.shape[0] == w.n_chunks * rank
    o_lin_ref = O.linformer_branch(qn, Kt, Vt)
    o_sp_ref = O.sparse_branch(qn, Kn, Vn, sel_gpu, w.N, False)
    out = Hn.f64(ctx.forward(qd, si, sc))
    o_lin = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_SPARSE))
    o_sp = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_LINEAR))
    assert ctx.device_status() == 0
    Hn.assert_close(o_sp, o_sp_ref, "O_sp")
    Hn.assert_close(o_lin, o_lin_ref, "O_lin (Linformer)")
    Hn.assert_close(out, o_lin_ref + o_sp_ref, "out")
    # whole segments only
    k, v = W.gen_kv_chunk(w, 0)
    with pytest.raises(hsa.HSAError) as e:
        ctx.append_kv(k[:100].to(cuda_device), v[:100].to(cuda_device))
    assert e.value.code in (hsa.HSA_ERR_UNSUPPORTED, hsa.HSA_ERR_OUT_OF_PAGES)
    ctx.destroy()


@pytest.mark.parametrize("n_segs,k_scale,split_blocks,gates,rank", [
    (1, None, 0, None, 128),          # one compressed step: both softmax groups start in different segments
    (2, None, 0, "head", 128),        # gated merge of the two segments' results
    (4, (0.05, 12.0), 0, None, 128),  # later segments / blocks dominate: both segments overflow the fixed reference
    (4, None, 4, None, 128),          # long lists split over CTAs: the two-launch form
    (3, None, 0, None, 192),          # three compressed pages per segment: an odd page count, a half-filled tile
    (1, None, 0, None, 64),           # the smallest rank: one compressed page in all
])
def test_linformer_segments_inside_the_forward_kernel(n_segs, k_scale, split_blocks, gates, rank, cuda_device):
    """The Linformer form runs as one launch whose loop walks the compressed pool first and the
    selected pages second, each with its own accumulator, exponent reference and row sums.  Cases:
    a single compressed step, gates, a history whose later parts outweigh the first step by far more
    than the fixed reference allows (the tile is redone with running maxima in both segments), the
    split-list configuration, which keeps the form with two launches, and ranks that are not a
    multiple of the compression kernel's 128-row tile."""
    from paper_2609_34606_b200 import hsa
    base = W.WORKLOADS["mid_linformer"]
    w = W.Workload("linf_case", H=base.H, d=128, Lq=300, chunk=base.chunk, n_chunks=n_segs, topk=6, seed=90 + n_segs)
    seg = w.chunk
    ek, ev = W.gen_linformer_weights(w, rank, seg)
    ctx = hsa.HSAContext(w.H, w.d, max_pages=w.n_blocks, max_q_tokens=max(w.Lq, w.chunk), max_topk=w.n_blocks,
                         lin_mode=hsa.HSA_LIN_LINFORMER, lin_rank=rank, lin_seg_tokens=seg,
                         e_k=ek.to(cuda_device), e_v=ev.to(cuda_device), device=cuda_device,
                         split_blocks=split_blocks)
    for pool in (ctx.k_pool, ctx.v_pool, ctx.kc_pool, ctx.vc_pool):
        pool.fill_(0xFF)
    K, V = W.gen_history(w)
    if k_scale is not None:
        K = K.float()
        K[:seg] *= k_scale[0]     # the first segment (and the first blocks) barely score
        K[seg:] *= k_scale[1]     # everything later scores far higher
        K = K.to(torch.bfloat16)
    for c in range(n_segs):
        ctx.append_kv(K[c * seg:(c + 1) * seg].to(cuda_device), V[c * seg:(c + 1) * seg].to(cuda_device))
    q = W.gen_query(w)
    qd = q.to(cuda_device)
    qn, Kn, Vn = Hn.f32(q), Hn.f32(K), Hn.f32(V)
    allsel = [[np.arange(w.n_blocks, dtype=np.int32)] for _ in range(w.H)]
    si, sc = Hn.selection_to_device(allsel, ctx.max_topk, cuda_device)
    g_lin = g_sp = None
    wl = ws = 1.0
    if gates:
        g_lin, g_sp = W.gen_gates(w, per_dim=False)
        wl, ws = Hn.f64(g_lin)[..., None], Hn.f64(g_sp)[..., None]
        g_lin, g_sp = g_lin.to(cuda_device), g_sp.to(cuda_device)
    Kt, Vt = O.linformer_compress(Kn, Vn, Hn.f32(ek), Hn.f32(ev), seg)
    if k_scale is not None:
        # logits of a few hundred: the bf16 rounding of the stored compressed rows (0.4 % of a logit)
        # is no longer small against 1, so this case takes the rows as the pool holds them
        Kt = Hn.f64(torch.from_numpy(Kt).to(torch.bfloat16))
        Vt = Hn.f64(torch.from_numpy(Vt).to(torch.bfloat16))
    o_lin_ref = O.linformer_branch(qn, Kt, Vt)
    o_sp_ref = O.dense_attention(qn, Kn, Vn, w.N, False)   # every block selected
    assert ctx.safe_pass_tiles() == 0
    out = Hn.f64(ctx.forward(qd, si, sc, g_lin=g_lin, g_sp=g_sp))
    o_lin = Hn.f64(ctx.forward(qd, si, sc, flags=hsa.HSA_FWD_NO_SPARSE))
    assert ctx.device_status() == 0
    redone = ctx.safe_pass_tiles()
    assert (redone > 0) == (k_scale is not None)
    tol = dict(rel_fro=1e-2, max_abs=4e-2 if k_scale is not None else 2e-2)
    for got, ref, what in ((o_lin, o_lin_ref, "O_lin"), (out, wl * o_lin_ref + ws * o_sp_ref, "out")):
        e = Hn.err_stats(got, ref)
        assert e["rel_fro"] <= tol["rel_fro"] and e["max_abs"] <= tol["max_abs"], (what, e)
    ctx.destroy()


def test_linformer_form_with_one_selection_per_query_tile(cuda_device):
    """The compressed segment in front of per-tile lists: every query tile walks the same compressed
    pool, then its own selection."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_linformer"]
    rank, seg, gtok = 128, w.chunk, 128
    ek, ev = W.gen_linformer_weights(w, rank, seg)
    ctx = hsa.HSAContext(w.H, w.d, max_pages=w.n_blocks, max_q_tokens=max(w.Lq, w.chunk), max_topk=w.n_blocks,
                         lin_mode=hsa.HSA_LIN_LINFORMER, lin_rank=rank, lin_seg_tokens=seg,
                         e_k=ek.to(cuda_device), e_v=ev.to(cuda_device), device=cuda_device)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    qd = q.to(cuda_device)
    budgets = W.gen_budgets(w)
    qn, Kn, Vn = Hn.f32(q), Hn.f32(K), Hn.f32(V)
    si, sc = ctx.select_blocks(qd, budgets.to(cuda_device), group_tokens=gtok)
    sel_gpu = Hn.selection_lists(si, sc)
    sel_ref, scores = O.select_blocks(qn, Kn, w.N, False, budgets.tolist(), gtok)
    Hn.check_selection(sel_gpu, sel_ref, scores)
    assert len(sel_gpu[0]) == (w.Lq + gtok - 1) // gtok and any(
        list(sel_gpu[0][0]) != list(sel_gpu[0][g]) for g in range(1, len(sel_gpu[0]))), "the tiles' lists should differ"
    Kt, Vt = O.linformer_compress(Kn, Vn, Hn.f32(ek), Hn.f32(ev), seg)
    ref = O.linformer_branch(qn, Kt, Vt) + O.sparse_branch(qn, Kn, Vn, sel_gpu, w.N, False, gtok)
    out = Hn.f64(ctx.forward(qd, si, sc, group_tokens=gtok))
    assert ctx.device_status() == 0
    Hn.assert_close(out, ref, "out")
    ctx.destroy()


@pytest.mark.parametrize("name,group_tokens", [("mid_mix", 0), ("mid_d128", 0), ("mid_d128", 128), ("cfg1_sharp", 0)])
def test_head_adaptive_selection(name, group_tokens, cuda_device):
    """Cumulative-mass selection with the Gini threshold map (tau_max = 1.00, tau_min = 0.35, the
    paper's best setting) against the oracle; a prefix length may differ only where the cumulative
    mass at the boundary is within 1e-6 of the threshold."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS[name]
    order = W.gen_page_order(w, w.n_blocks)
    ctx = hsa.HSAContext(w.H, w.d, max_pages=w.n_blocks, max_q_tokens=max(w.Lq, w.chunk), max_topk=w.n_blocks,
                         adaptive=True, page_order=order, device=cuda_device)
    K, V = Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w)
    qd = q.to(cuda_device)
    qn, Kn, Vn = Hn.f32(q), Hn.f32(K), Hn.f32(V)
    tmin, tmax = 0.35, 1.0
    si, sc, gt = ctx.select_blocks_adaptive(qd, tmin, tmax, group_tokens=group_tokens)
    assert ctx.device_status() == 0
    sel_gpu = Hn.selection_lists(si, sc)
    sel_ref, gini, tau = O.adaptive_selection(qn, Kn, w.N, False, tmin, tmax, group_tokens)
    assert np.allclose(gt[0].cpu().numpy(), gini, atol=1e-5) and np.allclose(gt[1].cpu().numpy(), tau, atol=1e-5)
    s = O.block_scores(qn, Kn, group_tokens)
    for h in range(w.H):
        for g in range(len(sel_ref[h])):
            a, b = list(sel_gpu[h][g]), list(sel_ref[h][g])
            if a != b:
                # tolerated only at a knife-edge of the cumulative mass
                p = O.block_weights(s[h, g], np.ones(s.shape[2], bool))
                cum = np.cumsum(np.sort(p)[::-1])
                k = min(len(a), len(b))
                assert abs(len(a) - len(b)) <= 1 and abs(cum[k - 1] - tau[h]) <= 1e-6, (h, g, len(a), len(b))
            assert a == sorted(set(a)) and len(a) >= 1
    # the selection drives the forward pass like any other
    ref = O.hsa_forward(qn, Kn, Vn, w.N, False, sel_gpu, group_tokens)
    out = Hn.f64(ctx.forward(qd, si, sc, group_tokens=group_tokens))
    Hn.assert_close(out, ref["out"], "out")
    ctx.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("name,causal", [("mid_d128", False), ("mid_mix", False), ("mid_causal", True), ("mid_d64", False)])
def test_inter_and_intra_chunk_granularity(name, causal, cuda_device):
    """128-token inter-chunk blocks against the head budgets plus the chunk's own 64-token pages
    (always on, then with their own budgets); the page lists drive the unchanged forward kernel."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS[name]
    ctx = Hn.build_context(w, cuda_device, causal=causal)
    K, V = Hn.append_history(ctx, w, cuda_device)
    Kn, Vn = Hn.f32(K), Hn.f32(V)
    q = W.gen_query(w)
    qn, qd = Hn.f32(q), q.to(cuda_device)
    N = Kn.shape[0]
    q_pos0 = w.q_pos0
    p0 = max(0, (N - w.chunk)) // 64            # page that holds the first token of the last chunk
    budgets = W.gen_budgets(w)
    intra_b = torch.full((w.H,), 2, dtype=torch.int32)

    def cands_of(pages, ranges):
        first = {t0 // 64: c for c, (t0, _) in enumerate(ranges)}
        return sorted({first[p] for p in pages if p in first})

    for inter_pages, first_page, ib in ((2, -1, None), (2, p0, None), (2, p0, intra_b), (1, p0, intra_b)):
        si, sc = ctx.select_blocks_ex(qd, budgets.to(cuda_device), inter_block_pages=inter_pages,
                                      intra_first_page=first_page,
                                      intra_budgets=None if ib is None else ib.to(cuda_device),
                                      q_pos0=q_pos0, causal=causal)
        assert ctx.device_status() == 0
        got = Hn.selection_lists(si, sc)
        ref, scores = O.select_blocks_mixed(qn, Kn, q_pos0, causal, budgets.tolist(), inter_pages, first_page,
                                            None if ib is None else ib.tolist())
        ranges, n_inter = O.mixed_candidates(N, inter_pages, first_page)
        for h in range(w.H):
            a, b = got[h][0].tolist(), ref[h][0].tolist()
            assert a == sorted(set(a))
            if a != b:   # only candidates whose score ties the weakest selected one may differ
                ca, cb = cands_of(a, ranges), cands_of(b, ranges)
                assert len(ca) == len(cb)
                diff = sorted(set(ca) ^ set(cb))
                for part in (range(0, n_inter), range(n_inter, len(ranges))):
                    sel_part = [c for c in cb if c in part]
                    d_part = [c for c in diff if c in part]
                    if d_part:
                        kth = min(scores[h, 0, c] for c in sel_part)
                        assert all(abs(scores[h, 0, c] - kth) <= Hn.TIE_EPS for c in d_part), (h, d_part)
        # the forward kernel runs on the page lists as they are
        rows = W.sample_rows(w, n_random=64).numpy()
        out = Hn.f64(ctx.forward(qd, si, sc, q_pos0=q_pos0, causal=causal, flags=hsa.HSA_FWD_NO_LINEAR))
        o_ref = O.sparse_branch(qn, Kn, Vn, got, q_pos0, causal, rows=rows)
        Hn.assert_close(out[rows], o_ref[rows], "O_sp")
    ctx.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["mid_d128", "mid_shuffle", "mid_d64"])
def test_kv_page_retrieval_mask_and_tier_migration(name, cuda_device):
    """Stage-2 page retrieval against the oracle, the retrieved pages as a candidate mask of the
    selection, and eviction / restore of blocks to pinned host memory (bit-exact round trip)."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS[name]
    ctx = Hn.build_context(w, cuda_device)
    K, V = Hn.append_history(ctx, w, cuda_device)
    Kn, Vn = Hn.f32(K), Hn.f32(V)
    q = W.gen_query(w)
    qn, qd = Hn.f32(q), q.to(cuda_device)
    N = Kn.shape[0]
    nblk = O.n_blocks(N)
    kvb = max(2, nblk // 5)                                   # five or six KV pages, the last one short
    ids, scores = ctx.retrieve_kv_pages(qd, kvb, top_kp=2, with_scores=True)
    ref_ids, alpha = O.retrieve_kv_pages(qn, Kn, kvb, 2)
    assert np.allclose(scores.cpu().numpy(), alpha, rtol=1e-5, atol=1e-6)
    got_ids = ids.cpu().tolist()
    if got_ids != ref_ids.tolist():                           # only pages that tie the weakest kept one may differ
        kth = alpha[ref_ids].min()
        assert all(abs(alpha[j] - kth) <= Hn.TIE_EPS for j in set(got_ids) ^ set(ref_ids.tolist()))
    assert ctx.retrieve_kv_pages(qd, kvb, top_kp=64).cpu().tolist() == list(range((nblk + kvb - 1) // kvb))

    # the retrieved pages restrict the selection (budgets larger than what they hold included)
    budgets = torch.tensor([3 if h % 2 == 0 else 10 ** 6 for h in range(w.H)], dtype=torch.int32)
    for inter_pages in (1, 2):
        si, sc = ctx.select_blocks_ex(qd, budgets.to(cuda_device), inter_block_pages=inter_pages, kv_pages=ids,
                                      kv_page_blocks=kvb)
        got = Hn.selection_lists(si, sc)
        ref, s = O.select_blocks_mixed(qn, Kn, N, False, budgets.tolist(), inter_pages, -1, None,
                                       kv_pages=got_ids, kv_page_blocks=kvb)
        for h in range(w.H):
            a, b = got[h][0].tolist(), ref[h][0].tolist()
            assert len(a) == len(b) and all(p // kvb in got_ids for p in a)
            if a != b:
                ca, cb = {p // inter_pages for p in a}, {p // inter_pages for p in b}
                kth = min(s[h, 0, c] for c in cb)
                assert all(abs(s[h, 0, c] - kth) <= Hn.TIE_EPS for c in ca ^ cb), h
    assert ctx.device_status() == 0

    # tier migration: evict the blocks outside the retrieved pages, poison their tiles, restore
    out0 = ctx.forward(qd, si, sc).clone()
    allsel = Hn.selection_to_device([[np.arange(nblk, dtype=np.int32)] for _ in range(w.H)], ctx.max_topk, cuda_device)
    full0 = ctx.forward(qd, allsel[0], allsel[1]).clone()
    evict_page = min(j for j in range((nblk + kvb - 1) // kvb) if j not in got_ids)   # a page that was not kept
    lo, hi = evict_page * kvb, min(nblk, evict_page * kvb + kvb)
    if hi > lo:
        hk, hv = ctx.evict_blocks(lo, hi - lo)
        torch.cuda.synchronize()
        assert not ctx.block_resident(lo) and not ctx.block_resident(hi - 1)
        assert ctx.block_resident(got_ids[0] * kvb)
        order = W.gen_page_order(w, w.n_blocks)
        pages = list(range(lo, hi)) if order is None else [int(order[b]) for b in range(lo, hi)]
        kp = ctx.k_pool.view(torch.bfloat16).view(-1, w.H, 64, w.d)
        vp = ctx.v_pool.view(torch.bfloat16).view(-1, w.H, 64, w.d)
        assert torch.equal(hk, kp[pages].cpu()) and torch.equal(hv, vp[pages].cpu())
        kp[pages] = float("nan")
        vp[pages] = float("nan")
        # a selection restricted to the retrieved pages does not touch the evicted tiles
        assert torch.equal(ctx.forward(qd, si, sc), out0)
        ctx.restore_blocks(lo, hk, hv)
        assert ctx.block_resident(lo)
        assert torch.equal(ctx.forward(qd, allsel[0], allsel[1]), full0)
    ctx.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("name,causal", [("mid_d128", False), ("mid_mix", False), ("mid_causal", True), ("mid_d64", False)])
def test_long_lists_split_over_ctas_and_merged(name, causal, cuda_device):
    """A (query tile, head) whose list is longer than split_blocks runs as several CTAs; the last
    one to finish merges their partial accumulators.  With a small split_blocks every tile of these
    workloads is split (lists of unequal lengths per head, odd block counts, a partial last block),
    and the result must match the oracle and the unsplit kernel."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS[name]
    q = W.gen_query(w)
    qn, qd = Hn.f32(q), q.to(cuda_device)
    outs = {}
    for sb in (0, 6):
        ctx = Hn.build_context(w, cuda_device, causal=causal, split_blocks=sb)
        K, V = Hn.append_history(ctx, w, cuda_device)
        nblk = ctx.n_blocks
        # head h keeps every block but the first h (so the heads differ in length and in parity)
        sel = [[np.arange(min(h, nblk - 1), nblk, dtype=np.int32)] for h in range(w.H)]
        si, sc = Hn.selection_to_device(sel, ctx.max_topk, cuda_device)
        for flags in (0, hsa.HSA_FWD_NO_LINEAR):
            for rep in range(3):                       # tickets must be back at zero after each launch
                out = ctx.forward(qd, si, sc, q_pos0=w.q_pos0, causal=causal, flags=flags)
                assert ctx.device_status() == 0
                if rep == 0:
                    outs[(sb, flags)] = out.clone()
                else:
                    assert torch.equal(out, outs[(sb, flags)])
        if sb:
            Kn, Vn = Hn.f32(K), Hn.f32(V)
            ref = O.hsa_forward(qn, Kn, Vn, w.q_pos0, causal, sel, linear_form="state")
            Hn.assert_close(Hn.f64(outs[(sb, hsa.HSA_FWD_NO_LINEAR)]), ref["O_sp"], "O_sp")
            Hn.assert_close(Hn.f64(outs[(sb, 0)]), ref["out"], "out")
        ctx.destroy()
    for flags in (0, hsa.HSA_FWD_NO_LINEAR):
        d = (outs[(6, flags)].float() - outs[(0, flags)].float()).abs().max()
        assert float(d) <= 2e-2


@pytest.mark.gpu
@pytest.mark.parametrize("name,grid_form", [("mid_d128", False), ("mid_mix", False), ("mid_d128", True), ("mid_mix", True)])
def test_steps_replayed_from_cuda_graphs_are_bit_identical(name, grid_form, cuda_device):
    """append + select + forward captured in CUDA graphs (the cooperative launch and the
    programmatic-dependent launches are ordinary graph nodes) give exactly what the same calls give
    issued one by one -- with a different query chunk in the captured buffer at every replay (so a
    stage of the selection kernel that ran ahead of its grid barrier would read the previous
    replay's sums), two graphs captured one after the other and replayed out of capture order, two
    selection calls per graph, and eager calls in between."""
    w = W.WORKLOADS[name]
    ctx = Hn.build_context(w, cuda_device, max_topk=max(w.n_blocks, 1), grid_barrier_select=grid_form)
    Hn.append_history(ctx, w, cuda_device, n_chunks=w.n_chunks - 1)
    k, v = (t.to(cuda_device) for t in W.gen_kv_chunk(w, w.n_chunks - 1))
    qs = [W.gen_query(w, step=i).to(cuda_device) for i in range(4)]
    budgets = W.gen_budgets(w).to(cuda_device)
    n0 = ctx.n_tokens
    state0, ksum0 = ctx.state.clone(), ctx.ksum.clone()

    def step(q, sel, out, scratch_sel):
        ctx.state.copy_(state0)
        ctx.ksum.copy_(ksum0)
        ctx.rewind(n0)
        ctx.append_kv(k, v)
        ctx.select_blocks(out, budgets, sel=scratch_sel)   # a selection on other data first: its sums
        ctx.select_blocks(q, budgets, sel=sel)              # and keys are what a missed barrier would reuse
        ctx.forward(q, sel[0], sel[1], out=out)

    def eager(q):
        sel, out = ctx.alloc_selection(w.Lq), torch.zeros_like(q)
        step(q, sel, out, ctx.alloc_selection(w.Lq))
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        return sel[0].clone(), sel[1].clone(), out.clone()

    refs = [eager(q) for q in qs]
    graphs = []
    for _ in range(2):
        qb = torch.zeros_like(qs[0])
        sel_g, out_g, scr = ctx.alloc_selection(w.Lq), torch.zeros_like(qb), ctx.alloc_selection(w.Lq)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step(qb, sel_g, out_g, scr)
        graphs.append((g, qb, sel_g, out_g))
    # a call issued directly after captures that have not been replayed yet
    e = eager(qs[1])
    assert torch.equal(e[2].view(torch.int16), refs[1][2].view(torch.int16)) and torch.equal(e[1], refs[1][1])

    def check(got_sel, got_out, ref):
        assert torch.equal(got_sel[1], ref[1])
        for h in range(w.H):
            n = int(ref[1][h, 0])
            assert torch.equal(got_sel[0][h, 0, :n], ref[0][h, 0, :n]), h
        assert torch.equal(got_out.view(torch.int16), ref[2].view(torch.int16))

    for gi, qi in [(1, 0), (0, 1), (0, 2), (1, 3), (1, 1), (0, 0), (1, 2)]:
        g, qb, sel_g, out_g = graphs[gi]
        qb.copy_(qs[qi])
        out_g.copy_(qs[(qi + 1) % 4])        # the first selection of the graph scores this tensor
        sel_g[1].fill_(-1)
        g.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        check(sel_g, out_g, refs[qi])
        if gi == 0 and qi == 2:              # an eager step between replays
            e = eager(qs[3])
            check((e[0], e[1]), e[2], refs[3])
    assert ctx.n_tokens == n0 + w.chunk
    ctx.destroy()


@pytest.mark.gpu
def test_grid_barrier_wait_that_runs_out_is_reported_and_leaves_the_context_usable(cuda_device):
    """The one place where CTAs wait for each other in global memory is the grid barrier of the
    selection kernel's grid-barrier form (the default form synchronises the CTAs of a head through
    hardware cluster barriers).  Its wait is bounded: with the bound set to a few milliseconds and the barrier's arrive count
    put where the last arrival can never be seen, the kernel must end by itself, report
    HSA_ERR_DEVICE_TIMEOUT, leave every list of the call empty (a forward call on it is the linear
    branch alone), and the next call must be clean."""
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_d128"]
    ctx = Hn.build_context(w, cuda_device, grid_barrier_select=True)
    Hn.append_history(ctx, w, cuda_device)
    q = W.gen_query(w).to(cuda_device)
    budgets = W.gen_budgets(w).to(cuda_device)
    ref_idx, ref_cnt = ctx.select_blocks(q, budgets)
    assert ctx.device_status() == 0 and int(ref_cnt.sum()) > 0
    words = ctx.barrier_words()
    assert int(words[0]) == 0                  # the arrive count is back at zero after every launch
    ctx.set_wait_limit_ns(5_000_000)
    words[0] = 0x40000000                      # no arrival will ever be the last one
    idx, cnt = ctx.alloc_selection(w.Lq)
    cnt.fill_(7)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    ctx.select_blocks(q, budgets, sel=(idx, cnt))
    t1.record()
    torch.cuda.synchronize()
    assert t0.elapsed_time(t1) < 1000.0        # milliseconds: the wait gave up at its bound
    assert int(cnt.abs().sum()) == 0
    out = ctx.forward(q, idx, cnt)
    lin = ctx.forward(q, idx, cnt, flags=hsa.HSA_FWD_NO_SPARSE)
    # (two different kernels: the same values up to the last bf16 bit)
    assert float((out.float() - lin.float()).abs().max()) <= 1e-3 and float(lin.float().abs().max()) > 1e-2
    assert ctx.device_status() == hsa.HSA_ERR_DEVICE_TIMEOUT
    assert ctx.barrier_words().tolist() == [0, 0] and ctx.device_status() == 0
    idx2, cnt2 = ctx.select_blocks(q, budgets)
    assert ctx.device_status() == 0
    assert torch.equal(cnt2, ref_cnt) and torch.equal(idx2, ref_idx)
    ctx.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("name,group_tokens,causal", [("mid_d128", 0, False), ("mid_d128", 128, False), ("mid_mix", 0, False),
                                                      ("mid_causal", 128, True), ("mid_d64", 0, False), ("cfg2", 0, False),
                                                      ("cfg2", 128, False)])
def test_cluster_and_grid_barrier_forms_of_the_selection_agree(name, group_tokens, causal, cuda_device):
    """The selection kernel has two forms (one thread-block cluster per head with hardware cluster
    barriers; one cooperative launch with two grid barriers).  Both run the same stages on the same
    data in the same order, so their lists must be identical bit for bit -- plain, per query tile,
    and with the two sparse granularities."""
    w = W.WORKLOADS[name]
    res = []
    for grid_form in (False, True):
        ctx = Hn.build_context(w, cuda_device, causal=causal, grid_barrier_select=grid_form,
                               max_topk=w.topk if name == "cfg2" else None)
        Hn.append_history(ctx, w, cuda_device, n_chunks=min(w.n_chunks, 4) if name == "cfg2" else None)
        q = W.gen_query(w).to(cuda_device)
        budgets = W.gen_budgets(w).to(cuda_device)
        q_pos0 = ctx.n_tokens - (w.Lq if causal else 0)
        a = ctx.select_blocks(q, budgets, q_pos0=q_pos0, causal=causal, group_tokens=group_tokens)
        p0 = max(0, ctx.n_tokens - w.chunk) // 64
        b = ctx.select_blocks_ex(q, budgets, inter_block_pages=2, intra_first_page=p0, q_pos0=q_pos0, causal=causal,
                                 group_tokens=group_tokens) if name != "cfg2" else a
        assert ctx.device_status() == 0
        res.append((Hn.selection_lists(*a), Hn.selection_lists(*b)))
        ctx.destroy()
    for x, y in zip(res[0], res[1]):
        for h in range(w.H):
            assert len(x[h]) == len(y[h])
            for g in range(len(x[h])):
                assert x[h][g].tolist() == y[h][g].tolist(), (h, g)
    assert sum(len(l) for hl in res[0][0] for l in hl) > 0


@pytest.mark.gpu
@pytest.mark.parametrize("n_rep,budget", [(40, 7), (300, 129), (600, 1), (600, 599), (6400, 1000)])
def test_selection_exact_ties_go_to_the_lower_block_index(n_rep, budget, cuda_device):
    """A history made of one 64-token block repeated n_rep times, followed by one distinct block:
    the repeated blocks have bit-identical pooled scores, so the budget cuts through a group of exact
    ties, which must go to the lower block indices (in every thread's range of the compaction, with
    one key per thread and with several; the longest case is beyond what a thread keeps in registers
    and takes the form that walks shared memory).  Checked against the oracle's selection as well."""
    from paper_2609_34606_b200 import hsa
    H, d = 2, 128
    gen = torch.Generator().manual_seed(1234 + n_rep)
    blk_k = torch.randn(64, H, d, generator=gen).to(torch.bfloat16)
    blk_v = torch.randn(64, H, d, generator=gen).to(torch.bfloat16)
    last_k = (torch.randn(64, H, d, generator=gen) * 3).to(torch.bfloat16)
    last_v = torch.randn(64, H, d, generator=gen).to(torch.bfloat16)
    K = torch.cat([blk_k.repeat(n_rep, 1, 1), last_k], 0)
    V = torch.cat([blk_v.repeat(n_rep, 1, 1), last_v], 0)
    n_blocks = n_rep + 1
    step = 64 * 50  # tokens per append
    ctx = hsa.HSAContext(H, d, max_pages=n_blocks, max_q_tokens=step, max_topk=n_blocks, device=cuda_device)
    for t0 in range(0, K.shape[0], step):
        ctx.append_kv(K[t0:t0 + step].to(cuda_device), V[t0:t0 + step].to(cuda_device))
    q = torch.randn(200, H, d, generator=gen).to(torch.bfloat16)
    budgets = torch.tensor([budget, budget + 1], dtype=torch.int32)
    si, sc = ctx.select_blocks(q.to(cuda_device), budgets.to(cuda_device))
    assert ctx.device_status() == 0
    got = Hn.selection_lists(si, sc)
    ref, scores = O.select_blocks(Hn.f64(q), Hn.f64(K), K.shape[0], False, budgets.numpy())
    for h in range(H):
        b = int(budgets[h])
        s = scores[h, 0]
        # (over thousands of blocks numpy's block means differ in the last bit from block to block:
        # there the oracle's own list is not held to the lowest indices, the GPU's is)
        exact = bool(np.all(s[:n_rep] == s[0]))
        assert exact or (n_rep > 1000 and np.ptp(s[:n_rep]) < 1e-12), "the repeated blocks must tie in the oracle too"
        # the distinct block either beats the ties or not; the rest of the budget is the lowest indices
        want = [n_rep] if s[n_rep] > s[0] else []
        want = sorted(list(range(b - len(want))) + want)
        assert got[h][0].tolist() == want
        if exact:
            assert ref[h][0].tolist() == want
    ctx.destroy()
