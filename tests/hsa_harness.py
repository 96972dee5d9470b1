"""Shared helpers for the GPU parity tests: run a workload through the C-ABI
path and through the CPU oracle on the identical bf16 inputs, and compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import hsa_oracle as O
from paper_2609_34606_b200 import workloads as W

# tolerances of the benchmark spec for bf16 inputs with fp32 accumulation
MAX_ABS = 2e-2
MEAN_ABS = 2e-3
REL_FRO = 1e-2      # additional relative check (outputs are small for N(0,1) inputs)
TIE_EPS = 1e-6


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def build_context(w: W.Workload, device, max_topk=None, causal=None, extra_pages=0, lin_mode=1,
                  gate_act=0, split_blocks=0, grid_barrier_select=False, feature_map=0):
    from paper_2609_34606_b200 import hsa
    max_pages = w.n_blocks + extra_pages
    order = W.gen_page_order(w, max_pages)
    ctx = hsa.HSAContext(w.H, w.d, max_pages=max_pages, max_q_tokens=max(w.Lq, w.chunk),
                         max_topk=max_topk or max(w.n_blocks, 1), lin_mode=lin_mode,
                         gate_act=gate_act, causal=w.causal if causal is None else causal,
                         page_order=order, device=device, split_blocks=split_blocks,
                         grid_barrier_select=grid_barrier_select, feature_map=feature_map)
    # poison the pools (0xFFFF is a bf16 NaN): anything read but never written shows up
    ctx.k_pool.fill_(0xFF)
    ctx.v_pool.fill_(0xFF)
    return ctx


def append_history(ctx, w: W.Workload, device, n_chunks=None):
    """Appends the history chunk by chunk; returns the CPU copies (bf16) for the oracle."""
    ks, vs = [], []
    for c in range(w.n_chunks if n_chunks is None else n_chunks):
        k, v = W.gen_kv_chunk(w, c)
        ctx.append_kv(k.to(device), v.to(device))
        ks.append(k)
        vs.append(v)
    return torch.cat(ks, 0), torch.cat(vs, 0)


def selection_lists(sel_idx: torch.Tensor, sel_cnt: torch.Tensor):
    idx, cnt = sel_idx.cpu().numpy(), sel_cnt.cpu().numpy()
    H, G = cnt.shape
    return [[idx[h, g, :cnt[h, g]].copy() for g in range(G)] for h in range(H)]


def selection_to_device(sel, max_topk, device):
    H, G = len(sel), len(sel[0])
    idx = torch.zeros(H, G, max_topk, dtype=torch.int32)
    cnt = torch.zeros(H, G, dtype=torch.int32)
    for h in range(H):
        for g in range(G):
            n = len(sel[h][g])
            idx[h, g, :n] = torch.from_numpy(np.asarray(sel[h][g], dtype=np.int32))
            cnt[h, g] = n
    return idx.to(device), cnt.to(device)


def check_selection(sel_gpu, sel_ref, scores):
    """Bit-exact sets except for blocks whose score ties the k-th score within TIE_EPS."""
    for h in range(len(sel_ref)):
        for g in range(len(sel_ref[h])):
            a, b = np.asarray(sel_gpu[h][g]), np.asarray(sel_ref[h][g])
            assert len(a) == len(b), (h, g, len(a), len(b))
            assert list(a) == sorted(set(a.tolist())), "ascending, no duplicates"
            diff = np.setxor1d(a, b)
            if diff.size:
                kth = scores[h, g, b].min()
                assert np.all(np.abs(scores[h, g, diff] - kth) <= TIE_EPS), (h, g, diff)


def err_stats(got: np.ndarray, ref: np.ndarray):
    d = np.abs(got - ref)
    fro = np.linalg.norm(ref)
    return {"max_abs": float(d.max()) if d.size else 0.0,
            "mean_abs": float(d.mean()) if d.size else 0.0,
            "rel_fro": float(np.linalg.norm(got - ref) / fro) if fro > 0 else float(np.linalg.norm(got - ref))}


def assert_close(got, ref, what="out", rel=True):
    s = err_stats(got, ref)
    assert s["max_abs"] <= MAX_ABS, (what, s)
    assert s["mean_abs"] <= MEAN_ABS, (what, s)
    if rel:
        assert s["rel_fro"] <= REL_FRO, (what, s)
    return s


def oracle_inputs(w: W.Workload, K: torch.Tensor, V: torch.Tensor, q: torch.Tensor):
    return f32(q), f32(K), f32(V)


def run_case(w: W.Workload, device, group_tokens=0, gates=None, gate_act=0, check_state=True, fmap="elu1"):
    """Full path on the GPU and in the oracle; returns a dict of error statistics."""
    from paper_2609_34606_b200 import hsa
    ctx = build_context(w, device, gate_act=gate_act, feature_map=1 if fmap == "relu" else 0)
    K, V = append_history(ctx, w, device)
    q = W.gen_query(w)
    qd = q.to(device)
    budgets = W.gen_budgets(w)
    qn, Kn, Vn = oracle_inputs(w, K, V, q)
    res = {}
    if check_state:
        S_ref, z_ref = O.linear_state(Kn, Vn, fmap=fmap)
        kbar = O.block_key_means(Kn)
        cnts = np.array([O.block_count(b, w.N) for b in range(w.n_blocks)])
        ksum_ref = (kbar * cnts[:, None, None]).transpose(1, 0, 2)
        S, z, ksum = f64(ctx.S), f64(ctx.z), f64(ctx.ksum[:, :w.n_blocks])
        res["S_rel"] = np.linalg.norm(S - S_ref) / np.linalg.norm(S_ref)
        res["z_rel"] = np.linalg.norm(z - z_ref) / np.linalg.norm(z_ref)
        res["ksum_rel"] = np.linalg.norm(ksum - ksum_ref) / max(np.linalg.norm(ksum_ref), 1e-30)
        assert res["S_rel"] <= 1e-5 and res["z_rel"] <= 1e-5 and res["ksum_rel"] <= 1e-5, res
    sel_idx, sel_cnt = ctx.select_blocks(qd, budgets.to(device), q_pos0=w.q_pos0, causal=w.causal,
                                         group_tokens=group_tokens)
    sel_gpu = selection_lists(sel_idx, sel_cnt)
    sel_ref, scores = O.select_blocks(qn, Kn, w.q_pos0, w.causal, budgets.tolist(), group_tokens)
    check_selection(sel_gpu, sel_ref, scores)
    g_lin = g_sp = None
    gl_n = gs_n = None
    if gates is not None:
        g_lin, g_sp = W.gen_gates(w, per_dim=(gates == "dim"))
        gl_n, gs_n = f64(g_lin), f64(g_sp)
        g_lin, g_sp = g_lin.to(device), g_sp.to(device)
    # the oracle evaluates the GPU's own selection (identical up to forgiven ties)
    ref = O.hsa_forward(qn, Kn, Vn, w.q_pos0, w.causal, sel_gpu, group_tokens, gl_n, gs_n, gate_act, fmap=fmap)
    out = ctx.forward(qd, sel_idx, sel_cnt, q_pos0=w.q_pos0, causal=w.causal, group_tokens=group_tokens,
                      g_lin=g_lin, g_sp=g_sp)
    o_sp = ctx.forward(qd, sel_idx, sel_cnt, q_pos0=w.q_pos0, causal=w.causal,
                       group_tokens=group_tokens, flags=hsa.HSA_FWD_NO_LINEAR)
    o_lin = ctx.forward(qd, sel_idx, sel_cnt, q_pos0=w.q_pos0, causal=w.causal,
                        group_tokens=group_tokens, flags=hsa.HSA_FWD_NO_SPARSE)
    assert ctx.device_status() == 0
    res["O_sp"] = assert_close(f64(o_sp), ref["O_sp"], "O_sp")
    res["O_lin"] = assert_close(f64(o_lin), ref["O_lin"], "O_lin")
    res["out"] = assert_close(f64(out), ref["out"], "out")
    ctx.destroy()
    return res
