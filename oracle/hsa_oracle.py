"""Plain CPU fp64 oracle for one Hybrid Sparse Attention (HSA) forward pass.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the
benchmark's CPU-baseline / reference arm.  It shares no code with the CUDA
path and never imports it.  Everything is numpy float64; library matmuls and
sorts are used as steps, with no blocking, fusion or reordering beyond what
the cited definitions state.

Conventions
-----------
q        [Lq, H, d]  queries of the current chunk (float64)
K, V     [N,  H, d]  the whole KV history as one flat token stream (no pages:
                     paging is a storage detail of the GPU pool and must not
                     change any result)
Query i sits at absolute position p_i = q_pos0 + i.  A key j is visible to
query i iff j < N and (not causal or j <= p_i)  -- the mask M in {-inf, 0} of
the attention definition (Preliminaries, Eq. "attention").
History blocks are runs of BLOCK = 64 consecutive tokens; the last one may be
partial (Block Sparse Attention preliminaries: a block is a contiguous run of
B tokens; HKV: pages of consecutive KV).

Which passage each function follows is stated in its docstring.  Readings of
points the paper leaves open (feature map, tie-break, group granularity, gate
shape) are the ones listed in the design notes; those parts are
"parity unpinned" by the paper itself and are pinned instead by mathematical
identities in the CPU tests (see tests/test_oracle_*.py):
  * phi (feature map of the running-state linear branch): parity unpinned
  * tie order of equal scores: parity unpinned
  * Linformer rank / segment length defaults: parity unpinned
"""
from __future__ import annotations

import numpy as np

BLOCK = 64


# --------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------
def _f64(x):
    """Inputs may arrive as float32 arrays holding exact bf16 values (to save
    memory on long histories); all arithmetic is done in float64."""
    return np.asarray(x, dtype=np.float64)


def n_blocks(N: int) -> int:
    return (N + BLOCK - 1) // BLOCK


def block_count(b: int, N: int) -> int:
    """Number of valid tokens of history block b."""
    return max(0, min(BLOCK, N - BLOCK * b))


def group_bounds(Lq: int, group_tokens: int):
    """Query groups that share one selection: [start, end) token ranges.
    group_tokens == 0 means the whole chunk is one group (the page-retrieval
    score of HKV Stage 2 uses the average query of the whole chunk)."""
    if group_tokens <= 0:
        return [(0, Lq)]
    return [(s, min(Lq, s + group_tokens)) for s in range(0, Lq, group_tokens)]


def n_visible(N: int, p: int, causal: bool) -> int:
    """Keys 0..n_visible-1 are visible to a query at absolute position p."""
    if not causal:
        return N
    return max(0, min(N, p + 1))


# --------------------------------------------------------------------------
# dense attention: Preliminaries, Eq. "attention"
#   S = Q K^T / sqrt(d_k),  A = Softmax(S + M),  O = A V
# --------------------------------------------------------------------------
def dense_attention(q, K, V, q_pos0: int, causal: bool, scale: float | None = None):
    Lq, H, d = q.shape
    N = K.shape[0]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.zeros((Lq, H, d))
    j = np.arange(N)[None, :]
    p = (q_pos0 + np.arange(Lq))[:, None]
    vis = np.ones((Lq, N), bool) if not causal else (j <= p)
    for h in range(H):
        S = (_f64(q[:, h, :]) @ _f64(K[:, h, :]).T) * scale
        S = np.where(vis, S, -np.inf)
        m = S.max(axis=1, keepdims=True) if N > 0 else np.zeros((Lq, 1))
        m = np.where(np.isfinite(m), m, 0.0)
        P = np.exp(S - m)
        l = P.sum(axis=1, keepdims=True)
        A = np.divide(P, l, out=np.zeros_like(P), where=l > 0)
        out[:, h, :] = A @ _f64(V[:, h, :])
    return out


# --------------------------------------------------------------------------
# block scoring + per-head top-k
#   pooled map: Sparse branch paragraph ("pooled attention map for coarse
#   block selection"); score form: HKV Stage 2, alpha = Qbar^T Kbar / sqrt(d_k)
#   with Qbar the average query and Kbar the average key of the block.
#   Budgeted per-head top-k replaces the cumulative-mass rule here.
# --------------------------------------------------------------------------
def block_key_means(K):
    """kbar[b, h, :] = arithmetic mean of the valid keys of block b."""
    N, H, d = K.shape
    nb = n_blocks(N)
    kbar = np.zeros((nb, H, d))
    for b in range(nb):
        kbar[b] = _f64(K[BLOCK * b:min(N, BLOCK * (b + 1))]).mean(axis=0)
    return kbar


def block_scores(q, K, group_tokens: int = 0, scale: float | None = None):
    """s[h, g, b] = mean_{i in group g} q_i  .  mean_{j in block b} k_j  * scale."""
    Lq, H, d = q.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    groups = group_bounds(Lq, group_tokens)
    kbar = block_key_means(K)                      # [nb, H, d]
    s = np.zeros((H, len(groups), kbar.shape[0]))
    for g, (a, e) in enumerate(groups):
        qbar = _f64(q[a:e]).mean(axis=0)           # [H, d]
        for h in range(H):
            s[h, g, :] = (kbar[:, h, :] @ qbar[h]) * scale
    return s


def candidate_mask(N: int, q_pos0: int, group_end: int, causal: bool):
    """Blocks a group may select: at least one valid token and, under the
    causal mask, a first token at or before the group's last query position."""
    nb = n_blocks(N)
    first = BLOCK * np.arange(nb)
    cand = first < N
    if causal:
        cand &= first <= (q_pos0 + group_end - 1)
    return cand


def select_topk(scores_row, cand, budget: int):
    """The min(budget, ncand) candidates with the largest score; an exact tie is
    won by the lower block index; reported in ascending block index.
    budget < 0 means every candidate."""
    idx = np.nonzero(cand)[0]
    if budget < 0 or budget >= idx.size:
        return idx.astype(np.int32)
    if budget == 0:
        return np.zeros(0, np.int32)
    # stable sort on (-score) keeps the lower index first among exact ties
    order = idx[np.argsort(-scores_row[idx], kind="stable")]
    return np.sort(order[:budget]).astype(np.int32)


def select_blocks(q, K, q_pos0: int, causal: bool, budgets, group_tokens: int = 0,
                  scale: float | None = None):
    """Returns (sel, scores): sel[h][g] = ascending int32 array of block ids."""
    Lq, H, _ = q.shape
    N = K.shape[0]
    s = block_scores(q, K, group_tokens, scale)
    groups = group_bounds(Lq, group_tokens)
    sel = []
    for h in range(H):
        row = []
        for g, (_, e) in enumerate(groups):
            cand = candidate_mask(N, q_pos0, e, causal)
            row.append(select_topk(s[h, g], cand, int(budgets[h])))
        sel.append(row)
    return sel, s


# --------------------------------------------------------------------------
# Two sparse granularities (Sec. 3.3, "Inter- and intra-chunk sparse
# granularity"): history before the current chunk is partitioned into coarse
# blocks of B_inter = inter_pages * 64 tokens, the current chunk's own tokens
# into blocks of B_intra = 64; both go through the same block-sparse
# attention, so a selection is reported as a list of 64-token pages.
# The paper fixes the two block sizes only; that each kind has its own budget
# and that a coarse block is scored by the mean key over all its tokens are
# this implementation's readings.
# --------------------------------------------------------------------------
# --------------------------------------------------------------------------
# HKV Stage 2, page-level retrieval (Sec. 3.2): a KV page is a run of
# kv_page_blocks consecutive 64-token blocks (8 frames x 1560 tokens = 195
# blocks in the paper's setting); its score is
#     alpha_j = Qbar^T Kbar_j / sqrt(d_k)
# with the average query of the current chunk and the average key of the
# page, and the top-K_p pages (K_p = 4 in the paper) are kept.  The paper
# writes Qbar, Kbar_j in R^{d_k} and is silent on heads: here the score is
# averaged over the heads, so that one set of pages serves the whole layer
# (a reading of this implementation).
# --------------------------------------------------------------------------
def kv_page_scores(q, K, kv_page_blocks: int, scale: float | None = None):
    """alpha[j] for every KV page j that holds at least one token."""
    Lq, H, d = q.shape
    N = K.shape[0]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    ptok = BLOCK * int(kv_page_blocks)
    npages = (N + ptok - 1) // ptok
    qbar = _f64(q).mean(axis=0)                                   # [H, d]
    alpha = np.zeros(npages)
    for j in range(npages):
        kbar = _f64(K[ptok * j:min(N, ptok * (j + 1))]).mean(axis=0)   # [H, d]
        alpha[j] = float(np.mean(np.sum(qbar * kbar, axis=1))) * scale
    return alpha


def retrieve_kv_pages(q, K, kv_page_blocks: int, top_kp: int, scale: float | None = None):
    """Ascending ids of the top_kp best-scoring KV pages (ties to the lower id)."""
    alpha = kv_page_scores(q, K, kv_page_blocks, scale)
    return select_topk(alpha, np.ones(alpha.size, bool), int(top_kp)), alpha


def mixed_candidates(N: int, inter_pages: int, intra_first_page: int):
    """Token ranges [(t0, t1), ...] of the candidates in history order: runs of
    inter_pages pages below intra_first_page (the last run may be short), then
    single pages.  intra_first_page < 0 or beyond the history: no intra part.
    Returns (ranges, n_inter)."""
    nb = n_blocks(N)
    p0 = intra_first_page if 0 <= intra_first_page < nb else nb
    ip = max(1, int(inter_pages))
    ranges = []
    for first in range(0, p0, ip):
        last = min(p0, first + ip)
        ranges.append((BLOCK * first, min(N, BLOCK * last)))
    n_inter = len(ranges)
    for pg in range(p0, nb):
        ranges.append((BLOCK * pg, min(N, BLOCK * (pg + 1))))
    return ranges, n_inter


def select_blocks_mixed(q, K, q_pos0: int, causal: bool, budgets, inter_pages: int = 2,
                        intra_first_page: int = -1, intra_budgets=None, group_tokens: int = 0,
                        scale: float | None = None, kv_pages=None, kv_page_blocks: int = 0):
    """Per (head, group): the budgets[h] best inter-chunk candidates and the
    intra_budgets[h] best intra-chunk candidates (None: all of them), by the
    pooled score mean_q . mean_k(candidate) * scale; ties to the earlier
    candidate.  kv_pages (with kv_page_blocks): ids of the retrieved KV pages;
    an inter-chunk candidate with a page outside them is no candidate at all
    (the retrieved pages are what is resident, Sec. 3.2 "Active KV
    construction").
    Returns (sel, scores): sel[h][g] = ascending int32 page ids,
    scores[h, g, c] per candidate."""
    Lq, H, d = q.shape
    N = K.shape[0]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    ranges, n_inter = mixed_candidates(N, inter_pages, intra_first_page)
    groups = group_bounds(Lq, group_tokens)
    kbar = np.zeros((len(ranges), H, d))
    for c, (t0, t1) in enumerate(ranges):
        kbar[c] = _f64(K[t0:t1]).mean(axis=0)
    first_tok = np.array([t0 for t0, _ in ranges], dtype=np.int64)
    scores = np.zeros((H, len(groups), len(ranges)))
    sel = []
    for h in range(H):
        row = []
        for g, (a, e) in enumerate(groups):
            qbar = _f64(q[a:e, h]).mean(axis=0)
            scores[h, g] = (kbar[:, h, :] @ qbar) * scale
            cand = np.ones(len(ranges), bool)
            if causal:
                cand &= first_tok <= (q_pos0 + e - 1)
            inter = cand.copy()
            inter[n_inter:] = False
            if kv_pages is not None:
                allowed = set(int(j) for j in kv_pages)
                for c in range(n_inter):
                    first_pg, last_pg = ranges[c][0] // BLOCK, (ranges[c][1] - 1) // BLOCK
                    if any(pg // int(kv_page_blocks) not in allowed for pg in (first_pg, last_pg)):
                        inter[c] = False
            intra = cand.copy()
            intra[:n_inter] = False
            chosen = list(select_topk(scores[h, g], inter, int(budgets[h])))
            chosen += list(select_topk(scores[h, g], intra, -1 if intra_budgets is None else int(intra_budgets[h])))
            pages = []
            for c in sorted(chosen):
                t0, t1 = ranges[c]
                pages += list(range(t0 // BLOCK, (t1 + BLOCK - 1) // BLOCK))
            row.append(np.array(pages, dtype=np.int32))
        sel.append(row)
    return sel, scores


# --------------------------------------------------------------------------
# sparse branch: O_sp = SDPA_block(Q, K, V; S^(h))  (Sparse branch, Eq. 4),
# i.e. Eq. "attention" with M = 0 exactly on the visible keys of the selected
# blocks and -inf elsewhere.
# --------------------------------------------------------------------------
def sparse_branch(q, K, V, sel, q_pos0: int, causal: bool, group_tokens: int = 0,
                  scale: float | None = None, rows=None):
    """rows: optional index array of query rows to evaluate (others stay 0);
    every row is independent given the selection."""
    Lq, H, d = q.shape
    N = K.shape[0]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.zeros((Lq, H, d))
    groups = group_bounds(Lq, group_tokens)
    for h in range(H):
        for g, (a, e) in enumerate(groups):
            blocks = np.asarray(sel[h][g], dtype=np.int64)
            if blocks.size == 0:
                continue
            r = np.arange(a, e)
            if rows is not None:
                r = np.intersect1d(r, rows)
            if r.size == 0:
                continue
            J = (blocks[:, None] * BLOCK + np.arange(BLOCK)[None, :]).reshape(-1)
            J = J[J < N]
            Kj = _f64(K[J, h, :])
            Vj = _f64(V[J, h, :])
            step = max(1, int(2.5e7 // max(1, J.size)))      # bound the score matrix
            for c0 in range(0, r.size, step):
                rr = r[c0:c0 + step]
                S = (_f64(q[rr, h, :]) @ Kj.T) * scale
                if causal:
                    vis = J[None, :] <= (q_pos0 + rr)[:, None]
                    S = np.where(vis, S, -np.inf)
                m = S.max(axis=1, keepdims=True)
                m = np.where(np.isfinite(m), m, 0.0)
                P = np.exp(S - m)
                l = P.sum(axis=1, keepdims=True)
                A = np.divide(P, l, out=np.zeros_like(P), where=l > 0)
                out[rr, h, :] = A @ Vj
    return out


# --------------------------------------------------------------------------
# linear branch, running-state form (kernelised linear attention):
#   O_lin[i] = sum_{j vis} (phi(q_i).phi(k_j)) v_j / sum_{j vis} phi(q_i).phi(k_j)
# This is the "fixed-size hidden state" linear attention the Linear Branch
# appendix contrasts with Linformer; it is the form the measured path uses.
# phi is not given by the paper: phi(x) = elu(x) + 1 ("elu1", the default), or
# phi(x) = max(x, 0) ("relu").  With relu a query can have weight zero on every
# visible key, so that form divides by (sum of weights + 1e-6): a row without
# any weight is 0 / 1e-6 = 0.   (parity unpinned)
# --------------------------------------------------------------------------
RELU_EPS = 1e-6


def phi(x, fmap: str = "elu1"):
    x = _f64(x)
    if fmap == "relu":
        return np.maximum(x, 0.0)
    if fmap != "elu1":
        raise ValueError("fmap must be 'elu1' or 'relu'")
    return np.where(x > 0, x + 1.0, np.exp(np.minimum(x, 0.0)))


def _normalise(num, den, fmap: str):
    """num / den per row; elu1: rows without a visible key (den = 0) are 0; relu: num / (den + eps)."""
    if fmap == "relu":
        return num / (den + RELU_EPS)
    return np.divide(num, den, out=np.zeros_like(num), where=den > 0)


def linear_parallel(q, K, V, q_pos0: int, causal: bool, rows=None, fmap: str = "elu1"):
    """The definition written out: explicit [rows x N] weight matrix,
    masked, row-normalised."""
    Lq, H, d = q.shape
    N = K.shape[0]
    out = np.zeros((Lq, H, d))
    r_all = np.arange(Lq) if rows is None else np.asarray(rows)
    step = max(1, int(2.5e7 // max(1, N)))
    for h in range(H):
        fk = phi(K[:, h, :], fmap)
        for c0 in range(0, r_all.size, step):
            rr = r_all[c0:c0 + step]
            W = phi(q[rr, h, :], fmap) @ fk.T                 # [rows, N], all >= 0
            if causal:
                vis = np.arange(N)[None, :] <= (q_pos0 + rr)[:, None]
                W = np.where(vis, W, 0.0)
            den = W.sum(axis=1, keepdims=True)
            num = W @ _f64(V[:, h, :])
            out[rr, h, :] = _normalise(num, den, fmap)
    return out


def linear_state(K, V, upto: int | None = None, fmap: str = "elu1"):
    """S[h] = sum_j phi(k_j)^T v_j  (d x d),  z[h] = sum_j phi(k_j), over tokens j < upto."""
    N, H, d = K.shape
    n = N if upto is None else max(0, min(N, upto))
    S = np.zeros((H, d, d))
    z = np.zeros((H, d))
    for h in range(H):
        fk = phi(K[:n, h, :], fmap)
        S[h] = fk.T @ _f64(V[:n, h, :])
        z[h] = fk.sum(axis=0)
    return S, z


def linear_recurrent(q, K, V, q_pos0: int, causal: bool, fmap: str = "elu1"):
    """Token-by-token recurrence S_t = S_{t-1} + phi(k_t)^T v_t, z_t likewise.
    Query i reads the state after token min(p_i, N-1) if causal, else after the
    last token."""
    Lq, H, d = q.shape
    N = K.shape[0]
    out = np.zeros((Lq, H, d))
    # number of tokens each query must have absorbed before it reads the state
    need = np.array([n_visible(N, q_pos0 + i, causal) for i in range(Lq)])
    for h in range(H):
        S = np.zeros((d, d))
        z = np.zeros(d)
        fq = phi(q[:, h, :], fmap)
        order = np.argsort(need, kind="stable")
        t = 0
        for i in order:
            while t < need[i]:
                fk = phi(K[t, h, :], fmap)
                S += np.outer(fk, _f64(V[t, h, :]))
                z += fk
                t += 1
            den = fq[i] @ z
            if need[i] > 0:
                out[i, h, :] = (fq[i] @ S) / (den + RELU_EPS if fmap == "relu" else den)
    return out


def linear_chunked(q, K, V, q_pos0: int, causal: bool, boundary: int, fmap: str = "elu1"):
    """State of the tokens before `boundary` plus the explicitly masked part over
    tokens >= boundary: the split the GPU uses (state at a chunk boundary +
    intra-chunk part)."""
    Lq, H, d = q.shape
    N = K.shape[0]
    S0, z0 = linear_state(K, V, upto=boundary, fmap=fmap)
    out = np.zeros((Lq, H, d))
    p = q_pos0 + np.arange(Lq)
    jj = np.arange(boundary, N)
    for h in range(H):
        fq = phi(q[:, h, :], fmap)
        num = np.zeros((Lq, d))
        den = np.zeros(Lq)
        # the boundary state holds tokens < boundary; a causal query before the
        # boundary cannot use it as a whole, so this form requires p_i >= boundary-1
        if causal and np.any(p < boundary - 1):
            raise ValueError("chunked form needs every query at or after the boundary")
        num += fq @ S0[h]
        den += fq @ z0[h]
        if jj.size:
            W = fq @ phi(K[boundary:, h, :], fmap).T
            if causal:
                W = np.where(jj[None, :] <= p[:, None], W, 0.0)
            num += W @ _f64(V[boundary:, h, :])
            den += W.sum(axis=1)
        out[:, h, :] = _normalise(num, den[:, None], fmap)
    return out


def linear_from_state(q, S, z, fmap: str = "elu1"):
    """phi(q) S / (phi(q) z): applying a given state to the chunk's queries."""
    Lq, H, d = q.shape
    out = np.zeros((Lq, H, d))
    for h in range(H):
        fq = phi(q[:, h, :], fmap)
        den = (fq @ z[h])[:, None]
        num = fq @ S[h]
        out[:, h, :] = _normalise(num, den, fmap)
    return out


# --------------------------------------------------------------------------
# linear branch, Linformer form (Linear branch paragraph, Eq. 3 and the
# Linear Branch appendix): per fixed-length segment K~ = E_K^T K, V~ = E_V^T V
# (r x d), concatenated over complete segments; softmax attention over the
# compressed rows.
# --------------------------------------------------------------------------
def linformer_compress(K, V, E_K, E_V, L_seg: int):
    """E_K, E_V: [H, L_seg, r].  Returns K~, V~ of shape [n_seg * r, H, d]."""
    N, H, d = K.shape
    r = E_K.shape[2]
    n_seg = N // L_seg
    Kt = np.zeros((n_seg * r, H, d))
    Vt = np.zeros((n_seg * r, H, d))
    for s in range(n_seg):
        for h in range(H):
            Kt[s * r:(s + 1) * r, h, :] = _f64(E_K[h]).T @ _f64(K[s * L_seg:(s + 1) * L_seg, h, :])
            Vt[s * r:(s + 1) * r, h, :] = _f64(E_V[h]).T @ _f64(V[s * L_seg:(s + 1) * L_seg, h, :])
    return Kt, Vt


def linformer_branch(q, Kt, Vt, scale: float | None = None):
    """Softmax(Q K~^T / sqrt(d)) V~ : dense attention over the compressed rows."""
    return dense_attention(q, Kt, Vt, q_pos0=0, causal=False, scale=scale)


# --------------------------------------------------------------------------
# gated fusion (Gated fusion paragraph, Eq. 5):
#   O = O_lin * G_lin + O_sp * G_sp,  gates optionally through a sigmoid.
# --------------------------------------------------------------------------
def gate_weight(g, gate_act: int, shape):
    if g is None:
        return np.ones(shape)
    g = np.asarray(g, dtype=np.float64)
    if g.ndim == 2:
        g = g[:, :, None]
    w = 1.0 / (1.0 + np.exp(-g)) if gate_act == 1 else g
    return np.broadcast_to(w, shape)


def merge(O_lin, O_sp, g_lin=None, g_sp=None, gate_act: int = 0):
    return gate_weight(g_lin, gate_act, O_lin.shape) * O_lin + \
        gate_weight(g_sp, gate_act, O_sp.shape) * O_sp


# --------------------------------------------------------------------------
# whole forward
# --------------------------------------------------------------------------
def hsa_forward(q, K, V, q_pos0: int, causal: bool, sel, group_tokens: int = 0,
                g_lin=None, g_sp=None, gate_act: int = 0, scale: float | None = None,
                no_linear: bool = False, no_sparse: bool = False, rows=None,
                linear_form: str = "parallel", fmap: str = "elu1"):
    """out = gate(g_lin) * O_lin + gate(g_sp) * O_sp with a disabled branch
    contributing exactly 0.  linear_form: "parallel" (definition) or "state"
    (phi(q) S / phi(q) z, non-causal only; equal up to rounding order and used
    where the explicit weight matrix would not fit)."""
    Lq, H, d = q.shape
    O_sp = np.zeros((Lq, H, d))
    O_lin = np.zeros((Lq, H, d))
    if not no_sparse:
        O_sp = sparse_branch(q, K, V, sel, q_pos0, causal, group_tokens, scale, rows)
    if not no_linear:
        if linear_form == "state" and not causal:
            S, z = linear_state(K, V, fmap=fmap)
            O_lin = linear_from_state(q, S, z, fmap)
        else:
            O_lin = linear_parallel(q, K, V, q_pos0, causal, rows, fmap)
        if rows is not None:
            keep = np.zeros(Lq, bool)
            keep[np.asarray(rows)] = True
            O_lin[~keep] = 0.0
    out = merge(O_lin, O_sp, g_lin, g_sp, gate_act)
    return {"out": out, "O_sp": O_sp, "O_lin": O_lin}


# --------------------------------------------------------------------------
# head-adaptive block budgets (Appendix "Sparse Branch"): for head h and query
# group i, p_{i,:} are the block attention weights (softmax of the pooled
# scores over the candidate blocks), sigma sorts them in descending order,
#   K_i = min{k : sum_{m<=k} p_{sigma(m)} >= tau_h},     S(i) = first K_i blocks,
#   G^(h) = mean_i [ (1/N) sum_{m=1..N} (N - 2m + 1) p_{sigma(m)} ]   (Gini, Eq. 12),
#   tau_h = tau_min + G^(h) (tau_max - tau_min)                        (Eq. 13).
# Exact ties in the sort go to the lower block index.
# --------------------------------------------------------------------------
def block_weights(scores_row, cand):
    """Softmax of the candidate blocks' pooled scores (zeros elsewhere)."""
    p = np.zeros_like(scores_row)
    idx = np.nonzero(cand)[0]
    if idx.size:
        e = np.exp(scores_row[idx] - scores_row[idx].max())
        p[idx] = e / e.sum()
    return p


def gini_of_weights(p_sorted_desc):
    N = p_sorted_desc.size
    if N == 0:
        return 0.0
    m = np.arange(1, N + 1)
    return float(((N - 2 * m + 1) * p_sorted_desc).sum() / N)


def adaptive_selection(q, K, q_pos0: int, causal: bool, tau_min: float, tau_max: float,
                       group_tokens: int = 0, scale: float | None = None):
    """Returns (sel, gini, tau): sel[h][g] ascending block ids chosen by the cumulative-mass
    rule, gini[h], tau[h]."""
    Lq, H, _ = q.shape
    N = K.shape[0]
    s = block_scores(q, K, group_tokens, scale)
    groups = group_bounds(Lq, group_tokens)
    sel, gini, tau = [], np.zeros(H), np.zeros(H)
    for h in range(H):
        orders, weights, gs = [], [], []
        for g, (_, e) in enumerate(groups):
            cand = candidate_mask(N, q_pos0, e, causal)
            p = block_weights(s[h, g], cand)
            idx = np.nonzero(cand)[0]
            order = idx[np.argsort(-s[h, g][idx], kind="stable")]     # descending, ties -> lower index
            orders.append(order)
            weights.append(p[order])
            gs.append(gini_of_weights(p[order]))
        gini[h] = float(np.mean(gs)) if gs else 0.0
        tau[h] = tau_min + gini[h] * (tau_max - tau_min)
        row = []
        for order, pw in zip(orders, weights):
            if order.size == 0:
                row.append(np.zeros(0, np.int32))
                continue
            cum = np.cumsum(pw)
            hit = np.nonzero(cum >= tau[h])[0]
            k = int(hit[0]) + 1 if hit.size else order.size
            row.append(np.sort(order[:k]).astype(np.int32))
        sel.append(row)
    return sel, gini, tau
