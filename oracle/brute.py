"""Pure-Python brute force for tiny HSA cases (test infrastructure only).

Scalar loops and math.exp only: no numpy arithmetic, no matmul, no shared
helper with hsa_oracle.py.  It exists so that the numpy oracle can be checked
against something that does not share its vectorised code paths.
Inputs are nested lists / anything indexable as x[token][head][dim].
"""
from __future__ import annotations

import math

BLOCK = 64


def _dot(a, b):
    s = 0.0
    for x, y in zip(a, b):
        s += float(x) * float(y)
    return s


def _visible(j, N, p, causal):
    return j < N and (not causal or j <= p)


def attention_rows(q, K, V, N, H, d, Lq, q_pos0, causal, key_sets):
    """Softmax attention (Preliminaries, Eq. "attention") where query row i of head
    h may only look at the keys in key_sets[h][i] that are also visible."""
    scale = 1.0 / math.sqrt(d)
    out = [[[0.0] * d for _ in range(H)] for _ in range(Lq)]
    for i in range(Lq):
        p = q_pos0 + i
        for h in range(H):
            keys = [j for j in key_sets[h][i] if _visible(j, N, p, causal)]
            if not keys:
                continue
            s = [_dot(q[i][h], K[j][h]) * scale for j in keys]
            m = max(s)
            w = [math.exp(x - m) for x in s]
            tot = sum(w)
            for c in range(d):
                acc = 0.0
                for wj, j in zip(w, keys):
                    acc += wj * float(V[j][h][c])
                out[i][h][c] = acc / tot
    return out


def block_scores(q, K, N, H, d, Lq):
    """Whole-chunk group: mean query . mean key of the block / sqrt(d)
    (HKV Stage 2 score form)."""
    nb = (N + BLOCK - 1) // BLOCK
    scale = 1.0 / math.sqrt(d)
    s = [[0.0] * nb for _ in range(H)]
    for h in range(H):
        qbar = [sum(float(q[i][h][c]) for i in range(Lq)) / Lq for c in range(d)]
        for b in range(nb):
            toks = range(BLOCK * b, min(N, BLOCK * b + BLOCK))
            kbar = [sum(float(K[j][h][c]) for j in toks) / len(toks) for c in range(d)]
            s[h][b] = _dot(qbar, kbar) * scale
    return s


def topk_blocks(scores, cand, budget):
    """Largest `budget` candidate scores, lower index wins exact ties, ascending output."""
    idx = [b for b in range(len(scores)) if cand[b]]
    if budget < 0 or budget >= len(idx):
        return idx
    idx.sort(key=lambda b: (-scores[b], b))
    return sorted(idx[:budget])


def _phi(x, relu=False):
    x = float(x)
    if relu:
        return x if x > 0 else 0.0
    return x + 1.0 if x > 0 else math.exp(x)


def linear_rows(q, K, V, N, H, d, Lq, q_pos0, causal, relu=False):
    """sum_j phi(q).phi(k_j) v_j / sum_j phi(q).phi(k_j) over visible j (relu: the sum of weights
    plus 1e-6 in the denominator)."""
    out = [[[0.0] * d for _ in range(H)] for _ in range(Lq)]
    for h in range(H):
        fk = [[_phi(K[j][h][c], relu) for c in range(d)] for j in range(N)]
        for i in range(Lq):
            fq = [_phi(q[i][h][c], relu) for c in range(d)]
            p = q_pos0 + i
            num = [0.0] * d
            den = 0.0
            for j in range(N):
                if not _visible(j, N, p, causal):
                    continue
                w = _dot(fq, fk[j])
                den += w
                for c in range(d):
                    num[c] += w * float(V[j][h][c])
            if relu:
                out[i][h] = [x / (den + 1e-6) for x in num]
            elif den > 0:
                out[i][h] = [x / den for x in num]
    return out
