"""Seeded input generators: determinism, shapes and the structure the configs ask for."""
import numpy as np
import torch

from paper_2609_34606_b200 import workloads as W


def test_shapes_and_block_counts():
    for name, nb, tail in [("cfg1a", 32, 64), ("cfg2", 732, 16), ("cfg3", 4388, 32), ("cfg4", 2194, 48)]:
        w = W.WORKLOADS[name]
        assert w.n_blocks == nb and w.N - 64 * (nb - 1) == tail
    assert W.WORKLOADS["cfg1b"].q_pos0 == 2048 - 256 and W.WORKLOADS["cfg1a"].q_pos0 == 2048
    assert W.WORKLOADS["cfg5"].n_chunks * 4680 == 374400 and W.WORKLOADS["cfg5"].layers == 30


def test_deterministic_bf16():
    w = W.WORKLOADS["mid_d128"]
    k1, v1 = W.gen_kv_chunk(w, 3)
    k2, v2 = W.gen_kv_chunk(w, 3)
    assert k1.dtype == torch.bfloat16 and k1.shape == (w.chunk, w.H, w.d)
    assert torch.equal(k1, k2) and torch.equal(v1, v2)
    assert not torch.equal(k1, W.gen_kv_chunk(w, 4)[0])
    assert torch.equal(W.gen_query(w), W.gen_query(w))


def test_budget_set_and_page_order():
    w = W.WORKLOADS["cfg4"]
    b = W.gen_budgets(w)
    assert b.dtype == torch.int32 and b.shape == (12,)
    assert set(b.tolist()) <= set(w.budget_set)
    assert W.gen_budgets(W.WORKLOADS["cfg2"]).tolist() == [64] * 12
    p = W.gen_page_order(W.WORKLOADS["cfg3"], 4388)
    assert sorted(p.tolist()) == list(range(4388)) and p.tolist() != list(range(4388))
    assert W.gen_page_order(W.WORKLOADS["cfg2"], 732) is None


def test_mixture_structure():
    w = W.WORKLOADS["mid_mix"]
    mu = W.segment_means(w)
    s = W.query_segment(w)
    assert 0 <= s < mu.shape[0] - 1
    k, _ = W.gen_kv_chunk(w, 2 * s)          # first chunk of the queries' segment
    q = W.gen_query(w)
    assert np.allclose(k.float().mean(0).numpy(), mu[s].numpy(), atol=0.15)
    assert np.allclose(q.float().mean(0).numpy(), mu[s].numpy(), atol=0.15)


def test_sample_rows_cover_first_and_last_tile():
    w = W.WORKLOADS["cfg2"]
    r = W.sample_rows(w).tolist()
    assert set(range(128)) <= set(r) and set(range(4608, 4680)) <= set(r)
    assert len(r) <= 128 + 72 + 512 and r == sorted(r)
