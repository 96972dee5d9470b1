"""Seeded synthetic inputs for the HSA forward path.

This module holds input generation only -- none of the method's arithmetic --
so that the CUDA path's callers and the CPU oracle's callers can both draw the
identical bf16 bit patterns from it.  Everything is generated on the CPU with a
seeded torch.Generator, in fp32, and rounded to bf16.

Shapes follow the workload the paper measures on (Implementation Details and
HKV Stage 2): 1560 tokens per latent frame, 3-latent-frame chunks of 4680
tokens, a 1.3B-class video DiT layer with 12 heads of 128, histories of tens
of chunks.  Values are synthetic (N(0,1) or a Gaussian mixture with one mean
per scene segment); no dataset, prompt or weight of the paper's evaluation is
used or needed.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import torch

BLOCK = 64
ALL = -1  # budget value meaning "every candidate block"


@dataclass(frozen=True)
class Workload:
    name: str
    H: int
    d: int
    Lq: int                      # query chunk tokens
    chunk: int                   # tokens appended per history chunk
    n_chunks: int                # history chunks appended before the forward
    topk: int                    # uniform per-head budget (ignored if budget_set)
    seed: int
    causal: bool = False
    q_inside: bool = False       # True: the queries are the last Lq history tokens' positions
    shuffle_pages: bool = False
    mixture: bool = False        # keys from a per-segment Gaussian mixture
    seg_chunks: int = 5          # chunks per scene segment (mixture only)
    sigma: float = 0.3
    budget_set: Optional[tuple] = None   # draw per-head budgets uniformly from this set
    q_scale: float = 1.0
    layers: int = 1

    @property
    def N(self) -> int:
        return self.chunk * self.n_chunks

    @property
    def n_blocks(self) -> int:
        return (self.N + BLOCK - 1) // BLOCK

    @property
    def q_pos0(self) -> int:
        return self.N - self.Lq if self.q_inside else self.N


WORKLOADS = {
    # tiny case the oracle finishes in well under a second
    "cfg1a": Workload("cfg1a", H=2, d=64, Lq=256, chunk=256, n_chunks=8, topk=4, seed=0),
    "cfg1b": Workload("cfg1b", H=2, d=64, Lq=256, chunk=256, n_chunks=8, topk=4, seed=0,
                      causal=True, q_inside=True),
    "cfg1_sharp": Workload("cfg1_sharp", H=2, d=64, Lq=256, chunk=256, n_chunks=8, topk=4,
                           seed=0, q_scale=4.0),
    # one attention layer of a 1.3B-class video DiT, 10 history chunks
    "cfg2": Workload("cfg2", H=12, d=128, Lq=4680, chunk=4680, n_chunks=10, topk=64, seed=1),
    # long history, shuffled page table
    "cfg3": Workload("cfg3", H=12, d=128, Lq=4680, chunk=4680, n_chunks=60, topk=128, seed=2,
                     shuffle_pages=True),
    # head-adaptive budgets + scene-segment mixture
    "cfg4": Workload("cfg4", H=12, d=128, Lq=4680, chunk=4680, n_chunks=30, topk=64, seed=3,
                     mixture=True, budget_set=(0, 16, 32, 64, 128, ALL)),
    # full-stack rollout: 30 layers, 80 chunks
    "cfg5": Workload("cfg5", H=12, d=128, Lq=4680, chunk=4680, n_chunks=80, topk=64, seed=4,
                     layers=30),
    # reduced shapes used by the parity tests (several tiles + ragged tails)
    "mid_d128": Workload("mid_d128", H=3, d=128, Lq=333, chunk=333, n_chunks=7, topk=9, seed=11),
    "mid_d64": Workload("mid_d64", H=3, d=64, Lq=200, chunk=200, n_chunks=6, topk=5, seed=12),
    "mid_mix": Workload("mid_mix", H=6, d=128, Lq=300, chunk=300, n_chunks=12, topk=8, seed=13,
                        mixture=True, seg_chunks=2, budget_set=(0, 2, 4, 8, 16, ALL)),
    "mid_causal": Workload("mid_causal", H=2, d=128, Lq=300, chunk=300, n_chunks=5, topk=6,
                           seed=14, causal=True, q_inside=True),
    "mid_linformer": Workload("mid_linformer", H=3, d=128, Lq=300, chunk=328, n_chunks=4, topk=6, seed=16),
    # the layer's own sizes with three history chunks: Linformer segments of one chunk each
    "cfg2_linformer": Workload("cfg2_linformer", H=12, d=128, Lq=4680, chunk=4680, n_chunks=3, topk=64, seed=17),
    "mid_shuffle": Workload("mid_shuffle", H=2, d=128, Lq=260, chunk=260, n_chunks=9, topk=12,
                            seed=15, shuffle_pages=True),
}


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def _tensor_seed(w: Workload, kind: int, index: int, layer: int = 0) -> int:
    # distinct stream per (workload seed, tensor kind, chunk index, layer)
    return (w.seed * 1_000_003 + kind * 100_003 + index * 101 + layer * 7_919) % (2 ** 63 - 1)


def segment_means(w: Workload) -> torch.Tensor:
    """[n_segments, H, d] fp32 mixture means (mixture workloads only)."""
    n_seg = (w.n_chunks + w.seg_chunks - 1) // w.seg_chunks
    return torch.randn(n_seg, w.H, w.d, generator=_gen(_tensor_seed(w, 7, 0)))


def query_segment(w: Workload) -> int:
    """Scene segment the queries are drawn from: one strictly earlier than the last."""
    n_seg = (w.n_chunks + w.seg_chunks - 1) // w.seg_chunks
    if n_seg <= 1:
        return 0
    return int(torch.randint(0, n_seg - 1, (1,), generator=_gen(_tensor_seed(w, 8, 0))).item())


def gen_kv_chunk(w: Workload, c: int, layer: int = 0):
    """(k, v) of history chunk c: bf16 [chunk, H, d]."""
    k = torch.randn(w.chunk, w.H, w.d, generator=_gen(_tensor_seed(w, 1, c, layer)))
    v = torch.randn(w.chunk, w.H, w.d, generator=_gen(_tensor_seed(w, 2, c, layer)))
    if w.mixture:
        means = segment_means(w)
        mu = means[min(c // w.seg_chunks, means.shape[0] - 1)]  # chunks past the history: last segment
        k = mu[None] + w.sigma * k
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def gen_query(w: Workload, step: int = 0, layer: int = 0) -> torch.Tensor:
    """Queries of the current chunk: bf16 [Lq, H, d]."""
    q = torch.randn(w.Lq, w.H, w.d, generator=_gen(_tensor_seed(w, 3, step, layer)))
    if w.mixture:
        mu = segment_means(w)[query_segment(w)]
        q = mu[None] + w.sigma * q
    return (q * w.q_scale).to(torch.bfloat16)


def gen_budgets(w: Workload) -> torch.Tensor:
    """int32 [H] per-head block budgets (ALL = every candidate)."""
    if w.budget_set is None:
        return torch.full((w.H,), w.topk, dtype=torch.int32)
    choices = torch.tensor(w.budget_set, dtype=torch.int32)
    pick = torch.randint(0, len(w.budget_set), (w.H,), generator=_gen(_tensor_seed(w, 4, 0)))
    return choices[pick].to(torch.int32)


def gen_page_order(w: Workload, max_pages: int) -> Optional[torch.Tensor]:
    """int32 [max_pages]: physical page given to the b-th allocated block
    (a seeded random permutation), or None for the identity order."""
    if not w.shuffle_pages:
        return None
    return torch.randperm(max_pages, generator=_gen(_tensor_seed(w, 5, 0))).to(torch.int32)


def gen_gates(w: Workload, per_dim: bool = False):
    """Synthetic gate logits (g_lin, g_sp): bf16 [Lq, H] or [Lq, H, d]."""
    shape = (w.Lq, w.H, w.d) if per_dim else (w.Lq, w.H)
    g1 = torch.randn(*shape, generator=_gen(_tensor_seed(w, 6, 0)))
    g2 = torch.randn(*shape, generator=_gen(_tensor_seed(w, 6, 1)))
    return g1.to(torch.bfloat16), g2.to(torch.bfloat16)


def gen_history(w: Workload, layer: int = 0):
    """Whole history as two bf16 tensors [N, H, d] (concatenated chunks)."""
    ks, vs = zip(*(gen_kv_chunk(w, c, layer) for c in range(w.n_chunks)))
    return torch.cat(ks, 0), torch.cat(vs, 0)


def sample_rows(w: Workload, n_random: int = 512, tile: int = 128) -> torch.Tensor:
    """Row subset for sampled parity at full size: every row of the first and
    the last query tile plus n_random seeded random rows."""
    first = torch.arange(0, min(tile, w.Lq))
    last_start = ((w.Lq - 1) // tile) * tile
    last = torch.arange(last_start, w.Lq)
    rnd = torch.randperm(w.Lq, generator=_gen(_tensor_seed(w, 9, 0)))[:n_random]
    return torch.unique(torch.cat([first, last, rnd])).to(torch.int64)


def random_rows(w: Workload, n: int) -> torch.Tensor:
    """n distinct seeded query rows (all rows if n >= Lq)."""
    return torch.randperm(w.Lq, generator=_gen(_tensor_seed(w, 10, 0)))[:min(n, w.Lq)].to(torch.int64)


def gen_linformer_weights(w: Workload, rank: int, seg_tokens: int):
    """Synthetic Linformer projections (E_K, E_V): bf16 [H, seg_tokens, rank] ~ N(0, 1/seg_tokens)."""
    shape = (w.H, seg_tokens, rank)
    ek = torch.randn(*shape, generator=_gen(_tensor_seed(w, 11, 0))) / seg_tokens ** 0.5
    ev = torch.randn(*shape, generator=_gen(_tensor_seed(w, 11, 1))) / seg_tokens ** 0.5
    return ek.to(torch.bfloat16), ev.to(torch.bfloat16)
