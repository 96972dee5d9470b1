"""The allocation-free selection entry point against the regular one and against the oracle.

Some callers of this library cannot allocate device memory at the point where they need a block
selection (a stream being captured into a CUDA graph, a process whose device memory belongs to
another framework's pool, a service that forbids allocation after start-up).  For them
hsa_select_blocks_noalloc keeps its scratch in a fixed array inside the library.  This test calls
it through the C ABI twice in a row -- the second call reuses the scratch the first one left
behind -- and requires the same selection as hsa_select_blocks and as the CPU oracle; a causal
call and a call whose lists do not fit max_topk (reported through a caller-supplied status word)
follow.  The file name sorts last so that a run which stops at the first failure has already run
every other test."""
import pytest
import torch

import hsa_harness as Hn
from oracle import hsa_oracle as O
from paper_2609_34606_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_noalloc_selection_matches_regular_entry_point_twice(cuda_device):
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_mix"]           # per-head budgets drawn from {0, 2, 4, 8, 16, all}
    ctx = Hn.build_context(w, cuda_device)
    K, _ = Hn.append_history(ctx, w, cuda_device)
    Kn = Hn.f32(K)
    budgets = W.gen_budgets(w).to(cuda_device)
    ksum = ctx.ksum                      # fp32 [H, max_pages, d] view of the context's state
    for call, step in enumerate((0, 1)):  # two different query chunks, back to back
        qc = W.gen_query(w, step=step)
        q = qc.to(cuda_device)
        ref_idx, ref_cnt = ctx.select_blocks(q, budgets)
        idx = torch.full_like(ref_idx, -1)
        cnt = torch.full_like(ref_cnt, -1)
        before = torch.cuda.memory_allocated(cuda_device)
        hsa.hsa_select_blocks_noalloc(q, ksum, ctx.n_tokens, ctx.n_tokens, False, 0.0, budgets, idx, cnt)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(cuda_device) == before
        assert torch.equal(cnt, ref_cnt), call
        for h in range(w.H):
            n = int(ref_cnt[h, 0])
            assert torch.equal(idx[h, 0, :n], ref_idx[h, 0, :n]), (call, h)
        sel_ref, scores = O.select_blocks(Hn.f32(qc), Kn, w.N, False, budgets.cpu().tolist())
        Hn.check_selection(Hn.selection_lists(idx, cnt), sel_ref, scores)
    # sizes beyond the fixed scratch are refused with a clear error, before any launch
    with pytest.raises(hsa.HSAError) as e:
        big = torch.empty(1, dtype=torch.float32, device=cuda_device)
        hsa._lib.hsa_select_blocks_noalloc.restype = int
        rc = hsa._lib.hsa_select_blocks_noalloc(q.data_ptr(), 128 * 65, q.stride(0), q.stride(1), 32, 128,
                                                big.data_ptr(), 1 << 20, 64, 64, 0, 0.0, budgets.data_ptr(),
                                                4, idx.data_ptr(), cnt.data_ptr(), None, None)
        hsa._check(rc, "hsa_select_blocks_noalloc")
    assert e.value.code == hsa.HSA_ERR_OUT_OF_PAGES
    assert ctx.device_status() == 0
    ctx.destroy()


def test_noalloc_selection_causal_and_clamped_lists(cuda_device):
    from paper_2609_34606_b200 import hsa
    w = W.WORKLOADS["mid_causal"]        # the queries are the last chunk of the history, causal
    ctx = Hn.build_context(w, cuda_device)
    K, _ = Hn.append_history(ctx, w, cuda_device)
    qc = W.gen_query(w)
    q = qc.to(cuda_device)
    budgets = W.gen_budgets(w).to(cuda_device)
    status = torch.zeros(1, dtype=torch.int32, device=cuda_device)
    idx, cnt = ctx.alloc_selection(w.Lq)
    hsa.hsa_select_blocks_noalloc(q, ctx.ksum, ctx.n_tokens, w.q_pos0, True, 0.0, budgets, idx, cnt, status)
    sel_ref, scores = O.select_blocks(Hn.f32(qc), Hn.f32(K), w.q_pos0, True, budgets.cpu().tolist())
    Hn.check_selection(Hn.selection_lists(idx, cnt), sel_ref, scores)
    assert int(status.item()) == 0
    # "every candidate" against a list capacity of 3: the lists are cut and the caller's status word says so
    every = torch.full((w.H,), -1, dtype=torch.int32, device=cuda_device)
    idx3 = torch.zeros(w.H, 1, 3, dtype=torch.int32, device=cuda_device)
    cnt3 = torch.zeros(w.H, 1, dtype=torch.int32, device=cuda_device)
    hsa.hsa_select_blocks_noalloc(q, ctx.ksum, ctx.n_tokens, w.q_pos0, True, 0.0, every, idx3, cnt3, status)
    torch.cuda.synchronize()
    assert cnt3.flatten().tolist() == [3] * w.H and idx3[:, 0].cpu().tolist() == [[0, 1, 2]] * w.H
    assert int(status.item()) == hsa.HSA_ERR_DEVICE_BOUNDS
    assert ctx.device_status() == 0
    ctx.destroy()
