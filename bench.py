#!/usr/bin/env python
"""HSA forward-path benchmark: one JSON line per run.

A "step" is one pass of the whole hot path for one query chunk of the
1.3B-class video-DiT layer workload (H=12, d=128, chunk 4680 tokens, history
10 chunks = 46,800 tokens, top-64 blocks per head): undo the previous step's append
(hsa_rewind to the 9-chunk history, host bookkeeping only), then
hsa_append_kv (chunk 10) -> hsa_select_blocks -> hsa_forward.  By default the
step is captured once per input set in a CUDA graph and the timed loop replays
the graphs (`--launch eager` issues the same calls one by one instead).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 is launched by torchrun (one rank per GPU); every rank runs an
independent replica of the step (layers / heads partition with no collective in
the path), so the scaling is weak and `value` is the aggregate over ranks.
`--impl reference` times the CPU fp64 oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_34606_b200 import workloads as W  # noqa: E402



def ncu_traffic(workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one forward-kernel launch on `workload`, as
    recorded from the last ncu capture (a small tracked JSON beside the ncu summaries), or None."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    try:
        rec = json.load(open(path)).get("hsa_forward_kernel", {}).get(workload)
        return None if rec is None else float(rec["dram_bytes_read"]) + float(rec["dram_bytes_write"])
    except (OSError, ValueError, KeyError):
        return None


METRIC = "hsa_effective_tflops"
UNIT = "TFLOP/s"
RING = 4  # distinct (q, k, v, out) input sets rotated between steps (> L2 in total)


# ----------------------------------------------------------------------------- work model
def step_flops(w: W.Workload, sel_row_tokens, lin: str = "state", lin_rank: int = 0) -> dict:
    """Algorithmic FLOPs of one step (masked / unselected keys count as zero work).
    sel_row_tokens = sum over heads and query groups of (rows of the group) x (valid tokens of its
    selected blocks); with one selection per head that is Lq x the selected tokens of the head."""
    Lq, d, H = w.Lq, w.d, w.H
    sparse = 4.0 * d * float(sel_row_tokens)                          # QK^T + PV
    select = 2.0 * Lq * H * d + 2.0 * w.n_blocks * H * d
    if lin == "linformer":
        # compressed rows of all complete segments, softmax attention over them; the append projects
        # one segment: K~ = E_K^T K, V~ = E_V^T V
        lin_apply = 4.0 * Lq * (w.n_chunks * lin_rank) * d * H
        state = 2.0 * 2.0 * lin_rank * w.chunk * d * H
    else:
        lin_apply = 2.0 * Lq * d * (d + 1) * H                        # phi(Q) S and phi(Q) z
        state = 2.0 * w.chunk * d * (d + 1) * H                       # S += phi(K)^T V, z
    return {"forward": sparse + lin_apply, "append": state, "select": select,
            "total": sparse + lin_apply + state + select, "sparse": sparse, "linear": lin_apply}


def step_bytes(w: W.Workload, sel_tokens) -> dict:
    """Algorithmic HBM bytes per call (sel_tokens: valid tokens of the distinct selected blocks)."""
    Lq, d, H = w.Lq, w.d, w.H
    qo = Lq * H * d * 2
    fwd = 2 * qo + sel_tokens * d * 4 + H * d * d * 4
    app = 4 * w.chunk * H * d * 2 + H * d * d * 4 * 2
    sel = qo + w.n_blocks * H * d * 4
    return {"forward": float(fwd), "append": float(app), "select": float(sel)}


def workload_desc(w: W.Workload) -> str:
    return (f"{w.name}: H={w.H} d={w.d} chunk={w.Lq} history={w.N} tokens ({w.n_blocks} blocks of 64) " +
            (f"top-{w.topk} blocks/head" if not w.budget_set else f"budgets per head from {list(w.budget_set)} (-1 = all)"))


def load_peaks() -> dict:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons in the background."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device: torch.device):
        self.rows = []
        self.proc = None
        try:
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.rows.append((ts, float(parts[1]), float(parts[2]), parts[4:9]))
            except ValueError:
                continue

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float) -> dict:
        rows = [r for r in self.rows if t0 <= r[0] <= t1]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = sorted(r[1] for r in rows)
        names = ["active", "hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in rows:
            for n, v in zip(names[1:], r[3][1:]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": rows[0][2], "reasons": sorted(reasons),
                "samples": len(rows)}


# ----------------------------------------------------------------------------- ours
def bench_ours(args, rank: int, world: int):
    from paper_2609_34606_b200 import hsa
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    w = W.WORKLOADS[args.workload]
    gt = args.group_tokens
    lin_kw = {}
    if args.lin == "linformer":
        ek, ev = W.gen_linformer_weights(w, args.lin_rank, w.chunk)
        lin_kw = dict(lin_mode=hsa.HSA_LIN_LINFORMER, lin_rank=args.lin_rank, lin_seg_tokens=w.chunk,
                      e_k=ek.to(dev), e_v=ev.to(dev))
    ctx = hsa.HSAContext(w.H, w.d, max_pages=w.n_blocks, max_q_tokens=max(w.Lq, w.chunk),
                         max_topk=w.n_blocks if w.budget_set else max(w.topk, 1),
                         page_order=W.gen_page_order(w, w.n_blocks), device=dev, split_blocks=args.split_blocks, **lin_kw)
    for c in range(w.n_chunks - 1):
        k, v = W.gen_kv_chunk(w, c, layer=rank)
        ctx.append_kv(k.to(dev), v.to(dev))
    n_before = ctx.n_tokens
    # A step appends chunk n_chunks to the (n_chunks - 1)-chunk history; the next step first undoes that
    # append (hsa_rewind to the length before it: host bookkeeping only -- the state before the append
    # is still in the library's other state slot) and appends its own chunk.
    # host (pinned) and device copies of RING distinct input sets
    host, devs = [], []
    for r in range(RING):
        k, v = W.gen_kv_chunk(w, w.n_chunks - 1 + r, layer=rank)
        q = W.gen_query(w, step=r, layer=rank)
        hs = [t.pin_memory() for t in (q, k, v)]
        host.append(hs + [torch.empty_like(q).pin_memory()])
        devs.append([t.to(dev) for t in (q, k, v)] + [torch.empty(q.shape, dtype=torch.bfloat16, device=dev)])
    budgets = W.gen_budgets(w).to(dev)
    sel = ctx.alloc_selection(w.Lq, gt)

    def step(i, ev=None, from_host=False, with_forward=True):
        q, k, v, out = devs[i % RING]
        if from_host:
            hq, hk, hv, hout = host[i % RING]
            q.copy_(hq, non_blocking=True)
            k.copy_(hk, non_blocking=True)
            v.copy_(hv, non_blocking=True)
        ctx.rewind(n_before)
        if ev:
            ev[0].record()
        ctx.append_kv(k, v)
        if ev:
            ev[1].record()
        ctx.select_blocks(q, budgets, group_tokens=gt, sel=sel)
        if ev:
            ev[2].record()
        if with_forward:
            ctx.forward(q, sel[0], sel[1], group_tokens=gt, out=out)
        if ev:
            ev[3].record()
        if from_host:
            hout.copy_(out, non_blocking=True)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(dev) if (rank == 0 and not args.profile) else None
    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0, "device-side error during warm-up"
    cnt = sel[1].cpu()
    idx = sel[0].cpu()
    n_groups = cnt.shape[1]
    rows_of = lambda g: (min(w.Lq, (g + 1) * gt) - g * gt) if gt else w.Lq
    blk_tokens = lambda b: min(64, w.N - 64 * int(b))
    sel_row_tokens, distinct = 0, 0
    for h in range(w.H):
        seen = set()
        for g in range(n_groups):
            blocks = idx[h, g, :int(cnt[h, g])].tolist()
            sel_row_tokens += rows_of(g) * sum(blk_tokens(b) for b in blocks)
            seen.update(blocks)
        distinct += sum(blk_tokens(b) for b in seen)

    K = args.steps
    # eager pass with events between the calls: per-stage times (launch gaps included)
    Ks = max(3, min(K, 50))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(Ks)]
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s0.record()
    for i in range(Ks):
        step(i, evs[i])
    s1.record()
    torch.cuda.synchronize()
    ms_eager = s0.elapsed_time(s1) / Ks
    stage = [sum(evs[i][s].elapsed_time(evs[i][s + 1]) for i in range(Ks)) / Ks for s in range(3)]

    def capture(fn, n):
        """One CUDA graph holding fn(0), fn(1), ... fn(n - 1) (the input sets rotate inside fn)."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n):
                fn(i)
        return g

    def time_graph(g, n, reps=3):
        """Mean duration of one of the n calls held by the graph."""
        g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * n)

    # each call on its own, replayed from graphs: the kernels' own durations without launch gaps
    def only_append(i):
        ctx.rewind(n_before)
        ctx.append_kv(devs[i % RING][1], devs[i % RING][2])
    NK = 5 * RING  # calls per graph
    fwd = lambda flags: (lambda i: ctx.forward(devs[i % RING][0], sel[0], sel[1], group_tokens=gt,
                                               out=devs[i % RING][3], flags=flags))
    kern = {"append": time_graph(capture(only_append, NK), NK),
            "select": time_graph(capture(lambda i: ctx.select_blocks(devs[i % RING][0], budgets, group_tokens=gt,
                                                                     sel=sel), NK), NK),
            "forward": time_graph(capture(fwd(0), NK), NK),
            "linear_only": time_graph(capture(fwd(hsa.HSA_FWD_NO_SPARSE), NK), NK),
            "sparse_only": time_graph(capture(fwd(hsa.HSA_FWD_NO_LINEAR), NK), NK)}
    # the forward call inside the step: a graph of the same steps without it, subtracted from the full
    # one below (the kernel with its launch gap, behind the selection kernel and with the L2 contents
    # a step leaves; a kernel replayed on its own sees its pages in L2 and comes out a little faster)
    GSn = 2 * RING
    ms_step_no_fwd = time_graph(capture(lambda i: step(i, with_forward=False), GSn), GSn)
    ms_step_graph = time_graph(capture(step, GSn), GSn)
    step(0)  # leaves the context as a full step does

    # the timed loop: K steps, as replays of a graph that holds GS steps plus single-step graphs for
    # the remainder (or call by call with --launch eager)
    GS = 2 * RING
    if args.launch == "graph":
        g_many, g_one = capture(step, GS), [capture(lambda i, r=r: step(r), 1) for r in range(RING)]
        plan = [g_many] * (K // GS) + [g_one[i % RING] for i in range(K % GS)]
        run_all = lambda: [g.replay() for g in plan]
        warm = lambda: (g_many.replay(), [g.replay() for g in g_one])
    else:
        run_all = lambda: [step(i) for i in range(K)]
        warm = lambda: [step(i) for i in range(max(args.warmup, 3))]
    warm()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    wall0 = time.time()
    e0.record()
    run_all()
    e1.record()
    barrier()
    wall1 = time.time()
    ms_total = e0.elapsed_time(e1)
    status = ctx.device_status()

    # the last replayed step against the same step issued call by call: selection and output bit for bit
    last = (K - 1) % RING if (args.launch == "graph" and K % GS) or args.launch != "graph" else (GS - 1) % RING
    sel_replayed = (sel[0].clone(), sel[1].clone())
    out_replayed = devs[last][3].clone()
    step(last)
    torch.cuda.synchronize()
    cnt_e = sel[1].cpu()
    same = torch.equal(sel[1], sel_replayed[1]) and torch.equal(devs[last][3].view(torch.int16), out_replayed.view(torch.int16))
    same = same and all(torch.equal(sel[0][h, g, :int(cnt_e[h, g])], sel_replayed[0][h, g, :int(cnt_e[h, g])])
                        for h in range(w.H) for g in range(cnt_e.shape[1]))
    if not same or ctx.device_status() != 0:
        raise SystemExit("bench: the last replayed step differs from the same step issued call by call")

    # spread of the step time: each replay of the 8-step graph timed on its own (>= 20 repeats)
    reps = []
    if args.launch == "graph":
        evs_r = [torch.cuda.Event(enable_timing=True) for _ in range(25)]
        torch.cuda.synchronize()
        for i in range(24):
            evs_r[i].record()
            g_many.replay()
        evs_r[24].record()
        torch.cuda.synchronize()
        reps = sorted(evs_r[i].elapsed_time(evs_r[i + 1]) / GS for i in range(24))

    # clocks: sampled during the timed region; if that was too short for three samples, over an
    # identical loop run right after it (said so in the record)
    probe = None
    if sampler is not None:
        time.sleep(0.15)
        clocks = sampler.summary(wall0, wall1)
        if clocks["samples"] < 3:
            p0 = time.time()
            i = 0
            while time.time() - p0 < 1.5:
                run_all()
                i += 1
                if i % 4 == 0:
                    torch.cuda.synchronize()
            torch.cuda.synchronize()
            p1 = time.time()
            time.sleep(0.15)
            probe = sampler.summary(p0, p1)
    ms_lin_only, ms_sp_only = kern["linear_only"], kern["sparse_only"]
    if args.profile:
        if rank == 0:
            print(json.dumps({"profile_run": True, "launch": args.launch, "steps": K, "ms_per_step": ms_total / K,
                              "eager_ms_per_step": ms_eager,
                              "eager_stage_ms": {"append": stage[0], "select": stage[1], "forward": stage[2]},
                              "kernel_ms": kern, "forward_in_step_ms": ms_step_graph - ms_step_no_fwd}))
        ctx.destroy()
        return
    # end-to-end through the same API with host buffers: every step copies its inputs from pinned
    # host memory and its result back.  The copies run on their own streams, so that the upload of
    # step i + 1 and the download of step i - 1 overlap the kernels of step i (the RING device slots
    # give the look-ahead); the timed region runs from the first upload to the last download.
    Ke = max(3, min(K, 50))
    s_comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def e2e_loop(n):
        ev_in = [torch.cuda.Event() for _ in range(n)]
        ev_done = [torch.cuda.Event() for _ in range(n)]
        ev_out = [torch.cuda.Event() for _ in range(n)]
        for i in range(n):
            q, k, v, out = devs[i % RING]
            hq, hk, hv, hout = host[i % RING]
            with torch.cuda.stream(s_in):
                if i >= RING:
                    s_in.wait_event(ev_done[i - RING])      # the slot's previous step has read its inputs
                q.copy_(hq, non_blocking=True)
                k.copy_(hk, non_blocking=True)
                v.copy_(hv, non_blocking=True)
                ev_in[i].record(s_in)
            s_comp.wait_event(ev_in[i])
            if i >= RING:
                s_comp.wait_event(ev_out[i - RING])         # ... and its result has left the slot
            step(i)
            ev_done[i].record(s_comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                hout.copy_(out, non_blocking=True)
                ev_out[i].record(s_out)
        s_comp.wait_stream(s_out)

    e2e_loop(3)
    barrier()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    s_in.wait_event(g0)
    e2e_loop(Ke)
    g1.record()
    barrier()
    ms_e2e = g0.elapsed_time(g1) / Ke
    if sampler is not None:
        sampler.stop()

    from paper_2609_34606_b200 import sharding
    fl = step_flops(w, sel_row_tokens, args.lin, args.lin_rank)
    # whole job: the FLOPs of all ranks over the slowest rank's time
    agg_flops, sec_step = sharding.aggregate_throughput(fl["total"], ms_total / K * 1e-3, device=dev)
    agg_e2e, sec_e2e = sharding.aggregate_throughput(fl["total"], ms_e2e * 1e-3, device=dev)
    ms_step, ms_e2e = sec_step * 1e3, sec_e2e * 1e3
    by = step_bytes(w, distinct)
    peaks = load_peaks()
    if rank == 0:
        if probe is not None:
            clocks = dict(probe, note="timed region shorter than 3 samples; sampled over an identical "
                                      "1.5 s loop run right after it")
        tf = lambda f, ms: f / (ms * 1e-3) / 1e12
        fwd_tf = tf(fl["forward"], kern["forward"])
        line = {
            "metric": METRIC, "value": agg_flops / 1e12, "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_desc(w),
                       "selection": "one per head for the whole chunk" if not gt else f"one per {gt}-row query tile",
                       "linear_branch": ("running state (S, z)" if args.lin == "state" else
                                         f"Linformer form, rank {args.lin_rank}, segments of {w.chunk} tokens"),
                       "step": f"undo the previous step's append (back to the {w.n_chunks - 1}-chunk history) + hsa_append_kv + "
                               "hsa_select_blocks + hsa_forward",
                       "launch": (f"CUDA graphs: the timed loop replays a graph of {2 * RING} consecutive steps "
                                  "(single-step graphs for the remainder)"
                                  if args.launch == "graph" else "eager: every call issued from the host"),
                       "l2": f"inputs rotate over {RING} distinct (q,k,v,out) sets "
                             f"({RING * 4 * w.Lq * w.H * w.d * 2 / 1e6:.0f} MB > 126 MB L2)",
                       "replicas": world},
            "ms_per_chunk": ms_step,
            "ms_per_step_repeats": ({"n": len(reps), "min": reps[0], "median": reps[len(reps) // 2], "max": reps[-1]}
                                    if reps else None),
            "replay_check": "last replayed step == the same step issued call by call (selection and output bits)",
            "eager_ms_per_step": ms_eager,
            "eager_stage_ms": {"append": stage[0], "select": stage[1], "forward": stage[2]},
            "kernel_ms": {k2: kern[k2] for k2 in ("append", "select", "forward")},
            "kernel_gbs": {k2: by[k2] / kern[k2] / 1e6 for k2 in ("append", "select", "forward")},
            "flops_per_step": fl["total"],
            "forward_modes_ms": {"linear_only": ms_lin_only, "sparse_only": ms_sp_only,
                                 "linear_only_gbs": (2 * w.Lq * w.H * w.d * 2 + w.H * w.d * w.d * 4) / ms_lin_only / 1e6},
            "clocks": clocks,
            "e2e": {"value": agg_e2e / 1e12, "unit": UNIT, "ms_per_step": ms_e2e,
                    "h2d_bytes_per_step": 3 * w.Lq * w.H * w.d * 2, "d2h_bytes_per_step": w.Lq * w.H * w.d * 2},
            # per step: append_fused, state_reduce, hsa_forward and the selection -- two kernels (query
            # sums, then one cluster per head) for one list per head while a head has at most 192
            # score items of 32 blocks, one cooperative kernel otherwise
            "gpu_launches": (5 if (args.group_tokens == 0 and w.n_blocks <= 192 * 32) else 4) * K,
            # (the Linformer form has as many: page write + projection instead of the fused append and
            # its reduction, one forward launch that walks the compressed pool before the selected pages)
            "device_status": status,
            "roofline": {"kernel": "hsa_forward_kernel<128, false>", "bound": "tensor", "achieved": fwd_tf,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": fwd_tf / peaks["bf16_tflops"],
                         "traffic": ncu_traffic(w.name), "algorithmic_bytes": by["forward"],
                         "peak_source": peaks["source"] + " (burst)",
                         "frac_of_sustained": fwd_tf / peaks["bf16_tflops_sustained"],
                         "timing": "average duration of the call replayed from CUDA graphs, CUDA events",
                         "in_step_ms": ms_step_graph - ms_step_no_fwd,
                         "frac_in_step": tf(fl["forward"], ms_step_graph - ms_step_no_fwd) / peaks["bf16_tflops"],
                         "in_step_timing": "graph of 8 steps minus the same graph without the forward call, per step",
                         "append_hbm_frac": by["append"] / kern["append"] / 1e6 / peaks["hbm_gbs"],
                         "select_hbm_frac": by["select"] / kern["select"] / 1e6 / peaks["hbm_gbs"],
                         "linear_only_hbm_frac": (2 * w.Lq * w.H * w.d * 2 + w.H * w.d * w.d * 4) / ms_lin_only
                                                 / 1e6 / peaks["hbm_gbs"]},
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(w, rows=args.cpu_rows)
        print(json.dumps(line), flush=True)
    ctx.destroy()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- rollout (cfg5)
def bench_rollout(args, rank: int, world: int):
    """Full-stack rollout: `layers` contexts, n_chunks chunks; per chunk and layer append the chunk,
    select, forward (the history grows, so the calls are issued one by one: no graph fits).  Inputs
    rotate over a ring of 8 (q, k, v) triples per layer generated on the device (seeded N(0,1))."""
    from paper_2609_34606_b200 import hsa
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    w = W.WORKLOADS[args.workload]
    layers = args.layers or w.layers
    RR = 8
    ctxs = [hsa.HSAContext(w.H, w.d, max_pages=w.n_blocks, max_q_tokens=w.Lq, max_topk=w.topk, device=dev)
            for _ in range(layers)]
    g = torch.Generator(device=dev)
    ring = []
    for layer in range(layers):
        g.manual_seed(4_000_000 + 1000 * layer + rank)
        ring.append([[torch.randn(w.Lq, w.H, w.d, device=dev, generator=g).to(torch.bfloat16) for _ in range(3)]
                     for _ in range(RR)])
    outs = [torch.empty(w.Lq, w.H, w.d, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    budgets = W.gen_budgets(w).to(dev)
    sels = [c.alloc_selection(w.Lq) for c in ctxs]

    def rollout(n_chunks, evs=None):
        for c in range(n_chunks):
            if evs is not None:
                evs[c].record()
            for layer, ctx in enumerate(ctxs):
                q, k, v = ring[layer][c % RR]
                ctx.append_kv(k, v)
                ctx.select_blocks(q, budgets, sel=sels[layer])
                ctx.forward(q, sels[layer][0], sels[layer][1], out=outs[layer & 1])
        if evs is not None:
            evs[n_chunks].record()

    def reset():
        for ctx in ctxs:
            ctx.rewind(0)
            ctx.state.zero_()

    rollout(3)                    # warm-up
    torch.cuda.synchronize()
    assert all(c.device_status() == 0 for c in ctxs)
    sampler = ClockSampler(dev)
    runs = []
    for rep_i in range(2):        # the second rollout shows the run-to-run spread
        reset()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(w.n_chunks + 1)]
        torch.cuda.synchronize()
        t0 = time.time()
        rollout(w.n_chunks, evs)
        torch.cuda.synchronize()
        t1 = time.time()
        per_chunk = [evs[c].elapsed_time(evs[c + 1]) for c in range(w.n_chunks)]
        runs.append({"ms_total": evs[0].elapsed_time(evs[-1]), "wall": (t0, t1), "per_chunk": per_chunk})
    time.sleep(0.2)
    clocks = sampler.summary(runs[0]["wall"][0], runs[1]["wall"][1])
    sampler.stop()
    status = max(c.device_status() for c in ctxs)
    # work model: 64 full blocks per head from the first chunk on (a chunk alone is 73 blocks)
    fl = step_flops(w, w.Lq * w.topk * 64 * w.H)
    steps = w.n_chunks * layers
    best = min(runs, key=lambda r: r["ms_total"])
    ms_step = best["ms_total"] / steps
    pc = best["per_chunk"]
    print(json.dumps({
        "metric": METRIC, "value": fl["total"] / (ms_step * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1,
        "steps": steps, "warmup": 3 * layers, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name}: rollout of {w.n_chunks} chunks x {layers} layers, H={w.H} d={w.d} "
                               f"chunk={w.Lq}, top-{w.topk} blocks/head, history grows to {w.n_chunks * w.chunk} tokens",
                   "step": "hsa_append_kv + hsa_select_blocks + hsa_forward of one layer for one chunk",
                   "launch": "eager: every call issued from the host (the history grows every step)",
                   "l2": f"{layers} layers x {RR} rotating (q,k,v) triples, pools {layers * 2 * w.n_blocks * w.H * 64 * w.d * 2 / 1e9:.0f} GB"},
        "rollout_ms": [r["ms_total"] for r in runs],
        "ms_per_chunk_all_layers": {"first": pc[0], "median": sorted(pc)[len(pc) // 2], "last": pc[-1]},
        "flops_per_step": fl["total"], "clocks": clocks,
        # (the selection is two kernels while the history has at most 6144 blocks, one beyond that)
        "gpu_launches": layers * sum(5 if (c + 1) * w.chunk <= 6144 * 64 else 4 for c in range(w.n_chunks)),
        "device_status": status}),
        flush=True)
    for c in ctxs:
        c.destroy()


# ----------------------------------------------------------------------------- oracle (CPU)
def oracle_step(w: W.Workload, data, rows):
    """One bounded oracle step, stage by stage: block selection over the full history, the sparse
    branch on `rows` query rows, the linear branch (state from scratch, applied to the chunk), the
    merge.  Returns (seconds in all, selection, seconds per stage)."""
    from oracle import hsa_oracle as O
    q, K, V = data
    t = [time.perf_counter()]
    sel, _ = O.select_blocks(q, K, w.q_pos0, w.causal, W.gen_budgets(w).tolist())
    t.append(time.perf_counter())
    o_sp = O.sparse_branch(q, K, V, sel, w.q_pos0, w.causal, rows=rows)
    t.append(time.perf_counter())
    if w.causal:
        o_lin = O.linear_parallel(q, K, V, w.q_pos0, True, rows)
    else:
        S, z = O.linear_state(K, V)
        o_lin = O.linear_from_state(q, S, z)
    t.append(time.perf_counter())
    O.merge(o_lin, o_sp)
    t.append(time.perf_counter())
    stages = dict(zip(("select", "sparse", "linear", "merge"), (b - a for a, b in zip(t, t[1:]))))
    return t[-1] - t[0], sel, stages


def oracle_data(w: W.Workload):
    K, V = W.gen_history(w)
    q = W.gen_query(w)
    return q.float().numpy(), K.float().numpy(), V.float().numpy()


def oracle_value(w: W.Workload, sel, rows, seconds: float) -> float:
    sel_tokens = sum(min(64, w.N - 64 * int(b)) for h in range(w.H) for b in sel[h][0])
    fl = step_flops(w, w.Lq * sel_tokens)
    frac = len(rows) / w.Lq
    flops = fl["forward"] * frac + fl["select"] + fl["append"] * w.n_chunks  # state built from scratch
    return flops / seconds / 1e12


def cpu_baseline(w: W.Workload, rows: int = 256) -> dict:
    import numpy as np
    data = oracle_data(w)
    r = np.sort(W.random_rows(w, rows).numpy())
    secs, stage_sum = [], {}
    while sum(secs) < 10.0 and len(secs) < 8:      # about 10 s of CPU work in all
        sec, sel, stages = oracle_step(w, data, r)
        secs.append(sec)
        for k2, v2 in stages.items():
            stage_sum[k2] = stage_sum.get(k2, 0.0) + v2
    sec = sum(secs) / len(secs)
    return {"value": oracle_value(w, sel, r, sec), "unit": UNIT, "cores": len(os.sched_getaffinity(0)),
            "kind": "oracle", "seconds": sec, "repeats": len(secs),
            "stage_seconds": {k2: v2 / len(secs) for k2, v2 in stage_sum.items()},
            "sample": f"block selection over the full {w.N}-token history + linear state from scratch + both "
                      f"branches and merge on {len(r)} seeded query rows of {w.Lq}; algorithmic FLOPs of that "
                      "sample / wall time"}


def bench_reference(args, rank: int, world: int):
    if rank != 0:
        return
    import numpy as np
    w = W.WORKLOADS[args.workload]
    data = oracle_data(w)
    r = np.sort(W.random_rows(w, args.cpu_rows).numpy())
    K = max(1, min(args.steps, 5))
    Wm = max(0, min(args.warmup, 1))
    for _ in range(Wm):
        oracle_step(w, data, r)
    secs = []
    for _ in range(K):
        s, sel, _ = oracle_step(w, data, r)
        secs.append(s)
    sec = sum(secs) / len(secs)
    val = oracle_value(w, sel, r, sec)
    cores = len(os.sched_getaffinity(0))
    sample = (f"per step: block selection over the full {w.N}-token history + linear state from scratch + both "
              f"branches and merge on {len(r)} seeded query rows of {w.Lq}")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": Wm, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_desc(w)},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


# ----------------------------------------------------------------------------- context (third party)
def context_library_attention(args):
    """Context only -- neither the product nor the oracle: library attention kernels (torch SDPA back
    ends, flash_attn, flashinfer, whichever the image has) on dense, contiguous K and V of the size
    the workload's sparse branch selects (top-k blocks per head), i.e. the same FLOPs as the sparse
    branch without the page gather.  One JSON line."""
    w = W.WORKLOADS[args.workload]
    dev = torch.device("cuda:0")
    T = min(w.topk * W.BLOCK, w.N)
    gen = torch.Generator(device="cpu").manual_seed(1234)
    q, k, v = (torch.randn(1, w.H, n, w.d, generator=gen).to(torch.bfloat16).to(dev) for n in (w.Lq, T, T))
    flops = 4.0 * w.Lq * T * w.d * w.H

    def timeit(fn, n=50):
        for _ in range(5):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    res = {}
    from torch.nn.attention import SDPBackend, sdpa_kernel
    for name, be in (("torch_sdpa_cudnn", SDPBackend.CUDNN_ATTENTION), ("torch_sdpa_flash", SDPBackend.FLASH_ATTENTION)):
        try:
            with sdpa_kernel(be):
                ms = timeit(lambda: torch.nn.functional.scaled_dot_product_attention(q, k, v))
            res[name] = {"ms": ms, "tflops": flops / ms / 1e9}
        except Exception as e:  # a back end the build does not have
            res[name] = {"unavailable": type(e).__name__}
    try:
        from flash_attn import flash_attn_func
        q2, k2, v2 = (t.transpose(1, 2).contiguous() for t in (q, k, v))
        ms = timeit(lambda: flash_attn_func(q2, k2, v2))
        res["flash_attn"] = {"ms": ms, "tflops": flops / ms / 1e9}
    except Exception as e:
        res["flash_attn"] = {"unavailable": type(e).__name__}
    print(json.dumps({"context": "third-party attention kernels on dense contiguous K, V of the selected size "
                                 "(same FLOPs as the sparse branch, no page gather); not the product, not the oracle",
                      "workload": f"{w.name}: H={w.H} d={w.d} Lq={w.Lq} keys={T}", "flops": flops, "results": res}),
          flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000,
                    help="timed steps (the default makes the timed region about half a second long, so that the "
                         "clock samples belong to it)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--cpu-rows", type=int, default=4680)
    ap.add_argument("--layers", type=int, default=0, help="rollout workloads: number of layers (0 = the workload's)")
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"],
                    help="how the timed steps are issued: replayed CUDA graphs (default) or call by call")
    ap.add_argument("--group-tokens", type=int, default=0,
                    help="0: one selection per head for the whole chunk; 128: one per 128-row query tile")
    ap.add_argument("--lin", default="state", choices=["state", "linformer"],
                    help="linear branch: the running-state form (measured configuration) or the Linformer form")
    ap.add_argument("--lin-rank", type=int, default=256, help="Linformer projection rank")
    ap.add_argument("--split-blocks", type=int, default=0,
                    help="blocks per part when a long list is split over several CTAs (0 = the library's default)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile", action="store_true",
                    help="profiling run: set-up, warm-up and the K timed steps only (no clock probe loop, "
                         "no end-to-end loop, no CPU baseline), for use under ncu")
    ap.add_argument("--context", action="store_true",
                    help="context only: time library attention kernels (third party) on dense K, V of the "
                         "selected size and exit")
    ap.add_argument("--rank-check", action="store_true",
                    help="start the ranks, let them meet over gloo and report the aggregation of stand-in "
                         "numbers, then exit before any GPU is touched (checks the launcher on a CPU box)")
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be >= 1")
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.impl == "ours":
        # started by hand with --gpus N: start the N ranks ourselves (one process per GPU)
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "ours" and world != args.gpus:
        sys.exit(f"bench: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if args.rank_check:
        rank_check(rank, world)
    elif args.context:
        if rank == 0:
            context_library_attention(args)
    elif args.impl == "reference":
        bench_reference(args, rank, world)
    elif W.WORKLOADS[args.workload].layers > 1:
        if rank == 0:
            bench_rollout(args, rank, world)
    else:
        bench_ours(args, rank, world)


def rank_check(rank: int, world: int) -> None:
    """The multi-rank bookkeeping of bench_ours without a GPU: rendezvous, barrier, whole-job
    throughput of stand-in numbers (rank r: 1 unit of work in 1 + r seconds)."""
    import torch.distributed as dist
    from paper_2609_34606_b200 import sharding
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    thr, slowest = sharding.aggregate_throughput(1.0, 1.0 + rank)
    if rank == 0:
        print(json.dumps({"rank_check": True, "n_gpus": world, "local_rank": int(os.environ.get("LOCAL_RANK", "0")),
                          "value": thr, "slowest_s": slowest}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def spawn_ranks(n: int, argv, env=None) -> int:
    """Runs this script as n ranks under torch.distributed.run on this node (rendezvous on 127.0.0.1);
    returns the launcher's exit code."""
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd, env=env)


if __name__ == "__main__":
    main()
