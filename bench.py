#!/usr/bin/env python
"""Benchmark of the MoC hot path (pool -> route -> attend, + backward for the training
workload) on seeded synthetic inputs.

    python bench.py --gpus N --steps K --warmup W [--workload cfg2] [--impl reference]

One step = one pass of the whole hot path over one batch.  The headline value is the
selected-key attention throughput of the whole step: 4*d FLOPs per selected (query, key)
pair (10*d more with the backward), divided by the device time of the step, summed over
ranks.  Ranks are independent replicas (one process per GPU, no data-path collective;
rank r draws its inputs with seed r): weak scaling.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moc_sparse_attention_selected_key_tflops"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self._stop, self._t = index, [], threading.Event(), None

    def _loop(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout.strip()
                if out:
                    self.rows.append([f.strip() for f in out.splitlines()[0].split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._t = threading.Thread(target=self._loop, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=10)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measured_traffic(kernel: str, workload: str):
    """DRAM bytes per call from the committed ncu summary, or None when the kernel source has
    changed since the counters were taken (profiles/traffic.txt: kernel workload bytes sha1-of-source)."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) == 5 and parts[0] == kernel and parts[1] == workload:
                    with open(os.path.join(ROOT, parts[4]), "rb") as src:
                        if hashlib.sha1(src.read()).hexdigest() == parts[3]:
                            return float(parts[2])
    except Exception:
        pass
    return None


def max_over_ranks_ms(ms: float, world: int, device) -> float:
    """Slowest rank's time: ranks are independent replicas, so the job's step time is the max."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(flops_per_rank: float, world: int, ms_per_step: float) -> float:
    """Whole-job TFLOP/s: every rank does `flops_per_rank` per step in `ms_per_step`."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def step_flops(wl, pairs: int, with_bwd: bool) -> float:
    return (4.0 + (10.0 if with_bwd else 0.0)) * wl.head_dim * pairs


def route_bytes(wl) -> float:
    H, L, d, C, k = wl.n_heads, wl.n_tokens, wl.head_dim, wl.n_chunks, wl.top_k
    return 2.0 * (2 * L * d * H) + 4.0 * k * L * H + 2 * 4.0 * C * d * H   # K once + Q once + indices + desc write/read


def config_of(wl, with_bwd: bool, world: int) -> dict:
    """The workload's description, the same in both arms (what a run measured about it goes elsewhere)."""
    H, L, d = wl.n_heads, wl.n_tokens, wl.head_dim
    return {"workload": wl.name, "layout": wl.note, "heads": H, "head_dim": d, "tokens": L, "chunks": wl.n_chunks,
            "top_k": wl.top_k, "window": [wl.win_back, wl.win_fwd], "backward": with_bwd,
            "l2": "inputs larger than L2 (Q, K, V %.0f MB each); no flush" % (H * L * d * 2 / 1e6),
            "parallelism": f"replicas x{world}"}


def run_reference(args, wl):
    """The CPU oracle, as it stands, timed per step on a bounded sample of the workload:
    one head's descriptors and routing in full, attention on a seeded sample of its rows."""
    import numpy as np
    import oracle
    from oracle import Oracle
    from paper_2508_21058_b200 import workloads as W
    rows_per_step = args.ref_rows
    heads = [s % wl.n_heads for s in range(args.warmup + args.steps)]
    times, flops = [], []
    for s, h in enumerate(heads):
        x = {n: W.as_u16(t) for n, t in W.generate(wl, "cpu", ("q", "k", "v"), heads=[h]).items()}
        orc = Oracle.from_workload(wl, n_heads=1)
        rng = np.random.RandomState(100 + s)
        rows = np.stack([np.zeros(rows_per_step, np.int32),
                         np.sort(rng.randint(0, wl.n_tokens, rows_per_step)).astype(np.int32)], 1)
        t0 = time.perf_counter()
        desc = orc.chunk_pool(x["k"])
        sel = orc.route(x["q"], desc)
        orc.attend(x["q"], x["k"], x["v"], sel, rows)
        dt = time.perf_counter() - t0
        if s >= args.warmup:
            times.append(dt)
            flops.append(4.0 * wl.head_dim * orc.pair_count(sel, rows))
    total_t, total_f = sum(times), sum(flops)
    value = total_f / total_t / 1e12
    sample = (f"per step: descriptors + routing of one head in full ({wl.n_tokens} rows), attention on "
              f"{rows_per_step} seeded rows of that head")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(len(times), 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, args.bwd or args.workload == "cfg4", int(os.environ.get("WORLD_SIZE", "1"))),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def cpu_baseline(wl, budget_s: float):
    """Oracle attention on a bounded seeded row sample (sized from a short probe)."""
    import numpy as np
    import oracle
    from oracle import Oracle
    from paper_2508_21058_b200 import workloads as W
    x = {n: W.as_u16(t) for n, t in W.generate(wl, "cpu", ("q", "k", "v"), heads=[0]).items()}
    orc = Oracle.from_workload(wl, n_heads=1)
    t0 = time.perf_counter()
    sel = orc.route(x["q"], orc.chunk_pool(x["k"]))
    t_route = time.perf_counter() - t0
    rng = np.random.RandomState(42)

    def sample(n):
        return np.stack([np.zeros(n, np.int32), np.sort(rng.randint(0, wl.n_tokens, n)).astype(np.int32)], 1)

    probe = sample(64)
    t0 = time.perf_counter()
    orc.attend(x["q"], x["k"], x["v"], sel, probe)
    per_row = (time.perf_counter() - t0) / len(probe)
    n = int(max(64, min(2000000, budget_s / max(per_row, 1e-6))))
    rows = sample(n)
    t0 = time.perf_counter()
    orc.attend(x["q"], x["k"], x["v"], sel, rows)
    dt = time.perf_counter() - t0
    fl = 4.0 * wl.head_dim * orc.pair_count(sel, rows)
    return {"value": fl / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"attention of {n} seeded rows of head 0 ({dt:.1f} s); head-0 descriptors + routing took {t_route:.1f} s"}


def run_ours(wl, with_bwd, steps, warmup, world, local_rank, do_e2e):
    """Times `steps` passes of the hot path on one workload; returns the measurements of this rank
    (times already reduced to the slowest rank)."""
    import torch
    import torch.distributed as dist
    from paper_2508_21058_b200 import MocPlan, launch_count
    from paper_2508_21058_b200 import workloads as W

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def _rec():
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    tensors = ("q", "k", "v", "do") if with_bwd else ("q", "k", "v")
    x = W.generate(wl, "cuda", tensors)
    plan = MocPlan.from_workload(wl)
    ws = plan.new_workspace(with_bwd)
    H, L, d, C, k = wl.n_heads, wl.n_tokens, wl.head_dim, wl.n_chunks, wl.top_k
    desc = torch.empty((H, C, d), dtype=torch.float32, device="cuda")
    sel = torch.empty((H, L, k), dtype=torch.int32, device="cuda")
    O = torch.empty_like(x["q"])
    lse = torch.empty((H, L), dtype=torch.float32, device="cuda")
    grads = [torch.empty_like(x["q"]) for _ in range(3)] if with_bwd else None

    def step(q, kk, v, marks=None, out=None):
        o_, l_ = out if out is not None else (O, lse)
        ev = (lambda: marks.append(_rec())) if marks is not None else (lambda: None)
        ev()
        plan.moc_chunk_pool(kk, desc, ws)
        ev()
        plan.moc_route(q, desc, sel, ws)
        ev()
        plan.moc_attend(q, kk, v, sel, o_, l_, ws)
        ev()
        if with_bwd:
            plan.moc_attend_bwd(q, kk, v, o_, l_, x["do"], sel, *grads, ws)
            ev()

    for _ in range(max(warmup, 3)):
        step(x["q"], x["k"], x["v"])
    barrier()
    st, det = plan.moc_get_status(ws)
    if st != 0:
        raise SystemExit(f"device status {st} detail {det}")
    pairs = plan.moc_selected_pairs(ws)
    flops = step_flops(wl, pairs, with_bwd)

    # ---- timed region: inputs resident in HBM, device time by CUDA events on the launching stream
    marks_all = []
    n0 = launch_count()
    with ClockSampler(local_rank) as clocks:
        barrier()
        for _ in range(steps):
            m = []
            step(x["q"], x["k"], x["v"], m)
            marks_all.append(m)
        barrier()
    launches = launch_count() - n0
    total_ms = marks_all[0][0].elapsed_time(marks_all[-1][-1])
    seg = [sum(m[i].elapsed_time(m[i + 1]) for m in marks_all) / steps for i in range(len(marks_all[0]) - 1)]
    ms_per_step = max_over_ranks_ms(total_ms, world, "cuda") / steps
    out = {"pairs": pairs, "flops": flops, "ms_per_step": ms_per_step, "seg": seg, "launches": int(launches), "timed_ms": total_ms,
           "clocks": clocks.summary(), "workspace_bytes": plan.workspace_bytes(with_bwd), "e2e": None}

    # ---- end to end: host buffers in, host results out, copies inside the timed region
    if do_e2e:
        hq, hk, hv = (x[n].cpu().pin_memory() for n in ("q", "k", "v"))
        dq, dk, dv = (torch.empty_like(x[n]) for n in ("q", "k", "v"))
        hO = torch.empty(O.shape, dtype=O.dtype).pin_memory()
        hl = torch.empty(lse.shape, dtype=lse.dtype).pin_memory()
        hg = [torch.empty(O.shape, dtype=O.dtype).pin_memory() for _ in range(3)] if with_bwd else []

        def e2e_step():
            dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
            step(dq, dk, dv)
            hO.copy_(O, non_blocking=True); hl.copy_(lse, non_blocking=True)
            for a, b in zip(hg, grads or []):
                a.copy_(b, non_blocking=True)
            torch.cuda.current_stream().synchronize()

        n_e2e = max(2, min(steps, 5))
        e2e_step()
        barrier()
        e0 = _rec()
        for _ in range(n_e2e):
            e2e_step()
        e1 = _rec()
        barrier()
        te_serial_ms = max_over_ranks_ms(e0.elapsed_time(e1), world, "cuda")
        h2d = 3 * hq.numel() * 2
        d2h = hO.numel() * 2 + hl.numel() * 4 + sum(g.numel() * 2 for g in hg)
        out["e2e"] = {"value": job_value(flops, world, te_serial_ms / n_e2e), "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e, "copies": "serial with the compute"}
        if not with_bwd:
            # The same work with the copies on streams of their own and two sets of device buffers: step i's
            # inputs travel while step i - 1 computes and step i - 2's results go back.  Every step still copies
            # its own inputs in and its own results out inside the timed region.
            main = torch.cuda.current_stream()
            s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
            ins = [(dq, dk, dv), tuple(torch.empty_like(t) for t in (dq, dk, dv))]
            outs = [(O, lse), (torch.empty_like(O), torch.empty_like(lse))]
            n_pipe = 2 * n_e2e

            def pipelined(n):
                in_done, comp_done, out_done = [], [], []
                for i in range(n):
                    b = i & 1
                    with torch.cuda.stream(s_in):
                        if i >= 2:
                            s_in.wait_event(comp_done[i - 2])       # the buffers' previous user has computed
                        for dst, src in zip(ins[b], (hq, hk, hv)):
                            dst.copy_(src, non_blocking=True)
                        in_done.append(_rec())
                    main.wait_event(in_done[i])
                    if i >= 2:
                        main.wait_event(out_done[i - 2])            # the output buffers have gone back
                    step(*ins[b], out=outs[b])
                    comp_done.append(_rec())
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(comp_done[i])
                        hO.copy_(outs[b][0], non_blocking=True)
                        hl.copy_(outs[b][1], non_blocking=True)
                        out_done.append(_rec())
                main.wait_event(out_done[-1])

            s_in.wait_stream(main)
            s_out.wait_stream(main)
            pipelined(2)
            barrier()
            p0 = _rec()
            pipelined(n_pipe)
            p1 = _rec()
            barrier()
            tp_ms = max_over_ranks_ms(p0.elapsed_time(p1), world, "cuda")
            out["e2e"].update({"value": job_value(flops, world, tp_ms / n_pipe), "steps": n_pipe,
                               "copies": "on their own streams, two sets of device buffers (inputs of step i travel while step i-1 computes)",
                               "serial_value": job_value(flops, world, te_serial_ms / n_e2e)})
            del ins, outs
    plan.close()
    del x, ws, desc, sel, O, lse, grads
    torch.cuda.empty_cache()
    return out


def rooflines(wl, r, peaks, peak_kind):
    """Roofline objects of the attention call and of pooling + routing.  The attention peak is the measured bf16
    matmul rate of the regime the call was timed in: the burst figure when the whole timed region is short, the
    sustained one (seconds under the power cap) when it lasts long enough for the GPU to settle at its cap."""
    H, L, d = wl.n_heads, wl.n_tokens, wl.head_dim
    t_pool, t_route, t_att = r["seg"][0], r["seg"][1], r["seg"][2]
    att_flops = step_flops(wl, r["pairs"], False)
    att = att_flops / (t_att * 1e-3) / 1e12
    long_run = r.get("timed_ms", 0.0) >= 500.0
    peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
    roofline = {"kernel": "moc_attend (persistent tensor-core flash kernel over selected key chunks)",
                "bound": "tensor", "achieved": att, "peak": peak,
                "unit": "TFLOP/s", "frac": att / peak,
                "frac_of_burst": att / peaks["bf16_tflops"],
                "frac_of_sustained": att / peaks["bf16_tflops_sustained"],
                "traffic": measured_traffic("moc_attend", wl.name),
                "peak_source": f"{peak_kind} ({'sustained' if long_run else 'burst'} bf16 matmul; timed region {r.get('timed_ms', 0.0):.0f} ms)",
                "ms": t_att}
    rb = route_bytes(wl)
    gbs = rb / ((t_pool + t_route) * 1e-3) / 1e9
    routing = {"kernel": "moc_chunk_pool + moc_route", "bound": "hbm", "achieved": gbs,
               "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
               "pool_ms": t_pool, "route_ms": t_route, "pool_gbs": (2.0 * L * d * H) / (t_pool * 1e-3) / 1e9,
               "peak_source": peak_kind}
    return roofline, routing


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2",
                    help="cfg2 (the largest forward-only configuration) by default; cfg1, cfg4, cfg3-m<chunk>-p<percent>")
    ap.add_argument("--bwd", action="store_true", help="include moc_attend_bwd in the step (implied by cfg4)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--cpu-budget-s", type=float, default=15.0)
    ap.add_argument("--ref-rows", type=int, default=256)
    ap.add_argument("--heads", type=int, default=0, help="override the head count (profiling a smaller case)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2508_21058_b200 import workloads as W
    wl = W.workload(args.workload, seed=rank)
    if args.heads > 0:
        wl.n_heads = args.heads
        wl.name = f"{wl.name}-h{args.heads}"
    with_bwd = args.bwd or args.workload == "cfg4"

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    r = run_ours(wl, with_bwd, args.steps, args.warmup, world, local_rank, not args.no_e2e)
    # the other configurations, a few steps each, so that one run covers the small single-shot clip, the
    # multi-shot stream and the training step (forward + backward)
    others = {}
    if args.workload == "cfg2" and args.heads == 0 and not args.no_others:
        # (the single-shot clip's step is a few ms: 20 steps, so that the first launch after the barrier does not weigh)
        for name, bwd, n in (("cfg1", False, 20), ("cfg4", True, 3)):
            w2 = W.workload(name, seed=rank)
            others[name] = (w2, bwd, n, run_ours(w2, bwd, n, 3, world, local_rank, False))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_peaks()
    H, L, d, C, k = wl.n_heads, wl.n_tokens, wl.head_dim, wl.n_chunks, wl.top_k
    roofline, routing = rooflines(wl, r, peaks, peak_kind)
    seg = r["seg"]
    line = {"metric": METRIC, "value": job_value(r["flops"], world, r["ms_per_step"]), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": config_of(wl, with_bwd, world),
            "workload_stats": {"selected_pairs": r["pairs"], "sparsity_vs_dense": 1.0 - r["pairs"] / (float(H) * L * L),
                               "workspace_bytes": r["workspace_bytes"]},
            "segments_ms": {"pool": seg[0], "route": seg[1], "attend": seg[2], **({"attend_bwd": seg[3]} if with_bwd else {})},
            "roofline": roofline, "roofline_routing": routing, "clocks": r["clocks"], "gpu_launches": r["launches"]}
    if r["e2e"]:
        line["e2e"] = r["e2e"]
    if others:
        line["other_workloads"] = {}
        for name, (w2, bwd, n2, r2) in others.items():
            rf, rt = rooflines(w2, r2, peaks, peak_kind)
            s2 = r2["seg"]
            entry = {"steps": n2, "value": job_value(r2["flops"], world, r2["ms_per_step"]), "unit": UNIT, "backward": bwd,
                     "ms_per_step": r2["ms_per_step"],
                     "segments_ms": {"pool": s2[0], "route": s2[1], "attend": s2[2], **({"attend_bwd": s2[3]} if bwd else {})},
                     "attend_tflops": rf["achieved"], "attend_frac": rf["frac"], "attend_peak": rf["peak"],
                     "attend_frac_of_burst": rf["frac_of_burst"], "routing_gbs": rt["achieved"],
                     "routing_frac": rt["frac"], "selected_pairs": r2["pairs"], "workspace_bytes": r2["workspace_bytes"],
                     "clocks": r2["clocks"]}
            if bwd:
                entry["attend_bwd_tflops"] = 10.0 * w2.head_dim * r2["pairs"] / (s2[3] * 1e-3) / 1e12
            line["other_workloads"][name] = entry
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, args.cpu_budget_s)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
