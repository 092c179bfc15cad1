#!/usr/bin/env python
"""Benchmark of the two-stage verification path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3|cfg4|cfg2] [--impl ours|reference]

A step is one pass of the whole hot path — pyramidsd_verify: the statistics of both stages' rows in one
launch, then stage-1 finalisation, window build and stage-2 finalisation in another — over one batch of
seeded synthetic logits (workload configuration 3, "batched serving", by default: B=64, V=128256, bf16,
K_draft=16, K_qual=8). Metric: verified
positions per second (a position = one row pair actually verified: all B*K_d stage-1 rows plus the
stage-2 rows inside each sequence's window). Prints ONE JSON line on rank 0.

`--impl reference` times the CPU oracle (the only reference this method has) on the host cores.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified positions/s (two-stage verify, B*K*V logits streamed)"
UNIT = "positions/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def workload_from_name(name: str):
    from paper_2510_12966_b200 import workloads
    cfg = int(name.replace("cfg", ""))
    return cfg, workloads.CONFIGS[cfg]


def graph_replay_us_per_step(binding, step, steps_in_graph=16, replays=50):
    """The same calls replayed from a CUDA graph: device time per step with the host's launch path taken out.
    For the single-stream workloads, whose step is a few launches of a few microseconds each."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    try:
        with torch.cuda.stream(side):
            binding.set_stream()
            step(0)
            step(1)
            side.synchronize()
            with torch.cuda.graph(g, stream=side):
                binding.set_stream()
                for i in range(steps_in_graph):
                    step(i)
    finally:
        binding.set_stream()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (replays * steps_in_graph) * 1e3


def positions_per_step(w, out) -> int:
    """Rows actually verified: every stage-1 row, and stage-2 rows inside each sequence's window."""
    al_q, nt_q = out["accept_len_q"], out["next_token_q"]
    n2 = torch.clamp(al_q + (nt_q >= 0).to(torch.int32), max=w.K_q)
    return int(al_q.numel() * w.K_d + int(n2.sum().item()))


def run_ours(args):
    from paper_2510_12966_b200 import binding, workloads
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the verification path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    binding.load_library()
    binding.set_stream()
    schedule = {"fused": binding.TWO_STAGE_FUSED, "separate": binding.TWO_STAGE_SEPARATE, "auto": binding.TWO_STAGE_AUTO,
                "rows": binding.TWO_STAGE_FUSED_ROWS}[args.two_stage]
    cfg, w = workload_from_name(args.workload)
    if args.batch > 0:
        w = dataclasses.replace(w, B=args.batch, name=f"{w.name}[B={args.batch}]")
    if args.tau_q is not None or args.tau_t is not None:
        # other thresholds than the workload's (how the step depends on the share of rejected windows)
        w = dataclasses.replace(w, tau_q=w.tau_q if args.tau_q is None else args.tau_q,
                                tau_t=w.tau_t if args.tau_t is None else args.tau_t, name=f"{w.name}[tau overridden]")
    if args.logits_dtype and args.logits_dtype != w.dtype:
        w = dataclasses.replace(w, dtype=args.logits_dtype, name=f"{w.name}[{args.logits_dtype}]")
    es = 2 if w.dtype == "bf16" else 4

    # Each rank owns its own batch of B sequences (weak scaling; sequences are independent, no collective
    # on the data path). Two distinct rounds alternate so that a step never re-reads a buffer it just used;
    # one round (788 MB for cfg3) already exceeds the 126 MB L2.
    n_bufs = 2
    rounds = [workloads.make_pyramid_inputs(w.B, w.K_d, w.K_q, w.V, w.dtype, 1000 * cfg + 100 * rank + i, w.boost, w.sigma_q,
                                            w.sigma_d, device=dev) for i in range(n_bufs)]
    outs = [{k: torch.empty(w.B, dtype=torch.int32, device=dev)
             for k in ("accept_len_q", "next_token_q", "accept_len", "next_token")} for _ in range(n_bufs)]
    mode, seed = binding.FUZZY, 0
    div_kind = {"js": binding.DIV_JS, "kl": binding.DIV_KL, "tv": binding.DIV_TV}[args.div]

    # every rank's B sequences are a slice of one global batch of world * B: the sequence base keeps each row's
    # random draws those of the global batch
    def step(i):
        zd, zq, zt, tok = rounds[i % n_bufs]
        binding.verify_ex(zd, zq, zt, tok, w.tau_q, w.tau_t, mode, None, seed, 2 * i, seq_index_base=rank * w.B,
                          schedule=schedule, div_kind=div_kind, want_rows=False, want_window=False, out=outs[i % n_bufs])

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = binding.launch_count()
    # The timed region is K steps between a barrier + synchronize on both sides, CUDA events around it. It is
    # taken `regions` times back to back (K steps can be a few milliseconds) and the median region is reported.
    region_ms = []
    for _ in range(args.regions):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record()
        for i in range(args.steps):
            step(args.warmup + i)
        ev1.record()
        barrier()
        region_ms.append(ev0.elapsed_time(ev1))
    launches = (binding.launch_count() - launches0) // args.regions
    clocks = sampler.stop()
    # The same K steps once more with an event pair around every launch, for the per-kernel durations of the
    # roofline. Kept out of the pass above: the event records between launches cost a few microseconds each.
    timed_cap = 4096               # timed launches the library's event timing holds
    ev_steps = min(args.steps, timed_cap // 4)
    binding.kernel_timing_begin()
    for i in range(ev_steps):
        step(args.warmup + i)
    torch.cuda.synchronize()
    ms_rs, n_rs, ms_fin, n_fin = binding.kernel_timing_end()
    status = binding.last_status()
    if status != 0:
        raise SystemExit(f"bench.py: library status {status}")
    graph_us = graph_replay_us_per_step(binding, step) if (world == 1 and w.B <= 4) else None

    # positions and algorithmic bytes of the steps that were timed
    pos_by_buf = [positions_per_step(w, o) for o in outs]
    n_pos = sum(pos_by_buf[(args.warmup + i) % n_bufs] for i in range(args.steps))
    row_bytes = 2 * w.V * es
    # the statistics kernel streams each verified row pair once; the event pass covered the first ev_steps steps
    rs_bytes = sum(pos_by_buf[(args.warmup + i) % n_bufs] for i in range(ev_steps)) * row_bytes
    # statistics launches per step: 1 when one launch covers both stages, 2 when the call runs stage by stage (a
    # finalisation, one or three launches, is timed as one)
    stats_per_step = max(1, round(n_rs / ev_steps))

    # ---- acceptance rates and near ties of the rounds that were timed (one more call per round, with rows) ----
    acc = {"rows_q": 0, "acc_q": 0, "rows_t": 0, "acc_t": 0, "near_q": 0, "near_t": 0}
    for zd, zq, zt, tok in rounds:
        o = binding.verify_ex(zd, zq, zt, tok, w.tau_q, w.tau_t, mode, None, seed, 0, seq_index_base=rank * w.B, schedule=schedule,
                              div_kind=div_kind)
        torch.cuda.synchronize()
        nw = o["n_window"]
        inside = torch.arange(w.K_q, device=dev)[None, :] < nw[:, None]
        acc["rows_q"] += w.B * w.K_d
        acc["acc_q"] += int((o["div_q"] <= w.tau_q).sum())
        acc["rows_t"] += int(nw.sum())
        acc["acc_t"] += int(((o["div_t"] <= w.tau_t) & inside).sum())
        acc["near_q"] += int(((o["div_q"] - w.tau_q).abs() < 1e-4).sum())
        acc["near_t"] += int((((o["div_t"] - w.tau_t).abs() < 1e-4) & inside).sum())

    # ---- end to end through the host-pointer entry point: H2D of the step's inputs + D2H of its results ----
    e2e = None
    if not args.no_e2e:
        zd, zq, zt, tok = [t.cpu().pin_memory() for t in rounds[0]]
        hout = {k: torch.empty(w.B, dtype=torch.int32).pin_memory()
                for k in ("accept_len_q", "next_token_q", "accept_len", "next_token")}
        h2d = sum(t.numel() * t.element_size() for t in (zd, zq, zt, tok))
        d2h = 4 * w.B * 4
        e2e_steps = max(2, min(args.steps, 8))
        for _ in range(2):
            binding.verify_host(zd, zq, zt, tok, w.tau_q, w.tau_t, mode, seed, 0, out=hout)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(e2e_steps):
            binding.verify_host(zd, zq, zt, tok, w.tau_q, w.tau_t, mode, seed, 0, out=hout)
        e1.record()
        barrier()
        ms_e2e = e0.elapsed_time(e1)
        e2e_pos = pos_by_buf[0] * e2e_steps
        e2e = {"ms": ms_e2e, "pos": e2e_pos, "h2d": h2d, "d2h": d2h, "steps": e2e_steps}

    # ---- max over ranks, sum of positions ----
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor(region_ms + [e2e["ms"] if e2e else 0.0], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        region_ms, ms_e2e_max = t[:-1].tolist(), t[-1].item()
        c = torch.tensor([n_pos, e2e["pos"] if e2e else 0, launches], device=dev, dtype=torch.int64)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
        n_pos_all, e2e_pos_all, launches_all = int(c[0]), int(c[1]), int(c[2])
        if e2e:
            e2e["ms"] = ms_e2e_max
    else:
        n_pos_all, e2e_pos_all, launches_all = n_pos, (e2e["pos"] if e2e else 0), launches

    ms_total = statistics.median(region_ms)   # per region: the max over ranks
    if rank == 0:
        peaks, peak_kind = load_peaks()
        value = n_pos_all / (ms_total * 1e-3)
        achieved = rs_bytes / (ms_rs * 1e-3) / 1e9 if ms_rs > 0 else 0.0
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "timed_regions": args.regions, "ms_per_step_min_max": [min(region_ms) / args.steps, max(region_ms) / args.steps],
            "config": {"workload": f"{w.name}: B={w.B} per GPU, V={w.V}, {w.dtype} logits, K_draft={w.K_d}, "
                                   f"K_qual={w.K_q}, tau_q={w.tau_q}, tau_t={w.tau_t}, fuzzy mode, Philox seed 0, two-stage schedule {args.two_stage}"
                                   + {"js": "", "kl": ", divergence KL(large||small) in one pass", "tv": ", divergence total variation"}[args.div],
                       "logits_dtype": w.dtype, "arithmetic": "f32 (logits widened from %s)" % w.dtype,
                       "positions_per_step": n_pos / args.steps,
                       "acceptance": {"beta_qualifier_stage": acc["acc_q"] / max(acc["rows_q"], 1),
                                      "beta_target_stage": acc["acc_t"] / max(acc["rows_t"], 1),
                                      "rows_within_1e-4_of_tau": {"qualifier_stage": acc["near_q"], "target_stage": acc["near_t"]},
                                      "rows": {"qualifier_stage": acc["rows_q"], "target_stage": acc["rows_t"]}},
                       "l2_policy": "inputs larger than L2 (one round = %.0f MB), two rounds alternate" %
                                    ((2 * w.K_d + w.K_q) * w.B * w.V * es / 1e6),
                       "gb_per_s_whole_step": n_pos_all * row_bytes / (ms_total * 1e-3) / 1e9},
            "roofline": {"bound": "hbm", "kernel": "rowstats (per-row softmax/divergence statistics%s)" %
                                                   (", KL in one pass over the logits" if args.div == "kl" else ""),
                         "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                         "bytes_counted": "2*V*s per verified row pair (the call made); the least a two-stage call can "
                                          "read, qualifier rows once, is (2*K_d + K_q)/(2*(K_d + K_q)) of it",
                         "frac_on_fused_minimum_bytes": achieved / peaks["hbm_gbs"] * (2 * w.K_d + w.K_q) / (2.0 * (w.K_d + w.K_q)),
                         "traffic": None, "launches": n_rs, "avg_launch_ms": ms_rs / max(n_rs, 1),
                         "finalize_ms_per_launch": ms_fin / max(n_fin, 1),
                         # statistics time per step of the event pass over the step time of the timed pass
                         "share_of_step": (ms_rs / ev_steps) / (ms_total / args.steps)
                                          if ms_total > 0 else None,
                         "timing": "CUDA events around every launch, in a second pass over the same K steps"},
            "gpu_launches": launches_all, "clocks": clocks,
        }
        # The same kernel against the special-function unit, its first ceiling with bf16 logits: four ex2 per
        # index pair (two per pass; two in all when KL takes one pass), 16 results per clock and SM, 148 SMs at the
        # sampled SM clock.
        n_ex2 = {"js": 4.0, "kl": 2.0, "tv": 3.0}[args.div] * rs_bytes / (2 * es)   # KL in one pass: one ex2 per index and model
        xu_peak = 16.0 * 148 * (clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0) * 1e6
        line["roofline"]["special_function_unit"] = {
            "achieved": n_ex2 / (ms_rs * 1e-3) if ms_rs > 0 else 0.0, "peak": xu_peak, "unit": "ex2/s",
            "frac": (n_ex2 / (ms_rs * 1e-3) / xu_peak) if ms_rs > 0 else 0.0,
            "peak_kind": "16 results/clk/SM (measured) x 148 SMs x sampled SM clock"}
        if graph_us is not None:
            line["config"]["us_per_step_cuda_graph_replay"] = graph_us
        if e2e:
            line["e2e"] = {"value": e2e_pos_all / (e2e["ms"] * 1e-3), "unit": UNIT,
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": e2e["ms"] / e2e["steps"], "steps": e2e["steps"]}
        # Sec. 3.3's throughput model fed with the acceptance rates measured above and assumed model speeds
        b_qd, b_tq = acc["acc_q"] / max(acc["rows_q"], 1), acc["acc_t"] / max(acc["rows_t"], 1)
        line["analytic_model"] = {
            "beta_qd": b_qd, "beta_tq": b_tq, "ell_d": w.K_d, "ell_q": w.K_q,
            "assumed_tokens_per_s": {"draft": args.v_draft, "qualifier": args.v_qual, "target": args.v_target},
            "sd_tokens_per_s": binding.model_sd_throughput(b_tq, w.K_q, args.v_qual, args.v_target),
            "psd_tokens_per_s": binding.model_psd_throughput(b_qd, w.K_d, args.v_draft, args.v_qual, b_tq, w.K_q, args.v_target)}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, rounds, {"js": 0, "tv": 1, "kl": 2}[args.div])
        if world == 1 and args.div == "js" and w.B * (w.K_d + w.K_q) >= 148:
            # beside the line: the same workload with the KL divergence, whose statistics take one pass over the logits
            # (thresholds 2.0 / 1.0, under which about the same rows are accepted as with JS at the workload's own)
            kl_tau = (2.0, 1.0)

            def kl_step(i):
                zd, zq, zt, tok = rounds[i % n_bufs]
                binding.verify_ex(zd, zq, zt, tok, kl_tau[0], kl_tau[1], mode, None, seed, 2 * i, schedule=schedule,
                                  div_kind=binding.DIV_KL, want_rows=False, want_window=False, out=outs[i % n_bufs])
            kl_steps = min(args.steps, 100)
            for i in range(3):
                kl_step(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(kl_steps):
                kl_step(i)
            e1.record()
            torch.cuda.synchronize()
            kl_ms = e0.elapsed_time(e1) / kl_steps
            binding.kernel_timing_begin()
            for i in range(kl_steps):
                kl_step(i)
            torch.cuda.synchronize()
            kl_rs, kl_n, _, _ = binding.kernel_timing_end()
            kl_pos = sum(positions_per_step(w, outs[i % n_bufs]) for i in range(2)) / 2.0
            line["kl_divergence_one_pass"] = {
                "tau_q": kl_tau[0], "tau_t": kl_tau[1], "ms_per_step": kl_ms, "positions_per_s": kl_pos / (kl_ms * 1e-3),
                "rowstats_ms_per_launch": kl_rs / max(kl_n, 1), "rowstats_launches_per_step": kl_n / kl_steps,
                "rowstats_gb_per_s": kl_pos * row_bytes * kl_steps / (kl_rs * 1e-3) / 1e9 if kl_rs > 0 else None,
                # on the bytes of the call made, 2*V*s per verified row pair, as the line's roofline.frac; and on the
                # bytes actually read when one launch walks row triples (the qualifier's rows once)
                "frac_of_hbm_peak_on_call_bytes": (kl_pos * row_bytes * kl_steps / (kl_rs * 1e-3) / 1e9 / peaks["hbm_gbs"]) if kl_rs > 0 else None,
                "frac_of_hbm_peak_on_bytes_read": (kl_pos * row_bytes * kl_steps / (kl_rs * 1e-3) / 1e9 / peaks["hbm_gbs"] *
                                                   ((2 * w.K_d + w.K_q) / (2.0 * (w.K_d + w.K_q))
                                                    if (kl_n == kl_steps and args.two_stage in ("auto", "rows")) else 1.0)) if kl_rs > 0 else None,
                "note": "not the line's metric: div_kind = KL(large||small) instead of the Jensen-Shannon reading of Div"}
        line["traffic_note"] = "roofline.traffic is filled from the ncu capture summarised under profiles/"
        form = ("kl_" if args.div == "kl" else "tv_" if args.div == "tv" else "") + ("pairs" if args.two_stage == "fused" else "rows")
        traffic = read_profile_traffic(w, form) if stats_per_step == 1 else None
        if traffic is not None:
            line["roofline"]["traffic"] = traffic
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_single_stage(args):
    """Config 1: the tiny fp32 single-stage check (B=1, K=4, V=32000). A step = one fuzzy (tau=0.3) and one
    strict pyramidsd_verify_stage call on one round of inputs; 1 MB per step, so this line is a latency figure."""
    from paper_2510_12966_b200 import binding, workloads
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and int(os.environ.get("RANK", "0")) != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the verification path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    binding.load_library()
    binding.set_stream()
    w = workloads.CONFIGS[1]
    rounds = [workloads.workload_inputs(1, i, device=dev) for i in range(64)]
    outs = (torch.empty(w.B, dtype=torch.int32, device=dev), torch.empty(w.B, dtype=torch.int32, device=dev))

    def step(i):
        zs, zl, tok = rounds[i % 64]
        binding.verify_stage(zs, zl, tok, w.tau_q, binding.FUZZY, 0, i, *outs)
        binding.verify_stage(zs, zl, tok, w.tau_q, binding.STRICT, 0, i, *outs)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    launches0 = binding.launch_count()
    region_ms = []
    for _ in range(args.regions):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for i in range(args.steps):
            step(args.warmup + i)
        ev1.record()
        torch.cuda.synchronize()
        region_ms.append(ev0.elapsed_time(ev1))
    ms_total = statistics.median(region_ms)
    launches = (binding.launch_count() - launches0) // args.regions
    clocks = sampler.stop()
    binding.kernel_timing_begin()   # per-kernel durations: a second pass, so that the event records stay out of the step time
    for i in range(args.steps):
        step(args.warmup + i)
    torch.cuda.synchronize()
    ms_rs, n_rs, ms_fin, n_fin = binding.kernel_timing_end()
    graph_us = graph_replay_us_per_step(binding, step, steps_in_graph=64)
    peaks, peak_kind = load_peaks()
    pos = 2 * w.B * w.K_d * args.steps
    row_bytes = 2 * w.V * 4
    achieved = (n_rs * w.B * w.K_d * row_bytes) / (ms_rs * 1e-3) / 1e9 if ms_rs > 0 else 0.0
    print(json.dumps({
        "metric": METRIC, "value": pos / (ms_total * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "timed_regions": args.regions,
        "ms_per_step_min_max": [min(region_ms) / args.steps, max(region_ms) / args.steps],
        "config": {"workload": f"{w.name}: B=1, K=4, V=32000, fp32 logits, one fuzzy (tau=0.3) and one strict call per step, 64 rounds",
                   "l2_policy": "64 rounds of 1 MB stay in L2: this is a latency figure, not a bandwidth one",
                   "us_per_call": ms_total / args.steps / 2 * 1e3, "us_per_call_cuda_graph_replay": graph_us / 2},
        "roofline": {"bound": "hbm", "kernel": "rowstats (4 row pairs per launch: launch-latency-bound)", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                     "traffic": None, "launches": n_rs, "avg_launch_ms": ms_rs / max(n_rs, 1),
                     "finalize_ms_per_launch": ms_fin / max(n_fin, 1)},
        "gpu_launches": launches, "clocks": clocks}))


def run_fused(args):
    """Config 5: the fused LM-head + target verify. A step = one pyramidsd_verify_fused_lmhead call (two GEMM
    sweeps with the statistics in their epilogues, a row reduction, the finalisation). The bound is the
    tensor pipe: achieved = 2 sweeps x 2*M*d*V flops / device time of the sweep kernels."""
    from paper_2510_12966_b200 import binding, workloads
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and int(os.environ.get("RANK", "0")) != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the verification path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    binding.load_library()
    binding.set_stream()
    w = workloads.CONFIGS[5]
    if args.vocab > 0:
        w = dataclasses.replace(w, V=args.vocab, name=f"{w.name}[V={args.vocab}]")
    M = w.B * w.K_d
    h, w_t, z_q, tok = workloads.make_fused_inputs(w.B, w.K_d, w.V, w.d_model, seed=5000, sigma_q=w.sigma_q, device=dev)
    hs = [h, h.clone()]          # the weight (1.05 GB) stays resident like a model's; activations alternate
    zs = [z_q, z_q.clone()]

    kl = args.lmhead_div == "kl"
    div_kind = binding.DIV_KL if kl else binding.DIV_JS
    lm_mode = binding.ASSISTED if args.lmhead_mode == "assisted" else binding.FUZZY
    if args.lmhead_tau is not None:
        w = dataclasses.replace(w, tau_t=args.lmhead_tau)

    def step(i):
        return binding.verify_fused_lmhead(hs[i % 2], w_t, zs[i % 2], tok, w.tau_t, lm_mode, 0, i, want_rows=False,
                                           div_kind=div_kind)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    launches0 = binding.launch_count()
    region_ms = []
    for _ in range(args.regions):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for i in range(args.steps):
            out = step(args.warmup + i)
        ev1.record()
        torch.cuda.synchronize()
        region_ms.append(ev0.elapsed_time(ev1))
    ms_total = statistics.median(region_ms)
    launches = (binding.launch_count() - launches0) // args.regions
    clocks = sampler.stop()
    binding.kernel_timing_begin()   # per-kernel durations: a second pass, so that the event records stay out of the step time
    for i in range(args.steps):
        out = step(args.warmup + i)
    torch.cuda.synchronize()
    ms_sweeps, n_sw, ms_fin, n_fin = binding.kernel_timing_end()
    if binding.last_status() != 0:
        raise SystemExit("bench.py: library status != 0")
    peaks, peak_kind = load_peaks()
    # Jensen-Shannon runs the GEMM twice; KL once, plus a second sweep only when a rejected row needs residual masses:
    # never in the assisted mode, and not in the threshold mode while every position is accepted
    one_sweep = kl and (lm_mode == binding.ASSISTED or bool((out["accept_len"] == w.K_d).all().item()))
    sweeps = 1 if one_sweep else 2
    flops = sweeps * 2.0 * M * w.d_model * w.V
    achieved = flops * n_sw / (ms_sweeps * 1e-3) / 1e12 if ms_sweeps > 0 else 0.0
    # end to end: activations and qualifier logits come from pinned host memory every step, results go back
    e2e = None
    if not args.no_e2e:
        hh, zh, th = h.cpu().pin_memory(), z_q.cpu().pin_memory(), tok.cpu().pin_memory()
        res = torch.empty((2, w.B), dtype=torch.int32).pin_memory()
        n = max(2, min(args.steps, 8))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for it in range(n + 2):
            if it == 2:
                torch.cuda.synchronize()
                e0.record()
            hs[0].copy_(hh, non_blocking=True); zs[0].copy_(zh, non_blocking=True); tok.copy_(th, non_blocking=True)
            o = binding.verify_fused_lmhead(hs[0], w_t, zs[0], tok, w.tau_t, lm_mode, 0, it, want_rows=False, div_kind=div_kind)
            res[0].copy_(o["accept_len"], non_blocking=True); res[1].copy_(o["next_token"], non_blocking=True)
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        e2e = {"value": M * n / (e0.elapsed_time(e1) * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": hh.numel() * 2 + zh.numel() * 2 + th.numel() * 4, "d2h_bytes_per_step": 8 * w.B,
               "ms_per_step": e0.elapsed_time(e1) / n, "steps": n}
    # The sweeps run back to back for the whole timed region: when the power cap held the clocks down during it,
    # the denominator is the sustained GEMM figure (measured the same way), else the burst one.
    capped = "sw_power_cap" in (clocks.get("reasons") or []) and "bf16_tflops_sustained" in peaks
    tensor_peak = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
    tensor_kind = f"of {peak_kind} ({'sustained: sw_power_cap active during the timed region' if capped else 'burst'})"
    line = {
        "metric": METRIC, "value": M * args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 x bf16 -> f32 (GEMM), f32 (epilogue)", "data": "synthetic",
        "timed_regions": args.regions, "ms_per_step_min_max": [min(region_ms) / args.steps, max(region_ms) / args.steps],
        "config": {"workload": f"{w.name}: B={w.B}, K={w.K_d} (M={M}), d={w.d_model}, V={w.V}, LM-head weight bf16 [V, d], "
                               f"qualifier logits bf16, tau_t={w.tau_t}, {args.lmhead_mode} mode, Philox seed 0, divergence {'KL(large||small)' if kl else 'Jensen-Shannon'}, {sweeps} GEMM sweep(s)",
                   "all_positions_accepted": bool((out["accept_len"] == w.K_d).all().item()),
                   "l2_policy": "the weight (1.05 GB) is larger than L2 and is streamed twice per step"},
        "roofline": {"bound": "tensor", "kernel": "lmhead_sweep (two tcgen05 GEMM sweeps + row reduction)",
                     "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s", "frac": achieved / tensor_peak,
                     "frac_of_burst": achieved / peaks["bf16_tflops"],
                     "flops_counted": "the GEMM sweeps executed (%d); the method needs one h x W^T" % sweeps,
                     "achieved_on_one_gemm": achieved / sweeps, "frac_on_one_gemm": achieved / sweeps / tensor_peak,
                     "peak_kind": tensor_kind, "traffic": None, "launches": n_sw,
                     "avg_launch_ms": ms_sweeps / max(n_sw, 1), "finalize_ms_per_launch": ms_fin / max(n_fin, 1),
                     "weight_gb_per_s": sweeps * w.V * w.d_model * 2 * n_sw / (ms_sweeps * 1e-3) / 1e9 if ms_sweeps > 0 else 0.0},
        "gpu_launches": launches, "clocks": clocks,
    }
    if e2e:
        line["e2e"] = e2e
    if not args.no_cpu_baseline:
        import oracle
        oracle.build()
        cores = os.cpu_count() or 1
        nb = 2                     # sequences in the sample (16 rows, full vocabulary)
        t0 = time.perf_counter()
        zl = oracle.lmhead_logits(workloads.to_host_bits(h[:nb * w.K_d]), workloads.to_host_bits(w_t.T.contiguous()),
                                  n_threads=cores).reshape(nb, w.K_d, w.V)
        oracle.verify_stage_mixed(workloads.to_host_bits(z_q[:nb]), zl, tok[:nb].cpu().numpy(), np.float32(w.tau_t),
                                  oracle.FUZZY, 0, 0, n_threads=cores)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": nb * w.K_d / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {nb} sequences ({nb * w.K_d} rows, full vocabulary: double-precision GEMM + stage), {dt:.1f} s wall"}
    print(json.dumps(line))


def read_profile_traffic(w, form):
    """DRAM bytes per full-size rowstats launch (row-pair or row-triple form) from the committed ncu summary, if present."""
    path = os.path.join(ROOT, "profiles", "rowstats_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        t = json.load(f)
    per_row = t.get("dram_bytes_per_row", {}).get(f"V{w.V}_{w.dtype}_{form}")
    return None if per_row is None else per_row * w.B * (w.K_d + w.K_q)   # rows of the fused statistics launch


def cpu_baseline(w, rounds, div_kind=0):
    """The CPU oracle, as it stands, on a bounded sample: the resident rounds of the workload (two rounds
    of B sequences each), one oracle call per round on all host cores."""
    import oracle
    from paper_2510_12966_b200 import workloads
    oracle.build()
    cores = os.cpu_count() or 1
    pos, dt = 0, 0.0
    for r in rounds:
        zd, zq, zt, tok = [workloads.to_host_bits(t) for t in r]
        t0 = time.perf_counter()
        out = oracle.verify(zd, zq, zt, tok, np.float32(w.tau_q), np.float32(w.tau_t), oracle.FUZZY, 0, 0, div_kind=div_kind,
                            n_threads=cores)
        dt += time.perf_counter() - t0
        n2 = np.minimum(w.K_q, out["accept_len_q"] + (out["next_token_q"] >= 0))
        pos += w.B * w.K_d + int(n2.sum())
    # the same oracle on one core, on the first sequences of the first round
    nb = min(4, w.B)
    zd, zq, zt, tok = [workloads.to_host_bits(t[:nb]) for t in rounds[0]]
    t0 = time.perf_counter()
    out = oracle.verify(zd, zq, zt, tok, np.float32(w.tau_q), np.float32(w.tau_t), oracle.FUZZY, 0, 0, div_kind=div_kind, n_threads=1)
    dt1 = time.perf_counter() - t0
    pos1 = nb * w.K_d + int(np.minimum(w.K_q, out["accept_len_q"] + (out["next_token_q"] >= 0)).sum())
    return {"value": pos / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(rounds)} rounds of {w.name} ({w.B} sequences each, {pos} positions, {dt:.2f} s wall, "
                      f"about {dt * cores:.0f} core-seconds)",
            "one_core": {"value": pos1 / dt1, "unit": UNIT, "cores": 1,
                         "sample": f"first {nb} sequences of one round ({pos1} positions, {dt1:.2f} s)"}}


def run_reference(args):
    """The reference arm: the CPU oracle timed on the host cores (this method has no other reference)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2510_12966_b200 import workloads
    oracle.build()
    cfg, w = workload_from_name(args.workload)
    if args.tau_q is not None or args.tau_t is not None:
        w = dataclasses.replace(w, tau_q=w.tau_q if args.tau_q is None else args.tau_q,
                                tau_t=w.tau_t if args.tau_t is None else args.tau_t, name=f"{w.name}[tau overridden]")
    seqs = args.cpu_seqs if args.cpu_seqs > 0 else w.B
    cores = os.cpu_count() or 1
    rounds = [workloads.workload_inputs(cfg, i, device="cpu", B=seqs) for i in range(2)]
    hosts = [[workloads.to_host_bits(t) for t in r] for r in rounds]

    def step(i):
        zd, zq, zt, tok = hosts[i % 2]
        out = oracle.verify(zd, zq, zt, tok, np.float32(w.tau_q), np.float32(w.tau_t), oracle.FUZZY, 0, 2 * i,
                            div_kind={"js": 0, "tv": 1, "kl": 2}[args.div], n_threads=cores)
        n2 = np.minimum(w.K_q, out["accept_len_q"] + (out["next_token_q"] >= 0))
        return seqs * w.K_d + int(n2.sum())

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    pos = sum(step(args.warmup + i) for i in range(args.steps))
    dt = time.perf_counter() - t0
    value = pos / dt
    sample = f"{seqs} sequences per step of {w.name} (B={w.B} in the full workload), {cores} threads"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: V={w.V}, {w.dtype} logits, K_draft={w.K_d}, K_qual={w.K_q}, "
                               f"tau_q={w.tau_q}, tau_t={w.tau_t}, fuzzy mode, Philox seed 0; {sample}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)    # x 5 regions: ~0.25 s of timed work, long enough for the clock sampler
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="cfg3", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--logits-dtype", choices=["bf16", "f32"], default=None, help="override the workload's logits dtype (cfg4's fp32 run)")
    ap.add_argument("--cpu-seqs", type=int, default=0, help="sequences per step of the CPU-oracle reference arm (0: the workload's B)")
    ap.add_argument("--regions", type=int, default=5, help="the K-step timed region is taken this many times; the median is reported")
    ap.add_argument("--v-draft", type=float, default=900.0, help="assumed draft-model speed (tokens/s) for the analytic model line")
    ap.add_argument("--v-qual", type=float, default=400.0, help="assumed qualifier-model speed (tokens/s)")
    ap.add_argument("--v-target", type=float, default=150.0, help="assumed target-model speed (tokens/s)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size B (small profiling cases)")
    ap.add_argument("--vocab", type=int, default=0, help="override the vocabulary size V of cfg5 (small profiling cases)")
    ap.add_argument("--two-stage", choices=["fused", "separate", "auto", "rows"], default="auto",
                    help="schedule of the two stages (same results): one statistics launch for both (row pairs, or row "
                         "triples with `rows`), stage by stage, or the library's per-call choice (its default)")
    ap.add_argument("--lmhead-div", choices=["js", "kl"], default="js", help="divergence of the fused LM-head workload (cfg5)")
    ap.add_argument("--lmhead-mode", choices=["fuzzy", "assisted"], default="fuzzy", help="acceptance mode of cfg5")
    ap.add_argument("--lmhead-tau", type=float, default=None, help="threshold of cfg5 (default: the workload's)")
    ap.add_argument("--div", choices=["js", "kl", "tv"], default="js",
                    help="divergence of cfg2-cfg4: Jensen-Shannon (the reading taken for the paper's Div), KL(large||small), "
                         "whose terms separate and whose statistics take one pass over the logits, or total variation "
                         "(three ex2 per index pair instead of four)")
    ap.add_argument("--tau-q", type=float, default=None, help="override the qualifier-stage threshold of cfg2-cfg4")
    ap.add_argument("--tau-t", type=float, default=None, help="override the target-stage threshold of cfg2-cfg4")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "cfg5":
        run_fused(args)
    elif args.workload == "cfg1":
        run_single_stage(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
