#!/usr/bin/env python
"""Benchmark of the TreeSpark hot path: tree rounds per second on one B200 (or N independent
batch shards on N GPUs), with the roofline of the dominant kernel and the CPU oracle timed beside it.

A step is one round = ts_expand_tree (all scoring levels, survival/expansion, masks) followed by
ts_verify_tree (all target rows, the walk, the bonus token) for the whole batch.  Inputs are seeded
and synthetic (paper_2609_22098_b200.synth); several distinct input sets, together far larger than
L2, are rotated so that base logits and target logits never hit in L2 across rounds while the
Markov-head factors legitimately stay resident.  The timed rounds are replays of CUDA graphs, one per input
set, each holding every launch of one round as the library issues it (--no-graph times the direct calls; the
per-kernel figures always come from direct, instrumented calls).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload serve32] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_22098_b200 import shard, synth  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="serve32", choices=list(synth.WORKLOADS))
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--T", type=float, default=None)
    ap.add_argument("--theta", type=float, default=None)
    ap.add_argument("--sets", type=int, default=4, help="distinct input sets rotated through")
    ap.add_argument("--seed", type=int, default=2609)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--test-mode", type=int, default=0, help="library test switches (TS_TEST_*), e.g. 64 = every level of the expansion inside one cooperative launch")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-edge-stat", action="store_true", help="do not emit per-edge statistics")
    ap.add_argument("--no-graph", action="store_true",
                    help="time direct calls instead of replays of one CUDA graph per input set (the default captures "
                         "each set's round, all launches of expand + verify, once)")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def wait_first(self, limit=2.0):
        """nvidia-smi takes a moment to start: wait (bounded) for its first line."""
        t0 = time.monotonic()
        while self.proc and not self.lines and time.monotonic() - t0 < limit:
            time.sleep(0.01)

    def stop(self, t_lo=None, t_hi=None):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [ln for (t, ln) in self.lines if t_lo is not None and t_lo <= t <= t_hi]
        # samples inside the timed region when it is long enough to hold some, else every sample since the
        # warm-up began (the GPU runs the same rounds from there to the end of the timed region)
        for ln in (inside if inside else [ln for (_, ln) in self.lines]):
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "samples_in_timed_region": len(inside), "reasons": sorted(reasons)}


class InputSet:
    """One seeded instance of the workload on the device: base logits, anchors, prices, and (after
    the first untimed pass) the target logits of its tree."""

    def __init__(self, wl, seed, B, theta, A, W, device):
        Ufull = synth.make_base_logits(wl, seed + 2, device, B=B)
        self.Ufull = Ufull
        self.U = Ufull[:, :wl.D].contiguous()
        self.anchor = synth.make_anchor(wl, seed + 3, B=B).to(device)
        self.theta = synth.make_theta(wl, B=B, theta=theta).to(device)
        self.round_seed = seed + 7
        self.A, self.W = A, W
        self.Z = self.zoff = None

    def make_targets(self, wl, seed, tree):
        self.Z, self.zoff = synth.make_target_logits(wl, seed + 5, self.Ufull, self.A, self.W, self.anchor,
                                                     tree["n_nodes"], tree["tok"], tree["depth"], tree["node_hash"])
        self.Ufull = None  # only needed to synthesise Z


def tree_stats(wl, tree, verdict):
    """Algorithmic units of one round, from its outputs (host side, untimed)."""
    n = tree["n_nodes"].long().cpu()
    B, N = tree["tok"].shape
    lse = tree["node_lseT"].cpu()
    depth = torch.cat([torch.zeros(B, 1, dtype=torch.int32), tree["depth"].cpu()], 1)
    valid = torch.arange(N + 1).unsqueeze(0) <= n.unsqueeze(1)
    scored = valid & ~torch.isnan(lse)
    parents = int(scored.sum())
    urows = 0
    per_level = []
    for d in range(wl.D):
        act = int(((scored & (depth == d)).sum(1) > 0).sum())
        urows += act
        per_level.append(int((scored & (depth == d)).sum()))
    return dict(nodes=int(n.sum()), parents=parents, u_rows=urows, z_rows=int((n + 1).sum()),
                levels_used=sum(1 for p in per_level if p > 0), parents_per_level=per_level,
                acc=int(verdict["acc_len"].sum()), walk_rows=int((verdict["acc_len"].long() + 1).sum()),
                walk_passes=int(((verdict["flags"].long() >> 8) & 0xFFFF).sum()),
                # a request's reductions follow one another, one grid step each: the longest chain bounds the walk's steps
                walk_chain=int(((verdict["flags"].long() >> 8) & 0xFFFF).max()))


def snapshot(tree, verdict):
    """The defined part of a round's outputs (entries past n_nodes / acc_len are undefined)."""
    n = tree["n_nodes"].long()
    N = tree["tok"].shape[1]
    valid = torch.arange(N, device=n.device).unsqueeze(0) < n.unsqueeze(1)
    L = verdict["acc_len"].long()
    va = torch.arange(verdict["acc_tok"].shape[1], device=n.device).unsqueeze(0) < L.unsqueeze(1)
    return (torch.where(valid, tree["tok"], -1), torch.where(valid, tree["parent"], -2), tree["n_nodes"].clone(),
            verdict["acc_len"].clone(), torch.where(va, verdict["acc_tok"], -1), verdict["bonus_tok"].clone())


def workload_theta(args, wl, B):
    """The stopping threshold of the run: --theta if given; for the load sweep the seeded monotone
    load -> theta schedule at this batch size (the chain sentinel at the largest); the workload's own otherwise."""
    if args.theta is not None:
        return args.theta
    if wl.name == "sweep" and B in synth.SWEEP_BATCHES:
        return synth.sweep_theta(B, seed=args.seed)
    return wl.theta


def run_ours(args, rank, world, device):
    from paper_2609_22098_b200.binding import TreeSpark
    wl = synth.WORKLOADS[args.workload]
    B = args.batch or wl.B
    T = wl.temps[-1] if args.T is None else args.T
    theta = workload_theta(args, wl, B)
    es = 2 if wl.dtype == "bf16" else 4
    seed = shard.shard_seed(args.seed, rank)
    table = synth.make_calibration_table(wl, args.seed + 4, "fit")
    A, W = synth.make_head(wl, args.seed + 1, device)
    ts = TreeSpark(wl.V, wl.D, wl.r, wl.K, wl.Nmax, B, dtype=wl.torch_dtype, calib_mode=wl.calib_mode,
                   calib_table=table, device=device, test_mode=args.test_mode)
    sets = [InputSet(wl, seed + 100 * i, B, theta, A, W, device) for i in range(args.sets)]
    tree = ts.alloc_tree(B)
    verdict = ts.alloc_verdict(B)
    edge = not args.no_edge_stat

    # ---- pass 1 (untimed): trees -> target logits -> reference outputs of every set -------------
    stats, ref_out = [], []
    for s in sets:
        ts.expand_tree(s.U, A, W, s.anchor, s.theta, T, s.round_seed, out=tree)
        torch.cuda.synchronize()
        s.make_targets(wl, seed, tree)
        ts.verify_tree(s.U, A, W, s.Z, s.zoff, s.anchor, tree, T, s.round_seed, out=verdict, edge_stat=edge)
        torch.cuda.synchronize()
        assert int(tree["status"].abs().max()) == 0 and int(verdict["status"].abs().max()) == 0, "device status"
        stats.append(tree_stats(wl, tree, verdict))
        ref_out.append(snapshot(tree, verdict))

    def direct_round(i):
        s = sets[i % len(sets)]
        ts.expand_tree(s.U, A, W, s.anchor, s.theta, T, s.round_seed, out=tree)
        ts.verify_tree(s.U, A, W, s.Z, s.zoff, s.anchor, tree, T, s.round_seed, out=verdict, edge_stat=edge)

    # --graph: the same launches, recorded once per input set and replayed (the calls allocate nothing and
    # never synchronise, so a round is capturable as it stands)
    graphs, launches_per_round, graph_note = [], None, "direct calls"
    if not args.no_graph:
        try:
            ts.profile_read(reset=True)
            cap_stream = torch.cuda.Stream()
            cap_stream.wait_stream(torch.cuda.current_stream())
            for i in range(len(sets)):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=cap_stream):
                    direct_round(i)
                graphs.append(g)
            torch.cuda.current_stream().wait_stream(cap_stream)
            launches_per_round = sum(c for _, c in ts.profile_read(reset=True).values()) / len(sets)
            graph_note = "CUDA graph replay, one graph per input set"
        except Exception as e:   # capture refused: time direct calls and say so
            graphs, graph_note = [], f"direct calls (graph capture failed: {type(e).__name__})"
            torch.cuda.synchronize()

    def one_round(i):
        if graphs:
            graphs[i % len(graphs)].replay()
        else:
            direct_round(i)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    # ---- timed region -----------------------------------------------------------------------
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    sampler.wait_first()
    for i in range(args.warmup):
        one_round(i)
    ts.profile_read(reset=True)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_lo = time.monotonic()
    e0.record()
    for i in range(args.steps):
        one_round(args.warmup + i)
    e1.record()
    barrier()
    clocks = sampler.stop(t_lo, time.monotonic())
    total_ms = e0.elapsed_time(e1)
    launches = sum(c for _, c in ts.profile_read(reset=True).values())
    if graphs:
        launches = int(round(launches_per_round * args.steps))   # replayed launches are not seen by the library's counter
    last = (args.warmup + args.steps - 1) % len(sets)
    same = all(bool(torch.equal(a, b)) for a, b in zip(ref_out[last], snapshot(tree, verdict)))
    total_ms = shard.max_over_ranks(total_ms, device)   # the slowest rank's device time
    ms_per_step = total_ms / args.steps

    # ---- per-kernel device times (separate, instrumented loop; not the headline number) ----------
    ts.profile_enable(args.steps * (3 * wl.D + 8))
    torch.cuda.synchronize()
    for i in range(args.steps):
        direct_round(args.warmup + i)
    prof = ts.profile_read(reset=True)
    ts.profile_enable(0)
    kern = {k: {"ms_per_round": v[0] / args.steps, "launches_per_round": v[1] / args.steps} for k, v in prof.items() if v[1]}
    tot_kernel_ms = sum(v["ms_per_round"] for v in kern.values()) or 1.0
    for v in kern.values():
        v["share"] = v["ms_per_round"] / tot_kernel_ms

    # ---- algorithmic bytes ---------------------------------------------------------------------
    used = [stats[(args.warmup + i) % len(sets)] for i in range(args.steps)]
    mean = lambda k: sum(u[k] for u in used) / len(used)
    row_b = wl.V * es
    w_b = wl.r * wl.V * es
    # scoring: every needed base-logit row once, the head rows, and W once per round (19 MB: it stays in the 126 MB
    # L2 after the first level; the per-level figure is printed beside it as `alg_bytes_per_round_w_every_level`)
    bytes_score = mean("u_rows") * row_b + w_b + mean("parents") * wl.r * es
    bytes_score_w_levels = mean("u_rows") * row_b + mean("levels_used") * w_b + mean("parents") * wl.r * es
    bytes_zrows = mean("z_rows") * row_b
    bytes_round_all = mean("u_rows") * row_b + w_b + mean("parents") * wl.r * es + bytes_zrows
    bytes_round_min = mean("u_rows") * row_b + w_b + mean("parents") * wl.r * es + mean("walk_rows") * row_b
    peak, peak_src = measured_peak()
    dom = max(kern, key=lambda k: kern[k]["ms_per_round"]) if kern else None
    # walk: every residual reduction streams one target row and (recomputing the proposal) one base row;
    # its range of W is staged once per launch
    bytes_walk = mean("walk_passes") * 2 * row_b + w_b
    alg = {"score_tile": bytes_score, "expand_persistent": bytes_score, "zrow_stats": bytes_zrows, "verify_walk": bytes_walk}
    # DRAM bytes of the dominant kernel from a committed ncu capture of one round of this workload
    # (per launch: the round's bytes over the round's launches), null where none was captured
    traffic, traffic_src = None, None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if dom and os.path.exists(tpath):
        try:
            ent = json.load(open(tpath)).get(args.workload, {}).get(dom)
            if ent:
                traffic = ent["dram_bytes_per_round"] / ent["launches_per_round"]
                traffic_src = ent.get("source")
        except Exception:
            traffic = None
    roofline = None
    if dom:
        per_launch_ms = kern[dom]["ms_per_round"] / max(kern[dom]["launches_per_round"], 1e-9)
        a_bytes = alg.get(dom)
        achieved = (a_bytes / (kern[dom]["ms_per_round"] * 1e-3) / 1e9) if a_bytes else None
        roofline = {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": (achieved / peak) if achieved else None, "peak_source": f"of {peak_src}",
                    "traffic": traffic, "traffic_source": traffic_src,
                    "alg_bytes_per_launch": (a_bytes / max(kern[dom]["launches_per_round"], 1e-9)) if a_bytes else None,
                    "alg_bytes_per_round": a_bytes, "ms_per_launch": per_launch_ms,
                    "launches_per_round": kern[dom]["launches_per_round"], "share_of_kernel_time": kern[dom]["share"]}
        if dom in ("score_tile", "expand_persistent"):
            roofline["alg_bytes_per_round_w_every_level"] = bytes_score_w_levels
    sec = ms_per_step * 1e-3
    round_hbm = {"alg_bytes_all_rows": bytes_round_all, "alg_bytes_walk_rows_only": bytes_round_min,
                 "achieved_gbs": bytes_round_all / sec / 1e9, "frac_of_measured": bytes_round_all / sec / 1e9 / peak,
                 "frac_of_nominal_8TBs": bytes_round_all / sec / 1e9 / NOMINAL_HBM_GBS,
                 "edge_stat_emitted": edge}

    # ---- end to end through the host-buffer API ----------------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, ts, wl, sets[:2], A, W, T, B, world, device, barrier)

    out = {
        "metric": "tree_rounds_per_s", "value": world * 1e3 / ms_per_step, "unit": "rounds/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32" if wl.dtype == "f32" else "bf16 in, f32 accumulate",
        "data": "synthetic",
        "config": {"workload": f"{wl.name}: batch {B}, V={wl.V}, D={wl.D}, r={wl.r}, K={wl.K}, Nmax={wl.Nmax}, "
                               f"theta={theta}, T={T}, {wl.dtype} U/A/W/Z", "l2": f"{args.sets} rotating input sets, "
                               f"{sum(s.U.numel() * es + s.Z.numel() * es for s in sets) / 1e6:.0f} MB of U+Z > 126 MB L2",
                   "parallelism": f"batch shards x{world}, no collective",
                   "launch": graph_note},
        "parents_scored_per_s": world * mean("parents") / sec, "nodes_per_s": world * mean("nodes") / sec,
        "detail": {"mean_nodes_per_tree": mean("nodes") / B, "mean_parents_per_round": mean("parents"),
                   "mean_accepted_len": mean("acc") / B, "mean_z_rows": mean("z_rows"),
                   "mean_walk_reductions": mean("walk_passes"), "mean_longest_walk_chain": mean("walk_chain"),
                   "launches_per_round": launches / max(args.steps, 1),
                   "parents_per_level": used[0]["parents_per_level"], "outputs_reproduced": same},
        "clocks": clocks, "gpu_launches": launches, "kernels": kern,
        # the round's time in SM cycles (time x median SM clock under load): comparable across runs whose clocks differ
        "mcycles_per_step": (ms_per_step * 1e-3 * clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
        # the per-kernel milliseconds come from a separate loop with an event pair around every launch (no chaining
        # of launches there): multiply them by this factor to read them as parts of the timed round
        "kernels_chained_scale": ms_per_step / tot_kernel_ms,
        "roofline": roofline, "round_hbm": round_hbm,
        "e2e": e2e,
    }
    if rank == 0 and not args.no_cpu and world == 1:
        out["cpu_baseline"] = cpu_baseline(wl, table, sets[0], A, W, T, B)
    return out


def short_side_run(args, device, workload, steps=200):
    """Rounds/s of another configuration, timed the same way in a short run (context beside the headline
    workload: the single-request decode shape)."""
    import copy
    a2 = copy.copy(args)
    a2.workload, a2.steps, a2.warmup, a2.batch, a2.T, a2.theta = workload, steps, 5, None, None, None
    a2.no_e2e, a2.no_cpu = True, True
    r = run_ours(a2, 0, 1, device)
    return {"workload": r["config"]["workload"], "value": r["value"], "unit": r["unit"], "ms_per_step": r["ms_per_step"],
            "steps": steps, "parents_scored_per_s": r["parents_scored_per_s"], "nodes_per_s": r["nodes_per_s"],
            "detail": r["detail"]}


def allocate_side_run(args, device, steps=200):
    """Device time of ts_allocate_budget (batch-wide node budget, Section 4) on the headline batch: trees
    grown under a low price, then cut to half their nodes.  Every timed call starts from the same trees
    (restored outside the timed events).  The oracle's allocation is timed beside it on the host."""
    from oracle import allocate as orc_alloc
    from paper_2609_22098_b200.binding import TreeSpark
    wl = synth.WORKLOADS["serve32"]
    B, T = wl.B, wl.temps[-1]
    table = synth.make_calibration_table(wl, args.seed + 4, "fit")
    A, W = synth.make_head(wl, args.seed + 1, device)
    ts = TreeSpark(wl.V, wl.D, wl.r, wl.K, wl.Nmax, B, dtype=wl.torch_dtype, calib_mode=wl.calib_mode,
                   calib_table=table, device=device)
    s = InputSet(wl, args.seed + 900, B, 0.02, A, W, device)
    grown = ts.expand_tree(s.U, A, W, s.anchor, s.theta, T, s.round_seed)
    torch.cuda.synchronize()
    total = int(grown["n_nodes"].sum())
    budget = total // 2
    tree = {k: v.clone() for k, v in grown.items()}
    price = torch.zeros(4, dtype=torch.float32, device=device)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i in range(5 + steps):
        for k in tree:
            tree[k].copy_(grown[k])
        if i >= 5:
            ev[i - 5][0].record()
        ts.allocate_budget(tree, budget, price)
        if i >= 5:
            ev[i - 5][1].record()
    torch.cuda.synchronize()
    us = sorted(a.elapsed_time(b) * 1e3 for a, b in ev)
    kept = int(tree["n_nodes"].sum())
    g = {k: v.cpu() for k, v in grown.items()}
    t0 = time.perf_counter()
    keep, _ = orc_alloc.water_fill(g["n_nodes"].numpy(), g["logkey"].numpy(), g["pop_rank"].numpy(), budget)
    t_cpu = time.perf_counter() - t0
    words = (wl.Nmax + 63) // 64
    node_bytes = 9 * 4 + 8 + 4 + 8 * words          # per-node arrays read and written by the cut
    alg = total * 4 + total * 4 + (total + kept) * node_bytes
    return {"workload": f"serve32 trees grown at theta=0.02 ({total} nodes in {B} trees), budget {budget}",
            "us_per_call_median": us[len(us) // 2], "us_per_call_mean": sum(us) / len(us), "calls": steps,
            "kernels_per_call": 2, "nodes_kept": kept, "matches_oracle_sizes": tree["n_nodes"].cpu().tolist() == list(keep),
            "alg_bytes_per_call": alg, "bound": "launch latency (two small kernels; the bytes are noise)",
            "oracle_water_fill_ms": t_cpu * 1e3}


def calibrate_side_run(args, device, steps=200):
    """Device time of the calibration-statistics calls (Section 3.4) on the headline batch: one
    ts_calib_accumulate per verified round, and one ts_calib_refit over the accumulated cells."""
    from oracle import calibrate as orc_cal
    from paper_2609_22098_b200.binding import TreeSpark
    wl = synth.WORKLOADS["serve32"]
    B, T = wl.B, wl.temps[-1]
    table = synth.make_calibration_table(wl, args.seed + 4, "fit")
    A, W = synth.make_head(wl, args.seed + 1, device)
    ts = TreeSpark(wl.V, wl.D, wl.r, wl.K, wl.Nmax, B, dtype=wl.torch_dtype, calib_mode=wl.calib_mode,
                   calib_table=table, device=device)
    s = InputSet(wl, args.seed + 950, B, wl.theta, A, W, device)
    tree = ts.expand_tree(s.U, A, W, s.anchor, s.theta, T, s.round_seed)
    torch.cuda.synchronize()
    s.make_targets(wl, args.seed, tree)
    verdict = ts.verify_tree(s.U, A, W, s.Z, s.zoff, s.anchor, tree, T, s.round_seed)
    stats = ts.calib_new_stats()
    out_table = torch.empty(wl.D, 16, dtype=torch.float32, device=device)
    out_platt = torch.empty(4, dtype=torch.float64, device=device)

    def timed(fn):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(5 + steps):
            if i >= 5:
                ev[i - 5][0].record()
            fn()
            if i >= 5:
                ev[i - 5][1].record()
        torch.cuda.synchronize()
        us = sorted(a.elapsed_time(b) * 1e3 for a, b in ev)
        return us[len(us) // 2]

    att = ts.emit_attention_inputs(s.anchor, tree)
    att_us = timed(lambda: ts.emit_attention_inputs(s.anchor, tree, out=att))
    acc_us = timed(lambda: ts.calib_accumulate(tree, verdict, stats))
    fit_us = timed(lambda: ts.calib_refit(stats, 1, 4, None, out_table, out_platt))
    edges = int(tree["n_nodes"].sum())
    g = {k: v.cpu() for k, v in tree.items()}
    v = {k: t.cpu() for k, t in verdict.items()}
    ref = orc_cal.new_stats(wl.D)
    t0 = time.perf_counter()
    for b in range(B):
        orc_cal.accumulate(ref, wl.D, -10.0, 10.0, int(g["n_nodes"][b]), g["parent"][b].numpy(), g["depth"][b].numpy(),
                           g["q0"][b].numpy(), v["edge_stat"][b].numpy(), int(v["acc_len"][b]), v["acc_node"][b].numpy())
    t_cpu = time.perf_counter() - t0
    calls = 2 * (5 + steps)   # the same round was added this many times
    same = bool((stats.cpu().numpy()[..., :2] == ref[..., :2] * (calls // 2)).all())
    return {"workload": f"serve32 round ({edges} edges in {B} trees)", "accumulate_us_median": acc_us,
            "refit_us_median": fit_us, "platt": out_platt.cpu().tolist(),
            "counts_and_label_sums_equal_oracle": same, "oracle_accumulate_ms": t_cpu * 1e3,
            "attention_inputs_us_median": att_us,
            "attention_inputs_bytes": int(sum(t.numel() * t.element_size() for t in att.values())),
            "bound": "launch latency (one small kernel each)"}


def run_e2e(args, ts, wl, sets, A, W, T, B, world, device, barrier):
    """Same metric through the host-buffer API: every step copies that step's inputs (base logits,
    anchors, prices, target logits) from pinned host memory and reads the round's results back."""
    from paper_2609_22098_b200.binding import HostRound
    host = [HostRound.pin_inputs(s.U, s.anchor, s.theta, s.Z, s.zoff) for s in sets]
    hr = HostRound(ts, B, max(int(h["Z"].shape[0]) for h in host))
    steps = min(args.steps, 20)
    for i in range(2):
        hr.run(host[i % len(host)], A, W, T, sets[i % len(sets)].round_seed)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        res = hr.run(host[i % len(host)], A, W, T, sets[i % len(sets)].round_seed)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    ms = shard.max_over_ranks(ms, device)
    acc_last = int(res["acc_len"].sum())
    ref_last = {k: res[k].clone() for k in ("acc_len", "bonus_tok", "n_nodes")}   # the slots below reuse these buffers
    # the same steps with two rounds in flight: the copies of a step run beside the kernels of the step before
    for i in range(2):
        hr.submit(host[i % len(host)], A, W, T, sets[i % len(sets)].round_seed)
        hr.collect()
    barrier()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for i in range(steps):
        hr.submit(host[i % len(host)], A, W, T, sets[i % len(sets)].round_seed)
        if i > 0:
            res2 = hr.collect()
    res2 = hr.collect()
    p1.record()
    barrier()
    ms2 = shard.max_over_ranks(p0.elapsed_time(p1), device)
    same = all(bool(torch.equal(res2[k], ref_last[k])) for k in ref_last)
    return {"value": world * steps * 1e3 / ms, "unit": "rounds/s", "steps": steps,
            "h2d_bytes_per_step": hr.h2d_bytes, "d2h_bytes_per_step": hr.d2h_bytes,
            "acc_len_sum_last": acc_last,
            "two_in_flight": {"value": world * steps * 1e3 / ms2, "unit": "rounds/s", "same_results": same}}


def oracle_round_sample(orc, wl, U, A32, W32, anchor, theta, Z, zoff, T, seed, reqs, threads):
    """Expand + verify with the CPU oracle for the listed requests (as it stands, threads over requests)."""
    import oracle

    def one(b):
        ub = U[b].float().numpy()
        tr = orc.expand_tree(ub, A32, W32, int(anchor[b]), float(theta[b]), T, seed, b)
        r0 = int(zoff[b])
        zb = Z[r0:r0 + tr["n"] + 1].float().numpy()
        if zb.shape[0] < tr["n"] + 1:
            return tr, None
        return tr, orc.verify_tree(ub, A32, W32, zb, int(anchor[b]), tr, T, seed, b, want_edge_stat=True)

    return oracle.run_batch(one, list(reqs), threads)


def cpu_baseline(wl, table, s, A, W, T, B):
    import numpy as np
    import oracle
    cores = os.cpu_count() or 1
    orc = oracle.Oracle(wl.V, wl.D, wl.r, wl.K, wl.Nmax, calib_mode=wl.calib_mode,
                        calib_table=table.numpy().astype(np.float64))
    A32, W32 = A.cpu().float().numpy(), W.cpu().float().numpy()
    U, Z, zoff = s.U.cpu(), s.Z.cpu(), s.zoff.cpu()
    anchor, theta = s.anchor.cpu(), s.theta.cpu()
    sample = min(B, max(1, 2 * cores))
    threads = min(sample, cores)
    t0 = time.time()
    res, used = oracle_round_sample(orc, wl, U, A32, W32, anchor, theta, Z, zoff, T, s.round_seed, range(sample), threads)
    dt = time.time() - t0
    parents = sum(r[0]["n_scored"] for r in res)
    return {"value": (sample / B) / dt, "unit": "rounds/s", "cores": used, "host_cores": cores, "kind": "oracle",
            "sample": f"{sample} of {B} requests of one round (expand + verify with edge statistics), {dt:.1f} s wall",
            "parents_scored_per_s": parents / dt}


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    import numpy as np
    import oracle
    wl = synth.WORKLOADS[args.workload]
    B = args.batch or wl.B
    T = wl.temps[-1] if args.T is None else args.T
    theta = workload_theta(args, wl, B)
    cores = os.cpu_count() or 1
    table = synth.make_calibration_table(wl, args.seed + 4, "fit")
    A, W = synth.make_head(wl, args.seed + 1, "cpu")
    orc = oracle.Oracle(wl.V, wl.D, wl.r, wl.K, wl.Nmax, calib_mode=wl.calib_mode,
                        calib_table=table.numpy().astype(np.float64))
    A32, W32 = A.float().numpy(), W.float().numpy()
    sample = min(B, max(1, cores // 2))
    threads = min(sample, cores)
    wl_s = wl
    Ufull = synth.make_base_logits(wl_s, args.seed + 2, "cpu", B=sample)
    anchor = synth.make_anchor(wl_s, args.seed + 3, B=sample)
    th = synth.make_theta(wl_s, B=sample, theta=theta)
    U = Ufull[:, :wl.D].contiguous()
    # target logits need a tree: build them once from the oracle's own trees (untimed set-up)
    trees, _ = oracle.run_batch(lambda b: orc.expand_tree(U[b].float().numpy(), A32, W32, int(anchor[b]),
                                                          float(th[b]), T, args.seed + 7, b), list(range(sample)), threads)
    N = wl.Nmax
    n_nodes = torch.tensor([t["n"] for t in trees])
    tok = torch.stack([torch.from_numpy(t["tok"]) for t in trees])
    depth = torch.stack([torch.from_numpy(t["depth"]) for t in trees])
    nh = torch.stack([torch.from_numpy(t["node_hash"].astype(np.int64)) for t in trees])
    Z, zoff = synth.make_target_logits(wl, args.seed + 5, Ufull, A, W, anchor, n_nodes, tok, depth, nh)

    def step():
        return oracle_round_sample(orc, wl, U, A32, W32, anchor, th, Z, zoff, T, args.seed + 7, range(sample), threads)

    for _ in range(min(args.warmup, 1)):
        step()
    t0 = time.time()
    used = threads
    for _ in range(args.steps):
        _, used = step()
    dt = time.time() - t0
    val = args.steps * (sample / B) / dt
    return {"impl": "reference", "metric": "tree_rounds_per_s", "value": val, "unit": "rounds/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{wl.name}: batch {B}, V={wl.V}, D={wl.D}, r={wl.r}, K={wl.K}, Nmax={wl.Nmax}, "
                                   f"theta={theta}, T={T}, {wl.dtype} U/A/W/Z"},
            "cpu_baseline": {"value": val, "unit": "rounds/s", "cores": used, "host_cores": cores, "kind": "oracle",
                             "sample": f"each step = {sample} of {B} requests of one round (expand + verify), "
                                       f"value scaled to whole rounds"},
            "e2e": {"value": val, "unit": "rounds/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=device)
    out = run_ours(args, rank, world, device)
    if world == 1 and args.workload == "serve32" and not args.no_cpu and not args.no_e2e:
        # the default run also reports the single-request decode shape, briefly
        try:
            out["also"] = {"decode": short_side_run(args, device, "decode")}
        except Exception as e:  # the headline line must not depend on the side run
            out["also"] = {"decode": {"error": repr(e)}}
        try:
            out["also"]["allocate_budget"] = allocate_side_run(args, device)
        except Exception as e:
            out["also"]["allocate_budget"] = {"error": repr(e)}
        try:
            out["also"]["calibration"] = calibrate_side_run(args, device)
        except Exception as e:
            out["also"]["calibration"] = {"error": repr(e)}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
