#!/usr/bin/env python
"""Benchmark of the GRAFT draft-tree round on B200.

One step = one whole round over one batch of synthetic drafter outputs: graft_build_trees (vocab pass ->
SABA -> TDES edges -> best-first selection -> emission) followed by graft_accept.  Metric: trees/s (and
microseconds per round) at batch 64, L = 16, V = 151,936 bf16 (workload "M").  Prints one JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload M] [--impl graft|reference]

N > 1 (under torchrun): every rank runs the same per-GPU batch on its own sequences (weak scaling, no
data-path collective); the time is the max over ranks.  --impl reference times the CPU oracle, as it stands,
on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import graft_inputs as gi  # noqa: E402

METRIC = "draft trees built and verified-walked per second (batch 64, L=16, V=151,936 bf16)"
UNIT = "trees/s"
# DRAM bytes (read + write) of one vocab-pass launch on workload M: the mean of the two launches of the ncu
# capture summarised in profiles/vocab_pass_kernel_M.md.
NCU_VOCAB_TRAFFIC_BYTES_M = 324_300_000  # profiles/vocab_pass_kernel_M.md: mean of two launches, read + write
L2_BYTES = 126 * 1024 * 1024


MIN_KERNEL_SAMPLES = 32  # rounds whose kernels are timed one by one, whatever --steps is
MIN_CLOCK_WINDOW_S = 0.06  # the clock readings are taken over at least this long under the benchmark's load


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Reads SM clock, power and clock-event reasons through NVML while the benchmark runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples = []  # (t, sm_mhz, reasons_bitmask, power_w)
        self.stop_flag = False
        self.max_mhz = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((time.perf_counter(), mhz, int(reasons), pw))
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self, t0, t1):
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
                 0x80: "hw_power_brake", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting",
                 0x10: "sync_boost"}
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "window": "none"}
        win = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed rounds and the sampled rounds that follow them"
        if len(win) < 3:
            win, window = self.samples, "whole run"
        bits = 0
        for s in win:
            bits |= s[2]
        return {"sm_mhz": float(np.median([s[1] for s in win])), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(n for b, n in names.items() if bits & b), "samples": len(win), "window": window,
                "power_w_max": max(s[3] for s in win)}


def _dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def _host_inputs(w, lo, hi, n_buf):
    """n_buf independent input sets for sequences lo..hi-1 (set k uses sequence index b + k * 1_000_003)."""
    sets = []
    for k in range(n_buf):
        off = k * 1_000_003
        parts = [gi.batch_inputs(w, b + off, b + off + 1) for b in range(lo, hi)]
        s = {key: torch.cat([p[key] for p in parts]) for key in ("logits", "hidden", "root_token", "hist", "prefix_len")}
        s["seq_ids"] = [b + off for b in range(lo, hi)]
        sets.append(s)
    return sets


def run_graft(args):
    from paper_2608_20375_b200 import Graft, BF16, F32, shard_range  # noqa: F401
    import oracle  # CPU-baseline leg only

    rank, world, local = _dist_setup(args.gpus)
    w = gi.WORKLOADS[args.workload]
    batch = w.batch  # per GPU (weak scaling)
    lo = rank * batch
    dev = torch.device("cuda", local)
    dt = {"f32": 0, "bf16": 1}
    g = Graft(w.V, w.L, w.K, w.m, w.hidden_dim, batch, w.budget_min, w.budget_max, w.budget_step, w.beta, 1,
              dt[w.logits_dtype], dt[w.hidden_dtype])
    tb = gi.tdes_tables(w)
    P, Ct, u = tb["P"].to(dev), tb["C"].to(dev), tb["u"].to(dev)
    g.set_tdes_tables(P, Ct, u, tb["s"])
    saba_kw = gi.saba_defaults(w)
    g.set_saba(**saba_kw)
    if args.edge_rows is not None:
        g.set_edge_rows(args.edge_rows)

    logits_bytes = batch * w.L * w.V * (2 if w.logits_dtype == "bf16" else 4)
    n_buf = max(2, int(np.ceil(2.5 * L2_BYTES / logits_bytes)))  # rotating sets: > 2.5x L2 in total
    n_buf = min(n_buf, 8)
    host_sets = _host_inputs(w, lo, lo + batch, n_buf)
    dev_sets = [{k: (v.to(dev) if torch.is_tensor(v) else v) for k, v in s.items()} for s in host_sets]
    fixed = None if w.fixed_budget is None else torch.full((batch,), w.fixed_budget, dtype=torch.int32, device=dev)
    outs = [g.alloc_out(batch) for _ in range(n_buf)]
    a_len = torch.empty(batch, dtype=torch.int32, device=dev)
    a_path = torch.empty((batch, w.L), dtype=torch.int32, device=dev)
    bonus = torch.empty(batch, dtype=torch.int32, device=dev)

    def build(k):
        s = dev_sets[k]
        g.build_trees(s["logits"], s["hidden"], s["root_token"], s["hist"], s["prefix_len"], fixed, outs[k])

    # target next-token ids per input set: drawn independently of the trees, indexed by each node's depth
    tn_dev, tn_host = [], []
    for k in range(n_buf):
        build(k)
        torch.cuda.synchronize()
        depth = outs[k].depth.cpu().numpy()
        tn = np.stack([gi.target_next_from_depth(gi.target_tokens(w, sid), depth[i])
                       for i, sid in enumerate(host_sets[k]["seq_ids"])])
        tn_host.append(torch.from_numpy(tn).pin_memory())
        tn_dev.append(torch.from_numpy(tn).to(dev))

    def step(i):
        k = i % n_buf
        build(k)
        g.accept(outs[k], tn_dev[k], a_len, a_path, bonus)

    sampler = ClockSampler(local)
    sampler.start()
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    if args.cuda_graph:
        # one captured round per input set, replayed in the timed loop (the per-kernel events then come from eager
        # rounds: event records are not captured)
        eager_step = step
        side = torch.cuda.Stream()
        graphs = []
        for k in range(n_buf):
            side.wait_stream(torch.cuda.current_stream())
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=side):
                eager_step(k)
            graphs.append(gr)
        torch.cuda.synchronize()

        def step(i, timed=False):  # noqa: F811
            if timed:
                eager_step(i)
            else:
                graphs[i % n_buf].replay()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    # per-kernel CUDA events (recorded by the library on the launching stream around each of its kernels) are taken
    # on every TIMING_EVERY-th step of the timed region: four event records cost the stream a few microseconds
    # (a round with its four event records takes about 16 us longer than one without: in a long run every
    # steps/32-th round carries them, which still gives 32 samples and keeps their cost under 1 % of ms_per_step)
    timing_every = max(args.timing_every, args.steps // MIN_KERNEL_SAMPLES)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    launches0 = g.launch_count()
    n_timed = 0
    g.set_timing(1)  # (creates the library's events outside the timed region)
    g.set_timing(False)
    t_wall0 = time.perf_counter()
    ev0.record()
    for i in range(args.steps):
        timed = (i % timing_every) == timing_every - 1  # (never the first rounds after the synchronize)
        if timed:
            g.set_timing(2 if n_timed else 1)  # 1 = reset the call count, 2 = go on counting
            n_timed += 1
        if args.cuda_graph:
            step(i, timed)
        else:
            step(i)
        if timed:
            g.set_timing(False)
    ev1.record()
    torch.cuda.synchronize()
    launches = g.launch_count() - launches0
    ms_total = ev0.elapsed_time(ev1)
    # the per-kernel figures must not rest on a handful of events when the run is short: more sampled rounds follow the
    # timed loop (they are not part of ms_per_step) until at least MIN_KERNEL_SAMPLES rounds carry events; the clock
    # sampler's window takes them in
    n_t = g.read_timing()[0]
    extra = 0
    evx0, evx1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    evx0.record()
    while n_t + extra < MIN_KERNEL_SAMPLES or extra < 8:
        g.set_timing(2 if (n_t + extra) > 0 else 1)
        if args.cuda_graph:
            step(extra, True)
        else:
            step(extra)
        g.set_timing(False)
        extra += 1
    evx1.record()
    torch.cuda.synchronize()
    # a round that carries the per-kernel event records: longer than an ordinary one (the records cost time and keep a
    # kernel from setting up while the one ahead of it drains); the per-kernel intervals add up to this, not to ms_per_step
    instrumented_round_ms = evx0.elapsed_time(evx1) / extra
    # ... and a short run leaves the clock sampler (a reading every few milliseconds) nothing to read: the same rounds
    # go on, untimed, until the window under load holds a handful of readings
    i_more = 0
    while time.perf_counter() - t_wall0 < MIN_CLOCK_WINDOW_S:
        for _ in range(16):
            step(i_more)
            i_more += 1
        torch.cuda.synchronize()
    t_wall1 = time.perf_counter()
    barrier()
    n_t, vocab_ms, tdes_ms, tree_ms = g.read_timing()
    # what two event records cost the stream with nothing between them (the per-kernel figures above are intervals
    # between such records, so each holds one of these; reported beside them, not subtracted from `frac`)
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(64)]
    step(0)
    for a, b_ in pairs:
        a.record()
        b_.record()
        step(0)
    torch.cuda.synchronize()
    event_pair_ms = float(np.median([a.elapsed_time(b_) for a, b_ in pairs]))
    # the vocab pass alone, launched back to back over the same rotating inputs through its own entry point
    # (graft_vocab_pass) with one event pair around the whole series: its throughput with no event record between
    # launches, i.e. with each launch setting up while the one ahead drains, as inside an ordinary round
    vb_ids = torch.empty((batch, w.L, w.K), dtype=torch.int32, device=dev)
    vb_lp = torch.empty((batch, w.L, w.K), dtype=torch.float32, device=dev)
    vb_lse = torch.empty((batch, w.L), dtype=torch.float32, device=dev)
    vb_st = torch.empty((batch, w.L), dtype=torch.int32, device=dev)
    n_b2b = 200
    for i in range(8):
        g.vocab_pass(dev_sets[i % n_buf]["logits"], vb_ids, vb_lp, vb_lse, vb_st)
    evb0, evb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    evb0.record()
    for i in range(n_b2b):
        g.vocab_pass(dev_sets[i % n_buf]["logits"], vb_ids, vb_lp, vb_lse, vb_st)
    evb1.record()
    torch.cuda.synchronize()
    vocab_b2b_ms = evb0.elapsed_time(evb1) / n_b2b
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms_total], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / args.steps
    value = world * batch / (ms_step * 1e-3)
    mean_accept = float(a_len.float().mean().item())
    status_or = int(torch.stack([o.status for o in outs]).max().item())

    # ---- end to end through the host-buffer entry point (host <-> device copies inside the timed region)
    e2e_steps = max(3, min(args.steps, 10))
    pinned = [{k: v.pin_memory() for k, v in s.items() if torch.is_tensor(v)} for s in host_sets[:2]]
    h_out = g.alloc_out(batch, device="cpu", pinned=True)
    h_alen = torch.empty(batch, dtype=torch.int32).pin_memory()
    h_fixed = None if fixed is None else fixed.cpu().pin_memory()
    d_out = outs[0]

    def e2e_step(i):
        s = pinned[i % len(pinned)]
        g.build_trees_host(s["logits"], s["hidden"], s["root_token"], s["hist"], s["prefix_len"], h_fixed, h_out)
        # the verifier's answer arrives on the host; the walk runs on the device copy of the tree it was built from
        tnd = tn_host[i % len(pinned)].to(dev, non_blocking=True)
        for name in ("n_nodes", "token", "parent"):
            getattr(d_out, name).copy_(getattr(h_out, name), non_blocking=True)
        g.accept(d_out, tnd, a_len, a_path, bonus)
        h_alen.copy_(a_len, non_blocking=True)
        torch.cuda.synchronize()

    for i in range(2):
        e2e_step(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        e2e_step(i)
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([e2e_s], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    s0 = pinned[0]
    h2d = sum(s0[k].numel() * s0[k].element_size() for k in ("logits", "hidden", "root_token", "hist", "prefix_len"))
    h2d += tn_host[0].numel() * 4 + sum(getattr(h_out, n).numel() * 4 for n in ("n_nodes", "token", "parent"))
    d2h = sum(getattr(h_out, n).numel() * getattr(h_out, n).element_size() for n in
              ("n_nodes", "budget", "status", "token", "parent", "depth", "position", "path_score", "mask")) + batch * 4
    sampler.stop_flag = True
    sampler.join(timeout=2)

    if rank != 0:
        return
    peak, peak_kind = _peaks()
    vocab_s = vocab_ms * 1e-3 / max(1, n_t)
    # algorithmic bytes of the vocab-pass kernel: every logit once, plus (SABA) every hidden state once for the
    # adjacent-position cosines that the same kernel computes beside the stream
    hidden_bytes = 0 if w.fixed_budget is not None else batch * w.L * w.hidden_dim * (2 if w.hidden_dtype == "bf16" else 4)
    # `achieved` / `frac` count the logits alone (the definition of the vocab pass's roofline: logits bytes over kernel
    # time); the figures "with_hidden" add the hidden-state bytes that the same kernel also reads
    algo_bytes = logits_bytes
    achieved = algo_bytes / vocab_s / 1e9
    achieved_h = (logits_bytes + hidden_bytes) / vocab_s / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "us_per_round": ms_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: batch {batch} per GPU, L={w.L}, V={w.V} {w.logits_dtype} logits, "
                               f"hidden d={w.hidden_dim} {w.hidden_dtype}, K={w.K}, m={w.m}, beta={w.beta}, SABA budgets "
                               f"[{w.budget_min},{w.budget_max}] step {w.budget_step}, build_trees + accept",
                   "edge_rows": g.edge_rows(),
                   "parallelism": f"batch-sharded x{world}, no collective",
                   "l2_policy": f"{n_buf} rotating input sets of {logits_bytes / 1e6:.0f} MB each (> L2 of 126 MB)"},
        "gpu_launches": launches,
        "kernel_ms": {"vocab_pass": vocab_ms / max(1, n_t), "tdes_edges": tdes_ms / max(1, n_t),
                      "tree": tree_ms / max(1, n_t), "calls_averaged": n_t, "empty_event_pair": event_pair_ms,
                      "round_with_these_events": instrumented_round_ms,
                      "vocab_pass_back_to_back": vocab_b2b_ms},
        "roofline": {"bound": "hbm", "kernel": "vocab_pass_kernel", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8000": achieved / 8000.0, "algorithmic_bytes": algo_bytes,
                     "achieved_with_hidden": achieved_h, "frac_with_hidden": achieved_h / peak,
                     "algorithmic_bytes_with_hidden": logits_bytes + hidden_bytes,
                     "frac_net_of_event_pair": algo_bytes / max(1e-9, vocab_s - event_pair_ms * 1e-3) / 1e9 / peak,
                     "frac_back_to_back": algo_bytes / (vocab_b2b_ms * 1e-3) / 1e9 / peak,
                     "traffic": NCU_VOCAB_TRAFFIC_BYTES_M if w.name == "M" else None},
        "e2e": {"value": world * batch / e2e_s, "unit": UNIT, "ms_per_step": e2e_s * 1e3, "steps": e2e_steps,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
        "clocks": sampler.summary(t_wall0, t_wall1),
        "mean_accepted_len": mean_accept, "status_or": status_or,
    }
    # ---- CPU baseline: the oracle as it stands, on this machine's host cores, on a bounded sample
    if world == 1 and not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        threads = min(cores, 32)
        sp = oracle.SabaParams(**saba_kw)
        # whole batches of the input sets, round after round, until about 10 s have passed (>= 150 core-seconds)
        done, rounds, t0 = 0, 0, time.perf_counter()
        while time.perf_counter() - t0 < 10.0 and rounds < 64:
            s = host_sets[rounds % len(host_sets)]
            fb = None if w.fixed_budget is None else np.full((batch,), w.fixed_budget, dtype=np.int32)
            orc = oracle.build_trees(s["logits"], s["hidden"], s["root_token"].numpy(), s["hist"].numpy(),
                                     s["prefix_len"].numpy(), fb, sp, (w.budget_min, w.budget_max, w.budget_step),
                                     tb["P"].numpy(), tb["C"].numpy(), tb["u"].numpy(), tb["s"], w.beta, w.K,
                                     threads=threads)
            for i in range(batch):
                tn = gi.target_next_from_depth(gi.target_tokens(w, s["seq_ids"][i]), orc["depth"][i])
                oracle.accept(int(orc["n_nodes"][i]), orc["token"][i], orc["parent"][i], tn, w.L)
            done += batch
            rounds += 1
        dt_s = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": done / dt_s, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{rounds} rounds over the {batch} sequences of the input sets, "
                                          f"{threads} threads, {dt_s:.1f} s"}
    print(json.dumps(line))


def run_reference(args):
    """The oracle (plain C, fp64), as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle
    w = gi.WORKLOADS[args.workload]
    cores = os.cpu_count() or 1
    threads = min(cores, 32, w.batch)
    n_seq = threads  # one sequence per thread and step: a bounded sample of the batch
    tb = gi.tdes_tables(w)
    saba_kw = gi.saba_defaults(w)
    sp = oracle.SabaParams(**saba_kw)
    sets = _host_inputs(w, 0, n_seq, 2)
    P, Ct, u = tb["P"].numpy(), tb["C"].numpy(), tb["u"].numpy()
    ys = [[gi.target_tokens(w, sid) for sid in s["seq_ids"]] for s in sets]

    def step(i):
        s = sets[i % 2]
        fb = None if w.fixed_budget is None else np.full(n_seq, w.fixed_budget, np.int32)
        orc = oracle.build_trees(s["logits"], s["hidden"], s["root_token"].numpy(), s["hist"].numpy(),
                                 s["prefix_len"].numpy(), fb, sp, (w.budget_min, w.budget_max, w.budget_step), P, Ct, u,
                                 tb["s"], w.beta, w.K, threads=threads)
        for j in range(n_seq):
            tn = gi.target_next_from_depth(ys[i % 2][j], orc["depth"][j])
            oracle.accept(int(orc["n_nodes"][j]), orc["token"][j], orc["parent"][j], tn, w.L)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(i)
    dt_s = (time.perf_counter() - t0) / args.steps
    value = n_seq / dt_s
    sample = f"{n_seq} of the {w.batch} sequences per step, one round each, {threads} threads"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: batch {w.batch}, L={w.L}, V={w.V} {w.logits_dtype} logits, hidden "
                               f"d={w.hidden_dim}, K={w.K}, SABA budgets [{w.budget_min},{w.budget_max}]; CPU oracle on "
                               f"a sample of {n_seq} sequences per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_overlap(args):
    """--overlap-verifier-ms T: the batch as two micro-batches with contexts and streams of their own, a stub verifier
    (a chain of GEMMs of about T ms) between build and walk; sequential schedule against overlapped one, on one GPU.
    Prints its own JSON line (not the benchmark's metric)."""
    from paper_2608_20375_b200 import Graft, MicroBatch, run_rounds, join

    w = gi.WORKLOADS[args.workload]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n_micro, mb_batch = 2, w.batch // 2
    dt = {"f32": 0, "bf16": 1}
    tb = gi.tdes_tables(w)
    P, Ct, u = tb["P"].to(dev), tb["C"].to(dev), tb["u"].to(dev)
    micro = []
    for i in range(n_micro):
        g = Graft(w.V, w.L, w.K, w.m, w.hidden_dim, mb_batch, w.budget_min, w.budget_max, w.budget_step, w.beta, 1,
                  dt[w.logits_dtype], dt[w.hidden_dtype])
        g.set_tdes_tables(P, Ct, u, tb["s"])
        g.set_saba(**gi.saba_defaults(w))
        micro.append(MicroBatch(g, mb_batch, w.L))
    n_buf = 4  # input sets per micro-batch: 8 x 156 MB of logits in rotation (> L2)
    sets = [[{k: (v.to(dev) if torch.is_tensor(v) else v)
              for k, v in _host_inputs(w, (i * n_buf + k) * mb_batch, (i * n_buf + k + 1) * mb_batch, 1)[0].items()}
             for k in range(n_buf)] for i in range(n_micro)]
    tn = torch.zeros((mb_batch, micro[0].graft.nmax), dtype=torch.int32, device=dev)
    a = torch.randn(4096, 4096, device=dev, dtype=torch.bfloat16)
    # size the stub: GEMMs of 4096^3 until one verification takes about the requested time
    def chain(n):
        y = a
        for _ in range(n):
            y = torch.mm(y, a)
        return y
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    chain(8)
    torch.cuda.synchronize()
    e0.record()
    chain(32)
    e1.record()
    torch.cuda.synchronize()
    per_gemm = e0.elapsed_time(e1) / 32
    n_gemm = max(1, int(round(args.overlap_verifier_ms / per_gemm)))

    def draft(i, r):
        return sets[i][r % n_buf]

    def verify(i, r, out):
        chain(n_gemm)
        return tn

    def build_only(i, r, out):
        return tn

    def timed(fn_verify, overlap, rounds):
        run_rounds(micro, 8, draft, fn_verify, overlap=overlap)
        join(micro)
        torch.cuda.synchronize()
        e0.record()
        run_rounds(micro, rounds, draft, fn_verify, overlap=overlap)
        join(micro)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / rounds

    rounds = args.steps
    res = {
        "build_walk_only_ms": timed(build_only, False, rounds),
        "sequential_ms": timed(verify, False, rounds),
        "overlapped_ms": timed(verify, True, rounds),
    }
    e0.record()
    for _ in range(rounds):
        chain(n_gemm)
        chain(n_gemm)
    e1.record()
    torch.cuda.synchronize()
    res["verifier_only_ms"] = e0.elapsed_time(e1) / rounds
    print(json.dumps({
        "kind": "micro-batch overlap (two micro-batches, one round of each per step)", "workload": args.workload,
        "micro_batches": n_micro, "batch_per_micro_batch": mb_batch, "rounds": rounds,
        "stub_verifier": f"{n_gemm} bf16 GEMMs of 4096^3 per micro-batch round ({per_gemm * n_gemm:.3f} ms alone)",
        **{k: round(v, 5) for k, v in res.items()},
        "overlapped_over_sequential": round(res["overlapped_ms"] / res["sequential_ms"], 4),
    }))


def run_tdes_loss(args):
    """--tdes-loss: the TDES training objective forward + backward (graft_tdes_loss) on one synthetic batch of traces
    at the paper's shapes; prints its own JSON line (not the benchmark's metric)."""
    from paper_2608_20375_b200 import Graft
    import oracle  # CPU-baseline leg only

    V, L, K, m = 151936, 16, 32, 128
    n_groups, n_pairs, n_edges = 32768, 131072, 262144
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    g = Graft(V, L, K, m, 32, 1, 16, 32, 16, 0.2, 1, 0, 0)
    w = gi.small(V=V, L=L, K=K, m=m, seed=20381)
    tb = gi.tdes_tables(w)
    P, Ct, u = tb["P"].to(dev), tb["C"].to(dev), tb["u"].to(dev)
    g.set_tdes_tables(P, Ct, u, tb["s"])
    tr = gi.tdes_traces(V, L, K, n_groups, n_pairs, n_edges, seed=20382)
    groups = {k: torch.from_numpy(np.ascontiguousarray(v)).to(dev) for k, v in tr["groups"].items()}
    pairs, edges = torch.from_numpy(tr["pairs"]).to(dev), torch.from_numpy(tr["edges"]).to(dev)
    cfg = dict(gamma=0.5, w1=4.0, lambda_kl=1.0, lambda_pair=1.0, lambda_bce=0.25)
    loss = torch.zeros(4, dtype=torch.float64, device=dev)
    gP, gC = torch.zeros((V, m), device=dev), torch.zeros((V, m), device=dev)
    gu, gs = torch.zeros((L, m), device=dev), torch.zeros(1, device=dev)

    def step():
        g.tdes_loss(groups, pairs, edges, loss=loss, gP=gP, gC=gC, gu=gu, gs=gs, **cfg)

    for _ in range(max(3, args.warmup or 3)):
        step()
    torch.cuda.synchronize()
    steps = args.steps or 50
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    row = m * 4
    # rows gathered + gradient rows added, once each: a group reads 1 + K rows and adds to 1 + K, an edge 2 and 2
    alg = (n_groups * 2 * (1 + K) + n_pairs * 8 + n_edges * 4) * row
    items = n_groups + n_pairs + n_edges
    # the oracle on a slice of the same traces
    n_s = 512
    sub = {k: v[:n_s] for k, v in tr["groups"].items()}
    t0 = time.perf_counter()
    oracle.tdes_loss(tb["P"].numpy(), tb["C"].numpy(), tb["u"].numpy(), tb["s"], sub, tr["pairs"][:4 * n_s],
                     tr["edges"][:8 * n_s], **cfg)
    t_cpu = time.perf_counter() - t0
    hbm_peak, peak_kind = _peaks()
    print(json.dumps({
        "kind": "TDES training objective, forward + backward (graft_tdes_loss)",
        "shapes": {"V": V, "L": L, "K": K, "m": m, "groups": n_groups, "pairs": n_pairs, "edges": n_edges},
        "ms_per_step": round(ms, 4), "items_per_s": round(items / (ms * 1e-3)),
        "algorithmic_bytes": alg, "algorithmic_gbs": round(alg / (ms * 1e-3) / 1e9, 1),
        "hbm_peak_gbs": hbm_peak, "peak_kind": "of " + peak_kind,
        "note": "rows of hot tokens are served by L2, so the algorithmic rate is not bounded by the HBM peak",
        "cpu_oracle": {"items": 13 * n_s, "seconds": round(t_cpu, 3),
                       "items_per_s": round(13 * n_s / t_cpu)},
    }))


def run_saba_fit(args):
    """--saba-fit: the least-squares fit of the SABA models (graft_saba_fit) over synthetic replay logs; prints its own
    JSON line (not the benchmark's metric)."""
    from paper_2608_20375_b200 import Graft
    import oracle  # CPU-baseline leg only

    n = 16_000_000  # 36 bytes a round: 576 MB, well over L2
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    g = Graft(1000, 4, 4, 16, 8, 1, 8, 8, 8, 0.0, 1, 0, 0)
    lg = gi.saba_replay_logs(n, seed=20383)
    d = {k: torch.from_numpy(np.ascontiguousarray(v)).to(dev) for k, v in lg.items()}
    out = torch.zeros(10, dtype=torch.float64, device=dev)

    def step():
        g.saba_fit(d["state"], d["budget"], d["gain"], d["prefix_len"], d["latency"], out)

    for _ in range(max(3, args.warmup or 3)):
        step()
    torch.cuda.synchronize()
    steps = args.steps or 20
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    n_s = 2_000_000
    t0 = time.perf_counter()
    ref = oracle.saba_fit(**{k: v[:n_s] for k, v in lg.items()})
    t_cpu = time.perf_counter() - t0
    hbm_peak, peak_kind = _peaks()
    alg = n * 36
    print(json.dumps({
        "kind": "least-squares fit of the SABA gain and cost models (graft_saba_fit)", "rounds_logged": n,
        "ms_per_fit": round(ms, 4), "algorithmic_bytes": alg, "achieved_gbs": round(alg / (ms * 1e-3) / 1e9, 1),
        "hbm_peak_gbs": hbm_peak, "peak_kind": "of " + peak_kind, "frac": round(alg / (ms * 1e-3) / 1e9 / hbm_peak, 3),
        "fit": [float(x) for x in out.cpu().numpy()],
        "cpu_oracle": {"rounds": n_s, "seconds": round(t_cpu, 3), "rounds_per_s": round(n_s / t_cpu),
                       "phi": [float(x) for x in ref["phi"]], "c": [float(x) for x in ref["c"]]},
    }))


# ---- budget / beta sweeps on synthetic acceptance (the shape of the paper's Tables 2 and 3) --------------------------
SWEEP_BETAS = (0.0, 0.05, 0.1, 0.2, 0.4)
SWEEP_BUDGETS = (16, 32, 64, 128, 256, 512)


def sweep_arms(fixed_budget):
    """(name, beta, fixed budget or None = SABA): the component analysis, the beta sensitivity under SABA, and the
    accepted length against a fixed budget (where the gain of more nodes saturates)."""
    arms = [("DDTree (beta=0, fixed budget)", 0.0, fixed_budget), ("+TDES (beta=0.2, fixed budget)", 0.2, fixed_budget),
            ("+SABA (beta=0, SABA budget)", 0.0, None), ("GRAFT (beta=0.2, SABA budget)", 0.2, None)]
    arms += [(f"beta={b:g} (SABA budget)", b, None) for b in SWEEP_BETAS]
    return arms + [(f"fixed budget {n} (beta=0.2)", 0.2, n) for n in SWEEP_BUDGETS]


def sweep_cost_ms(saba_kw, n):
    """The modelled verification cost C_t(B) of a tree of n draft nodes: the piecewise-linear table of the workload."""
    return float(np.interp(n, saba_kw["pts_n"], saba_kw["pts_t"]))


def sweep_arm(w, x, beta, fixed_budget, dev, rounds=0):
    """One arm on inputs x (CPU tensors of gi.batch_inputs): trees, acceptance walk against the seeded targets, and
    (rounds > 0) the device time of build + walk.  Returns per-sequence arrays and the arm's summary."""
    from paper_2608_20375_b200 import Graft
    dt = {"f32": 0, "bf16": 1}
    batch = x["logits"].shape[0]
    g = Graft(w.V, w.L, w.K, w.m, w.hidden_dim, batch, w.budget_min, w.budget_max, w.budget_step, beta, 1,
              dt[w.logits_dtype], dt[w.hidden_dtype])
    tb = gi.tdes_tables(w)
    keep = [tb["P"].to(dev), tb["C"].to(dev), tb["u"].to(dev)]
    g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
    saba_kw = gi.saba_defaults(w)
    g.set_saba(**saba_kw)
    d = {k: x[k].to(dev) for k in ("logits", "hidden", "root_token", "hist", "prefix_len")}
    fixed = None if fixed_budget is None else torch.full((batch,), int(fixed_budget), dtype=torch.int32, device=dev)
    out = g.alloc_out(batch)
    a_len = torch.empty(batch, dtype=torch.int32, device=dev)
    a_path = torch.empty((batch, w.L), dtype=torch.int32, device=dev)
    bonus = torch.empty(batch, dtype=torch.int32, device=dev)

    def build():
        g.build_trees(d["logits"], d["hidden"], d["root_token"], d["hist"], d["prefix_len"], fixed, out)

    build()
    torch.cuda.synchronize()
    depth = out.depth.cpu().numpy()
    seq_ids = x.get("seq_ids", list(range(batch)))
    tn = np.stack([gi.target_next_from_depth(gi.target_tokens(w, sid), depth[i]) for i, sid in enumerate(seq_ids)])
    tn_d = torch.from_numpy(tn).to(dev)
    g.accept(out, tn_d, a_len, a_path, bonus)
    torch.cuda.synchronize()
    us = None
    if rounds > 0:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            build()
            g.accept(out, tn_d, a_len, a_path, bonus)
        e0.record()
        for _ in range(rounds):
            build()
            g.accept(out, tn_d, a_len, a_path, bonus)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / rounds
    nodes = out.n_nodes.cpu().numpy().astype(np.int64) - 1   # draft nodes (the root is not counted)
    acc = a_len.cpu().numpy().astype(np.int64)
    budget = out.budget.cpu().numpy().astype(np.int64)
    cost = np.array([sweep_cost_ms(saba_kw, n) for n in nodes])
    res = dict(nodes=nodes, accepted=acc, budget=budget, status=out.status.cpu().numpy(),
               avg_nodes=float(nodes.mean()), mean_accepted=float(acc.mean()), mat=float(acc.mean() + 1.0),
               modelled_verify_ms=float(cost.mean()), us_per_round=us)
    # tokens committed per round (accepted draft tokens + the bonus token) over the round's modelled cost: the
    # verification cost of every sequence's tree plus the measured construction time of the batch
    build_ms = 0.0 if us is None else us * 1e-3
    res["tokens_per_modelled_ms"] = float(((acc + 1.0) / (cost + build_ms)).mean())
    g.destroy()
    return res


def run_sweep(args):
    """`--sweep`: the fixed-budget / beta sweeps in the shape of the paper's component analysis (Table 2) and beta
    sensitivity (Table 3; Sec. 4.3), on the synthetic inputs of a configured workload and its seeded targets.  The
    targets are synthetic (drawn from the boosted token sets, independently of the TDES tables, which are random): the
    numbers show the mechanics of the two knobs -- tree size against accepted length and cost -- not the paper's gains,
    which come from a scorer distilled from a target model."""
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = gi.WORKLOADS[args.workload]
    x = gi.batch_inputs(w)
    x["seq_ids"] = list(range(w.batch))
    rows = []
    for name, beta, fixed in sweep_arms(args.sweep_fixed_budget):
        r = sweep_arm(w, x, beta, fixed, dev, rounds=args.steps)
        rows.append(dict(arm=name, beta=beta, budget=("SABA" if fixed is None else int(fixed)),
                         avg_nodes=round(r["avg_nodes"], 2), mean_accepted=round(r["mean_accepted"], 4),
                         mat=round(r["mat"], 4), modelled_verify_ms=round(r["modelled_verify_ms"], 4),
                         us_per_round=round(r["us_per_round"], 2),
                         tokens_per_modelled_ms=round(r["tokens_per_modelled_ms"], 5),
                         status_or=int(np.bitwise_or.reduce(r["status"]))))
    base = rows[0]["tokens_per_modelled_ms"]
    for r in rows:
        r["vs_ddtree"] = round(r["tokens_per_modelled_ms"] / base, 4)
    print(json.dumps({"sweep": "component analysis and beta sensitivity on synthetic acceptance",
                      "workload": w.name, "batch": w.batch, "rounds_timed": args.steps, "data": "synthetic",
                      "targets": "seeded synthetic continuations (per-depth match rate decays 0.9 -> 0.3)",
                      "fixed_budget": args.sweep_fixed_budget, "rows": rows}))


def run_styles(args):
    """`--styles`: the round's kernels (the library's own CUDA events) on degenerate inputs of the benchmark's shape:
    ordinary logits, logits on coarse grids, flat rows, one or two dominant tokens over an exactly flat rest, sharply
    peaked rows, masked vocabularies, ramps (graft_inputs.styled_logits).  One JSON line."""
    from paper_2608_20375_b200 import Graft
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w0 = gi.WORKLOADS[args.workload]
    rng = np.random.default_rng(5)
    rows = []
    for style in gi.STYLES:
        w = gi.small(batch=w0.batch, L=w0.L, V=w0.V, K=w0.K, budget_min=w0.budget_min, budget_max=w0.budget_max,
                     budget_step=w0.budget_step, m=w0.m, hidden_dim=256, logits_dtype=w0.logits_dtype,
                     hidden_dtype=w0.hidden_dtype, beta=w0.beta if args.styles_beta is None else args.styles_beta,
                     seed=123)
        g = Graft(w.V, w.L, w.K, w.m, w.hidden_dim, w.batch, w.budget_min, w.budget_max, w.budget_step, w.beta, 1,
                  1 if w.logits_dtype == "bf16" else 0, 1 if w.hidden_dtype == "bf16" else 0)
        tb = gi.tdes_tables(w)
        keep = [tb["P"].to(dev), tb["C"].to(dev), tb["u"].to(dev)]
        g.set_tdes_tables(keep[0], keep[1], keep[2], tb["s"])
        g.set_saba(**gi.saba_defaults(w))
        x = gi.batch_inputs(w, 0, 8)  # eight sequences, repeated to the batch
        gen = torch.Generator().manual_seed(w.seed)
        rep = (w.batch + 7) // 8
        z = gi.styled_logits(x["logits"].float(), style, rng, gen, w.K).to(x["logits"].dtype).repeat(rep, 1, 1)[:w.batch].to(dev)
        h = x["hidden"].repeat(rep, 1, 1)[:w.batch].to(dev)
        root, hist, pre = (x[k].repeat(rep)[:w.batch].to(dev) for k in ("root_token", "hist", "prefix_len"))
        out = g.alloc_out(w.batch)
        for _ in range(3):
            g.build_trees(z, h, root, hist, pre, None, out)
        torch.cuda.synchronize()
        g.set_timing(1)
        for _ in range(args.steps):
            g.build_trees(z, h, root, hist, pre, None, out)
        torch.cuda.synchronize()
        n, a, b_, c = g.read_timing()
        rows.append(dict(style=style, vocab_pass_us=round(a / n * 1e3, 1), tdes_edges_us=round(b_ / n * 1e3, 1),
                         tree_us=round(c / n * 1e3, 1), budget_min=int(out.budget.min()), budget_max=int(out.budget.max()),
                         status_or=int(out.status.max())))
        g.destroy()
    print(json.dumps({"styles": "per-kernel times of the round on degenerate inputs", "shape": w0.name,
                      "beta": w.beta, "rounds_timed": args.steps, "rows": rows}))


def run_rows(args):
    """`--rows`: the vocab pass alone, launched back to back, on rows that defeat its top-K filter
    (graft_inputs.adversarial_rows): every row of the batch is the same shape, rolled differently per sequence so
    that the CTAs' segments cut it in different places.  One JSON line."""
    from paper_2608_20375_b200 import Graft
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = gi.WORKLOADS[args.workload]
    bf16 = w.logits_dtype == "bf16"
    g = Graft(w.V, w.L, w.K, w.m, 8, w.batch, w.budget_min, w.budget_max, w.budget_step, 0.0, 1, 1 if bf16 else 0, 0)
    ids = torch.empty((w.batch, w.L, w.K), dtype=torch.int32, device=dev)
    lp = torch.empty((w.batch, w.L, w.K), dtype=torch.float32, device=dev)
    lse = torch.empty((w.batch, w.L), dtype=torch.float32, device=dev)
    rs = torch.empty((w.batch, w.L), dtype=torch.int32, device=dev)
    gen = torch.Generator().manual_seed(11)
    out = []
    for name, row in gi.adversarial_rows(w.V, gen):
        r = row.to(torch.bfloat16 if bf16 else torch.float32).to(dev)
        # two input sets (each larger than L2 at the benchmark's shapes), every row rolled by its own offset
        sets = []
        for k in range(2):
            z = torch.stack([torch.roll(r, (131 * i + 7919 * k) % w.V) for i in range(w.batch * w.L)])
            sets.append(z.reshape(w.batch, w.L, w.V).contiguous())
        for _ in range(3):
            for z in sets:
                g.vocab_pass(z, ids, lp, lse, rs)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        torch.cuda.synchronize()
        ev[0].record()
        for _ in range(args.steps):
            for z in sets:
                g.vocab_pass(z, ids, lp, lse, rs)
        ev[1].record()
        torch.cuda.synchronize()
        out.append(dict(row=name, vocab_pass_us=round(ev[0].elapsed_time(ev[1]) * 1e3 / (2 * args.steps), 1),
                        status_or=int(rs.max())))
        del sets
    g.destroy()
    print(json.dumps({"rows": "the vocab pass alone, back to back, on rows that defeat its filter", "shape": w.name,
                      "launches_timed": 2 * args.steps, "times": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="M", choices=sorted(gi.WORKLOADS))
    ap.add_argument("--impl", default="graft", choices=["graft", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--timing-every", type=int, default=16,
                    help="record the per-kernel events on every n-th timed step (at least; steps/32 in a long run)")
    ap.add_argument("--cuda-graph", action="store_true", help="replay captured rounds in the timed loop")
    ap.add_argument("--edge-rows", type=int, default=None,
                    help="depths scored ahead of the expansion (default: the library's)")
    ap.add_argument("--overlap-verifier-ms", type=float, default=None,
                    help="instead of the benchmark: two micro-batches on two streams around a stub verifier of this "
                         "duration, sequential against overlapped schedule")
    ap.add_argument("--tdes-loss", action="store_true",
                    help="instead of the benchmark: time the TDES training objective (forward + backward)")
    ap.add_argument("--saba-fit", action="store_true",
                    help="instead of the benchmark: time the least-squares fit of the SABA models")
    ap.add_argument("--styles", action="store_true",
                    help="instead of the benchmark: the round's kernels timed on degenerate inputs (own JSON line)")
    ap.add_argument("--styles-beta", type=float, default=None,
                    help="with --styles: the weight of the edge scores instead of the workload's (0: none, as in DDTree)")
    ap.add_argument("--rows", action="store_true",
                    help="instead of the benchmark: the vocab pass timed on rows that defeat its filter (own JSON line)")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the benchmark: fixed-budget / beta sweeps on synthetic acceptance (own JSON line)")
    ap.add_argument("--sweep-fixed-budget", type=int, default=256, help="the fixed budget of the DDTree-style arms")
    args = ap.parse_args()
    if args.styles and args.impl == "graft":
        args.steps = 20 if args.steps is None else args.steps
        run_styles(args)
        return
    if args.rows and args.impl == "graft":
        args.steps = 10 if args.steps is None else args.steps
        run_rows(args)
        return
    if args.sweep and args.impl == "graft":
        if "--workload" not in sys.argv:
            args.workload = "C5"
        args.steps = 20 if args.steps is None else args.steps
        run_sweep(args)
        return
    if args.saba_fit and args.impl == "graft":
        run_saba_fit(args)
        return
    if args.tdes_loss and args.impl == "graft":
        run_tdes_loss(args)
        return
    if args.overlap_verifier_ms is not None and args.impl == "graft":
        args.steps = 200 if args.steps is None else args.steps
        run_overlap(args)
        return
    if args.impl == "reference":
        args.steps = 10 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 1000 if args.steps is None else args.steps
        args.warmup = max(3, 20 if args.warmup is None else args.warmup)
        try:
            run_graft(args)
        finally:
            import torch.distributed as dist
            if dist.is_available() and dist.is_initialized():
                dist.destroy_process_group()


if __name__ == "__main__":
    main()
