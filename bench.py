#!/usr/bin/env python
"""Benchmark of the eventually consistent collectives on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]

One "step" is one epoch of the headline workload (P=16 ranks, n=2^24 fp32 per
rank, segments of 65536 elements, seeded three-round arrival schedule): a reset
and three ec_allreduce_apply calls - the first produces the partial result from
what has arrived, the next two fold the late segments in.  The metric is the
algorithmic GB/s of those applies: bytes of every newly folded (rank, segment)
plus bytes of result written (and read back, for segments that already held a
partial result), computed from the actual masks.

Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank runs an
independent replica on its own GPU - the path has no exchange between GPUs -
and the line reports the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

HEADLINE = dict(P=16, n=1 << 24, seg=65536, p_first=0.7, seed=1002, seed_sched=2002)
NOMINAL_HBM_GBS = 8000.0
WORKLOAD = "config 2: P=16 x n=2^24 fp32 N(0,1), seg 65536, sum, 3-round arrival schedule; step = reset + 3 applies"

# dram__bytes_read.sum + dram__bytes_write.sum of the three apply launches of one headline epoch, from one
# one-pass ncu capture that leaves the caches alone: reads 750.4 + 192.2 + 212.9 MB, writes 66.5 + 36.2 + 38.7 MB.
# Below the algorithmic bytes because about half of the 64 MiB result is found in L2 by the next round.  A stored
# value, not measured by this run (the line says so in roofline.traffic_source).
NCU_TRAFFIC_BYTES_PER_EPOCH = 1_296_705_920


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------------------------
# algorithmic bytes of one apply, from the masks
# --------------------------------------------------------------------------------------------
def popcount64(a: np.ndarray) -> np.ndarray:
    a = a.astype(np.uint64)
    c = np.zeros(a.shape, dtype=np.int64)
    for b in range(64):
        c += ((a >> np.uint64(b)) & np.uint64(1)).astype(np.int64)
    return c


def apply_bytes(prev_mask, mask, P, n, seg, in_bytes, out_bytes, first_apply):
    """Bytes one apply must move: inputs of the newly notified (rank, segment) pairs, the result
    segments it writes, and the result segments it first reads (those that held a partial result)."""
    S = (n + seg - 1) // seg
    seg_len = np.minimum(seg, n - np.arange(S) * seg).astype(np.int64)
    if mask is None:
        mask = np.full((S, (P + 63) // 64), np.uint64(2 ** 64 - 1))
        if P % 64:
            mask[:, -1] = np.uint64((1 << (P % 64)) - 1)
    prev = np.zeros_like(mask) if prev_mask is None else prev_mask
    new = mask & ~prev
    n_new = popcount64(new).sum(axis=1)
    had = popcount64(prev).sum(axis=1) > 0
    written = (n_new > 0) | (first_apply & ~had)
    read_back = (n_new > 0) & had
    total = (n_new * seg_len * in_bytes).sum() + (written * seg_len * out_bytes).sum() \
        + (read_back * seg_len * out_bytes).sum()
    words = mask.size * 8 * 2 + S * 4
    return int(total + words)


# --------------------------------------------------------------------------------------------
# clocks during the timed region
# --------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines: list[str] = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def wait_first(self, timeout=8.0):
        """Block until nvidia-smi has produced a sample (it takes a moment to start)."""
        t0 = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - t0 < timeout:
            time.sleep(0.02)

    def stop(self, t_begin=None, t_end=None) -> dict:
        """Summary of the samples taken inside [t_begin, t_end] (host clock); if the window is too
        short to hold three samples, of every sample since the sampler started (warm-up included)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = []
        for ts, line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                rows.append((ts, float(f[1]), float(f[2]), float(f[3]), f[5:9]))
            except ValueError:
                continue
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        window = "timed region"
        if len(inside) < 3:
            inside, window = rows, "warm-up + timed region + end-to-end leg (timed region shorter than 3 samples)"
        reasons = set()
        for r in inside:
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        busy = [r for r in inside if r[3] > 300.0] or inside        # samples under load (power well above idle)
        return {"sm_mhz": statistics.median(r[1] for r in busy) if busy else None,
                "sm_max_mhz": max(r[2] for r in inside) if inside else None,
                "power_w_max": max(r[3] for r in inside) if inside else None,
                "reasons": sorted(reasons), "samples": len(inside), "window": window}


# --------------------------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------------------------
def make_headline_host(scale_n=None):
    from paper_2203_17063_b200 import inputs
    cfg = dict(HEADLINE)
    if scale_n:
        cfg["n"] = scale_n
    S = (cfg["n"] + cfg["seg"] - 1) // cfg["seg"]
    bufs = inputs.rank_buffers("normal_f32", cfg["seed"], cfg["P"], cfg["n"])
    rounds = inputs.arrival_rounds(cfg["seed_sched"], cfg["P"], S, cfg["p_first"])
    masks = inputs.cumulative_masks(rounds)
    return cfg, bufs, masks


def epoch_bytes(cfg, masks, in_b=4, out_b=4):
    per_round, prev = [], None
    for t, m in enumerate(masks):
        per_round.append(apply_bytes(prev, m, cfg["P"], cfg["n"], cfg["seg"], in_b, out_b, t == 0))
        prev = m
    return per_round


def ev_ms(pairs):
    return [a.elapsed_time(b) for a, b in pairs]


def mean_ci(xs):
    m = statistics.fmean(xs)
    if len(xs) < 2:
        return m, 0.0
    return m, 1.96 * statistics.stdev(xs) / (len(xs) ** 0.5)


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2203_17063_b200 import binding as ec

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    from paper_2203_17063_b200.replicas import Replicas
    rep = Replicas(backend="nccl", device=dev)     # N independent replicas; shared: barrier, max time, summed work
    barrier = rep.barrier

    peak, peak_kind = measured_peaks()
    cfg, h_bufs, h_masks = make_headline_host()
    P, n, seg = cfg["P"], cfg["n"], cfg["seg"]
    S = n // seg
    per_round_bytes = epoch_bytes(cfg, h_masks)
    step_bytes = sum(per_round_bytes)

    stream = torch.cuda.Stream(device=dev)
    st = stream.cuda_stream
    # pinned host copies (the end-to-end leg copies from these every step)
    pin_bufs = [torch.from_numpy(b).pin_memory() for b in h_bufs]
    d_bufs = [t.to(dev) for t in pin_bufs]
    d_masks = [torch.from_numpy(m.view(np.int64)).to(dev) for m in h_masks]
    d_res = torch.empty(n, dtype=torch.float32, device=dev)
    d_cnt = torch.empty(S, dtype=torch.int32, device=dev)
    pin_res = torch.empty(n, dtype=torch.float32).pin_memory()
    pin_cnt = torch.empty(S, dtype=torch.int32).pin_memory()
    ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg, device=dev)
    if args.threads or args.tile:
        ar.set_tile(args.threads, args.tile)
    if args.apply_path == "direct":
        ar.set_path(0)
    table = (C.c_void_p * P)(*[t.data_ptr() for t in d_bufs])
    L = ec.lib()

    def epoch(events=None):
        L.ec_allreduce_reset(ar._h, st)
        for t in range(len(d_masks)):
            if events is not None:
                events[t][0].record(stream)
            rc = ar.apply_raw(table, d_masks[t].data_ptr(), d_res.data_ptr(), d_cnt.data_ptr(), st)
            if events is not None:
                events[t][1].record(stream)
            if rc != 0:
                raise ec.EcError(rc, "ec_allreduce_apply")

    with torch.cuda.stream(stream):
        clocks = ClockSampler(local_rank)
        clocks.start()
        clocks.wait_first()
        for _ in range(args.warmup):
            epoch()
        barrier()
        t_host0 = time.perf_counter()
        K = args.steps
        # The timed region: exactly K steps between two events, nothing else in the stream (an event between two launches
        # keeps the second from starting as a programmatic dependent of the first and costs about a tenth of a step).
        t_all0 = torch.cuda.Event(enable_timing=True)
        t_all1 = torch.cuda.Event(enable_timing=True)
        t_all0.record(stream)
        for k in range(K):
            epoch()
        t_all1.record(stream)
        barrier()
        # Right after it, the same steps once more with an event around every launch and every step: kernel durations
        # for the roofline, step times for the confidence interval.  Every step when K <= 32, else every 8th.
        SAMPLE = 1 if K <= 32 else 8
        sampled = [k for k in range(K) if k % SAMPLE == 0]
        step_ev = {k: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for k in sampled}
        apply_ev = {k: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                        for _ in d_masks] for k in sampled}
        for k in range(K):
            if k in step_ev:
                step_ev[k][0].record(stream)
                epoch(apply_ev[k])
                step_ev[k][1].record(stream)
            else:
                epoch()
        barrier()
        t_host1 = time.perf_counter()
    if args.profile_only:
        clocks.stop()
        if rank == 0:
            print(json.dumps({"profile_only": True, "steps": K, "ms_per_step": t_all0.elapsed_time(t_all1) / K}))
        return
    total_ms = t_all0.elapsed_time(t_all1)
    steps_ms = ev_ms(list(step_ev.values()))
    round_ms = [[a.elapsed_time(b) for a, b in ev] for ev in apply_ev.values()]   # [sampled steps][rounds]
    kernel_ms_total = sum(sum(r) for r in round_ms)
    launches = K * len(d_masks)

    # ---- end to end: host buffers in, result out, copies inside the timed region ------------------
    e2e_steps = max(3, min(10, K))
    h2d = sum(t.numel() * t.element_size() for t in pin_bufs) + sum(m.numel() * 8 for m in d_masks)
    d2h = pin_res.numel() * 4 + pin_cnt.numel() * 4
    pin_masks = [torch.from_numpy(m.view(np.int64)).pin_memory() for m in h_masks]
    # One ec_allreduce_epoch_host call per step: it uploads the P host buffers and the masks, runs the epoch and reads
    # the result back, all on one stream.  Two streams (each with its context, staging area and host result) alternate,
    # so that the read-back of one step runs while the next step's uploads are under way (PCIe carries both directions).
    rounds = len(pin_masks)
    lanes = []
    for i in range(2):
        a_i = ar if i == 0 else ec.Allreduce(P, n, ec.F32, ec.SUM, seg, device=dev)
        if i and (args.threads or args.tile):
            a_i.set_tile(args.threads, args.tile)
        if i and args.apply_path == "direct":
            a_i.set_path(0)
        nbytes = a_i.host_staging_bytes(rounds)
        lanes.append({
            "ar": a_i, "stream": stream if i == 0 else torch.cuda.Stream(device=dev),
            "staging": torch.empty(nbytes, dtype=torch.uint8, device=dev), "bytes": nbytes,
            "res": pin_res if i == 0 else torch.empty_like(pin_res).pin_memory(),
            "cnt": pin_cnt if i == 0 else torch.empty_like(pin_cnt).pin_memory(),
            "done": torch.cuda.Event()})
    host_table = (C.c_void_p * P)(*[t.data_ptr() for t in pin_bufs])
    mask_table = (C.c_void_p * rounds)(*[t.data_ptr() for t in pin_masks])

    def e2e_epoch(i):
        ln = lanes[i & 1]
        rc = ln["ar"].epoch_host_raw(host_table, mask_table, rounds, ln["res"].data_ptr(), ln["cnt"].data_ptr(),
                                     ln["staging"].data_ptr(), ln["bytes"], ln["stream"].cuda_stream)
        if rc != 0:
            raise ec.EcError(rc, "ec_allreduce_epoch_host")
        ln["done"].record(ln["stream"])

    torch.cuda.synchronize(dev)
    e2e_epoch(0)
    e2e_epoch(1)
    torch.cuda.synchronize(dev)
    if not (torch.equal(lanes[0]["res"], lanes[1]["res"]) and torch.equal(pin_res, d_res.cpu())):
        raise RuntimeError("end-to-end result differs from the device-resident result")
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    lanes[1]["stream"].wait_event(e0)
    for i in range(e2e_steps):
        e2e_epoch(i)
    stream.wait_event(lanes[0]["done"])
    stream.wait_event(lanes[1]["done"])                      # the last results have reached the host
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    clock_info = clocks.stop(t_host0, t_host1)

    max_over_ranks = rep.max
    total_ms_max = max_over_ranks(total_ms)
    e2e_ms_max = max_over_ranks(e2e_ms)
    value = world * step_bytes * K / (total_ms_max * 1e-3) / 1e9
    e2e_value = world * step_bytes / (e2e_ms_max * 1e-3) / 1e9
    achieved = step_bytes * len(round_ms) / (kernel_ms_total * 1e-3) / 1e9
    m_step, ci_step = mean_ci(steps_ms)

    line = {
        "metric": "ec_allreduce_apply_GBps",
        "value": round(value, 2),
        "unit": "GB/s",
        "n_gpus": world,
        "steps": K,
        "warmup": args.warmup,
        "ms_per_step": round(total_ms_max / K, 5),
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "f32",
        "data": "synthetic",
        "config": {
            "workload": WORKLOAD,
            "schedule": "fixed rank order; each (rank, segment) arrives in round 1 with probability 0.7, else in round 2 or 3",
            "parallelism": "replicas only (no exchange between GPUs)" if world > 1 else "1 GPU",
            "algorithmic_bytes_per_step": step_bytes,
            "algorithmic_bytes_per_round": per_round_bytes,
            "elements_per_s": round(world * n * K / (total_ms_max * 1e-3), 1),
            "input_elements_per_s": round(world * P * n * K / (total_ms_max * 1e-3), 1),
            "l2": "rank buffers (1 GiB) exceed L2 every step; the 64 MiB result is carried between rounds as in the workload",
            "ms_per_step_mean_ci95": [round(m_step, 5), round(ci_step, 5)],
            "ms_per_step_median_min": [round(statistics.median(steps_ms), 5), round(min(steps_ms), 5)],
            "timing": f"value: two events around the {K} timed steps, nothing else in the stream; the per-launch and per-step "
                      f"events (roofline, confidence interval) come from the same {K} steps run once more right after, "
                      + ("an event pair on every step" if SAMPLE == 1 else f"an event pair on every {SAMPLE}th step")
                      + " (events between the launches cost about a tenth of a step: ms_per_step_mean_ci95 includes them)",
            "ms_per_round_mean": [round(statistics.fmean(r[t] for r in round_ms), 5) for t in range(len(d_masks))],
            "GBps_per_round": [round(per_round_bytes[t] / (statistics.fmean(r[t] for r in round_ms) * 1e-3) / 1e9, 1)
                               for t in range(len(d_masks))],
        },
        "roofline": {
            "bound": "hbm",
            "kernel": "apply_bulk_kernel<f32,sum> (all three launches of an epoch)",
            "achieved": round(achieved, 1),
            "peak": peak,
            "peak_kind": f"of {peak_kind}",
            "unit": "GB/s",
            "frac": round(achieved / peak, 4),
            "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBS, 4),
            "traffic": NCU_TRAFFIC_BYTES_PER_EPOCH // 3,
            "traffic_source": "stored: one ncu capture of this workload's three launches (profiles/), not measured by this run",
            "traffic_note": "DRAM bytes per launch, averaged over the three launches of an epoch; achieved uses the "
                            "algorithmic bytes of the same three launches (they include the re-read of the partial "
                            "result, about half of which L2 serves), achieved_dram the stored DRAM bytes",
            "achieved_dram": round(NCU_TRAFFIC_BYTES_PER_EPOCH * len(round_ms) / (kernel_ms_total * 1e-3) / 1e9, 1),
            "frac_dram_of_measured": round(NCU_TRAFFIC_BYTES_PER_EPOCH * len(round_ms) / (kernel_ms_total * 1e-3) / 1e9 / peak, 4),
            "frac_dram_of_nominal_8TBps": round(NCU_TRAFFIC_BYTES_PER_EPOCH * len(round_ms) / (kernel_ms_total * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
        },
        "e2e": {"value": round(e2e_value, 2), "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_ms_max, 3), "steps": e2e_steps},
        "gpu_launches": launches,
        "clocks": clock_info,
    }

    if rank == 0 and world == 1:
        line["cpu_baseline"] = cpu_baseline(cfg, h_bufs, h_masks, per_round_bytes, budget_s=args.cpu_seconds)
        if not args.no_extras:
            del h_bufs, pin_bufs, d_bufs
            ar.destroy()
            ex = extras(args, dev, stream, peak)
            line["extras"] = ex
            # the results the target names, as plain numbers beside the workload (short keys: they survive truncation)
            c3, c3p, km = ex["config3_P32_bf16_n2^25"], ex["config3_P32_bf16_n2^25_pairwise"], ex["config5_kmeans_N2^22_D32_K64_P64"]
            line["config"].update({
                "cfg2_round_GBps_1": line["config"]["GBps_per_round"][0], "cfg2_round_GBps_2": line["config"]["GBps_per_round"][1],
                "cfg2_round_GBps_3": line["config"]["GBps_per_round"][2],
                "cfg3_P32_bf16_all_at_once_GBps": c3["all_at_once"]["GBps"], "cfg3_all_at_once_frac_8TBps": c3["all_at_once"]["frac_8TBps"],
                "cfg3_all_at_once_frac_measured": c3["all_at_once"]["frac_measured"],
                "cfg3_round_GBps_1": c3["rounds"][0]["GBps"], "cfg3_round_GBps_2": c3["rounds"][1]["GBps"],
                "cfg3_round_GBps_3": c3["rounds"][2]["GBps"],
                "cfg3_round_frac_8TBps_1": round(c3["rounds"][0]["GBps"] / NOMINAL_HBM_GBS, 4),
                "cfg3_round_frac_8TBps_2": round(c3["rounds"][1]["GBps"] / NOMINAL_HBM_GBS, 4),
                "cfg3_round_frac_8TBps_3": round(c3["rounds"][2]["GBps"] / NOMINAL_HBM_GBS, 4),
                "cfg3_pairwise_GBps": c3p["all_at_once"]["GBps"], "cfg3_pairwise_frac_8TBps": c3p["all_at_once"]["frac_8TBps"],
                "cfg5_kmeans_iterations_per_s": km["iterations_per_s"],
                "cfg5_kmeans_every_tile_searched_iterations_per_s": km["iterations_per_s_every_tile_searched"],
                "cfg5_kmeans_every_tile_searched_frac_of_hbm_measured": km["every_tile_searched_frac_of_hbm_measured"],
                "cfg5_kmeans_first_full_iteration_ms": km["first_full_iteration_ms"],
            })
    rep.close()
    if rank == 0:
        print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# the CPU checker as a timed baseline (never tuned for this)
# --------------------------------------------------------------------------------------------
def cpu_baseline(cfg, h_bufs, h_masks, per_round_bytes, budget_s=15.0):
    import oracle
    P, n, seg = cfg["P"], cfg["n"], cfg["seg"]
    threads = oracle.max_threads()
    ref = oracle.Allreduce(P, n, oracle.F32, oracle.SUM, seg)
    res = np.empty(n, dtype=np.float32)
    cnt = np.empty((n + seg - 1) // seg, dtype=np.uint32)
    times = []
    t_start = time.perf_counter()
    while True:
        ref.reset()
        t0 = time.perf_counter()
        for m in h_masks:
            ref.apply(h_bufs, m, res, cnt, threads=threads)
        times.append(time.perf_counter() - t0)
        if time.perf_counter() - t_start > budget_s or len(times) >= 20:
            break
    best = min(times)
    return {"value": round(sum(per_round_bytes) / best / 1e9, 3), "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": f"{len(times)} full epochs of the same workload (n={n}, 3 rounds), best of them; "
                      f"mean {statistics.fmean(times) * 1e3:.1f} ms per epoch",
            "host_cpus": os.cpu_count()}


# --------------------------------------------------------------------------------------------
# the other workloads (reported beside the headline; parity for them is in tests/)
# --------------------------------------------------------------------------------------------
def time_calls(stream, fn, reps, warm=3, before=None):
    import torch
    with torch.cuda.stream(stream):
        for _ in range(warm):
            if before:
                before()
            fn()
        torch.cuda.synchronize()
        evs = []
        for _ in range(reps):
            if before:
                before()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize()
    return ev_ms(evs)


def time_rotating(stream, fns, reps, before=None):
    """Cold-cache timing of a call whose working set fits in L2: the repetitions rotate over `fns`, the same call on
    distinct buffer sets that together exceed twice the L2 capacity, so that every timed call finds none of its data
    cached.  One untimed round over all sets first."""
    import torch
    with torch.cuda.stream(stream):
        for fn in fns:
            if before:
                before()
            fn()
        torch.cuda.synchronize()
        evs = []
        for r in range(reps):
            if before:
                before()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fns[r % len(fns)]()
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize()
    return ev_ms(evs)


L2_BYTES = 126 * 1024 * 1024


def extras(args, dev, stream, peak):
    import torch
    from paper_2203_17063_b200 import binding as ec
    from paper_2203_17063_b200 import inputs
    out = {}
    st = stream.cuda_stream
    L = ec.lib()
    reps = max(10, min(args.steps, 50))

    def allreduce_case(name, P, n, seg, dtype, kind, seed, sched_seed, p_first, last_round, order=ec.ORDER_FIXED, **kw):
        S = (n + seg - 1) // seg
        h = inputs.rank_buffers(kind, seed, P, n, **kw)
        if kind == "normal_bf16":
            d = [torch.from_numpy(b.view(np.int16)).to(dev).view(torch.bfloat16) for b in h]
        else:
            d = [torch.from_numpy(b).to(dev) for b in h]
        del h
        in_b = d[0].element_size()
        out_dt = ec.OUT_TORCH[dtype]
        out_b = torch.empty(0, dtype=out_dt).element_size()
        masks = inputs.cumulative_masks(inputs.arrival_rounds(sched_seed, P, S, p_first, last_round)) if last_round > 1 else [None]
        d_masks = [None if m is None else torch.from_numpy(m.view(np.int64)).to(dev) for m in masks]
        res = torch.empty(n, dtype=out_dt, device=dev)
        cnt = torch.empty(S, dtype=torch.int32, device=dev)
        ar = ec.Allreduce(P, n, dtype, ec.SUM, seg, order, device=dev)
        if args.threads or args.tile:
            ar.set_tile(args.threads, args.tile)
        if args.apply_path == "direct":
            ar.set_path(0)
        table = (C.c_void_p * P)(*[t.data_ptr() for t in d])
        cfgd = dict(P=P, n=n, seg=seg)
        rb = epoch_bytes(cfgd, masks, in_b, out_b) if masks[0] is not None else [apply_bytes(None, None, P, n, seg, in_b, out_b, True)]
        entry = {}
        # all at once
        full_bytes = apply_bytes(None, None, P, n, seg, in_b, out_b, True)
        ms = time_calls(stream, lambda: ar.apply_raw(table, None, res.data_ptr(), cnt.data_ptr(), st), reps,
                        before=lambda: L.ec_allreduce_reset(ar._h, st))
        m, ci = mean_ci(ms)
        entry["all_at_once"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(full_bytes / m / 1e6, 1),
                                "frac_measured": round(full_bytes / m / 1e6 / peak, 4),
                                "frac_8TBps": round(full_bytes / m / 1e6 / NOMINAL_HBM_GBS, 4), "bytes": full_bytes}
        if masks[0] is not None:
            with torch.cuda.stream(stream):
                per = [[] for _ in masks]
                for k in range(reps + 3):
                    L.ec_allreduce_reset(ar._h, st)
                    evs = []
                    for t, dm in enumerate(d_masks):
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record(stream)
                        ar.apply_raw(table, dm.data_ptr(), res.data_ptr(), cnt.data_ptr(), st)
                        b.record(stream)
                        evs.append((a, b))
                    torch.cuda.synchronize()
                    if k >= 3:
                        for t, (a, b) in enumerate(evs):
                            per[t].append(a.elapsed_time(b))
            entry["rounds"] = [{"ms": round(statistics.fmean(p), 5), "GBps": round(rb[t] / statistics.fmean(p) / 1e6, 1),
                                "frac_measured": round(rb[t] / statistics.fmean(p) / 1e6 / peak, 4), "bytes": rb[t]}
                               for t, p in enumerate(per)]
        ar.destroy()
        out[name] = entry

    def ssp_case(name, P, n, seg, seed, sched_seed, p_first):
        """Stale-synchronous apply on the config-2 shape: clocks 10 / 9 / 8 where the three-round schedule has
        rounds 1 / 2 / 3; slack 0, 1, 2 accept about 70 %, 85 %, 100 % of the contributions."""
        S = n // seg
        h = inputs.rank_buffers("normal_f32", seed, P, n)
        d = [torch.from_numpy(b).to(dev) for b in h]
        del h
        rounds = inputs.arrival_rounds(sched_seed, P, S, p_first)
        clocks = (10 - (rounds.T - 1)).astype(np.uint32)
        d_clocks = torch.from_numpy(clocks.view(np.int32)).to(dev)
        res = torch.empty(n, dtype=torch.float32, device=dev)
        cnt = torch.empty(S, dtype=torch.int32, device=dev)
        clk = torch.empty(S, dtype=torch.int32, device=dev)
        wait = torch.empty(S, dtype=torch.int32, device=dev)
        ar = ec.Allreduce(P, n, ec.F32, ec.SUM, seg, device=dev)
        table = (C.c_void_p * P)(*[t.data_ptr() for t in d])
        entry = {}
        for slack in (0, 1, 2):
            accepted = int((clocks >= 10 - slack).sum())
            nbytes = accepted * seg * 4 + n * 4 + S * P * 4 + 3 * S * 4
            ms = time_calls(stream, lambda: L.ec_allreduce_ssp_apply(ar._h, table, P, n, ec.F32, ec.SUM, seg,
                                                                     d_clocks.data_ptr(), 10, slack, res.data_ptr(),
                                                                     cnt.data_ptr(), clk.data_ptr(), wait.data_ptr(), st), reps)
            m, ci = mean_ci(ms)
            entry[f"slack{slack}"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(nbytes / m / 1e6, 1),
                                      "frac_measured": round(nbytes / m / 1e6 / peak, 4), "bytes": nbytes,
                                      "accepted_fraction": round(accepted / (S * P), 4)}
        ar.destroy()
        out[name] = entry

    allreduce_case("config1_P4_f32_n2^20", 4, 1 << 20, 16384, ec.F32, "uniform_f32", 1001, 0, 1.0, 1)
    ssp_case("ssp_apply_P16_f32_n2^24", 16, 1 << 24, 65536, 1002, 2002, 0.7)
    allreduce_case("config2_P16_f32_n2^24_all_at_once", 16, 1 << 24, 65536, ec.F32, "normal_f32", 1002, 2002, 0.7, 1)
    allreduce_case("config3_P32_bf16_n2^25", 32, 1 << 25, 131072, ec.BF16, "normal_bf16", 1003, 2003, 0.9, 3, sigma=1e-3)
    allreduce_case("config3_P32_bf16_n2^25_pairwise", 32, 1 << 25, 131072, ec.BF16, "normal_bf16", 1003, 2003, 0.9, 1,
                   order=ec.ORDER_PAIRWISE, sigma=1e-3)
    allreduce_case("config4_P256_i64_n2^20", 256, 1 << 20, 8192, ec.I64, "int64_below", 1004, 2004, 0.8, 2, bound=1 << 20)

    # config 1 again with a cold cache: 21 MB per call, so 13 buffer sets (> 2 x L2) in rotation
    P, n, seg = 4, 1 << 20, 16384
    nsets = 2 * L2_BYTES // ((P + 1) * n * 4) + 1
    c1_sets = []
    for k in range(nsets):
        bufs = [torch.from_numpy(b).to(dev) for b in inputs.rank_buffers("uniform_f32", 1001 + 7 * k, P, n)]
        c1_sets.append((bufs, (C.c_void_p * P)(*[t.data_ptr() for t in bufs]), torch.empty(n, device=dev)))
    c1_cnt = torch.empty(n // seg, dtype=torch.int32, device=dev)
    ar1 = ec.Allreduce(P, n, ec.F32, ec.SUM, seg, device=dev)
    ms = time_rotating(stream, [(lambda tb=tb, r=r: ar1.apply_raw(tb, None, r.data_ptr(), c1_cnt.data_ptr(), st)) for _, tb, r in c1_sets],
                       reps, before=lambda: L.ec_allreduce_reset(ar1._h, st))
    m, ci = mean_ci(ms)
    c1_bytes = apply_bytes(None, None, P, n, seg, 4, 4, True)
    out["config1_P4_f32_n2^20"]["cold"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(c1_bytes / m / 1e6, 1),
                                           "frac_measured": round(c1_bytes / m / 1e6 / peak, 4), "buffer_sets": nsets}
    out["config1_P4_f32_n2^20"]["all_at_once"]["cache"] = "warm: the 21 MB working set stays in L2 between repetitions"
    ar1.destroy()
    del c1_sets

    # AlltoAll at the paper's largest message size: 64 ranks (16 nodes x 4 processes), 32 KiB per block
    P, B = 64, 32768
    g = torch.Generator(device="cpu").manual_seed(77)
    a_send = [torch.randint(0, 256, (P * B,), dtype=torch.uint8, generator=g).to(dev) for _ in range(P)]
    a_recv = [torch.empty(P * B, dtype=torch.uint8, device=dev) for _ in range(P)]
    a_cnt = torch.empty(P, dtype=torch.int32, device=dev)
    a_mask = torch.from_numpy(inputs.pack_mask(inputs.bernoulli_mask(2006, 0, P, P, 0.8).T.copy()).view(np.int64)).to(dev)
    st_tbl = (C.c_void_p * P)(*[t.data_ptr() for t in a_send])
    rt_tbl = (C.c_void_p * P)(*[t.data_ptr() for t in a_recv])
    entry = {}
    for label, mptr, frac in (("all_arrived", None, 1.0), ("80pct_arrived", a_mask.data_ptr(), None)):
        ms = time_calls(stream, lambda: L.ec_alltoall(st_tbl, rt_tbl, P, B, mptr, a_cnt.data_ptr(), st), reps)
        m, ci = mean_ci(ms)
        blocks = P * P if mptr is None else int(a_cnt.sum().item())
        nbytes = 2 * blocks * B
        entry[label] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(nbytes / m / 1e6, 1),
                        "frac_measured": round(nbytes / m / 1e6 / peak, 4), "bytes": nbytes}
    entry["note"] = "read + write of every notified block; 2 x 128 MiB working set, partly L2-resident when repeated (warm)"
    a_send2 = [t.clone() for t in a_send]
    a_recv2 = [torch.empty_like(t) for t in a_recv]
    st_tbl2 = (C.c_void_p * P)(*[t.data_ptr() for t in a_send2])
    rt_tbl2 = (C.c_void_p * P)(*[t.data_ptr() for t in a_recv2])
    ms = time_rotating(stream, [lambda: L.ec_alltoall(st_tbl, rt_tbl, P, B, None, a_cnt.data_ptr(), st),
                                lambda: L.ec_alltoall(st_tbl2, rt_tbl2, P, B, None, a_cnt.data_ptr(), st)], reps)
    m, ci = mean_ci(ms)
    nbytes = 2 * P * P * B
    entry["all_arrived_cold"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(nbytes / m / 1e6, 1),
                                 "frac_measured": round(nbytes / m / 1e6 / peak, 4), "bytes": nbytes,
                                 "buffer_sets": 2, "note": "two 256 MiB buffer sets in rotation: nothing of a call's data is in L2"}
    out["alltoall_P64_32KiB_blocks"] = entry
    del a_send, a_recv, a_send2, a_recv2

    # Broadcast with the paper's data thresholds (a quarter, half, three quarters, all of the vector): 16 ranks, 64 MiB
    P, n, seg = 16, 1 << 24, 65536
    b_src = torch.randn(n, device=dev)
    b_dst = [b_src if r == 0 else torch.empty(n, device=dev) for r in range(P)]
    b_words = torch.empty(n // seg, dtype=torch.int64, device=dev)
    b_tbl = (C.c_void_p * P)(*[t.data_ptr() for t in b_dst])
    entry = {}
    for frac in (0.25, 0.5, 0.75, 1.0):
        ms = time_calls(stream, lambda: L.ec_bcast(b_src.data_ptr(), b_tbl, P, 0, n, ec.F32, seg, frac,
                                                   b_words.data_ptr(), st), reps)
        m, ci = mean_ci(ms)
        nbytes = int(frac * n) * 4 * P                      # read once, written P - 1 times
        entry[f"threshold_{int(frac * 100)}"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(nbytes / m / 1e6, 1),
                                                 "frac_measured": round(nbytes / m / 1e6 / peak, 4), "bytes": nbytes}
    entry["note"] = "root in place; bytes = delivered prefix read once + written to 15 receive buffers"
    out["bcast_P16_f32_n2^24"] = entry
    del b_src, b_dst

    # config 4 gather
    P = 256
    counts = inputs.gather_counts(1004, P)
    hb = inputs.gather_buffers(1004, counts)
    arrived = inputs.bernoulli_mask(2004, 0, P, 1, 0.8)[:, 0]
    db = [torch.from_numpy(b).to(dev) for b in hb]
    total = int(counts.sum())
    d_counts = torch.from_numpy(counts).to(dev)
    d_mask = torch.from_numpy(inputs.pack_mask(arrived[:, None]).reshape(-1).view(np.int64)).to(dev)
    d_displs = torch.empty(P + 1, dtype=torch.int64, device=dev)
    d_out = torch.empty(total, dtype=torch.int64, device=dev)
    d_status = torch.empty(1, dtype=torch.int32, device=dev)
    table = (C.c_void_p * P)(*[t.data_ptr() for t in db])
    gbytes = 2 * 8 * int(counts[arrived].sum()) + P * 8 * 2
    ms = time_calls(stream, lambda: L.ec_allgatherv(table, d_counts.data_ptr(), P, ec.I64, d_mask.data_ptr(),
                                                    d_displs.data_ptr(), d_out.data_ptr(), total,
                                                    d_status.data_ptr(), st), reps)
    m, ci = mean_ci(ms)
    out["config4_allgatherv_P256_i64"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(gbytes / m / 1e6, 1),
                                          "frac_measured": round(gbytes / m / 1e6 / peak, 4),
                                          "bytes": gbytes, "note": "warm: the 109 MB working set is L2-resident when repeated"}
    g_sets = [(table, d_out)]
    for k in range(3):
        db_k = [t.clone() for t in db]
        g_sets.append(((C.c_void_p * P)(*[t.data_ptr() for t in db_k]), torch.empty_like(d_out), db_k))
    ms = time_rotating(stream, [(lambda tb=gs[0], o=gs[1]: L.ec_allgatherv(tb, d_counts.data_ptr(), P, ec.I64, d_mask.data_ptr(),
                                                                           d_displs.data_ptr(), o.data_ptr(), total,
                                                                           d_status.data_ptr(), st)) for gs in g_sets], reps)
    m, ci = mean_ci(ms)
    out["config4_allgatherv_P256_i64"]["cold"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(gbytes / m / 1e6, 1),
                                                  "frac_measured": round(gbytes / m / 1e6 / peak, 4), "buffer_sets": len(g_sets)}
    # a gather large enough to be cold by itself: the same counts x 8 (about 870 MB moved)
    counts8 = counts * 8
    big = [torch.empty(int(c), dtype=torch.int64, device=dev).random_() for c in counts8]
    total8 = int(counts8.sum())
    d_counts8 = torch.from_numpy(counts8).to(dev)
    d_out8 = torch.empty(total8, dtype=torch.int64, device=dev)
    table8 = (C.c_void_p * P)(*[t.data_ptr() for t in big])
    gbytes8 = 2 * 8 * int(counts8[arrived].sum()) + P * 8 * 2
    ms = time_calls(stream, lambda: L.ec_allgatherv(table8, d_counts8.data_ptr(), P, ec.I64, d_mask.data_ptr(),
                                                    d_displs.data_ptr(), d_out8.data_ptr(), total8,
                                                    d_status.data_ptr(), st), reps)
    m, ci = mean_ci(ms)
    out["config4_allgatherv_P256_i64"]["counts_x8"] = {"ms": round(m, 5), "ci95": round(ci, 5), "GBps": round(gbytes8 / m / 1e6, 1),
                                                       "frac_measured": round(gbytes8 / m / 1e6 / peak, 4), "bytes": gbytes8}
    del db, d_out, g_sets, big, d_out8

    # The allreduce inside a config 5 iteration on its own: 64 ranks x 64 centroid rows of 36 floats (590 KB), one row a
    # segment, arrival probability 0.75.  Warm (everything in L2, as between the kernels of an iteration) and cold (a
    # buffer of twice the L2 size is overwritten before every timed call).
    P, Kc, Dc = 64, 64, 32
    n5, seg5 = Kc * (Dc + 4), Dc + 4
    rows5 = torch.randn(P, n5, device=dev)
    tab5 = (C.c_void_p * P)(*[rows5[r].data_ptr() for r in range(P)])
    mask5 = torch.from_numpy(inputs.pack_mask(inputs.bernoulli_mask(2005, 0, P, Kc, 0.75)).view(np.int64)).to(dev)
    res5 = torch.empty(n5, device=dev)
    cnt5 = torch.empty(Kc, dtype=torch.int32, device=dev)
    ar5 = ec.Allreduce(P, n5, ec.F32, ec.SUM, seg5, device=dev)
    call5 = lambda: ar5.apply_raw(tab5, mask5.data_ptr(), res5.data_ptr(), cnt5.data_ptr(), st)
    reset5 = lambda: L.ec_allreduce_reset(ar5._h, st)
    bytes5 = int(0.75 * P * n5 * 4) + n5 * 4 + Kc * 4
    entry = {"bytes_about": bytes5}
    ms = time_rotating(stream, [call5], reps, before=reset5)
    m, ci = mean_ci(ms)
    entry["warm"] = {"us": round(m * 1e3, 2), "ci95_us": round(ci * 1e3, 2), "GBps": round(bytes5 / m / 1e6, 1)}
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
    def cold_before():
        flush.fill_(1)
        reset5()
    ms = time_rotating(stream, [call5], reps, before=cold_before)
    m, ci = mean_ci(ms)
    entry["cold"] = {"us": round(m * 1e3, 2), "ci95_us": round(ci * 1e3, 2), "GBps": round(bytes5 / m / 1e6, 1),
                     "how": "252 MB written before every timed call"}
    entry["note"] = "a launch with three dependent trips to memory: latency, not bandwidth"
    out["config5_allreduce_P64_K64_D32"] = entry
    ar5.destroy()
    del flush, rows5

    out["config5_kmeans_N2^22_D32_K64_P64"] = kmeans_case(dev, stream, reps=5)
    out["mf_ssp_U2^17_I2^14_k32_nnz2^23_P16"] = mf_case(dev, stream)
    return out


def mf_case(dev, stream, iters=20):
    """Matrix factorisation over the stale-synchronous allreduce (stands in for the paper's MovieLens experiment):
    2^17 users, 2^14 items, 32 factors, 2^23 synthetic ratings, 16 ranks, item segments of 64 rows; each
    contribution is delivered fresh with probability 0.5, otherwise reused until it is older than the slack."""
    import torch
    from paper_2203_17063_b200 import binding as ec
    from paper_2203_17063_b200 import inputs
    U, I, k, nnz, P, seg_rows = 1 << 17, 1 << 14, 32, 1 << 23, 16, 64
    d = inputs.mf_ratings(1006, U, I, 16, nnz, P)
    pu, qi = inputs.mf_init_factors(1006, U, I, k, 0.3)
    dd = {key: torch.from_numpy(d[key]).to(dev) for key in ("user_ptr", "user_item", "user_val", "rank_item_ptr",
                                                             "item_user", "item_val")}
    d_pu, d_qi = torch.from_numpy(pu).to(dev), torch.from_numpy(qi).to(dev)
    S = (I + seg_rows - 1) // seg_rows
    masks = [torch.from_numpy(m.view(np.int64)).to(dev) for m in inputs.mf_refresh_masks(2006, iters + 2, P, S, 0.5)]
    key_after = f"mse_after_{iters}_iterations"
    sse = torch.empty(1, dtype=torch.float64, device=dev)
    out = {}
    for label, slack, use_masks in (("synchronous", 0, False), ("slack1_half_fresh", 1, True), ("slack2_half_fresh", 2, True)):
        mf = ec.MatrixFactorization(dd, U, I, P, d_pu, d_qi, 1e-3, 0.05, seg_rows)
        with torch.cuda.stream(stream):
            for t in range(2):
                mf.iterate(masks[t] if use_masks else None, slack, stream)
            mf.get(sse=sse, stream=stream)
            torch.cuda.synchronize()
            mse0 = float(sse.item()) / nnz
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for t in range(iters):
                mf.iterate(masks[t + 2] if use_masks else None, slack, stream)
            b.record(stream)
            mf.get(sse=sse, stream=stream)
            torch.cuda.synchronize()
        ms = a.elapsed_time(b)
        out[label] = {"iterations_per_s": round(iters / (ms * 1e-3), 1), "ms_per_iteration": round(ms / iters, 4),
                      "mse_before": round(mse0, 5), key_after: round(float(sse.item()) / nnz, 5)}
        mf.destroy()
    out["note"] = ("5 launches per iteration: refresh decision, item gradients of the refreshed (rank, segment) pairs, "
                   "ec_allreduce_ssp_apply over 16 x 2 MiB, user step, item step; mse = mean squared error at the start "
                   "of the last iteration")
    return out


def kmeans_case(dev, stream, reps=5, iters=20, profile_only=False, bounds=True, refresh=32):
    """Config 5: N = 2^22 points, D = 32, K = 64, P = 64 ranks, 20 Lloyd iterations with seeded masks."""
    import torch
    from paper_2203_17063_b200 import binding as ec
    from paper_2203_17063_b200 import inputs
    st = stream.cuda_stream
    N, D, K, P = 1 << 22, 32, 64, 64
    pts, comp, _ = inputs.kmeans_mixture(1005, N, D, K)
    init = inputs.kmeans_first_of_component(pts, comp, K)
    masks = [torch.from_numpy(m.view(np.int64)).to(dev) for m in inputs.kmeans_masks(2005, iters, P, K, 0.75)]
    d_pts = torch.from_numpy(pts).to(dev)
    d_init = torch.from_numpy(init).to(dev)
    km = ec.KMeans(d_pts, K, P, d_init)
    if profile_only:                 # which leg a profiler capture looks at: distance bounds on / off, sums afresh every `refresh`
        km.set_bounds(bounds)
        km.set_refresh(refresh)
    with torch.cuda.stream(stream):
        for t in range(3):
            km.iterate_raw(masks[t].data_ptr(), st)
        runs = []
        first_ms = []
        for rep in range(reps):
            km.set_centroids(d_init, stream)
            km.set_refresh(refresh)     # forgets labels and running sums: every repetition is a fresh run of 20 iterations
            a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            a.record(stream)
            km.iterate_raw(masks[0].data_ptr(), st)
            c.record(stream)
            for t in range(1, iters):
                km.iterate_raw(masks[t].data_ptr(), st)
            b.record(stream)
            torch.cuda.synchronize()
            runs.append(a.elapsed_time(b))
            first_ms.append(a.elapsed_time(c))
        if profile_only:
            km.destroy()
            return {"ms_per_iteration": statistics.fmean(runs) / iters}
        lab = torch.empty(N, dtype=torch.int32, device=dev)
        ms_assign = time_calls(stream, lambda: km.assign(d_init, lab, stream), 10)
        part = torch.empty(P, K, D + 4, device=dev)
        ms_part = time_calls(stream, lambda: km.partials(lab, part, stream), 10)
        # the same 20 iterations with every tile searched in every iteration (the distance bounds switched off)
        km.set_bounds(False)
        km.set_centroids(d_init, stream)
        km.iterate_raw(masks[0].data_ptr(), st)      # (the full first iteration is reported on its own: not in this leg)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for t in range(iters):
            km.iterate_raw(masks[t].data_ptr(), st)
        b.record(stream)
        torch.cuda.synchronize()
        ms_no_bounds = a.elapsed_time(b)
        # ... and with every iteration summing all points as well (the running sums switched off, too)
        km.set_refresh(1)
        km.set_centroids(d_init, stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for t in range(iters):
            km.iterate_raw(masks[t].data_ptr(), st)
        b.record(stream)
        torch.cuda.synchronize()
        ms_full_sums = a.elapsed_time(b)
        km.set_refresh(32)
        km.set_bounds(True)
        # the same 20 iterations with the candidate search on the fp32 pipes instead of the tensor cores
        km.set_path(1)
        km.set_centroids(d_init, stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for t in range(iters):
            km.iterate_raw(masks[t].data_ptr(), st)
        b.record(stream)
        torch.cuda.synchronize()
        ms_fp32_path = a.elapsed_time(b)
        km.set_path(0)
        tc_status = km.tc_status(stream)
        km.destroy()
        del d_pts
        churn = kmeans_churn_leg(dev, stream, N, D, K, P, iters, masks)
    m, ci = mean_ci(runs)
    peak, _ = measured_peaks()
    iter_bytes = N * D * 4 + N * 4            # the points once, the labels once (centroids and partial rows are < 1 %)
    res = {
        "iterations_per_s": round(iters / (m * 1e-3), 1), "ms_per_20_iterations": round(m, 3), "ci95": round(ci, 3),
        "first_full_iteration_ms": round(statistics.fmean(first_ms), 4),
        "timed": "every repetition is a fresh run: labels and running sums forgotten, so its first iteration searches and "
                 "sums every point; every_tile_searched: 20 iterations after one untimed full one",
        "what_iterations_per_s_is": "the library's default: every iteration produces the labels, sums and centroids of a full Lloyd "
                                    "iteration (bit-identical to the legs below, tested), but tiles whose distance bounds prove that no "
                                    "label can change are not searched again; the two legs below switch that off",
        "path": "tensor cores (bulk tensor copies, tcgen05 tf32 candidate search + bf16 one-hot sums GEMM, exact fp32 re-decision); "
                "iterations after the first sum only the points whose label changed and search only the tiles whose distance "
                "bounds allow a change",
        "overlapping_mixture": churn,
        "tensor_core_status_word": tc_status,
        "iterations_per_s_every_tile_searched": round(iters / (ms_no_bounds * 1e-3), 1),
        "every_tile_searched_iteration_GBps": round(iter_bytes / (ms_no_bounds / iters) / 1e6, 1),
        "every_tile_searched_frac_of_hbm_measured": round(iter_bytes / (ms_no_bounds / iters) / 1e6 / peak, 4),
        "iterations_per_s_all_points_summed_every_iteration": round(iters / (ms_full_sums * 1e-3), 1),
        "assign_only_ms": round(statistics.fmean(ms_assign), 4),
        "standalone_partials_ms": round(statistics.fmean(ms_part), 4),
        "fp32_path_iterations_per_s": round(iters / (ms_fp32_path * 1e-3), 1),
        "note": "on this well-separated mixture the labels settle after the first iteration, so the later ones read 12 bytes of "
                "bounds and label per point instead of the points; with every tile searched an iteration is bound by HBM "
                "(537 MB of points + 17 MB of labels); the fp32 path is bound by the FMA pipe "
                "(N*K*D fused multiply-adds = 0.23 ms at 148 SMs x 128 lanes x 1.965 GHz)",
    }
    return res


def kmeans_churn_leg(dev, stream, N, D, K, P, iters, masks):
    """The same shape on a mixture whose components overlap (centres in a box of 2.5 instead of 10, start from K random
    points): labels keep moving, so the running sums and the distance bounds have work to do in every iteration."""
    import torch
    from paper_2203_17063_b200 import binding as ec
    from paper_2203_17063_b200 import inputs
    st = stream.cuda_stream
    pts, _, _ = inputs.kmeans_mixture(3005, N, D, K, sigma=1.0, box=2.5)
    init = pts[np.random.default_rng(3006).choice(N, K, replace=False)].copy()
    d_pts = torch.from_numpy(pts).to(dev)
    d_init = torch.from_numpy(init).to(dev)
    km = ec.KMeans(d_pts, K, P, d_init)
    out = {}
    lab_a = torch.empty(N, dtype=torch.int32, device=dev)
    lab_b = torch.empty(N, dtype=torch.int32, device=dev)
    for label, bounds in (("bounds_on", True), ("bounds_off", False)):
        km.set_bounds(bounds)
        km.set_centroids(d_init, stream)
        km.set_refresh(32)
        moved = []
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for t in range(iters):
            km.iterate_raw(masks[t].data_ptr(), st)
        b.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(b)
        if bounds:                                # how many labels move per iteration (a second, untimed run)
            km.set_centroids(d_init, stream)
            km.set_refresh(32)
            for t in range(iters):
                km.iterate_raw(masks[t].data_ptr(), st)
                km.get(labels=lab_a if t % 2 == 0 else lab_b, stream=stream)
                if t:
                    moved.append(float((lab_a != lab_b).float().mean().item()))
            out["labels_moved_per_iteration_min_median_max"] = [round(min(moved), 5), round(statistics.median(moved), 5), round(max(moved), 5)]
        out[label + "_iterations_per_s"] = round(iters / (ms * 1e-3), 1)
    km.destroy()
    return out


# --------------------------------------------------------------------------------------------
# reference arm: the CPU checker, timed as it stands on the host cores
# --------------------------------------------------------------------------------------------
def run_reference(args, rank):
    if rank != 0:
        return
    # the same workload at its full size: every step one whole 3-round epoch (about 15-20 ms on 16 cores)
    cfg, h_bufs, h_masks = make_headline_host()
    per_round = epoch_bytes(cfg, h_masks)
    import oracle
    threads = oracle.max_threads()
    ref = oracle.Allreduce(cfg["P"], cfg["n"], oracle.F32, oracle.SUM, cfg["seg"])
    res = np.empty(cfg["n"], dtype=np.float32)
    cnt = np.empty((cfg["n"] + cfg["seg"] - 1) // cfg["seg"], dtype=np.uint32)

    def epoch():
        ref.reset()
        for m in h_masks:
            ref.apply(h_bufs, m, res, cnt, threads=threads)

    for _ in range(args.warmup):
        epoch()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        epoch()
    dt = time.perf_counter() - t0
    value = round(sum(per_round) * args.steps / dt / 1e9, 3)
    sample = f"each step = one whole 3-round epoch of the headline workload (n={cfg['n']} per rank, nothing cut)"
    print(json.dumps({
        "impl": "reference", "metric": "ec_allreduce_apply_GBps", "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "parallelism": "host cores (CPU checker)", "algorithmic_bytes_per_step": sum(per_round)},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--profile-only", action="store_true", help="warm-up and timed steps only (for ncu captures)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="headline workload only")
    ap.add_argument("--apply-path", default="default", choices=["default", "direct"],
                    help="direct: force the direct-load apply kernel (ec_allreduce_set_path(0)) where bulk staging is the default")
    ap.add_argument("--workload", default="headline", choices=["headline", "kmeans", "mf"],
                    help="kmeans: time only the K-means driver (config 5) and print its own JSON line")
    ap.add_argument("--kmeans-bounds", default="on", choices=["on", "off"], help="with --workload kmeans --profile-only: distance bounds")
    ap.add_argument("--kmeans-refresh", type=int, default=32, help="with --workload kmeans --profile-only: all points summed every N-th iteration")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="time budget of the CPU baseline leg")
    ap.add_argument("--threads", type=int, default=0, help="expert: threads per block of the apply kernel")
    ap.add_argument("--tile", type=int, default=0, help="expert: elements per block of the apply kernel")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if world != args.gpus and world == 1 and args.gpus > 1:
        raise SystemExit("launch with torchrun for --gpus > 1")
    if args.workload == "kmeans":
        import torch
        torch.cuda.set_device(local_rank)
        dev = torch.device("cuda", local_rank)
        print(json.dumps({"workload": "kmeans", **kmeans_case(dev, torch.cuda.Stream(device=dev), reps=max(1, min(args.steps, 5)),
                                                               profile_only=args.profile_only, bounds=args.kmeans_bounds == "on",
                                                               refresh=args.kmeans_refresh)}))
        return
    if args.workload == "mf":
        import torch
        torch.cuda.set_device(local_rank)
        dev = torch.device("cuda", local_rank)
        print(json.dumps({"workload": "mf", **mf_case(dev, torch.cuda.Stream(device=dev), iters=max(1, min(args.steps, 20)))}))
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
