#!/usr/bin/env python
"""Benchmark of the value-driven memory hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
append a few new experiences (Eq. 1), retrieve for a batch of queries (two-phase
value-driven retrieval, Section 3.2) and update the value estimates of everything
that was retrieved from per-query rewards (Eq. 4).

Prints ONE JSON line.  `value` is retrieval queries/s with every input already in
HBM; `e2e` is the same step through host buffers (new rows, queries and update
batches copied host->device, results device->host, inside the timed region).
Besides the headline leg (exactly --steps steps) the line carries a `sustained`
block (the same step for about a second, whatever --steps says) and, on one GPU,
an `also` list with the other regimes: the small batches of the bandwidth-bound
bank and the two tensor-bound workloads, each timed for at least half a second.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl evk|reference]
                  [--workload large_hbm|...] [--batch B] [--layout replicated|rows]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "retrieval queries/sec at N=1M, d=1024 bf16"
UNIT = "queries/s"
NOMINAL_HBM_GBS = 8000.0          # the HBM3e figure the bandwidth target is quoted against
# DRAM bytes (read + written) per scanned bank entry of width 1024, from one ncu capture of the
# scan kernel; see TRAFFIC_SOURCE.  The bank is read once per launch, so traffic grows with the rows.
SCAN_DRAM_BYTES_PER_ENTRY = 541.86e6 / 262147
TRAFFIC_SOURCE = ("ncu dram__bytes_read.sum + dram__bytes_write.sum of one score_mma_kernel launch, "
                  "262,147 rows x 1024 bf16 (512 MiB), 64 queries, k1=128: 537.81 + 4.04 MB = 2,067.0 B per entry "
                  "against 2,048 B algorithmic; scaled by the rows one launch scans")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps of the headline leg (0: about a second of them)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="evk", choices=["evk", "reference"])
    ap.add_argument("--workload", default="large_hbm")
    ap.add_argument("--batch", type=int, default=0, help="query batch size (0: the workload's largest)")
    ap.add_argument("--scoring", default="auto", choices=["auto", "stream", "tensor"])
    ap.add_argument("--layout", default="replicated", choices=["replicated", "rows"],
                    help="several GPUs: every rank holds the bank and serves its own queries, or the bank is "
                         "split by rows and every rank scans its shard for all queries")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="headline and sustained legs only")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "power_w": statistics.median(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle_sample(wl, bank_bits, q_tab, b, seconds, seed=0):
    """The CPU checker as it stands, on a bounded sample of the workload's queries."""
    import oracle
    from paper_2603_10846_b200 import synth
    import torch
    queries = synth.bf16_bits(synth.make_queries(wl, max(b, 1), "cpu", salt=99 + seed).to(dtype=torch.bfloat16))
    n_done, t0 = 0, time.perf_counter()
    ids_all = []
    while n_done < queries.shape[0]:
        ids, _, _, _ = oracle.retrieve(bank_bits, queries[n_done:n_done + 1], q_tab[0], wl.k1, wl.k2, wl.w)
        ids_all.append(ids.reshape(-1))
        n_done += 1
        if time.perf_counter() - t0 >= seconds:
            break
    ids = np.concatenate(ids_all)
    oracle.q_update_f32(q_tab[0], ids, np.ones(ids.size, np.float32), wl.alpha)
    dt = time.perf_counter() - t0
    return n_done / dt, n_done, dt, oracle.threads()


def run_reference(args):
    """--impl reference: the CPU checker timed on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2603_10846_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    b = args.batch or max(wl.batches)
    if args.steps <= 0:
        args.steps = 5
    bank_bits = synth.bf16_bits(synth.make_bank(wl, "cpu").to(dtype=torch.bfloat16))
    q_tab = synth.make_q_tables(wl)
    total = args.steps + args.warmup
    queries = synth.bf16_bits(synth.make_queries(wl, total + 1, "cpu", salt=7).to(dtype=torch.bfloat16))
    q = q_tab[0].copy()

    def step(i, rows):
        nonlocal q
        ids, _, _, _ = oracle.retrieve(bank_bits[:rows], queries[i:i + 1], q[:rows], wl.k1, wl.k2, wl.w)
        flat = ids.reshape(-1)
        q[:rows] = oracle.q_update_f32(q[:rows], flat, np.ones(flat.size, np.float32), wl.alpha)

    # size the per-step sample so that the whole run stays near two minutes
    t0 = time.perf_counter()
    step(total, wl.n)
    t_full = time.perf_counter() - t0
    frac = min(1.0, 120.0 / max(total * t_full, 1e-9))
    rows = wl.n if frac >= 1.0 else max(min(wl.n, 65536), int(wl.n * frac))
    for i in range(args.warmup):
        step(i, rows)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i, rows)
    dt = time.perf_counter() - t0
    value = args.steps * (rows / wl.n) / dt          # queries/s against the full N-entry bank
    cores = oracle.threads()
    sample = (f"per step 1 of {b} queries against the first {rows} of {wl.n} bank rows and that query's updates; "
              f"throughput scaled by rows/N")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(wl, b)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def scan_roofline(evk, kind, n_score_launches, wl, b, rows, scan_ms, peaks, clocks, step_ms, leg_ms):
    """The roofline record of the phase-1 scan kernel for one leg: every fraction, against every
    denominator (the measured copy figure, the nominal HBM figure, the burst and the sustained GEMM)."""
    queries_per_launch = b / max(n_score_launches, 1)
    bytes_per_launch = rows * wl.d * 2 + queries_per_launch * wl.d * 2
    flops_per_launch = 2.0 * queries_per_launch * rows * wl.d
    launch_ms = scan_ms / max(n_score_launches, 1)
    gbs = bytes_per_launch / (launch_ms * 1e-3) / 1e9
    tflops = flops_per_launch / (launch_ms * 1e-3) / 1e12
    # arithmetic intensity of a scan is `queries_per_launch` flop per byte; the ridge of this
    # machine sits near 256, beyond it the tensor cores bound the kernel
    tensor_bound = queries_per_launch >= 256
    # the sustained GEMM figure where the kernel ran inside a long stretch of tensor work (steps of
    # several ms, or a leg the power cap had time to act on), else the burst one
    reasons = (clocks or {}).get("reasons", [])
    sustained = step_ms > 5.0 or (leg_ms > 300.0 and "sw_power_cap" in reasons)
    tensor_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    traffic = None
    if kind == evk.EVK_SCORING_TENSOR and wl.d == 1024:
        traffic = SCAN_DRAM_BYTES_PER_ENTRY * rows
    sm_mhz = (clocks or {}).get("sm_mhz")
    return {
        "bound": "tensor" if tensor_bound else "hbm",
        "achieved": tflops if tensor_bound else gbs,
        "peak": tensor_peak if tensor_bound else peaks["hbm_gbs"],
        "unit": "TFLOP/s" if tensor_bound else "GB/s",
        "frac": (tflops / tensor_peak) if tensor_bound else gbs / peaks["hbm_gbs"],
        "traffic": traffic, "traffic_source": TRAFFIC_SOURCE if traffic else None,
        "peak_source": peaks["source"],
        "peak_kind": ("sustained" if sustained else "burst") if tensor_bound else "copy",
        "kernel": "score_stream" if kind == evk.EVK_SCORING_STREAM else "score_mma",
        "launches_per_step": n_score_launches, "ms_per_launch": launch_ms,
        "gbs": gbs, "tflops": tflops,
        "frac_of_copy_hbm": gbs / peaks["hbm_gbs"],
        "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBS,
        # against a read-only stream of the same bank through the same copy engine, measured in this run
        "frac_of_read_only_hbm": gbs / peaks["hbm_read_gbs"] if peaks.get("hbm_read_gbs") else None,
        "frac_of_burst_tensor": tflops / peaks["bf16_tflops"],
        "frac_of_sustained_tensor": tflops / peaks["bf16_tflops_sustained"],
        # clock-normalised duration: compare legs that ran at different SM clocks
        "ms_x_sm_ghz": launch_ms * sm_mhz / 1e3 if sm_mhz else None,
    }


class Bank:
    """One workload's resident state on this rank plus the synthetic inputs of its steps."""

    def __init__(self, evk, synth, parallel, wl, dev, rank, world, scoring, layout):
        import torch
        self.evk, self.synth, self.parallel, self.wl, self.dev = evk, synth, parallel, wl, dev
        self.rank, self.world, self.layout = rank, world, layout
        self.torch = torch
        self.id_offset = 0
        n_local = wl.n
        if layout == "rows" and world > 1:
            begin, end = parallel.row_shard(wl.n, rank, world)
            self.id_offset, n_local = begin, end - begin
        self.n_local = n_local
        # room for the rows the steps append (at most ~8 % of the bank over all legs)
        self.capacity = n_local + max(4096, n_local // 12)
        bank = synth.make_bank(wl, dev)
        self.q_tab = synth.make_q_tables(wl)
        self.mem = evk.evk_mem_create(wl.d, self.capacity, device=dev)
        evk.evk_mem_set_scoring(self.mem, {"auto": evk.EVK_SCORING_AUTO, "stream": evk.EVK_SCORING_STREAM,
                                           "tensor": evk.EVK_SCORING_TENSOR}[scoring])
        evk.evk_mem_insert(self.mem, bank[self.id_offset:self.id_offset + n_local])
        for s in range(2):
            evk.evk_q_write(self.mem, s, torch.from_numpy(
                np.ascontiguousarray(self.q_tab[s][self.id_offset:self.id_offset + n_local])).to(dev))
        del bank
        self.new_rows = synth.gaussian_unit(16, wl.d, 77 + rank, dev)
        self.new_rows_host = self.new_rows.cpu().pin_memory()

    def inputs(self, b, n_batches):
        """Query batches, per-query rewards and (for a workload with its own update stream) update batches."""
        torch, wl, dev, synth = self.torch, self.wl, self.dev, self.synth
        # under the row layout every rank sees the same global batch; replicas serve batches of their own
        salt_rank = 0 if self.layout == "rows" else self.rank
        query_sets = [synth.make_queries(wl, b, dev, salt=1 + i + 1000 * salt_rank) for i in range(n_batches)]
        rng = np.random.Generator(np.random.PCG64([9, salt_rank]))
        rewards_q = torch.from_numpy((rng.random((n_batches, b)) < 0.4).astype(np.float32)).to(dev)
        r_sets = [rewards_q[j].repeat_interleave(wl.k2).contiguous() for j in range(n_batches)]
        own_updates = None
        if wl.update_ids == "zipf":
            own_updates = []
            for j in range(n_batches):
                u_ids, u_r = synth.make_updates(wl, round_idx=j + 1000 * salt_rank)
                own_updates.append((torch.from_numpy(u_ids).to(dev), torch.from_numpy(u_r).to(dev)))
        return query_sets, r_sets, own_updates


def check_status(evk, mem):
    st = evk.evk_last_status(mem)
    if st != 0:
        raise RuntimeError(f"device status {st}: {evk.strerror(st)}")


def run_leg(bk: Bank, b: int, warmup: int, steps: int = 0, min_seconds: float = 0.0, parts=("device",),
            sample_clocks=True, peaks=None):
    """Times one configuration on a resident bank.  steps > 0: exactly that many timed steps;
    otherwise as many as fill min_seconds.  parts: "device" (inputs resident), "e2e" (host buffers),
    "retrieve" (retrieval alone), "update" (value update alone)."""
    import torch
    import torch.distributed as dist
    evk, wl, mem, dev, world, rank = bk.evk, bk.wl, bk.mem, bk.dev, bk.world, bk.rank
    rows_layout = bk.layout == "rows" and world > 1
    n_batches = 16
    query_sets, r_sets, own_updates = bk.inputs(b, n_batches)
    n_upd = wl.n_updates if own_updates else b * wl.k2
    ids_out = torch.empty((b, wl.k2), dtype=torch.int32, device=dev)
    scores_out = torch.empty((b, wl.k2), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    res = {"B": b, "updates_per_step": int(n_upd * (1 if rows_layout else world))}

    def retrieve(qs, stage):
        if rows_layout:
            ids, sc = bk.parallel.retrieve_row_sharded(evk, mem, qs, stage, wl.k1, wl.k2, wl.w, bk.id_offset)
            return ids
        evk.evk_retrieve(mem, qs, stage, wl.k1, wl.k2, wl.w, out=(ids_out, scores_out))
        return ids_out

    def update(ids_flat, r_flat, stage):
        if rows_layout:
            # every rank sees the whole batch and applies, in array order, the pairs whose entry it owns
            ids_flat, r_flat = bk.parallel.own_updates(ids_flat, r_flat, bk.id_offset, bk.id_offset + bk.n_local)
        else:
            # replicas stay identical: every rank applies every rank's updates, in rank order
            ids_flat, r_flat = bk.parallel.gather_update_batches(ids_flat, r_flat)
        if ids_flat.numel():
            evk.evk_q_update(mem, ids_flat, stage, r_flat, wl.alpha)

    def step(i, n_new, events=None):
        stage = i % 2
        if n_new:
            evk.evk_mem_insert(mem, bk.new_rows[:n_new], evk.EVK_STAGE_ALL)
        if events is not None:
            evk.evk_mem_profile_scoring(mem, events[0], events[1])
        ids = retrieve(query_sets[i % n_batches], stage)
        if own_updates:
            update(own_updates[i % n_batches][0], own_updates[i % n_batches][1], stage)
        else:
            update(ids.reshape(-1), r_sets[i % n_batches], stage)

    def pick_steps(per_step_ms):
        if steps > 0:
            return steps
        return int(min(20000, max(10, np.ceil(1e3 * min_seconds / max(per_step_ms, 1e-3)))))

    def rows_per_step(k):
        # appended experiences (Eq. 1): 16 per step, fewer where that would grow the bank by more
        # than about 1 % over the leg (the workload's N is what the metric is quoted on)
        if bk.n_local < 1024:
            return 0
        room = bk.capacity - evk.evk_mem_size(mem) - 64
        return int(max(0, min(16, 0.01 * bk.n_local / max(k, 1), room / max(2 * k + warmup + 8, 1))))

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world > 1:
            t = torch.tensor([ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return ms

    if "device" in parts:
        for i in range(max(warmup, 3)):
            step(i, 1 if bk.n_local >= 1024 else 0)
        torch.cuda.synchronize()
        check_status(evk, mem)
        # a short probe sizes a time-based leg
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(5):
            step(i, 0)
        c.record(stream)
        torch.cuda.synchronize()
        k = pick_steps(a.elapsed_time(c) / 5)
        n_new = rows_per_step(k)
        kind, n_score_launches = evk.evk_retrieve_plan(mem, b, wl.k1)
        n_ev = (k + 3) // 4
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]
        for e0, e1 in pairs:     # create the underlying events
            e0.record(stream)
            e1.record(stream)
        size_start = evk.evk_mem_size(mem)
        launches_before = evk.evk_launch_count(mem)
        sync_all()
        sampler = ClockSampler(dev.index)
        if rank == 0 and sample_clocks:
            sampler.start()
        t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_start.record(stream)
        for i in range(k):
            # the scoring kernel is bracketed by events on every 4th step only: an event between two
            # kernels keeps the second from starting early behind the first
            step(i, n_new, pairs[i // 4] if (i % 4 == 0 and not rows_layout) else None)
        t_stop.record(stream)
        sync_all()
        clocks = sampler.stop() if (rank == 0 and sample_clocks) else None
        elapsed_ms = max_over_ranks(t_start.elapsed_time(t_stop))
        check_status(evk, mem)
        size_end = evk.evk_mem_size(mem)
        rows = 0.5 * (size_start + size_end)
        res.update({"steps": k, "ms_per_step": elapsed_ms / k, "elapsed_ms": elapsed_ms,
                    "queries_per_s": (b if rows_layout else world * b) * k / (elapsed_ms * 1e-3),
                    "rows_appended_per_step": n_new, "rows_scanned": rows,
                    "gpu_launches": int(evk.evk_launch_count(mem) - launches_before), "clocks": clocks})
        if not rows_layout:
            scan_ms = statistics.mean(p0.elapsed_time(p1) for p0, p1 in pairs)
            res["roofline"] = scan_roofline(evk, kind, n_score_launches, wl, b, rows, scan_ms, peaks, clocks,
                                            elapsed_ms / k, elapsed_ms)

    if "retrieve" in parts:
        # the retrieval alone (sample pass, thresholds, scan, merge, rerank), inputs resident
        for i in range(3):
            retrieve(query_sets[i % n_batches], 0)
        torch.cuda.synchronize()
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(5):
            retrieve(query_sets[i % n_batches], i % 2)
        c.record(stream)
        torch.cuda.synchronize()
        iters = int(min(5000, max(10, np.ceil(250.0 / max(a.elapsed_time(c) / 5, 1e-3)))))
        a.record(stream)
        for i in range(iters):
            retrieve(query_sets[i % n_batches], i % 2)
        c.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(c) / iters
        size_now = evk.evk_mem_size(mem)
        gbs = size_now * wl.d * 2 / (ms * 1e-3) / 1e9
        res["retrieve_only"] = {"ms": ms, "iters": iters, "queries_per_s": b / (ms * 1e-3), "bank_gbs": gbs,
                                "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                                "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBS,
                                "tflops": 2.0 * b * size_now * wl.d / (ms * 1e-3) / 1e12}

    if "update" in parts:
        # the value update alone (Eq. 4), one batch of the step's size per call
        if own_updates:
            u_batches = own_updates
        else:
            u_batches = [(ids_out.reshape(-1).clone(), r_sets[j]) for j in range(4)]
        longest = int(torch.bincount(u_batches[0][0].clamp(min=0).to(torch.int64)).max().item()) if n_upd else 0
        for i in range(3):
            evk.evk_q_update(mem, u_batches[i % len(u_batches)][0], i % 2, u_batches[i % len(u_batches)][1], wl.alpha)
        torch.cuda.synchronize()
        iters = 200
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(iters):
            evk.evk_q_update(mem, u_batches[i % len(u_batches)][0], i % 2, u_batches[i % len(u_batches)][1], wl.alpha)
        c.record(stream)
        torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(c) / iters
        check_status(evk, mem)
        res["update_only"] = {"us_per_batch": us, "updates": int(n_upd), "iters": iters,
                              "updates_per_s": n_upd / (us * 1e-6) if us > 0 else None,
                              "longest_duplicate_chain": longest}

    if "e2e" in parts and not rows_layout:
        # end to end: every input of the step starts in pinned host memory, the result ends there
        q_host = [query_sets[j].cpu().pin_memory() for j in range(4)]
        ids_h = torch.empty((b, wl.k2), dtype=torch.int32).pin_memory()
        sc_h = torch.empty((b, wl.k2), dtype=torch.float32).pin_memory()
        r_h = [r_sets[j].cpu().pin_memory() for j in range(4)]
        upd_h = [(u.cpu().pin_memory(), r.cpu().pin_memory()) for u, r in own_updates[:4]] if own_updates else None
        k = res.get("steps") or pick_steps(1.0)
        n_new = rows_per_step(k)

        evk.evk_mem_set_host_staging(mem, 8 << 20)

        def e2e_step(i):
            stage = i % 2
            if n_new:
                evk.evk_mem_insert_host(mem, bk.new_rows_host[:n_new], evk.EVK_STAGE_ALL)
            evk.evk_retrieve_host(mem, q_host[i % 4], stage, wl.k1, wl.k2, wl.w, ids_h, sc_h)
            if upd_h:
                evk.evk_q_update_host(mem, upd_h[i % len(upd_h)][0], stage, upd_h[i % len(upd_h)][1], wl.alpha)
            else:
                evk.evk_q_update_host(mem, ids_h.reshape(-1), stage, r_h[i % 4], wl.alpha)

        for i in range(3):
            e2e_step(i)
        sync_all()
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(k):
            e2e_step(i)
        c.record(stream)
        sync_all()
        e2e_ms = max_over_ranks(a.elapsed_time(c))
        check_status(evk, mem)
        res["e2e"] = {"value": world * b * k / (e2e_ms * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": n_new * wl.d * 2 + b * wl.d * 2 + n_upd * 8,
                      "d2h_bytes_per_step": b * wl.k2 * 8, "ms_per_step": e2e_ms / k, "steps": k,
                      "step": f"evk_mem_insert_host ({n_new} rows) + evk_retrieve_host + evk_q_update_host, all from pinned host "
                              "arrays, through a page-locked staging buffer (evk_mem_set_host_staging): the result is read "
                              "on the host every step"}
        evk.evk_mem_set_host_staging(mem, 0)
    return res


def workload_name(wl, b):
    """The same string in both arms, so that their lines can be matched."""
    return f"{wl.name}: N={wl.n}, d={wl.d} bf16, B={b}, k1={wl.k1}, k2={wl.k2}, w={wl.w}"


def describe_step(wl, b, res):
    upd = ("the retrieved ids (B*k2), one reward per query" if wl.update_ids != "zipf"
           else f"{wl.n_updates} popularity-skewed ids of the workload's own stream")
    return (f"insert {res.get('rows_appended_per_step', 0)} + retrieve {b} + update "
            f"{res['updates_per_step']} ({upd})")


def compact(name, b, res):
    """One `also` entry: what the regime's leg measured."""
    rf = res.get("roofline", {})
    ck = res.get("clocks") or {}
    out = {"workload": name, "B": b, "steps": res["steps"], "seconds": res["elapsed_ms"] / 1e3,
           "ms_per_step": res["ms_per_step"], "queries_per_s": res["queries_per_s"],
           "scan_ms": rf.get("ms_per_launch"), "bound": rf.get("bound"),
           "sm_mhz": ck.get("sm_mhz"), "clock_samples": ck.get("samples"), "reasons": ck.get("reasons"),
           "sw_power_cap": "sw_power_cap" in (ck.get("reasons") or []),
           "ms_x_sm_ghz": rf.get("ms_x_sm_ghz")}
    if rf.get("bound") == "hbm":
        out.update({"scan_gbs": rf["gbs"], "frac_of_copy_hbm": rf["frac_of_copy_hbm"],
                    "frac_of_nominal_hbm": rf["frac_of_nominal_hbm"]})
    else:
        out.update({"scan_tflops": rf.get("tflops"), "frac_of_burst_tensor": rf.get("frac_of_burst_tensor"),
                    "frac_of_sustained_tensor": rf.get("frac_of_sustained_tensor")})
    for key in ("retrieve_only", "update_only"):
        if key in res:
            out[key] = res[key]
    return out


def run_evk(args):
    import torch
    import torch.distributed as dist
    from paper_2603_10846_b200 import evk, parallel, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        if args.layout == "rows":
            os.environ.setdefault("NCCL_DEBUG", "INFO")      # the communicator's set-up lines stay in the log
        dist.init_process_group("nccl", device_id=dev)

    peaks = measured_peaks()
    wl = synth.WORKLOADS[args.workload]
    b = args.batch or max(wl.batches)
    bk = Bank(evk, synth, parallel, wl, dev, rank, world, args.scoring, args.layout)
    rows_layout = args.layout == "rows" and world > 1

    # ---- calibration: what a kernel that only reads can reach on this GPU, on this bank ----
    read_gbs = None
    if wl.n * wl.d * 2 > 126e6:
        stream = torch.cuda.current_stream()
        for _ in range(3):
            evk.evk_mem_read_probe(bk.mem)
        torch.cuda.synchronize()
        times = []
        for _ in range(20):
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            evk.evk_mem_read_probe(bk.mem)
            c.record(stream)
            torch.cuda.synchronize()
            times.append(a.elapsed_time(c))
        check_status(evk, bk.mem)
        read_bytes = (evk.evk_mem_size(bk.mem) * wl.d * 2 // 32768) * 32768
        read_gbs = {"best": read_bytes / (min(times) * 1e-3) / 1e9, "mean": read_bytes / (statistics.mean(times) * 1e-3) / 1e9,
                    "launches": len(times), "how": "evk_mem_read_probe: the stored rows streamed once into shared memory, "
                                                   "32 KB bulk copies, one block per SM, CUDA events around each launch"}
        peaks["hbm_read_gbs"] = read_gbs["mean"]

    # ---- headline: exactly --steps steps (or about a second of them) ----
    head = run_leg(bk, b, args.warmup, steps=args.steps, min_seconds=1.0,
                   parts=("device", "retrieve", "update", "e2e"), peaks=peaks)
    # ---- the same step for about a second whatever --steps says: the power cap has time to act ----
    sustained = run_leg(bk, b, 3, min_seconds=1.0, parts=("device",), peaks=peaks)

    also = []
    if world == 1 and not args.no_also and args.workload == "large_hbm" and not args.batch:
        for bb in sorted(set(wl.batches) - {b}):
            also.append(compact(wl.name, bb, run_leg(bk, bb, 3, min_seconds=0.5, parts=("device", "retrieve"),
                                                     peaks=peaks)))

    line = None
    if rank == 0:
        rf = head.get("roofline")
        line = {
            "metric": METRIC, "value": head["queries_per_s"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "strong" if rows_layout else "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(wl, b), "step": describe_step(wl, b, head),
                       "l2": ("inputs larger than L2 (bank %.2f GiB scanned every step)"
                              % (head["rows_scanned"] * wl.d * 2 / 2 ** 30))
                       if head["rows_scanned"] * wl.d * 2 > 126e6 else
                       "bank of %.1f MiB fits in L2 and is not flushed between steps: a parity workload, not a bench line"
                       % (head["rows_scanned"] * wl.d * 2 / 2 ** 20),
                       "parallelism": ("bank split by rows over the ranks: local phase 1, one all-gather of "
                                       "B*k1*12 bytes per rank, merge and phase 2 on every rank, owner-applied updates"
                                       if rows_layout else
                                       "replicated bank, queries sharded by rank, update batches all-gathered")
                       if world > 1 else "single GPU",
                       "e2e_step": (head.get("e2e") or {}).get("step")},
            "entries_scanned_per_s": head["queries_per_s"] * head["rows_scanned"] * (world if rows_layout else 1),
            "roofline": rf,
            "e2e": {k: v for k, v in (head.get("e2e") or {}).items() if k != "step"} or None,
            "retrieve_only": head.get("retrieve_only"),
            "update_only": head.get("update_only"),
            "gpu_launches": head["gpu_launches"],
            "clocks": head["clocks"],
            "hbm_read_only": read_gbs,
            "sustained": {"steps": sustained["steps"], "seconds": sustained["elapsed_ms"] / 1e3,
                          "ms_per_step": sustained["ms_per_step"], "queries_per_s": sustained["queries_per_s"],
                          "roofline": sustained.get("roofline"), "clocks": sustained["clocks"]},
        }

    # ---- the other regimes, one GPU only (they would hold the other ranks' GPUs idle) ----
    if world == 1 and not args.no_also and args.workload == "large_hbm" and not args.batch:
        bank_bits = None
        if not args.no_cpu_baseline:
            bank_bits = synth.bf16_bits(evk.evk_bank_read(bk.mem, 0, wl.n))
        q_tab = bk.q_tab
        del bk
        torch.cuda.empty_cache()
        for name in ("clustered", "large_compute"):
            wl2 = synth.WORKLOADS[name]
            bk2 = Bank(evk, synth, parallel, wl2, dev, rank, world, args.scoring, "replicated")
            b2 = max(wl2.batches)
            leg = run_leg(bk2, b2, 3, min_seconds=0.5, parts=("device", "retrieve", "update"), peaks=peaks)
            entry = compact(name, b2, leg)
            entry["config"] = workload_name(wl2, b2)
            entry["step"] = describe_step(wl2, b2, leg)
            also.append(entry)
            del bk2
            torch.cuda.empty_cache()
        line["also"] = also
        if line["roofline"] is not None:
            # the same regimes in brief, beside the headline kernel's record
            line["roofline"]["also"] = [
                {"workload": e["workload"], "B": e["B"], "bound": e["bound"], "ms_per_launch": e["scan_ms"],
                 "frac_of_copy_hbm": e.get("frac_of_copy_hbm"), "frac_of_nominal_hbm": e.get("frac_of_nominal_hbm"),
                 "frac_of_burst_tensor": e.get("frac_of_burst_tensor"),
                 "frac_of_sustained_tensor": e.get("frac_of_sustained_tensor")} for e in also]
            line["roofline"]["sustained"] = {k: sustained["roofline"][k] for k in
                                             ("ms_per_launch", "achieved", "frac", "frac_of_nominal_hbm")}
        if bank_bits is not None:
            v, n_done, dt, cores = time_oracle_sample(wl, bank_bits, q_tab, b, args.cpu_seconds)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{n_done} of {b} queries against the full bank plus their updates, {dt:.1f} s"}
    elif rank == 0 and world == 1 and not args.no_cpu_baseline:
        bank_bits = synth.bf16_bits(evk.evk_bank_read(bk.mem, 0, wl.n))
        v, n_done, dt, cores = time_oracle_sample(wl, bank_bits, bk.q_tab, b, args.cpu_seconds)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{n_done} of {b} queries against the full bank plus their updates, {dt:.1f} s"}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_evk(args)


if __name__ == "__main__":
    main()
