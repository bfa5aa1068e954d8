#!/usr/bin/env python
"""Benchmark of the value-driven memory hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
append a few new experiences (Eq. 1), retrieve for a batch of queries (two-phase
value-driven retrieval, Section 3.2) and update the value estimates of everything
that was retrieved from per-query rewards (Eq. 4).

Prints ONE JSON line.  `value` is retrieval queries/s with every input already in
HBM; `e2e` is the same loop through the host-buffer entry points (queries copied
host->device and results device->host inside the timed region).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl evk|reference]
                  [--workload large_hbm|...] [--batch B]
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
SCAN_DRAM_BYTES_PER_ENTRY = 542.93e6 / 262224      # d = 1024: 2,070.5 B against 2,048 B algorithmic
UNIT = "queries/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps (0: about a second of them)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="evk", choices=["evk", "reference"])
    ap.add_argument("--workload", default="large_hbm")
    ap.add_argument("--batch", type=int, default=0, help="query batch size (0: the workload's largest)")
    ap.add_argument("--scoring", default="auto", choices=["auto", "stream", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
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
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
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
        "config": {"workload": f"{wl.name}: N={wl.n}, d={wl.d} bf16, B={b}, k1={wl.k1}, k2={wl.k2}, w={wl.w}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


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
        dist.init_process_group("nccl", device_id=dev)

    wl = synth.WORKLOADS[args.workload]
    b = args.batch or max(wl.batches)
    if args.steps <= 0:
        # long enough for several clock samples: the scan of one step reads the bank once
        # (about 6 TB/s) or does 2*B*N*d flop (about 1.2 PFLOP/s), whichever takes longer
        est_ms = max(wl.n * wl.d * 2 / 6.0e9, 2.0 * b * wl.n * wl.d / 1.2e12) + 0.06
        args.steps = int(min(2000, max(20, 1000.0 / est_ms)))
    # experiences appended per step (Eq. 1): 16, fewer where that would grow the bank by more
    # than about 3 % over the run (the workload's N is what the metric is quoted on)
    n_new = 0 if wl.n < 1024 else max(1, min(16, int(0.03 * wl.n / (args.warmup + args.steps))))
    total_steps = args.warmup + args.steps
    capacity = wl.n + n_new * (2 * total_steps + 8)

    # ---- resident state: every rank holds a replica of the bank and serves its own batches ----
    bank = synth.make_bank(wl, dev)
    q_tab = synth.make_q_tables(wl)
    mem = evk.evk_mem_create(wl.d, capacity, device=dev)
    evk.evk_mem_set_scoring(mem, {"auto": evk.EVK_SCORING_AUTO, "stream": evk.EVK_SCORING_STREAM,
                                  "tensor": evk.EVK_SCORING_TENSOR}[args.scoring])
    evk.evk_mem_insert(mem, bank)
    for s in range(2):
        evk.evk_q_write(mem, s, torch.from_numpy(q_tab[s]).to(dev))
    del bank
    n_batches = min(total_steps, 16)
    query_sets = [synth.make_queries(wl, b, dev, salt=1 + i + 1000 * rank) for i in range(n_batches)]
    new_rows = synth.gaussian_unit(max(n_new, 1), wl.d, 77 + rank, dev)
    rng = np.random.Generator(np.random.PCG64([9, rank]))
    rewards_q = torch.from_numpy((rng.random((n_batches, b)) < 0.4).astype(np.float32)).to(dev)
    # one reward per query, shared by the k2 items of its context
    r_sets = [rewards_q[j].repeat_interleave(wl.k2).contiguous() for j in range(n_batches)]
    # a workload with its own stream of update batches (popularity-skewed ids) uses those
    own_updates = None
    if wl.update_ids == "zipf":
        own_updates = []
        for j in range(n_batches):
            u_ids, u_r = synth.make_updates(wl, round_idx=j + 1000 * rank)
            own_updates.append((torch.from_numpy(u_ids).to(dev), torch.from_numpy(u_r).to(dev)))
    n_upd = wl.n_updates if own_updates else b * wl.k2
    ids_out = torch.empty((b, wl.k2), dtype=torch.int32, device=dev)
    scores_out = torch.empty((b, wl.k2), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def gather_updates(ids_flat, rewards_flat):
        """Replicas stay identical: every rank applies every rank's updates, in rank order."""
        return parallel.gather_update_batches(ids_flat, rewards_flat)

    def step(i, events=None):
        stage = i % 2
        qs = query_sets[i % n_batches]
        if n_new:
            evk.evk_mem_insert(mem, new_rows, evk.EVK_STAGE_ALL)
        if events is not None:
            evk.evk_mem_profile_scoring(mem, events[0], events[1])
        evk.evk_retrieve(mem, qs, stage, wl.k1, wl.k2, wl.w, out=(ids_out, scores_out))
        if own_updates:
            ids_flat, r_flat = gather_updates(*own_updates[i % n_batches])
        else:
            ids_flat, r_flat = gather_updates(ids_out.reshape(-1), r_sets[i % n_batches])
        evk.evk_q_update(mem, ids_flat, stage, r_flat, wl.alpha)

    # ---- device-resident timing ----
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    assert evk.evk_last_status(mem) == 0
    kind, n_score_launches = evk.evk_retrieve_plan(mem, b, wl.k1)
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, c in pairs:     # create the underlying events
        a.record(stream)
        c.record(stream)
    launches_before = evk.evk_launch_count(mem)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        # the scoring kernel is bracketed by events on every 4th step only: an event between two
        # kernels keeps the second from starting early behind the first
        step(args.warmup + i, pairs[i] if i % 4 == 0 else None)
    t_stop.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = t_start.elapsed_time(t_stop)
    gpu_launches = evk.evk_launch_count(mem) - launches_before
    score_ms = [pairs[i][0].elapsed_time(pairs[i][1]) for i in range(0, args.steps, 4)]
    assert evk.evk_last_status(mem) == 0

    # ---- the retrieval alone (scoring + top-k1 + rerank), device-resident, for the roofline of the path ----
    r_iters = max(10, min(args.steps, 50))
    r_start, r_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(3):
        evk.evk_retrieve(mem, query_sets[i % n_batches], 0, wl.k1, wl.k2, wl.w, out=(ids_out, scores_out))
    torch.cuda.synchronize()
    r_start.record(stream)
    for i in range(r_iters):
        evk.evk_retrieve(mem, query_sets[i % n_batches], i % 2, wl.k1, wl.k2, wl.w, out=(ids_out, scores_out))
    r_stop.record(stream)
    torch.cuda.synchronize()
    retrieve_ms = r_start.elapsed_time(r_stop) / r_iters

    # ---- the value update alone (Eq. 4), one batch of the step's size per launch ----
    if own_updates:
        u_batches = own_updates
    else:
        u_batches = [(ids_out.reshape(-1).clone(), r_sets[j]) for j in range(min(4, n_batches))]
    longest_chain = int(torch.bincount(u_batches[0][0].clamp(min=0).to(torch.int64)).max().item()) if n_upd else 0
    u_start, u_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(3):
        evk.evk_q_update(mem, u_batches[i % len(u_batches)][0], i % 2, u_batches[i % len(u_batches)][1], wl.alpha)
    torch.cuda.synchronize()
    u_start.record(stream)
    for i in range(r_iters):
        evk.evk_q_update(mem, u_batches[i % len(u_batches)][0], i % 2, u_batches[i % len(u_batches)][1], wl.alpha)
    u_stop.record(stream)
    torch.cuda.synchronize()
    update_us = 1e3 * u_start.elapsed_time(u_stop) / r_iters
    assert evk.evk_last_status(mem) == 0

    # ---- end to end through the host-buffer entry points ----
    q_host = [query_sets[j % n_batches].cpu().pin_memory() for j in range(4)]
    ids_h = torch.empty((b, wl.k2), dtype=torch.int32).pin_memory()
    sc_h = torch.empty((b, wl.k2), dtype=torch.float32).pin_memory()
    r_h = [r_sets[j % n_batches].cpu().pin_memory() for j in range(4)]
    upd_h = None
    if own_updates:
        upd_h = [(u.cpu().pin_memory(), r.cpu().pin_memory()) for u, r in own_updates[:4]]
    e2e_steps = args.steps

    def e2e_step(i):
        stage = i % 2
        evk.evk_retrieve_host(mem, q_host[i % 4], stage, wl.k1, wl.k2, wl.w, ids_h, sc_h)
        if upd_h:
            evk.evk_q_update_host(mem, upd_h[i % len(upd_h)][0], stage, upd_h[i % len(upd_h)][1], wl.alpha)
        else:
            evk.evk_q_update_host(mem, ids_h.reshape(-1), stage, r_h[i % 4], wl.alpha)

    for i in range(3):
        e2e_step(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e_start, e_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_start.record(stream)
    for i in range(e2e_steps):
        e2e_step(i)
    e_stop.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e_start.elapsed_time(e_stop)
    assert evk.evk_last_status(mem) == 0

    if world > 1:
        t = torch.tensor([elapsed_ms, e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms, e2e_ms = t.tolist()

    if rank == 0:
        peaks = measured_peaks()
        value = world * b * args.steps / (elapsed_ms * 1e-3)
        e2e_value = world * b * e2e_steps / (e2e_ms * 1e-3)
        # roofline of the dominant kernel (phase-1 scoring): each launch reads the bank once
        # rows scanned by the launches that were timed (the bank grows by n_new rows per step)
        size = wl.n + n_new * (args.warmup + (args.steps + 1) / 2.0)
        size_end = evk.evk_mem_size(mem)             # what the retrieval-only loop scanned
        queries_per_launch = b / max(n_score_launches, 1)
        bytes_per_launch = size * wl.d * 2 + queries_per_launch * wl.d * 2
        launch_ms = statistics.mean(score_ms) / max(n_score_launches, 1)
        achieved = bytes_per_launch / (launch_ms * 1e-3) / 1e9
        flops_per_launch = 2.0 * queries_per_launch * size * wl.d
        # DRAM bytes per launch: read + written bytes per bank entry from one ncu capture of the scan
        # kernel on a 262,224-row case (profiles/score_mma_clustered_b64.md), scaled by the rows scanned
        # (the bank is read once, so traffic grows with the rows); unknown for the streaming kernel
        traffic = SCAN_DRAM_BYTES_PER_ENTRY * size if (kind == evk.EVK_SCORING_TENSOR and wl.d == 1024) else None
        tflops = flops_per_launch / (launch_ms * 1e-3) / 1e12
        # arithmetic intensity of a scan is `queries_per_launch` flop per byte; the ridge of this
        # machine sits near 256, beyond it the tensor cores bound the kernel
        tensor_bound = queries_per_launch >= 256
        # the sustained GEMM figure where the kernel ran inside a long stretch of tensor work (steps of
        # several ms, or a timed region that the power cap had time to act on), else the burst one
        sustained = elapsed_ms / args.steps > 5.0 or (elapsed_ms > 300.0 and "sw_power_cap" in (clocks or {}).get("reasons", []))
        tensor_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
        roofline = {"bound": "tensor" if tensor_bound else "hbm",
                    "achieved": tflops if tensor_bound else achieved,
                    "peak": tensor_peak if tensor_bound else peaks["hbm_gbs"],
                    "unit": "TFLOP/s" if tensor_bound else "GB/s",
                    "frac": (tflops / tensor_peak) if tensor_bound else achieved / peaks["hbm_gbs"],
                    "traffic": traffic, "peak_source": peaks["source"],
                    "peak_kind": ("sustained" if sustained else "burst") if tensor_bound else "copy", "gbs": achieved,
                    "kernel": "score_stream" if kind == evk.EVK_SCORING_STREAM else "score_mma",
                    "launches_per_step": n_score_launches, "ms_per_launch": launch_ms,
                    "tflops": flops_per_launch / (launch_ms * 1e-3) / 1e12}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{wl.name}: N={wl.n}, d={wl.d} bf16, B={b}, k1={wl.k1}, k2={wl.k2}, w={wl.w}; "
                                   f"step = insert {n_new} + retrieve {b} + update {n_upd * world}",
                       "l2": ("inputs larger than L2 (bank %.2f GiB scanned every step)" % (size * wl.d * 2 / 2 ** 30))
                       if size * wl.d * 2 > 126e6 else
                       "bank of %.1f MiB fits in L2 and is not flushed between steps: a parity workload, not a bench line"
                       % (size * wl.d * 2 / 2 ** 20),
                       "parallelism": "replicated bank, queries sharded by rank, update batches all-gathered"
                       if world > 1 else "single GPU"},
            "entries_scanned_per_s": value * size,
            "roofline": roofline,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": b * wl.d * 2 + n_upd * 8,
                    "d2h_bytes_per_step": b * wl.k2 * 8, "ms_per_step": e2e_ms / e2e_steps},
            "retrieve_only": {"ms": retrieve_ms, "queries_per_s": b / (retrieve_ms * 1e-3),
                              "bank_gbs": size_end * wl.d * 2 / (retrieve_ms * 1e-3) / 1e9,
                              "frac_of_measured_hbm": size_end * wl.d * 2 / (retrieve_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            "update_only": {"us_per_batch": update_us, "updates": int(n_upd),
                            "updates_per_s": n_upd / (update_us * 1e-6) if update_us > 0 else None,
                            "longest_duplicate_chain": longest_chain},
            "gpu_launches": int(gpu_launches),
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            bank_bits = synth.bf16_bits(evk.evk_bank_read(mem, 0, wl.n))
            v, n_done, dt, cores = time_oracle_sample(wl, bank_bits, q_tab, b, args.cpu_seconds)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{n_done} of {b} queries against the full bank plus their updates, {dt:.1f} s"}
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
