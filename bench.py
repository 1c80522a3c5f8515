#!/usr/bin/env python
"""Benchmark of the batched strategy-timeline engine.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole hot path over one synthetic search: evaluate every candidate
of the 64-device workload (every stage composition, 38.8 M candidates), find the best one,
select the 1024 fastest and emit their full per-device timelines.  The headline value is
candidates per second with the event table already resident in HBM; ``e2e`` times the same
through host buffers (table upload, result download).  One JSON line is printed by rank 0.

With N > 1 (launched under torchrun) every rank runs its own search (seed 1 + rank): the path
shards by independent problems, no collective is on the data path, scaling is weak.
``--impl reference`` times the CPU oracle, as it stands, on a bounded sample of the same
workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2306_08423_b200 import sharding  # noqa: E402
from paper_2306_08423_b200 import workloads as W  # noqa: E402

TOP_K = 1024
# 32-bit integer instructions a recurrence cell (one max + one add) needs: on int64 a compare
# pair, two selects, add and add-with-carry; on uint32 (used where an entry's time bound is
# below 2^32) one max and one add.
INT_OPS_PER_CELL_64, INT_OPS_PER_CELL_32 = 6, 2
RECORD_BYTES = 40
# DRAM read + write bytes per launch set of the timed workload come from the one-pass ncu counters
# summarised in profiles/bench_config1_dram_bytes.md, which records beside each figure a hash of the
# kernel sources it was taken on: a figure whose sources have changed since reads as null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "bench_config1_dram_bytes.md")
KERNEL_SOURCES = {
    "eval": ("eval_thread.cuh", "eval_kernels.cu", "recurrence.cuh", "smem_stage.cuh", "interleaved.cuh",
             "bidirectional.cuh", "costs.cuh", "engine.h"),
    "emit": ("emit_kernels.cu", "recurrence.cuh", "interleaved.cuh", "bidirectional.cuh", "costs.cuh",
             "smem_stage.cuh", "engine.h"),
}


def sources_hash(kind: str) -> str:
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kind]:
        with open(os.path.join(ROOT, "paper_2306_08423_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(kind: str):
    """Bytes of the line `traffic: kernel=<kind> sources=<hash> bytes=<n>` if the hash is current."""
    import re
    try:
        text = open(TRAFFIC_FILE).read()
    except OSError:
        return None
    m = re.search(rf"traffic: kernel={kind} sources=([0-9a-f]+) bytes=(\d+)", text)
    return int(m.group(2)) if m and m.group(1) == sources_hash(kind) else None


SM_COUNT, SCHEDULERS_PER_SM, LANES = 148, 4, 32      # issue slots: one warp instruction per scheduler and clock


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


# ----------------------------------------------------------------------------------------------
# reference arm: the CPU oracle on a bounded sample

def oracle_sample_rate(w, n_total, sample, threads):
    import oracle
    idx = np.unique(np.linspace(0, n_total - 1, sample).astype(np.int64))
    t0 = time.perf_counter()
    values, _ = oracle.eval_indices_parallel(w.table, w.space, idx, threads, replicate=False)
    dt = time.perf_counter() - t0
    oracle_sample_rate.last = (idx, values)            # what the oracle computed, for the caller to compare
    return len(idx) / dt, dt, len(idx)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = W.config1()
    n_total, cells = W.count_candidates_and_cells(w.table, w.space)
    threads = os.cpu_count() or 1
    oracle_sample_rate(w, n_total, 4000, threads)                          # warms the thread pool
    rate, dt, ns = oracle_sample_rate(w, n_total, 40_000, threads)         # calibration, untimed
    sample = int(max(40_000, min(4_000_000, rate * 8.0)))                  # about 8 s per step
    for _ in range(args.warmup):
        oracle_sample_rate(w, n_total, max(500, sample // 20), threads)
    times, counts = [], []
    for _ in range(args.steps):
        r, dt, ns = oracle_sample_rate(w, n_total, sample, threads)
        times.append(dt); counts.append(ns)
    value = sum(counts) / sum(times)
    desc = f"{counts[0]} evenly strided candidates of {n_total} per step"
    line = {
        "impl": "reference", "metric": "strategy_candidates_per_sec", "value": value, "unit": "candidates/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * sum(times) / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": w.name, "candidates": n_total, "sample_per_step": counts[0]},
        "events_per_sec": value * cells / n_total,
        "cpu_baseline": {"value": value, "unit": "candidates/s", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "candidates/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        with open(self.tmp.name) as f:
            rows = [r.strip().split(", ") for r in f if r.strip()]
        os.unlink(self.tmp.name)
        sm, names = [], ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); out["sm_max_mhz"] = float(r[1])
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.strip() == "Active":
                    reasons.add(name)
        if sm:
            out["sm_mhz"] = statistics.median(sm)
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


# ----------------------------------------------------------------------------------------------
# our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2306_08423_b200 import engine as E

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peaks, peak_kind = measured_peaks()

    # weak: every rank runs its own search (seed 1 + rank).  shard: the ranks split ONE search
    # (seed 1) into contiguous candidate ranges, select among their own candidates, exchange only
    # their short lists of winners (one all-gather of 2 x 1024 words) and emit a slice of the
    # merged winners each; no other traffic between GPUs.
    shard = args.mode == "shard"
    w = W.config1(seed=1 if shard else sharding.rank_seed(1, rank))
    table, space = w.table, w.space
    n_total, cells = W.count_candidates_and_cells(table, space)
    N = table.n_devices
    my_first, my_count = sharding.shard_range(n_total, rank, world) if shard else (0, n_total)
    emit_first, emit_n = sharding.shard_range(TOP_K, rank, world) if shard else (0, TOP_K)
    k_loc = min(TOP_K, my_count)
    ctx = E.Context(local)
    stream = torch.cuda.current_stream()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    E.distsim_load_event_table(ctx, table)
    assert E.distsim_set_space(ctx, space) == n_total
    d_best = torch.empty(2, dtype=torch.int64, device=dev)                  # (batch time, index) of this rank's best candidate
    batch = torch.empty(my_count, dtype=torch.int64, device=dev)
    top_i = torch.empty(TOP_K, dtype=torch.int64, device=dev)
    top_t = torch.empty(TOP_K, dtype=torch.int64, device=dev)
    merging = shard and world > 1
    loc_i = torch.full((TOP_K,), torch.iinfo(torch.int64).max, dtype=torch.int64, device=dev) if merging else top_i
    loc_t = torch.full((TOP_K,), torch.iinfo(torch.int64).max, dtype=torch.int64, device=dev) if merging else top_t
    offsets = torch.empty(emit_n * N + 1, dtype=torch.int64, device=dev)
    busy = torch.empty(emit_n * N, dtype=torch.int64, device=dev)
    util = torch.empty(emit_n * N, dtype=torch.float64, device=dev)

    loc_i_k, loc_t_k = loc_i[:k_loc], loc_t[:k_loc]                  # views made once, outside the timed steps
    top_mine = top_i[emit_first:emit_first + emit_n]

    def search():
        """Evaluation, best candidate and the 1024 fastest in one asynchronous call; with the
        search split over ranks, the ranks' lists are gathered and merged on every rank."""
        E.distsim_eval_select(ctx, my_first, my_count, batch, k_loc, loc_i_k, loc_t_k, d_best, to_host=False)
        if merging:
            gt, gi = sharding.gather_topk_lists(loc_t, loc_i)
            E.distsim_merge_topk(ctx, gt, gi, gt.numel(), TOP_K, top_i, top_t)

    def emit(rec, cap):
        return E.distsim_emit_timelines(ctx, top_mine, emit_n, rec, cap, offsets, busy, util)

    flush = torch.empty(256 * 2**20, dtype=torch.uint8, device=dev)          # > L2 (126 MB)

    # sizing pass (untimed): how many records this rank's share of the 1024 fastest needs, and the
    # shape the timed steps' emission is provisioned with (they never wait on the host)
    search()
    total_records = emit(None, 0)
    shape = E.distsim_emit_shape_of_last_plan(ctx)
    capacity = total_records + total_records // 8 + 1024
    records = torch.empty(capacity * 5, dtype=torch.int64, device=dev)

    def step(timers=None):
        e0, e1, e2, e3 = (ev(), ev(), ev(), ev()) if timers is not None else (None,) * 4
        if timers is not None:
            e0.record(stream)
        # the search (the library records events around its evaluation and its selection
        # launches itself), then the winners' timelines
        search()
        if timers is not None:
            e2.record(stream)
        E.distsim_emit_timelines_async(ctx, top_mine, emit_n, records, capacity, shape, offsets, busy, util)
        if timers is not None:
            e3.record(stream)
            timers.append((e0, e1, e2, e3))
            e3.synchronize()
            phases.append(E.distsim_testing_last_phase_ms(ctx))
        return d_best, total_records

    phases = []
    E.distsim_testing_time_phases(ctx, True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
        flush.fill_(1)
    gpu_id = str(local)
    try:
        gpu_id = str(torch.cuda.get_device_properties(local).uuid)
        if not gpu_id.startswith("GPU-"):
            gpu_id = "GPU-" + gpu_id
    except Exception:
        gpu_id = str(local)
    barrier()
    sampler = ClockSampler(gpu_id) if rank == 0 else None
    launches0 = ctx.launch_count
    timers = []
    for _ in range(args.steps):
        best, tot = step(timers)
        flush.fill_(1)                         # evict L2 between timed iterations
    barrier()
    launches = ctx.launch_count - launches0
    best = (int(top_i[0]), int(top_t[0]))             # (index, batch time): head of the (merged) list of the last timed step
    # the asynchronous emissions found their provisions sufficient: the record count of the last
    # step, and no error left in the context (a synchronising call would report it)
    assert int(offsets[-1]) == total_records, (int(offsets[-1]), total_records)
    E.distsim_argmin(ctx, batch, my_first, my_count)
    # keep the clock sampler running through the end-to-end loop as well
    step_ms = [t[0].elapsed_time(t[3]) for t in timers]
    eval_ms = [p[0] for p in phases]
    sel_ms = [p[1] for p in phases]
    emit_ms = [t[2].elapsed_time(t[3]) for t in timers]
    total_ms = sum(step_ms)

    # ---- end to end through host buffers ----------------------------------------------------
    h_top_i = torch.empty(TOP_K, dtype=torch.int64).pin_memory()
    h_top_t = torch.empty(TOP_K, dtype=torch.int64).pin_memory()
    h_off = torch.empty(emit_n * N + 1, dtype=torch.int64).pin_memory()
    h_busy = torch.empty(emit_n * N, dtype=torch.int64).pin_memory()
    h_util = torch.empty(emit_n * N, dtype=torch.float64).pin_memory()
    h_rec = torch.empty(capacity * 5, dtype=torch.int64).pin_memory()
    h2d = sum(a.nbytes for a in (table.class_mp, table.class_b, table.fwd_ns, table.bwd_ns,
                                 table.layer_is_expert, table.grad_bytes, space.m_list)) + 128

    def e2e_step():
        E.distsim_load_event_table(ctx, table)                    # host -> device
        E.distsim_set_space(ctx, space)
        search()
        tot = emit(records, capacity)
        h_top_i.copy_(top_i, non_blocking=True); h_top_t.copy_(top_t, non_blocking=True)
        h_off.copy_(offsets, non_blocking=True); h_busy.copy_(busy, non_blocking=True)
        h_util.copy_(util, non_blocking=True)
        h_rec[: tot * 5].copy_(records[: tot * 5], non_blocking=True)
        torch.cuda.synchronize()
        return 16 + 2 * TOP_K * 8 + h_off.numel() * 8 + h_busy.numel() * 16 + tot * RECORD_BYTES

    def results_only_step():
        """As e2e_step, but the multi-GB record buffer stays on the device."""
        E.distsim_load_event_table(ctx, table)
        E.distsim_set_space(ctx, space)
        search()
        emit(records, capacity)
        h_top_i.copy_(top_i, non_blocking=True); h_top_t.copy_(top_t, non_blocking=True)
        h_off.copy_(offsets, non_blocking=True); h_busy.copy_(busy, non_blocking=True)
        h_util.copy_(util, non_blocking=True)
        torch.cuda.synchronize()

    results_only_step()
    t0 = time.perf_counter()
    for _ in range(3):
        results_only_step()
    results_only_s = (time.perf_counter() - t0) / 3

    e2e_step()
    barrier()
    e2e_times = []
    d2h = 0
    n_e2e = max(1, min(args.steps, 3))
    for _ in range(n_e2e):
        flush.fill_(1)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        d2h = e2e_step()
        e2e_times.append(time.perf_counter() - t0)
    serial_s = sum(e2e_times) / len(e2e_times)

    # The same steps with the download of a step's results overlapped with the next step's upload,
    # search and emission: two record buffers on the device and in pinned host memory, the
    # copies on a stream of their own, an event per buffer in each direction.
    records2 = (records, torch.empty_like(records))
    h_rec2 = (h_rec, torch.empty(capacity * 5, dtype=torch.int64).pin_memory())
    h_small = [[torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (top_i, top_t, offsets, busy, util)] for _ in range(2)]
    d_small = [[torch.empty_like(t) for t in (top_i, top_t, offsets, busy, util)] for _ in range(2)]
    copy_stream = torch.cuda.Stream(device=dev)
    emitted = [torch.cuda.Event(), torch.cuda.Event()]
    downloaded = [torch.cuda.Event(), torch.cuda.Event()]

    def overlapped_steps(n):
        for i in range(n):
            b = i & 1
            E.distsim_load_event_table(ctx, table)                # host -> device
            E.distsim_set_space(ctx, space)
            search()
            if i >= 2:
                stream.wait_event(downloaded[b])                  # the buffer's last download has ended
            tot = emit(records2[b], capacity)
            for dst, src in zip(d_small[b], (top_i, top_t, offsets, busy, util)):
                dst.copy_(src, non_blocking=True)                 # the next step overwrites these
            emitted[b].record(stream)
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(emitted[b])
                for dst, src in zip(h_small[b], d_small[b]):
                    dst.copy_(src, non_blocking=True)
                h_rec2[b][: tot * 5].copy_(records2[b][: tot * 5], non_blocking=True)
                downloaded[b].record(copy_stream)
        torch.cuda.synchronize()
        return tot

    overlapped_steps(2)
    barrier()
    n_ovl = 2 * n_e2e + 2
    flush.fill_(1)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    tot = overlapped_steps(n_ovl)
    e2e_times = [(time.perf_counter() - t0) / n_ovl]
    overlap_ok = bool(torch.equal(h_rec2[(n_ovl - 1) & 1][: tot * 5], records2[(n_ovl - 1) & 1][: tot * 5].cpu())
                      and torch.equal(h_small[(n_ovl - 1) & 1][0], top_i.cpu()))
    # what the link gives: the same records copied device -> pinned host, nothing else running
    pe0, pe1 = ev(), ev()
    h_rec[: tot * 5].copy_(records[: tot * 5], non_blocking=True)
    torch.cuda.synchronize()
    pe0.record(stream)
    for _ in range(3):
        h_rec[: tot * 5].copy_(records[: tot * 5], non_blocking=True)
    pe1.record(stream)
    torch.cuda.synchronize()
    d2h_gbs = 3 * tot * RECORD_BYTES / (pe0.elapsed_time(pe1) * 1e-3) / 1e9
    barrier()
    clocks = sampler.stop() if sampler else None

    # ---- max over ranks -----------------------------------------------------------------------
    total_ms_max = sharding.max_over_ranks(total_ms, device=dev)
    e2e_s_max = sharding.max_over_ranks(sum(e2e_times) / len(e2e_times), device=dev)
    serial_s_max = sharding.max_over_ranks(serial_s, device=dev)
    ms_per_step = total_ms_max / args.steps
    job_candidates = n_total if shard else world * n_total           # candidates the whole job evaluates per step
    job_cells = cells if shard else world * cells
    value = job_candidates / (ms_per_step * 1e-3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- rooflines -----------------------------------------------------------------------------
    # integer peaks, measured now with dependency-free instruction streams
    from paper_2306_08423_b200 import probes
    sink = torch.zeros(1, dtype=torch.int64, device=dev)

    def probe(mode):
        pe0, pe1 = ev(), ev()
        probes.distsim_bench_int_issue_probe(148 * 16, 2000, mode, sink)
        pe0.record(stream)
        ops = probes.distsim_bench_int_issue_probe(148 * 16, 20000, mode, sink)
        pe1.record(stream)
        torch.cuda.synchronize()
        return ops / (pe0.elapsed_time(pe1) * 1e-3) / 1e9
    int_peak_gops = probe(0)
    cell64_peak, cell32_peak, cmpsel_peak = probe(1) / 6, probe(3) / 2, probe(2)      # G cells/s, G instr/s
    cell32_fused_peak = probe(4) / 2                                                 # G cells/s, one fused add-max per cell
    cell32_peak = max(cell32_peak, cell32_fused_peak)
    sm_mhz = (clocks or {}).get("sm_mhz") or peaks.get("sm_max_mhz", 1965.0)
    cells_all, cells_32 = E.distsim_testing_space_cells(ctx)
    assert cells_all == cells
    if merging:
        # this rank evaluated its slice only: its share of the cells, taken as the share of the
        # candidates (rank 0's slice holds the short pipelines, so the fraction below is indicative)
        cells, cells_32 = int(cells * my_count / n_total), int(cells_32 * my_count / n_total)
    eval_s = statistics.mean(eval_ms) * 1e-3
    alg_ops = cells_32 * INT_OPS_PER_CELL_32 + (cells - cells_32) * INT_OPS_PER_CELL_64
    achieved_gops = alg_ops / eval_s / 1e9
    # time the recurrence cells alone would take at the measured cell rates of this device
    cell_floor_s = (cells_32 / cell32_peak + (cells - cells_32) / cell64_peak) / 1e9
    issue_peak_gops = SM_COUNT * SCHEDULERS_PER_SM * LANES * sm_mhz * 1e-3
    roofline = {"bound": "alu", "kernel": "eval_thread_kernel (+ lock-step kernel on small rows)",
                "achieved": achieved_gops, "peak": achieved_gops * eval_s / cell_floor_s,
                "unit": "G 32-bit integer operations/s (2 per uint32 cell: max and add; 6 per int64 cell)",
                "frac": cell_floor_s / eval_s, "traffic": recorded_traffic("eval"),
                "peak_kind": "measured in this run: the rate at which dependency-free chains of the same recurrence "
                             "cell issue (uint32 cells as one fused add-max, int64 cells as six instructions), "
                             "blended by the workload's share of each width; frac = time the cells alone take at "
                             "those rates / evaluation time",
                "derived_issue_slot_peak": issue_peak_gops,
                "frac_of_derived_issue_slots": achieved_gops / issue_peak_gops,
                "traffic_note": "DRAM read + write bytes of the four evaluation launches of one step (ncu, one pass; "
                                "null when the kernels changed after the counters were taken); algorithmic: 8 B per "
                                f"candidate = {8 * n_total} B, part of which is still in the L2 when the launches end",
                "derived_note": "148 SMs x 4 schedulers x 32 lanes x SM clock sampled during the run (one "
                                "instruction per scheduler and clock); a uint32 cell's max and add fuse into one "
                                "add-max instruction that issues at half rate, so this is also the cell bound x 2",
                "add_xor_probe_Ginstr_per_s": int_peak_gops, "frac_of_add_xor_probe": achieved_gops / int_peak_gops,
                "cells": cells, "cells_32bit": cells_32, "ms_per_launch_set": statistics.mean(eval_ms),
                "cell_rate_peaks_Gcells_per_s": {"uint32": cell32_peak, "uint32_fused_add_max": cell32_fused_peak,
                                                 "int64": cell64_peak},
                "peak_derived": {"issue_slots_Ginstr_per_s": SM_COUNT * SCHEDULERS_PER_SM * LANES * sm_mhz * 1e-3,
                                 "half_rate_max_Gcells_per_s": SM_COUNT * SCHEDULERS_PER_SM * LANES / 2 * sm_mhz * 1e-3,
                                 "sm_mhz": sm_mhz,
                                 "note": "148 SMs x 4 schedulers x 32 lanes x SM clock; integer max (and the fused "
                                         "add-max) issues at half rate, one per cell"},
                "frac_of_derived_half_rate_max": (cells / eval_s / 1e9) /
                                                 (SM_COUNT * SCHEDULERS_PER_SM * LANES / 2 * sm_mhz * 1e-3),
                "compare_select_peak_Ginstr_per_s": cmpsel_peak,
                "frac_of_cell_rate_floor": cell_floor_s / eval_s}
    emit_bytes = tot * RECORD_BYTES + emit_n * N * 24 + 8
    emit_gbs = emit_bytes / (statistics.mean(emit_ms) * 1e-3) / 1e9
    roofline_emit = {"bound": "hbm", "kernel": "emit_items_kernel (+plan, scan, devices, buckets)",
                     "achieved": emit_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": emit_gbs / peaks["hbm_gbs"], "traffic": recorded_traffic("emit"), "peak_kind": peak_kind,
                     "traffic_note": "DRAM read + write bytes of emit_items_kernel + emit_buckets_kernel of one step "
                                     "(ncu, one pass); the bucket-lane records are still in the L2 when they end",
                     "bytes_per_step": emit_bytes, "ms": statistics.mean(emit_ms)}

    line = {
        "metric": "strategy_candidates_per_sec", "value": value, "unit": "candidates/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "strong" if shard else "weak", "vs_baseline": None,
        "dtype": "int64",
        "dtype_note": "int64 nanoseconds at the boundary; exact uint32 arithmetic inside entries whose time bound is below 2^32",
        "data": "synthetic",
        "config": {"workload": w.name, "candidates": n_total, "recurrence_cells": job_cells // (1 if shard else world), "devices": N,
                   "layers": table.n_layers, "top_k_emitted": TOP_K, "records_emitted": tot,
                   "l2": "256 MB flush between timed iterations",
                   "emission": "distsim_emit_timelines_async, provisioned by the shape of one untimed sizing pass; "
                               "no host wait inside a step",
                   "seed": "1 on every rank" if shard else "1 + rank",
                   "mode": "one search split over the ranks by candidate range; 2 x 1024-word lists all-gathered and merged"
                           if shard else "one search per rank"},
        "events_per_sec": job_cells / (ms_per_step * 1e-3),
        "phase_ms": {"eval": statistics.mean(eval_ms), "argmin_topk": statistics.mean(sel_ms),
                     "emit": statistics.mean(emit_ms)},
        "eval_only": {"candidates_per_sec": my_count / eval_s, "events_per_sec": cells / eval_s},
        "best": {"index": best[0], "batch_ns": best[1]},
        "roofline": roofline, "roofline_emit": roofline_emit,
        "e2e": {"value": job_candidates / e2e_s_max, "unit": "candidates/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s_max * 1e3,
                "note": "table upload, search, emission and the download of every emitted record over PCIe in every "
                        "step; a step's download runs on a copy stream beside the next step's work (two record "
                        "buffers), the time is that of the whole loop / its steps",
                "steps": n_ovl, "downloads_match_device": overlap_ok,
                "d2h_copy_GB_per_sec_measured": d2h_gbs,
                "frac_of_d2h_copy_rate": (d2h / e2e_s_max / 1e9) / d2h_gbs,
                "one_step_at_a_time": {"value": job_candidates / serial_s_max,
                                       "unit": "candidates/s", "ms_per_step": serial_s_max * 1e3},
                "records_left_on_device": {"value": job_candidates / results_only_s, "unit": "candidates/s",
                                           "ms_per_step": results_only_s * 1e3}},
        "gpu_launches": launches, "clocks": clocks,
    }

    failed = False
    if world == 1:
        if not args.no_workloads:
            line["workloads"] = other_workloads(E, ctx, torch, dev, peaks, cell32_peak, cell64_peak)
        if not args.no_cpu:
            import oracle
            oracle.build()
            threads = os.cpu_count() or 1
            oracle_sample_rate(w, n_total, 4000, threads)                   # warms the thread pool
            rate, dt, ns = oracle_sample_rate(w, n_total, 40_000, threads)  # calibration
            sample = int(max(40_000, min(4_000_000, rate * 15.0)))          # about 15 s of work
            rate, dt, ns = oracle_sample_rate(w, n_total, sample, threads)
            line["cpu_baseline"] = {"value": rate, "unit": "candidates/s", "cores": threads, "kind": "oracle",
                                    "sample": f"{ns} evenly strided candidates of {n_total}, {dt:.1f} s"}
            # the batch array the timed steps wrote, against the oracle's values at the same indices
            o_idx, o_val = oracle_sample_rate.last
            got = batch[torch.from_numpy(o_idx).to(dev)].cpu().numpy()
            mismatches = int((got != o_val).sum())
            o_order = np.lexsort((o_idx, o_val))
            line["verified"] = {"candidates": int(len(o_idx)), "mismatches": mismatches,
                                "best_not_above_sample_minimum": bool(best[1] <= int(o_val[o_order[0]])),
                                "what": "batch times of the timed steps vs the CPU oracle, bit-exact"}
            failed = mismatches != 0 or not line["verified"]["best_not_above_sample_minimum"]
    ctx.close()
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    if world == 1 and not args.no_cpu and failed:
        sys.exit(1)


def other_workloads(E, ctx, torch, dev, peaks, cell32_peak, cell64_peak):
    """Evaluation rate on the other search workloads and emission rate on the 1024 fastest
    candidates of the 1024-device workload (device-resident, CUDA events)."""
    out = {}
    stream = torch.cuda.current_stream()
    # the 64-device workload once more with the two further schedules in its space: interleaved
    # 1F1B with two chunks per device and bidirectional pipelines (a warp per candidate)
    more = W.config1()
    more.space.sched_mask, more.space.v_max = 27, 2
    more.name = "config1_with_interleaved_and_bidirectional"
    for w in (W.CONFIGS[0](), W.CONFIGS[2](), W.CONFIGS[3](), more):
        n, cells = W.count_candidates_and_cells(w.table, w.space)
        E.distsim_load_event_table(ctx, w.table)
        E.distsim_set_space(ctx, w.space)
        batch = torch.empty(n, dtype=torch.int64, device=dev)
        # A small search is over before the host has issued the next launch, so a host-driven loop
        # would time the host.  One evaluation is captured into a CUDA graph and replayed back to
        # back: the device time of the library's own launches, nothing else.
        for _ in range(3):
            E.distsim_eval_strategies(ctx, 0, n, batch)
        best = E.distsim_argmin(ctx, batch, 0, n)
        # replays per sample: ten of a short evaluation, fewer of one that takes milliseconds
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        E.distsim_eval_strategies(ctx, 0, n, batch)
        p1.record(stream)
        torch.cuda.synchronize()
        reps = max(1, min(10, int(20.0 / max(p0.elapsed_time(p1), 1e-3))))
        times, how = [], f"cuda graph of one evaluation, replayed {reps}x per sample"
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                E.distsim_eval_strategies(ctx, 0, n, batch)
            stream = torch.cuda.current_stream()
            for it in range(8 if reps > 1 else 5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(reps):
                    graph.replay()
                e1.record(stream)
                torch.cuda.synchronize()
                if it >= (3 if reps > 1 else 2):
                    times.append(e0.elapsed_time(e1) * 1e-3 / reps)
            del graph
        except RuntimeError:
            how = "8 evaluations issued back to back per sample (graph capture unavailable)"
            torch.cuda.synchronize()
            stream = torch.cuda.current_stream()
            for it in range(8):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(8):
                    E.distsim_eval_strategies(ctx, 0, n, batch)
                e1.record(stream)
                torch.cuda.synchronize()
                if it >= 3:
                    times.append(e0.elapsed_time(e1) * 1e-3 / 8)
        assert E.distsim_argmin(ctx, batch, 0, n) == best
        t = statistics.median(times)
        _, cells_32 = E.distsim_testing_space_cells(ctx)
        # time the cells alone would take at this device's measured 32-bit / 64-bit cell rates
        floor_s = (cells_32 / cell32_peak + (cells - cells_32) / cell64_peak) / 1e9
        out[w.name] = {"candidates": n, "cells": cells, "cells_32bit": cells_32, "eval_ms": t * 1e3,
                       "candidates_per_sec": n / t, "events_per_sec": cells / t,
                       "frac_of_cell_rate_floor": floor_s / t, "best_index": best[0], "best_batch_ns": best[1],
                       "timed": how}
    # emission: still loaded with the 1024-device workload?  reload it to be explicit
    w = W.config4()
    n, _ = W.count_candidates_and_cells(w.table, w.space)
    N = w.table.n_devices
    E.distsim_load_event_table(ctx, w.table)
    E.distsim_set_space(ctx, w.space)
    batch = torch.empty(n, dtype=torch.int64, device=dev)
    E.distsim_eval_strategies(ctx, 0, n, batch)
    top = torch.empty(w.top_k, dtype=torch.int64, device=dev)
    E.distsim_topk(ctx, batch, 0, n, w.top_k, top)
    chunk = 128                       # candidates per call: about 10 GB of records
    sizes = [E.distsim_emit_timelines(ctx, top[i:i + chunk], min(chunk, w.top_k - i), None, 0)
             for i in range(0, w.top_k, chunk)]
    cap = max(sizes) + 1024
    records = torch.empty(cap * 5, dtype=torch.int64, device=dev)
    offsets = torch.empty(chunk * N + 1, dtype=torch.int64, device=dev)
    busy = torch.empty(chunk * N, dtype=torch.int64, device=dev)
    util = torch.empty(chunk * N, dtype=torch.float64, device=dev)
    for i in range(0, 2 * chunk, chunk):                                     # warm-up
        E.distsim_emit_timelines(ctx, top[i:i + chunk], chunk, records, cap, offsets, busy, util)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0
    e0.record(stream)
    for i in range(0, w.top_k, chunk):
        c = min(chunk, w.top_k - i)
        total += E.distsim_emit_timelines(ctx, top[i:i + c], c, records, cap, offsets, busy, util)
    e1.record(stream)
    torch.cuda.synchronize()
    t = e0.elapsed_time(e1) * 1e-3
    nbytes = total * RECORD_BYTES + w.top_k * N * 24
    out[w.name] = {"candidates": w.top_k, "records": total, "bytes": nbytes, "seconds": t,
                   "records_per_sec": total / t, "GB_per_sec": nbytes / t / 1e9,
                   "frac_of_measured_hbm": nbytes / t / 1e9 / peaks["hbm_gbs"],
                   "frac_of_nominal_8TBs": nbytes / t / 1e9 / 8000.0,
                   "chunk_candidates": chunk, "buffer_GB": cap * RECORD_BYTES / 1e9}
    # The same emission brought to the host: 32 candidates per call into one of two device buffers,
    # each downloaded to pinned memory on a copy stream while the next call writes the other.
    del records
    torch.cuda.empty_cache()
    small = 32
    sizes = [E.distsim_emit_timelines(ctx, top[i:i + small], min(small, w.top_k - i), None, 0)
             for i in range(0, w.top_k, small)]
    cap2 = max(sizes) + 1024
    d_rec = [torch.empty(cap2 * 5, dtype=torch.int64, device=dev) for _ in range(2)]
    h_rec = [torch.empty(cap2 * 5, dtype=torch.int64).pin_memory() for _ in range(2)]
    copy_stream = torch.cuda.Stream(device=dev)
    emitted = [torch.cuda.Event(), torch.cuda.Event()]
    downloaded = [torch.cuda.Event(), torch.cuda.Event()]
    # the link alone: one buffer copied device -> pinned host
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h_rec[0].copy_(d_rec[0], non_blocking=True)
    torch.cuda.synchronize()
    c0.record(stream)
    h_rec[0].copy_(d_rec[0], non_blocking=True)
    c1.record(stream)
    torch.cuda.synchronize()
    link_gbs = cap2 * RECORD_BYTES / (c0.elapsed_time(c1) * 1e-3) / 1e9
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    moved = 0
    for k, i in enumerate(range(0, w.top_k, small)):
        b, c = k & 1, min(small, w.top_k - i)
        if k >= 2:
            stream.wait_event(downloaded[b])
        got = E.distsim_emit_timelines(ctx, top[i:i + c], c, d_rec[b], cap2, offsets[: c * N + 1], busy[: c * N], util[: c * N])
        emitted[b].record(stream)
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(emitted[b])
            h_rec[b][: got * 5].copy_(d_rec[b][: got * 5], non_blocking=True)
            downloaded[b].record(copy_stream)
        moved += got * RECORD_BYTES
    torch.cuda.synchronize()
    t2 = time.perf_counter() - t0
    last = (w.top_k - 1) // small
    ok = bool(torch.equal(h_rec[last & 1][: got * 5], d_rec[last & 1][: got * 5].cpu()))
    out[w.name]["to_host"] = {"seconds": t2, "GB_per_sec": moved / t2 / 1e9, "d2h_copy_GB_per_sec_measured": link_gbs,
                              "frac_of_d2h_copy_rate": moved / t2 / 1e9 / link_gbs, "chunk_candidates": small,
                              "last_download_matches_device": ok,
                              "how": "two device buffers and two pinned host buffers; a chunk's download runs on a copy "
                                     "stream beside the emission of the next chunk"}
    return out


def profile_case(name):
    """Small, bounded invocations for profiler captures (no timing, no JSON line):
    eval1  - evaluation of a 2 M-candidate slice of the 64-device workload (a pp = 16 row, m = 16 and 32)
    eval1m128 - the m = 128 entry of the same row (1 M candidates, 4.0e9 cells)
    eval1m1 - the m = 1 entry of the same row (1 M candidates: unranking and set-up only)
    eval0  - evaluation of the whole tiny workload (88 candidates)
    eval3  - evaluation of the whole 256-device MoE workload (650 k candidates)
    eval2  - evaluation of the whole 1024-device workload (4 176 candidates, long pipelines)
    eval2pp64 - the pp = 64 rows of the same workload (lock-step kernel, two warps per candidate)
    emit4  - emission of 16 of the fastest candidates of the 1024-device workload (~1.9 GB)
    emit1  - emission of the 1024 fastest candidates of the 64-device workload (~1.8 GB)
    emit4x128 - as emit4 for 128 candidates, one call of the benchmark's size (~10 GB; for
             one-pass launch lists only)
    select1 - the 1024 fastest of the whole 64-device workload (evaluation, then three selections)
    evalx  - 400 000 candidates of the 64-device workload's interleaved (two chunks per device) and
             bidirectional-pipeline rows (a warp per candidate)"""
    import torch
    from paper_2306_08423_b200 import engine as E
    torch.cuda.set_device(0)
    ctx = E.Context(0)
    if name in ("eval0", "eval1", "eval1m1", "eval1m128", "eval3", "eval2", "eval2pp64"):
        w = {"eval0": W.config0, "eval3": W.config3, "eval2": W.config2, "eval2pp64": W.config2}.get(name, W.config1)()
        E.distsim_load_event_table(ctx, w.table)
        n = E.distsim_set_space(ctx, w.space)
        first, count = 0, n
        if name == "eval2pp64":
            # the first pp = 64 row (mp = 1): 256 micro-batch counts x 2 schedules
            off = 0
            for mp, pp, dp, ms, parts, n_sched, _v in W.space_shape(w.table, w.space):
                if (mp, pp) == (1, 64):
                    first, count = off, len(ms) * parts * n_sched
                off += len(ms) * parts * n_sched
        elif name in ("eval1", "eval1m1", "eval1m128"):
            # whole entries of the (mp = 1, pp = 16) row, 980 628 candidates each:
            # eval1 m = 16 and 32, eval1m128 m = 128
            off = 0
            for mp, pp, dp, ms, parts, n_sched, _v in W.space_shape(w.table, w.space):
                if (mp, pp) == (1, 16):
                    e0, ne = (4, 2) if name == "eval1" else (ms.index(128 if name == "eval1m128" else 1), 1)
                    first, count = off + e0 * parts * n_sched, ne * parts * n_sched
                off += len(ms) * parts * n_sched
        batch = torch.empty(count, dtype=torch.int64, device="cuda")
        for _ in range(3):
            E.distsim_eval_strategies(ctx, first, count, batch)
        print(name, "best", E.distsim_argmin(ctx, batch, first, count))
    elif name == "select1":
        w = W.config1()
        E.distsim_load_event_table(ctx, w.table)
        n = E.distsim_set_space(ctx, w.space)
        batch = torch.empty(n, dtype=torch.int64, device="cuda")
        top_i = torch.empty(TOP_K, dtype=torch.int64, device="cuda")
        top_t = torch.empty(TOP_K, dtype=torch.int64, device="cuda")
        E.distsim_eval_strategies(ctx, 0, n, batch)
        for _ in range(3):
            E.distsim_topk(ctx, batch, 0, n, TOP_K, top_i, top_t)
        print(name, "k-th time", int(top_t[-1]))
    elif name == "evalx":
        w = W.config1()
        w.space.sched_mask, w.space.v_max = 24, 2
        E.distsim_load_event_table(ctx, w.table)
        n = E.distsim_set_space(ctx, w.space)
        # a slice that ends in the bidirectional row of the first (mp, pp): both kinds of candidates
        rows = W.space_shape(w.table, w.space)
        first_two_rows = sum(len(ms) * parts * n_sched for (_mp, _pp, _dp, ms, parts, n_sched, _v) in rows[:2])
        count = min(n, 400_000)
        first = max(0, first_two_rows - count // 2)
        batch = torch.empty(count, dtype=torch.int64, device="cuda")
        for _ in range(3):
            E.distsim_eval_strategies(ctx, first, count, batch)
        print(name, "candidates", count, "of", n, "best", E.distsim_argmin(ctx, batch, first, count))
    elif name in ("emit4", "emit4x128", "emit1"):
        k = {"emit4": 16, "emit4x128": 128, "emit1": TOP_K}[name]
        w = W.config4() if name != "emit1" else W.config1()
        E.distsim_load_event_table(ctx, w.table)
        n = E.distsim_set_space(ctx, w.space)
        batch = torch.empty(n, dtype=torch.int64, device="cuda")
        E.distsim_eval_strategies(ctx, 0, n, batch)
        top = torch.empty(k, dtype=torch.int64, device="cuda")
        E.distsim_topk(ctx, batch, 0, n, k, top)
        total = E.distsim_emit_timelines(ctx, top, k, None, 0)
        records = torch.empty(total * 5, dtype=torch.int64, device="cuda")
        for _ in range(2):
            E.distsim_emit_timelines(ctx, top, k, records, total)
        print(name, "records", total, "bytes", total * RECORD_BYTES)
    else:
        raise SystemExit(f"unknown profile case {name}")
    torch.cuda.synchronize()
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--mode", choices=["weak", "shard"], default="weak",
                    help="N > 1: weak = one search per rank; shard = one search split over the ranks")
    ap.add_argument("--no-workloads", action="store_true", help="skip the per-workload summary")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--profile-case", default=None, help="eval0 | eval1 | eval1m1 | eval1m128 | eval2 | eval2pp64 | eval3 | emit1 | emit4 | emit4x128: small run for ncu")
    args = ap.parse_args()
    if args.profile_case:
        profile_case(args.profile_case)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
