#!/usr/bin/env python
"""Benchmark of the batched LLMem estimator on B200.

One "step" is one pass of the whole hot path over the stress grid (65,536 deep/wide
decoders, about 5.8e9 allocate/free events, materialised as int64):

    event counts + offsets  ->  expansion with fused page rounding  ->  segmented
    prefix-sum + max  ->  largest batch per capacity  ->  Algorithm 1 selection

By default the expansion and the scan run as one kernel (llmem_expand_scan: the list is
written to HBM once and folded from shared memory); --two-pass times the separate
llmem_expand_events and llmem_scan_peak kernels instead.  Either way the kernels of the
other path are timed alone after the step and reported next to it.

`value` is alloc-events per second over all ranks with the configurations already
resident in HBM; `e2e` is the same pass through the public API starting from pinned
host buffers, with every step's host<->device copies inside the timed region (the steps
run as a two-stage pipeline: step i + 1's inputs come in while step i computes).  The roofline
block reports the dominant kernel against the measured HBM copy bandwidth.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Under torchrun every rank runs the same work on its own seeded grid (no exchange
step exists in this method); times are the maximum over ranks.  With --scaling strong the
ranks share one grid instead: contiguous shards balanced by event count, results gathered
over NCCL and checked against the fused estimate of the whole grid.

At one GPU the default run adds three short legs under "secondary": the fused estimate of
the large sweep, the max-batch search with Algorithm 1 selection, and the whole shape grid
through the materialised path in slabs, each with its own roofline entry.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2404_10933_b200 import grids  # noqa: E402

METRIC = "alloc-events/sec (configs/sec in configs_per_sec, % of HBM roofline in roofline)"
UNIT = "events/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per event (dram__bytes_read.sum + dram__bytes_write.sum over events) of the two
# HBM-bound kernels, from an ncu capture of a 4096-configuration run (summary kept under
# profiles/; traffic grows in proportion to the number of events).  Set an entry
# to None when its kernel changes after the capture.
NCU_TRAFFIC_BYTES_PER_EVENT = {"expand": 7.8251, "scan": 8.0143, "expand_scan": 7.8269}
# the same for the owner kernel that takes lists of short and medium segments (64-shape capture)
NCU_TRAFFIC_BYTES_PER_EVENT_OWNERS = 8.0487


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_id: str):
        self.device_index = device_id
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.device_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()
        # nvidia-smi's start-up (driver enumeration) can hold up work submission for tens of
        # milliseconds: let it finish, i.e. wait for the first sample, before anything is timed
        deadline = time.time() + 10.0
        while not self.rows and time.time() < deadline and self.proc.poll() is None:
            time.sleep(0.05)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15 and len(r) >= 9] or \
               [r for _, r in self.rows if len(r) >= 9]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = [float(r[1]) for r in rows]
        reasons = set()
        for r in rows:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                               r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(rows[0][2]), "reasons": sorted(reasons),
                "samples": len(rows), "power_w_max": max(float(r[3]) for r in rows)}


# ---------------------------------------------------------------------------
# CPU oracle legs (the only places that may execute oracle/)
# ---------------------------------------------------------------------------
def oracle_sample(sample_configs: int):
    cfgs = grids.g5_stress(0, sample_configs)
    return cfgs


def time_oracle(cfgs, threads: int):
    """One pass of the hot path by the oracle as it stands: explicit list, rounding and linear
    scan per configuration (level 1), then its bisecting search and Algorithm 1 over the same
    capacities and batch range as the CUDA arm."""
    import oracle
    oracle.lib()
    caps = grids.g4_capacities()
    t0 = time.perf_counter()
    r = oracle.estimate(cfgs, level=1, threads=threads)
    oracle.max_batch(cfgs, caps, grids.G4_BMAX, level=2, threads=threads)
    oracle.select_method(cfgs, caps, grids.G4_BMAX, level=2, threads=threads)
    dt = time.perf_counter() - t0
    return int(r["count"].sum()), dt


def cpu_baseline(sample_configs: int = grids.G5_CONFIGS):
    cores = os.cpu_count() or 1
    events, dt = time_oracle(oracle_sample(sample_configs), cores)
    one_n = max(1, sample_configs // 32)
    one_events, one_dt = time_oracle(oracle_sample(one_n), 1)
    return {"value": events / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "configs_per_sec": sample_configs / dt,
            "single_thread": {"value": one_events / one_dt, "unit": UNIT, "cores": 1,
                              "sample": f"first {one_n} configurations, {one_dt:.2f} s"},
            "sample": f"all {sample_configs} stress-grid configurations "
                      f"({events} events), level-1 oracle (explicit list, round, scan) + its bisecting search and selection, "
                      f"{cores} threads, {dt:.2f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cores = os.cpu_count() or 1
    # each step a bounded sample of the workload, sized so that the whole run stays near 10-20 s
    sample = int(min(4096, max(256, 4096 * 100 // max(args.steps, 1))))
    cfgs = oracle_sample(sample)
    for _ in range(max(args.warmup, 0)):
        time_oracle(cfgs[:256], cores)
    t_total, ev_total = 0.0, 0
    for _ in range(args.steps):
        ev, dt = time_oracle(cfgs, cores)
        t_total += dt
        ev_total += ev
    value = ev_total / t_total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic", "configs_per_sec": sample * args.steps / t_total,
        "config": {"workload": "G5 stress grid (materialised int64 event lists), bounded sample",
                   "sample_configs": sample, "events_per_step": ev_total // args.steps},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"each step: first {sample} stress-grid configurations, level-1 oracle + its search and selection, "
                                   f"{cores} threads"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------
class HotPath:
    """Holds device buffers for one grid and runs one step of the hot path."""

    def __init__(self, llmem, torch, cfgs: np.ndarray, caps: np.ndarray, bmax: int, one_pass: bool):
        self.llmem, self.torch = llmem, torch
        self.one_pass = one_pass
        # counts(3) + [expand_scan(1) + finish(1) | expand(1) + scan(1) + finish(1)] + max_batch(1) + select(1)
        self.kernels_per_step = 7 if one_pass else 8
        self.n = len(cfgs)
        self.bmax = bmax
        self.host_cfg = torch.from_numpy(cfgs.view(np.uint8).reshape(-1, 64)).pin_memory()
        self.host_caps = torch.from_numpy(caps).pin_memory()
        self.cfg = self.host_cfg.cuda()
        self.caps = self.host_caps.cuda()
        offsets, _ = llmem.event_counts(self.cfg)
        self.total = int(offsets[-1].item())
        self.delta = torch.empty(self.total, dtype=torch.int64, device="cuda")
        self.scan_scratch = torch.empty(max(llmem.scratch_bytes(llmem.OP_SCAN_PEAK, self.n, self.total),
                                            llmem.scratch_bytes(llmem.OP_EXPAND_SCAN, self.n, self.total)),
                                        dtype=torch.uint8, device="cuda")
        self.ev = {k: [] for k in (("expand_scan",) if one_pass else ("expand", "scan"))}
        self.side = torch.cuda.Stream()
        self.fork = torch.cuda.Event()
        self.host_out = {
            "peak": torch.empty(self.n, dtype=torch.int64).pin_memory(),
            "method": torch.empty((self.n, len(caps)), dtype=torch.int32).pin_memory(),
            "batch": torch.empty((self.n, len(caps)), dtype=torch.int32).pin_memory(),
        }

    def _materialise_and_search(self, cfg, caps, offsets, total, record):
        """Rows a2-a6 for configurations and offsets already on the device."""
        llmem, torch = self.llmem, self.torch
        main = torch.cuda.current_stream()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)] if record else None
        if record:
            e[0].record()
        if self.one_pass:
            # expansion, page rounding and segmented scan in one kernel: the list is written once
            r = llmem.expand_scan(cfg, offsets, total, fuse_round=True, out=self.delta, scratch=self.scan_scratch)
            if record:
                e[1].record()
                self.ev["expand_scan"].append((e[0], e[1]))
            bs, _ = llmem.max_batch(cfg, caps, self.bmax, want_status=False)
            sel = llmem.select_method(cfg, caps, self.bmax, want_bs_list=False, want_status=False)
        else:
            delta = llmem.expand_events(cfg, offsets, total, fuse_round=True, out=self.delta)
            if record:
                e[1].record()
            # the searches (integer ALU, a few bytes per configuration) do not depend on the event
            # list: queued on a second stream once the expansion is done, they run underneath the scan
            self.fork.record(main)
            self.side.wait_event(self.fork)
            with torch.cuda.stream(self.side):
                bs, _ = llmem.max_batch(cfg, caps, self.bmax, want_status=False)
                sel = llmem.select_method(cfg, caps, self.bmax, want_bs_list=False, want_status=False)
            r = llmem.scan_peak(delta, offsets, cfg, scratch=self.scan_scratch)
            if record:
                e[2].record()
                self.ev["expand"].append((e[0], e[1]))
                self.ev["scan"].append((e[1], e[2]))
            main.wait_stream(self.side)
        return r, bs, sel

    def step(self, record=True):
        offsets, _ = self.llmem.event_counts(self.cfg)
        r, bs, sel = self._materialise_and_search(self.cfg, self.caps, offsets, self.total, record)
        return {"peak": r["peak"], "index": r["index"], "bs": bs, "method": sel["method"],
                "batch": sel["batch"], "offsets": offsets}

    def run_e2e(self, steps: int):
        """`steps` end-to-end steps as a two-stage pipeline, the way a caller with a stream of
        batches would drive the library: while step i computes on the main stream, the copy
        stream brings in the configurations of step i + 1, counts their events and hands the
        total to the host (which needs it to size the list), and afterwards takes step i's
        results back.  Every step still moves its own inputs and outputs; nothing is reused
        between steps but the buffers."""
        torch, llmem = self.torch, self.llmem
        main, copy = torch.cuda.current_stream(), self.side
        if not hasattr(self, "host_total"):
            self.host_total = torch.zeros(2, dtype=torch.int64).pin_memory()

        def stage(k):
            copy.wait_stream(main) if k == 0 else None
            with torch.cuda.stream(copy):
                cfg = self.host_cfg.to("cuda", non_blocking=True)
                caps = self.host_caps.to("cuda", non_blocking=True)
                offsets, _ = llmem.event_counts(cfg)
                self.host_total[k % 2:k % 2 + 1].copy_(offsets[-1:], non_blocking=True)
                ready = torch.cuda.Event()
                ready.record(copy)
            return cfg, caps, offsets, ready

        nxt = stage(0)
        for i in range(steps):
            cfg, caps, offsets, ready = nxt
            ready.synchronize()                               # the host needs this step's event total
            total = int(self.host_total[i % 2])
            if total > self.delta.numel():
                self.delta = torch.empty(total, dtype=torch.int64, device="cuda")
            main.wait_event(ready)
            for t in (cfg, caps, offsets):
                t.record_stream(main)
            if i + 1 < steps:
                nxt = stage(i + 1)
            if self.one_pass:
                r = llmem.expand_scan(cfg, offsets, total, fuse_round=True, out=self.delta, scratch=self.scan_scratch)
            else:
                delta = llmem.expand_events(cfg, offsets, total, fuse_round=True, out=self.delta)
                r = llmem.scan_peak(delta, offsets, cfg, scratch=self.scan_scratch)
            llmem.max_batch(cfg, caps, self.bmax, want_status=False)
            sel = llmem.select_method(cfg, caps, self.bmax, want_bs_list=False, want_status=False)
            done = torch.cuda.Event()
            done.record(main)
            copy.wait_event(done)
            with torch.cuda.stream(copy):
                self.host_out["peak"].copy_(r["peak"], non_blocking=True)
                self.host_out["method"].copy_(sel["method"], non_blocking=True)
                self.host_out["batch"].copy_(sel["batch"], non_blocking=True)
            for t in (r["peak"], sel["method"], sel["batch"]):
                t.record_stream(copy)
        main.wait_stream(copy)
        main.synchronize()

    def time_kernel(self, what, reps=5):
        """Mean launch time (ms) of one of the HBM-bound kernels on the resident grid."""
        llmem, torch = self.llmem, self.torch
        offsets, _ = llmem.event_counts(self.cfg)
        ts = []
        for _ in range(reps + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if what == "expand":
                llmem.expand_events(self.cfg, offsets, self.total, fuse_round=True, out=self.delta)
            elif what == "scan":
                llmem.scan_peak(self.delta, offsets, self.cfg, scratch=self.scan_scratch)
            else:
                llmem.expand_scan(self.cfg, offsets, self.total, fuse_round=True, out=self.delta,
                                  scratch=self.scan_scratch)
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.mean(ts[1:])

    @property
    def h2d_bytes(self):
        return self.host_cfg.numel() + self.host_caps.numel() * 8

    @property
    def d2h_bytes(self):
        return 8 + sum(t.numel() * t.element_size() for t in self.host_out.values())


def run_ours(args):
    import torch
    if not torch.cuda.is_available():
        print(json.dumps({"error": "no CUDA device: the estimator has no CPU fallback"}))
        return 2
    import paper_2404_10933_b200 as llmem
    llmem.lib()  # fail loudly if the CUDA library is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    # under torchrun (any world size, one rank included) time through the process group
    if world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ):
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    from paper_2404_10933_b200 import multi

    def max_over_ranks(x: float) -> float:
        return multi.reduce_scalar(x, "max", device="cuda")

    def sum_over_ranks(x: float) -> float:
        return multi.reduce_scalar(x, "sum", device="cuda")

    n_cfg = args.configs
    caps = grids.g4_capacities()
    strong = args.scaling == "strong"
    shard_lo, whole = 0, None
    if strong:
        # one grid for all ranks: contiguous shards balanced by event count (the counts come from
        # llmem_event_counts on this rank's device; every rank computes the same cut)
        whole = grids.g5_stress(0, n_cfg)
        whole_offsets, _ = llmem.event_counts(whole)
        counts = torch.diff(whole_offsets).cpu().numpy()
        shard_lo, shard_hi = multi.shard_of(n_cfg, counts, rank, world)
        cfgs = whole[shard_lo:shard_hi]
        del whole_offsets
    else:
        cfgs = grids.g5_stress(0, n_cfg, seed_offset=rank)     # weak scaling: one full grid per rank
    hp = HotPath(llmem, torch, cfgs, caps, grids.G4_BMAX, one_pass=not args.two_pass)

    # ---- device-resident timing ----
    for _ in range(args.warmup):
        hp.step(record=False)
    hp.ev = {k: [] for k in hp.ev}
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
    except Exception:
        gpu_id = str(torch.cuda.current_device())
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    start.record()
    marks = []  # an event after every step: where the time of the region went, step by step
    for _ in range(args.steps):
        out = hp.step()
        marks.append(torch.cuda.Event(enable_timing=True))
        marks[-1].record()
    stop.record()
    barrier()
    wall1 = time.time()
    ms = max_over_ranks(start.elapsed_time(stop))
    per_step = [a.elapsed_time(b) for a, b in zip([start] + marks[:-1], marks)]
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    total_events_all = sum_over_ranks(float(hp.total))
    configs_all = sum_over_ranks(float(hp.n))
    value = total_events_all * args.steps / (ms * 1e-3)

    kernel_ms = {k: statistics.mean(a.elapsed_time(b) for a, b in v) for k, v in hp.ev.items()}
    status = llmem.lib().llmem_scratch_status(int(hp.scan_scratch.data_ptr()), None)
    if status != 0:
        print(json.dumps({"error": f"device status {status}"}))
        return 3
    # the two paths must agree on the device (cheap self-check outside the timed region)
    fused = llmem.estimate_batch(hp.cfg, want_status=False)
    agree = bool(torch.equal(fused["peak"], out["peak"]) and torch.equal(fused["index"], out["index"]))
    gathered_ok = None
    if strong:
        # the shards' results, gathered over the process group, against the fused estimate of the
        # whole grid computed on rank 0
        everything = {k: multi.gather_slices(out[k], n_cfg, shard_lo, device="cuda") for k in ("peak", "index", "method", "batch")}
        if rank == 0:
            ref = llmem.estimate_batch(whole, want_status=False)
            ref_sel = llmem.select_method(whole, caps, grids.G4_BMAX, want_bs_list=False, want_status=False)
            gathered_ok = bool(torch.equal(everything["peak"], ref["peak"]) and torch.equal(everything["index"], ref["index"]) and
                               torch.equal(everything["method"], ref_sel["method"]) and
                               torch.equal(everything["batch"], ref_sel["batch"]))
            del ref, ref_sel
        del everything

    # ---- end to end from host buffers ----
    hp.run_e2e(min(args.warmup, 3))
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    e2e_steps = max(1, min(args.steps, 100))
    hp.run_e2e(e2e_steps)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1))
    # what came back to the host must be what the device-resident step computed
    e2e_agree = bool(torch.equal(hp.host_out["peak"], out["peak"].cpu()) and
                     torch.equal(hp.host_out["method"], out["method"].cpu()) and
                     torch.equal(hp.host_out["batch"], out["batch"].cpu()))
    e2e_value = total_events_all * e2e_steps / (e2e_ms * 1e-3)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    peak_gbs, peak_src = measured_peaks()
    bytes_per_launch = 8.0 * hp.total          # 8 algorithmic bytes per event for each of the three kernels
    others = {k: hp.time_kernel(k) for k in ("expand", "scan", "expand_scan") if k not in kernel_ms}
    dom = max(kernel_ms, key=kernel_ms.get)
    achieved = bytes_per_launch / (kernel_ms[dom] * 1e-3) / 1e9

    def entry(ms_):
        g = bytes_per_launch / (ms_ * 1e-3) / 1e9
        return {"ms": ms_, "gbs": g, "frac": g / peak_gbs}
    roofline = {
        "bound": "hbm",
        "kernel": {"expand": "expand_kernel (8 B written / event)", "scan": "scan_kernel (8 B read / event)",
                   "expand_scan": "expand_scan_kernel (8 B written / event; the scan reads shared memory)"}[dom],
        "achieved": achieved, "peak": peak_gbs, "unit": "GB/s", "frac": achieved / peak_gbs,
        "peak_source": peak_src,
        "traffic": (NCU_TRAFFIC_BYTES_PER_EVENT[dom] * hp.total
                    if NCU_TRAFFIC_BYTES_PER_EVENT.get(dom) is not None else None),
        "traffic_note": "ncu dram bytes per event on a 4096-configuration capture, scaled by events",
        "algorithmic_bytes": bytes_per_launch,
        "per_kernel": {k: entry(v) for k, v in kernel_ms.items()},
        "other_path_kernels": {"note": "the kernels of the path not taken by the timed step, timed alone "
                                       "after it on the same grid (5 launches each)",
                               **{k: entry(v) for k, v in others.items()}},
        "frac_of_nominal_8000": achieved / 8000.0,
        "note": "the measured peak is a copy (read + write); a stream that only writes, or only reads, can exceed it: "
                "above 1 the fraction of the nominal 8 TB/s is the one to read",
    }
    step_text = ("event_counts + expand_scan (expansion, page rounding and segmented scan in one kernel, list "
                 "written to HBM once) + max_batch + select_method" if hp.one_pass else
                 "event_counts + expand(fused rounding) + scan_peak on the main stream; max_batch + "
                 "select_method concurrently on a second stream; both joined before the step ends")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "step_ms": {"median": statistics.median(per_step), "min": min(per_step), "max": max(per_step),
                    "note": "device time of the single timed steps on this rank (ms_per_step is the whole region / steps: "
                            "one pause of the box inside a short region shows as a large max here)"},
        "scaling": args.scaling, "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "configs_per_sec": configs_all * args.steps / (ms * 1e-3),
        "config": {"workload": "G5 stress grid: deep/wide decoders, materialised int64 event lists",
                   "configs_per_gpu": hp.n, "events_per_gpu": hp.total, "capacities": len(caps),
                   "bmax": grids.G4_BMAX,
                   "parallelism": (f"one grid cut into {world} contiguous shards balanced by event count; results "
                                   "gathered over NCCL outside the timed region" if strong else
                                   f"replicas x{world} (independent configs, no collective)"),
                   "l2": "event list (8 B/event) far larger than the 126 MB L2; no flush needed",
                   "path": "one-pass" if hp.one_pass else "two-pass", "step": step_text},
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": hp.h2d_bytes,
                "d2h_bytes_per_step": hp.d2h_bytes, "ms_per_step": e2e_ms / e2e_steps,
                "inputs": "configuration records and capacities from pinned host memory, every step",
                "outputs": "peak[n] int64, method[n, capacities] and batch[n, capacities] int32 to pinned host memory, "
                           "and the event total the host needs to size the list; peak positions, per-method "
                           "batches and status stay on the device"},
        "gpu_launches": hp.kernels_per_step * args.steps,
        "clocks": clocks,
        "fused_equals_materialised": agree, "e2e_equals_resident": e2e_agree,
    }
    if strong:
        line["gathered_equals_whole_grid"] = gathered_ok
    if world == 1 and args.secondary:
        # the other grids, shortly, with their own rooflines (device memory of the headline is released first)
        del hp, out, fused
        torch.cuda.empty_cache()
        line["secondary"] = {
            "g3": leg_estimate(llmem, torch, max(20, min(args.steps, 200)), args.warmup),
            "g4": leg_search(llmem, torch, max(5, min(args.steps, 20)), args.warmup),
            "g2": leg_slabs(llmem, torch, max(3, min(args.steps, 5)), args.warmup),
        }
        torch.cuda.empty_cache()
        line["secondary"]["classes"] = leg_classes(llmem, torch, 3, 1)
    if args.cpu_baseline:
        line["cpu_baseline"] = cpu_baseline()
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    ok = agree and e2e_agree and gathered_ok is not False
    if "secondary" in line:
        ok = ok and line["secondary"]["g2"]["fused_equals_materialised"] and line["secondary"]["g4"]["selection_equals_search"]
    return 0 if ok else 4


# ---------------------------------------------------------------------------
# secondary workloads: the kernels that generate events in registers (integer-ALU bound)
# and the shape grid through the materialised path in slabs
# ---------------------------------------------------------------------------
# Lane instructions executed per unit of work, as warp instructions with all 32 lanes busy
# (ncu smsp__thread_inst_executed.sum / 32 / units), from captures of these kernels on reduced
# grids (profiles/register_kernels_g3_g4_ncu.md); None once a kernel changes after the capture.
# Counting lane instructions keeps divergence from passing for throughput: a warp instruction
# issued for 20 of 32 lanes counts as 20/32.
NCU_LANE_INSTR_PER_UNIT = {"estimate_kernel": 21.78, "max_batch_kernel": 5.14, "select_kernel": 26.76}


def _gpu_id(torch):
    try:
        return "GPU-" + str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
    except Exception:
        return str(torch.cuda.current_device())


def _timed_steps(torch, step, steps, warmup, flush=None):
    """Mean device time (ms) of `steps` calls of step(), CUDA events on the current stream, L2
    flushed before every timed call when `flush` is given; clocks sampled meanwhile."""
    for _ in range(max(warmup, 3)):
        step()
    sampler = ClockSampler(_gpu_id(torch))
    sampler.start()
    time.sleep(0.3)
    torch.cuda.synchronize()
    wall0 = time.time()
    total_ms = 0.0
    for _ in range(steps):
        if flush is not None:
            flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step()
        e1.record()
        torch.cuda.synchronize()
        total_ms += e0.elapsed_time(e1)
    clocks = sampler.stop(wall0, time.time())
    return total_ms / steps, clocks


def _alu_roofline(torch, llmem, units, ms, clocks):
    """Issue-rate roofline of a per-configuration kernel: achieved = lane instructions of the
    model (as full warp instructions) per second, peak = SMs x 4 schedulers x sampled clock."""
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    mhz = clocks.get("sm_mhz") or 1965.0
    peak = sm * 4 * mhz * 1e6
    probe = {name: llmem.int_rate(kind) for kind, name in enumerate(("add_xor", "mad", "add_mad"))}
    instr = None
    if all(NCU_LANE_INSTR_PER_UNIT.get(k) is not None for k in units):
        instr = sum(NCU_LANE_INSTR_PER_UNIT[k] * u for k, u in units.items())
    return {"bound": "alu", "unit": "warp-instr/s", "peak": peak,
            "achieved": (instr / (ms * 1e-3)) if instr else None,
            "frac": (instr / (ms * 1e-3) / peak) if instr else None,
            "achieved_is": "lane instructions / 32 (ncu smsp__thread_inst_executed per unit x units / time): "
                           "idle lanes of a diverged warp do not count",
            "peak_source": "148 SMs x 4 schedulers x sampled SM clock (one warp instruction per cycle each)",
            "measured_issue_rates": probe,
            "frac_of_measured_add_mad": (instr / (ms * 1e-3) / probe["add_mad"]) if instr else None,
            "traffic": None}


def leg_estimate(llmem, torch, steps, warmup, n=None, repeat=16):
    """Fused estimate (no list) of the large sweep; also of the sweep repeated `repeat` times
    (2^24 configurations), where launch ramp and tail no longer weigh."""
    n = grids.G3_CONFIGS if n is None else n
    host = grids.g3_sweep(0, n)
    dev = llmem.to_device(host)
    big = dev.repeat(repeat, 1).contiguous()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    events = int(llmem.event_counts(dev)[0][-1].item())
    ms, clocks = _timed_steps(torch, lambda: llmem.estimate_batch(dev), steps, warmup, flush)
    ms_big, _ = _timed_steps(torch, lambda: llmem.estimate_batch(big), max(3, steps // 4), warmup, flush)
    ms_dnn, _ = _timed_steps(torch, lambda: llmem.estimate_batch(dev, estimator="dnnmem"), max(3, steps // 4), warmup, flush)
    roof = _alu_roofline(torch, llmem, {"estimate_kernel": n}, ms, clocks)
    roof_big = _alu_roofline(torch, llmem, {"estimate_kernel": n * repeat}, ms_big, clocks)
    return {"metric": "configs per second (fused estimate)", "value": n / (ms * 1e-3), "unit": "configs/s",
            "steps": steps, "ms_per_step": ms, "dtype": "int64",
            "config": {"workload": "G3 large sweep: fused estimate, event runs summed in registers (no list materialised)",
                       "configs": n, "virtual_events_per_config": events / n,
                       "l2": "256 MB write between timed steps flushes L2"},
            "roofline": roof,
            "repeated": {"configs": n * repeat, "ms_per_step": ms_big, "value": n * repeat / (ms_big * 1e-3),
                         "unit": "configs/s", "frac": roof_big["frac"],
                         "frac_of_measured_add_mad": roof_big["frac_of_measured_add_mad"]},
            "second_estimator": {"what": "the DNNMem-style estimate of Section 3.1 on the same records (those of another "
                                         "method than the conventional one get status 2)",
                                 "ms_per_step": ms_dnn, "value": n / (ms_dnn * 1e-3), "unit": "configs/s"},
            "gpu_launches": steps, "clocks": clocks}


def leg_search(llmem, torch, steps, warmup, shapes=None):
    """Largest-batch search (shapes x 4 methods x 16 degrees x 9 capacities) and Algorithm 1
    selection (shapes x 16 degrees x 9 capacities); the selection's batches are compared with
    the search's on the device."""
    shapes = grids.G4_SHAPES if shapes is None else shapes
    caps_np = grids.g4_capacities()
    caps = torch.from_numpy(caps_np).cuda()
    host = [grids.g4_search_grid(0, shapes), grids.g4_select_grid(0, shapes)]
    dev = [llmem.to_device(h) for h in host]
    units = {"max_batch_kernel": len(host[0]) * len(caps_np), "select_kernel": len(host[1]) * len(caps_np)}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def step():
        a = llmem.max_batch(dev[0], caps, grids.G4_BMAX, want_status=False)
        b = llmem.select_method(dev[1], caps, grids.G4_BMAX, want_bs_list=True, want_status=False)
        return a, b
    (bs, _), sel = step()
    # the four batches Algorithm 1 compared are those of the search grid, shape by shape
    bs4 = bs.clamp(min=0).reshape(shapes, 4, grids.G4_DEGREES, len(caps_np)).permute(0, 2, 3, 1).reshape(-1, len(caps_np), 4)
    agree = bool(torch.equal(sel["bs_list"], bs4))
    ms, clocks = _timed_steps(torch, step, steps, warmup, flush)
    n_units = units["max_batch_kernel"] + 4 * units["select_kernel"]
    return {"metric": "searches per second (max batch + Algorithm 1)", "value": n_units / (ms * 1e-3),
            "unit": "searches/s", "steps": steps, "ms_per_step": ms, "dtype": "int64",
            "config": {"workload": "G4 max-batch search + Algorithm 1 selection, batch 1..4096, a certain bracket from the near-linear page count and probes inside it, in registers",
                       "shapes": shapes, "searches": units["max_batch_kernel"], "selections": units["select_kernel"],
                       "l2": "256 MB write between timed steps flushes L2"},
            "roofline": _alu_roofline(torch, llmem, units, ms, clocks),
            "gpu_launches": 2 * steps, "clocks": clocks, "selection_equals_search": agree}


def leg_slabs(llmem, torch, steps, warmup, shapes=None):
    """The whole shape grid (3.8 M configurations, 4.3e10 events, 345 GB as int64) through the
    materialised path in slabs of 2^32 events sharing one 32 GiB list buffer.  One step = event
    counts of the grid, slab boundaries cut on the device, then per slab event counts,
    expansion with fused rounding and segmented scan (llmem_expand_scan)."""
    shapes = grids.G2_SHAPES if shapes is None else max(1, min(shapes, grids.G2_SHAPES))
    cfgs = grids.g2_shape_grid(0, shapes)
    dev = llmem.to_device(cfgs)
    budget = 1 << 32
    r = llmem.estimate_in_slabs(dev, budget)
    events = int(llmem.event_counts(dev)[0][-1].item())
    slabs = len(r["bounds"]) - 1
    fused = llmem.estimate_batch(dev)
    agree = bool(torch.equal(fused["peak"], r["peak"]) and torch.equal(fused["index"], r["index"]))
    del r, fused
    steps = max(1, min(steps, 20))
    ms, clocks = _timed_steps(torch, lambda: llmem.estimate_in_slabs(dev, budget), steps, warmup)
    peak_gbs, peak_src = measured_peaks()
    achieved = 8.0 * events / (ms * 1e-3) / 1e9
    return {"metric": METRIC, "value": events / (ms * 1e-3), "unit": UNIT, "steps": steps, "ms_per_step": ms,
            "dtype": "int64", "configs_per_sec": len(cfgs) / (ms * 1e-3),
            "config": {"workload": "G2 shape grid, materialised int64 event lists in slabs", "configs": len(cfgs),
                       "events": events, "slabs": slabs, "events_per_slab_max": budget,
                       "l2": "every slab's list is far larger than the 126 MB L2"},
            "roofline": {"bound": "hbm", "kernel": "whole step (per slab: counts, descriptor table, expand_scan_owned_kernel, "
                                                   "finishing pass; host slab loop)",
                         "achieved": achieved, "peak": peak_gbs, "unit": "GB/s", "frac": achieved / peak_gbs,
                         "frac_of_nominal_8000": achieved / 8000.0, "peak_source": peak_src,
                         "traffic": (NCU_TRAFFIC_BYTES_PER_EVENT_OWNERS * events
                                     if NCU_TRAFFIC_BYTES_PER_EVENT_OWNERS is not None else None),
                         "traffic_note": "ncu dram bytes per event of expand_scan_owned_kernel on a 64-shape capture, scaled by events",
                         "algorithmic_bytes": 8.0 * events},
            "gpu_launches": steps * (4 + slabs * 7), "clocks": clocks, "fused_equals_materialised": agree}


# lists of the shape grid by length: [lo, hi) events per list
LENGTH_CLASSES = ((1, 150), (150, 400), (400, 1500), (1500, 6000), (6000, 25000), (25000, 1 << 31))


def leg_classes(llmem, torch, steps, warmup, only=None):
    """Throughput by list length: about 4e8 events of shape-grid configurations from one length
    class each (the class's configurations repeated), through llmem_expand_scan,
    llmem_expand_events and llmem_scan_peak with CUDA events; `only` picks one class by number
    (for a profiler capture).  The lists (3.2 GB) are larger than L2."""
    import numpy as np
    cfgs = grids.g2_shape_grid(0, 512)
    counts = torch.diff(llmem.event_counts(llmem.to_device(cfgs))[0]).cpu().numpy()
    target = 400_000_000
    rows = []
    for k, (lo, hi) in enumerate(LENGTH_CLASSES):
        if only is not None and k != only:
            continue
        idx = np.nonzero((counts >= lo) & (counts < hi))[0]
        idx = idx[:int(np.searchsorted(np.cumsum(counts[idx]), target)) + 1]
        sub = np.tile(cfgs[idx], max(1, int(target // max(1, counts[idx].sum()))))
        dev = llmem.to_device(sub)
        offsets, _ = llmem.event_counts(dev)
        total = int(offsets[-1].item())
        delta = torch.empty(total, dtype=torch.int64, device="cuda")
        scratch = torch.empty(max(llmem.scratch_bytes(op, len(sub), total)
                                  for op in (llmem.OP_SCAN_PEAK, llmem.OP_EXPAND_SCAN, llmem.OP_EXPAND)),
                              dtype=torch.uint8, device="cuda")
        fused = llmem.estimate_batch(dev)
        row = {"events_per_list": [lo, hi], "lists": len(sub), "events": total, "mean_events": total / len(sub)}
        calls = (("expand_scan", lambda: llmem.expand_scan(dev, offsets, total, fuse_round=True, out=delta, scratch=scratch)),
                 ("expand", lambda: llmem.expand_events(dev, offsets, total, fuse_round=True, out=delta, scratch=scratch)),
                 ("scan", lambda: llmem.scan_peak(delta, offsets, dev, scratch=scratch)))
        for name, call in calls:  # the scan reads the list the expansion before it wrote
            best = None
            for it in range(max(warmup, 1) + max(steps, 1)):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                res = call()
                e1.record()
                torch.cuda.synchronize()
                if it >= max(warmup, 1):
                    best = e0.elapsed_time(e1) if best is None else min(best, e0.elapsed_time(e1))
            if name != "expand" and not (torch.equal(res["peak"], fused["peak"]) and torch.equal(res["index"], fused["index"])):
                raise SystemExit(f"{name} disagrees with the fused estimate on class {lo}..{hi}")
            row[name] = {"ms": best, "gbs": 8.0 * total / best / 1e6}
        rows.append(row)
        del dev, delta, scratch
    peak_gbs, peak_src = measured_peaks()
    return {"metric": METRIC, "unit": UNIT, "steps": steps, "dtype": "int64",
            "value": sum(r["events"] for r in rows) / sum(r["expand_scan"]["ms"] * 1e-3 for r in rows),
            "ms_per_step": sum(r["expand_scan"]["ms"] for r in rows),
            "config": {"workload": "shape-grid lists by length class, 4e8 events each: expand_scan / expand / scan",
                       "l2": "each list (3.2 GB) is larger than the 126 MB L2"},
            "classes": rows, "peak": peak_gbs, "peak_source": peak_src}


def run_secondary_workload(args):
    """--workload g3 | g4 | g2 | classes alone: one JSON line for that leg."""
    import torch
    import paper_2404_10933_b200 as llmem
    llmem.lib()
    torch.cuda.set_device(0)
    reduced = args.configs != grids.G5_CONFIGS
    if args.workload == "g3":
        leg = leg_estimate(llmem, torch, args.steps, args.warmup, min(args.configs, grids.G3_CONFIGS) if reduced else None)
    elif args.workload == "g4":
        leg = leg_search(llmem, torch, args.steps, args.warmup, min(args.configs, grids.G4_SHAPES) if reduced else None)
    elif args.workload == "classes":
        leg = leg_classes(llmem, torch, min(args.steps, 10), min(args.warmup, 3), args.length_class)
    else:
        leg = leg_slabs(llmem, torch, args.steps, args.warmup, args.configs if reduced else None)
    line = {"n_gpus": 1, "warmup": max(args.warmup, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "data": "synthetic", **leg}
    print(json.dumps(line))
    ok = leg.get("fused_equals_materialised", True) and leg.get("selection_equals_search", True)
    return 0 if ok else 4


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000,
                    help="timed steps (default 1000, about 6 s: long enough that a stray 0.1 s stall of the box does not move the result)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--configs", type=int, default=grids.G5_CONFIGS,
                    help="configurations of the stress grid per GPU (default: the full grid)")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--scaling", choices=("weak", "strong"), default="weak",
                    help="weak (default): every rank its own seeded grid; strong: one grid cut into shards balanced by event count")
    ap.add_argument("--no-secondary", dest="secondary", action="store_false",
                    help="skip the short legs on the other grids that a one-GPU run appends under 'secondary'")
    ap.add_argument("--two-pass", action="store_true",
                    help="time llmem_expand_events + llmem_scan_peak as separate kernels instead of llmem_expand_scan")
    ap.add_argument("--workload", choices=("g5", "g3", "g4", "g2", "classes"), default="g5",
                    help="g5 (default): the full hot path on the stress grid; g3 / g4: the in-register kernels; "
                         "g2: the shape grid through the materialised path in slabs; classes: the three list "
                         "entry points on shape-grid lists of one length class at a time")
    ap.add_argument("--length-class", type=int, default=None, choices=range(len(LENGTH_CLASSES)),
                    help="with --workload classes: only this class (0 = the shortest lists)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.workload != "g5":
        return run_secondary_workload(args)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world == 1 and args.gpus > 1:
        # launched without torchrun: re-launch one rank per GPU
        import socket
        with socket.socket() as sock:  # a port nobody else on this machine is using right now
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        return subprocess.call(cmd)
    if int(os.environ.get("RANK", "0")) != 0:
        args.cpu_baseline = False
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
