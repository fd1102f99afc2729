#!/usr/bin/env python
"""Benchmark of the batched model-variant selection path.

One step = one pass of the whole path over the 16M-query configuration (C3): one
`infaas_select_batch` over all 2^24 queries against the current load snapshot, then one
`infaas_load_update` that tallies those decisions, advances every queue by the time the
batch spans (256 windows' worth) and rebuilds the scan lists.  `value` is queries decided
per second with inputs resident in HBM; `e2e` repeats it with host buffers and the copies
inside the timed region.  The per-window pipeline (one update every 65,536 queries) and
the selection kernel alone are reported beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "queries decided/sec"
UNIT = "queries/s"
ALGO_BYTES_PER_QUERY = 12          # 2 (task) + 4 (slo) + 2 (min acc) read, 4 (decision) written
FALLBACK_HBM_GBS = 6650.0
ISSUE_PER_SM_CLK = 4
SELECT_STAT_LAUNCHES = 200         # the selection kernel's statistic comes from at least this many launches
# Counters of one selection-kernel launch on the 2^24-query workload under ncu (one capture,
# never taken from the run itself): DRAM bytes read + written, warp-instructions executed and
# L1 data-pipe wavefronts (shared memory + global; one per clock and SM at most).  They belong
# to the kernel source whose digest is recorded with them: when csrc/select.cu or
# csrc/common.cuh no longer match, every figure derived from them is reported as null.
NCU_CAPTURE = {
    "source_sha256_16": "dad366acf5783ebe",
    "workload": "C3",
    "dram_bytes": 134.58e6 + 26.87e6,
    "warp_instructions": 39.94e6,
    "l1_wavefronts": 11.32e6,          # 79.5 % of one per SM and elapsed clock over the launch
}
# end-to-end leg: shares of the batch per chunk (the rest is the last chunk)
E2E_CHUNK_SHARES = (0.36, 0.26, 0.18, 0.11, 0.06)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3", choices=["C2", "C3", "C4", "C5"])
    ap.add_argument("--queries", type=int, default=0, help="override the query count (testing)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the windowed / e2e legs")
    ap.add_argument("--check", action="store_true",
                    help="replay all steps on the CPU oracle and compare the final state (small --queries)")
    ap.add_argument("--split-update", action="store_true",
                    help="with one rank too, update through tally / count exchange / advance (the N > 1 path)")
    return ap.parse_args()


def kernel_source_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("select.cu", "common.cuh"):
        with open(os.path.join(ROOT, "paper_1905_13348_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_capture(workload_name: str):
    """The stored ncu counters, or None if they were taken on another kernel source or workload."""
    if NCU_CAPTURE["workload"] != workload_name or NCU_CAPTURE["source_sha256_16"] != kernel_source_digest():
        return None
    return NCU_CAPTURE


def on_chip_limits(cap, sel_ms: float, sm_mhz, sm_count: int):
    if not sm_mhz or cap is None:
        return None
    clk = sm_count * sm_mhz * 1e6 * sel_ms * 1e-3              # SM-clocks available to the launch
    return {"issue_slot_frac": cap["warp_instructions"] / (ISSUE_PER_SM_CLK * clk),
            "l1_data_pipe_frac": cap["l1_wavefronts"] / clk,
            "how": "ncu instruction and L1 wavefront counts of one launch / (SMs x sampled clock x event time)",
            "counters_of_source": cap["source_sha256_16"]}


def make_workload(name: str, queries: int):
    from paper_1905_13348_b200 import workloads as W
    if name == "C5":
        kw = {"n_windows": max(1, queries // 65536)} if queries else {}
    else:
        kw = {"n_queries": queries} if queries else {}
    return W.make(name, **kw)


def batch_window_us(w) -> int:
    """Length of the time the whole query array spans (all its windows)."""
    if w.window:
        return min(2**32 - 1, max(1, w.n_queries // w.window) * w.window_us)
    return 1_000_000


def workload_config(w, world: int = 1) -> dict:
    """Same dictionary for both arms (the reference arm times the oracle on the same workload)."""
    return {"workload": f"{w.name}: {w.recipe}", "n_tasks": w.n_tasks, "n_variants": w.n_variants,
            "n_queries": w.n_queries, "window_queries": w.window, "window_us": w.window_us,
            "step": "select_batch(all queries) + load_update(all decisions)",
            "l2": "GPU arm: two rotating input sets; per-step working set 12 B/query > 126 MB L2, no flush",
            "parallelism": (f"dp{world}: each rank decides its own queries against a replicated catalog; "
                            "one all-reduce of the per-variant counts per step") if world > 1 else "1 gpu"}


# ----------------------------------------------------------------------------------------
# clocks (read-only sampling during the timed region)
# ----------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake", 0x2: "applications_clocks_setting"}

    def __init__(self, cuda_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(cuda_index).uuid)
            uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # sampling is best effort
            self.error = repr(e)
        self._t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                for b, name in self.REASONS.items():
                    if bits & b:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0)          # back to back: an NVML query takes a fraction of a millisecond

    def __enter__(self):
        if self._h is not None:
            self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._h is not None:
            self._t.join()

    def summary(self) -> dict:
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------
# CPU oracle legs (the only place the benchmark touches oracle/)
# ----------------------------------------------------------------------------------------
def oracle_step(o, w, lo, hi, threads, window_us):
    d = o.select(w.task[lo:hi], w.slo_us[lo:hi], w.min_acc_bp[lo:hi], threads)
    o.load_update(d, window_us)
    return d


def cpu_baseline(w, target_s: float = 10.0, single_s: float = 6.0):
    """The oracle as it stands, on this host's cores, on a prefix of the same workload: all
    hardware threads (`value`) and one thread.  Also returns what the second roofline needs:
    the integer operations a 32-wide scan of the pruned lists would spend on the sample's
    decisions (oracle-side lists at the workload's initial load), scaled to the whole batch."""
    from oracle import OracleCatalog
    threads = os.cpu_count() or 1

    def timed(nthreads, seconds):
        o = OracleCatalog(w.rows, w.n_tasks)
        probe = min(w.n_queries, 1 << 16 if nthreads == 1 else 1 << 18)
        t0 = time.perf_counter()
        oracle_step(o, w, 0, probe, nthreads, 1000)
        rate = probe / max(1e-9, time.perf_counter() - t0)
        n = int(min(w.n_queries, max(probe, rate * seconds)))
        o = OracleCatalog(w.rows, w.n_tasks)
        t0 = time.perf_counter()
        d = o.select(w.task[:n], w.slo_us[:n], w.min_acc_bp[:n], nthreads)
        o.load_update(d, batch_window_us(w))
        return n, time.perf_counter() - t0, d

    n, dt, dec = timed(threads, target_s)
    n1, dt1, _ = timed(1, single_s)
    o = OracleCatalog(w.rows, w.n_tasks)
    ops = o.scan_ops(w.task[:n], dec) * (w.n_queries / n)
    base = {"value": n / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"first {n} of {w.n_queries} queries of {w.name}, select + load update, "
                      f"{dt:.1f} s wall on {threads} threads ({dt * threads:.0f} core-seconds)",
            "single_thread": {"value": n1 / dt1, "unit": UNIT, "cores": 1,
                              "sample": f"first {n1} queries, {dt1:.1f} s on one thread"}}
    return base, ops


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host, same metric and workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import OracleCatalog
    w = make_workload(args.workload, args.queries)
    threads = os.cpu_count() or 1
    o = OracleCatalog(w.rows, w.n_tasks)
    probe = min(w.n_queries, 1 << 18)
    t0 = time.perf_counter()
    oracle_step(o, w, 0, probe, threads, 1000)
    rate = probe / max(1e-9, time.perf_counter() - t0)
    total_steps = args.steps + args.warmup
    per_step = int(min(w.n_queries, max(1 << 14, rate * 90.0 / max(1, total_steps))))
    o = OracleCatalog(w.rows, w.n_tasks)
    wus = max(1, int(batch_window_us(w) * per_step / w.n_queries))
    for _ in range(args.warmup):
        oracle_step(o, w, 0, per_step, threads, wus)
    t0 = time.perf_counter()
    for k in range(args.steps):
        lo = (k * per_step) % max(1, w.n_queries - per_step + 1)
        oracle_step(o, w, lo, lo + per_step, threads, wus)
    dt = time.perf_counter() - t0
    value = args.steps * per_step / dt
    sample = f"{per_step} queries of {w.name} per step (select + load update)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32",
        "data": "synthetic", "config": workload_config(w, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ----------------------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_1905_13348_b200 as P
    from paper_1905_13348_b200 import sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = make_workload(args.workload, args.queries)
    n = w.n_queries
    wus_batch = batch_window_us(w)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks, local)

    def dev_i(a, view):
        return torch.from_numpy(a.view(view)).to(dev)

    # two rotating copies of the inputs: the working set (2 x 8 B + 4 B per query) is far
    # larger than L2, so no step starts with its inputs cached
    inputs = [(dev_i(w.task, np.int16), dev_i(w.slo_us, np.int32), dev_i(w.min_acc_bp, np.int16))
              for _ in range(2)]
    d_dec = torch.empty(n, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    # N > 1: every rank decides its own 2^24 queries of a window N times as long against the
    # same catalog; the per-variant counts are summed over the ranks (NCCL all-reduce of
    # n_variants u32) before every rank advances its catalog with them
    split = world > 1 or args.split_update
    d_cnt = torch.zeros(w.n_variants, dtype=torch.int32, device=dev) if split else None
    wus_step = min(2**32 - 1, wus_batch * world)

    def update(dec, st):
        if not split:
            P.infaas_load_update(cat, dec, wus_step, stream=st)
        else:
            P.infaas_tally(cat, dec, stream=st)
            P.infaas_pending_counts(cat, d_cnt, set=False, stream=st)
            with torch.cuda.stream(st):
                sharding.allreduce_sum_(d_cnt)
            P.infaas_pending_counts(cat, d_cnt, set=True, stream=st)
            P.infaas_advance(cat, wus_step, stream=st)

    def step(k, evs=None):
        t, s, a = inputs[k & 1]
        if evs is not None:
            evs[0].record(stream)
        P.infaas_select_batch(cat, t, s, a, d_dec, stream=stream)
        if evs is not None:
            evs[1].record(stream)
        update(d_dec, stream)
        if evs is not None:
            evs[2].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    warm = max(3, args.warmup)
    for k in range(warm):
        step(k)
    P.infaas_catalog_get_state(cat)          # also resizes the staging buffer to the live lists
    # the K timed steps, then (untimed for `value`) as many more as the selection kernel's
    # statistic needs; the clock sampler runs over both
    n_stat = max(args.steps, SELECT_STAT_LAUNCHES)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_stat)]
    barrier()
    with ClockSampler(local) as clocks:
        for k in range(args.steps):
            step(k, evs[k])
        barrier()
        for k in range(args.steps, n_stat):
            step(k, evs[k])
        torch.cuda.synchronize()
    total_ms = evs[0][0].elapsed_time(evs[args.steps - 1][2])
    sel_ms = [e[0].elapsed_time(e[1]) for e in evs]
    upd_ms = [e[1].elapsed_time(e[2]) for e in evs]
    total_ms = sharding.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = world * n / (ms_per_step * 1e-3)
    state = P.infaas_catalog_get_state(cat)
    info = P.infaas_catalog_get_info(cat)
    dec_host = d_dec.cpu().numpy().view(np.uint32)
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count

    if args.check:
        check_against_oracle(w, world, warm + n_stat, wus_step, state, dec_host)

    peak, peak_kind = measured_hbm_peak()
    sel_avg_ms = sum(sel_ms) / len(sel_ms)
    achieved = ALGO_BYTES_PER_QUERY * n / (sel_avg_ms * 1e-3) / 1e9
    cap = ncu_capture(w.name) if n == (1 << 24) else None
    clk = clocks.summary()
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": workload_config(w, world),
        "gpu_launches": 3 * args.steps,
        "kernels_ms": {"select": sel_avg_ms, "select_median": statistics.median(sel_ms),
                       "select_launches_timed": len(sel_ms),
                       "tally_plus_rebuild": sum(upd_ms) / len(upd_ms)},
        "roofline": {"bound": "hbm", "kernel": "select_kernel", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "traffic": None if cap is None else cap["dram_bytes"],
                     "launches_timed": len(sel_ms)},
        # the same launch against the SM's own limits at the clock sampled during the run:
        # issue slots (4 warp-instructions per SM and clock) and the L1 data pipe (1 wavefront)
        "on_chip_limits": on_chip_limits(cap, sel_avg_ms, clk.get("sm_mhz"), sm_count),
        "clocks": clk,
        "decisions": {"feasible": int(((dec_host >> 31) == 0).sum()),
                      "no_feasible": int((((dec_host >> 31) == 1) & (dec_host != 0xFFFFFFFF)).sum()),
                      "invalid": int((dec_host == 0xFFFFFFFF).sum()),
                      "queued_max": int(state["queued"].max())},
        "lookup": dict(info, staged_in_shared_memory=info["image_bytes"] <= info["image_smem"]),
    }

    if not args.no_extras:
        out["select_only"] = {"value": world * n / (sel_avg_ms * 1e-3), "unit": UNIT, "ms": sel_avg_ms}
        out["e2e"] = e2e_leg(P, cat, w, dev, update, max(3, min(10, args.steps)), world, dist)
        if w.window and world == 1:
            # from the workload's own initial state, whatever the steps above left behind
            cat_w = P.infaas_catalog_load(w.rows, w.n_tasks, local)
            out["windowed"] = windowed_leg(P, cat_w, w, inputs[0], d_dec, world)
            cat_w.free()
            out["stateful"] = stateful_leg(P, w, inputs, d_dec, local, peak)
            out["autoscale"] = autoscale_leg(P, w, inputs[0], d_dec, local)
            out["workers"] = workers_leg(P, w, cat, d_dec, peak)
    else:
        out["e2e"] = None
    cat.free()
    if rank == 0 and world == 1:
        out["int_pipe"] = int_pipe_leg(P, dev, local)
        if not args.no_cpu_baseline:
            out["cpu_baseline"], scan_ops = cpu_baseline(w)
            # the second roofline: the feasibility scan's integer operations at the measured
            # integer-pipe rate; the slower of the two bounds is the binding one
            t_hbm = ALGO_BYTES_PER_QUERY * n / (peak * 1e9)
            t_int = scan_ops / out["int_pipe"]["lane_ops_per_s"]
            out["roofline_scan_ops"] = {
                "bound": "alu", "ops_per_launch": scan_ops, "peak": out["int_pipe"]["lane_ops_per_s"],
                "unit": "lane-ops/s", "achieved": scan_ops / (sel_avg_ms * 1e-3),
                "frac": t_int / (sel_avg_ms * 1e-3), "time_at_peak_ms": 1e3 * t_int,
                "how": "3 x 32 x ceil(position / 32) per feasible query, 9 x list length per query without "
                       "a feasible variant; lists and decisions from the oracle on the CPU-baseline sample, "
                       "scaled to the batch; the kernel itself looks positions up instead of scanning"}
            out["binding_roofline"] = {"name": "scan_ops" if t_int > t_hbm else "hbm",
                                       "hbm_time_ms": 1e3 * t_hbm, "scan_ops_time_ms": 1e3 * t_int,
                                       "frac_of_binding": max(t_int, t_hbm) / (sel_avg_ms * 1e-3)}
        if not args.no_extras:
            del inputs, d_dec
            torch.cuda.empty_cache()
            out["per_config"] = per_config_leg(P, local, peak, {w.name: (sel_avg_ms, n, info)})
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def check_against_oracle(w, world, steps_run, wus_step, state, dec_host):
    """--check: replay every step on the CPU oracle (each step's decisions tallied `world` times,
    which is what the summed counts of `world` ranks with the same queries amount to) and
    compare the final load state and the last decisions.  Meant for small --queries."""
    from oracle import OracleCatalog
    o = OracleCatalog(w.rows, w.n_tasks)
    d = None
    for _ in range(steps_run):
        d = o.select(w.task, w.slo_us, w.min_acc_bp, os.cpu_count() or 1)
        o.load_update(np.tile(d, world), wus_step)
    # the last step's decisions were taken before its update
    if not np.array_equal(d, dec_host):
        raise SystemExit("--check: decisions of the last step differ from the oracle's")
    if not np.array_equal(o.queued, state["queued"]) or not np.array_equal(o.served_total, state["served_total"]):
        raise SystemExit("--check: load state differs from the oracle's")
    print(f"check ok: {steps_run} steps, world {world}", file=sys.stderr)


def int_pipe_leg(P, dev, local):
    """Sustained 32-bit integer lane-operations per second over all SMs (add, xor, compare,
    conditional add in independent chains), with the SM clock sampled meanwhile."""
    import torch
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        P.infaas_intpipe_probe(2048, sink, stream=stream)
    reps = 10
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    with ClockSampler(local) as clocks:
        e0.record(stream)
        for _ in range(reps):
            ops = P.infaas_intpipe_probe(8192, sink, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    sms = torch.cuda.get_device_properties(local).multi_processor_count
    mhz = clocks.summary().get("sm_mhz")
    rate = ops / (ms * 1e-3)
    return {"lane_ops_per_s": rate, "ms_per_launch": ms, "lane_ops_per_launch": ops, "sm_mhz": mhz,
            "lane_ops_per_sm_clk": rate / (sms * mhz * 1e6) if mhz else None,
            "how": "infaas_intpipe_probe: 2 CTAs x 1024 threads per SM, 8 independent chains per thread"}


def per_config_leg(P, local, peak, known):
    """Selection kernel alone on every configuration at its full size (one launch over all its
    queries against the catalog's initial load): mean CUDA-event time and fraction of the HBM
    roofline.  `known`: configurations already measured in this run."""
    import torch
    from paper_1905_13348_b200 import workloads as W
    dev = torch.device("cuda", local)
    stream = torch.cuda.current_stream()
    res = {}
    for name in ("C1", "C2", "C3", "C4", "C5"):
        if name in known:
            ms, n, info = known[name]
            note = "the benchmark step's state"
        else:
            w = W.make(name)
            n = w.n_queries
            cat = P.infaas_catalog_load(w.rows, w.n_tasks, local)
            # enough rotating sets of inputs and outputs that no launch finds its data in L2
            sets = max(1, min(64, -(-(300 << 20) // (12 * n))))
            inp = [(torch.from_numpy(w.task.view(np.int16)).to(dev), torch.from_numpy(w.slo_us.view(np.int32)).to(dev),
                    torch.from_numpy(w.min_acc_bp.view(np.int16)).to(dev), torch.empty(n, dtype=torch.int32, device=dev))
                   for _ in range(sets)]
            reps = 30
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            for k in range(3 + reps):
                if k >= 3:
                    evs[k - 3][0].record(stream)
                P.infaas_select_batch(cat, *inp[k % sets], stream=stream)
                if k >= 3:
                    evs[k - 3][1].record(stream)
            torch.cuda.synchronize()
            ms = sum(a.elapsed_time(b) for a, b in evs) / reps
            info = P.infaas_catalog_get_info(cat)
            cat.free()
            del inp
            note = f"initial load; {sets} rotating sets of inputs and outputs"
        gbs = ALGO_BYTES_PER_QUERY * n / (ms * 1e-3) / 1e9
        res[name] = {"n_queries": n, "select_ms": ms, "gbs": gbs, "frac_of_hbm_peak": gbs / peak,
                     "image_bytes": info["image_bytes"], "image_in_shared_memory": info["image_bytes"] <= info["image_smem"],
                     "longest_list": info["longest_list"], "state": note}
    return res


def e2e_leg(P, cat, w, dev, update, steps, world, dist):
    """Same step with HOST inputs and outputs: pinned host arrays are copied to the device,
    decided, and the decisions copied back, all inside the timed region.  The work is chunked
    and pipelined over three streams so that upload, kernels and download overlap; every step's
    selection still sees the load update of the step before."""
    import torch
    n = w.n_queries
    h_task = torch.from_numpy(w.task.view(np.int16)).pin_memory()
    h_slo = torch.from_numpy(w.slo_us.view(np.int32)).pin_memory()
    h_acc = torch.from_numpy(w.min_acc_bp.view(np.int16)).pin_memory()
    h_dec = torch.empty(n, dtype=torch.int32).pin_memory()
    # two sets of device arrays: the upload of one step runs while the previous step's last
    # chunk is still being decided, downloaded and tallied
    dsets = [(torch.empty(n, dtype=torch.int16, device=dev), torch.empty(n, dtype=torch.int32, device=dev),
              torch.empty(n, dtype=torch.int16, device=dev), torch.empty(n, dtype=torch.int32, device=dev))
             for _ in range(2)]
    # few, large copies (each costs some 4-10 us of set-up on top of its bytes), shrinking
    # towards the end so that little is left to do after the last upload
    bounds, lo = [], 0
    for share in E2E_CHUNK_SHARES:
        hi = min(n, lo + max(8, int(n * share) // 8 * 8))
        if hi > lo:
            bounds.append((lo, hi))
        lo = hi
    if lo < n:
        bounds.append((lo, n))
    up, comp, down = (torch.cuda.Stream(dev) for _ in range(3))
    ev_up = [[torch.cuda.Event() for _ in bounds] for _ in range(2)]
    ev_sel = [[torch.cuda.Event() for _ in bounds] for _ in range(2)]
    ev_updated = [torch.cuda.Event() for _ in range(2)]      # the step that used this set has been tallied
    ev_down = [torch.cuda.Event() for _ in range(2)]         # ... and its decisions are on the host
    main = torch.cuda.current_stream()
    for st in (up, comp, down):
        st.wait_stream(main)
    for s_ in range(2):
        ev_updated[s_].record(comp)
        ev_down[s_].record(down)
    host = [tuple(x[lo:hi] for x in (h_task, h_slo, h_acc, h_dec)) for lo, hi in bounds]
    devv = [[tuple(x[lo:hi] for x in dset) for lo, hi in bounds] for dset in dsets]
    count = [0]

    def step():
        # upload, selection (+ the load update, which the next step's selection must see) and
        # download each on a stream of their own, chained per chunk by events
        k = count[0] & 1
        count[0] += 1
        up.wait_event(ev_updated[k])           # the inputs of the step before last have been read
        comp.wait_event(ev_down[k])            # ... and its decisions copied out
        for i, (ht, hs, ha, hd) in enumerate(host):
            dt_, ds, da, dd = devv[k][i]
            with torch.cuda.stream(up):
                dt_.copy_(ht, non_blocking=True)
                ds.copy_(hs, non_blocking=True)
                da.copy_(ha, non_blocking=True)
                ev_up[k][i].record(up)
            comp.wait_event(ev_up[k][i])
            P.infaas_select_batch(cat, dt_, ds, da, dd, stream=comp)
            ev_sel[k][i].record(comp)
            down.wait_event(ev_sel[k][i])
            with torch.cuda.stream(down):
                hd.copy_(dd, non_blocking=True)
        ev_down[k].record(down)
        update(dsets[k][3], comp)
        ev_updated[k].record(comp)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([dt], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dt = float(t.item())
    return {"value": world * n * steps / dt, "unit": UNIT, "h2d_bytes_per_step": 8 * n,
            "d2h_bytes_per_step": 4 * n, "ms_per_step": 1e3 * dt / steps, "steps": steps,
            "how": f"pinned host -> device copies, select and download per chunk ({len(bounds)} chunks of "
                   "decreasing size; upload / select + load update / download streams chained by events; "
                   "two sets of device arrays, so a step's upload overlaps the end of the step before); "
                   "host wall clock around synchronize"}


def windowed_leg(P, cat, w, inp, d_dec, world):
    """The workload as a stream of windows: select one window, update the load, repeat.
    All windows are captured once into a CUDA graph (the calls only launch kernels), so the
    timing shows the device-side dependency chain and not the Python call overhead.  The
    catalog keeps its load from one pass over the windows to the next: the timed passes are
    the fourth to the eighth, when the queues have settled."""
    import torch
    t, s, a = inp
    W_ = w.window
    nwin = w.n_queries // W_
    side = torch.cuda.Stream()

    def run(stream):
        for k in range(nwin):
            lo, hi = k * W_, (k + 1) * W_
            P.infaas_select_update(cat, t[lo:hi], s[lo:hi], a[lo:hi], d_dec[lo:hi], w.window_us, stream=stream)

    # the same chain of dependent launches with nothing in them: what the window costs before any work
    tick = torch.zeros(1, device=t.device)

    def run_empty(stream):
        for _ in range(2 * nwin):
            tick.add_(1.0)

    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        run(side)                      # plain pass first (also warms the kernels up)
        side.synchronize()
        t0 = time.perf_counter()
        run(side)
        side.synchronize()
        eager_ms = 1e3 * (time.perf_counter() - t0)
        P.infaas_catalog_get_state(cat, stream=side)   # lets the library re-plan its shared memory for the lists as they are now
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            run(side)
        graph.replay()
        side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 5
        e0.record(side)
        for _ in range(reps):
            graph.replay()
        e1.record(side)
        side.synchronize()
        floor_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(floor_graph, stream=side):
            run_empty(side)
        floor_graph.replay()
        side.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(side)
        for _ in range(reps):
            floor_graph.replay()
        f1.record(side)
        side.synchronize()
    ms = e0.elapsed_time(e1) / reps
    floor_ms = f0.elapsed_time(f1) / reps
    info = P.infaas_catalog_get_info(cat, stream=side)
    return {"value": world * nwin * W_ / (ms * 1e-3), "unit": UNIT, "windows": nwin,
            "windows_before_timing": 3 * nwin, "lists_after": {k: info[k] for k in ("image_bytes", "longest_list", "list_entries")},
            "window_queries": W_, "us_per_window": 1e3 * ms / nwin, "gpu_launches_per_window": 2,
            "us_per_window_floor": 1e3 * floor_ms / nwin,
            "floor_how": "the same graph shape with two one-element kernels per window instead of selection and rebuild",
            "how": "CUDA graph of all windows, one infaas_select_update per window (selection with its own "
                   "tally, then the rebuild)", "us_per_window_python_calls": 1e3 * eager_ms / nwin}


def stateful_leg(P, w, inputs, d_dec, local, peak):
    """The same workload with a life-cycle state and a loading latency per variant
    (state-aware selection; states move with the load at every update): the selection kernel
    over all queries against the initial states, then the stream of windows."""
    import torch
    from paper_1905_13348_b200 import workloads as W
    state, load = W.variant_states(w.n_variants)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks, local)
    P.infaas_catalog_set_states(cat, state, load)
    stream = torch.cuda.current_stream()
    reps = 20
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for k in range(3 + reps):
        t, s, a = inputs[k & 1]
        if k >= 3:
            evs[k - 3][0].record(stream)
        P.infaas_select_batch(cat, t, s, a, d_dec, stream=stream)
        if k >= 3:
            evs[k - 3][1].record(stream)
    torch.cuda.synchronize()
    sel_ms = sum(e0.elapsed_time(e1) for e0, e1 in evs) / reps
    dec = d_dec.cpu().numpy().view(np.uint32)
    ok = dec[(dec >> 31) == 0]
    info = P.infaas_catalog_get_info(cat)
    win = windowed_leg(P, cat, w, inputs[0], d_dec, 1)
    end = P.infaas_catalog_get_states(cat)
    cat.free()
    gbs = ALGO_BYTES_PER_QUERY * w.n_queries / (sel_ms * 1e-3) / 1e9
    return {"select_ms": sel_ms, "select_gbs": gbs, "select_frac_of_hbm_peak": gbs / peak,
            "decisions": {"active": int((state[ok] == 1).sum()), "inactive": int((state[ok] == 0).sum()),
                          "no_feasible": int((((dec >> 31) == 1) & (dec != 0xFFFFFFFF)).sum()),
                          "invalid": int((dec == 0xFFFFFFFF).sum())},
            "states_start": np.bincount(state, minlength=4).tolist(),
            "states_after_windows": np.bincount(end, minlength=4).tolist(),
            "list_entries": info["list_entries"], "image_bytes": info["image_bytes"],
            "windowed_us_per_window": win["us_per_window"], "windowed_value": win["value"], "unit": UNIT}


def autoscale_leg(P, w, inp, d_dec, local):
    """Scaling-up step of the Model-Autoscaler on one window's tallies: every variant that
    served queries in the window runs one instance, each task's SLO is the median SLO of its
    queries, slack 1.05 (the paper's value), lambda 0.1/s.  One small kernel per window."""
    import torch
    from paper_1905_13348_b200 import workloads as W
    t, s, a = inp
    W_ = w.window
    cat = P.infaas_catalog_load(w.rows, w.n_tasks, local)
    _, load = W.variant_states(w.n_variants)
    P.infaas_catalog_set_states(cat, np.ones(w.n_variants, np.uint8), load)
    P.infaas_select_batch(cat, t[:W_], s[:W_], a[:W_], d_dec[:W_])
    P.infaas_tally(cat, d_dec[:W_])
    torch.cuda.synchronize()
    dec = d_dec[:W_].cpu().numpy().view(np.uint32)
    served = np.bincount(dec[(dec >> 31) == 0], minlength=w.n_variants)
    slo = np.array([np.median(w.slo_us[:W_][w.task[:W_] == k]) if (w.task[:W_] == k).any() else 0
                    for k in range(w.n_tasks)], np.uint32)
    P.infaas_autoscale_config(cat, (served > 0).astype(np.uint32), slo)
    d_v = torch.empty(w.n_tasks, dtype=torch.int32, device="cuda")
    d_d = torch.empty(w.n_tasks, dtype=torch.int32, device="cuda")
    # 50 calls in one CUDA graph: the kernel is far shorter than a Python call
    side = torch.cuda.Stream()
    reps = 50
    with torch.cuda.stream(side):
        for _ in range(3):
            P.infaas_autoscale_step(cat, w.window_us, 105, 100, d_v, d_d, stream=side)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(reps):
                P.infaas_autoscale_step(cat, w.window_us, 105, 100, d_v, d_d, stream=side)
        graph.replay()
        side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        graph.replay()
        e1.record(side)
        side.synchronize()
    us = 1e3 * e0.elapsed_time(e1) / reps
    v = d_v.cpu().numpy().view(np.uint32)
    d = d_d.cpu().numpy().view(np.uint32)
    cat.free()
    act = v < 0xFFFFFFFE
    return {"us_per_step": us, "tasks": w.n_tasks, "window_queries": W_, "window_us": w.window_us,
            "tasks_scaling": int(act.sum()), "tasks_with_headroom": int((v == 0xFFFFFFFF).sum()),
            "tasks_escalated": int((v == 0xFFFFFFFE).sum()), "instances_added": int(d[act].sum()),
            "how": "50 calls in one CUDA graph",
            "bound": "latency (one CTA per task over ~30 B per variant)"}


def workers_leg(P, w, cat, d_dec, peak):
    """Worker choice for all decisions of the batch: 1,000 workers over four hardware codes,
    half of the variants loaded on one to three of them.  A gather: 4 B read + 4 B written per
    query."""
    import torch
    rng = np.random.Generator(np.random.PCG64([7, 0]))
    n_workers = 1000
    loaded = np.flatnonzero(rng.random(w.n_variants) < 0.5)
    iv = np.repeat(loaded, rng.integers(1, 4, loaded.size)).astype(np.uint32)
    P.infaas_workers_config(cat, iv, rng.integers(0, n_workers, iv.size).astype(np.uint32),
                            rng.integers(0, 1000, iv.size).astype(np.uint32),
                            rng.integers(0, 4, n_workers).astype(np.uint8),
                            rng.integers(0, 10000, n_workers).astype(np.uint32))
    d_w = [torch.empty_like(d_dec) for _ in range(2)]
    stream = torch.cuda.current_stream()
    reps = 20
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for k in range(3 + reps):
        if k >= 3:
            evs[k - 3][0].record(stream)
        P.infaas_assign_workers(cat, d_dec, d_w[k & 1], stream=stream)
        if k >= 3:
            evs[k - 3][1].record(stream)
    torch.cuda.synchronize()
    ms = sum(e0.elapsed_time(e1) for e0, e1 in evs) / reps
    gbs = 8 * w.n_queries / (ms * 1e-3) / 1e9
    return {"ms": ms, "gbs": gbs, "frac_of_hbm_peak": gbs / peak, "bytes_per_query": 8, "workers": n_workers,
            "instances": int(iv.size), "assigned": int((d_w[0] != -1).sum().item()),
            "l2": "decisions + two output buffers = 201 MB > 126 MB L2"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
