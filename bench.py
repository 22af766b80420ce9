#!/usr/bin/env python
"""Benchmark of the strategy-search path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 3] [--impl reference]

A step is one pass of the whole path over one batch of synthetic search
instances: cost model -> validation -> layer-wise min-plus recurrence ->
optimum -> plan backtrack.  Prints ONE JSON line (rank 0).

Metric: DP cell updates per second (cells = sum_i L_i * (M+1) * S); searches/s
and min-plus relaxations/s are reported beside it.  With N > 1 every rank runs
its own batch of independent instances (no exchange on the data path; weak
scaling); the time is the maximum over ranks.

--impl reference times the CPU oracle (plain C, one instance per thread) on a
bounded sample of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2504_03662_b200 import inputs  # noqa: E402

METRIC, UNIT = "dp_cell_updates_per_s", "cells/s"
# Integer-ALU peak of one B200: 148 SMs x 64 int32 lanes x 1.965 GHz, one fused add-min
# (one min-plus relaxation) per lane per clock.
ALU_PEAK_GOPS = 148 * 64 * 1.965
# DRAM bytes (read + write) per LAYER of the layer_tiled_kernel, from the committed ncu captures under
# profiles/ (captured on the first layers of the same batch: the kernel's traffic grows in proportion
# to the layers a launch covers, so a launch over Lmax-1 layers moves (Lmax-1) times this).
NCU_TRAFFIC_BYTES_PER_LAYER = {"config3_heterogeneous": 533.6e6, "config4_research_sweep": 541.1e6}


def workload_for(k: int, rank: int = 0, batch: int = 0, layers: int = 0):
    """Workload k; ranks > 0 of a multi-GPU run get other instances of the same shape (other seed / other jitter)."""
    if rank and k in (0, 4):
        w = inputs.CONFIGS[k](seed=(0 if k == 0 else 7) + 1000 * rank)
    else:
        w = inputs.CONFIGS[k]()
    if rank and w.has_model:
        # the same model searched under other measured rates: two draws per instance scale the FLOP rate and the
        # link bandwidth by a factor in [0.8, 1.2), as the heterogeneous workload does on rank 0
        u = inputs._unit(inputs.splitmix64(3 + 1000 * rank, 2 * w.B)).reshape(w.B, 2)
        w.inst["flops_rate"] = 1e15 * (0.8 + 0.4 * u[:, 0])
        w.inst["bw_tp"] = w.inst["bw_dp"] = 450e9 * (0.8 + 0.4 * u[:, 1])
    if batch or layers:
        # trimmed copy of the workload (first `batch` instances, first `layers` layers) for profiler captures
        w = w.take(slice(0, batch or w.B))
        if layers and layers < w.Lmax:
            w.Lmax = layers
            w.L = np.minimum(w.L, layers).astype(np.int32)
            if w.has_model:
                w.layers = np.ascontiguousarray(w.layers[:, :layers])
            else:
                w.time_q = np.ascontiguousarray(w.time_q[:, :layers]); w.mem_q = np.ascontiguousarray(w.mem_q[:, :layers])
        w.name += f"[B={w.B},L={w.Lmax}]"
    return w


def input_checksums(w) -> dict:
    """FNV-1a-64 of the first 64 KiB of every input array of the workload (hex)."""
    arrays = (("L", w.L), ("layers", w.layers), ("strat", w.strat), ("inst", w.inst),
              ("time_q", w.time_q), ("mem_q", w.mem_q), ("trans_q", w.trans_q))
    return {name: f"{inputs.fnv1a64(a):016x}" for name, a in arrays if a is not None}


def spawn_ranks(n: int) -> int:
    """Re-run this command as n ranks of one node (one process per GPU, NCCL rendezvous on the loopback address)."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


# ------------------------------------------------------------------ CPU oracle legs

ORACLE_RELAX_PER_S_PER_THREAD = 1.3e9          # what the plain C oracle does on one host core (measured on the GPU machine's hosts)


def oracle_sample_size(w, threads: int, seconds: float):
    """(instances, layers) of a sample of the workload that keeps `threads` oracle threads busy for about `seconds`."""
    per_layer = (w.M + 1) * w.S * w.S
    budget = seconds * ORACLE_RELAX_PER_S_PER_THREAD               # relaxations per thread
    layers = int(w.Lmax)
    if per_layer * max(1, layers - 1) > budget:                     # one instance is already too long: fewer layers
        layers = max(2, int(budget / per_layer) + 1)
        return min(threads, w.B), layers
    per_thread = max(1, int(budget / (per_layer * max(1, layers - 1))))
    return min(w.B, threads * per_thread), layers


def oracle_sample(w, max_layers: int, threads: int, instances: int = 0):
    """First `instances` (default: one per thread) instances, first `max_layers` layers each: integer tables from the oracle's cost model."""
    from oracle import oracle
    k = min(instances or threads, w.B)
    items = []
    for i in range(k):
        Li = min(int(w.L[i]), max_layers)
        if w.has_model:
            _, _, tq, mq, xq = oracle.eval_costs(w.layers[0 if w.layers.shape[0] == 1 else i], w.strat, w.inst[i], Li)
        else:
            tq, mq, xq = w.time_q[i, :Li], w.mem_q[i, :Li], w.trans_q[i]
        items.append((np.ascontiguousarray(tq), np.ascontiguousarray(mq), np.ascontiguousarray(xq)))
    cells = sum(t.shape[0] for t, _, _ in items) * (w.M + 1) * w.S
    return items, cells


def oracle_run(w, items, threads: int) -> float:
    """Seconds for the oracle to search every sampled instance (one instance per thread)."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle

    def one(it):
        return oracle.search(it[0], it[1], it[2], w.M)["opt_cost"]

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(one, items))
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle
    oracle.build()
    w = workload_for(args.workload)
    threads = min(os.cpu_count() or 1, w.B)
    n_inst, max_layers = oracle_sample_size(w, threads, 4.0)         # ~4 s of work per thread and step
    items, cells = oracle_sample(w, max_layers, threads, n_inst)
    for _ in range(args.warmup):
        oracle_run(w, items, threads)
    ts = [oracle_run(w, items, threads) for _ in range(args.steps)]
    t = sum(ts) / len(ts)
    value = cells / t
    sample = f"first {len(items)} instances x first {max_layers} layers per step, one instance at a time per thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "Lmax": w.Lmax, "S": w.S, "M": w.M, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.rows, self.proc, self.uuid = [], None, uuid

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = [n for k, n in enumerate(names) if any(len(r) >= 7 and r[3 + k] == "Active" for r in self.rows)]
        pw = [float(r[2]) for r in self.rows if len(r) >= 7 and r[2].replace(".", "").isdigit()]
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(self.rows[0][1]), "reasons": reasons,
                "samples": len(sm), "power_w_max": max(pw) if pw else None}


# ------------------------------------------------------------------ GPU arm

def time_steps(torch, fn, steps, warmup, barrier):
    """CUDA-event time of `steps` calls of fn on the current stream, in seconds (after warm-up, barriers both sides)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record()
    for k in range(steps):
        fn()
        ev[k + 1].record()                                       # between steps: lets median and best be reported
    torch.cuda.synchronize()
    barrier()
    LAST_STEP_MS[:] = [ev[k].elapsed_time(ev[k + 1]) for k in range(steps)]
    return ev[0].elapsed_time(ev[steps]) * 1e-3


LAST_STEP_MS: list = []       # per-step durations of the most recent time_steps call


def cost_model_scaled(torch, galv, hbm_gbs, barrier, copies=8192):
    """The cost-model kernels alone on `copies` instances of the heterogeneous stack: large enough to be
    bandwidth-bound (the benchmark's own batch is launch-latency-bound).  Bytes counted: the int32 outputs."""
    import numpy as np
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import _dev_bytes
    w = inputs.config3(B=copies)
    dev = torch.device("cuda", galv.device)
    shape = gb.make_shape(w.B, w.Lmax, w.S, w.M, 0)
    L = torch.from_numpy(np.ascontiguousarray(w.L, np.int32)).to(dev)
    layers, strat, inst = _dev_bytes(w.layers, dev), _dev_bytes(w.strat, dev), _dev_bytes(w.inst, dev)
    tq = torch.empty(w.B, w.Lmax, w.S, dtype=torch.int32, device=dev)
    mq = torch.empty_like(tq)
    xq = torch.empty(w.B, w.S, w.S, dtype=torch.int32, device=dev)
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    stride = 0 if w.layers.shape[0] == 1 else w.Lmax
    fn = lambda: galv.galv_eval_costs(shape, L, layers, stride, strat, inst, None, None, tq, mq, xq, status)
    t = time_steps(torch, fn, 10, 3, barrier) / 10
    nbytes = 4 * (2 * tq.numel() + xq.numel())
    return {"instances": copies, "elements": tq.numel(), "ms": t * 1e3, "bytes_written": nbytes,
            "gb_per_s": nbytes / t / 1e9, "frac_of_hbm": nbytes / t / 1e9 / hbm_gbs}


def launches_per_step(w, cluster: bool = False) -> int:
    if cluster:                                   # the cost model's kernel, ONE cluster kernel for the whole search, backtrack
        return (1 if w.has_model else 0) + 1 + 1
    # the cost model's kernel, validate + schedule + base layer, ONE cooperative launch over all layers,
    # copy-last + finalize, backtrack; where the shape allows the packed 16-bit path, the kernel that packs
    # the trans rows and the launch of the other inner-loop variant (it returns at once) come on top
    packable = w.S <= 64 and w.S % 4 == 0
    return (1 if w.has_model else 0) + 3 + 1 + 2 + 1 + (2 if packable else 0)


def bench_workload(torch, galv, w, steps, warmup, barrier, flags=1):
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    sb = SearchBuffers(galv, w, flags)
    for _ in range(warmup):
        sb.step()
    galv.galv_set_profiling(True)                                # one event pair around the layer launches of every timed search
    t = time_steps(torch, sb.step, steps, 0, barrier)
    step_ms = sorted(LAST_STEP_MS)
    layer_ms, layer_min, layer_max, layer_n = galv.galv_layer_loop_ms_stats()   # mean over the timed searches (the last 64)
    path = galv.galv_dp_search_path(sb.shape, sb.workspace)                     # which kernel ran
    packed, cluster = path == gb.PATH_TILED_PACKED, path == gb.PATH_CLUSTER
    galv.galv_set_profiling(False)
    res = sb.results()
    out = {"seconds": t, "ms_per_step": t / steps * 1e3, "cells_per_s": w.cells * steps / t,
           "relax_per_s": w.relaxations * steps / t, "searches_per_s": w.B * steps / t,
           "layer_kernel_ms_avg": layer_ms / max(1, w.Lmax - 1), "layer_loop_ms": layer_ms, "packed": packed, "cluster": cluster,
           "ms_median": statistics.median(step_ms), "ms_best": step_ms[0], "layer_loop_ms_min": layer_min, "layer_loop_ms_max": layer_max, "layer_loop_launches_timed": layer_n,
           "feasible": int((res["status"] == 0).sum()), "opt_cost_sum": int(res["opt_cost"][res["status"] == 0].sum())}
    return sb, out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=3, help="workload index 0..4 (3: heterogeneous stack, the whole path)")
    ap.add_argument("--impl", default="galv", choices=["galv", "reference"])
    ap.add_argument("--no-others", action="store_true", help="skip the side measurements of the other workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiler captures)")
    ap.add_argument("--no-packed", action="store_true", help="keep the 32-bit inner loop where the packed 16-bit one would run")
    ap.add_argument("--no-cluster", action="store_true", help="keep the tiled kernels where the small-batch cluster kernel would run")
    ap.add_argument("--instance", type=int, default=-1, help="search only this instance of the workload (single re-search latency)")
    ap.add_argument("--cost-model-only", action="store_true", help="only the bandwidth-sized cost-model pass (profiler captures); prints its figures")
    ap.add_argument("--skip-dominated", action="store_true", help="run with GALV_SKIP_DOMINATED (profiler captures; the roofline keys then do not apply)")
    ap.add_argument("--argmin-table", action="store_true", help="run with GALV_STORE_ARGMIN as well (profiler captures; the roofline keys then do not apply)")
    ap.add_argument("--batch", type=int, default=0, help="trim the workload to its first instances (profiler captures)")
    ap.add_argument("--layers", type=int, default=0, help="trim the workload to its first layers (profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "galv" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))            # no launcher around this process: start the ranks here

    import torch
    import torch.distributed as dist
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import HostSearch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the search has no CPU path")
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if torch.cuda.device_count() < world:
        raise SystemExit(f"bench.py: {world} ranks but only {torch.cuda.device_count()} CUDA device(s) are visible")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        if rank == 0:
            print(f"[bench] communicator: backend nccl {'.'.join(map(str, torch.cuda.nccl.version()))}, {world} ranks on one node, "
                  f"used for the barrier and the max over ranks only (no collective on the data path)", file=sys.stderr)

    def barrier():
        if world > 1:
            dist.barrier()

    def max_over_ranks(x: float) -> float:
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    galv = gb.Galv(local)
    for _ in range(8):                                           # bring the clocks up before short workloads are timed
        galv.galv_probe_int_alu(0, 4096)
    if args.cost_model_only:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except OSError:
            pass
        print(json.dumps({"cost_model_scaled": cost_model_scaled(torch, galv, peaks.get("hbm_gbs", 6650.0), lambda: None),
                          "hbm_peak": "of measured" if peaks else "of fallback"}))
        galv.close()
        return
    w = workload_for(args.workload, rank, args.batch, args.layers)
    if args.instance >= 0:
        w = w.take([args.instance])
        w.name += f"[instance {args.instance}]"
    uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", "")

    with ClockSampler(uuid) as clk:
        sb, r = bench_workload(torch, galv, w, args.steps, args.warmup, barrier,
                               flags=1 | (gb.KERNEL_NO_PACKED if args.no_packed else 0) | (gb.SKIP_DOMINATED if args.skip_dominated else 0)
                                     | (gb.KERNEL_NO_CLUSTER if args.no_cluster else 0) | (gb.STORE_ARGMIN if args.argmin_table else 0))
    t = max_over_ranks(r["seconds"])
    clocks = clk.summary()
    value = world * w.cells * args.steps / t
    kernel_s = r["layer_loop_ms"] * 1e-3                     # the one launch that runs every layer
    relax_per_launch = w.relaxations
    achieved = relax_per_launch / kernel_s / 1e9
    del sb
    torch.cuda.empty_cache()

    # end to end through the host-buffer entry point: pinned host inputs -> device -> search -> host results
    e2e = None
    if not args.no_e2e:
        hs = HostSearch(galv, w, gb.STORE_C_FULL)
        for _ in range(args.warmup):
            hs.run()
        torch.cuda.synchronize(); barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            hs.run()
        torch.cuda.synchronize(); barrier()
        te = max_over_ranks(time.perf_counter() - t0)
        e2e = {"value": world * w.cells * args.steps / te, "unit": UNIT, "ms_per_step": te / args.steps * 1e3,
               "h2d_bytes_per_step": hs.h2d, "d2h_bytes_per_step": hs.d2h}
        del hs
        torch.cuda.empty_cache()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": t / args.steps * 1e3, "ms_median": r["ms_median"], "ms_best": r["ms_best"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "Lmax": w.Lmax, "S": w.S, "M": w.M, "per_gpu_batch": w.B,
                   "tables": "full C kept (int32), plan re-derived along the path",
                   "l2": "tables far larger than L2 (no flush needed)", "parallelism": f"instances x{world}"},
        "searches_per_s": world * w.B * args.steps / t, "relaxations_per_s": world * w.relaxations * args.steps / t,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step(w, r["cluster"]) * args.steps,
        "roofline": {"bound": "alu", "achieved": achieved, "peak": ALU_PEAK_GOPS * (2 if r["packed"] else 1), "unit": "G add-min/s",
                     "frac": achieved / (ALU_PEAK_GOPS * (2 if r["packed"] else 1)),
                     "frac_of_32bit_peak": achieved / ALU_PEAK_GOPS,
                     "inner_loop": ("packed 16-bit add-min on rebased costs, two relaxations per instruction" if r["packed"]
                                    else "32-bit fused add-min, one relaxation per instruction"),
                     "traffic": (NCU_TRAFFIC_BYTES_PER_LAYER[w.name] * (w.Lmax - 1)
                                 if w.name in NCU_TRAFFIC_BYTES_PER_LAYER else None),
                     "traffic_unit": "bytes per launch (ncu dram read+write per layer x layers)",
                     "algorithmic_bytes_per_launch": 2 * 4 * w.B * w.S * w.m_pitch * (w.Lmax - 1),
                     "algorithmic_ops_per_launch": relax_per_launch,
                     "kernel": ("cluster_search_kernel (one thread-block cluster per instance, all layers in one launch)" if r["cluster"] else
                                "layer_tiled_kernel (one cooperative launch over all layers"
                                + (", packed 16-bit variant)" if r["packed"] else ")")),
                     "launch_ms": r["layer_loop_ms"], "launch_ms_min": r["layer_loop_ms_min"],
                     "launch_ms_max": r["layer_loop_ms_max"], "launches_timed": r["layer_loop_launches_timed"],
                     "peak_source": "derived: 148 SMs x 64 int32 lanes x 1.965 GHz, one fused add-min per lane per clock"
                                    + (" (two relaxations each in the packed 16-bit form)" if r["packed"] else "")},
    }

    line["inputs_fnv1a64"] = input_checksums(w)
    line["kernel_variant"] = line["roofline"]["kernel"]
    if rank == 0:
        # The ALU peak measured on this GPU, in the run itself, by register-only probes of the very instruction the
        # inner loop issues (relaxations per second: the packed instruction counts as the two it performs).
        rf = line["roofline"]
        rf["peak_derived"] = rf["peak"]
        try:
            fused = galv.galv_probe_int_alu(0, 4096) / 1e9
            packed = galv.galv_probe_int_alu(3, 4096) / 1e9
            rf["peak_measured"] = packed if r["packed"] else fused
            rf["frac_of_measured"] = achieved / rf["peak_measured"]
            rf["probe_fused_addmin_gops"] = fused
            rf["probe_packed_addmin_u16x2_gops"] = packed
            rf["probe_add_then_min_gops"] = galv.galv_probe_int_alu(1, 4096) / 1e9
            rf["probe_add_xor_2ops_gops"] = galv.galv_probe_int_alu(2, 4096) / 1e9
            rf["probe_min3_gops"] = galv.galv_probe_int_alu(4, 4096) / 1e9
            rf["peak_measured_source"] = ("galv_probe_int_alu kind 3 (__viaddmin_u16x2, two relaxations per instruction)" if r["packed"]
                                          else "galv_probe_int_alu kind 0 (__viaddmin_s32)")
        except gb.GalvError as e:      # diagnostic only
            rf["peak_measured"] = None
            rf["probe_error"] = str(e)
        # HBM side of the roofline: every table cell written once and read once by the next layer
        from paper_2504_03662_b200.binding import make_shape
        pitch = make_shape(w.B, w.Lmax, w.S, w.M).m_pitch
        hbm_bytes = 2 * 4 * int(np.sum(w.L)) * w.S * pitch
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except OSError:
            pass
        hbm_gbs = peaks.get("hbm_gbs", 6650.0)
        line["roofline"]["t_alu_ms"] = w.relaxations / (line["roofline"]["peak"] * 1e9) * 1e3
        line["roofline"]["t_hbm_ms"] = hbm_bytes / (hbm_gbs * 1e9) * 1e3
        line["roofline"]["hbm_peak"] = f"{hbm_gbs} GB/s " + ("of measured" if peaks else "of fallback")
        line["roofline"]["step_frac_of_bound"] = max(line["roofline"]["t_alu_ms"], line["roofline"]["t_hbm_ms"]) / (t / args.steps * 1e3)

    if rank == 0 and world == 1 and not args.no_others:
        # The same step with GALV_SKIP_INFEASIBLE: tiles wholly below the feasibility frontier get their +inf
        # results without loads or relaxations.  Same tables; reported beside the headline, which does all the work.
        sbs, rs = bench_workload(torch, galv, w, max(5, args.steps // 2), 3, barrier, flags=1 | gb.SKIP_INFEASIBLE)
        line["with_infeasible_skip"] = {"ms_per_step": rs["ms_per_step"], "cells_per_s": rs["cells_per_s"],
                                        "searches_per_s": rs["searches_per_s"], "opt_cost_sum": rs["opt_cost_sum"],
                                        "note": "part of the cells is produced without relaxations: no ALU-roofline fraction"}
        line["opt_cost_sum"] = r["opt_cost_sum"]
        del sbs
        torch.cuda.empty_cache()
        if r["packed"]:
            # The same step with GALV_SKIP_DOMINATED (and with both flags): row pairs that cannot win in any
            # column of a tile are left out of the inner loop.  Same tables; how much is left out depends on the
            # spread of the costs, so it stands beside the headline, which does all the relaxations.
            for key, fl in (("with_dominated_rows_skipped", gb.SKIP_DOMINATED), ("with_both_skips", gb.SKIP_DOMINATED | gb.SKIP_INFEASIBLE)):
                sbd, rd = bench_workload(torch, galv, w, max(5, args.steps // 2), 3, barrier, flags=1 | fl)
                line[key] = {"ms_per_step": rd["ms_per_step"], "cells_per_s": rd["cells_per_s"],
                             "searches_per_s": rd["searches_per_s"], "opt_cost_sum": rd["opt_cost_sum"],
                             "launch_ms": rd["layer_loop_ms"],
                             "hbm_frac": hbm_bytes / (rd["layer_loop_ms"] * 1e-3) / (hbm_gbs * 1e9),
                             "roofline": {"bound": "hbm", "achieved": hbm_bytes / (rd["layer_loop_ms"] * 1e-3) / 1e9, "peak": hbm_gbs,
                                          "unit": "GB/s", "frac": hbm_bytes / (rd["layer_loop_ms"] * 1e-3) / (hbm_gbs * 1e9),
                                          "traffic": None, "peak_source": "of measured" if peaks else "of fallback",
                                          "algorithmic_bytes_per_launch": hbm_bytes},
                             "note": "part of the relaxations is proved unnecessary and left out: no ALU-roofline fraction"}
                del sbd
                torch.cuda.empty_cache()
        if r["packed"]:
            # the same step with the 32-bit inner loop (one relaxation per instruction), against its own peak
            sb3, r3 = bench_workload(torch, galv, w, max(5, args.steps // 2), 3, barrier, flags=1 | gb.KERNEL_NO_PACKED)
            line["inner_loop_32bit"] = {"ms_per_step": r3["ms_per_step"], "cells_per_s": r3["cells_per_s"],
                                        "launch_ms": r3["layer_loop_ms"], "opt_cost_sum": r3["opt_cost_sum"],
                                        "alu_frac": w.relaxations / (r3["layer_loop_ms"] * 1e-3) / 1e9 / ALU_PEAK_GOPS,
                                        "peak": ALU_PEAK_GOPS}
            del sb3
            torch.cuda.empty_cache()
        # Cost-only search: no table kept, two layers roll in the workspace (optimum per instance, no plan).
        # All the relaxations are done; the tables' HBM footprint is 2 layers instead of Lmax.
        sbc, rc = bench_workload(torch, galv, w, max(5, args.steps // 2), 3, barrier, flags=0)
        line["cost_only"] = {"ms_per_step": rc["ms_per_step"], "cells_per_s": rc["cells_per_s"],
                             "searches_per_s": rc["searches_per_s"], "opt_cost_sum": rc["opt_cost_sum"],
                             "alu_frac": w.relaxations / (rc["layer_loop_ms"] * 1e-3) / 1e9 / (ALU_PEAK_GOPS * (2 if rc["packed"] else 1)),
                             "packed": rc["packed"],
                             "table_bytes": 2 * 4 * w.B * w.S * sbc.shape.m_pitch,
                             "note": "optimum per instance without a plan; same relaxations, two-layer rolling buffer"}
        del sbc
        torch.cuda.empty_cache()
        others = {}
        for k in (0, 1, 2, 4):
            wk = workload_for(k)
            sbk, rk = bench_workload(torch, galv, wk, max(5, args.steps // 2), 3, barrier)
            o = {key: rk[key] for key in ("ms_per_step", "cells_per_s", "relax_per_s", "searches_per_s")}
            o["alu_frac"] = rk["relax_per_s"] / (ALU_PEAK_GOPS * 1e9 * (2 if rk["packed"] else 1))
            o["packed"] = rk["packed"]
            o["kernel"] = "cluster" if rk["cluster"] else "tiled"
            o["layer_loop_ms"] = rk["layer_loop_ms"]
            if k in (1, 2, 4):
                # with both opt-in flags (work proved unnecessary left out; same tables): no ALU-roofline fraction
                sbd, rd = bench_workload(torch, galv, wk, max(5, args.steps // 2), 3, barrier,
                                         flags=1 | gb.SKIP_DOMINATED | gb.SKIP_INFEASIBLE)
                pitch4 = make_shape(wk.B, wk.Lmax, wk.S, wk.M).m_pitch
                o["with_both_skips"] = {"ms_per_step": rd["ms_per_step"], "cells_per_s": rd["cells_per_s"], "launch_ms": rd["layer_loop_ms"],
                                        "hbm_frac": 2 * 4 * int(np.sum(wk.L)) * wk.S * pitch4 / (rd["layer_loop_ms"] * 1e-3) / (hbm_gbs * 1e9),
                                        "opt_cost_sum": rd["opt_cost_sum"], "opt_cost_sum_plain": rk["opt_cost_sum"]}
                del sbd
            if rk["cluster"]:
                # the same step on the tiled kernels (what a batch this small ran on before the cluster kernel)
                sbt, rt = bench_workload(torch, galv, wk, max(5, args.steps // 2), 3, barrier, flags=1 | gb.KERNEL_NO_CLUSTER)
                o["tiled_kernels_only"] = {"ms_per_step": rt["ms_per_step"], "layer_loop_ms": rt["layer_loop_ms"], "packed": rt["packed"],
                                           "opt_cost_sum": rt["opt_cost_sum"], "opt_cost_sum_cluster": rk["opt_cost_sum"]}
                del sbt
            # the same step replayed from a CUDA graph (launch latency matters for the small workloads)
            g = torch.cuda.CUDAGraph()
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                sbk.step()
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=s):
                    sbk.step()
                tg = time_steps(torch, g.replay, max(5, args.steps // 2), 3, barrier)
            o["graph_ms_per_step"] = tg / max(5, args.steps // 2) * 1e3
            others[wk.name] = o
            del sbk, g
            torch.cuda.empty_cache()
        line["others"] = others
        # One model searched again at run time (the paper's monitoring / optimisation loop): a batch of ONE instance.
        single = {}
        for k, inst in ((1, 15), (2, 56)):                       # micro-batch 16 of the GPT-style stack; b = 8, one stage of 96 layers
            wk = workload_for(k).take([inst])
            e = {}
            for key, fl in (("cluster_kernel", 1), ("tiled_kernels_only", 1 | gb.KERNEL_NO_CLUSTER)):
                sb1, r1 = bench_workload(torch, galv, wk, 50, 5, barrier, flags=fl)
                e[key] = {"ms_per_step": r1["ms_per_step"], "layer_loop_ms": r1["layer_loop_ms"], "opt_cost_sum": r1["opt_cost_sum"],
                          "kernel": "cluster" if r1["cluster"] else ("tiled packed" if r1["packed"] else "tiled 32-bit"),
                          "us_per_layer": r1["layer_loop_ms"] * 1e3 / max(1, wk.Lmax - 1)}
                del sb1
            single[f"{wk.name}[instance {inst}]"] = e
        line["single_instance_research"] = single
        # The argmin-table mode (one launch per layer, at least three ALU operations per relaxation), plain and
        # with dominated rows left out: whole steps on config 4 and on the first 40 layers of config 3
        # (its full argmin + cost tables would not leave room for the other buffers of this run).
        amode = {}
        for wk in (workload_for(3, 0, 0, 40), workload_for(4)):
            for key, fl in (("plain", 0), ("dominated_rows_skipped", gb.SKIP_DOMINATED)):
                sba, ra = bench_workload(torch, galv, wk, 5, 3, barrier, flags=gb.STORE_ARGMIN | fl)
                amode.setdefault(wk.name, {})[key] = {"ms_per_step": ra["ms_per_step"], "layer_loop_ms": ra["layer_loop_ms"],
                                                      "cells_per_s": ra["cells_per_s"], "opt_cost_sum": ra["opt_cost_sum"]}
                del sba
                torch.cuda.empty_cache()
        line["argmin_table_mode"] = amode
        line["cost_model_scaled"] = cost_model_scaled(torch, galv, hbm_gbs, barrier)

    if rank == 0 and world == 1 and not args.no_cpu:
        from oracle import oracle
        oracle.build()
        threads = min(os.cpu_count() or 1, w.B, 32)
        n_inst, max_layers = oracle_sample_size(w, threads, 15.0)    # ~15 s of work per thread
        items, cells = oracle_sample(w, max_layers, threads, n_inst)
        tc = oracle_run(w, items, threads)
        t1 = oracle_run(w, items[:1], 1)                          # the same search on one core
        line["cpu_baseline"] = {"value": cells / tc, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": tc,
                                "sample": f"first {len(items)} instances x first {max_layers} layers, one instance at a time per thread",
                                "single_core_value": cells / len(items) / t1}
    elif rank == 0:
        line["cpu_baseline"] = None

    if rank == 0:
        print(json.dumps(line))
    galv.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
