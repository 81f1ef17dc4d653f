#!/usr/bin/env python
"""Benchmark of the placement-semantics sweep.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload C4|C3|...] [--models M] [--window-log2 L]

One step = one pass of the whole hot path over one batch of synthetic input,
on the stress configuration (4096 shapes, N up to 2^14, 6 963 200 000 points):

  derive   per-model records from the shape table
  topk     fused sweep, per-model 64 smallest by (comm, mem, idx) under 192 GB
  pareto   fused sweep, per-model memory-vs-communication frontier under
           {80, 192} GB with a 64 GB per-step host-link budget
  compact  filter + stream compaction of a window (valid points under 80 GB)
  material all five output arrays of the same window

`value` counts every point each phase evaluates, per second, device-timed with
inputs resident in HBM; `e2e` times the same step through the C interface with
the shape table in pinned host memory and every result copied back to the host.
Before anything is timed, sampled outputs are compared bit for bit with the CPU
oracle; a run that is not bit-exact reports no throughput.

`--impl reference` times the CPU oracle itself (a deliberately plain program)
on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_02311_b200 import synth  # noqa: E402

GB = synth.GB
VALID = 1 | 2 | 4
METRIC = "placement evaluations/sec (bit-exact vs oracle)"
UNIT = "evals/s"
BYTES_PER_POINT_MATERIALISE = 36


def ncu_counters():
    """Figures only a profiler can give (executed instructions per point, pipe
    utilisation, DRAM traffic), from the tracked summary of the last capture.
    They describe the kernels of the commit named there, on the stress
    configuration; the bench prints that commit and uses them on that workload
    only."""
    try:
        return json.load(open(os.path.join(ROOT, "profiles", "ncu_counters.json")))
    except Exception:
        return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4")
    ap.add_argument("--models", type=int, default=None, help="shrink the shape table (tests)")
    ap.add_argument("--window-log2", type=int, default=25)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity", action="store_true")
    return ap.parse_args()


def workload(name: str, n_models, rank: int = 0):
    space = synth.config(name, n_models=n_models)
    if rank:
        # weak scaling: every rank sweeps its own table of the same distribution
        seeds = {"C1": 0, "C2": 1, "C3": 2, "C4": 3}
        if name in seeds:
            kw = {}
            if name in ("C3", "C4"):
                kw = dict(max_layers=160, max_hidden_mult=256)
            if name == "C4":
                kw.update(seqs=(2048, 4096, 8192, 16384, 32768), max_micro_batch=64)
            space["models"] = synth.zoo(len(space["models"]), seeds[name] + 1000 * rank, **kw)
    return space


TOPK_FILTER = dict(require_flags=VALID, comm_kind=1)
TOPK_CAPS = [192 * GB]
TOPK_K = 64
PARETO_FILTER = dict(require_flags=VALID, comm_kind=1, host_cap=64 * GB)
PARETO_CAPS = [80 * GB, 192 * GB]
PARETO_MAX = 64
COMPACT_FILTER = dict(require_flags=VALID, cap_bytes=80 * GB)


def window_of(size: int, window_log2: int):
    count = min(size, 1 << window_log2)
    first = (size - count) // 2 // 625 * 625 + 311 if size > count else 0   # not group aligned
    first = min(first, size - count)
    return first, count


# ---------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(prefix="clocks_", suffix=".csv")
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.fh,
                stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, reasons = [], set()
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1]))
                    out["sm_max_mhz"] = float(p[2])
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------- oracle legs
def oracle_step(osp, first, count, model_count, threads):
    """One pass of the hot path by the CPU oracle on `model_count` models and a
    window; returns evaluations done."""
    from oracle import oracle as O
    osp.sweep(TOPK_FILTER, TOPK_CAPS, O.KIND_TOPK, TOPK_K, model_count=model_count, n_threads=threads)
    osp.sweep(PARETO_FILTER, PARETO_CAPS, O.KIND_PARETO, PARETO_MAX, model_count=model_count,
              n_threads=threads)
    osp.compact_range(first, count, COMPACT_FILTER)
    osp.eval_range(first, count)
    ppm = osp.points_per_model
    # the oracle evaluates a model once per capacity: 1 + 2 passes; the window twice
    return model_count * ppm * (len(TOPK_CAPS) + len(PARETO_CAPS)) + 2 * count


def cpu_baseline(space, gpu_topk=None, threads=None):
    """The oracle as it stands, timed on a bounded sample of the workload.  Its
    result is not thrown away: the top-k tables of every model it sweeps are
    compared with the GPU's (`gpu_topk` = (entries, counts)); returns the
    baseline record and the number of models compared (None on a mismatch)."""
    from oracle import oracle as O
    threads = threads or O.hardware_threads()
    osp = O.Space(space)
    n_models = min(len(space["models"]), 96 * threads)      # about 15 s of CPU work
    t0 = time.perf_counter()
    o_e, o_c = osp.sweep(TOPK_FILTER, TOPK_CAPS, O.KIND_TOPK, TOPK_K, model_count=n_models, n_threads=threads)
    dt = time.perf_counter() - t0
    evals = n_models * osp.points_per_model
    compared = 0
    if gpu_topk is not None:
        g_e, g_c = gpu_topk
        same = g_e[:n_models].tobytes() == o_e[:n_models].tobytes() and np.array_equal(g_c[:n_models], o_c[:n_models])
        compared = n_models if same else None
    return {"value": evals / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"top-k sweep of the first {n_models} models ({evals} points) in {dt:.2f} s"}, compared


def run_reference(args):
    from oracle import oracle as O
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    space = workload(args.workload, args.models)
    osp = O.Space(space)
    threads = O.hardware_threads()
    model_count = min(len(space["models"]), threads)
    first, count = window_of(osp.size, 18)
    for _ in range(args.warmup):
        oracle_step(osp, first, count, 1, threads)
    t0 = time.perf_counter()
    evals = 0
    for _ in range(args.steps):
        evals += oracle_step(osp, first, count, model_count, threads)
    dt = time.perf_counter() - t0
    value = evals / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
        "data": "synthetic",
        "config": {"workload": f"{args.workload} (CPU oracle on a bounded sample)",
                   "models": int(model_count), "window_points": int(count)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{model_count} models x (top-k + 2-cap Pareto) + window of "
                                   f"{count} points, per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------- ours
def aggregate_over_ranks(dist, device, total_ms, e2e_ms, world, points_per_step, steps, e2e_steps):
    """Whole-job figures: every rank processed `points_per_step` points per step
    (weak scaling, no data-path collective); the job's time is the slowest rank's.
    Returns (value, e2e_value, total_ms_max, e2e_ms_max)."""
    import torch
    t = torch.tensor([total_ms, e2e_ms], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms_max, e2e_ms_max = float(t[0]), float(t[1])
    value = points_per_step * steps * world / (total_ms_max * 1e-3)
    e2e_value = points_per_step * e2e_steps * world / (e2e_ms_max * 1e-3)
    return value, e2e_value, total_ms_max, e2e_ms_max


def parity_gate(ps, gs, space, first):
    """Sampled outputs against the oracle, bit for bit."""
    from oracle import oracle as O
    osp = O.Space(space)
    nm = len(space["models"])
    sample = sorted(set([0, nm // 3, nm - 1]))
    threads = O.hardware_threads()
    g_e, g_c = gs.sweep(TOPK_FILTER, TOPK_CAPS, ps.REDUCE_TOPK, TOPK_K)
    p_e, p_c = gs.sweep(PARETO_FILTER, PARETO_CAPS, ps.REDUCE_PARETO, PARETO_MAX)
    for m in sample:
        o_e, o_c = osp.sweep(TOPK_FILTER, TOPK_CAPS, O.KIND_TOPK, TOPK_K, model_first=m,
                             model_count=1, n_threads=1)
        if g_e[m].tobytes() != o_e[m].tobytes() or g_c[m].tolist() != o_c[m].tolist():
            return f"top-k mismatch at model {m}"
        o_e, o_c = osp.sweep(PARETO_FILTER, PARETO_CAPS, O.KIND_PARETO, PARETO_MAX, model_first=m,
                             model_count=1, n_threads=1)
        if p_e[m].tobytes() != o_e[m].tobytes() or p_c[m].tolist() != o_c[m].tolist():
            return f"Pareto mismatch at model {m}"
    n = min(1 << 18, gs.size - first)
    got = gs.eval_batch(first, n)
    want = osp.eval_range(first, n)
    for k in want:
        if not np.array_equal(got[k], want[k]):
            return f"materialise mismatch in {k}"
    got = gs.compact(first, n, COMPACT_FILTER)
    want = osp.compact_range(first, n, COMPACT_FILTER)
    for k in want:
        if not np.array_equal(got[k], want[k]):
            return f"compaction mismatch in {k}"
    del threads
    return None


def run_ours(args):
    import torch
    import paper_2601_02311_b200.ps as ps

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()
    ctx = ps.Context(local_rank, stream)

    space = workload(args.workload, args.models, rank)
    gs = ctx.space(space)
    size, ppm, nm = gs.size, gs.points_per_model, gs.n_models
    first, count = window_of(size, args.window_log2)

    parity = "skipped"
    if not args.no_parity:
        err = parity_gate(ps, gs, space, first)
        if err:
            print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "error": "parity: " + err}))
            sys.exit(1)
        parity = ("bit-exact: top-k and Pareto tables of 3 sampled models, a 2^18-point window materialised "
                  "and compacted")

    # device buffers (caller-owned outputs)
    topk_out, topk_cnt = gs.alloc_sweep(len(TOPK_CAPS), TOPK_K)
    par_out, par_cnt = gs.alloc_sweep(len(PARETO_CAPS), PARETO_MAX)
    mat = gs.alloc_outputs(count)
    cmp_out = gs.alloc_outputs(count)
    cmp_idx = torch.empty(count, dtype=torch.int64, device=dev)
    cmp_n = torch.zeros(1, dtype=torch.int64, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    # pinned host mirrors for the end-to-end leg
    models_pinned = torch.from_numpy(np.ascontiguousarray(space["models"]).view(np.uint8).copy()).pin_memory()
    h_topk = torch.empty_like(topk_out, device="cpu").pin_memory()
    h_topk_cnt = torch.empty_like(topk_cnt, device="cpu").pin_memory()
    h_par = torch.empty_like(par_out, device="cpu").pin_memory()
    h_par_cnt = torch.empty_like(par_cnt, device="cpu").pin_memory()
    h_mat = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in mat.items()}
    h_cmp = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in cmp_out.items()}
    h_cmp_idx = torch.empty_like(cmp_idx, device="cpu").pin_memory()

    phases = ("derive", "topk", "pareto", "compact", "materialise")
    phase_points = {"derive": 0, "topk": size, "pareto": size, "compact": count, "materialise": count}
    points_per_step = sum(phase_points.values())
    launches_per_step = 1 + 2 * len(TOPK_CAPS) + 2 + 3 + 1

    def step(events=None):
        def mark(i):
            if events is not None:
                events[i].record(stream)
        mark(0)
        gs.rederive()
        mark(1)
        gs.sweep_into(TOPK_FILTER, TOPK_CAPS, ps.REDUCE_TOPK, TOPK_K, topk_out, topk_cnt)
        mark(2)
        gs.sweep_into(PARETO_FILTER, PARETO_CAPS, ps.REDUCE_PARETO, PARETO_MAX, par_out, par_cnt)
        mark(3)
        gs.eval_batch_into(first, count, cmp_out, COMPACT_FILTER, cmp_idx, cmp_n)
        mark(4)
        gs.eval_batch_into(first, count, mat)
        mark(5)

    copy_stream = torch.cuda.Stream(device=dev)
    mat_done = torch.cuda.Event()

    def e2e_step():
        # same work as step(); the window is materialised first so that its copy to
        # the host (1.2 GB over PCIe, the longest part) runs on a second stream while
        # the sweeps compute
        gs.set_models(models_pinned)                     # host -> device inside the call
        gs.eval_batch_into(first, count, mat)
        mat_done.record(stream)
        copy_stream.wait_event(mat_done)
        with torch.cuda.stream(copy_stream):
            for k in mat:
                h_mat[k].copy_(mat[k], non_blocking=True)
        gs.eval_batch_into(first, count, cmp_out, COMPACT_FILTER, cmp_idx, cmp_n)
        gs.sweep_into(TOPK_FILTER, TOPK_CAPS, ps.REDUCE_TOPK, TOPK_K, topk_out, topk_cnt)
        gs.sweep_into(PARETO_FILTER, PARETO_CAPS, ps.REDUCE_PARETO, PARETO_MAX, par_out, par_cnt)
        h_topk.copy_(topk_out, non_blocking=True)
        h_topk_cnt.copy_(topk_cnt, non_blocking=True)
        h_par.copy_(par_out, non_blocking=True)
        h_par_cnt.copy_(par_cnt, non_blocking=True)
        n = int(cmp_n.item())                            # survivors (synchronises the main stream)
        h_cmp_idx[:n].copy_(cmp_idx[:n], non_blocking=True)
        for k in cmp_out:
            h_cmp[k][:n].copy_(cmp_out[k][:n], non_blocking=True)
        torch.cuda.synchronize()                         # both streams
        d2h = (h_topk.numel() + h_topk_cnt.numel() * 4 + h_par.numel() + h_par_cnt.numel() * 4 + 8 +
               n * (8 + BYTES_PER_POINT_MATERIALISE) + count * BYTES_PER_POINT_MATERIALISE)
        return d2h

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        step()
    ctx.check_status()

    # ---- device-timed steps
    sampler = ClockSampler(local_rank)
    sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(args.steps)]
    barrier()
    wall0 = time.perf_counter()
    for s in range(args.steps):
        flush.fill_(1)                                   # L2 flush, outside the step's events
        step(ev[s])
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()
    ctx.check_status()
    step_ms = [ev[s][0].elapsed_time(ev[s][5]) for s in range(args.steps)]
    total_ms = float(sum(step_ms))
    phase_ms = {p: float(np.mean([ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(args.steps)]))
                for i, p in enumerate(phases)}

    # ---- end to end through the C interface, host buffers
    for _ in range(2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    d2h = 0
    e2e_steps = max(3, min(args.steps, 5))
    for _ in range(e2e_steps):
        d2h = e2e_step()
    barrier()
    e2e_s = time.perf_counter() - t0
    ctx.check_status()

    # ---- integer-pipe peak, measured in this run
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    blocks = torch.cuda.get_device_properties(dev).multi_processor_count * 8
    ctx.int_peak(blocks, 2000, sink)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    ops = ctx.int_peak(blocks, 40000, sink)
    e1.record(stream)
    torch.cuda.synchronize()
    int_peak = ops / (e0.elapsed_time(e1) * 1e-3)

    # ---- Algorithm 1 batched (ps_select), measured beside the step, not inside it
    n_sel = 1 << 24
    sel_q = synth.select_queries(4096, 17)                                  # (4096, 8) u64 on the host
    rec = np.zeros(4096, dtype=ps.SELECT_QUERY_DTYPE)                       # 32-byte records
    rec["param_elems"], rec["layer_elems"], rec["device_bytes"] = sel_q[:, 0], sel_q[:, 1], sel_q[:, 2]
    rec["n_devices"] = sel_q[:, 3]
    rec["w_param"], rec["w_grad"], rec["w_opt"] = sel_q[:, 4], sel_q[:, 5], sel_q[:, 6]
    rec["fast_interconnect"] = sel_q[:, 7]
    d_sel_q = torch.from_numpy(rec.view(np.uint8).reshape(4096, 32).copy()).to(dev).repeat(n_sel // 4096, 1).contiguous()
    d_sel_o = torch.empty(n_sel * 4, dtype=torch.int64, device=dev)
    for _ in range(3):
        ctx.select_into(d_sel_q, n_sel, d_sel_o)
    torch.cuda.synchronize()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(stream)
    for _ in range(10):
        ctx.select_into(d_sel_q, n_sel, d_sel_o)
    s1.record(stream)
    torch.cuda.synchronize()
    select_ms = s0.elapsed_time(s1) / 10

    # ---- the sweeps when they may skip what the filter rejects at sight, beside the step
    # (never instead of it: the step evaluates every point)
    skip_ms = {}
    for name_, filt_, caps_, kind_, k_, out_, cnt_ in (
            ("topk_skip", TOPK_FILTER, TOPK_CAPS, ps.REDUCE_TOPK, TOPK_K, topk_out, topk_cnt),
            ("pareto_skip", PARETO_FILTER, PARETO_CAPS, ps.REDUCE_PARETO, PARETO_MAX, par_out, par_cnt)):
        f_skip = dict(filt_, skip_rejected=1)
        for _ in range(3):
            gs.sweep_into(f_skip, caps_, kind_, k_, out_, cnt_)
        torch.cuda.synchronize()
        times = []
        for _ in range(10):
            flush.fill_(1)
            k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            k0.record(stream)
            gs.sweep_into(f_skip, caps_, kind_, k_, out_, cnt_)
            k1.record(stream)
            torch.cuda.synchronize()
            times.append(k0.elapsed_time(k1))
        skip_ms[name_] = float(np.mean(times))
    ctx.check_status()

    # ---- compaction with every point surviving (the output-bound case), beside the step
    dense_filter = dict(require_flags=0)                                    # no capacity, no flags: all survive
    for _ in range(3):
        gs.eval_batch_into(first, count, cmp_out, dense_filter, cmp_idx, cmp_n)
    torch.cuda.synchronize()
    dense_ms = []
    for _ in range(10):
        flush.fill_(1)
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(stream)
        gs.eval_batch_into(first, count, cmp_out, dense_filter, cmp_idx, cmp_n)
        d1.record(stream)
        torch.cuda.synchronize()
        dense_ms.append(d0.elapsed_time(d1))
    dense_ms = float(np.mean(dense_ms))
    dense_survivors = int(cmp_n.item())
    ctx.check_status()

    # ---- aggregate over ranks: max time, summed points
    value, e2e_value, total_ms_max, e2e_ms_max = aggregate_over_ranks(
        dist, dev, total_ms, e2e_s * 1e3, world, points_per_step, args.steps, e2e_steps)

    if rank == 0:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        hbm_peak = peaks.get("hbm_gbs", 6650.0)
        hbm_src = "measured" if "hbm_gbs" in peaks else "fallback"
        ncu = ncu_counters()
        captured = ncu["workloads"].get(args.workload) if (ncu is not None and args.models is None) else None
        ncu_commit = ncu["captured_at_commit"] if ncu else None

        def alu_roofline(kernel_key, label, ms):
            """The sweep against the integer issue rate measured in this run.  `frac` is the
            issue-slot fraction: executed thread-instructions of all kinds per point (ncu) x
            points/s over the add/xor issue peak.  `alu_pipe_frac` is ncu's ALU-pipe
            utilisation (integer and logic instructions only) -- the figure to hold against
            an integer-ALU target.  Both come from the capture named in `counters_commit`
            and are given on the workload of that capture only."""
            k = captured["kernels"].get(kernel_key) if captured else None
            ops = k["thread_instr_per_point"] if k else None
            achieved = ops * size / (ms * 1e-3) / 1e12 if k else None
            return {"bound": "alu", "kernel": label, "achieved": achieved, "peak": int_peak / 1e12,
                    "unit": "T thread-instructions/s", "frac": achieved / (int_peak / 1e12) if k else None,
                    "frac_is": "issue-slot fraction (all executed instructions)",
                    "alu_pipe_frac": k["alu_pipe_active"] if k else None,
                    "alu_pipe_frac_is": "ncu ALU-pipe utilisation of the captured launch",
                    "issue_active_ncu": k["issue_active"] if k else None,
                    "traffic": k["dram_bytes_per_launch"] if k else None,
                    "ops_per_point": ops, "counters_commit": ncu_commit if k else None,
                    "evals_per_s": size / (ms * 1e-3),
                    "peak_source": "k_int_peak (add+xor chains on both integer pipes) measured in this run"}

        mat_gbs = BYTES_PER_POINT_MATERIALISE * count / (phase_ms["materialise"] * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms_max / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
            "data": "synthetic",
            "config": {"workload": f"{args.workload}: {nm} shapes x {ppm} points = {size} points per "
                                   "sweep; step = derive + top-64 sweep (192 GB) + Pareto sweep "
                                   "({80,192} GB, 64 GB host budget) + compaction and "
                                   f"materialisation of a {count}-point window",
                       "points_per_step": points_per_step, "window_points": count,
                       "l2": "flushed between steps (256 MiB write); window outputs exceed L2",
                       "table_checksum": "%016x" % synth.table_checksum(space["models"]),
                       "parity": parity},
            "phases_ms": phase_ms,
            "phases_evals_per_s": {p: (phase_points[p] / (phase_ms[p] * 1e-3) if phase_points[p] else None)
                                   for p in phases},
            "wall_s_timed_region": wall,
            "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"],
                       "reasons": clocks["reasons"], "samples": clocks["samples"]},
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": int(models_pinned.numel()), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": launches_per_step * args.steps,
            # the dominant kernel of a step is the Pareto sweep (its share is in phases_ms)
            "roofline": alu_roofline("k_sweep_pareto", "k_sweep<Pareto> (+ merge)", phase_ms["pareto"]),
            "roofline_topk": alu_roofline("k_sweep_topk", "k_sweep<top-k> (+ merge)", phase_ms["topk"]),
            "roofline_hbm": {"bound": "hbm", "kernel": "k_eval<materialise>", "achieved": mat_gbs,
                             "peak": hbm_peak, "unit": "GB/s", "frac": mat_gbs / hbm_peak,
                             "traffic": (int(captured["kernels"]["k_eval_materialise"]["dram_bytes_per_point"] * count)
                                         if captured and "k_eval_materialise" in captured["kernels"] else None),
                             "counters_commit": (ncu_commit if captured and "k_eval_materialise" in captured["kernels"]
                                                 else None),
                             "peak_source": hbm_src + " (of measured)" if hbm_src == "measured" else hbm_src + " (of fallback)"},
        }
        dense_gbs = (BYTES_PER_POINT_MATERIALISE + 8) * dense_survivors / (dense_ms * 1e-3) / 1e9
        line["roofline_compact_dense"] = {
            "bound": "hbm", "kernel": "k_compact_count + k_tile_scan + k_eval<write>, every point survives",
            "achieved": dense_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": dense_gbs / hbm_peak,
            "ms": dense_ms, "survivors": dense_survivors, "bytes_per_survivor": BYTES_PER_POINT_MATERIALISE + 8,
            "traffic": None}
        line["sweeps_skipping_rejected_ms"] = dict(skip_ms, note="same results; factorisations whose composition "
                                                   "flags miss a required one are not evaluated; not part of the "
                                                   "step or of `value`")
        line["select"] = {"queries": n_sel, "ms": select_ms, "queries_per_s": n_sel / (select_ms * 1e-3),
                          "GB/s": 64 * n_sel / (select_ms * 1e-3) / 1e9,
                          "frac_of_hbm_peak": 64 * n_sel / (select_ms * 1e-3) / 1e9 / hbm_peak}
        if not args.no_cpu_baseline and world == 1:
            gpu_topk = None
            if not args.no_parity:
                e = topk_out.cpu().numpy().view(ps.ENTRY_DTYPE).reshape(nm, len(TOPK_CAPS), TOPK_K)
                c = topk_cnt.cpu().numpy().view(np.uint32).reshape(nm, len(TOPK_CAPS))
                gpu_topk = (e, c)
            line["cpu_baseline"], compared = cpu_baseline(space, gpu_topk)
            if compared is None:
                print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT,
                                  "error": "parity: top-k tables differ from the CPU-baseline sweep"}))
                sys.exit(1)
            if compared:
                line["config"]["parity"] += f"; top-k tables of {compared} of {nm} models (the CPU-baseline sweep)"
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
