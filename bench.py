#!/usr/bin/env python
"""Benchmark of the row-reduction hot path (RMSNorm, softmax, cross-entropy forward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--sweep [--out FILE]]

One "step" is one pass of the whole hot path over one batch of synthetic bf16 input:
RMSNorm [8192, 8192], last-dim softmax [16384, 8192] and fused cross-entropy
[4096, 128256] - one large shape from each benchmark configuration, every working set
larger than the 126 MB L2.  ``value`` is algorithmic bytes per second (the bytes the
method itself must move: activation read + write, logits read, weights / targets / losses)
with inputs resident in HBM; ``e2e`` is the same metric through the host-buffer entry
points with the host<->device copies inside the timed region.  One JSON line is printed
by rank 0.  With N > 1 (torchrun) every rank processes its own batch (rows are independent:
weak scaling, no data-path collective) and the cross-entropy mean is made global with one
16-byte all-gather per step.

``--impl reference`` times the fp64 CPU checker on the host cores on a bounded sample of
the same workload.  ``--sweep`` additionally times every benchmark shape one by one, beside a
plain copy (or read) of the same size, prints the table to stderr and writes it to the file
``--out`` names (not part of the JSON line contract).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "achieved HBM GB/s (algorithmic bytes / time) over RMSNorm + softmax + cross-entropy forward"
WORKLOAD = {
    "rmsnorm": (8192, 8192),
    "softmax": (16384, 8192),
    "xent": (4096, 128256),
}
WORKLOAD_NAME = "rmsnorm[8192x8192] + softmax[16384x8192] + xent[4096x128256], bf16"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# ncu dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel
# (cross-entropy row kernel at [4096, 128256]): the [2048, 128256] capture summarised in
# profiles/kernels_ncu_set_full.md, 499.62 MB read + 4.05 MB written, scaled by rows (x2).
NCU_TRAFFIC_BYTES_DOMINANT = {"xent": 1007342592}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(op, rows, D, n_valid=None):
    if op == "rmsnorm":
        return 4 * rows * D + 2 * D
    if op == "layernorm":
        return 4 * rows * D + 4 * D
    if op == "rowsum":
        return 2 * rows * D + 4 * rows
    if op == "softmax":
        return 4 * rows * D
    nv = rows if n_valid is None else n_valid
    return 2 * D * nv + 12 * rows + 4       # ignored rows are never read


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Polls NVML for SM clock and throttle reasons while a timed region runs.  Every sample
    carries its host time, so a region can be summarised as a whole or per time window."""

    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap", "hw_power_brake")

    def __init__(self, index, period=0.005):
        self.samples = []          # (host time, SM MHz, set of active reasons)
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self.period = period
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        bits = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, frozenset(k for k, bit in bits.items() if mask & bit)))
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self, t_lo=None, t_hi=None):
        sel = [(m, r) for t, m, r in self.samples
               if (t_lo is None or t >= t_lo) and (t_hi is None or t < t_hi)]
        if not sel and t_lo is not None:   # a window shorter than the polling period: the next sample after it began
            sel = [(m, r) for t, m, r in self.samples if t >= t_lo][:1]
        med = float(np.median([m for m, _ in sel])) if sel else None
        reasons = sorted(set().union(*[r for _, r in sel])) if sel else []
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(sel)}


# --------------------------------------------------------------------------- timed blocks
MIN_TIMED_S = 1.0          # the device-timed region lasts at least this long, whatever --steps says
SUSTAINED_AFTER_S = 0.3    # blocks that start later than this are the sustained regime
IDLE_BEFORE_S = 1.0        # the GPU idles this long before a timed region, so its first block is a burst


def timed_blocks(run_block, est_block_ms, device_index, min_s=MIN_TIMED_S, sync=None):
    """Runs `run_block` (K steps, enqueued without a synchronise) back to back until at least
    `min_s` seconds of device time have been timed, a CUDA event between blocks.  Returns the
    per-block milliseconds, each block's start offset in seconds, and the clock samples."""
    nblocks = max(3, int(np.ceil(min_s * 1e3 / max(est_block_ms, 1e-3))))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(nblocks + 1)]
    time.sleep(IDLE_BEFORE_S)
    if sync is not None:
        sync()
    with ClockSampler(device_index) as clk:
        t0 = time.perf_counter()
        ev[0].record()
        for b in range(nblocks):
            run_block()
            ev[b + 1].record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
    ms = np.array([ev[b].elapsed_time(ev[b + 1]) for b in range(nblocks)])
    starts = np.concatenate([[0.0], np.cumsum(ms)[:-1]]) * 1e-3
    return ms, starts, clk, t0, t1


def regimes(ms, starts, clk, t0, t1):
    """Block time (ms) and clocks of the burst regime (the first block), the sustained regime
    (median of the blocks that start after SUSTAINED_AFTER_S of load) and of all blocks (median)."""
    late = starts >= SUSTAINED_AFTER_S
    if not late.any():
        late[-1] = True
    t_first_end = t0 + ms[0] * 1e-3
    return {
        "burst": {"block_ms": float(ms[0]), "blocks": 1, "clocks": clk.summary(t0, max(t_first_end, t0 + 0.05))},
        "sustained": {"block_ms": float(np.median(ms[late])), "blocks": int(late.sum()),
                      "clocks": clk.summary(t0 + SUSTAINED_AFTER_S, t1)},
        "all": {"block_ms": float(np.median(ms)), "blocks": int(len(ms)), "clocks": clk.summary(t0, t1)},
    }


# --------------------------------------------------------------------------- reference arm
def run_reference(args, rank, world):
    """The fp64 CPU checker, as it stands, on the host cores, on a bounded sample."""
    if rank != 0:
        return
    import oracle
    from paper_2603_21331_b200 import synth
    cores = oracle.set_threads(0)
    sample = {"rmsnorm": (256, 8192), "softmax": (128, 8192), "xent": (16, 128256)}
    x, w = synth.rmsnorm_inputs(*sample["rmsnorm"], seed=2000)
    xs = synth.softmax_inputs(*sample["softmax"], seed=3000)
    lg, tg = synth.xent_inputs(*sample["xent"], seed=4000)
    xb, wb, xsb, lgb, tgn = (synth.to_bits(x), synth.to_bits(w), synth.to_bits(xs), synth.to_bits(lg),
                             tg.numpy())
    nbytes = (algorithmic_bytes("rmsnorm", *sample["rmsnorm"]) + algorithmic_bytes("softmax", *sample["softmax"])
              + algorithmic_bytes("xent", *sample["xent"], n_valid=int((tgn != -100).sum())))

    def step():
        oracle.rmsnorm(xb, wb, 1e-6)
        oracle.softmax(xsb)
        oracle.xent(lgb, tgn)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    gbs = nbytes * args.steps / dt / 1e9
    desc = ("per step: rmsnorm 256 rows + softmax 128 rows of D=8192, xent 16 rows of V=128256 "
            "(same row lengths as the GPU workload, fewer rows)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD_NAME, "sample": desc},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def cpu_baseline_leg():
    """Bounded sample (about 10-30 s of CPU work) of the workload through the CPU checker."""
    import oracle
    from paper_2603_21331_b200 import synth
    cores = oracle.set_threads(0)
    sample = {"rmsnorm": (2048, 8192), "softmax": (1024, 8192), "xent": (128, 128256)}
    x, w = synth.rmsnorm_inputs(*sample["rmsnorm"], seed=2000)
    xs = synth.softmax_inputs(*sample["softmax"], seed=3000)
    lg, tg = synth.xent_inputs(*sample["xent"], seed=4000)
    xb, wb, xsb, lgb, tgn = (synth.to_bits(x), synth.to_bits(w), synth.to_bits(xs), synth.to_bits(lg),
                             tg.numpy())
    nbytes = (algorithmic_bytes("rmsnorm", *sample["rmsnorm"]) + algorithmic_bytes("softmax", *sample["softmax"])
              + algorithmic_bytes("xent", *sample["xent"], n_valid=int((tgn != -100).sum())))
    reps, dt = 0, 0.0
    t0 = time.perf_counter()
    while True:
        oracle.rmsnorm(xb, wb, 1e-6)
        oracle.softmax(xsb)
        oracle.xent(lgb, tgn)
        reps += 1
        dt = time.perf_counter() - t0
        if dt > 10.0:
            break
    return {"value": nbytes * reps / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": (f"{reps} passes over rmsnorm 2048x8192 + softmax 1024x8192 + xent 128x128256 "
                       f"({dt:.1f} s, OpenMP over rows)")}


def speed_of_light(ak, dev, iters=30):
    """In-process HBM ceilings: the library's plain streaming copy (512 MiB -> 512 MiB, bytes
    = read + write) and plain streaming read (1 GiB), CUDA events, trimmed mean."""
    n = 512 << 20
    src = torch.empty((2 * n,), dtype=torch.uint8, device=dev)
    src.fill_(3)
    dst = torch.empty((n,), dtype=torch.uint8, device=dev)
    sink = torch.zeros((1,), dtype=torch.int32, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    l = ak.lib()

    def timed(fn, nbytes):
        # burst: a handful of isolated launches; sustained: back-to-back launches for ~0.25 s
        # after ~0.25 s of the same load (the regime the K-step timed region runs in)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(iters):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ts = np.sort(np.array(ts))
        k = iters // 10
        burst = nbytes / (float(ts[k:iters - k].mean()) * 1e-3) / 1e9
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(20):
                    fn_on(side.cuda_stream)
        torch.cuda.current_stream().wait_stream(side)
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < 0.25:
            g.replay()
            torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 0
        a.record()
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < 0.25:
            g.replay()
            reps += 1
            if reps % 4 == 0:
                torch.cuda.synchronize()
        b.record()
        torch.cuda.synchronize()
        sustained = nbytes * 20 * reps / (a.elapsed_time(b) * 1e-3) / 1e9
        return burst, sustained

    fn_on = lambda s: l.ak_sol_copy(src.data_ptr(), dst.data_ptr(), n, s)
    copy_b, copy_s = timed(lambda: fn_on(st), 2 * n)
    fn_on = lambda s: l.ak_sol_read(src.data_ptr(), 2 * n, sink.data_ptr(), s)
    read_b, read_s = timed(lambda: fn_on(st), 2 * n)
    return {"copy_GB/s": copy_s, "read_GB/s": read_s, "copy_burst_GB/s": copy_b, "read_burst_GB/s": read_b,
            "how": "ak_sol_copy 512 MiB->512 MiB (read+write bytes), ak_sol_read 1 GiB; sustained = CUDA-graph "
                   "replays for 0.25 s after 0.25 s of the same load; burst = isolated launches, trimmed mean"}


# --------------------------------------------------------------------------- our arm
def run_ours(args, rank, world, local_rank):
    import paper_2603_21331_b200 as ak
    from paper_2603_21331_b200 import synth

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the ops have no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    # AK_BENCH_DIST=1 takes the multi-GPU code path (eager steps + the NCCL mean exchange, a process
    # group, barriers, max over ranks) with ONE rank, so that path can be exercised on one GPU
    multi = world > 1 or bool(os.environ.get("AK_BENCH_DIST"))
    dist = None
    if multi:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device(dev))

    seed0 = 100 * rank
    (rr, rd), (sr, sd), (xr, xv) = WORKLOAD["rmsnorm"], WORKLOAD["softmax"], WORKLOAD["xent"]
    x, w = synth.rmsnorm_inputs(rr, rd, synth.case_seed(2, 3) + seed0, device=dev)
    xs = synth.softmax_inputs(sr, sd, synth.case_seed(3, 4) + seed0, device=dev)
    lg, tg = synth.xent_inputs(xr, xv, synth.case_seed(4, 2) + seed0, device=dev)
    y = torch.empty_like(x)
    ys = torch.empty_like(xs)
    loss = torch.empty((xr,), dtype=torch.float32, device=dev)
    mean = torch.empty((1,), dtype=torch.float32, device=dev)
    n_valid = int((tg != -100).sum())
    nbytes = {"rmsnorm": algorithmic_bytes("rmsnorm", rr, rd), "softmax": algorithmic_bytes("softmax", sr, sd),
              "xent": algorithmic_bytes("xent", xr, xv, n_valid)}
    step_bytes = sum(nbytes.values())

    def step():
        ak.ak_rmsnorm_fwd(x, w, y, eps=1e-6)
        ak.ak_softmax_fwd(xs, ys)
        ak.ak_xent_fwd(lg, tg, -100, loss, mean)

    def global_mean():
        # the one real exchange of the path: (sum, count) per rank, summed in rank order
        from paper_2603_21331_b200 import parallel
        return parallel.global_xent_mean(loss, tg, -100)

    for _ in range(max(args.warmup, 3)):
        step()
        if multi:
            global_mean()
    torch.cuda.synchronize()
    if multi:
        dist.barrier()
        torch.cuda.synchronize()

    K = args.steps
    # ---- timed region.  One GPU: the step is captured once into a CUDA graph and a block is K
    # replays of it (no host launch gaps between the kernels).  Several GPUs: a block is K eager
    # steps, each followed by the 16-byte mean exchange over NCCL.  Blocks of K steps repeat, a CUDA
    # event between them, until at least MIN_TIMED_S of device time: `value` and `ms_per_step` come
    # from the median block; the first block (after a second of idling) is the burst regime, the
    # blocks that start after SUSTAINED_AFTER_S of load are the sustained one (power cap reached).
    use_graph = not multi and not os.environ.get("AK_BENCH_EAGER")
    launches0 = ak.ak_launch_count()
    step()
    if multi:
        global_mean()
    torch.cuda.synchronize()
    kernels_per_step = ak.ak_launch_count() - launches0

    def graph_of(fn):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        return g

    def block_runner(fn_or_graph):
        def run():
            for _ in range(K):
                fn_or_graph()
        return run

    def probe_ms(run_block):
        a_ev, b_ev = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_ev.record()
        run_block()
        b_ev.record()
        torch.cuda.synchronize()
        return a_ev.elapsed_time(b_ev)

    def sync_ranks():
        if multi:
            dist.barrier()
        torch.cuda.synchronize()

    if use_graph:
        graph = graph_of(step)
        run_step_block = block_runner(graph.replay)
    else:
        graph = None

        def eager_step():
            step()
            if multi:
                global_mean()
        run_step_block = block_runner(eager_step)
    est = probe_ms(run_step_block)
    ms, starts, clk, t0, t1 = timed_blocks(run_step_block, est, local_rank, sync=sync_ranks)
    if multi:
        t = torch.tensor(ms, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = t.cpu().numpy()
        starts = np.concatenate([[0.0], np.cumsum(ms)[:-1]]) * 1e-3
        dist.barrier()
    step_reg = regimes(ms, starts, clk, t0, t1)
    launches = kernels_per_step * K * len(ms)
    total_ms = float(ms.sum())

    # ---- instrumented pass: per-op durations behind `per_op` and `roofline`.  Events cannot sit
    # inside a replayed graph, so each op gets its own single-op CUDA graph; a block is K replays of
    # it back to back on the same stream and buffers, duration = block / K (kernel time plus the
    # graph's kernel-to-kernel gap; for cross-entropy the streaming kernel and its 1-CTA finish
    # kernel).  Blocks and regimes as for the step.  The eager per-call interval (host launch gaps
    # included) is reported beside it.
    op_fns = {"rmsnorm": lambda: ak.ak_rmsnorm_fwd(x, w, y, eps=1e-6),
              "softmax": lambda: ak.ak_softmax_fwd(xs, ys),
              "xent": lambda: ak.ak_xent_fwd(lg, tg, -100, loss, mean)}
    op_reg, op_ms_eager = {}, {}
    for op, fn in op_fns.items():
        run_op_block = block_runner(graph_of(fn).replay)
        est = probe_ms(run_op_block)
        o_ms, o_starts, o_clk, o_t0, o_t1 = timed_blocks(run_op_block, est, local_rank,
                                                         min_s=SUSTAINED_AFTER_S + 0.4)
        op_reg[op] = regimes(o_ms, o_starts, o_clk, o_t0, o_t1)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(min(K, 200))]
    for e in ev:
        e[0].record()
        op_fns["rmsnorm"]()
        e[1].record()
        op_fns["softmax"]()
        e[2].record()
        op_fns["xent"]()
        e[3].record()
    torch.cuda.synchronize()
    for j, op in enumerate(("rmsnorm", "softmax", "xent")):
        op_ms_eager[op] = float(np.mean([e[j].elapsed_time(e[j + 1]) for e in ev]))

    peak, peak_kind = measured_peak()
    rows_of = {"rmsnorm": rr, "softmax": sr, "xent": xr}

    def op_entry(op, reg):
        us = reg["block_ms"] / K * 1e3
        gbs = nbytes[op] / (us * 1e-6) / 1e9
        mhz = reg["clocks"]["sm_mhz"]
        return {"us": us, "GB/s": gbs, "rows_per_s": rows_of[op] / (us * 1e-6), "frac_of_measured_peak": gbs / peak,
                "frac_of_8TBs": gbs / NOMINAL_HBM_GBS, "sm_mhz": mhz, "us_x_mhz": (us * mhz if mhz else None),
                "blocks": reg["blocks"]}

    per_op = {op: op_entry(op, op_reg[op]["all"]) for op in op_reg}
    for op in per_op:
        per_op[op]["us_eager_call_interval"] = op_ms_eager[op] * 1e3
    dominant = max(per_op, key=lambda o: per_op[o]["us"])

    def step_entry(reg):
        ms_step = reg["block_ms"] / K
        return {"value": step_bytes * world / (ms_step * 1e-3) / 1e9, "ms_per_step": ms_step,
                "blocks": reg["blocks"], "clocks": reg["clocks"]}

    value = step_entry(step_reg["all"])["value"]
    sol = speed_of_light(ak, dev)
    for op in per_op:
        ceiling = sol["read_GB/s"] if op == "xent" else sol["copy_GB/s"]
        per_op[op]["frac_of_in_process_ceiling"] = per_op[op]["GB/s"] / ceiling
    regime_out = {}
    for name in ("burst", "sustained"):
        e = step_entry(step_reg[name])
        e["per_op"] = {op: op_entry(op, op_reg[op][name]) for op in op_reg}
        e["roofline_frac"] = e["per_op"][dominant]["frac_of_measured_peak"]
        regime_out[name] = e

    out = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": step_reg["all"]["block_ms"] / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME, "l2": "every op's working set (268 MB / 537 MB / 1.05 GB) "
                   "exceeds the 126 MB L2; no flush needed", "parallelism": f"rows sharded x{world}",
                   "io_dtype": "bf16",
                   "timed_region": (("blocks of K replays of a CUDA graph holding one step" if graph is not None
                                     else "blocks of K eager steps + NCCL mean exchange")
                                    + f", repeated for >= {MIN_TIMED_S} s of device time after {IDLE_BEFORE_S} s of "
                                      "idling; value / ms_per_step = median block; burst = first block; sustained "
                                      f"= median of the blocks starting after {SUSTAINED_AFTER_S} s"),
                   "blocks": int(len(ms)), "timed_seconds": total_ms * 1e-3},
        "rows_per_s": sum(rows_of.values()) * world / (step_reg["all"]["block_ms"] / K * 1e-3),
        "burst": regime_out["burst"], "sustained": regime_out["sustained"],
        "per_op": per_op,
        "roofline": {"bound": "hbm", "kernel": f"{dominant} {WORKLOAD[dominant][0]}x{WORKLOAD[dominant][1]}",
                     "achieved": per_op[dominant]["GB/s"], "peak": peak, "peak_kind": f"of {peak_kind}",
                     "unit": "GB/s", "frac": per_op[dominant]["GB/s"] / peak,
                     "frac_burst": regime_out["burst"]["roofline_frac"],
                     "frac_sustained": regime_out["sustained"]["roofline_frac"],
                     "frac_of_nominal_8TBs": per_op[dominant]["GB/s"] / NOMINAL_HBM_GBS,
                     "traffic": NCU_TRAFFIC_BYTES_DOMINANT.get(dominant), "algorithmic_bytes": nbytes[dominant],
                     "note": "duration = median block of K back-to-back replays of a single-op CUDA graph / K, "
                             "same stream and buffers (for cross-entropy: streaming kernel + 1-CTA finish kernel); "
                             "frac_burst / frac_sustained: first block after idling / blocks after "
                             f"{SUSTAINED_AFTER_S} s of load"},
        "gpu_launches": launches,
        "clocks": step_reg["all"]["clocks"],
        "speed_of_light": sol,
    }

    # ---- end to end: host buffers in pinned memory, copies inside the timed region
    if rank == 0 or multi:
        xh, wh, yh = x.cpu().pin_memory(), w.cpu(), torch.empty(x.shape, dtype=x.dtype).pin_memory()
        xsh, ysh = xs.cpu().pin_memory(), torch.empty(xs.shape, dtype=xs.dtype).pin_memory()
        lgh, tgh = lg.cpu().pin_memory(), tg.cpu()
        lossh = torch.empty((xr,), dtype=torch.float32).pin_memory()
        meanh = torch.empty((1,), dtype=torch.float32).pin_memory()

        def e2e_step():
            ak.ak_rmsnorm_fwd_host(xh, wh, yh, 1e-6)
            ak.ak_softmax_fwd_host(xsh, ysh)
            ak.ak_xent_fwd_host(lgh, tgh, lossh, meanh)

        e2e_steps = max(2, min(K, 5))
        e2e_step()
        torch.cuda.synchronize()
        if multi:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        if multi:
            t = torch.tensor([dt], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            dt = float(t.item())
        h2d = xh.numel() * 2 + wh.numel() * 2 + xsh.numel() * 2 + lgh.numel() * 2 + tgh.numel() * 8
        d2h = yh.numel() * 2 + ysh.numel() * 2 + lossh.numel() * 4 + 4
        out["e2e"] = {"value": step_bytes * e2e_steps * world / dt / 1e9, "unit": "GB/s",
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                      "ms_per_step": dt / e2e_steps * 1e3,
                      "note": "pinned host buffers -> ak_*_fwd_host (chunked copy/compute/copy pipeline); PCIe-bound"}
        ak.lib().ak_host_arena_release()

    if rank == 0 and world == 1:
        out["widened_rows"] = [
            {"op": r["op"], "rows": r["rows"], "D": r["D"], "us": round(r["us_trimmed_mean"], 2),
             "GB/s": round(r["GB/s"], 1), "frac_of_measured_peak": round(r["GB/s"] / peak, 4)}
            for r in run_sweep(ak, synth, dev, peak, shapes=WIDENED, iters=60, write=False, accuracy=False)]
        out["cpu_baseline"] = cpu_baseline_leg()
    elif rank == 0:
        out["cpu_baseline"] = None

    if args.sweep and rank == 0:
        run_sweep(ak, synth, dev, peak, out_path=args.out)

    if multi:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


# --------------------------------------------------------------------------- per-shape sweep
SWEEP = list(
    [("rmsnorm", 8192, d) for d in (1024, 2048, 4096, 8192, 16384)]
    + [("rmsnorm", r, 4096) for r in (1, 17, 65536, 262144)] + [("rmsnorm", 8192, 4099), ("rmsnorm", 8192, 8190), ("rmsnorm", 4096, 65536), ("rmsnorm", 16, 128256)]
    + [("softmax", 16384, d) for d in (512, 1024, 2048, 4096, 8192, 32768)]
    + [("softmax", 262144, 4096), ("softmax", 16384, 4099), ("softmax", 4096, 65536), ("softmax", 4096, 128256),
       ("softmax", 16, 128256), ("softmax", 1, 128256), ("softmax", 4096, 128257)]
    + [("xent", 4096, v) for v in (32000, 50304, 128256, 128257)] + [("xent", 16384, 128256), ("xent", 16, 128256)]
    + [("layernorm", 8192, 4096), ("layernorm", 4096, 5120), ("layernorm", 8192, 8192), ("layernorm", 65536, 4096),
       ("layernorm", 4096, 32768), ("layernorm", 8192, 4099), ("layernorm", 8192, 8190),
       ("layernorm", 4096, 65536), ("layernorm", 16, 128256)]
    + [("rowsum", 8192, 4096), ("rowsum", 16384, 4096), ("rowsum", 8192, 8192), ("rowsum", 65536, 1024), ("rowsum", 65536, 8192),
       ("rowsum", 4096, 128256), ("rowsum", 8192, 4099), ("rowsum", 16, 128256), ("rowsum", 1, 1 << 24)]
    # element-type variants ("op.f16" / "op.f32"): the paper's Table 4 shapes were measured in FP16
    + [("rmsnorm.f16", 8192, 4096), ("rmsnorm.f16", 8192, 8192), ("rmsnorm.f32", 8192, 8192),
       ("softmax.f16", 16384, 4096), ("softmax.f16", 16384, 8192), ("softmax.f32", 16384, 8192),
       ("xent.f16", 4096, 50304), ("xent.f16", 4096, 128256), ("xent.f32", 4096, 50304)]
)
SWEEP_DTYPES = {"f16": torch.float16, "f32": torch.float32}
# vocabulary-parallel cross-entropy as one of 8 ranks sees it: its [rows, V/8] shard -> partial
# kernel, then the merge over 8 ranks' partial buffers (the 7 others' stand-ins are copies)
SWEEP += [("xent_vp8", 4096, 128256 // 8), ("xent_vp8", 16384, 128256 // 8)]
# rotary embedding, the paper's Table 4 shapes 2 x 32 x {2k, 4k} x 128 (rows = 64 sequences x S)
SWEEP += [("rope.f16", 64 * 2048, 128), ("rope.f16", 64 * 4096, 128), ("rope.bf16", 64 * 4096, 128),
          ("rope.f32", 64 * 4096, 128), ("rope.bf16", 64 * 16384, 128)]
SWEEP_DTYPES["bf16"] = torch.bfloat16


def time_op(fn_for_set, nsets, iters=200, warmup=20):
    """Paper's protocol: CUDA events, 200 samples, trimmed mean (drop top/bottom 10%).
    Consecutive launches rotate over `nsets` disjoint buffer sets (>= 1 GiB in total when
    one set is smaller than that) so no launch finds its input in L2.  Each sample is one
    replay of a CUDA graph holding a batch of back-to-back launches (at least one per buffer
    set, at least ~300 us of work), so short kernels are not timed at the host's launch rate;
    the reported time is the sample divided by the launches in it."""
    for i in range(warmup):
        fn_for_set(i % nsets)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(nsets):
        fn_for_set(i)
    b.record()
    torch.cuda.synchronize()
    est_us = max(a.elapsed_time(b) * 1e3 / nsets, 1.0)
    per_graph = nsets * max(1, int(np.ceil(300.0 / est_us / nsets)))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(per_graph):
                fn_for_set(i % nsets)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for ea, eb in evs:
        ea.record()
        graph.replay()
        eb.record()
    torch.cuda.synchronize()
    t = np.sort(np.array([ea.elapsed_time(eb) for ea, eb in evs])) / per_graph
    k = iters // 10
    return float(t[k:iters - k].mean()) * 1e3, float(t[0]) * 1e3, float(np.median(t)) * 1e3


def sweep_accuracy(ak, synth, op, rows, D, bufs):
    """Errors of the outputs of buffer set 0 against the CPU checker on a sample of rows, a
    bitwise repeat check, and the checker's own speed on that sample (1 thread and all
    threads), scaled to the full number of rows."""
    import oracle
    n = int(max(1, min(rows, 64, (1 << 22) // D)))
    idx = np.unique(np.concatenate([[0, rows - 1], np.random.default_rng(rows + D).integers(0, rows, n)]))
    it = torch.from_numpy(idx).to(bufs[0].device)
    widen = lambda t: (t.cpu().view(torch.int16).numpy().view(np.uint16).astype(np.uint32) << 16
                       ).view(np.float32).astype(np.float64)
    cores = oracle.set_threads(0)

    def timed_oracle(fn):
        t0 = time.perf_counter()
        ref = fn()
        t_all = time.perf_counter() - t0
        oracle.set_threads(1)
        t0 = time.perf_counter()
        fn()
        t_one = time.perf_counter() - t0
        oracle.set_threads(cores)
        return ref, t_one * rows / len(idx), t_all * rows / len(idx)

    if op.startswith("rope."):
        dts = op.split(".")[1]
        x, y = bufs
        first = y.clone()
        ak.ak_rope_fwd(x, y)
        same = torch.equal(first.view(torch.uint8), y.view(torch.uint8))
        S = x.shape[1]
        pos = np.sort(np.unique(np.concatenate([[0, S - 1], np.random.default_rng(S).integers(0, S, 14)])))
        refs, t1, tn, gots = [], 0.0, 0.0, []
        for p in pos:   # one position of every sequence at a time: the checker gets [64, 1, Dh] at offset p
            xs = x[:, int(p):int(p) + 1].contiguous()
            ref, a, b = timed_oracle(lambda: oracle.rope(synth.to_elems(xs), dts, pos_offset=int(p)))
            refs.append(ref); t1 += a; tn += b
            gots.append(y[:, int(p):int(p) + 1].cpu().double().numpy())
        ref, got = np.concatenate(refs, axis=1), np.concatenate(gots, axis=1)
        err = np.abs(got - ref)
        tol = {"bf16": 1.6e-2, "f16": 1e-3, "f32": 1e-5}[dts]
        scale = rows / (64.0 * len(pos)) * len(idx) / rows   # timed_oracle scaled by rows / len(idx)
        return {"max_abs_err": float(err.max()),
                "max_err_over_tolerance": float((err / (tol * np.maximum(1.0, np.abs(ref)))).max()),
                "bitwise_repeat": bool(same), "sampled_rows": int(64 * len(pos)),
                "oracle_s_1_thread_scaled": t1 * scale, "oracle_s_all_threads_scaled": tn * scale,
                "oracle_threads": cores}
    if op == "xent_vp8":
        lg, tg, parts = bufs
        V = 8 * D
        tgt = torch.where(tg == -100, tg, tg % D)   # keep the targets inside this shard
        part = ak.ak_xent_vp_partial(lg, tgt, 0, V, 1)
        # the other seven shards: all-(-inf) columns contribute (max, sum) = (-inf, 0)
        stack = torch.zeros((8,) + tuple(part.shape), dtype=torch.float32, device=part.device)
        stack[:, :, 0, 0] = float("-inf")
        stack[0] = part
        loss, _ = ak.ak_xent_vp_merge(stack, tgt, V)
        again, _ = ak.ak_xent_vp_merge(stack, tgt, V)
        same = torch.equal(loss.view(torch.int32), again.view(torch.int32))
        ref, t1, tn = timed_oracle(lambda: oracle.xent(synth.to_bits(lg[it]), tgt[it].cpu().numpy())[0])
        got = loss[it].cpu().double().numpy()
        torch.cuda.synchronize()
        err = np.abs(got - ref)
        return {"max_abs_err": float(err.max()),
                "max_err_over_tolerance": float((err / (1e-5 * np.maximum(1.0, np.abs(ref)))).max()),
                "bitwise_repeat": bool(same), "sampled_rows": int(len(idx)),
                "oracle_s_1_thread_scaled": t1, "oracle_s_all_threads_scaled": tn, "oracle_threads": cores}
    if "." in op:
        base, dts = op.split(".")
        tol = {"f16": 1e-3, "f32": 1e-5}[dts] if base != "xent" else 1e-5
        if base == "rmsnorm":
            x, w, y = bufs
            first = y.clone()
            ak.ak_rmsnorm_fwd_dt(x, w, y, eps=1e-6)
            same = torch.equal(first.view(torch.uint8), y.view(torch.uint8))
            ref, t1, tn = timed_oracle(lambda: oracle.rmsnorm_dt(synth.to_elems(x[it]), synth.to_elems(w), 1e-6, dts))
            got = y[it].cpu().double().numpy()
        elif base == "softmax":
            x, y = bufs
            first = y.clone()
            ak.ak_softmax_fwd_dt(x, y)
            same = torch.equal(first.view(torch.uint8), y.view(torch.uint8))
            ref, t1, tn = timed_oracle(lambda: oracle.softmax_dt(synth.to_elems(x[it]), dts))
            got = y[it].cpu().double().numpy()
        else:
            lg, tg = bufs
            first, _ = ak.ak_xent_fwd_dt(lg, tg)
            loss, _ = ak.ak_xent_fwd_dt(lg, tg)
            same = torch.equal(first.view(torch.int32), loss.view(torch.int32))
            ref, t1, tn = timed_oracle(lambda: oracle.xent_dt(synth.to_elems(lg[it]), tg[it].cpu().numpy(), dts)[0])
            got = loss[it].cpu().double().numpy()
        torch.cuda.synchronize()
        err = np.abs(got - ref)
        return {"max_abs_err": float(err.max()),
                "max_err_over_tolerance": float((err / (tol * np.maximum(1.0, np.abs(ref)))).max()),
                "bitwise_repeat": bool(same), "sampled_rows": int(len(idx)),
                "oracle_s_1_thread_scaled": t1, "oracle_s_all_threads_scaled": tn, "oracle_threads": cores}
    if op == "rmsnorm":
        x, w, y = bufs
        first = y.clone()
        ak.ak_rmsnorm_fwd(x, w, y, eps=1e-6)
        same = torch.equal(first.view(torch.int16), y.view(torch.int16))
        ref, t1, tn = timed_oracle(lambda: oracle.rmsnorm(synth.to_bits(x[it]), synth.to_bits(w), 1e-6))
        got = widen(y[it])
    elif op == "layernorm":
        x, g, b, y = bufs
        first = y.clone()
        ak.ak_layernorm_fwd(x, g, b, y, eps=1e-5)
        same = torch.equal(first.view(torch.int16), y.view(torch.int16))
        ref, t1, tn = timed_oracle(lambda: oracle.layernorm(synth.to_bits(x[it]), synth.to_bits(g),
                                                            synth.to_bits(b), 1e-5))
        got = widen(y[it])
    elif op == "rowsum":
        x, out = bufs
        first = out.clone()
        ak.ak_rowsum_fwd(x, out)
        same = torch.equal(first.view(torch.int32), out.view(torch.int32))
        ref, t1, tn = timed_oracle(lambda: oracle.rowsum(synth.to_bits(x[it])))
        got = out[it].cpu().double().numpy()
    elif op == "softmax":
        x, y = bufs
        first = y.clone()
        ak.ak_softmax_fwd(x, y)
        same = torch.equal(first.view(torch.int16), y.view(torch.int16))
        ref, t1, tn = timed_oracle(lambda: oracle.softmax(synth.to_bits(x[it])))
        got = widen(y[it])
    else:
        lg, tg, loss, mean, ws = bufs
        first = loss.clone()
        ak.ak_xent_fwd_ws(lg, tg, ws, -100, loss, mean)
        same = torch.equal(first.view(torch.int32), loss.view(torch.int32))
        ref, t1, tn = timed_oracle(lambda: oracle.xent(synth.to_bits(lg[it]), tg[it].cpu().numpy())[0])
        got = loss[it].cpu().double().numpy()
    torch.cuda.synchronize()
    err = np.abs(got - ref)
    rel = err / np.maximum(np.abs(ref), 1e-30)
    if op == "rowsum":   # no bf16 output: report the error relative to sum |x| (fp32 accumulation)
        mag = np.abs(widen(x[it])).sum(axis=1)
        return {"max_abs_err": float(err.max()), "max_err_over_sum_abs_x": float((err / np.maximum(mag, 1e-30)).max()),
                "bitwise_repeat": bool(same), "sampled_rows": int(len(idx)),
                "oracle_s_1_thread_scaled": t1, "oracle_s_all_threads_scaled": tn, "oracle_threads": cores}
    return {"max_abs_err": float(err.max()), "max_rel_err_where_ref_ge_1e-3": float(rel[np.abs(ref) >= 1e-3].max()
                                                                               if (np.abs(ref) >= 1e-3).any() else 0.0),
            "max_err_over_tolerance": float((err / ((1.6e-2 if op != "xent" else 1e-5) * np.maximum(1.0, np.abs(ref)))).max()),
            "bitwise_repeat": bool(same), "sampled_rows": int(len(idx)),
            "oracle_s_1_thread_scaled": t1, "oracle_s_all_threads_scaled": tn, "oracle_threads": cores}


# The ops added beyond the three headline ones, at the paper's Table 4 shapes (LayerNorm 8192 x 4096,
# reduce 16384 x 4096, rotary 2 x 32 x 2k x 128 in FP16), an FP16 variant, and the vocabulary-parallel
# cross-entropy as one of eight ranks runs it: timed briefly in every default run ("widened_rows").
WIDENED = [("layernorm", 8192, 4096), ("rowsum", 16384, 4096), ("rope.f16", 64 * 2048, 128),
           ("rmsnorm.f16", 8192, 8192), ("xent_vp8", 4096, 128256 // 8),
           # rows split over thread-block clusters: a vocabulary-sized softmax, training- and decoding-sized
           ("softmax", 4096, 128256), ("softmax", 16, 128256)]


def size_matched_sol(ak, op_base, sets, nsets, esize, rows, D, iters):
    """The library's plain copy (read-only ops: plain read) over buffers of the op's own size,
    same timing protocol and buffer rotation: what this GPU gives a kernel of that size that
    does no arithmetic.  Returns microseconds, or None where the buffers do not fit the aid."""
    nbytes = esize * rows * D
    if nbytes % 16 or any(t[0].data_ptr() % 16 for t in sets):
        return None
    l = ak.lib()
    if op_base in ("xent", "rowsum", "xent_vp8"):
        sink = torch.zeros((1,), dtype=torch.int32, device=sets[0][0].device)
        fn = lambda i: l.ak_sol_read(sets[i][0].data_ptr(), nbytes, sink.data_ptr(),
                                     torch.cuda.current_stream().cuda_stream)
    else:
        dst = [t[-1] for t in sets]
        if any(d.data_ptr() % 16 or d.numel() * d.element_size() != nbytes for d in dst):
            return None
        fn = lambda i: l.ak_sol_copy(sets[i][0].data_ptr(), dst[i].data_ptr(), nbytes,
                                     torch.cuda.current_stream().cuda_stream)
    us, _, _ = time_op(fn, nsets, iters=iters)
    return us


def run_sweep(ak, synth, dev, peak, shapes=None, iters=200, write=True, accuracy=True, out_path=None):
    rows_out = []
    only = os.environ.get("AK_SWEEP_OPS") if shapes is None else None
    for op, rows, D in (SWEEP if shapes is None else shapes):
        if only and op not in only.split(",") and not ("." in op and "dtypes" in only.split(",")):
            continue
        base, _, dts = op.partition(".")
        esize = 4 if dts == "f32" else 2
        one_set = (1 if base in ("xent", "rowsum", "xent_vp8") else 2) * esize * rows * D
        nsets = int(max(1, min(64, -(-(1 << 30) // one_set))))
        sets = []
        for s in range(nsets):
            if base == "rope":
                x = synth.rope_inputs(64, rows // 64, D, 7900 + s, device=dev, dtype=SWEEP_DTYPES[dts])
                sets.append((x, torch.empty_like(x)))
            elif op == "xent_vp8":
                lg, tg = synth.xent_inputs(rows, D, 7800 + s, device=dev)
                sets.append((lg, tg, torch.zeros((8, rows, 2, 2), dtype=torch.float32, device=dev)))
            elif dts:
                tdt = SWEEP_DTYPES[dts]
                if base == "rmsnorm":
                    x, w = synth.rmsnorm_inputs(rows, D, 7500 + s, device=dev, dtype=tdt)
                    sets.append((x, w, torch.empty_like(x)))
                elif base == "softmax":
                    x = synth.softmax_inputs(rows, D, 7600 + s, device=dev, dtype=tdt)
                    sets.append((x, torch.empty_like(x)))
                else:
                    sets.append(synth.xent_inputs(rows, D, 7700 + s, device=dev, dtype=tdt))
            elif op == "rmsnorm":
                x, w = synth.rmsnorm_inputs(rows, D, 7000 + s, device=dev)
                sets.append((x, w, torch.empty_like(x)))
            elif op == "layernorm":
                x, g, b = synth.layernorm_inputs(rows, D, 7300 + s, device=dev)
                sets.append((x, g, b, torch.empty_like(x)))
            elif op == "rowsum":
                x, _, _ = synth.layernorm_inputs(rows, D, 7400 + s, device=dev)
                sets.append((x, torch.empty((rows,), dtype=torch.float32, device=dev)))
            elif op == "softmax":
                x = synth.softmax_inputs(rows, D, 7100 + s, device=dev)
                sets.append((x, torch.empty_like(x)))
            else:
                lg, tg = synth.xent_inputs(rows, D, 7200 + s, device=dev)
                nws = ak.ak_xent_workspace_bytes(rows, D)
                sets.append((lg, tg, torch.empty((rows,), dtype=torch.float32, device=dev),
                             torch.empty((1,), dtype=torch.float32, device=dev),
                             torch.empty((nws,), dtype=torch.uint8, device=dev) if nws else None))
        if base == "rope":
            fn = lambda i: ak.ak_rope_fwd(sets[i][0], sets[i][1])
            nb = 2 * esize * rows * D
        elif op == "xent_vp8":
            def fn(i):
                lg, tg, parts = sets[i]
                ak.ak_xent_vp_partial(lg, tg, 0, 8 * D, 1, partial=parts[0])
                ak.ak_xent_vp_merge(parts, tg, 8 * D)
            nv = int((sets[0][1] != -100).sum())
            nb = 2 * D * nv + 8 * rows + (8 + 1) * 16 * rows + 12 * rows + 4
        elif dts:
            scale = esize // 2   # algorithmic_bytes counts 2-byte elements
            if base == "rmsnorm":
                fn = lambda i: ak.ak_rmsnorm_fwd_dt(sets[i][0], sets[i][1], sets[i][2], eps=1e-6)
                nb = algorithmic_bytes(base, rows, D) * scale
            elif base == "softmax":
                fn = lambda i: ak.ak_softmax_fwd_dt(sets[i][0], sets[i][1])
                nb = algorithmic_bytes(base, rows, D) * scale
            else:
                fn = lambda i: ak.ak_xent_fwd_dt(sets[i][0], sets[i][1])
                nv = int((sets[0][1] != -100).sum())
                nb = 2 * scale * D * nv + 12 * rows + 4
        elif op == "rmsnorm":
            fn = lambda i: ak.ak_rmsnorm_fwd(sets[i][0], sets[i][1], sets[i][2], eps=1e-6)
            nb = algorithmic_bytes(op, rows, D)
        elif op == "layernorm":
            fn = lambda i: ak.ak_layernorm_fwd(sets[i][0], sets[i][1], sets[i][2], sets[i][3], eps=1e-5)
            nb = algorithmic_bytes(op, rows, D)
        elif op == "rowsum":
            fn = lambda i: ak.ak_rowsum_fwd(sets[i][0], sets[i][1])
            nb = algorithmic_bytes(op, rows, D)
        elif op == "softmax":
            fn = lambda i: ak.ak_softmax_fwd(sets[i][0], sets[i][1])
            nb = algorithmic_bytes(op, rows, D)
        else:
            fn = lambda i: ak.ak_xent_fwd_ws(sets[i][0], sets[i][1], sets[i][4], -100, sets[i][2], sets[i][3])
            nb = algorithmic_bytes(op, rows, D, int((sets[0][1] != -100).sum()))
        us, us_min, us_med = time_op(fn, nsets, iters=iters)
        gbs = nb / (us * 1e-6) / 1e9
        # errors against the CPU checker and its timing belong to the per-shape CPU-baseline report
        # (before the copy below overwrites the outputs: the repeat check compares with what the
        # timed launches left in buffer set 0)
        acc = sweep_accuracy(ak, synth, op, rows, D, sets[0]) if accuracy else {}
        sol_us = size_matched_sol(ak, base, sets, nsets, esize, rows, D, max(iters // 2, 30)) if write else None
        rows_out.append({"op": op, "rows": rows, "D": D, "us_trimmed_mean": us, "us_min": us_min,
                         "us_median": us_med, "GB/s": gbs, "frac_of_8TBs": gbs / NOMINAL_HBM_GBS,
                         "frac_of_measured_copy": gbs / peak, "rows_per_s": rows / (us * 1e-6),
                         "buffer_sets": nsets, "large_shape": one_set >= (250 << 20),
                         "us_size_matched_copy": sol_us,
                         "frac_of_size_matched_copy": (sol_us / us if sol_us else None), **acc})
        del sets
        torch.cuda.empty_cache()
    if not write:
        return rows_out
    if out_path:
        os.makedirs(os.path.dirname(os.path.abspath(out_path)), exist_ok=True)
        with open(out_path, "w") as f:
            json.dump(rows_out, f, indent=1)
    for r in rows_out:
        sm = r["frac_of_size_matched_copy"]
        print(f"# {r['op']:11s} {r['rows']:7d} x {r['D']:6d}  {r['us_trimmed_mean']:9.1f} us  "
              f"{r['GB/s']:7.0f} GB/s  {100 * r['frac_of_8TBs']:5.1f}% of 8TB/s  "
              f"{100 * r['frac_of_measured_copy']:5.1f}% of copy  "
              + (f"{100 * sm:5.1f}% of a copy / read of its size" if sm else ""), file=sys.stderr)


def run_case(args):
    """A few launches of ONE op at one shape (for profiler captures on a small case):
    --case op:rows:D, e.g. xent:1024:128256.  Prints per-launch event times."""
    import paper_2603_21331_b200 as ak
    from paper_2603_21331_b200 import synth
    op, rows, D = args.case.split(":")
    rows, D = int(rows), int(D)
    dev = "cuda:0"
    torch.cuda.set_device(0)
    if op == "rope":   # rows = 64 sequences x S positions, D = head dimension, fp16 as in the paper
        x = synth.rope_inputs(64, rows // 64, D, 7900, device=dev, dtype=torch.float16)
        y = torch.empty_like(x)
        fn = lambda: ak.ak_rope_fwd(x, y)
        nb = 4 * rows * D
    elif op == "rmsnorm":
        x, w = synth.rmsnorm_inputs(rows, D, 7000, device=dev)
        y = torch.empty_like(x)
        fn = lambda: ak.ak_rmsnorm_fwd(x, w, y, eps=1e-6)
        nb = algorithmic_bytes(op, rows, D)
    elif op == "layernorm":
        x, gamma, beta = synth.layernorm_inputs(rows, D, 7300, device=dev)
        y = torch.empty_like(x)
        fn = lambda: ak.ak_layernorm_fwd(x, gamma, beta, y, eps=1e-5)
        nb = algorithmic_bytes(op, rows, D)
    elif op == "rowsum":
        x, _, _ = synth.layernorm_inputs(rows, D, 7400, device=dev)
        out = torch.empty((rows,), dtype=torch.float32, device=dev)
        fn = lambda: ak.ak_rowsum_fwd(x, out)
        nb = algorithmic_bytes(op, rows, D)
    elif op == "softmax":
        x = synth.softmax_inputs(rows, D, 7100, device=dev)
        y = torch.empty_like(x)
        fn = lambda: ak.ak_softmax_fwd(x, y)
        nb = algorithmic_bytes(op, rows, D)
    else:
        lg, tg = synth.xent_inputs(rows, D, 7200, device=dev)
        loss = torch.empty((rows,), dtype=torch.float32, device=dev)
        mean = torch.empty((1,), dtype=torch.float32, device=dev)
        nws = ak.ak_xent_workspace_bytes(rows, D)
        ws = torch.empty((nws,), dtype=torch.uint8, device=dev) if nws else None
        fn = lambda: ak.ak_xent_fwd_ws(lg, tg, ws, -100, loss, mean)
        nb = algorithmic_bytes(op, rows, D, int((tg != -100).sum()))
    for _ in range(args.warmup):
        fn()
    torch.cuda.synchronize()
    times = []
    for _ in range(args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b) * 1e3)
    print(json.dumps({"case": args.case, "algorithmic_bytes": nb, "us": times,
                      "GB/s_best": nb / (min(times) * 1e-6) / 1e9}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, help="op:rows:D - run a few launches of one op (profiling aid)")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--out", default=None, help="file the --sweep table is written to (JSON)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.case:
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_case(args)
        return
    if args.impl == "reference":
        args.steps = 5 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, rank, world)
        return
    args.steps = 100 if args.steps is None else args.steps
    args.warmup = 10 if args.warmup is None else args.warmup
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
