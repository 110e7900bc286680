#!/usr/bin/env python
"""Throughput of one two-way compressed dist-EF-blockSGDM step (Algorithm 4) on B200.

A "step" is the worker side of all M workers (one ef_worker_step_all launch, or M
ef_worker_step calls with --per-worker-calls) plus one ef_server_step over one batch of
synthetic gradients.  The default workload is the flat 2^28-parameter layout (256 blocks of
2^20, M = 7).  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]
                  [--graph] [--per-worker-calls] [--weight-decay L] [--diagnostics] [--blocks N]

With N > 1 (launched by torch.distributed.run) every rank owns its own block range of an
N-times larger problem (blocks are independent in the method, so there is no data-path
collective): weak scaling, value = parameters processed by all ranks per second.

--impl reference times the CPU oracle (plain single-threaded C++) on a bounded sample of the
same workload; it is a deliberately slow program, reported for context.
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

from paper_1905_10936_b200 import workloads as wl

METRIC = "parameters/sec through one two-way compressed dist-EF-blockSGDM step (M workers)"
UNIT = "params/s"

# DRAM traffic per launch of the worker kernel measured by ncu (dram__bytes_read.sum +
# dram__bytes_write.sum), in bytes per parameter; see profiles/ for the capture it comes from.
NCU_WORKER_TRAFFIC_BYTES_PER_PARAM = 20.10   # 37.766e9 bytes per 7-worker launch at d = 2^28


# --------------------------------------------------------------------------- byte counts
def worker_call_bytes(d: int, B: int) -> float:
    """Algorithmic bytes of one ef_worker_step: read g, m, e; write m, e; write 1 bit per
    element; write one fp32 scale per block."""
    return 20.125 * d + 4.0 * B


def server_call_bytes(d: int, B: int, M: int) -> float:
    """Algorithmic bytes of one ef_server_step: read M bits, etilde, x; write etilde, x, 1 bit
    per element; read M and write one scale per block."""
    return (16.0 + (M + 1) / 8.0) * d + 4.0 * B * (M + 1)


def step_bytes(d: int, B: int, M: int) -> float:
    return M * worker_call_bytes(d, B) + server_call_bytes(d, B, M)


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        self.period = period_s
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(device_index).uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    _NAMES = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
        0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown",
    }

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in self._NAMES.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self) -> dict:
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- CPU oracle legs
def time_oracle(w: wl.Workload, n_blocks: int, steps: int, warmup: int):
    """Times the oracle, as it stands, on the first n_blocks blocks of the workload.
    Returns (params_per_s, seconds_per_step, d_sample)."""
    from oracle import Oracle
    sizes = w.sizes[:n_blocks]
    sub = wl.custom_workload(w.name + "-sample", sizes, w.M, w.mu, w.eta, steps, w.law,
                             w.scale_range, config_id=w.config_id)
    orc = Oracle(sub.offsets, sub.M, sub.mu, sub.eta)
    es = sub.element_scales("cpu")
    grads = [sub.draw_grad(0, i, "cpu", es).numpy() for i in range(sub.M)]
    elapsed = 0.0
    for t in range(warmup + steps):
        t0 = time.perf_counter()
        for i in range(sub.M):
            orc.worker_step(i, grads[i])
        orc.server_step()
        if t >= warmup:
            elapsed += time.perf_counter() - t0
    return sub.d * steps / elapsed, elapsed / steps, sub.d


def oracle_ns_per_param(M: int) -> float:
    # rough cost model used only to size the sample: ~18 ns per worker-element, ~20 ns per
    # server-element on one host core
    return 18.0 * M + 20.0


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = load_workload(args)
    budget_s = 90.0
    per_block = np.mean(w.sizes) * oracle_ns_per_param(w.M) * 1e-9
    n_blocks = int(max(1, min(w.B, budget_s / ((args.steps + args.warmup) * per_block))))
    value, s_per_step, d_s = time_oracle(w, n_blocks, args.steps, args.warmup)
    sample = (f"first {n_blocks} of {w.B} blocks ({d_s} of {w.d} parameters), M={w.M}, "
              f"{args.steps} timed steps; single-threaded C++ oracle")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": s_per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "d": w.d, "B": w.B, "M": w.M, "mu": w.mu, "eta": w.eta},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- CUDA path
def run_ours(args) -> None:
    from paper_1905_10936_b200.engine import EFEngine
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = load_workload(args)
    K, W = args.steps, args.warmup
    # all work of the context runs on this (non-default) stream, which is also made current
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    eng = EFEngine(w.offsets, w.M, w.mu, w.eta, stream=stream, weight_decay=args.weight_decay > 0,
                   diagnostics=args.diagnostics)
    if args.weight_decay > 0:
        eng.set_weight_decay(args.weight_decay)
    es = w.element_scales(dev)
    stride = (w.d + 3) // 4 * 4
    gall = torch.zeros(w.M, stride, dtype=torch.float32, device=dev)   # pre-staged in HBM
    grads = [w.draw_grad(0, i, dev, es, out=gall[i, :w.d]) for i in range(w.M)]
    del es
    batched = not args.per_worker_calls

    def worker_calls():
        if batched:
            eng.worker_step_all(gall)          # all M workers in one launch
        else:
            for i in range(w.M):
                eng.worker_step(i, grads[i])

    def one_step():
        worker_calls()
        eng.server_step()

    for _ in range(W):
        one_step()
    barrier()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    sampler = ClockSampler(local_rank)
    launches0 = eng.launch_count
    sampler.start()
    barrier()
    for k in range(K):
        ev[k][0].record()
        worker_calls()
        ev[k][1].record()
        eng.server_step()
        ev[k][2].record()
    barrier()
    clocks = sampler.stop()
    launches = eng.launch_count - launches0
    total_ms = ev[0][0].elapsed_time(ev[K - 1][2])
    launches_per_step_worker = 1 if batched else w.M
    worker_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / (K * launches_per_step_worker)
    server_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / K
    if world > 1:
        tt = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())

    # ---- the same step replayed from a CUDA graph (launch gaps shrink; matters for small layouts)
    graph_info = None
    if args.graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            one_step()
        for _ in range(3):
            g.replay()
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(K):
            g.replay()
        g1.record()
        barrier()
        g_ms = g0.elapsed_time(g1)
        if world > 1:
            tt = torch.tensor([g_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            g_ms = float(tt.item())
        graph_info = {"ms_per_step": g_ms / K, "value": world * w.d * K / (g_ms * 1e-3),
                      "unit": UNIT, "note": "one whole step captured once, replayed K times"}
        del g

    # ---- end to end: host gradients in, packed update out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        del eng
        torch.cuda.empty_cache()
        eng2 = EFEngine(w.offsets, w.M, w.mu, w.eta, host_staging=True, stream=stream)
        hgrads = []
        for i in range(w.M):
            h = torch.empty(w.d, dtype=torch.float32).pin_memory()
            h.copy_(grads[i])
            hgrads.append(h)
        hwords = torch.empty(eng2.W, dtype=torch.int32).pin_memory()
        hscales = torch.empty(eng2.B, dtype=torch.float32).pin_memory()
        Ke = max(2, min(K, args.e2e_steps))

        def e2e_step():
            for i in range(w.M):
                eng2.worker_step_host(i, hgrads[i])
            eng2.server_step()
            eng2.read_update_host(hwords, hscales)

        for _ in range(2):
            e2e_step()
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        s0.record()
        for _ in range(Ke):
            e2e_step()
        s1.record()
        barrier()
        wall_ms = (time.perf_counter() - t0) * 1e3
        e2e_ms = max(s0.elapsed_time(s1), 0.0)
        if world > 1:
            tt = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            e2e_ms = float(tt.item())
        e2e = {"value": world * w.d * Ke / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(w.M * w.d * 4),
               "d2h_bytes_per_step": int(eng2.W * 4 + eng2.B * 4),
               "steps": Ke, "ms_per_step": e2e_ms / Ke, "wall_ms_per_step": wall_ms / Ke,
               "note": "pinned host gradients -> ef_worker_step_host (double-buffered H2D on a "
                       "copy stream) -> ef_server_step -> ef_read_update_host"}
        del eng2, hgrads

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_hbm_peak()
    wbytes = worker_call_bytes(w.d, w.B) * (w.M if batched else 1)
    sbytes = server_call_bytes(w.d, w.B, w.M) + (8.0 * w.d if args.weight_decay > 0 else 0.0)
    w_gbs = wbytes / (worker_ms * 1e-3) / 1e9
    s_gbs = sbytes / (server_ms * 1e-3) / 1e9
    state_gib = eng_state_gib(w)
    line = {
        "metric": METRIC, "value": world * w.d * K / (total_ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": total_ms / K,
        "steps_per_sec": K / (total_ms * 1e-3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "d": w.d, "B": w.B, "M": w.M, "mu": w.mu, "eta": w.eta,
                   "weight_decay": args.weight_decay, "diagnostics": bool(args.diagnostics),
                   "worker_calls": "ef_worker_step_all" if batched else "ef_worker_step x M",
                   "per_gpu": "each rank owns one such layout (block-range shard of an "
                              "N-times larger problem)",
                   "l2": f"no flush: state+gradients {state_gib:.1f} GiB per GPU, far larger "
                         "than the 126 MB L2"},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches * world),
        "roofline": {
            "kernel": "ef_worker_kernel", "call": ("ef_worker_step_all: M workers per launch" if batched
                                                   else "ef_worker_step: one worker per launch"),
            "bound": "hbm", "achieved": w_gbs, "peak": peak,
            "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": w_gbs / peak,
            "frac_of_8000_nominal": w_gbs / 8000.0,
            "bytes_per_launch": wbytes, "ms_per_launch": worker_ms,
            "traffic": (NCU_WORKER_TRAFFIC_BYTES_PER_PARAM * w.d * (w.M if batched else 1)
                        if NCU_WORKER_TRAFFIC_BYTES_PER_PARAM else None),
        },
        "roofline_server": {
            "kernel": "ef_server_kernel + ef_apply_kernel", "bound": "hbm", "achieved": s_gbs,
            "peak": peak, "unit": "GB/s", "frac": s_gbs / peak,
            "frac_of_8000_nominal": s_gbs / 8000.0, "bytes_per_call": sbytes,
            "ms_per_call": server_ms,
        },
        "step_gbs": step_bytes(w.d, w.B, w.M) / (total_ms / K * 1e-3) / 1e9,
    }
    if graph_info is not None:
        line["cuda_graph"] = graph_info
    if world == 1 and not args.no_cpu_baseline:
        per_block = np.mean(w.sizes) * oracle_ns_per_param(w.M) * 1e-9
        steps_c = 2
        n_blocks = int(max(1, min(w.B, 15.0 / ((steps_c + 1) * per_block))))
        v, s_per_step, d_s = time_oracle(w, n_blocks, steps_c, 1)
        line["cpu_baseline"] = {
            "value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"first {n_blocks} of {w.B} blocks ({d_s} of {w.d} parameters), M={w.M}, "
                      f"{steps_c} timed steps after 1 warm-up; single-threaded C++ oracle; "
                      f"host has {os.cpu_count()} cores"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def eng_state_gib(w: wl.Workload) -> float:
    return (w.d * 4.0 * (2 * w.M + 2) + w.d * 4.0 * w.M) / 2 ** 30


def load_workload(args) -> wl.Workload:
    w = wl.make_workload(args.config)
    if args.blocks and args.blocks < w.B:
        w = wl.custom_workload(f"{w.name}-first{args.blocks}blocks", w.sizes[:args.blocks], w.M,
                               w.mu, w.eta, w.steps, w.law, w.scale_range, config_id=w.config_id)
    if args.workers and args.workers != w.M:
        w = wl.custom_workload(f"{w.name}-M{args.workers}", w.sizes, args.workers, w.mu, w.eta,
                               w.steps, w.law, w.scale_range, config_id=w.config_id)
    return w


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=4, help="workload 1..5 (default: flat 2^28)")
    ap.add_argument("--blocks", type=int, default=0,
                    help="use only the first N blocks of the workload (small cases for profiling)")
    ap.add_argument("--workers", type=int, default=0,
                    help="override the number of simulated workers M of the workload")
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--per-worker-calls", action="store_true",
                    help="step the workers with M ef_worker_step calls instead of one ef_worker_step_all")
    ap.add_argument("--weight-decay", type=float, default=0.0,
                    help="enable the weight-decay side path (adds a d-float momentum to the server call)")
    ap.add_argument("--diagnostics", action="store_true",
                    help="worker steps also record the per-block diagnostic sums")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--graph", action="store_true",
                    help="also time the step replayed from a CUDA graph (extra key cuda_graph)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
