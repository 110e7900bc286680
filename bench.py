#!/usr/bin/env python
"""Throughput of one two-way compressed dist-EF-blockSGDM step (Algorithm 4) on B200.

A "step" is the worker side of all M workers (one ef_worker_step_all launch, or M
ef_worker_step calls with --per-worker-calls) plus one ef_server_step over one batch of
synthetic gradients (up to three batches are kept in HBM and rotated).  The default workload is
the flat 2^28-parameter layout (256 blocks of 2^20, M = 7).  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]
                  [--workload ef|signum|topk|ps [--push] [--process-group]] [--scaling weak|strong]
                  [--graph] [--ceiling] [--library-flags F]
                  [--per-worker-calls] [--weight-decay L] [--diagnostics] [--blocks N] [--workers M]

Keys beyond the common ones: `roofline` (worker launch), `roofline_server` (server call),
`sustained` (300 more back-to-back steps with the clocks sampled), `e2e` (host gradients in, packed
update out), `cpu_baseline` (the oracle on one host core), `cuda_graph` (--graph) and
`stream_ceiling` (--ceiling: no-compute kernels with the step kernels' access mix).

With N > 1 (launched by torch.distributed.run): --scaling weak (default) gives every rank one
whole layout (a block-range shard of an N-times larger problem; no data-path collective);
--scaling strong cuts ONE layout into N equal element ranges, blocks included, and all-reduces
one fp64 sum per cut block and call.

--workload ps: the sharded parameter server (one worker and one server shard per rank), with
the ranks emulated on one GPU (the pieces timed one by one) or, with --process-group or under
torchrun with N > 1, over the real process group; --push stores the messages directly into the
peers' buffers instead of packing them and calling collectives.

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
METRIC_SIGNUM = "parameters/sec through one signum-with-majority-vote step (M workers)"
UNIT = "params/s"

# DRAM traffic of the worker kernel from ncu (dram__bytes_read.sum + dram__bytes_write.sum) on
# the small case of the flat layout (its first 64 blocks: d = 2^26, M = 7, one launch of
# ef_worker_step_all), in bytes per worker-parameter; traffic grows in proportion to d*M on this
# layout (every CTA streams one 4096-element chunk), so a full launch is this figure x d x M.
# The capture is summarised in profiles/; the figure is reported for that layout only.
NCU_WORKER_TRAFFIC = {"workload": "C4-flat-2^28", "bytes_per_worker_param": 20.01,
                      "captured_on": "first 64 blocks (d = 2^26), M = 7, scaled by d*M"}


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


def vote_worker_call_bytes(d: int, B: int) -> float:
    """signum worker: read g, m; write m; write 1 bit per element."""
    return 12.125 * d


def vote_server_call_bytes(d: int, B: int, M: int) -> float:
    """signum server: read M bits and x; write x and 1 bit per element."""
    return (8.0 + (M + 1) / 8.0) * d


def config_dict(w) -> dict:
    """Names the workload; identical in both arms (descriptive extras go under "run")."""
    gib = eng_state_gib(w)
    return {"workload": w.name, "d": w.d, "B": w.B, "M": w.M, "mu": w.mu, "eta": w.eta,
            "l2": f"no flush: state + one gradient batch = {gib:.2f} GiB per GPU vs 126 MB of L2"
                  if gib * 2 ** 30 > 4 * 126e6 else
                  f"no flush: state + one gradient batch = {gib * 1024:.0f} MiB per GPU fits the "
                  "126 MB L2 (launch-latency-bound layout, reported as such)"}


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
def time_oracle(w: wl.Workload, n_blocks: int, steps: int, warmup: int, workload: str = "ef"):
    """Times the oracle, as it stands, on the first n_blocks blocks of the workload.
    Returns (params_per_s, seconds_per_step, d_sample)."""
    from oracle import Oracle, SignumOracle
    sizes = w.sizes[:n_blocks]
    sub = wl.custom_workload(w.name + "-sample", sizes, w.M, w.mu, w.eta, steps, w.law,
                             w.scale_range, config_id=w.config_id)
    orc = (SignumOracle if workload == "signum" else Oracle)(sub.offsets, sub.M, sub.mu, sub.eta)
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
    value, s_per_step, d_s = time_oracle(w, n_blocks, args.steps, args.warmup, args.workload)
    sample = (f"first {n_blocks} of {w.B} blocks ({d_s} of {w.d} parameters), M={w.M}, "
              f"{args.steps} timed steps; single-threaded C++ oracle")
    line = {
        "impl": "reference", "metric": METRIC_SIGNUM if args.workload == "signum" else METRIC,
        "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        # time one step of the WHOLE workload takes at the sampled rate (blocks are independent,
        # the oracle's cost is linear in the number of parameters); the sample's own step time
        # is given beside it
        "ms_per_step": w.d / value * 1e3, "ms_per_sample_step": s_per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": config_dict(w),
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

    def max_over_ranks(ms: float) -> float:
        if world == 1:
            return ms
        tt = torch.tensor([ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        return float(tt.item())

    w_full = load_workload(args)
    strong = args.scaling == "strong" and world > 1
    if strong:
        # ONE layout cut into equal element ranges (blocks are cut where a rank's share ends
        # inside one): this rank builds and steps only its own range.  The only data-path
        # exchange is an all-reduce of B doubles per call, and only if some block is cut.
        sh = wl.shard_elements(w_full.sizes, world, rank)
        w = wl.custom_workload(f"{w_full.name}[elements {sh.elem_lo}:{sh.elem_hi}]", sh.local_sizes or [4],
                               w_full.M, w_full.mu, w_full.eta, w_full.steps, w_full.law,
                               w_full.scale_range, config_id=1000 * w_full.config_id + rank)
        job_params = w_full.d                       # total work is fixed as N grows
    else:
        w = w_full                                  # every rank owns one whole layout
        job_params = world * w_full.d
    K, W = args.steps, args.warmup
    # all work of the context runs on this (non-default) stream, which is also made current
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    dshard = None
    if strong:
        from paper_1905_10936_b200.sharded import DistributedShard
        dshard = DistributedShard(w_full.sizes, w.M, w.mu, w.eta, rank, world, stream=stream,
                                  weight_decay=args.weight_decay > 0, extra_flags=args.library_flags)
        eng = dshard.eng
    else:
        eng = EFEngine(w.offsets, w.M, w.mu, w.eta, stream=stream, weight_decay=args.weight_decay > 0,
                       diagnostics=args.diagnostics, extra_flags=args.library_flags)
    if args.weight_decay > 0:
        eng.set_weight_decay(args.weight_decay)
    es = w.element_scales(dev)
    stride = (w.d + 3) // 4 * 4
    # Gradient batches pre-staged in HBM and rotated step by step (fresh values every step as
    # far as memory allows: up to 3 batches within a quarter of the device memory)
    free_b, total_b = torch.cuda.mem_get_info(dev)
    batch_bytes = w.M * stride * 4
    nbatch = int(max(1, min(3, args.grad_batches or 3, (total_b // 4) // max(batch_bytes, 1))))
    galls = []
    for bidx in range(nbatch):
        ga = torch.zeros(w.M, stride, dtype=torch.float32, device=dev)
        for i in range(w.M):
            w.draw_grad(bidx, i, dev, es, out=ga[i, :w.d])
        galls.append(ga)
    del es
    batched = not args.per_worker_calls
    step_no = [0]
    signum = args.workload == "signum"
    step_all = eng.vote_worker_step_all if signum else eng.worker_step_all
    step_one = eng.vote_worker_step if signum else eng.worker_step
    server_call = eng.vote_server_step if signum else eng.server_step
    if dshard is not None:              # cut layout: the step calls go through the exchange
        assert not signum and batched, "--scaling strong runs the default workload with batched worker calls"
        step_all, server_call = dshard.worker_step_all, dshard.server_step
    w_bytes_fn = vote_worker_call_bytes if signum else worker_call_bytes
    s_bytes_fn = vote_server_call_bytes if signum else server_call_bytes

    def worker_calls():
        ga = galls[step_no[0] % nbatch]
        if batched:
            step_all(ga)                       # all M workers in one launch
        else:
            for i in range(w.M):
                step_one(i, ga[i, :w.d])

    def one_step():
        worker_calls()
        server_call()
        step_no[0] += 1

    for _ in range(W):
        one_step()
    barrier()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    sampler = ClockSampler(local_rank, period_s=0.002)
    launches0 = eng.launch_count
    sampler.start()
    barrier()
    for k in range(K):
        ev[k][0].record()
        worker_calls()
        ev[k][1].record()
        server_call()
        ev[k][2].record()
        step_no[0] += 1
    barrier()
    clocks = sampler.stop()
    launches = eng.launch_count - launches0
    total_ms = ev[0][0].elapsed_time(ev[K - 1][2])
    launches_per_step_worker = 1 if batched else w.M
    worker_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / (K * launches_per_step_worker)
    server_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / K
    total_ms = max_over_ranks(total_ms)
    if clocks.get("sm_mhz"):
        clocks["ms_per_step_x_sm_mhz"] = total_ms / K * clocks["sm_mhz"]

    # ---- sustained: many back-to-back steps (the board reaches its power limit after ~1 s)
    sustained = None
    if args.sustained_steps > 0:
        Ks = args.sustained_steps
        s_sampler = ClockSampler(local_rank, period_s=0.01)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        s_sampler.start()
        s0.record()
        for _ in range(Ks):
            one_step()
        s1.record()
        barrier()
        s_clk = s_sampler.stop()
        s_ms = max_over_ranks(s0.elapsed_time(s1))
        sustained = {"steps": Ks, "ms_per_step": s_ms / Ks, "value": job_params * Ks / (s_ms * 1e-3),
                     "unit": UNIT, "seconds": s_ms * 1e-3, "sm_mhz": s_clk.get("sm_mhz"),
                     "sm_max_mhz": s_clk.get("sm_max_mhz"), "reasons": s_clk.get("reasons"),
                     "clock_samples": s_clk.get("samples"),
                     "step_gbs": (w.M * w_bytes_fn(w.d, w.B) + s_bytes_fn(w.d, w.B, w.M))
                                 / (s_ms / Ks * 1e-3) / 1e9}

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
        g_ms = max_over_ranks(g0.elapsed_time(g1))
        graph_info = {"ms_per_step": g_ms / K, "value": job_params * K / (g_ms * 1e-3),
                      "unit": UNIT, "note": "one whole step captured once, replayed K times"}
        del g

    # ---- ceiling of a no-compute kernel with the worker step's access mix (3 reads, 2 writes)
    ceiling = None
    if args.ceiling:
        ceiling = stream_ceilings(eng, galls[0], w, stream)

    # ---- end to end: host gradients in, packed update out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        hsrc = galls[0]
        del eng
        torch.cuda.empty_cache()
        eng2 = EFEngine(w.offsets, w.M, w.mu, w.eta, host_staging=True, stream=stream)
        hgrads = []
        for i in range(w.M):
            h = torch.empty(w.d, dtype=torch.float32).pin_memory()
            h.copy_(hsrc[i, :w.d])
            hgrads.append(h)
        hwords = torch.empty(eng2.W, dtype=torch.int32).pin_memory()
        hscales = torch.empty(eng2.B, dtype=torch.float32).pin_memory()
        Ke = max(2, min(K, args.e2e_steps))

        def e2e_step():
            for i in range(w.M):
                (eng2.vote_worker_step_host if signum else eng2.worker_step_host)(i, hgrads[i])
            (eng2.vote_server_step if signum else eng2.server_step)()
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
        e2e_ms = max_over_ranks(max(s0.elapsed_time(s1), 0.0))
        e2e = {"value": job_params * Ke / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(w.M * w.d * 4),
               "d2h_bytes_per_step": int(eng2.W * 4 + eng2.B * 4),
               "steps": Ke, "ms_per_step": e2e_ms / Ke, "wall_ms_per_step": wall_ms / Ke,
               "note": ("pinned host gradients -> ef_vote_worker_step_host (double-buffered H2D on a copy "
                        "stream) -> ef_vote_server_step -> ef_read_update_host; PCIe-bound" if signum else
                        "pinned host gradients -> ef_worker_step_host (double-buffered H2D on a "
                        "copy stream) -> ef_server_step -> ef_read_update_host; PCIe-bound")}
        del eng2, hgrads

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_hbm_peak()
    wbytes = w_bytes_fn(w.d, w.B) * (w.M if batched else 1)
    sbytes = s_bytes_fn(w.d, w.B, w.M) + (8.0 * w.d if args.weight_decay > 0 else 0.0)
    w_gbs = wbytes / (worker_ms * 1e-3) / 1e9
    s_gbs = sbytes / (server_ms * 1e-3) / 1e9
    plain = (args.weight_decay == 0 and not args.diagnostics and world == 1 and not signum)
    traffic = None
    if plain and w.name == NCU_WORKER_TRAFFIC["workload"]:
        traffic = NCU_WORKER_TRAFFIC["bytes_per_worker_param"] * w.d * (w.M if batched else 1)
    line = {
        "metric": METRIC_SIGNUM if signum else METRIC,
        "value": job_params * K / (total_ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": total_ms / K,
        "steps_per_sec": K / (total_ms * 1e-3),
        "higher_is_better": True, "scaling": args.scaling if world > 1 else "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(w_full),
        "run": {"workload": args.workload, "library_flags": args.library_flags,
                "weight_decay": args.weight_decay, "diagnostics": bool(args.diagnostics),
                "worker_calls": "ef_worker_step_all" if batched else "ef_worker_step x M",
                "gradient_batches_rotated": nbatch,
                "per_gpu": ("every rank owns one whole layout (a block-range shard of an N-times "
                            "larger problem); no data-path collective" if args.scaling == "weak" or world == 1
                            else f"one layout cut into {world} equal element ranges (workloads.shard_elements, "
                                 "blocks cut where needed); each rank builds and steps only its own range; "
                                 "one all-reduce of B doubles per call if a block is cut")},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches * world),
        "roofline": {
            "kernel": "ef_vote_worker_kernel" if signum else "ef_worker_kernel",
            "call": ("all M workers in one launch" if batched else "one worker per launch"),
            "bound": "hbm", "achieved": w_gbs, "peak": peak,
            "peak_kind": f"of {peak_kind} (a 1:1 copy; context for a kernel that reads 60% of its bytes)",
            "unit": "GB/s", "frac": w_gbs / peak,
            "frac_of_8000_nominal": w_gbs / 8000.0,
            "bytes_per_launch": wbytes, "ms_per_launch": worker_ms,
            "traffic": traffic,
            "traffic_source": NCU_WORKER_TRAFFIC["captured_on"] if traffic else None,
        },
        "roofline_server": {
            "kernel": ("ef_vote_server_kernel" if signum else
                       "ef_server_kernel (+ ef_apply_kernel where the update is not fused)"),
            "bound": "hbm", "achieved": s_gbs,
            "peak": peak, "unit": "GB/s", "frac": s_gbs / peak,
            "frac_of_8000_nominal": s_gbs / 8000.0, "bytes_per_call": sbytes,
            "ms_per_call": server_ms,
        },
        "step_gbs": (w.M * w_bytes_fn(w.d, w.B) + s_bytes_fn(w.d, w.B, w.M)) / (total_ms / K * 1e-3) / 1e9,
    }
    if sustained is not None:
        line["sustained"] = sustained
    if graph_info is not None:
        line["cuda_graph"] = graph_info
    if ceiling is not None:
        line["stream_ceiling"] = ceiling
        line["roofline"]["frac_of_stream_ceiling"] = w_gbs / ceiling["3r2w_gbs"]
        line["roofline_server"]["frac_of_stream_ceiling"] = s_gbs / ceiling["1r1w_gbs"]
    if world == 1 and not args.no_cpu_baseline:
        per_block = np.mean(w.sizes) * oracle_ns_per_param(w.M) * 1e-9
        steps_c = 2
        n_blocks = int(max(1, min(w.B, 15.0 / ((steps_c + 1) * per_block))))
        v, s_per_step, d_s = time_oracle(w, n_blocks, steps_c, 1, args.workload)
        line["cpu_baseline"] = {
            "value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"first {n_blocks} of {w.B} blocks ({d_s} of {w.d} parameters), M={w.M}, "
                      f"{steps_c} timed steps after 1 warm-up; single-threaded C++ oracle; "
                      f"host has {os.cpu_count()} cores"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def stream_ceilings(eng, gall: torch.Tensor, w: wl.Workload, stream) -> dict:
    """Rates of the library's no-compute stream kernels (ef_stream_probe) on buffers of this
    workload's size: the ceiling a kernel with the same read/write mix can reach."""
    from paper_1905_10936_b200 import binding as ef
    n = (w.d // 4096) * 4096
    a = gall[0, :n]
    b = torch.empty(n, dtype=torch.float32, device=gall.device)
    c = torch.empty(n, dtype=torch.float32, device=gall.device)
    out = {}
    for mode, key, bytes_per_elem in ((ef.EF_PROBE_3R2W, "3r2w_gbs", 20.0),
                                      (ef.EF_PROBE_1R1W, "1r1w_gbs", 8.0)):
        reps = max(3, min(50, int(2e10 / (bytes_per_elem * n))))
        for _ in range(3):
            ef.ef_stream_probe(mode, a.data_ptr(), b.data_ptr(), c.data_ptr(), n, stream.cuda_stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            ef.ef_stream_probe(mode, a.data_ptr(), b.data_ptr(), c.data_ptr(), n, stream.cuda_stream)
        e1.record()
        torch.cuda.synchronize()
        out[key] = bytes_per_elem * n * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9
    out["note"] = (f"no-compute float4 stream kernels on {n} elements per buffer, one 4096-element "
                   "chunk per CTA: 3 reads + 2 writes (the worker step's mix) and 1 read + 1 write")
    return out


def run_topk(args) -> None:
    """The top-k compressor (ef_topk_compress) on a vector of the workload's size: one "step" is
    one call (threshold search, ordered scatter of k index/value pairs, residual)."""
    from paper_1905_10936_b200 import binding as ef
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = load_workload(args)
    n, k = w.d, max(1, int(w.d * args.topk_fraction))
    K, W = args.steps, args.warmup
    if args.impl == "reference":
        from oracle import topk_compress
        ns = min(n, 1 << 22)
        v = w.draw_grad(0, 0, "cpu")[:ns].numpy()
        t0 = time.perf_counter()
        for _ in range(K):
            topk_compress(v, max(1, int(ns * args.topk_fraction)))
        value = ns * K / (time.perf_counter() - t0)
        line = {"impl": "reference", "metric": "elements/sec through the top-k compressor", "value": value,
                "unit": "elements/s", "n_gpus": args.gpus, "steps": K, "warmup": W, "ms_per_step": n / value * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": config_dict(w),
                "cpu_baseline": {"value": value, "unit": "elements/s", "cores": 1, "kind": "oracle",
                                 "sample": f"first {ns} of {n} elements, sort-based definition"},
                "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line), flush=True)
        return
    torch.cuda.set_device(0)
    v = w.draw_grad(0, 0, "cuda", w.element_scales("cuda"))
    ws = torch.empty(ef.ef_topk_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    idx = torch.empty(k, dtype=torch.int64, device="cuda")
    val = torch.empty(k, device="cuda")
    resid = torch.empty(n, device="cuda")
    st = torch.cuda.current_stream().cuda_stream

    def call():
        ef.ef_topk_compress(v.data_ptr(), n, k, idx.data_ptr(), val.data_ptr(), resid.data_ptr(),
                            ws.data_ptr(), ws.numel(), st)
    for _ in range(W):
        call()
    torch.cuda.synchronize()
    sampler = ClockSampler(0, period_s=0.002)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    e0.record()
    for _ in range(K):
        call()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / K
    peak, kind = measured_hbm_peak()
    nbytes = 16.0 * n + 12.0 * k           # three reads of v, one write of the residual, k pairs
    line = {"metric": "elements/sec through the top-k compressor", "value": n / (ms * 1e-3), "unit": "elements/s",
            "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config_dict(w),
            "run": {"workload": "topk", "n": n, "k": k}, "clocks": clocks, "e2e": None, "gpu_launches": 9 * K,
            "roofline": {"kernel": "ef_topk_* (9 launches per call)", "bound": "hbm",
                         "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": peak, "peak_kind": f"of {kind}",
                         "unit": "GB/s", "frac": nbytes / (ms * 1e-3) / 1e9 / peak, "traffic": None,
                         "bytes_per_launch": nbytes}}
    print(json.dumps(line), flush=True)


def run_ps_group(args) -> None:
    """The paper's setting over a process group: one rank per GPU (torchrun), rank r = worker r
    and the server of one block range, M = world size.  --push: buffers in symmetric memory, the
    kernels store the messages into the peers' buffers, two one-element all-reduces per iteration;
    otherwise all-to-all and all-gather.  Timed as the whole iteration, max over ranks."""
    import torch.distributed as dist
    from paper_1905_10936_b200 import ps
    from paper_1905_10936_b200.engine import EFEngine
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29541")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    w0 = load_workload(args)
    w = wl.custom_workload(f"{w0.name}-M{world}", w0.sizes, world, w0.mu, w0.eta, w0.steps, w0.law,
                           w0.scale_range, config_id=w0.config_id)
    K, W = args.steps, args.warmup
    eng = EFEngine(w.offsets, world, w.mu, w.eta, one_local_worker=True)
    if args.push:
        recv, update, recv_ptrs, update_ptrs = ps.symmetric_buffers(w.sizes, rank, world, dev)
        rk = ps.Rank(eng, w.sizes, rank, world, recv=recv, update=update)
        rk.connect(recv_ptrs, update_ptrs)
    else:
        rk = ps.Rank(eng, w.sizes, rank, world)
    flag = torch.zeros(1, device=dev)
    grad = w.draw_grad(0, rank, "cuda", w.element_scales("cuda"))

    def one():
        if args.push:
            ps.step_push(rk, grad, flag)
        else:
            ps.step(rk, grad)

    for _ in range(W):
        one()
    dist.barrier(); torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(K):
        one()
    e1.record()
    dist.barrier(); torch.cuda.synchronize()
    tt = torch.tensor([e0.elapsed_time(e1)], device=dev, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    ms = float(tt.item()) / K
    if rank == 0:
        units = rk.total_units
        line = {"metric": "parameters/sec through one iteration of the sharded parameter-server protocol "
                          "(one worker and one server shard per GPU)",
                "value": w.d / (ms * 1e-3), "unit": "params/s", "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic", "config": config_dict(w),
                "run": {"workload": "ps", "variant": "push" if args.push else "collective", "ranks": world,
                        "process_group": "nccl",
                        "exchange_bytes_per_rank": {"out": 4 * units * (world - 1) // world,
                                                    "in": 4 * units * (world - 1) // world}},
                "e2e": None, "gpu_launches": int(eng.launch_count)}
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


def run_ps(args) -> None:
    """The paper's setting in pieces on ONE GPU: G ranks (rank r = worker r + the server of one
    block range) stepped one after the other, the exchange replaced by device copies.  Times the
    pieces a real rank would run between its collectives; the exchange itself cannot be measured
    on one device and is given analytically (bytes per rank and phase).  --push times the push
    variant instead: the worker kernel stores its message into the servers' receive buffers and
    the servers store their update slices into every rank's update buffer (here all on one
    device, so the stores that would cross NVLink are local)."""
    from paper_1905_10936_b200 import ps
    from paper_1905_10936_b200.engine import EFEngine
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = load_workload(args)
    G, K, W = w.M, args.steps, args.warmup
    torch.cuda.set_device(0)
    ranks = [ps.Rank(EFEngine(w.offsets, G, w.mu, w.eta, one_local_worker=True), w.sizes, r, G) for r in range(G)]
    es = w.element_scales("cuda")
    grads = [w.draw_grad(0, i, "cuda", es) for i in range(G)]
    names = (["worker_step_push", "server_step_range", "push_update", "apply_update"] if args.push else
             ["worker_step", "pack_message", "server_step_range", "pack_update", "apply_update"])
    if args.push:
        ps.connect_emulated(ranks)
    acc = {n: 0.0 for n in names}

    def timed(name, fn, record):
        if not record:
            fn()
            return
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        pending.append((name, e0, e1))

    for it in range(W + K):
        rec = it >= W
        pending = []
        if args.push:
            for rk, g in zip(ranks, grads):
                timed("worker_step_push", lambda: rk.engine.worker_step_push(0, g, rk.block_dst), rec)
            for rk in ranks:
                m = rk.mine
                if m.b1 > m.b0:
                    timed("server_step_range", lambda: rk.engine.server_step_range(m.b0, m.b1, rk.recv), rec)
                    timed("push_update", lambda: rk.engine.push_message(-1, m.b0, m.b1, rk.update_dst), rec)
            for rk in ranks:
                timed("apply_update", lambda: rk.engine.apply_update(0, rk.B, rk.update), rec)
            torch.cuda.synchronize()
            for name, e0, e1 in pending:
                acc[name] += e0.elapsed_time(e1)
            continue
        for rk, g in zip(ranks, grads):
            timed("worker_step", lambda: rk.engine.worker_step(0, g), rec)
            timed("pack_message", lambda: rk.engine.pack_message(0, 0, rk.B, rk.send), rec)
        for dst in ranks:                                   # stands in for the all-to-all
            m = dst.mine
            for src in ranks:
                if m.units:
                    dst.recv[src.rank, :m.units].copy_(src.send[m.unit0:m.unit0 + m.units])
        for rk in ranks:
            m = rk.mine
            if m.b1 > m.b0:
                timed("server_step_range", lambda: rk.engine.server_step_range(m.b0, m.b1, rk.recv), rec)
                timed("pack_update", lambda: rk.engine.pack_message(-1, m.b0, m.b1,
                                                                    rk.update[m.unit0:m.unit0 + m.units]), rec)
        for dst in ranks:                                   # stands in for the all-gather
            for src in ranks:
                p = src.mine
                if src is not dst and p.units:
                    dst.update[p.unit0:p.unit0 + p.units].copy_(src.update[p.unit0:p.unit0 + p.units])
        for rk in ranks:
            timed("apply_update", lambda: rk.engine.apply_update(0, rk.B, rk.update), rec)
        torch.cuda.synchronize()
        for name, e0, e1 in pending:
            acc[name] += e0.elapsed_time(e1)
    per_rank_ms = {n: acc[n] / (K * G) for n in names}      # average over ranks and steps
    total_ms = sum(per_rank_ms.values())
    units = ranks[0].total_units
    line = {"metric": "parameters/sec per rank through one iteration of the sharded parameter-server "
                      "protocol (compute pieces only; ranks emulated one after the other on one GPU)",
            "value": w.d / (total_ms * 1e-3), "unit": "params/s", "n_gpus": 1, "steps": K, "warmup": W,
            "ms_per_step": total_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": config_dict(w),
            "run": {"workload": "ps", "variant": "push" if args.push else "collective", "ranks": G,
                    "ms_per_rank": per_rank_ms,
                    "bytes_per_rank": {"worker_step": worker_call_bytes(w.d, w.B),
                                       "server_step_range": (8.0 + (G + 1) / 8.0) * w.d / G,
                                       "apply_update": 8.125 * w.d},
                    "exchange_bytes_per_rank": {"all_to_all_out": 4 * units * (G - 1) // G,
                                                "all_gather_in": 4 * units * (G - 1) // G},
                    "note": "the exchange is not timed: on NVLink at the pool's measured 770 GB/s per "
                            "direction the two phases would take "
                            f"{2 * 4 * units * (G - 1) / G / 770e9 * 1e6:.0f} us per iteration"},
            "e2e": None, "gpu_launches": int(sum(rk.engine.launch_count for rk in ranks))}
    print(json.dumps(line), flush=True)


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
    ap.add_argument("--workload", choices=["ef", "signum", "topk", "ps"], default="ef",
                    help="ef: dist-EF-blockSGDM (default, the headline); signum: the paper's "
                         "comparison method, signum with majority vote, on the same layouts; "
                         "topk: the top-k compressor on one vector of the layout's size; "
                         "ps: the one-worker-per-rank protocol with a block-sharded server, its "
                         "compute pieces timed with the M ranks emulated on one GPU")
    ap.add_argument("--process-group", action="store_true",
                    help="--workload ps: run over the torch.distributed process group (one rank per GPU; "
                         "implied under torchrun with more than one rank) instead of emulating the ranks")
    ap.add_argument("--push", action="store_true",
                    help="--workload ps: the push variant (messages stored where their readers are)")
    ap.add_argument("--topk-fraction", type=float, default=0.01, help="k / n for --workload topk")
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
    ap.add_argument("--library-flags", type=int, default=0,
                    help="extra EF_FLAG_* bits for ef_init (A/B comparisons: 512 = per-thread staging in "
                         "the server kernel, 1024 = programmatic instead of ordinary launches)")
    ap.add_argument("--sustained-steps", type=int, default=300,
                    help="extra back-to-back steps timed as one region with the clocks sampled "
                         "(key `sustained`; 0 = skip)")
    ap.add_argument("--scaling", choices=["weak", "strong"], default="weak",
                    help="N > 1: weak = every rank owns one whole layout; strong = one layout cut "
                         "into block ranges, each rank builds only its own")
    ap.add_argument("--grad-batches", type=int, default=0,
                    help="gradient batches kept in HBM and rotated (default: up to 3)")
    ap.add_argument("--ceiling", action="store_true",
                    help="also time the library's no-compute stream kernels (key `stream_ceiling`)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.workload == "topk":
        run_topk(args)
    elif args.workload == "ps":
        if args.process_group or int(os.environ.get("WORLD_SIZE", "1")) > 1:
            run_ps_group(args)
        else:
            run_ps(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
