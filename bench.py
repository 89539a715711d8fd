#!/usr/bin/env python
"""Benchmark of the KroQuant online activation quantizer on B200.

One *step* = one denoising-step-like pass of the quantizer over a FLUX.1-schnell-shaped
layer stack: 28 consecutive calls, 14 on X[4608, 3072] and 14 on X[4608, 12288]
(interleaved), each call with its own input buffer, output buffers and factor set,
captured in one CUDA graph.  The 28 inputs total 1.98 GB, far beyond the 126 MB L2, so
every call reads its input from HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` = algorithmic bytes moved per second by the
whole job (2 B read + 0.5 B codes + 1/32 B scale per element), inputs resident in HBM;
`e2e` = the same metric with pinned-host inputs and outputs, copies inside the timed
region.  `--impl reference` times the CPU oracle on a bounded sample of the same
workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_21446_b200 import workloads as W  # noqa: E402

METRIC = "quantizer_hbm_throughput"
UNIT = "GB/s"
CALLS_PER_STEP = 28
SHAPES = [(4608, 3072), (4608, 12288)]
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per launch of the tensor-core kernel from the Nsight Compute captures
# summarised under profiles/ (dram__bytes_read.sum + dram__bytes_write.sum); None = not captured.
NCU_TRAFFIC_BYTES = {(4608, 3072): 28.36e6, (4608, 12288): 125.3e6}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def step_bytes() -> float:
    return sum(W.algorithmic_bytes(t, d) for t, d in SHAPES) * (CALLS_PER_STEP // 2)


def step_tokens() -> int:
    return sum(t for t, _ in SHAPES) * (CALLS_PER_STEP // 2)


# --------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines: list[str] = []
        self.first = 0            # samples [first, last) were taken between mark_begin() and mark_end()
        self.last = None

    def mark_begin(self):
        self.first = len(self.lines)

    def mark_end(self):
        self.last = len(self.lines)

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def count(self) -> int:
        return len(self.lines)

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        # the samples of the marked region and one on either side of it (all of them if nothing was marked)
        lo = max(0, self.first - 1)
        hi = len(self.lines) if self.last is None else min(len(self.lines), self.last + 1)
        for ln in self.lines[lo:hi]:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [v for v in sm if v > 0.5 * max(sm)] or sm
        return {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(mx)),
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------
# reference arm: the CPU oracle on a bounded sample
# --------------------------------------------------------------------------------------
SAMPLE = "calls 0 and 1 of the 28-call step (the full X[4608,3072] and X[4608,12288] tensors)"


def oracle_sample_inputs():
    return [(W.gen_activations(sp), W.gen_factors(3, layer=layer))
            for layer, sp in enumerate(W.flux_specs())]


def time_oracle(steps: int, warmup: int):
    """The cpu_baseline leg: the C oracle, as it stands, on the sample.  Returns its throughput and
    the outputs of its last pass (the timed GPU calls 0 and 1 are compared with them)."""
    from oracle import c_oracle as co
    inputs = oracle_sample_inputs()
    byts = sum(W.algorithmic_bytes(*x.shape) for x, _ in inputs)
    outs = []

    def one():
        outs.clear()
        for x, g in inputs:
            outs.append(co.quantize(x, g))
    for _ in range(max(warmup, 1)):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = (time.perf_counter() - t0) / steps
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return byts / dt / 1e9, dt, cores, outs


ONE_THREAD_ROWS = 512


def time_oracle_one_thread():
    """The same oracle on ONE host thread, on the first 512 token rows of each of the two sample tensors
    (the work is uniform over rows).  The oracle's OpenMP team size is set through its own runtime; nothing
    in the oracle changes."""
    import ctypes
    from oracle import c_oracle as co
    co.lib()                                           # loads the oracle (and with it the OpenMP runtime)
    try:
        omp = ctypes.CDLL("libgomp.so.1")
        n_before = int(omp.omp_get_max_threads())
        omp.omp_set_num_threads(1)
    except OSError:
        return None
    try:
        inputs = [(x[:ONE_THREAD_ROWS], g) for x, g in oracle_sample_inputs()]
        byts = sum(W.algorithmic_bytes(*x.shape) for x, _ in inputs)
        for x, g in inputs:
            co.quantize(x, g)
        t0 = time.perf_counter()
        for x, g in inputs:
            co.quantize(x, g)
        dt = time.perf_counter() - t0
    finally:
        omp.omp_set_num_threads(n_before)
    return {"value": byts / dt / 1e9, "unit": UNIT, "cores": 1,
            "sample": f"first {ONE_THREAD_ROWS} token rows of each sample tensor, {dt:.2f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 10))
    gbs, dt, cores, _ = time_oracle(steps, min(args.warmup, 2))
    sample = f"{SAMPLE} per step, C oracle (fp64, OpenMP over token rows)"
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 2), "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": "flux_step_28_calls (bounded sample)", "l2": "oracle on host cores"},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------
# multi-GPU plumbing: one process per GPU, token rows / calls sharded, no data-path collective
# --------------------------------------------------------------------------------------
def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def relaunch_under_torchrun(argv, n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this same command line with
    torch.distributed.run on this node (rendezvous on 127.0.0.1) and pass their output through."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


class Ranks:
    """torch.distributed reduced to what the bench needs: barrier and max / sum over ranks."""

    def __init__(self, backend: str, device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.dist = None
        self.device = device
        if self.world > 1:
            import torch.distributed as dist
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            if backend == "nccl":
                dist.init_process_group("nccl", device_id=device)
            else:
                dist.init_process_group(backend)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def _reduce(self, value: float, op) -> float:
        if self.dist is None:
            return value
        import torch
        t = torch.tensor([value], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=op)
        return float(t.item())

    def max(self, value: float) -> float:
        return self._reduce(value, self.dist.ReduceOp.MAX) if self.dist is not None else value

    def sum(self, value: float) -> float:
        return self._reduce(value, self.dist.ReduceOp.SUM) if self.dist is not None else value

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def run_dist_selftest(args):
    """The launch / barrier / max-over-ranks logic of the bench on CPU ranks (gloo) with a stub step: every rank
    'processes' step_bytes() in a time that depends on its rank; rank 0 prints the line the real bench would."""
    ranks = Ranks("gloo")
    ranks.barrier()
    t_rank = 1e-3 * (1 + ranks.rank)                     # the slowest rank sets the step time
    t = ranks.max(t_rank)
    units = ranks.sum(float(step_bytes()))
    ranks.barrier()
    if ranks.rank == 0:
        print(json.dumps({"selftest": "dist", "n_gpus": ranks.world, "ms_per_step": t * 1e3,
                          "value": units / t / 1e9, "unit": UNIT, "scaling": "weak"}), flush=True)
    ranks.close()


# --------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------
def build_inputs(torch, B, device):
    """28 distinct input buffers: the seeded FLUX-shaped tensors, rolled by i token rows."""
    specs = W.flux_specs()
    base = []
    for sp in specs:
        bits = W.gen_activations(sp)
        base.append((bits, torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)))
    calls = []
    for i in range(CALLS_PER_STEP):
        k = i % 2
        bits, x0 = base[k]
        shift = i // 2
        x = torch.roll(x0, shifts=shift, dims=0).contiguous() if shift else x0
        G = W.gen_factors(3, layer=i)
        t, d = x.shape
        calls.append({
            "shift": shift, "shape_idx": k, "X": x, "G": G, "factors": B.Factors.create(G),
            "q": torch.empty((t, d // 2), dtype=torch.uint8, device=device),
            "s": torch.empty((t, d // 32), dtype=torch.uint8, device=device),
            "sv": torch.from_numpy(W.gen_channel_scales(3, d, layer=i)).to(device),
        })
    return base, calls


def capture(torch, fns, stream):
    with torch.cuda.stream(stream):
        for f in fns:
            f()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for f in fns:
                f()
    return g


def capture_overlapped(torch, calls, fn, stream, n_streams=3):
    """The same calls, captured with call i on stream i % n_streams (fork from `stream`, join back): the
    calls are independent (own inputs, outputs, factors), so consecutive kernels may overlap."""
    sides = [torch.cuda.Stream() for _ in range(n_streams - 1)]
    lanes = [stream] + sides
    with torch.cuda.stream(stream):
        for c in calls:
            fn(c, stream)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for sd in sides:
                sd.wait_stream(stream)
            for i, c in enumerate(calls):
                fn(c, lanes[i % n_streams])
            for sd in sides:
                stream.wait_stream(sd)
    return g


def time_graph(torch, dist, g, stream, steps, warmup, sampler=None):
    """W untimed replays, then exactly `steps` timed replays between two events on `stream`.
    The clock sampler (nvidia-smi, 20 ms period) is started first and the GPU idles until its first samples have
    arrived (the tool takes some hundred milliseconds to start); the reported clocks are those of the samples taken
    during the timed region and of one on either side; untimed replays keep the load up until that last one arrives."""
    with torch.cuda.stream(stream):
        if sampler:
            sampler.start()
            t_end = time.perf_counter() + 4.0
            while sampler.proc is not None and sampler.count() < 2 and time.perf_counter() < t_end:
                time.sleep(0.01)
        for _ in range(warmup):
            g.replay()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if sampler:
            sampler.mark_begin()
        a.record(stream)
        for _ in range(steps):
            g.replay()
        b.record(stream)
        torch.cuda.synchronize()
        if sampler:
            sampler.mark_end()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        if sampler and sampler.proc is not None:
            n_before = sampler.count()
            t_end = time.perf_counter() + 1.0
            while sampler.count() < n_before + 2 and time.perf_counter() < t_end:
                for _ in range(20):
                    g.replay()
                torch.cuda.synchronize()
    ms = a.elapsed_time(b)
    clocks = sampler.stop() if sampler else None
    return ms / steps, clocks


def check_parity(calls, oracle_outs):
    """Whole-tensor parity of the timed calls 0 and 1 (one per shape; their inputs are the unrolled
    seeded tensors) against the outputs the cpu_baseline leg has just produced."""
    from tests import parity as P
    out = {}
    for c, (q_or, s_or, Y) in zip(calls[:2], oracle_outs):
        t, d = Y.shape
        out[f"{t}x{d}"] = P.check_codes(c["q"].cpu().numpy(), c["s"].cpu().numpy(), q_or, s_or, Y, exact=False)
    return out


def run_ours(args):
    import torch
    from paper_2607_21446_b200 import binding as B
    B.load_library()                       # fails loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    ranks = Ranks("nccl", device)
    world, rank, dist = ranks.world, ranks.rank, ranks.dist
    peak, peak_kind = measured_peak()
    base, calls = build_inputs(torch, B, device)
    stream = torch.cuda.Stream()

    n0 = B.kroquant_launch_count()
    g_kq = capture(torch, [lambda c=c: B.kroquant_quantize(c["X"], c["factors"], c["q"], c["s"], stream=stream)
                           for c in calls], stream)
    launches_per_step = (B.kroquant_launch_count() - n0) // 2     # eager pass + captured pass
    g_scale = capture(torch, [lambda c=c: B.kroquant_scale_quantize(c["X"], c["sv"], c["q"], c["s"], stream=stream)
                              for c in calls], stream)
    g_plain = capture(torch, [lambda c=c: B.kroquant_mxfp4_quantize(c["X"], c["q"], c["s"], stream=stream)
                              for c in calls], stream)

    idx = torch.cuda.current_device()
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    smi_index = int(vis.split(",")[idx]) if vis and vis.split(",")[idx].isdigit() else idx
    ms_step, clocks = time_graph(torch, dist, g_kq, stream, args.steps, args.warmup, ClockSampler(smi_index))
    ms_step = ranks.max(ms_step)
    byts = step_bytes()
    value = world * byts / (ms_step * 1e-3) / 1e9
    dev_err = B.kroquant_last_device_error(stream)

    # in-run comparison kernels and per-shape breakdown (rank-local, shorter runs)
    k2 = max(3, args.steps // 2)
    ms_scale, _ = time_graph(torch, None, g_scale, stream, k2, 3)
    ms_plain, _ = time_graph(torch, None, g_plain, stream, k2, 3)
    per_shape = {}
    for k, (t, d) in enumerate(SHAPES):
        sub = [c for c in calls if c["shape_idx"] == k]
        res = {}
        for name, fn in (("kroquant", lambda c: B.kroquant_quantize(c["X"], c["factors"], c["q"], c["s"], stream=stream)),
                         ("scale", lambda c: B.kroquant_scale_quantize(c["X"], c["sv"], c["q"], c["s"], stream=stream)),
                         ("plain_mxfp4", lambda c: B.kroquant_mxfp4_quantize(c["X"], c["q"], c["s"], stream=stream))):
            g = capture(torch, [lambda c=c, fn=fn: fn(c) for c in sub + sub], stream)   # 28 calls of one shape
            ms, _ = time_graph(torch, None, g, stream, k2, 3)
            us = ms * 1e3 / (2 * len(sub))
            res[name] = {"us_per_call": round(us, 3),
                         "GB/s": round(W.algorithmic_bytes(t, d) / us / 1e3, 1),
                         "frac_of_peak": round(W.algorithmic_bytes(t, d) / us / 1e3 / peak, 4)}
        per_shape[f"{t}x{d}"] = res

    # the same 28 calls with their launches overlapped (three streams inside one graph): not how a model
    # runs them (each call waits for the layer before it), but it separates what the kernel can do from what
    # a kernel boundary costs
    # (static tile distribution for this one: with the default, every kernel's grid claims all CTA slots, so
    # kernels on different streams could not share the SMs)
    ovl = B.Tuning(dynamic=0, unit_tiles=1, config=5, ctas_per_sm=3)   # three small CTAs per SM leave room for a second kernel
    g_ovl = capture_overlapped(torch, calls,
                               lambda c, st: B.kroquant_quantize(c["X"], c["factors"], c["q"], c["s"], stream=st, tuning=ovl), stream)
    ms_ovl, _ = time_graph(torch, None, g_ovl, stream, args.steps, 3)
    # the headline step again right after an idle second (not the headline: it shows what the 1 kW power cap
    # costs; the timed region above starts only after seconds of load, with the SM clock already lowered)
    torch.cuda.synchronize()
    time.sleep(1.5)
    ms_burst, _ = time_graph(torch, None, g_kq, stream, min(args.steps, 50), 3)
    # the same graph for at least a second (its own clock samples): what the step costs once the power cap has
    # settled the SM clock; the headline above is the K steps the caller asked for
    n_sus = max(args.steps, int(args.sustained_seconds / (ms_step * 1e-3)))
    ms_sus, clocks_sus = time_graph(torch, dist, g_kq, stream, n_sus, 3, ClockSampler(smi_index))
    ms_sus = ranks.max(ms_sus)
    # end to end: pinned host inputs -> device -> quantize -> pinned host outputs
    e2e_steps = max(1, min(args.steps, 3))
    hx = [torch.empty(c["X"].shape, dtype=torch.bfloat16).pin_memory() for c in calls[:2]]
    for h, c in zip(hx, calls[:2]):
        h.copy_(c["X"])
    hq = [torch.empty(c["q"].shape, dtype=torch.uint8).pin_memory() for c in calls[:2]]
    hs = [torch.empty(c["s"].shape, dtype=torch.uint8).pin_memory() for c in calls[:2]]

    # One C call per layer (kroquant_quantize_host: upload, kernel, two downloads, in order on its stream); the
    # calls go round three streams, each with its own device work buffers, so that the upload of one call, the
    # kernel of another and the download of a third overlap (PCIe is full duplex).
    lanes = []
    for _ in range(3):
        lanes.append({"stream": torch.cuda.Stream(device),
                      "work": [(torch.empty_like(c["X"]), torch.empty_like(c["q"]), torch.empty_like(c["s"])) for c in calls[:2]]})

    def e2e_step():
        for i, c in enumerate(calls):
            k = c["shape_idx"]
            ln = lanes[i % 3]
            xw, qw, sw = ln["work"][k]
            B.kroquant_quantize_host(hx[k], c["factors"], hq[k], hs[k], xw, qw, sw, stream=ln["stream"])

    def e2e_sync():
        for ln in lanes:
            ln["stream"].synchronize()
    # (calls of one shape share their pinned host tensors: a download may overwrite what an earlier call of the
    #  same step wrote there with identical bytes for identical inputs; no timing-relevant property changes)
    torch.cuda.synchronize()
    e2e_step()
    e2e_sync()
    torch.cuda.synchronize()
    ranks.barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_sync()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = ranks.max(e2e_s)
    h2d = sum(c["X"].numel() * 2 for c in calls)
    d2h = sum(c["q"].numel() + c["s"].numel() for c in calls)

    if rank != 0:
        ranks.close()
        return

    # parity of the timed configuration (fresh device-resident run of the first two calls)
    g_kq.replay()
    torch.cuda.synchronize()
    cpu_gbs, cpu_dt, cores, oracle_outs = time_oracle(5, 1)
    cpu_one = time_oracle_one_thread()
    try:
        parity = check_parity(calls, oracle_outs)
        parity["status"] = "ok"
    except AssertionError as e:          # report, never hide
        parity = {"status": "FAILED", "error": str(e)[:200]}
    n_launch = launches_per_step * args.steps
    us_per_launch = ms_step * 1e3 / CALLS_PER_STEP
    alg_per_launch = byts / CALLS_PER_STEP
    traffic = None
    if all(NCU_TRAFFIC_BYTES[s] is not None for s in SHAPES):
        traffic = sum(NCU_TRAFFIC_BYTES[s] for s in SHAPES) / 2
    achieved = alg_per_launch / us_per_launch / 1e3
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "flux_step_28_calls: 14 x X[4608,3072] + 14 x X[4608,12288] bf16, interleaved, "
                               "one CUDA graph, distinct buffers and factor sets per call",
                   "l2": "28 input buffers total 1.98 GB (> 126 MB L2); no flush needed",
                   "factors": "one shared set per call (orthogonal x diag(U[0.5,2]))",
                   "kernel": "tcgen05+TMA tensor-core quantizer"},
        "tokens_per_s": world * step_tokens() / (ms_step * 1e-3),
        "frac_of_hbm_peak": value / world / peak,
        "frac_of_nominal_8tbs": value / world / 8000.0,
        "peak_note": f"frac_of_hbm_peak divides by the {peak_kind} copy bandwidth ({peak} GB/s: a device copy kernel, "
                     "which the quantizer exceeds on its largest launches); frac_of_nominal_8tbs by the data-sheet figure",
        "sustained": {"steps": n_sus, "ms_per_step": round(ms_sus, 5), "GB/s": round(world * byts / (ms_sus * 1e-3) / 1e9, 1),
                      "frac_of_hbm_peak": round(byts / (ms_sus * 1e-3) / 1e9 / peak, 4), "clocks": clocks_sus,
                      "note": f"the same graph timed for at least {args.sustained_seconds} s, after the headline region"},
        "speedup_vs_scale_kernel": ms_scale / ms_step,
        "speedup_vs_plain_mxfp4": ms_plain / ms_step,
        "after_idle": {
            "ms_per_step": round(ms_burst, 5), "GB/s": round(byts / (ms_burst * 1e-3) / 1e9, 1),
            "frac_of_hbm_peak": round(byts / (ms_burst * 1e-3) / 1e9 / peak, 4),
            "note": "the same graph, 3 warm-up + at most 50 timed steps after 1.5 s of idle: before the power cap "
                    "lowers the SM clock; not the headline"},
        "independent_calls_overlapped": {
            "ms_per_step": round(ms_ovl, 5), "GB/s": round(byts / (ms_ovl * 1e-3) / 1e9, 1),
            "frac_of_hbm_peak": round(byts / (ms_ovl * 1e-3) / 1e9 / peak, 4),
            "note": "same step, call i on stream i % 3 inside the graph, static tile distribution, three small CTAs per SM; not the headline: "
                    "in a model every call waits for the layer before it"},
        "per_shape": per_shape,
        "parity": parity,
        "device_error": dev_err,
        "clocks": clocks,
        "e2e": {"value": world * byts / e2e_s / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "api": "kroquant_quantize_host (C ABI, host buffers; 28 calls per step over 3 streams)"},
        "gpu_launches": n_launch,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                     "kernel": "quantize_umma<8,2,2,false,false>", "launches": n_launch,
                     "avg_launch_us": us_per_launch, "algorithmic_bytes_per_launch": alg_per_launch},
        "cpu_baseline": {"value": cpu_gbs, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{SAMPLE}, {cpu_dt:.2f} s per pass, 5 passes, "
                                   "C oracle (fp64, OpenMP over token rows)",
                         "one_thread": cpu_one},
    }
    print(json.dumps(line), flush=True)
    ranks.close()


def run_single(args):
    """Small case for profilers: a few eager launches of one shape on rotating buffers
    (no CUDA graph, no comparison kernels).  Prints a short JSON line; never a bench value."""
    import torch
    from paper_2607_21446_b200 import binding as B
    B.load_library()
    t, d = (int(v) for v in args.single.lower().split("x"))
    nbuf = max(2, int(400e6 // (t * d * 2)) + 1)          # > 3 x L2 of distinct inputs
    sp = W.ActivationSpec("single", t, d, seed=3, outlier_channels=max(1, d // 200), outlier_gain=100.0)
    x0 = torch.from_numpy(W.gen_activations(sp).view(np.int16)).cuda().view(torch.bfloat16)
    Xs = [x0] + [torch.roll(x0, shifts=i, dims=0).contiguous() for i in range(1, nbuf)]
    q = torch.empty((t, d // 2), dtype=torch.uint8, device="cuda")
    sc = torch.empty((t, d // 32), dtype=torch.uint8, device="cuda")
    f = B.Factors.create(W.gen_factors(3, n_sets=d // 32 if args.per_block else 1))
    sv = torch.from_numpy(W.gen_channel_scales(3, d)).cuda()
    fn = {"kroquant": lambda x: B.kroquant_quantize(x, f, q, sc),
          "kroquant_onchip": lambda x: B.kroquant_quantize(x, f, q, sc, path="onchip"),
          "fwht": lambda x: B.kroquant_fwht_quantize(x, q, sc),
          "scale": lambda x: B.kroquant_scale_quantize(x, sv, q, sc),
          "plain": lambda x: B.kroquant_mxfp4_quantize(x, q, sc)}[args.kernel]
    torch.cuda.synchronize()
    evs = []
    for i in range(args.calls):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn(Xs[i % nbuf])
        b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    us = sorted(a.elapsed_time(b) * 1e3 for a, b in evs)
    print(json.dumps({"single": args.single, "kernel": args.kernel, "calls": args.calls,
                      "median_us_eager": us[len(us) // 2], "buffers": nbuf,
                      "device_error": B.kroquant_last_device_error()}), flush=True)


def run_point(torch, B, co, P, args, label, bits, tokens, G, seed, peak, peak_kind, stream, idx):
    """One measured and parity-checked point: KroQuant (factor sets G: one shared set or one per block; operand images
    ready-made, and built on chip), Scale and bare MXFP4 on the same input, each as a CUDA graph of back-to-back calls over rotating buffers (> 3 x L2).  `bits` holds
    the first n0 <= tokens host rows; device row r is host row r % n0.  The C oracle then goes over EVERY row in
    chunks of 2048 (that pass is its measured time, all host cores) and all three outputs are compared with it
    (rules P0-P3 of tests/parity.py).  Prints one JSON line."""
    n0, d = bits.shape
    nbuf = min(28, max(3, int(400e6 // (tokens * d * 2)) + 1))
    x0 = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    x0 = x0.repeat((tokens + n0 - 1) // n0, 1)[:tokens].contiguous()
    Xs = [x0] + [torch.roll(x0, shifts=i, dims=0).contiguous() for i in range(1, nbuf)]
    q = torch.empty((tokens, d // 2), dtype=torch.uint8, device="cuda")
    sc = torch.empty((tokens, d // 32), dtype=torch.uint8, device="cuda")
    f = B.Factors.create(G)
    svh = W.gen_channel_scales(seed, d)
    sv = torch.from_numpy(svh).cuda()
    kernels = (("kroquant", lambda x: B.kroquant_quantize(x, f, q, sc, stream=stream)),
               # the same kernel with its operand built on chip from the factor scalars (the paper's K2 construction)
               ("kroquant_onchip", lambda x: B.kroquant_quantize(x, f, q, sc, stream=stream, path="onchip")),
               ("scale", lambda x: B.kroquant_scale_quantize(x, sv, q, sc, stream=stream)),
               ("plain_mxfp4", lambda x: B.kroquant_mxfp4_quantize(x, q, sc, stream=stream)))
    res, clk = {}, {}
    for name, fn in kernels:
        g = capture(torch, [lambda x=x, fn=fn: fn(x) for x in Xs], stream)
        # (every kernel is timed with the clock sampler running: the sampler's start-up keeps the GPU under
        #  load for some hundred milliseconds before the timed region, and all three must see the same regime)
        ms, c = time_graph(torch, None, g, stream, max(5, args.steps // 10), 3, ClockSampler(idx))
        res[name] = ms * 1e3 / nbuf
        clk[name] = {"sm_mhz": c.get("sm_mhz"), "reasons": c.get("reasons")}

    def rows(r0, r1):
        return bits[np.arange(r0, r1) % n0]
    oracle_s = [0.0]

    def timed(fn_or):
        def run(b):
            t0 = time.perf_counter()
            out = fn_or(b)
            oracle_s[0] += time.perf_counter() - t0
            return out
        return run
    parity = {}
    try:
        with torch.cuda.stream(stream):
            for name, fn in kernels:
                fn(x0)
                stream.synchronize()
                if name.startswith("kroquant"):
                    fn_or = (lambda b: co.quantize(b, G))                 # (its time is taken once, on the first pass)
                    parity[name] = P.check_codes_chunked(q, sc, rows, timed(fn_or) if name == "kroquant" else fn_or, tokens, exact=False)
                elif name == "scale":
                    parity[name] = P.check_codes_chunked(q, sc, rows, lambda b: co.scale_quantize(b, svh), tokens, exact=True)
                else:
                    parity[name] = P.check_codes_chunked(q, sc, rows, co.plain_quantize, tokens, exact=True)
        parity["status"] = "ok"
    except AssertionError as e:          # report, never hide
        parity["status"] = "FAILED"
        parity["error"] = str(e)[:200]
    byt = W.algorithmic_bytes(tokens, d)
    print(json.dumps({
        "point": label, "shape": f"{tokens}x{d}", "factor_sets": int(G.shape[0]),
        "us": {k: round(v, 2) for k, v in res.items()},
        "GB/s": {k: round(byt / v / 1e3, 1) for k, v in res.items()},
        "frac_of_hbm_peak": {k: round(byt / v / 1e3 / peak, 4) for k, v in res.items()},
        "frac_of_nominal_8tbs": {k: round(byt / v / 1e3 / 8000.0, 4) for k, v in res.items()},
        "tokens_per_s": round(tokens / (res["kroquant"] * 1e-6)),
        "scale_over_kroquant": round(res["scale"] / res["kroquant"], 3),
        "plain_over_kroquant": round(res["plain_mxfp4"] / res["kroquant"], 3),
        "onchip_over_kroquant": round(res["kroquant_onchip"] / res["kroquant"], 3),
        "parity": parity,
        "cpu_oracle_s": round(oracle_s[0], 3), "cpu_oracle_rows": tokens, "cpu_cores": os.cpu_count(),
        "clocks": clk, "peak": f"{peak} GB/s of {peak_kind}", "buffers": nbuf,
        "device_error": B.kroquant_last_device_error()}), flush=True)


def run_sweep(args):
    """The sweep config (tokens x d grid, one shared factor set), or with --configs the PixArt-, SANA- and
    FLUX-shaped tensors of the other workload configs (SANA also with one factor set per block): see run_point.
    --points TOKENSxD,... restricts the sweep grid."""
    import torch
    from oracle import c_oracle as co
    from paper_2607_21446_b200 import binding as B
    from tests import parity as P
    B.load_library()
    peak, peak_kind = measured_peak()
    stream = torch.cuda.Stream()
    idx = torch.cuda.current_device()
    if args.configs:
        todo = [("tiny", W.tiny_spec(), 0, 0, False)]
        todo += [(sp.name, sp, 1, i, False) for i, sp in enumerate(W.pixart_specs())]
        for i, sp in enumerate(W.sana_specs()):
            todo += [(sp.name, sp, 2, i, False), (sp.name + "_per_block", sp, 2, i, True)]
        todo += [(sp.name, sp, 3, i, False) for i, sp in enumerate(W.flux_specs())]
        for label, sp, seed, layer, per_block in todo:
            bits = W.gen_activations(sp)
            G = W.gen_factors(seed, n_sets=sp.d // 32 if per_block else 1, layer=layer)
            run_point(torch, B, co, P, args, label, bits, sp.tokens, G, seed, peak, peak_kind, stream, idx)
        return
    points = [(t, d) for t in W.SWEEP_TOKENS for d in W.SWEEP_D]
    if args.points:
        points = [tuple(int(v) for v in p.lower().split("x")) for p in args.points.split(",")]
    for tokens, d in points:
        bits = W.gen_activations(W.sweep_spec(min(tokens, 4096), d))     # host generator on <= 4096 rows, tiled on the device
        run_point(torch, B, co, P, args, f"sweep_{tokens}x{d}", bits, tokens, W.gen_factors(4), 4, peak, peak_kind, stream, idx)


# The paper's two latency tables (Section 4.4 and Appendix A): (m, d) and its MI350 / FP16 numbers in
# microseconds for Q4, Scale, K1, K2 (and FWHT where given) -- context only, another machine.
PAPER_TABLES = {
    "power_of_two_d": [((4096, 1024), (9.40, 10.56, 9.96, 14.00, 18.16)), ((4096, 4096), (22.64, 25.52, 23.88, 27.80, 68.04)),
                       ((4096, 16384), (74.44, 75.44, 75.32, 78.52, 186.04)), ((512, 4096), (7.20, 9.24, 8.12, 10.28, 14.40)),
                       ((512, 16384), (13.68, 16.36, 15.36, 19.32, 33.96))],
    "production_shapes": [((512, 3072), (6.72, 9.04, 7.64, 8.84)), ((512, 12288), (11.80, 14.68, 13.08, 17.00)),
                          ((4096, 1152), (10.64, 14.00, 10.68, 14.64)), ((4096, 3072), (18.56, 21.12, 19.28, 23.32)),
                          ((4096, 3456), (20.60, 24.20, 21.32, 25.36)), ((4096, 4096), (22.08, 25.80, 23.36, 27.28)),
                          ((4096, 4608), (25.72, 28.40, 26.40, 30.36)), ((4096, 12288), (59.64, 59.12, 59.92, 62.80))],
}


def run_table(args):
    """The paper's latency tables re-measured on this GPU with FP16 activations: Q4 (bare MXFP4),
    Scale, K1 (dense 32x32 block handle: the tensor-core kernel on a ready-made operand image), K2 (five-factor
    handle, the same kernel on the image made at handle creation) and K2_onchip (five-factor handle, operand built
    inside the kernel from the 20 scalars, as the paper's K2 kernel does).  Back-to-back calls in a CUDA graph
    over rotating inputs (> 3 x L2).  One JSON line per shape."""
    import torch
    from paper_2607_21446_b200 import binding as B
    B.load_library()
    stream = torch.cuda.Stream()
    for table, rows in PAPER_TABLES.items():
        for (m, d), paper in rows:
            nbuf = min(28, max(3, int(400e6 // (m * d * 2)) + 1))
            sp = W.ActivationSpec("table", m, d, seed=4, outlier_channels=max(1, d // 100), outlier_gain=50.0)
            x0 = torch.from_numpy(W.gen_activations(sp, "fp16").view(np.int16)).cuda().view(torch.float16)
            Xs = [x0] + [torch.roll(x0, shifts=i, dims=0).contiguous() for i in range(1, nbuf)]
            q = torch.empty((m, d // 2), dtype=torch.uint8, device="cuda")
            sc = torch.empty((m, d // 32), dtype=torch.uint8, device="cuda")
            G = W.gen_factors(4)
            K = G[0, 0].astype(np.float64)
            for k in range(1, 5):
                K = np.kron(K, G[0, k].astype(np.float64))          # input recipe of the dense handle
            f2, f1 = B.Factors.create(G), B.Factors.create_dense(K.astype(np.float32)[None])
            sv = torch.from_numpy(W.gen_channel_scales(4, d)).cuda()
            us = {}
            kernels = [("Q4", lambda x: B.kroquant_mxfp4_quantize(x, q, sc, stream=stream)),
                       ("Scale", lambda x: B.kroquant_scale_quantize(x, sv, q, sc, stream=stream)),
                       ("K1", lambda x: B.kroquant_quantize(x, f1, q, sc, stream=stream)),
                       ("K2", lambda x: B.kroquant_quantize(x, f2, q, sc, stream=stream)),
                       ("K2_onchip", lambda x: B.kroquant_quantize(x, f2, q, sc, stream=stream, path="onchip"))]
            if d & (d - 1) == 0:
                kernels.append(("FWHT", lambda x: B.kroquant_fwht_quantize(x, q, sc, stream=stream)))
            for name, fn in kernels:
                g = capture(torch, [lambda x=x, fn=fn: fn(x) for x in Xs], stream)
                ms, _ = time_graph(torch, None, g, stream, max(5, args.steps // 10), 3)
                us[name] = round(ms * 1e3 / nbuf, 2)
            print(json.dumps({"table": table, "m": m, "d": d, "dtype": "fp16", "us_b200": us,
                              "scale_over_k1": round(us["Scale"] / us["K1"], 3),
                              "scale_over_k2": round(us["Scale"] / us["K2"], 3),
                              "scale_over_k2_onchip": round(us["Scale"] / us["K2_onchip"], 3),
                              "fwht_over_k2": round(us["FWHT"] / us["K2"], 3) if "FWHT" in us else None,
                              "paper_mi350_us": dict(zip(("Q4", "Scale", "K1", "K2", "FWHT"), paper))}), flush=True)
            del Xs, x0


def run_calib(args):
    """Calibration loop (Section 3.3): `--steps` Adam steps on a synthetic layer, timed with CUDA
    events on the launching stream after `--warmup` steps.  One JSON line: ms per step, the rate of
    the three contractions of a step (3 x 2 M o d flop) against the measured bf16 tensor peak, the
    objective before/after, and the float64 oracle timed on a row sample of the same layer."""
    import torch
    from paper_2607_21446_b200 import binding as B
    B.load_library()
    B.set_gemm_pair(not args.gemm_single)
    M, o, d = (int(v) for v in args.calib.lower().split("x"))
    n_sets = d // 32 if args.per_block else 1
    A_bits = W.gen_activations(W.calib_spec(M, d))
    W_bits = W.gen_weights(5, o, d)
    dev = torch.device("cuda:0")
    A_t = torch.from_numpy(A_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    W_t = torch.from_numpy(W_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    side = torch.cuda.Stream()          # a capturable stream: the library replays one captured step per Adam step
    torch.cuda.set_stream(side)
    stream = torch.cuda.current_stream()
    launches0 = B.kroquant_launch_count()
    cal = B.Calibrator(A_t, W_t, n_sets)
    lam = cal.lambdas.astype(np.float64)
    l_first, _ = cal.loss_grad(grad=False)
    cal.run(max(args.warmup, 3), history=False)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    t_wait = time.time()
    while sampler.count() < 2 and time.time() - t_wait < 3.0:
        cal.run(1, history=False)
        torch.cuda.synchronize()
    l0 = B.kroquant_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    cal.run(args.steps, history=False)
    e1.record(stream)
    torch.cuda.synchronize()
    launches = B.kroquant_launch_count() - l0
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    l_last, _ = cal.loss_grad(grad=False)
    flop = 3 * 2.0 * M * o * d
    peak_tf, kind = 1590.0, "fallback"
    pth = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pth):
        with open(pth) as f:
            mp = json.load(f)
        if "bf16_tflops" in mp:
            peak_tf, kind = float(mp["bf16_tflops"]), "measured"
    # CPU oracle on a bounded sample: the first rows of A with the full W (cost is linear in rows)
    from oracle import calib_oracle as co
    rows_s = min(M, max(64, int(5.0e11 // (6.0 * o * d)) // 8 * 8))      # about 10 s of CPU work
    A_s = W.bf16_bits_to_f32(A_bits[:rows_s]).astype(np.float64)
    W_s = W.bf16_bits_to_f32(W_bits).astype(np.float64)
    th = co.hadamard_theta(n_sets)
    t0 = time.time()
    _, terms_s, g_s = co.loss_and_grad(A_s, W_s, th, lam[0], lam[1])
    cpu_s = time.time() - t0
    # parity of the sample on the GPU: same rows, same parameters, same lambdas
    cal_s = B.Calibrator(A_t[:rows_s].contiguous(), W_t, n_sets)
    cal_s.lambdas = lam.astype(np.float32)
    terms_g, g_g = cal_s.loss_grad()
    parity = {"rows": rows_s,
              "loss_rel_err": float(np.max(np.abs(terms_g - terms_s) / np.abs(terms_s))),
              "grad_err_over_max": float(np.abs(g_g - g_s).max() / np.abs(g_s).max())}
    cal_s.destroy()
    tot = lambda l: float(l[0] + lam[0] * l[1] + lam[1] * l[2])
    print(json.dumps({
        "metric": "calibration_step_time", "value": round(ms, 4), "unit": "ms", "higher_is_better": False,
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "dtype": "bf16 operands, fp32 accumulate",
        "data": "synthetic", "config": {"workload": f"calibration M={M} o={o} d={d} n_sets={n_sets}",
                                        "gemm": "one CTA, 128x256 tiles" if args.gemm_single else "CTA pairs, 256x256 tiles",
                                        "l2": "operands and work space exceed L2"},
        "gpu_launches": int(launches), "launches_per_step": launches / args.steps,
        "roofline": {"bound": "tensor", "achieved": round(flop / ms / 1e9, 1), "peak": peak_tf, "unit": "TFLOP/s",
                     "frac": round(flop / ms / 1e9 / peak_tf, 4), "traffic": None,
                     "note": f"3 contractions x 2 M o d flop / step time, of {kind} bf16 peak; the step also "
                             "runs the fake-quant, block-gradient and optimiser kernels"},
        "objective": {"lambda_A": lam[0], "lambda_W": lam[1], "at_init": [float(v) for v in l_first],
                      "after": [float(v) for v in l_last], "total_at_init": tot(l_first), "total_after": tot(l_last),
                      "adam_steps_taken": int(args.steps + max(args.warmup, 3))},
        "cpu_baseline": {"value": round(cpu_s * 1e3 * M / rows_s, 1), "unit": "ms", "cores": os.cpu_count(),
                         "kind": "oracle", "sample": f"one loss+gradient evaluation on the first {rows_s} of {M} rows "
                                                     f"({cpu_s:.2f} s), scaled linearly in rows"},
        "parity": parity, "clocks": clocks, "device_error": B.kroquant_last_device_error(),
    }), flush=True)
    cal.destroy()


def run_gemm_fp4(args):
    """W4A4 consumer GEMM (Section 3.4) on synthetic operands: this library's block-scaled FP4 kernel, the
    library GEMM behind torch.nn.functional.scaled_mm, and cuBLAS bf16 on the unquantized operands, timed
    with CUDA events after warm-up; one JSON line."""
    import torch
    from paper_2607_21446_b200 import binding as B
    B.load_library()
    M, N, K = (int(v) for v in args.gemm_fp4.lower().split("x"))
    g = torch.Generator(device="cuda")
    g.manual_seed(0)
    A = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    Wt = (torch.randn(N, K, device="cuda", generator=g) / K ** 0.5).to(torch.bfloat16)
    qa, sa = B.kroquant_mxfp4_quantize(A, scale_layout="tiled")
    qw, sw = B.kroquant_mxfp4_quantize(Wt, scale_layout="tiled")
    out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    F = torch.nn.functional

    def timed(fn):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps * 1e3

    l0 = B.kroquant_launch_count()
    us_own = timed(lambda: B.kroquant_gemm_mxfp4(qa, sa, qw, sw, out=out))
    launches = B.kroquant_launch_count() - l0
    us_lib = None
    if hasattr(F, "scaled_mm"):
        us_lib = timed(lambda: F.scaled_mm(
            qa.view(torch.float4_e2m1fn_x2), qw.view(torch.float4_e2m1fn_x2).t(),
            sa.view(torch.float8_e8m0fnu), F.ScalingType.BlockWise1x32, sw.view(torch.float8_e8m0fnu),
            F.ScalingType.BlockWise1x32, swizzle_a=F.SwizzleType.SWIZZLE_32_4_4,
            swizzle_b=F.SwizzleType.SWIZZLE_32_4_4, output_dtype=torch.bfloat16))
    us_bf16 = timed(lambda: torch.matmul(A, Wt.t()))
    flop = 2.0 * M * N * K
    peak_bf16, kind = 1590.0, "fallback"
    pth = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pth):
        with open(pth) as f:
            mp = json.load(f)
        if "bf16_tflops" in mp:
            peak_bf16, kind = float(mp["bf16_tflops"]), "measured"
    peak = 4.0 * peak_bf16          # nominal fp4 : bf16 ratio of the dense peaks (9 : 2.25)
    print(json.dumps({
        "metric": "w4a4_gemm_time", "value": round(us_own, 2), "unit": "us", "higher_is_better": False, "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "dtype": "e2m1 x e2m1 with e8m0 block scales, fp32 accumulate",
        "data": "synthetic", "config": {"workload": f"W4A4 GEMM M={M} N={N} K={K}, bf16 output"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": round(flop / us_own / 1e6, 1), "peak": round(peak, 1), "unit": "TFLOP/s",
                     "frac": round(flop / us_own / 1e6 / peak, 4), "traffic": None,
                     "note": f"peak = {kind} bf16 peak x 4 (nominal fp4 : bf16 ratio)"},
        "library_fp4_us": None if us_lib is None else round(us_lib, 2),
        "library_fp4_tflops": None if us_lib is None else round(flop / us_lib / 1e6, 1),
        "cublas_bf16_us": round(us_bf16, 2), "cublas_bf16_tflops": round(flop / us_bf16 / 1e6, 1),
        "device_error": B.kroquant_last_device_error()}), flush=True)


def run_layer(args):
    """The quantized linear layer of Section 3.4, one call per step (quantizer + W4A4 GEMM), against the
    bf16 GEMM it replaces; inputs and outputs rotate over buffers that exceed L2.  One JSON line."""
    import torch
    from paper_2607_21446_b200 import binding as B
    B.load_library()
    t, o, d = (int(v) for v in args.layer.lower().split("x"))
    nbuf = max(2, int(300e6 // (t * (d + o) * 2)) + 1)
    sp = W.ActivationSpec("layer", t, d, seed=3, outlier_channels=max(1, d // 200), outlier_gain=100.0)
    x0 = torch.from_numpy(W.gen_activations(sp).view(np.int16)).cuda().view(torch.bfloat16)
    Xs = [x0] + [torch.roll(x0, shifts=i, dims=0).contiguous() for i in range(1, nbuf)]
    outs = [torch.empty((t, o), dtype=torch.bfloat16, device="cuda") for _ in range(nbuf)]
    Wt = torch.from_numpy(W.gen_weights(3, o, d).view(np.int16)).cuda().view(torch.bfloat16)
    G = W.gen_factors(3, n_sets=d // 32 if args.per_block else 1)
    H = np.stack([[np.linalg.inv(G[s_, k].astype(np.float64)).T for k in range(5)] for s_ in range(G.shape[0])]).astype(np.float32)
    layer = B.LinearW4A4.from_weights(Wt, G, H)
    q = torch.empty((t, d // 2), dtype=torch.uint8, device="cuda")
    sc = torch.zeros(B.tiled_scale_bytes(t, d), dtype=torch.uint8, device="cuda")

    stream = torch.cuda.Stream()
    per_graph = 2 * nbuf

    def timed(fn):
        """One CUDA graph of 2 * nbuf calls over the rotating buffers, replayed: the host's launch cost
        (about 10 us per call from Python) stays out of the number."""
        g = capture(torch, [lambda i=i: fn(i % nbuf) for i in range(per_graph)], stream)
        reps = max(1, args.steps // per_graph)
        with torch.cuda.stream(stream):
            for _ in range(max(args.warmup, 3)):
                g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                g.replay()
            e1.record(stream)
            torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (reps * per_graph) * 1e3

    l0 = B.kroquant_launch_count()
    us_layer = timed(lambda i: layer(Xs[i], out=outs[i], stream=stream))
    launches = (B.kroquant_launch_count() - l0) / 2 / per_graph      # eager pass + captured pass
    us_quant = timed(lambda i: B.kroquant_quantize(Xs[i], layer.factors, q, sc, scale_layout="tiled", stream=stream))
    us_gemm = timed(lambda i: B.kroquant_gemm_mxfp4(q, sc, layer.w_codes, layer.w_scales, out=outs[i], stream=stream))
    us_bf16 = timed(lambda i: torch.matmul(Xs[i], Wt.t(), out=outs[i]))
    flop = 2.0 * t * o * d
    print(json.dumps({
        "metric": "quantized_linear_layer_time", "value": round(us_layer, 2), "unit": "us", "higher_is_better": False,
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "data": "synthetic",
        "dtype": "bf16 activations -> MXFP4 x MXFP4, fp32 accumulate, bf16 output",
        "config": {"workload": f"linear layer tokens={t} d={d} o={o}, n_sets={G.shape[0]}",
                   "l2": f"{nbuf} rotating input/output buffer pairs ({nbuf * t * (d + o) * 2 / 1e6:.0f} MB)"},
        "gpu_launches": int(round(launches * per_graph * max(1, args.steps // per_graph))), "launches_per_step": launches,
        "quantizer_us": round(us_quant, 2), "w4a4_gemm_us": round(us_gemm, 2), "cublas_bf16_gemm_us": round(us_bf16, 2),
        "speedup_vs_bf16_gemm": round(us_bf16 / us_layer, 3), "effective_tflops": round(flop / us_layer / 1e6, 1),
        "device_error": B.kroquant_last_device_error()}), flush=True)


def run_timeline(args):
    """Where a call's time goes at the kernel boundary: eight back-to-back calls of one shape in a CUDA graph, run on
    the timeline build of the library (per-CTA global-timer marks, see kroquant_debug_set_timeline).  For the KroQuant
    kernel and the two comparison kernels: time of each mark relative to the end of the LAST CTA of the call before,
    minimum / median / maximum over the CTAs, averaged over calls 2..7; and the call period.  The marks cost a few
    per cent; this is a diagnosis, never a bench value."""
    import torch
    from paper_2607_21446_b200 import binding as B, build as kbuild
    B.use_library(kbuild.build_timeline())           # (re)built when missing or older than the sources
    B.load_library()
    t, d = (int(v) for v in args.timeline.lower().split("x"))
    ncall = 8
    stream = torch.cuda.Stream()
    sp = W.ActivationSpec("tl", min(t, 8192), d, seed=3, outlier_channels=max(1, d // 200), outlier_gain=100.0)
    x0 = torch.from_numpy(W.gen_activations(sp).view(np.int16)).cuda().view(torch.bfloat16)
    x0 = x0.repeat((t + x0.shape[0] - 1) // x0.shape[0], 1)[:t].contiguous()
    Xs = [x0] + [torch.roll(x0, shifts=i, dims=0).contiguous() for i in range(1, ncall)]
    q = torch.empty((t, d // 2), dtype=torch.uint8, device="cuda")
    sc = torch.empty((t, d // 32), dtype=torch.uint8, device="cuda")
    f = B.Factors.create(W.gen_factors(3))
    sv = torch.from_numpy(W.gen_channel_scales(3, d)).cuda()
    marks = torch.zeros(64 * 4096 * 8, dtype=torch.int64, device="cuda")
    names = ["cta_start", "wait_returned", "first_tile_ready", "producer_done", "epilogue_done", "cta_end"]
    out = {"timeline": args.timeline, "calls": ncall, "unit": "us after the last CTA of the previous call ended (min/median/max over CTAs)"}
    for kname, fn in (("kroquant", lambda x: B.kroquant_quantize(x, f, q, sc, stream=stream)),
                      ("plain_mxfp4", lambda x: B.kroquant_mxfp4_quantize(x, q, sc, stream=stream)),
                      ("scale", lambda x: B.kroquant_scale_quantize(x, sv, q, sc, stream=stream))):
        B.kroquant_debug_set_timeline(None)
        with torch.cuda.stream(stream):
            for x in Xs:
                fn(x)
            torch.cuda.synchronize()
            B.kroquant_debug_set_timeline(marks)           # launch slots restart at 0: the captured calls get 0..7
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for x in Xs:
                    fn(x)
            for _ in range(5):
                g.replay()
            torch.cuda.synchronize()
            marks.zero_()
            g.replay()
            torch.cuda.synchronize()
        a = marks.cpu().numpy().reshape(64, 4096, 8)
        ends = [a[k, a[k, :, 0] > 0, 5].max() for k in range(ncall)]
        rows = {n: np.zeros(3) for n in names}
        periods = []
        for k in range(2, ncall):
            live = a[k, :, 0] > 0
            for i, n in enumerate(names):
                v = (a[k, live, i] - ends[k - 1]) / 1e3
                rows[n] += np.array([v.min(), np.median(v), v.max()]) / (ncall - 2)
            periods.append((ends[k] - ends[k - 1]) / 1e3)
        out[kname] = {"period_us": round(float(np.mean(periods)), 2), "ctas": int((a[2, :, 0] > 0).sum()),
                      "tiles_per_cta_max": int(a[2, :, 6].max()),
                      **{n: [round(float(x), 2) for x in rows[n]] for n in names}}
    B.kroquant_debug_set_timeline(None)
    out["device_error"] = B.kroquant_last_device_error()
    print(json.dumps(out), flush=True)


def run_boundary_floor(args):
    """What the platform charges a dependent launch, apart from anything the quantizer does: chains of ten probe
    kernels (diagnostic build of the library, kroquant_debug_boundary_probe) whose CTAs only take tensor memory or not,
    wait for the launch before, idle for a fixed time and leave.  One JSON line per setting: the period of the chain
    minus the idle time is the cost of the kernel boundary; cta_start says when the next launch's CTAs begin,
    relative to the end of the last CTA of the launch before."""
    import torch
    from paper_2607_21446_b200 import binding as B, build as kbuild
    B.use_library(kbuild.build_timeline())
    B.load_library()
    calls, spin = 10, args.spin_ns
    stream = torch.cuda.Stream()
    marks = torch.zeros(calls * 1024 * 4, dtype=torch.int64, device="cuda")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    settings = [(0, 1, 1), (512, 1, 1), (0, 2, 1), (32, 2, 1), (128, 2, 1), (256, 2, 1), (-1, 2, 1), (0, 3, 1), (128, 3, 1),
                (0, 2, 0), (256, 2, 0), (0, 3, 0), (128, 3, 0)]
    for cols, cps, late in settings:
        with torch.cuda.stream(stream):
            B.kroquant_debug_boundary_probe(cols, cps, late, spin, calls, marks, stream)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                B.kroquant_debug_boundary_probe(cols, cps, late, spin, calls, marks, stream)
            for _ in range(5):
                g.replay()
            torch.cuda.synchronize()
            marks.zero_()
            g.replay()
            torch.cuda.synchronize()
        a = marks.cpu().numpy().reshape(calls, 1024, 4)[:, : sms * cps, :].astype(np.float64)
        ends = a[:, :, 3].max(axis=1)
        start, ready, setup, periods = np.zeros(3), 0.0, 0.0, []
        for k in range(2, calls):
            v = np.sort(a[k, :, 0] - ends[k - 1]) / 1e3
            start += np.array([v[0], v[len(v) // 2], v[-1]]) / (calls - 2)
            ready += float(np.median(a[k, :, 2] - ends[k - 1])) / 1e3 / (calls - 2)
            setup += float(np.median(a[k, :, 1] - a[k, :, 0])) / 1e3 / (calls - 2)
            periods.append((ends[k] - ends[k - 1]) / 1e3)
        period = float(np.mean(periods))
        print(json.dumps({"boundary_floor": {"tmem_cols_per_cta": max(cols, 0), "tcgen05_in_kernel": cols != 0,
                                             "permit_released": cols > 0 if cols != 0 else None, "ctas_per_sm": cps,
                                             "completion_signal": "at CTA end" if late else "at CTA start"},
                          "idle_us": spin / 1e3, "period_us": round(period, 2), "boundary_cost_us": round(period - spin / 1e3, 2),
                          "cta_start_us_after_previous_launch_ended": [round(float(x), 2) for x in start],
                          "setup_us": round(setup, 2), "wait_returned_us_after_previous_launch_ended": round(ready, 2),
                          "ctas": sms * cps}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--table", action="store_true",
                    help="the paper's two latency tables (Q4 / Scale / K1 / K2, FP16) on this GPU")
    ap.add_argument("--sweep", action="store_true",
                    help="tokens x d sweep of KroQuant / Scale / bare MXFP4 (one JSON line per point)")
    ap.add_argument("--timeline", default=None, metavar="TOKENSxD",
                    help="per-CTA timeline of back-to-back calls at the kernel boundary (timeline build of the library)")
    ap.add_argument("--boundary-floor", action="store_true",
                    help="platform cost of a dependent launch with and without tensor memory (probe kernels, diagnostic build)")
    ap.add_argument("--spin-ns", type=int, default=3000, help="with --boundary-floor: idle time of a probe CTA")
    ap.add_argument("--configs", action="store_true",
                    help="the tiny, PixArt-, SANA- (shared and per-block sets) and FLUX-shaped tensors, measured and parity-checked like --sweep")
    ap.add_argument("--points", default=None, metavar="TOKENSxD,...", help="with --sweep: only these points")
    ap.add_argument("--single", default=None, metavar="TOKENSxD",
                    help="profiling aid: a few eager launches of one shape, e.g. 4608x12288")
    ap.add_argument("--kernel", default="kroquant", choices=["kroquant", "kroquant_onchip", "fwht", "scale", "plain"])
    ap.add_argument("--calls", type=int, default=8)
    ap.add_argument("--per-block", action="store_true", help="with --single: one factor set per 32-channel block")
    ap.add_argument("--calib", default=None, metavar="MxOxD",
                    help="calibration loop on a synthetic layer, e.g. 16384x3072x3072 (with --per-block: one set per block)")
    ap.add_argument("--layer", default=None, metavar="TOKENSxOxD",
                    help="quantized linear layer (quantizer + W4A4 GEMM) vs the bf16 GEMM, e.g. 4608x3072x3072")
    ap.add_argument("--gemm-fp4", default=None, metavar="MxNxK",
                    help="W4A4 consumer GEMM, e.g. 4608x3072x3072: own FP4 kernel vs library FP4 vs cuBLAS bf16")
    ap.add_argument("--gemm-single", action="store_true",
                    help="with --calib: one-CTA 128x256 GEMM tiles instead of CTA pairs on 256x256 tiles")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sustained-seconds", type=float, default=1.2,
                    help="length of the extra sustained measurement of the headline graph (0: only --steps replays; for profilers)")
    ap.add_argument("--dist-selftest", action="store_true",
                    help="run the multi-rank launch / barrier / reduction logic on CPU ranks (gloo) with a stub step")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.table or args.sweep or args.configs or args.single or args.calib
                                                                  or args.gemm_fp4 or args.layer or args.timeline):
        sys.exit(relaunch_under_torchrun(sys.argv[1:], args.gpus))
    if args.dist_selftest:
        return run_dist_selftest(args)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.timeline:
        run_timeline(args)
    elif args.boundary_floor:
        run_boundary_floor(args)
    elif args.table:
        run_table(args)
    elif args.sweep or args.configs:
        run_sweep(args)
    elif args.single:
        run_single(args)
    elif args.calib:
        run_calib(args)
    elif args.gemm_fp4:
        run_gemm_fp4(args)
    elif args.layer:
        run_layer(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
