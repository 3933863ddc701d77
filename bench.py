#!/usr/bin/env python
"""Benchmark of the SLiM compressed linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload: the LLaMA-2-70B decode layer set, the largest configuration that fits one GPU.  One
step = the seven linears of one transformer block (2 x 8192->8192, 2 x 8192->1024 grouped-query
k/v, 2 x 8192->28672, 1 x 28672->8192; int4 2:4 weights, per-layer fp32 scale, bf16 adapters of
rank 0.1 x the smaller dimension) run once at batch 1 and once at batch 16: 14 small-batch calls,
each on the weight copy slim_decode_layout_hint names for its shape and batch (the packed format
through slim_linear_fwd, or the decode-tiled copy through slim_linear_fwd_tiled; both made once,
outside the timed region).
Every linear has its own copy of weight and adapters; the set is 563 MB, so each call reads its
operands from HBM (the L2 holds 126 MB).  The step is captured in a CUDA graph and replayed; time
is taken with CUDA events on the launching stream, max over ranks.  Prints one JSON line, which
also carries per-case tables for the 7B / 13B / 70B shapes, prefill tables (2048 and 4096 tokens,
rank sweep on the 70B shapes), an end-to-end figure through the host-buffer entry point and the CPU
oracle timed on the host's cores.

With N > 1 every rank runs the same step on its own GPU (independent replicas, no collective on
the data path).

--impl reference times the CPU oracle (oracle/) on the host's cores on the same workload:
each step runs each distinct (shape, batch) call once and weights it by how often the block uses it.
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
sys.path.insert(0, ROOT)

from paper_2410_09615_b200 import inputs  # noqa: E402

METRIC = "slim_linear_us_per_call"
UNIT = "us/call"
MODEL = "70b"
WORKLOAD = "llama2_70b_decode_layer_set"
BATCHES = (1, 16)
SHAPES = inputs.LLAMA2_SHAPES[MODEL]           # (name, d_in, d_out, count per block)
CALLS_PER_STEP = sum(c for *_x, c in SHAPES) * len(BATCHES)
HBM_FALLBACK_GBS = 6650.0                      # an earlier copy-bandwidth measurement on B200
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126e6

# DRAM traffic of one launch of the dominant kernel relative to the call's algorithmic bytes, from an
# ncu capture (dram__bytes_read.sum + dram__bytes_write.sum) whose summary is kept with the other
# profiler summaries.  None = no capture of the current kernel: the bench then reports traffic null.
# DRAM bytes / algorithmic bytes of one launch, from the ncu captures summarised under profiles/ (one
# case per kernel; traffic grows with the bytes streamed, so other cases are scaled by their bytes).
# Set an entry to None when its kernel changes after the capture.
NCU_TRAFFIC = {
    "decode_kernel": {"ratio": 1.007, "case": "8192,8192,832,16"},
    "decode_tiled_kernel": {"ratio": 1.035, "case": "8192,28672,832,1"},
    "source": "profiles/decode_kernels_llama2_70b_decode_layer_set.md",
}


def algorithmic_bytes(d_in, d_out, r, b):
    """Bytes one forward call must move: 3 bits per dense weight (4-bit code of
    the kept half plus 2-bit index each), bf16 adapters, X, Y and the scale."""
    return 0.375 * d_out * d_in + 2.0 * r * (d_in + d_out) + 2.0 * b * (d_in + d_out) + 4.0


def algorithmic_bytes_q(d_in, d_out, r, b):
    """The same with quantized adapters: 4 bits per adapter element plus one bf16 scale per 128."""
    groups = r * (d_in // 128) + d_out * ((r + 127) // 128)
    return 0.375 * d_out * d_in + 0.5 * r * (d_in + d_out) + 2.0 * groups + 2.0 * b * (d_in + d_out) + 4.0


def executed_flops(d_in, d_out, r, b):
    return 2.0 * b * d_out * d_in / 2.0 + 2.0 * b * r * (d_in + d_out)


def dense_equiv_flops(d_in, d_out, r, b):
    return 2.0 * b * d_out * d_in + 2.0 * b * r * (d_in + d_out)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback"


def dense_tflops_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while a region runs
    (NVML, read-only)."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = (pynvml.nvmlDeviceGetHandleByUUID(index) if isinstance(index, (str, bytes))
                      else pynvml.nvmlDeviceGetHandleByIndex(index))
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def _reason_names(self, mask):
        nv = self.nv
        table = [("hw_slowdown", "nvmlClocksEventReasonHwSlowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("sw_power_cap", "nvmlClocksEventReasonSwPowerCap", "nvmlClocksThrottleReasonSwPowerCap"),
                 ("hw_power_brake", "nvmlClocksEventReasonHwPowerBrakeSlowdown", "nvmlClocksThrottleReasonHwPowerBrakeSlowdown")]
        out = []
        for name, a, b in table:
            bit = getattr(nv, a, None) or getattr(nv, b, None)
            if bit and (mask & bit):
                out.append(name)
        return out

    def _once(self):
        try:
            self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            try:
                mask = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
            except Exception:
                mask = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            self.reasons.update(self._reason_names(mask))
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._once()
            time.sleep(self.period)

    def start(self):
        if self.ok:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        if self.ok and self._thr:
            self._once()
            self._stop.set()
            self._thr.join()

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------ host data
def host_layers(model=MODEL, ratio=0.1, cfg=4, batches=BATCHES):
    """The distinct layers of one block of `model`, generated once on the host with the recipe of
    paper_2410_09615_b200/inputs.py."""
    out = []
    for li, (name, d_in, d_out, count) in enumerate(inputs.LLAMA2_SHAPES[model]):
        r = inputs.rank_for_ratio(ratio, d_in, d_out)
        wseed = 1000 * cfg + 10 * li
        s, codes, mask = inputs.make_weights(d_out, d_in, wseed)
        L, R = inputs.make_adapters(d_out, d_in, r, wseed)
        out.append(dict(name=name, d_in=d_in, d_out=d_out, r=r, count=count, s=s, codes=codes, mask=mask,
                        L=L, R=R, X={b: inputs.make_activations(b, d_in, wseed + bi) for bi, b in enumerate(batches)}))
    return out


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except Exception:
        pass
    return "unknown"


# ------------------------------------------------------------------ reference arm
def oracle_step(layers, oracle):
    """One pass of the oracle over each distinct (layer shape, batch) pair; returns the time of the whole
    block (each pair weighted by the number of such linears) and the raw wall time."""
    t_weighted, t_raw = 0.0, 0.0
    for ly in layers:
        for b in BATCHES:
            t0 = time.perf_counter()
            oracle.linear_fwd(ly["X"][b], ly["ovals"], ly["ometa"], ly["s"], ly["L"], ly["R"])
            dt = time.perf_counter() - t0
            t_raw += dt
            t_weighted += dt * ly["count"]
    return t_weighted, t_raw


SAMPLE_TEXT = ("each step runs the oracle once per distinct (layer shape, batch) pair of the block, all token rows and all "
               "output columns, and weights the time by the number of such linears in the block (2/2/2/1)")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    layers = host_layers()
    for ly in layers:
        ly["ovals"], ly["ometa"] = oracle.pack(ly["codes"], ly["mask"])
        del ly["codes"], ly["mask"]
    for _ in range(args.warmup):
        oracle_step(layers, oracle)
    total = sum(oracle_step(layers, oracle)[0] for _ in range(args.steps))
    ms_per_step = 1e3 * total / args.steps
    value = 1e3 * ms_per_step / CALLS_PER_STEP
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "batches": list(BATCHES), "calls_per_step": CALLS_PER_STEP},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": SAMPLE_TEXT, "cpu": cpu_model()},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------ GPU arm
KERNEL_OF = {"slim_linear_fwd": "decode_kernel", "slim_linear_fwd_tiled": "decode_tiled_kernel"}


def weight_copy(ly):
    """One more copy of a layer's device tensors, in both weight formats."""
    return {"tiled": ly["tiled"].clone(), "vals": ly["vals"].clone(), "meta": ly["meta"].clone(),
            "L": ly["Ld"].clone(), "R": ly["Rd"].clone()}


def decode_call(K, lib, ly, b, c, ws, ws_bytes, status, tiled=None):
    """(C function, arguments without the stream, name) of one small-batch call on the copy `c`: the
    decode-tiled weight through slim_linear_fwd_tiled when slim_decode_layout_hint says so (or `tiled`
    forces it), else the packed weight through slim_linear_fwd."""
    import ctypes
    P = ctypes.c_void_p
    if tiled is None:
        tiled = K.slim_decode_layout_hint(b, ly["d_out"], ly["d_in"], ly["r"]) == K.LAYOUT_DECODE_TILED
    head = (P(ly["Xd"][b].data_ptr()), b)
    tail = (ctypes.c_float(ly["s"]), P(c["L"].data_ptr()), P(c["R"].data_ptr()), ly["r"], ly["d_out"], ly["d_in"],
            P(ly["Yd"][b].data_ptr()), P(ws.data_ptr()), ws_bytes, P(status.data_ptr()))
    if tiled:
        return lib.slim_linear_fwd_tiled, head + (P(c["tiled"].data_ptr()), K.LAYOUT_DECODE_TILED) + tail, "slim_linear_fwd_tiled"
    return lib.slim_linear_fwd, head + (P(c["vals"].data_ptr()), P(c["meta"].data_ptr())) + tail, "slim_linear_fwd"


def run_ours(args):
    import ctypes
    import torch
    import torch.distributed as dist
    from paper_2410_09615_b200 import binding as K
    from paper_2410_09615_b200 import build, replicas

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    lib = K.lib()
    dev = torch.device("cuda", local)
    P = ctypes.c_void_p

    # ---- weights: packed by slim_pack and repacked by slim_repack_tiled on the GPU; one copy per linear
    layers = host_layers()
    for ly in layers:
        codes_d, mask_d = torch.from_numpy(ly["codes"]).to(dev), torch.from_numpy(ly["mask"]).to(dev)
        ly["vals"], ly["meta"] = K.slim_pack(codes_d, mask_d)
        del codes_d, mask_d, ly["codes"], ly["mask"]
        ly["tiled"] = K.slim_repack_tiled(ly["vals"], ly["meta"])
        ly["Ld"], ly["Rd"] = K.bf16_from_bits(ly["L"], dev), K.bf16_from_bits(ly["R"], dev)
        ly["Xd"] = {b: K.bf16_from_bits(ly["X"][b], dev) for b in BATCHES}
        ly["Yd"] = {b: torch.empty((b, ly["d_out"]), dtype=torch.bfloat16, device=dev) for b in BATCHES}
        ly["copies"] = [weight_copy(ly) for _ in range(ly["count"])]
    ws_bytes = max(K.slim_workspace_bytes(b, ly["d_out"], ly["d_in"], ly["r"]) for ly in layers for b in BATCHES)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    K.slim_workspace_reset(ws)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    set_bytes = sum(c["tiled"].numel() + 2 * c["L"].numel() + 2 * c["R"].numel() for ly in layers for c in ly["copies"])
    torch.cuda.synchronize()

    # the 14 calls of one step: the block at batch 1, then the block at batch 16; every call goes to the
    # weight copy and entry point slim_decode_layout_hint names for its shape and batch
    step_calls = [(ly, b, decode_call(K, lib, ly, b, copy, ws, ws_bytes, status)) for b in BATCHES for ly in layers for copy in ly["copies"]]
    assert len(step_calls) == CALLS_PER_STEP

    def issue_step(stream_ptr):
        for _ly, _b, (fn, a, name) in step_calls:
            rc = fn(*a, stream_ptr)
            if rc != 0:
                raise RuntimeError(f"{name} failed: {K.strerror(rc)}")

    stream = torch.cuda.Stream(device=dev)
    sp = P(stream.cuda_stream)
    with torch.cuda.stream(stream):
        issue_step(sp)                      # first call fills the per-device cache outside any capture
    stream.synchronize()
    launches_per_step = 0
    for _ly, _b, (fn, a, _name) in step_calls:
        fn(*a, sp)
        launches_per_step += lib.slim_last_launch_count()
    stream.synchronize()

    graph, launch_mode = None, "stream"
    if not args.no_graph:
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                issue_step(P(torch.cuda.current_stream().cuda_stream))
            graph, launch_mode = g, "cuda_graph"
        except Exception as e:             # capture refused: time plain stream launches
            sys.stderr.write(f"[bench] graph capture failed ({e}); timing stream launches\n")
            torch.cuda.synchronize()
            graph = None

    def run_steps(n):
        with torch.cuda.stream(stream):
            for _ in range(n):
                if graph is not None:
                    graph.replay()
                else:
                    issue_step(sp)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        gpu_id = local
    sampler = ClockSampler(gpu_id)
    if not sampler.ok:
        sampler = ClockSampler(local)
    run_steps(args.warmup)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    with torch.cuda.stream(stream):
        e0.record(stream)
    run_steps(args.steps)
    with torch.cuda.stream(stream):
        e1.record(stream)
    barrier()
    sampler.stop()
    elapsed_ms = e0.elapsed_time(e1)
    if K.read_status(status) != 0:
        raise RuntimeError(f"device status {K.read_status(status):#x}")
    elapsed_ms = replicas.max_over_ranks(elapsed_ms, dev)
    ms_per_step = elapsed_ms / args.steps
    value = replicas.whole_job_us_per_call(ms_per_step, CALLS_PER_STEP, world)

    # ---- roofline of the dominant kernel over the timed region
    step_bytes = sum(algorithmic_bytes(ly["d_in"], ly["d_out"], ly["r"], b) for ly, b, _ in step_calls)
    kernels = sorted({KERNEL_OF[name] for _ly, _b, (_fn, _a, name) in step_calls})
    peak, peak_kind = measured_peaks()
    achieved = step_bytes / (ms_per_step * 1e-3) / 1e9
    ratios = {k: NCU_TRAFFIC.get(k) for k in kernels}
    traffic = None if any(v is None for v in ratios.values()) else sum(
        ratios[KERNEL_OF[name]]["ratio"] * algorithmic_bytes(ly["d_in"], ly["d_out"], ly["r"], b)
        for ly, b, (_fn, _a, name) in step_calls) / len(step_calls)
    roofline = {"bound": "hbm", "kernel": "+".join(kernels), "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "traffic": traffic,
                "traffic_kind": None if traffic is None else
                "per launch, scaled by algorithmic bytes from the captures in " + NCU_TRAFFIC["source"] + ": " +
                ", ".join(f"{k} x{v['ratio']} (case {v['case']})" for k, v in ratios.items()),
                "bytes_per_launch": step_bytes / len(step_calls), "avg_launch_us": 1e3 * ms_per_step / len(step_calls)}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "batches": list(BATCHES), "calls_per_step": CALLS_PER_STEP,
                       "layers": [[ly["name"], ly["d_in"], ly["d_out"], ly["r"], ly["count"]] for ly in layers],
                       "weight_format": "per call the copy slim_decode_layout_hint names (slim_pack / slim_repack_tiled once, "
                                        "outside the timed region): " + ", ".join(sorted({
                                            f"{ly['name']}@b{b}:{'tiled' if name.endswith('tiled') else 'packed'}"
                                            for ly, b, (_f, _a, name) in step_calls})),
                       "l2": f"inputs larger than L2: every linear has its own copy, {set_bytes / 1e6:.0f} MB per step pass",
                       "launch": launch_mode, "parallelism": f"replicas x{world}"},
            "gpu_launches": launches_per_step * args.steps, "roofline": roofline,
            "clocks": sampler.summary()}

    # ---- end to end through the host-buffer entry point
    line["e2e"] = time_e2e(K, lib, layers, step_calls, ws, ws_bytes, status, stream, args, world, barrier)
    if rank == 0 and not args.skip_extras:
        tables, prefill_rows = [], []
        tables += per_case_table(K, lib, layers, "70b", ws, ws_bytes, status, stream, peak)
        prefill_rows += prefill_table(K, layers, "70b", stream, 4096, sweep=True)
        host70 = layers
        for model, cfg in (("7b", 1), ("13b", 3)):
            small = host_layers(model, 0.1, cfg)
            for ly in small:
                ly["vals"], ly["meta"] = K.slim_pack(torch.from_numpy(ly["codes"]).to(dev), torch.from_numpy(ly["mask"]).to(dev))
                del ly["codes"], ly["mask"]
                ly["tiled"] = K.slim_repack_tiled(ly["vals"], ly["meta"])
                ly["Ld"], ly["Rd"] = K.bf16_from_bits(ly["L"], dev), K.bf16_from_bits(ly["R"], dev)
                ly["Xd"] = {b: K.bf16_from_bits(ly["X"][b], dev) for b in BATCHES}
                ly["Yd"] = {b: torch.empty((b, ly["d_out"]), dtype=torch.bfloat16, device=dev) for b in BATCHES}
            wsb = max(K.slim_workspace_bytes(b, ly["d_out"], ly["d_in"], ly["r"]) for ly in small for b in BATCHES)
            ws2 = ws if wsb <= ws_bytes else K.new_workspace(16, max(l["d_out"] for l in small), max(l["d_in"] for l in small), small[0]["r"])
            tables += per_case_table(K, lib, small, model, ws2, ws2.numel(), status, stream, peak)
            prefill_rows += prefill_table(K, small, model, stream, 2048)
            del small
        line["per_case"] = tables
        # batches between the two of the step, on the two large 70B layers: where the layout hint changes sides
        big = [ly for ly in host70 if ly["d_in"] * ly["d_out"] >= (1 << 27)]
        ws_mid = torch.empty(max(K.slim_workspace_bytes(b, l["d_out"], l["d_in"], l["r"]) for l in big for b in (2, 4, 8)),
                             dtype=torch.uint8, device=dev)
        K.slim_workspace_reset(ws_mid)
        line["per_case_batch_sweep"] = per_case_table(K, lib, big, "70b", ws_mid, ws_mid.numel(), status, stream, peak, batches=(2, 4, 8))
        del ws_mid
        # the step's two kernels apart: bytes and time of the 70B rows each of them serves, weighted by
        # the number of such linears in the block
        count = {ly["name"]: ly["count"] for ly in host70}
        by = {}
        for row in tables:
            if row.get("model") == "70b" and "us" in row:
                k = by.setdefault(row["kernel"], {"bytes": 0.0, "us": 0.0, "launches": 0})
                n = count[row["layer"]]
                k["bytes"] += n * algorithmic_bytes(row["d_in"], row["d_out"], row["r"], row["b"])
                k["us"] += n * row["us"]
                k["launches"] += n
        line["roofline"]["dominant_kernel"] = max(by, key=lambda k: by[k]["us"])      # its own figures: by_kernel
        line["roofline"]["by_kernel"] = {
            name: {"launches_per_step": k["launches"], "avg_launch_us": round(k["us"] / k["launches"], 3),
                   "achieved": round(k["bytes"] / k["us"] / 1e3, 1), "frac": round(k["bytes"] / k["us"] / 1e3 / peak, 4),
                   "share_of_step_time": round(k["us"] / sum(v["us"] for v in by.values()), 4)}
            for name, k in by.items()}
        line["prefill"] = prefill_rows
        line["roofline_prefill"] = prefill_roofline(prefill_rows)
        line["pack"] = time_pack(K, host70[0], stream)
        line["quantized_adapters"] = quantized_adapter_table(K, lib, host70, stream, peak)
    if rank == 0 and world == 1 and not args.skip_cpu:
        line["cpu_baseline"] = time_cpu_baseline(layers)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def time_graph_of_calls(fn, calls, stream, replays=10):
    """Median per-call time (us) of a CUDA graph holding `calls` of the C function `fn`, replayed."""
    import ctypes
    import torch
    P = ctypes.c_void_p
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        cur = P(torch.cuda.current_stream().cuda_stream)
        for a in calls:
            fn(*a, cur)
    times = []
    with torch.cuda.stream(stream):
        for _ in range(3):
            g.replay()
        for _ in range(replays):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            g.replay()
            a1.record(stream)
            a1.synchronize()
            times.append(1e3 * a0.elapsed_time(a1) / len(calls))
    return float(np.median(times)), float(np.min(times))


def per_case_table(K, lib, layers, model, ws, ws_bytes, status, stream, peak, batches=BATCHES):
    """Per (layer, batch): us/call of both small-batch kernels over rotating copies (> 2x L2 between
    reuses); `us` is the one slim_decode_layout_hint names, with its algorithmic GB/s and fraction of
    the HBM roofline."""
    import torch
    rows = []
    for ly in layers:
        per_copy = ly["tiled"].numel() + 2 * ly["Ld"].numel() + 2 * ly["Rd"].numel()
        n_copies = int(np.ceil(2 * L2_BYTES / per_copy)) + 1
        copies = [weight_copy(ly) for _ in range(n_copies)]
        torch.cuda.synchronize()
        for b in batches:
            if b not in ly["Xd"]:
                g = torch.Generator(device=ly["Ld"].device)
                g.manual_seed(1000 + b)
                ly["Xd"][b] = torch.randn((b, ly["d_in"]), device=ly["Ld"].device, generator=g).bfloat16()
                ly["Yd"][b] = torch.empty((b, ly["d_out"]), dtype=torch.bfloat16, device=ly["Ld"].device)
            hint_tiled = K.slim_decode_layout_hint(b, ly["d_out"], ly["d_in"], ly["r"]) == K.LAYOUT_DECODE_TILED
            t = {}
            for tiled in (False, True):
                trip = [decode_call(K, lib, ly, b, c, ws, ws_bytes, status, tiled=tiled) for c in copies] * 3
                try:
                    t[tiled] = time_graph_of_calls(trip[0][0], [a for _f, a, _n in trip], stream)
                except Exception as e:
                    t[tiled] = None
                    sys.stderr.write(f"[bench] {model} {ly['name']} b={b} tiled={tiled}: {str(e)[:80]}\n")
            if t[hint_tiled] is None:
                rows.append({"model": model, "layer": ly["name"], "b": b, "error": "call failed"})
                continue
            med, best = t[hint_tiled]
            nbytes = algorithmic_bytes(ly["d_in"], ly["d_out"], ly["r"], b)
            gbs = nbytes / (med * 1e-6) / 1e9
            rows.append({"model": model, "layer": ly["name"], "d_in": ly["d_in"], "d_out": ly["d_out"], "r": ly["r"], "b": b,
                         "kernel": "decode_tiled_kernel" if hint_tiled else "decode_kernel",
                         "us": round(med, 3), "us_min": round(best, 3), "GBs": round(gbs, 1),
                         "frac_measured": round(gbs / peak, 4), "frac_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4),
                         "roofline_us": round(nbytes / peak / 1e3, 3),
                         "us_other_kernel": None if t[not hint_tiled] is None else round(t[not hint_tiled][0], 3)})
        del copies
    return rows


def quantized_adapter_table(K, lib, layers, stream, peak):
    """The 70B layers at batch 1 and 16 through slim_linear_fwd_q (adapters as int4 codes with a bf16
    scale per 128 elements) beside slim_linear_fwd on the same packed weight with bf16 adapters:
    bytes per call, us per call over rotating copies, fraction of the HBM roofline on the smaller bytes."""
    import ctypes
    import torch
    P = ctypes.c_void_p
    rows = []
    for ly in layers:
        d_in, d_out, r = ly["d_in"], ly["d_out"], ly["r"]
        Lq, Ls = K.slim_pack_adapter(ly["Ld"])
        Rq, Rs = K.slim_pack_adapter(ly["Rd"])
        per_copy = ly["vals"].numel() + ly["meta"].numel() + 2 * ly["Ld"].numel() + 2 * ly["Rd"].numel()
        n_copies = int(np.ceil(2 * L2_BYTES / per_copy)) + 1
        copies = [dict(vals=ly["vals"].clone(), meta=ly["meta"].clone(), L=ly["Ld"].clone(), R=ly["Rd"].clone(),
                       Lq=Lq.clone(), Ls=Ls.clone(), Rq=Rq.clone(), Rs=Rs.clone()) for _ in range(n_copies)]
        wsq = torch.empty(max(K.slim_workspace_bytes_q(b, d_out, d_in, r) for b in BATCHES), dtype=torch.uint8, device=Lq.device)
        K.slim_workspace_reset(wsq)
        status = torch.zeros(1, dtype=torch.int32, device=Lq.device)
        torch.cuda.synchronize()
        for b in BATCHES:
            head = (P(ly["Xd"][b].data_ptr()), b)
            tail = (r, d_out, d_in, P(ly["Yd"][b].data_ptr()), P(wsq.data_ptr()), wsq.numel(), P(status.data_ptr()))
            plain = [head + (P(c["vals"].data_ptr()), P(c["meta"].data_ptr()), ctypes.c_float(ly["s"]), P(c["L"].data_ptr()),
                             P(c["R"].data_ptr())) + tail for c in copies] * 3
            quant = [head + (P(c["vals"].data_ptr()), P(c["meta"].data_ptr()), ctypes.c_float(ly["s"]), P(c["Lq"].data_ptr()),
                             P(c["Ls"].data_ptr()), P(c["Rq"].data_ptr()), P(c["Rs"].data_ptr())) + tail for c in copies] * 3
            try:
                t_plain, _ = time_graph_of_calls(lib.slim_linear_fwd, plain, stream)
                t_q, _ = time_graph_of_calls(lib.slim_linear_fwd_q, quant, stream)
            except Exception as e:
                rows.append({"layer": ly["name"], "b": b, "error": str(e)[:80]})
                continue
            lib.slim_linear_fwd_q(*quant[0], P(stream.cuda_stream))
            launches = lib.slim_last_launch_count()
            nb, nq = algorithmic_bytes(d_in, d_out, r, b), algorithmic_bytes_q(d_in, d_out, r, b)
            rows.append({"layer": ly["name"], "d_in": d_in, "d_out": d_out, "r": r, "b": b,
                         "path": "decode kernel on codes and scales" if launches == 1 else "adapters expanded to bf16 first",
                         "bytes_bf16_adapters": nb, "bytes_quantized": nq, "bytes_ratio": round(nb / nq, 3),
                         "us_bf16_adapters": round(t_plain, 3), "us_quantized": round(t_q, 3),
                         "speedup": round(t_plain / t_q, 3), "frac_measured_quantized": round(nq / (t_q * 1e-6) / 1e9 / peak, 4)})
        torch.cuda.synchronize()
        if K.read_status(status) != 0:
            raise RuntimeError(f"device status {K.read_status(status):#x}")
        del copies
    return rows


def prefill_table(K, layers, model, stream, tokens, sweep=False):
    """The layers of one model at `tokens` tokens (tcgen05 prefill kernel on the packed weight): us/call,
    dense-equivalent TFLOP/s (the 2:4 product counted as if dense, adapters at face value) and its
    fraction of the sparse bf16 peak, taken as twice the measured dense bf16 peak.  `sweep`: ranks of
    0, 0.05, 0.1 and 0.2 x the smaller dimension instead of 0.1 only."""
    import torch
    dense_peak, kind = dense_tflops_peak()
    rows = []
    for ly in layers:
        X = K.bf16_from_bits(inputs.make_activations(tokens, ly["d_in"], 7))
        Y = torch.empty((tokens, ly["d_out"]), dtype=torch.bfloat16, device=X.device)
        for ratio in ((0.0, 0.05, 0.1, 0.2) if sweep else (0.1,)):
            r = inputs.rank_for_ratio(ratio, ly["d_in"], ly["d_out"])
            if r == ly["r"]:
                Ld, Rd = ly["Ld"], ly["Rd"]
            elif r == 0:
                Ld = Rd = None
            else:
                Lh, Rh = inputs.make_adapters(ly["d_out"], ly["d_in"], r, 77)
                Ld, Rd = K.bf16_from_bits(Lh), K.bf16_from_bits(Rh)
            ws = K.new_workspace(tokens, ly["d_out"], ly["d_in"], r)
            with torch.cuda.stream(stream):
                for _ in range(3):
                    K.slim_linear_fwd(X, ly["vals"], ly["meta"], ly["s"], Ld, Rd, Y=Y, workspace=ws)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                n = 10
                e0.record(stream)
                for _ in range(n):
                    K.slim_linear_fwd(X, ly["vals"], ly["meta"], ly["s"], Ld, Rd, Y=Y, workspace=ws)
                e1.record(stream)
                e1.synchronize()
            us = 1e3 * e0.elapsed_time(e1) / n
            tf = dense_equiv_flops(ly["d_in"], ly["d_out"], r, tokens) / (us * 1e-6) / 1e12
            rows.append({"model": model, "layer": ly["name"], "d_in": ly["d_in"], "d_out": ly["d_out"], "r": r, "tokens": tokens,
                         "kernel": K.KERNEL_NAMES[K.slim_select_kernel(tokens, ly["d_out"], ly["d_in"], r)],
                         "us": round(us, 2), "dense_equiv_TFLOPs": round(tf, 1),
                         "executed_TFLOPs": round(executed_flops(ly["d_in"], ly["d_out"], r, tokens) / (us * 1e-6) / 1e12, 1),
                         "frac_of_sparse_peak": round(tf / (2 * dense_peak), 4), "sparse_peak_TFLOPs": 2 * dense_peak,
                         "peak_kind": f"2 x dense bf16 of {kind}", "frac_of_nominal_4500": round(tf / 4500.0, 4)})
            del ws
        del X, Y
    return rows


def prefill_roofline(rows):
    """One structured entry for the prefill kernel: the 2048-token 7B rows at rank 0.1 taken together
    (dense-equivalent flops of the three shapes / their summed time)."""
    sel = [r for r in rows if r.get("model") == "7b" and "us" in r]
    if not sel:
        return None
    flops = sum(dense_equiv_flops(r["d_in"], r["d_out"], r["r"], r["tokens"]) for r in sel)
    us = sum(r["us"] for r in sel)
    peak = sel[0]["sparse_peak_TFLOPs"]
    ach = flops / (us * 1e-6) / 1e12
    return {"bound": "tensor", "kernel": "prefill_kernel", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
            "peak_kind": sel[0]["peak_kind"], "workload": "llama2_7b layer shapes, 2048 tokens, rank 416 (one call per distinct shape)",
            "traffic": None, "flops": "dense-equivalent: 2 b d_in d_out + 2 b r (d_in + d_out)"}


def time_pack(K, ly, stream):
    """slim_pack and slim_repack_tiled of one layer (offline steps, outside the per-call metric)."""
    import torch
    s, codes_h, mask_h = inputs.make_weights(ly["d_out"], ly["d_in"], 5)
    codes, mask = torch.from_numpy(codes_h).cuda(), torch.from_numpy(mask_h).cuda()
    vals, meta = K.slim_pack(codes, mask)
    tiled = K.slim_repack_tiled(vals, meta)
    out = {"layer": [ly["d_in"], ly["d_out"]]}
    with torch.cuda.stream(stream):
        for name, fn, nbytes in (("pack", lambda: K.slim_pack(codes, mask, vals, meta, check=False), 2.375),
                                 ("repack_tiled", lambda: K.slim_repack_tiled(vals, meta, out=tiled), 0.75)):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(3):
                fn()
            a0.record(stream)
            for _ in range(10):
                fn()
            a1.record(stream)
            a1.synchronize()
            us = 1e3 * a0.elapsed_time(a1) / 10
            out[name] = {"us": round(us, 2), "GBs": round(nbytes * ly["d_out"] * ly["d_in"] / us / 1e3, 1)}
    # the producers before them: SLiM-Quant scale search on float32 weights, adapter quantization
    Wf = torch.randn((ly["d_out"], ly["d_in"]), device="cuda") * 0.02
    A = ly["Rd"]
    with torch.cuda.stream(stream):
        for name, fn, nbytes in (("slim_quant", lambda: K.slim_quant(Wf), 13.0 * ly["d_out"] * ly["d_in"]),
                                 ("pack_adapter_R", lambda: K.slim_pack_adapter(A), 2.516 * A.numel())):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(2):
                fn()
            a0.record(stream)
            for _ in range(5):
                fn()
            a1.record(stream)
            a1.synchronize()
            us = 1e3 * a0.elapsed_time(a1) / 5
            out[name] = {"us": round(us, 2), "GBs": round(nbytes / us / 1e3, 1)}
    out["bytes"] = ("pack: 2 B read + 0.375 B written per dense weight; repack: 0.375 B read + 0.375 B written; "
                    "slim_quant: three passes over the float32 weights (largest magnitude, histogram, codes) + 1 B written, "
                    "and a fixed search of 29 candidates over the histogram; pack_adapter: 2 B read + 0.516 B written per element")
    return out


def time_e2e(K, lib, layers, step_calls, ws, ws_bytes, status, stream, args, world, barrier):
    """Same step through the host-buffer entry points: X comes from pinned host memory
    and Y goes back to pinned host memory inside every call."""
    import ctypes
    import torch
    from paper_2410_09615_b200 import replicas
    P = ctypes.c_void_p
    host = {}
    for ly in layers:
        for b in BATCHES:
            xh = K.bf16_from_bits(ly["X"][b], "cpu").pin_memory()
            yh = torch.empty((b, ly["d_out"]), dtype=torch.bfloat16).pin_memory()
            host[(ly["name"], b)] = (xh, yh)
    calls, h2d, d2h = [], 0, 0
    for ly, b, (_fn, a, name) in step_calls:
        xh, yh = host[(ly["name"], b)]
        # (X_host, b, weight (two arguments), s, L, R, r, d_out, d_in, Y_host, x_dev, y_dev, ws, ws_bytes, status)
        fn = lib.slim_linear_fwd_tiled_host if name == "slim_linear_fwd_tiled" else lib.slim_linear_fwd_host
        calls.append((fn, (P(xh.data_ptr()), b, a[2], a[3], a[4], a[5], a[6], a[7], a[8], a[9], P(yh.data_ptr()),
                           P(ly["Xd"][b].data_ptr()), P(ly["Yd"][b].data_ptr()), a[11], a[12], a[13])))
        h2d += xh.numel() * 2
        d2h += yh.numel() * 2
    sp = P(stream.cuda_stream)
    steps = max(1, min(args.steps, 100))

    def run(n):
        for _ in range(n):
            for fn, c in calls:
                rc = fn(*c, sp)
                if rc != 0:
                    raise RuntimeError(f"host-buffer call failed: {K.strerror(rc)}")

    run(min(args.warmup, 10))
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    run(steps)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    ms = replicas.max_over_ranks(ms, "cuda")
    return {"value": replicas.whole_job_us_per_call(ms / steps, CALLS_PER_STEP, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": steps, "api": "slim_linear_fwd_host / slim_linear_fwd_tiled_host"}


def time_cpu_baseline(layers, repeats=2):
    """The oracle, as it stands, on the host's cores: the whole step (a bounded sample: one pass over
    each distinct (shape, batch) pair per repeat), plus a single-thread timing of the smallest layer."""
    import oracle
    host = []
    for ly in layers:
        h = dict(ly)
        h["ovals"], h["ometa"] = ly["vals"].cpu().numpy(), ly["meta"].cpu().numpy()
        host.append(h)
    t_weighted, t_raw = 0.0, 0.0
    for _ in range(repeats):
        tw, tr = oracle_step(host, oracle)
        t_weighted += tw
        t_raw += tr
    out = {"value": 1e6 * t_weighted / repeats / CALLS_PER_STEP, "unit": UNIT, "cores": oracle.num_threads(),
           "kind": "oracle", "cpu": cpu_model(),
           "sample": f"{SAMPLE_TEXT}; repeated {repeats} times ({t_raw:.1f} s of wall time on all cores)"}
    # single thread: one call of the smallest layer at batch 16 in a child process pinned to one OpenMP thread
    small = min(host, key=lambda h: h["d_in"] * h["d_out"])
    try:
        code = ("import sys, time; sys.path.insert(0, %r); import numpy as np, oracle; "
                "from paper_2410_09615_b200 import inputs; "
                "s, c, m = inputs.make_weights(%d, %d, 9); v, mt = oracle.pack(c, m); L, R = inputs.make_adapters(%d, %d, %d, 9); "
                "X = inputs.make_activations(16, %d, 9); oracle.linear_fwd(X, v, mt, s, L, R); t = time.perf_counter(); "
                "oracle.linear_fwd(X, v, mt, s, L, R); print(time.perf_counter() - t, oracle.num_threads())"
                % (ROOT, small["d_out"], small["d_in"], small["d_out"], small["d_in"], small["r"], small["d_in"]))
        res = {}
        for label, env in (("one_thread", {"OMP_NUM_THREADS": "1"}), ("all_threads", {})):
            o = subprocess.run([sys.executable, "-c", code], env={**os.environ, **env}, capture_output=True, text=True, timeout=600)
            sec, thr = o.stdout.split()[-2:]
            res[label] = {"us": round(1e6 * float(sec), 1), "threads": int(thr)}
        out["single_thread"] = {"case": [small["d_in"], small["d_out"], small["r"], 16], **res}
    except Exception as e:
        out["single_thread"] = {"error": str(e)[:100]}
    return out


def run_single_case(args):
    """Plain stream launches of one (d_in, d_out, r, b) case, L2 flushed between them: the command a
    profiler captures.  b <= 16: the copy --layout names; above: slim_linear_fwd on the packed weight."""
    import torch
    from paper_2410_09615_b200 import binding as K, build
    build.build()
    d_in, d_out, r, b = (int(x) for x in args.case.split(","))
    s, codes, mask = inputs.make_weights(d_out, d_in, 1)
    L, R = inputs.make_adapters(d_out, d_in, r, 1)
    vals, meta = K.slim_pack(torch.from_numpy(codes).cuda(), torch.from_numpy(mask).cuda())
    use_tiled = b <= 16 and (args.layout == "tiled" or (args.layout == "hint" and
                             K.slim_decode_layout_hint(b, d_out, d_in, r) == K.LAYOUT_DECODE_TILED))
    tiled = K.slim_repack_tiled(vals, meta) if use_tiled else None
    Ld = K.bf16_from_bits(L) if r else None
    Rd = K.bf16_from_bits(R) if r else None
    X = K.bf16_from_bits(inputs.make_activations(b, d_in, 1))
    ws = K.new_workspace(b, d_out, d_in, r)
    Y = torch.empty((b, d_out), dtype=torch.bfloat16, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    for _ in range(args.calls):
        flush.zero_()                       # evict the weights from L2 between calls
        e0.record()
        if tiled is not None:
            K.slim_linear_fwd_tiled(X, tiled, d_out, s, Ld, Rd, Y=Y, workspace=ws)
        else:
            K.slim_linear_fwd(X, vals, meta, s, Ld, Rd, Y=Y, workspace=ws)
        e1.record()
        e1.synchronize()
        times.append(1e3 * e0.elapsed_time(e1))
    print(json.dumps({"case": [d_in, d_out, r, b], "calls": args.calls, "us_median": float(np.median(times)),
                      "us_min": float(np.min(times)), "path": "tiled decode" if tiled is not None else
                      K.KERNEL_NAMES[K.slim_select_kernel(b, d_out, d_in, r)],
                      "algorithmic_bytes": algorithmic_bytes(d_in, d_out, r, b)}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, help="d_in,d_out,r,b: run plain launches of one case (for profilers)")
    ap.add_argument("--calls", type=int, default=5)
    ap.add_argument("--layout", choices=["hint", "packed", "tiled"], default="hint",
                    help="with --case and b <= 16: which weight copy (default: what slim_decode_layout_hint names)")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA graph")
    ap.add_argument("--skip-extras", action="store_true", help="skip the per-case and prefill tables and the pack timing")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the CPU-oracle baseline")
    args = ap.parse_args()
    if args.case:
        return run_single_case(args)
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        args.steps = min(args.steps, 3)       # the oracle takes seconds per step
        args.warmup = min(args.warmup, 1)
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
