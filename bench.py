#!/usr/bin/env python
"""Benchmark of one DualDiffusion verification step on B200.

A step is one pass of the whole hot path over one batch of synthetic input:
one dd_bidir_attention call (one layer's full-sequence bidirectional attention)
followed by one dd_verify call (KL mode), on the LLaDA-8B-shaped workload
(attention B=1,H=32,N=1024,D=128; logits [1,256,126464], tau=0.5, k=32).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is the device-timed latency of a step
with the inputs resident in HBM; `e2e` is the same step through the host-buffer
entry points with the host<->device copies inside the timed region.
--impl reference times the CPU oracle on the host cores instead (a deliberately
slow baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_05250_b200 import synth  # noqa: E402

CFG = 1
ATT = synth.ATTENTION_CONFIGS[CFG]
VER = synth.VERIFY_CONFIGS[CFG]
WORKLOAD = ("cfg1 LLaDA-8B-shaped verify step: attention B=1,H=32,N=1024,D=128 bf16 + "
            "dd_verify KL mode on logits [1,256,126464] bf16, all 256 positions flagged, tau=0.5, k=32")
L2_BYTES = 126 * 1024 * 1024
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
# profiles/ (None until a capture of that kernel exists).
NCU_TRAFFIC_BYTES = {"attention": 25.27e6, "verify": 136.55e6}


def attention_flops():
    return 4.0 * ATT["B"] * ATT["H"] * ATT["N"] ** 2 * ATT["D"]


def attention_bytes():
    return 4.0 * ATT["B"] * ATT["H"] * ATT["N"] * ATT["D"] * 2


def verify_bytes(n_flagged):
    # both logit rows of every flagged position once, plus token/flag/outputs per position
    return n_flagged * VER["V"] * 2 * 2 + VER["B"] * VER["P"] * 14.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- clocks


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only)."""

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples = []          # (t, sm_mhz, reasons_bitmask)
        self.sm_max = None
        self._stop = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, int(reasons)))
            except Exception:
                pass
            self._stop.wait(self.period)

    def stop(self):
        self._stop.set()

    def summary(self, t0, t1):
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}
        win = [s for s in self.samples if t0 <= s[0] <= t1]
        if not win:
            win = self.samples[-3:]
        if not win:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0}
        bits = 0
        for s in win:
            bits |= s[2]
        return {"sm_mhz": float(np.median([s[1] for s in win])), "sm_max_mhz": self.sm_max,
                "reasons": sorted(n for b, n in names.items() if bits & b), "samples": len(win)}


# ----------------------------------------------------------------------------- helpers


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), \
        int(os.environ.get("WORLD_SIZE", "1"))


def graph_chunk(K, cap=200):
    g = min(K, cap)
    while K % g:
        g -= 1
    return g


def max_over_ranks(values, device, distributed):
    """Element-wise maximum of a list of floats over all ranks (the job is as slow as its slowest rank)."""
    import torch
    vals = torch.tensor(list(values), dtype=torch.float64, device=device)
    if distributed:
        import torch.distributed as dist
        dist.all_reduce(vals, op=dist.ReduceOp.MAX)
    return [float(x) for x in vals.tolist()]


def bf16_tensor(bits, device=None, pin=False):
    import torch
    t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    if device is not None:
        return t.to(device, non_blocking=False)
    return t.pin_memory() if pin else t


# ----------------------------------------------------------------------------- CPU baseline (oracle)


def oracle_step_sample(oracle, att_in, ver_in, att_rows, ver_rows):
    """One bounded sample of a step on the host cores; returns seconds."""
    q, k, v = att_in
    dra, ver, tokens, flags = ver_in
    t0 = time.perf_counter()
    oracle.attention(q, k, v, ATT["D"] ** -0.5, rows=att_rows)
    oracle.verify(dra[:, :ver_rows], ver[:, :ver_rows], tokens[:, :ver_rows], flags[:, :ver_rows],
                  synth.MODE_KL, VER["tau"], VER["k"], VER["seed"])
    return time.perf_counter() - t0


def cpu_baseline(oracle, att_in, ver_in, budget_s=12.0):
    """The oracle as it stands on the whole cfg1 step, repeated for ~budget_s seconds."""
    att_rows = np.arange(ATT["N"], dtype=np.int32)
    times = []
    t_start = time.perf_counter()
    while not times or (time.perf_counter() - t_start < budget_s and len(times) < 64):
        times.append(oracle_step_sample(oracle, att_in, ver_in, att_rows, VER["P"]))
    return {"value": 1e3 * float(np.mean(times)), "unit": "ms", "cores": oracle.threads(), "kind": "oracle",
            "sample": f"the full cfg1 step (all {ATT['H']}x{ATT['N']} attention rows, all {VER['P']} logit rows), "
                      f"{len(times)} repetitions"}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    oracle.build()
    att_in = synth.attention_config_inputs(CFG)
    ver_in = synth.verify_config_inputs(CFG)
    K, W = args.steps, args.warmup
    # bounded sample per step so that K + W steps end within a few minutes
    full = oracle_step_sample(oracle, att_in, ver_in, np.arange(ATT["N"], dtype=np.int32), VER["P"])
    per_step_budget = 150.0 / max(1, K + W)
    frac = min(1.0, per_step_budget / max(full, 1e-9))
    n_att = max(1, int(ATT["N"] * frac))
    n_ver = max(1, int(VER["P"] * frac))
    att_rows = np.linspace(0, ATT["N"] - 1, n_att).astype(np.int32)
    for _ in range(W):
        oracle_step_sample(oracle, att_in, ver_in, att_rows, n_ver)
    t = 0.0
    for _ in range(K):
        t += oracle_step_sample(oracle, att_in, ver_in, att_rows, n_ver)
    # scale the sample to a whole step by the units processed (rows of each kernel)
    scale = 0.5 * (ATT["N"] / n_att + VER["P"] / n_ver)
    ms = 1e3 * t / K * scale
    sample = (f"{n_att}/{ATT['N']} attention query rows per head and {n_ver}/{VER['P']} logit rows per step, "
              f"time scaled to the whole step by rows")
    line = {
        "impl": "reference", "metric": "verify_step_latency_ms", "value": ms, "unit": "ms",
        "n_gpus": args.gpus, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD},
        "cpu_baseline": {"value": ms, "unit": "ms", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": ms, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------- GPU arm


def run_ours(args):
    import torch
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    distributed = world > 1
    if distributed:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2604_05250_b200 import binding as dd
    from paper_2604_05250_b200 import build
    build.build()
    dd.lib()

    K, W = args.steps, max(3, args.warmup)
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else local_rank)

    # ---- inputs: several distinct sets per kernel so that consecutive steps never hit L2
    att_sets = max(3, math.ceil(2.2 * L2_BYTES / attention_bytes()))
    ver_sets = 3
    base_seed = synth.config_seed(CFG) + 17 * rank
    att_host = [synth.attention_inputs(ATT["B"], ATT["H"], ATT["N"], ATT["D"], base_seed + s) for s in range(att_sets)]
    ver_host = [synth.verify_inputs(VER["B"], VER["P"], VER["V"], VER["flagged"], VER["err"], base_seed + s)
                for s in range(ver_sets)]
    n_flagged = int(ver_host[0][3].sum())
    att_dev = [tuple(bf16_tensor(x, dev) for x in s) + (torch.empty(ATT["B"], ATT["H"], ATT["N"], ATT["D"],
                                                                    dtype=torch.bfloat16, device=dev),)
               for s in att_host]
    ver_dev = []
    for dra, ver, tok, fl in ver_host:
        ver_dev.append(dict(dra=bf16_tensor(dra, dev), ver=bf16_tensor(ver, dev),
                            tok=torch.from_numpy(tok).to(dev), fl=torch.from_numpy(fl).to(dev),
                            ot=torch.empty(VER["B"], VER["P"], dtype=torch.int32, device=dev),
                            om=torch.empty(VER["B"], VER["P"], dtype=torch.uint8, device=dev),
                            osc=torch.empty(VER["B"], VER["P"], dtype=torch.float32, device=dev)))
    scale = ATT["D"] ** -0.5
    mode = synth.MODE_KL

    def attention_call(i):
        q, k, v, o = att_dev[i % att_sets]
        dd.bidir_attention(q, k, v, out=o, scale=scale)

    def verify_call(i):
        s = ver_dev[i % ver_sets]
        dd.verify(s["dra"], s["ver"], s["tok"], s["fl"], mode, VER["tau"], VER["k"], VER["seed"],
                  out_tokens=s["ot"], out_mask=s["om"], out_score=s["osc"])

    def step(i):
        attention_call(i)
        verify_call(i)

    stream = torch.cuda.Stream(device=dev)

    def timed(fn, n, use_graph=True):
        """Device time (ms) of n calls fn(0..n-1) on `stream`, CUDA events on that stream."""
        g = graph_chunk(n)
        launches = 0
        with torch.cuda.stream(stream):
            if use_graph:
                graph = torch.cuda.CUDAGraph()
                c0 = dd.launch_count()
                with torch.cuda.graph(graph, stream=stream):
                    for i in range(g):
                        fn(i)
                launches = (dd.launch_count() - c0) * (n // g)
                graph.replay()                      # untimed: first replay pays the upload
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            stream.synchronize()
            if distributed:
                dist.barrier()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            e0.record(stream)
            if use_graph:
                for _ in range(n // g):
                    graph.replay()
            else:
                c0 = dd.launch_count()
                for i in range(n):
                    fn(i)
                launches = dd.launch_count() - c0
            e1.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            if distributed:
                dist.barrier()
            t1 = time.perf_counter()
        return e0.elapsed_time(e1), launches, (t0, t1)

    sampler.start()
    with torch.cuda.stream(stream):
        for i in range(W):
            step(i)
    stream.synchronize()
    assert dd.attention_status() == 0

    use_graph = not args.no_graph
    total_ms, launches, window = timed(step, K, use_graph)
    att_ms, _, _ = timed(attention_call, K, use_graph)
    ver_ms, _, _ = timed(verify_call, K, use_graph)
    clocks = sampler.summary(*window)

    # ---- end to end: host buffers in, host results out, copies inside the timed region
    pin = lambda a: torch.from_numpy(a).pin_memory()  # noqa: E731
    e2e_steps = max(3, min(K, 20))
    hq, hk, hv = (bf16_tensor(x, pin=True) for x in att_host[0])
    ho = torch.empty(ATT["B"], ATT["H"], ATT["N"], ATT["D"], dtype=torch.bfloat16).pin_memory()
    hdra, hver = bf16_tensor(ver_host[0][0], pin=True), bf16_tensor(ver_host[0][1], pin=True)
    htok, hfl = pin(ver_host[0][2]), pin(ver_host[0][3])
    hot = torch.empty(VER["B"], VER["P"], dtype=torch.int32).pin_memory()
    hom = torch.empty(VER["B"], VER["P"], dtype=torch.uint8).pin_memory()
    hos = torch.empty(VER["B"], VER["P"], dtype=torch.float32).pin_memory()

    def e2e_step():
        dd.bidir_attention(hq, hk, hv, out=ho, scale=scale, host=True)
        dd.verify(hdra, hver, htok, hfl, mode, VER["tau"], VER["k"], VER["seed"],
                  out_tokens=hot, out_mask=hom, out_score=hos, host=True)

    with torch.cuda.stream(stream):
        for _ in range(3):
            e2e_step()
        stream.synchronize()
        if distributed:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
            stream.synchronize()               # the caller reads the step's result on the host
        e1.record(stream)
        stream.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    sampler.stop()
    h2d = 3 * attention_bytes() / 4 + 2 * VER["B"] * VER["P"] * VER["V"] * 2 + VER["B"] * VER["P"] * 5
    d2h = attention_bytes() / 4 + VER["B"] * VER["P"] * 9
    assert dd.attention_status() == 0

    # ---- max over ranks
    total_ms, att_ms, ver_ms, e2e_ms = max_over_ranks([total_ms, att_ms, ver_ms, e2e_ms], dev, distributed)
    ms_step, att_step, ver_step = total_ms / K, att_ms / K, ver_ms / K

    if rank == 0:
        peaks = measured_peaks()
        long_loop = att_ms > 1000.0
        att_peak = peaks["bf16_sustained"] if long_loop else peaks["bf16"]
        att_tflops = attention_flops() / (att_step * 1e-3) / 1e12
        ver_gbs = verify_bytes(n_flagged) / (ver_step * 1e-3) / 1e9
        kernels = {
            "attention": {"ms": att_step, "tflops": att_tflops, "frac_of_nominal_2250": att_tflops / NOMINAL_BF16_TFLOPS,
                          "frac_of_measured": att_tflops / att_peak,
                          "peak_used": f"{att_peak} TFLOP/s ({'sustained' if long_loop else 'burst'}, {peaks['source']})"},
            "verify": {"ms": ver_step, "gbs": ver_gbs, "frac_of_nominal_8000": ver_gbs / NOMINAL_HBM_GBS,
                       "frac_of_measured": ver_gbs / peaks["hbm"], "algorithmic_bytes": verify_bytes(n_flagged),
                       "peak_used": f"{peaks['hbm']} GB/s ({peaks['source']})"},
        }
        if ver_step >= att_step:
            roof = {"kernel": "verify_stream_kernel", "bound": "hbm", "achieved": ver_gbs, "peak": peaks["hbm"], "unit": "GB/s",
                    "frac": ver_gbs / peaks["hbm"], "traffic": NCU_TRAFFIC_BYTES["verify"], "peak_source": peaks["source"]}
        else:
            roof = {"kernel": "attention_kernel", "bound": "tensor", "achieved": att_tflops, "peak": att_peak,
                    "unit": "TFLOP/s", "frac": att_tflops / att_peak, "traffic": NCU_TRAFFIC_BYTES["attention"],
                    "peak_source": peaks["source"]}
        import oracle
        oracle.build()
        cpu = cpu_baseline(oracle, att_host[0], ver_host[0])
        line = {
            "metric": "verify_step_latency_ms", "value": ms_step, "unit": "ms", "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": f"inputs rotate over {att_sets} attention sets and {ver_sets} "
                       "logit sets, each group larger than 2x L2, so every step reads HBM",
                       "launch": "cuda_graph replay" if use_graph else "eager", "parallelism": f"replicas x{world}"},
            "throughput": {"value": world * 1e3 / ms_step, "unit": "verify_steps/s"},
            "clocks": clocks,
            "e2e": {"value": e2e_ms, "unit": "ms", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "steps": e2e_steps},
            "gpu_launches": int(launches),
            "roofline": roof,
            "kernels": kernels,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if distributed:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph")
    args = ap.parse_args()
    if args.steps < 1:
        ap.error("--steps must be >= 1")
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
