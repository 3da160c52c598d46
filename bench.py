#!/usr/bin/env python
"""Benchmark of one DualDiffusion verification step on B200.

A step is one pass of the whole hot path over one batch of synthetic input:
one dd_bidir_attention call (one layer's full-sequence bidirectional attention)
followed by one dd_verify call (KL mode), on the LLaDA-8B-shaped workload
(attention B=1,H=32,N=1024,D=128; logits [1,256,126464], tau=0.5, k=32).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is the device-timed latency of a step
with the inputs resident in HBM: the K steps are captured as one CUDA graph that
is replayed until the timed window is at least a quarter of a second, every
replay between two CUDA events, and the median over replays is reported (with
the 10th and 90th percentiles, and the eagerly launched latency beside it).
`e2e` is the same step through the host-buffer entry points with the
host<->device copies inside the timed region.  At one GPU the line also carries
`other_configs`: every other workload shape (batched serving, long context, the
sequence-length and vocabulary sweeps, the tiny case, the drafter's block
attention), each timed the same way with its own clock record.
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
NCU_TRAFFIC_BYTES = {"attention": 25.27e6, "verify": 134.9e6}


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


def percentiles(per_unit_ms):
    a = np.asarray(per_unit_ms, dtype=np.float64)
    return {"median": float(np.median(a)), "p10": float(np.percentile(a, 10)), "p90": float(np.percentile(a, 90)),
            "mean": float(a.mean()), "replays": int(a.size)}


def replay_timed(stream, enqueue, units_per_replay, min_window_s=0.25, min_replays=10, max_replays=2000,
                 barrier=None):
    """Device time of `enqueue()` (which puts `units_per_replay` units of work on `stream`), repeated
    until the timed window is at least `min_window_s`; every repetition lies between two CUDA
    events recorded on `stream`.  Returns (per-unit ms of every repetition, (t0, t1) host window)."""
    import torch
    with torch.cuda.stream(stream):
        enqueue()                                        # untimed: a graph's first replay pays the upload
        stream.synchronize()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        enqueue()
        p1.record(stream)
        stream.synchronize()
        probe_ms = max(p0.elapsed_time(p1), 1e-3)
        reps = int(min(max_replays, max(min_replays, math.ceil(1e3 * min_window_s / probe_ms))))
        events = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        if barrier is not None:
            barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        events[0].record(stream)
        for r in range(reps):
            enqueue()
            events[r + 1].record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        if barrier is not None:
            barrier()
        t1 = time.perf_counter()
    per_unit = [events[r].elapsed_time(events[r + 1]) / units_per_replay for r in range(reps)]
    return per_unit, (t0, t1)


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


def graph_of(stream, fn, n):
    """Captures fn(0..n-1) on `stream` into a CUDA graph; returns (graph, launches per replay)."""
    import torch
    from paper_2604_05250_b200 import binding as dd
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        c0 = dd.launch_count()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(n):
                fn(i)
        launches = dd.launch_count() - c0
    return graph, launches


def rotation(bytes_per_set, cap=24):
    """How many distinct input sets make consecutive launches miss L2."""
    return max(2, min(cap, int(2.2 * L2_BYTES // max(1, bytes_per_set)) + 1))


def device_logits(B, P, V, err, gen, want_drafter):
    """Logits drawn on the device by the recipe of synth.verify_inputs (verifier N(0, 2^2) with +8 at
    one token per position; drafter = verifier + N(0, 0.5^2), or an independent N(0, 2^2) row on a
    share `err` of the positions), rounded to bf16."""
    import torch
    dev = gen.device
    ver = torch.randn(B, P, V, device=dev, generator=gen)
    ver *= 2.0
    hot = torch.randint(0, V, (B, P, 1), device=dev, generator=gen)
    ver.scatter_add_(2, hot, torch.full((B, P, 1), 8.0, device=dev))
    dra = None
    if want_drafter:
        dra = torch.randn(B, P, V, device=dev, generator=gen)
        wrong = torch.rand(B, P, 1, device=dev, generator=gen) < err
        dra = torch.where(wrong, 2.0 * dra, ver + 0.5 * dra).to(torch.bfloat16)
    return dra, ver.to(torch.bfloat16)


def other_configs(dd, stream, sampler, peaks, quick=False):
    """Every workload shape other than the headline step, one entry each: median device time per
    launch over graph replays, algorithmic TFLOP/s or GB/s, roofline fractions, clocks."""
    import torch
    dev = torch.device("cuda", torch.cuda.current_device())
    gen = torch.Generator(device=dev)
    gen.manual_seed(4242)
    out = []
    window = 0.1 if quick else 0.25

    def record(name, op, shape, enqueue_one, n_sets, flops, nbytes, bound, note=None):
        # The inputs were drawn on the default stream and the launches go to `stream`: everything
        # queued so far has to finish first, both for the inputs themselves and because the caching
        # allocator may already have handed a generator's temporary (still to be read by a queued
        # kernel) to one of the output tensors.
        torch.cuda.synchronize()
        # a graph of enough launches to last a few milliseconds, replayed over the window
        with torch.cuda.stream(stream):
            for i in range(3):
                enqueue_one(i)
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            enqueue_one(0)
            e1.record(stream)
            stream.synchronize()
        one_ms = max(e0.elapsed_time(e1), 2e-3)
        n = int(min(200, max(n_sets, math.ceil(4.0 / one_ms))))
        n = ((n + n_sets - 1) // n_sets) * n_sets if n_sets <= 24 else n
        graph, launches = graph_of(stream, enqueue_one, n)
        per_launch, win = replay_timed(stream, graph.replay, n, min_window_s=window)
        st = percentiles(per_launch)
        sec = st["median"] * 1e-3
        entry = {"name": name, "op": op, "shape": shape, "ms": st["median"], "p10": st["p10"], "p90": st["p90"],
                 "replays": st["replays"], "launches_per_replay": n, "kernels_per_launch": launches // n,
                 "bound": bound, "clocks": sampler.summary(*win)}
        if flops:
            tf = flops / sec / 1e12
            entry.update(tflops=tf, frac_of_measured_burst=tf / peaks["bf16"],
                         frac_of_measured_sustained=tf / peaks["bf16_sustained"], frac_of_nominal_2250=tf / NOMINAL_BF16_TFLOPS)
        if nbytes:
            gb = nbytes / sec / 1e9
            entry.update(gbs=gb, algorithmic_bytes=nbytes, frac_of_measured_hbm=gb / peaks["hbm"],
                         frac_of_nominal_8000=gb / NOMINAL_HBM_GBS)
        if note:
            entry["note"] = note
        out.append(entry)
        del graph

    # ---- attention: the other configurations and the sequence-length sweep (H = 32, D = 128)
    att_shapes = [("cfg0 tiny", 1, 4, 128, 64, False), ("cfg2 batched serving", 16, 32, 512, 128, False),
                  ("cfg3 long context, planted rank-16 structure", 1, 32, 8192, 128, True)]
    att_shapes += [(f"sweep N={N}", 16384 // N, 32, N, 128, False) for N in synth.ATTENTION_SWEEP_N]
    att_shapes.append(("B=4 x N=1024", 4, 32, 1024, 128, False))
    for name, B, H, N, D, planted in att_shapes:
        per_set = 4 * B * H * N * D * 2
        ns = rotation(per_set)
        sets = []
        for _ in range(ns):
            q, k, v = (torch.randn(B, H, N, D, device=dev, generator=gen) for _ in range(3))
            if planted:
                # a shared rank-16 component of strength 3 in q and k (orthonormal W per head)
                w = torch.linalg.qr(torch.randn(B, H, D, 16, device=dev, generator=gen))[0].transpose(2, 3)
                q = q + 3.0 * torch.randn(B, H, N, 16, device=dev, generator=gen) @ w
                k = k + 3.0 * torch.randn(B, H, N, 16, device=dev, generator=gen) @ w
            sets.append(tuple(t.to(torch.bfloat16) for t in (q, k, v)))
        o = torch.empty(B, H, N, D, device=dev, dtype=torch.bfloat16)

        def call(i, sets=sets, o=o, D=D):
            q, k, v = sets[i % len(sets)]
            dd.bidir_attention(q, k, v, out=o, scale=D ** -0.5)
        flops = 4.0 * B * H * N * N * D
        bound = "tensor" if N >= 1024 else "hbm"
        record(name, "dd_bidir_attention", dict(B=B, H=H, N=N, D=D), call, ns, flops, float(per_set), bound,
               note=f"{ns} input sets in rotation" + ("; launch-bound" if N <= 128 else ""))
        del sets, o
    assert dd.attention_status() == 0

    # ---- the drafter's shape: a block of queries over stored keys
    for name, B, Nq, Nkv in [("drafter block B=64", 64, 32, 1024), ("drafter block B=16", 16, 32, 1024),
                             ("drafter block Nq=128 Nkv=4096", 16, 128, 4096)]:
        H, D = 32, 128
        per_set = (2 * Nkv + 2 * Nq) * B * H * D * 2
        ns = rotation(per_set)
        sets = [tuple(torch.randn(B, H, n, D, device=dev, generator=gen).to(torch.bfloat16) for n in (Nq, Nkv, Nkv))
                for _ in range(ns)]
        o = torch.empty(B, H, Nq, D, device=dev, dtype=torch.bfloat16)

        def call(i, sets=sets, o=o):
            q, k, v = sets[i % len(sets)]
            dd.block_attention(q, k, v, out=o)
        record(name, "dd_block_attention", dict(B=B, H=H, Nq=Nq, Nkv=Nkv, D=D), call, ns,
               4.0 * B * H * Nq * Nkv * D, float(per_set), "hbm" if Nq <= 256 else "tensor")
        del sets, o
    assert dd.attention_status() == 0

    # ---- verification: the other configurations and the vocabulary / masked-count sweep
    T, K_, C = synth.MODE_TRUST, synth.MODE_KL, synth.MODE_CONF
    ver_shapes = [("cfg0 tiny", 1, 128, 1024, 32, 0.10, 8, (T, K_, C)),
                  ("cfg2 batched serving", 16, 256, 126464, "uniform_25_100", 0.10, 16, (C,)),
                  ("cfg3 long context", 1, 512, 126464, "all", 0.10, 32, (T, K_))]
    for V in synth.VERIFY_SWEEP["V"]:
        for nflag in synth.VERIFY_SWEEP["flagged"]:
            modes = (T, K_, C) if (V == 126464 and nflag == 512) else (K_,)
            ver_shapes.append((f"sweep V={V} masked={nflag}", 1, 512, V, nflag, 0.20, 8 if nflag == 32 else 32, modes))
    # two shapes outside the configurations: a token excluded by both models (logit -inf at the same
    # index in every row, e.g. the mask token) on the cfg1 shape, and a sequence of 1024 positions
    ver_shapes.append(("cfg1 shape, one token excluded by both models", 1, 256, 126464, "all", 0.20, 32, (K_,)))
    ver_shapes.append(("P=1024 V=32000 masked=128", 1, 1024, 32000, 128, 0.20, 32, (K_,)))
    mode_name = {T: "TRUST", K_: "KL", C: "CONF"}
    for name, B, P, V, flagged, err, k, modes in ver_shapes:
        want_d = K_ in modes
        counts = synth.flag_counts(B, P, flagged, np.random.default_rng(7))
        flags_h = np.zeros((B, P), dtype=np.uint8)
        for b in range(B):
            flags_h[b, np.sort(np.random.default_rng(b).choice(P, size=counts[b], replace=False))] = 1
        n_flagged = int(flags_h.sum())
        flags = torch.from_numpy(flags_h).to(dev)
        per_set = n_flagged * V * 2 * (2 if want_d else 1)
        ns = rotation(per_set, cap=8)
        if B * P * V * 2 > (1 << 30):
            ns = 1                                   # one set is already many times the L2
        sets = [device_logits(B, P, V, err, gen, want_d) for _ in range(ns)]
        if "excluded" in name:
            for dra, ver in sets:
                dra[..., V - 128] = float("-inf")
                ver[..., V - 128] = float("-inf")
        tokens = torch.randint(0, V, (B, P), device=dev, dtype=torch.int32, generator=gen)
        ot = torch.empty(B, P, device=dev, dtype=torch.int32)
        om = torch.empty(B, P, device=dev, dtype=torch.uint8)
        osc = torch.empty(B, P, device=dev, dtype=torch.float32)
        for mode in modes:
            def call(i, sets=sets, mode=mode):
                dra, ver = sets[i % len(sets)]
                dd.verify(dra if mode == K_ else None, ver, tokens, flags, mode, 0.5, k, 0,
                          out_tokens=ot, out_mask=om, out_score=osc)
            nbytes = n_flagged * V * 2.0 * (2 if mode == K_ else 1) + B * P * 14.0
            record(f"{name} {mode_name[mode]}", "dd_verify", dict(B=B, P=P, V=V, flagged_rows=n_flagged, mode=mode_name[mode], k=k),
                   call, max(1, ns), 0.0, nbytes, "hbm",
                   note=(f"{ns} input sets in rotation" if ns > 1 else "one set, larger than the L2 many times over") +
                        ("; under 20 us: launch-bound" if nbytes < 2e7 else ""))
        if name.startswith("cfg2"):
            def call_u(i, sets=sets):
                dd.unmask(sets[i % len(sets)][1], tokens, flags, 0.5, 16, out_tokens=ot, out_mask=om, out_conf=osc)
            record("cfg2 shape, drafter's unmasking step", "dd_unmask", dict(B=B, P=P, V=V, masked_rows=n_flagged, k=16),
                   call_u, 1, 0.0, n_flagged * V * 2.0 + B * P * 14.0, "hbm")
        del sets
    assert dd.verify_status() == 0

    # ---- the verifier's language-model head fused with the verification algorithm (K = 4096)
    for name, B, P in [("fused LM head, cfg1 rows", 1, 256), ("fused LM head, cfg2 rows", 16, 256)]:
        K, V = 4096, 126464
        hs = [torch.randn(B, P, K, device=dev, generator=gen).to(torch.bfloat16) for _ in range(2)]
        ws = [(torch.randn(V, K, device=dev, generator=gen) * (2.0 / K ** 0.5)).to(torch.bfloat16) for _ in range(2)]
        tokens = torch.zeros(B, P, device=dev, dtype=torch.int32)
        flags = torch.ones(B, P, device=dev, dtype=torch.uint8)
        ot, om = torch.empty_like(tokens), torch.empty_like(flags)
        osc = torch.empty(B, P, device=dev, dtype=torch.float32)

        def call_lm(i, hs=hs, ws=ws):
            dd.lm_head_verify(None, None, hs[i % 2], ws[i % 2], tokens, flags, C, 0.5, 32, 0, out_tokens=ot, out_mask=om, out_score=osc)
        record(name, "dd_lm_head_verify", dict(B=B, P=P, K=K, V=V, mode="CONF", k=32), call_lm, 2,
               2.0 * B * P * K * V, float(V * K * 2 + B * P * K * 2), "tensor",
               note="two weight matrices in rotation (2 x 1.04 GB); bytes = weights and hidden states once")

        def call_lm_kl(i, hs=hs, ws=ws):
            dd.lm_head_verify(hs[(i + 1) % 2], ws[(i + 1) % 2], hs[i % 2], ws[i % 2], tokens, flags, K_, 0.5, 32, 0,
                              out_tokens=ot, out_mask=om, out_score=osc)
        record(name + ", KL (both heads)", "dd_lm_head_verify", dict(B=B, P=P, K=K, V=V, mode="KL", k=32), call_lm_kl, 2,
               4.0 * B * P * K * V, 2.0 * (V * K * 2 + B * P * K * 2), "tensor",
               note="the two matrices serve as drafter and verifier, roles swapped every call")
        del hs, ws
    assert dd.verify_status() == 0
    return out


def run_eager_other(dd, which, K, W):
    """K eagerly launched calls of one entry point on one of the other shapes (for profilers)."""
    import torch
    dev = torch.device("cuda", torch.cuda.current_device())
    gen = torch.Generator(device=dev)
    gen.manual_seed(99)
    if which == "drafter_block":
        B, H, Nq, Nkv, D = 64, 32, 32, 1024, 128
        sets = [tuple(torch.randn(B, H, n, D, device=dev, generator=gen).to(torch.bfloat16) for n in (Nq, Nkv, Nkv))
                for _ in range(2)]
        o = torch.empty(B, H, Nq, D, device=dev, dtype=torch.bfloat16)
        name = f"dd_block_attention B={B} H={H} Nq={Nq} Nkv={Nkv} D={D}"

        def call(i):
            q, k, v = sets[i % 2]
            dd.block_attention(q, k, v, out=o)
    elif which == "attention_cfg2":
        B, H, N, D = 16, 32, 512, 128          # many short work items: the persistent attention kernel
        sets = [tuple(torch.randn(B, H, N, D, device=dev, generator=gen).to(torch.bfloat16) for _ in range(3)) for _ in range(3)]
        o = torch.empty(B, H, N, D, device=dev, dtype=torch.bfloat16)
        name = f"dd_bidir_attention B={B} H={H} N={N} D={D}"

        def call(i):
            q, k, v = sets[i % 3]
            dd.bidir_attention(q, k, v, out=o)
    elif which in ("lm_head_small", "lm_head_small_kl"):
        # a small case of the fused head: 256 rows, K = 4096, a 32000-entry vocabulary (262 MB of
        # weights per matrix: larger than the L2, under 1 GB on the device)
        B, P, K_, V = 1, 256, 4096, 32000
        hs = [torch.randn(B, P, K_, device=dev, generator=gen).to(torch.bfloat16) for _ in range(2)]
        ws = [(torch.randn(V, K_, device=dev, generator=gen) * (2.0 / K_ ** 0.5)).to(torch.bfloat16) for _ in range(2)]
        tokens = torch.zeros(B, P, device=dev, dtype=torch.int32)
        flags = torch.ones(B, P, device=dev, dtype=torch.uint8)
        ot, om = torch.empty_like(tokens), torch.empty_like(flags)
        oc = torch.empty(B, P, device=dev, dtype=torch.float32)
        kl = which.endswith("_kl")
        name = f"dd_lm_head_verify {'KL' if kl else 'CONF'} on hidden [{B},{P},{K_}], weights [{V},{K_}]"

        def call(i):
            if kl:
                dd.lm_head_verify(hs[(i + 1) % 2], ws[(i + 1) % 2], hs[i % 2], ws[i % 2], tokens, flags, synth.MODE_KL,
                                  0.5, 32, 0, out_tokens=ot, out_mask=om, out_score=oc)
            else:
                dd.lm_head_verify(None, None, hs[i % 2], ws[i % 2], tokens, flags, synth.MODE_CONF, 0.5, 32, 0,
                                  out_tokens=ot, out_mask=om, out_score=oc)
    else:
        B, P, V = VER["B"], VER["P"], VER["V"]
        sets = [device_logits(B, P, V, 0.1, gen, False)[1] for _ in range(5)]
        tokens = torch.zeros(B, P, device=dev, dtype=torch.int32)
        flags = torch.ones(B, P, device=dev, dtype=torch.uint8)
        ot, om = torch.empty_like(tokens), torch.empty_like(flags)
        oc = torch.empty(B, P, device=dev, dtype=torch.float32)
        name = f"dd_unmask on logits [{B},{P},{V}], every position masked"

        def call(i):
            dd.unmask(sets[i % 5], tokens, flags, 0.5, 8, out_tokens=ot, out_mask=om, out_conf=oc)
    for i in range(W):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(K):
        call(i)
    e1.record()
    torch.cuda.synchronize()
    assert dd.attention_status() == 0 and dd.verify_status() == 0
    print(json.dumps({"mode": "eager-only", "workload": name, "steps": K, "warmup": W,
                      "ms_per_call": e0.elapsed_time(e1) / K}), flush=True)
    return 0


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
    barrier = (lambda: dist.barrier()) if distributed else None

    from paper_2604_05250_b200 import binding as dd
    from paper_2604_05250_b200 import build
    build.build()
    dd.lib()

    K, W = args.steps, max(3, args.warmup)
    if args.eager_only in ("drafter_block", "unmask_cfg1", "lm_head_small", "lm_head_small_kl", "attention_cfg2"):
        return run_eager_other(dd, args.eager_only, K, W)
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
    torch.cuda.synchronize()               # the inputs were copied on the default stream
    sampler.start()
    with torch.cuda.stream(stream):
        for i in range(W):
            step(i)
    stream.synchronize()
    assert dd.attention_status() == 0 and dd.verify_status() == 0

    if args.eager_only:
        # K eagerly launched steps and nothing else: the command profilers are pointed at
        with torch.cuda.stream(stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0 = dd.launch_count()
            e0.record(stream)
            for i in range(K):
                step(i)
            e1.record(stream)
            stream.synchronize()
        sampler.stop()
        if rank == 0:
            print(json.dumps({"mode": "eager-only", "workload": WORKLOAD, "steps": K, "warmup": W,
                              "ms_per_step": e0.elapsed_time(e1) / K, "gpu_launches": int(dd.launch_count() - c0)}),
                  flush=True)
        if distributed:
            dist.barrier()
            dist.destroy_process_group()
        return 0

    # ---- the K steps as a CUDA graph (in pieces of at most 200 steps), replayed over the window
    g = graph_chunk(K)

    def graph_runner(fn):
        graph, launches = graph_of(stream, fn, g)

        def run():
            for _ in range(K // g):
                graph.replay()
        return run, launches * (K // g), graph

    run_step, launches_per_pass, _g1 = graph_runner(step)
    per_step, window = replay_timed(stream, run_step, K, barrier=barrier)
    run_att, _, _g2 = graph_runner(attention_call)
    per_att, _ = replay_timed(stream, run_att, K, barrier=barrier)
    run_ver, _, _g3 = graph_runner(verify_call)
    per_ver, _ = replay_timed(stream, run_ver, K, barrier=barrier)
    clocks = sampler.summary(*window)

    # ---- the same steps launched eagerly through the C ABI (tensor maps encoded per call)
    eager_n = min(K, 200)

    def eager():
        for i in range(eager_n):
            step(i)
    per_eager, _ = replay_timed(stream, eager, eager_n, min_window_s=0.1, barrier=barrier)

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
    h2d = 3 * attention_bytes() / 4 + 2 * VER["B"] * VER["P"] * VER["V"] * 2 + VER["B"] * VER["P"] * 5
    d2h = attention_bytes() / 4 + VER["B"] * VER["P"] * 9
    assert dd.attention_status() == 0 and dd.verify_status() == 0

    # ---- max over ranks of every statistic
    st_step, st_att, st_ver, st_eager = (percentiles(x) for x in (per_step, per_att, per_ver, per_eager))
    keys = ("median", "p10", "p90", "mean")
    flat = [st[k] for st in (st_step, st_att, st_ver, st_eager) for k in keys] + [e2e_ms]
    flat = max_over_ranks(flat, dev, distributed)
    for n, st in enumerate((st_step, st_att, st_ver, st_eager)):
        for m, k in enumerate(keys):
            st[k] = flat[4 * n + m]
    e2e_ms = flat[-1]
    ms_step, att_step, ver_step = st_step["median"], st_att["median"], st_ver["median"]

    if rank == 0:
        peaks = measured_peaks()
        others = None
        if world == 1 and not args.no_other_configs:
            del att_dev, ver_dev
            torch.cuda.empty_cache()
            others = other_configs(dd, stream, sampler, peaks, quick=args.quick)
        sampler.stop()
        att_peak = peaks["bf16"]
        att_tflops = attention_flops() / (att_step * 1e-3) / 1e12
        ver_gbs = verify_bytes(n_flagged) / (ver_step * 1e-3) / 1e9
        kernels = {
            "attention": {"ms": att_step, "p10": st_att["p10"], "p90": st_att["p90"], "tflops": att_tflops,
                          "frac_of_nominal_2250": att_tflops / NOMINAL_BF16_TFLOPS,
                          "frac_of_measured": att_tflops / att_peak,
                          "peak_used": f"{att_peak} TFLOP/s (burst, {peaks['source']})"},
            "verify": {"ms": ver_step, "p10": st_ver["p10"], "p90": st_ver["p90"], "gbs": ver_gbs,
                       "frac_of_nominal_8000": ver_gbs / NOMINAL_HBM_GBS,
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
                       "launch": f"cuda_graph of {K} steps, replayed {st_step['replays']} times; value = median over replays",
                       "parallelism": f"replicas x{world}"},
            "latency": {"median_ms": st_step["median"], "p10_ms": st_step["p10"], "p90_ms": st_step["p90"],
                        "mean_ms": st_step["mean"], "replays": st_step["replays"],
                        "eager_median_ms": st_eager["median"], "eager_p10_ms": st_eager["p10"],
                        "eager_p90_ms": st_eager["p90"]},
            "throughput": {"value": world * 1e3 / ms_step, "unit": "verify_steps/s"},
            "clocks": clocks,
            "e2e": {"value": e2e_ms, "unit": "ms", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "steps": e2e_steps},
            "gpu_launches": int(launches_per_pass * st_step["replays"]),
            "roofline": roof,
            "kernels": kernels,
            "cpu_baseline": cpu,
        }
        if others is not None:
            line["other_configs"] = others
        print(json.dumps(line), flush=True)
    else:
        sampler.stop()
    if distributed:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def print_tables(path):
    """Markdown tables of a stored JSON line of this program (the last line of `path` that is one):
    the headline step, its two kernels, and every entry of `other_configs`."""
    with open(path) as f:
        d = json.loads([ln for ln in f if ln.startswith("{")][-1])
    ck, lat = d["clocks"], d["latency"]
    print(f"Headline ({d['config']['workload']}): {1e3 * d['value']:.2f} us per step (median; "
          f"p10 {1e3 * lat['p10_ms']:.2f}, p90 {1e3 * lat['p90_ms']:.2f}; eager launches "
          f"{1e3 * lat['eager_median_ms']:.2f} us); e2e {d['e2e']['value']:.3f} ms; SM clock median "
          f"{ck['sm_mhz']} of {ck['sm_max_mhz']} MHz, reasons {ck['reasons']}\n")
    print("| kernel | us | achieved | of measured | of nominal |")
    print("|---|---|---|---|---|")
    for name, k in d["kernels"].items():
        if "tflops" in k:
            print(f"| {name} | {1e3 * k['ms']:.2f} | {k['tflops']:.0f} TFLOP/s | {k['frac_of_measured']:.3f} (burst) | "
                  f"{k['frac_of_nominal_2250']:.3f} of 2250 |")
        else:
            print(f"| {name} | {1e3 * k['ms']:.2f} | {k['gbs']:.0f} GB/s | {k['frac_of_measured']:.3f} | "
                  f"{k['frac_of_nominal_8000']:.3f} of 8000 |")
    print("\n| workload | entry point | us (median) | p10 / p90 | achieved | of measured | of nominal | SM MHz (reasons) |")
    print("|---|---|---|---|---|---|---|---|")
    for e in d.get("other_configs", []):
        if e["bound"] == "tensor":
            perf = (f"{e['tflops']:.0f} TFLOP/s | {e['frac_of_measured_burst']:.3f} burst, "
                    f"{e['frac_of_measured_sustained']:.3f} sustained | {e['frac_of_nominal_2250']:.3f}")
        else:
            perf = f"{e['gbs']:.0f} GB/s | {e['frac_of_measured_hbm']:.3f} | {e['frac_of_nominal_8000']:.3f}"
        c = e["clocks"]
        print(f"| {e['name']} | {e['op']} | {1e3 * e['ms']:.1f} | {1e3 * e['p10']:.1f} / {1e3 * e['p90']:.1f} | {perf} | "
              f"{c['sm_mhz']} ({', '.join(c['reasons']) or 'none'}) |")
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-other-configs", action="store_true", help="time the headline step only")
    ap.add_argument("--quick", action="store_true", help="shorter timing windows for the other configurations")
    ap.add_argument("--eager-only", nargs="?", const="step", default=None, choices=["step", "drafter_block", "unmask_cfg1", "lm_head_small", "lm_head_small_kl", "attention_cfg2"],
                    help="launch K steps (or calls on one of the other shapes) eagerly and exit: for profilers")
    ap.add_argument("--tables", metavar="FILE", default=None,
                    help="print markdown tables of a stored JSON line of this program and exit (no GPU needed)")
    args = ap.parse_args()
    if args.tables:
        return print_tables(args.tables)
    if args.steps < 1:
        ap.error("--steps must be >= 1")
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
