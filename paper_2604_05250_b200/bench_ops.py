"""Device timings of the library's calls on shapes other than the benchmark step.

    python -m paper_2604_05250_b200.bench_ops [--op attention|block_attention|verify|unmask|all]
                                              [--iters N] [--no-graph]

One JSON line per shape: CUDA-event time per call (graph replay of `iters` calls, inputs
rotating over more than twice the L2 so that every call reads HBM), the algorithmic TFLOP/s and
GB/s, and their fractions of the measured peaks (MEASURED_PEAKS.json beside bench.py if present,
else the fallback figures).  Inputs are seeded random tensors made on the device; this module
measures, it checks nothing (the parity tests do).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
L2_BYTES = 126 * 1024 * 1024


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def timed(fn, iters, use_graph):
    """Mean device time (us) of fn(i), i = 0..iters-1."""
    import torch
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for i in range(3):
            fn(i, s)
        s.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if use_graph:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for i in range(iters):
                    fn(i, s)
            g.replay()
            s.synchronize()
            e0.record(s)
            g.replay()
            e1.record(s)
        else:
            e0.record(s)
            for i in range(iters):
                fn(i, s)
            e1.record(s)
        s.synchronize()
    return e0.elapsed_time(e1) * 1e3 / iters


def emit(op, shape, us, flops, nbytes, status):
    hbm, bf16, src = peaks()
    tf, gb = flops / (us * 1e-6) / 1e12, nbytes / (us * 1e-6) / 1e9
    print(json.dumps({"op": op, "shape": shape, "us": round(us, 2), "tflops": round(tf, 1), "gbs": round(gb, 1),
                      "frac_tensor": round(tf / bf16, 3), "frac_hbm": round(gb / hbm, 3), "peaks": src,
                      "status": status}), flush=True)


def n_sets(bytes_per_set, cap=24):
    return max(2, min(cap, int(2.2 * L2_BYTES // max(1, bytes_per_set)) + 1))


def bench_attention(dd, iters, use_graph, block):
    import torch
    dev = torch.device("cuda")
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    if not block:
        shapes = [dict(B=1, H=32, Nq=1024, Nkv=1024), dict(B=16, H=32, Nq=512, Nkv=512), dict(B=4, H=32, Nq=1024, Nkv=1024),
                  dict(B=64, H=32, Nq=256, Nkv=256), dict(B=2, H=32, Nq=4096, Nkv=4096), dict(B=1, H=32, Nq=8192, Nkv=8192)]
    else:
        shapes = [dict(B=16, H=32, Nq=32, Nkv=1024), dict(B=64, H=32, Nq=32, Nkv=1024),
                  dict(B=64, H=32, Nq=32, Nkv=1024, ragged=True), dict(B=16, H=32, Nq=32, Nkv=1024, layout="bnhd"),
                  dict(B=16, H=32, Nq=128, Nkv=4096), dict(B=1, H=32, Nq=32, Nkv=1024)]
    D = 128
    for sh in shapes:
        B, H, Nq, Nkv = sh["B"], sh["H"], sh["Nq"], sh["Nkv"]
        layout = sh.get("layout", "bhnd")
        per_set = (2 * Nkv + Nq) * B * H * D * 2

        def mk(N):
            shape = (B, H, N, D) if layout == "bhnd" else (B, N, H, D)
            return torch.randn(*shape, device=dev, generator=g).to(torch.bfloat16)
        sets = [(mk(Nq), mk(Nkv), mk(Nkv)) for _ in range(n_sets(per_set))]
        out = torch.empty_like(sets[0][0])
        kv, keys = None, B * Nkv
        if sh.get("ragged"):
            kv = torch.randint(Nkv // 4, Nkv + 1, (B,), device=dev, dtype=torch.int32, generator=g)
            keys = int(kv.sum())
        it = max(10, min(iters, int(2e5 / max(1.0, per_set / 5e6))))

        def call(i, s):
            q, k, v = sets[i % len(sets)]
            if block:
                dd.block_attention(q, k, v, kv_len=kv, layout=layout, out=out, stream=s)
            else:
                dd.bidir_attention(q, k, v, out=out, stream=s)
        us = timed(call, it, use_graph)
        emit("block_attention" if block else "attention", sh, us, 4.0 * H * Nq * keys * D,
             (2 * keys + 2 * B * Nq) * H * D * 2, dd.attention_status())
        del sets, out


def bench_verify(dd, iters, use_graph, unmask):
    import torch
    dev = torch.device("cuda")
    g = torch.Generator(device=dev)
    g.manual_seed(2)
    shapes = [dict(B=1, P=256, V=126464), dict(B=16, P=256, V=126464, flagged=0.625), dict(B=1, P=512, V=126464),
              dict(B=1, P=512, V=32000)]
    for sh in shapes:
        B, P, V = sh["B"], sh["P"], sh["V"]
        tensors = 1 if unmask else 2
        per_set = B * P * V * 2 * tensors
        sets = []
        for _ in range(n_sets(per_set, cap=6)):
            ver = (torch.randn(B, P, V, device=dev, generator=g) * 2).to(torch.bfloat16)
            dra = None if unmask else (ver.float() + 0.5 * torch.randn(B, P, V, device=dev, generator=g)).to(torch.bfloat16)
            sets.append((dra, ver))
        tokens = torch.randint(0, V, (B, P), device=dev, dtype=torch.int32, generator=g)
        flags = (torch.rand(B, P, device=dev, generator=g) < sh.get("flagged", 1.0)).to(torch.uint8)
        ot = torch.empty(B, P, device=dev, dtype=torch.int32)
        om = torch.empty(B, P, device=dev, dtype=torch.uint8)
        osc = torch.empty(B, P, device=dev, dtype=torch.float32)
        it = max(10, min(iters, int(4e4 / max(1.0, per_set / 1e8))))

        def call(i, s):
            dra, ver = sets[i % len(sets)]
            if unmask:
                dd.unmask(ver, tokens, flags, 0.5, 8, out_tokens=ot, out_mask=om, out_conf=osc, stream=s)
            else:
                dd.verify(dra, ver, tokens, flags, dd.DD_MODE_KL, 0.5, 32, 7, out_tokens=ot, out_mask=om,
                          out_score=osc, stream=s)
        us = timed(call, it, use_graph)
        nflag = int(flags.sum())
        emit("unmask" if unmask else "verify_kl", dict(sh, flagged_rows=nflag), us, 0.0,
             nflag * V * 2.0 * tensors + B * P * 14.0, dd.verify_status())
        del sets


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="all", choices=["attention", "block_attention", "verify", "unmask", "all"])
    ap.add_argument("--iters", type=int, default=200)
    ap.add_argument("--no-graph", action="store_true")
    args = ap.parse_args()
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("needs a CUDA device: the library has no CPU fallback")
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    from paper_2604_05250_b200 import binding as dd
    from paper_2604_05250_b200 import build
    build.build()
    dd.lib()
    use_graph = not args.no_graph
    if args.op in ("attention", "all"):
        bench_attention(dd, args.iters, use_graph, block=False)
    if args.op in ("block_attention", "all"):
        bench_attention(dd, args.iters, use_graph, block=True)
    if args.op in ("verify", "all"):
        bench_verify(dd, args.iters, use_graph, unmask=False)
    if args.op in ("unmask", "all"):
        bench_verify(dd, args.iters, use_graph, unmask=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
