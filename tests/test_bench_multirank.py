"""Host-side logic of bench.py with more than one rank, on CPU (gloo, world size 2).

The path has no exchange step: ranks are independent replicas, so what a multi-rank run adds is
the rendezvous, the max-over-ranks timing and the rule that only rank 0 reports.
"""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def torchrun(nproc, script_args, port, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + script_args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_with_gloo(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import torch, torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, local_rank, world = bench.dist_env()
        assert world == 2 and rank == dist.get_rank()
        got = bench.max_over_ranks([1.0 + rank, 10.0 - rank, 5.0], torch.device("cpu"), True)
        dist.barrier()
        if rank == 0:
            print(json.dumps(got))
        dist.destroy_process_group()
    """))
    r = torchrun(2, [str(script)], 29631)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("[")]
    assert len(lines) == 1 and json.loads(lines[0]) == [2.0, 10.0, 5.0]


def test_reference_arm_reports_from_rank0_only():
    r = torchrun(2, ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"], 29632)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["metric"] == "verify_step_latency_ms" and d["higher_is_better"] is False
