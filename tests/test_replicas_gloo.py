"""The multi-GPU path of the benchmark is N independent replicas plus measurement plumbing (barrier, max over ranks).
These tests run that plumbing as two `gloo` processes on CPU, rendezvous on 127.0.0.1."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_ranks(body: str, world: int = 2, timeout: int = 120):
    script = textwrap.dedent("""
        import json, os, sys
        sys.path.insert(0, %r)
        from paper_2101_03961_b200.replicas import Replicas
        reps = Replicas("gloo")
    """ % ROOT) + textwrap.dedent(body) + "\nreps.close()\n"
    port = _free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=timeout)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_max_over_ranks_and_single_reporter():
    outs = _run_ranks("""
        reps.barrier()
        slowest = reps.max_over_ranks(10.0 + 5.0 * reps.rank)          # rank 1 is slower: 15 ms
        value = reps.tokens_per_second(32768, slowest)
        if reps.is_reporting_rank:
            print(json.dumps({"n_gpus": reps.world, "ms": slowest, "value": value}))
    """)
    assert outs[1].strip() == ""                                       # only rank 0 prints the line
    line = json.loads(outs[0])
    assert line["n_gpus"] == 2 and line["ms"] == 15.0
    assert abs(line["value"] - 2 * 32768 / 15e-3) < 1e-6               # whole-job tokens/s at the slowest rank's time


def test_ranks_see_their_own_environment():
    outs = _run_ranks("""
        print(json.dumps({"rank": reps.rank, "world": reps.world, "local": reps.local_rank,
                          "max": reps.max_over_ranks(float(reps.rank))}))
    """)
    seen = sorted((json.loads(o)["rank"], json.loads(o)["local"], json.loads(o)["max"]) for o in outs)
    assert seen == [(0, 0, 1.0), (1, 1, 1.0)]


def test_single_process_needs_no_process_group():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, "-c", textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        from paper_2101_03961_b200.replicas import Replicas
        import torch.distributed as dist
        r = Replicas()
        r.barrier()
        assert r.world == 1 and r.is_reporting_rank and not dist.is_initialized()
        assert r.max_over_ranks(3.5) == 3.5 and r.tokens_per_second(1000, 2.0) == 500000.0
        r.close()
        print("ok")
    """ % ROOT)], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stderr[-2000:]


def test_reference_arm_other_ranks_do_no_work():
    # under torchrun the CPU-oracle arm runs on rank 0 only; other ranks exit 0 without output
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == "", out.stderr[-2000:]
