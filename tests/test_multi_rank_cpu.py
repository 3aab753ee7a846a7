"""World-size-2 check of the benchmark's multi-GPU plumbing on CPU (gloo).  The path shards by tokens with no
data-path collective; ranks only meet in a barrier and a MAX reduction of their device times.  The worker calls the
functions bench.py itself runs on every rank (init_ranks, rank0_first, barrier_all, max_over_ranks,
whole_job_tflops, finish_ranks), with the gloo backend in place of nccl."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    import numpy as np, torch, torch.distributed as dist
    sys.path.insert(0, %r)
    import bench
    from paper_2607_02461_b200 import synth
    rank, world, local = bench.init_ranks("gloo")
    marker = sys.argv[1]
    # rank 0 "builds" first; the other ranks must see the result once they are past the barrier
    bench.rank0_first(rank, world, lambda: open(marker, "w").write("built"))
    seen = os.path.exists(marker)
    # every rank draws its own tokens (weak scaling) and the same weights
    x = synth.activations(8, 256, 1000 + 1 + 100 * rank)
    w = synth.weights(16, 256, 2010)
    bench.barrier_all(world, cuda=False)
    ms = bench.max_over_ranks(1.5 + rank, world)             # this rank's "device time"
    value = bench.whole_job_tflops(world, 3.0e9, ms)
    xs = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    ws = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    ok = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(xs, torch.tensor([int(x.astype(np.int64).sum())]))
    dist.all_gather(ws, torch.tensor([int(w.astype(np.int64).sum())]))
    dist.all_gather(ok, torch.tensor([int(seen)]))
    if rank == 0:
        print(json.dumps({"max_t": ms, "value": value, "x": [int(v) for v in xs], "w": [int(v) for v in ws],
                          "seen": [int(v) for v in ok], "world": world}))
    bench.finish_ranks(world)
""") % ROOT


def test_token_sharded_replicas_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(script), str(tmp_path / "built.marker")]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["world"] == 2
    assert out["max_t"] == 2.5                     # the slowest rank sets the step time
    assert abs(out["value"] - 2 * 3.0e9 / 2.5e-3 / 1e12) < 1e-12      # both ranks' work over that time
    assert out["seen"] == [1, 1]                   # nobody passed the barrier before rank 0 had "built"
    assert out["x"][0] != out["x"][1]              # different tokens per rank
    assert out["w"][0] == out["w"][1]              # replicated weights


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    env = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        assert bench.init_ranks("gloo") == (0, 1, 0)
        assert bench.max_over_ranks(3.25, 1) == 3.25
        assert bench.rank0_first(0, 1, lambda: 7) == 7
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v


def test_gpus_flag_starts_its_own_ranks(monkeypatch):
    """`python bench.py --gpus 2` without a launcher re-runs itself under torch.distributed.run with two local ranks;
    under a launcher (WORLD_SIZE set) or with one GPU it does not."""
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    calls = []
    monkeypatch.setattr(subprocess, "call", lambda cmd: calls.append(cmd) or 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "3"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    try:
        bench.spawn_ranks_if_needed(argparse.Namespace(gpus=2))
        raised = None
    except SystemExit as e:
        raised = e.code
    assert raised == 0 and len(calls) == 1
    cmd = calls[0]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd
    assert cmd[cmd.index("--nproc-per-node") + 1] == "2" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "2", "--steps", "3"] and cmd[-5].endswith("bench.py")
    monkeypatch.setenv("WORLD_SIZE", "2")
    assert bench.spawn_ranks_if_needed(argparse.Namespace(gpus=2)) is False
    monkeypatch.delenv("WORLD_SIZE")
    assert bench.spawn_ranks_if_needed(argparse.Namespace(gpus=1)) is False
    assert len(calls) == 1


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0 and res.stdout.strip() == ""
