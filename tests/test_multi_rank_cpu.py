"""World-size-2 check of the benchmark's multi-GPU plumbing on CPU (gloo): the path shards by tokens with
no data-path collective; ranks only meet in a barrier and a MAX reduction of their device times."""
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
    from paper_2607_02461_b200 import synth
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    # every rank draws its own tokens (weak scaling) and the same weights
    x = synth.activations(8, 256, 1000 + 1 + 100 * rank)
    w = synth.weights(16, 256, 2010)
    t = torch.tensor([1.5 + rank], dtype=torch.float64)       # this rank's "device time"
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    xs = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    ws = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(xs, torch.tensor([int(x.astype(np.int64).sum())]))
    dist.all_gather(ws, torch.tensor([int(w.astype(np.int64).sum())]))
    if rank == 0:
        print(json.dumps({"max_t": t.item(), "x": [int(v) for v in xs], "w": [int(v) for v in ws], "world": world}))
    dist.destroy_process_group()
""") % ROOT


def test_token_sharded_replicas_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    import json
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["world"] == 2
    assert out["max_t"] == 2.5                     # the slowest rank sets the step time
    assert out["x"][0] != out["x"][1]              # different tokens per rank
    assert out["w"][0] == out["w"][1]              # replicated weights


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0 and res.stdout.strip() == ""
