"""World-size-2 gloo run of the benchmark's multi-rank logic (sharding by batch, max-over-ranks timing)."""
import json
import os
import socket
import subprocess
import sys
import textwrap


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_rank_batches_and_max_reduce_with_gloo(repo_root, tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import json, os, sys
        sys.path.insert(0, {repo_root!r})
        import torch, torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        w = bench.load_workload("tiny", seed_shift=rank)              # every rank draws its own batch
        digest = float(w.q.float().abs().sum())
        value, ms = bench.aggregate_over_ranks(dist, torch.device("cpu"), kv_bytes=1000 * (rank + 1),
                                               steps=4, total_ms=10.0 * (rank + 1))
        out = [None] * world
        dist.all_gather_object(out, (rank, digest, value, ms))
        if rank == 0:
            print(json.dumps(out))
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", env["MASTER_PORT"], str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("[[")][-1]
    got = json.loads(line)
    assert [g[0] for g in got] == [0, 1]
    assert got[0][1] != got[1][1]                      # different seeds -> different batches
    # time = max over ranks (20 ms), bytes = sum over ranks (3000 per step, 4 steps)
    for g in got:
        assert abs(g[3] - 20.0) < 1e-9
        assert abs(g[2] - 3000 * 4 / (20.0e-3) / 1e12) < 1e-18
