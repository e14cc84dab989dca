"""Host-side logic of the N>1 benchmark path on CPU (gloo, world size 2): per-rank streams, max-over-ranks
timing, and the reference arm running on rank 0 only.  The path has no data-path collective: ranks are replicas."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.rank_workload("medium", 1 / 512, rank)
    tok, off = w.queries.materialize()
    mine = dict(seed=w.recipe["seed"], n=w.queries.n, head=tok[:8].tolist(), arr=w.arrivals[:4].tolist())
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    slow = bench.reduce_max([1.0 + rank, 5.0 - rank], torch.device("cpu"), True)
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump(dict(gathered=gathered, slow=slow), f)
    dist.destroy_process_group()


def test_two_ranks_get_their_own_streams_and_the_slowest_rank_decides(tmp_path):
    out = str(tmp_path / "r.json")
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    r = json.load(open(out))
    a, b = r["gathered"]
    assert a["seed"] != b["seed"] and a["n"] == b["n"]          # same recipe and size, different stream
    assert a["head"] != b["head"] and a["arr"] != b["arr"]
    assert r["slow"] == [2.0, 5.0]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True)
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
