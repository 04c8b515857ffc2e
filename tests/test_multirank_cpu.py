"""World-size-2 checks of the benchmark's multi-rank plumbing on CPU (gloo): the update has
no data-path collective, so ranks meet only to agree on the slowest rank's time; each rank
works on its own independently seeded tensor set; the reference arm runs on rank 0 only."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import bench
    from paper_2004_13336_b200 import workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = 1.0 + 0.5 * rank                       # rank 1 is the slow one
    agreed = bench.reduce_max(my_ms, "cpu")
    wl = W.tiny()
    wl.seed = bench.rank_seed(wl.seed, rank)
    g = W.make_grads_one(wl, 0, "cpu")
    mine = torch.tensor([float(g[0][0])], dtype=torch.float64)
    both = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(both, mine)
    out[rank] = (agreed, bench.job_value(wl.N, world, agreed), [float(b) for b in both])
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_own_distinct_tensors():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 1.5
    n = 45792
    assert res[0][1] == res[1][1] == 2 * n / 1.5e-3
    assert res[0][2] == res[1][2] and res[0][2][0] != res[0][2][1]     # different seeds, different data


def test_single_process_reduce_is_identity():
    import bench
    assert bench.reduce_max(2.5, "cpu") == 2.5
    assert bench.job_value(1000, 4, 2.0) == 4 * 1000 / 2e-3


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True)
    assert r.returncode == 0
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"
