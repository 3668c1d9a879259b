"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The path shards over images with no
exchange step, so what has to hold is host logic only: every rank draws its own batch, and the
whole-job figures are the slowest rank's time and the sum of the ranks' work."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2509_22323_b200 import inputs
    wl = inputs.WORKLOADS["tiny"]
    q = inputs.make_tensor(wl, 0, bench.rank_step(rank, 0), 0)
    ms, flops, launches = bench.aggregate(dist, torch.device("cpu"), 10.0 + 5.0 * rank, 1.0e9 * (rank + 1), 4 + rank)
    dist.barrier()
    torch.save({"ms": ms, "flops": flops, "launches": launches, "q_sum": float(q.float().abs().sum())},
               os.path.join(out_dir, f"r{rank}.pt"))
    dist.destroy_process_group()


def test_two_ranks_aggregate_and_draw_their_own_batches(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(tmp_path, f"r{r}.pt")) for r in range(world)]
    for r in res:
        assert r["ms"] == 15.0                  # max over ranks
        assert r["flops"] == 3.0e9              # sum over ranks
        assert r["launches"] == 9
    assert res[0]["q_sum"] != res[1]["q_sum"]   # different batches per rank


def test_single_process_aggregate_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(None, torch.device("cpu"), 1.5, 2.0, 3) == (1.5, 2.0, 3)
    assert bench.rank_step(0, 3) == 3 and bench.rank_step(2, 3) == 2003


def test_bench_refuses_more_gpus_than_visible_and_mismatched_world_size():
    """`python bench.py --gpus N` outside a launcher starts its N ranks itself; with fewer devices than that it
    refuses (exit 2) before doing any work, and under a launcher --gpus must agree with WORLD_SIZE."""
    import subprocess
    n_dev = torch.cuda.device_count()
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(n_dev + 2), "--steps", "3"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 2 and "CUDA device" in r.stderr and r.stdout.strip() == ""
    env["WORLD_SIZE"] = "4"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "3"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode != 0 and "WORLD_SIZE=4" in r.stderr
