"""CPU, two gloo ranks: the whole-job aggregation bench.py applies when it runs one replica per GPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r measured 10 + r ms, committed 100 * (r + 1) tokens, and 1000 * (r + 1) tokens/s end to end
    ms, tokens, e2e = bench.aggregate_over_ranks(dist, torch, 10.0 + rank, 100 * (rank + 1), 1000.0 * (rank + 1), "cpu")
    dist.barrier()
    out.put((rank, ms, tokens, e2e))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, tokens, e2e in got:
        assert ms == 11.0 and tokens == 300 and e2e == 3000.0


def test_single_rank_passes_values_through():
    import bench
    assert bench.aggregate_over_ranks(None, torch, 5.0, 7, 9.0, "cpu") == (5.0, 7, 9.0)


def test_asking_for_more_gpus_than_there_are_fails_loudly():
    """`python bench.py --gpus 2` outside a launcher starts the ranks itself; without two GPUs it must exit
    non-zero and print no result line (never a line that says n_gpus: 1)."""
    import subprocess
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        return
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "8"], capture_output=True,
                       text=True, timeout=300)
    assert r.returncode != 0
    assert "n_gpus" not in r.stdout and "GPU" in r.stderr
