"""The multi-rank path of bench.py on CPU: two gloo ranks act as two replicas;
the job's value is all ranks' work over the slowest rank's time."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, results):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    r, w = bench.init_dist("gloo")
    assert (r, w) == (rank, world) and bench.dist_env() == (rank, rank, world)
    bench.barrier()
    slowest = bench.max_over_ranks(1.0 + rank)          # rank 1 is slower
    results[rank] = (slowest, bench.aggregate_value(10.0, world, slowest))
    bench.barrier()


def test_two_replicas_aggregate():
    world, port = 2, 29500 + os.getpid() % 2000
    mgr = mp.Manager()
    results = mgr.dict()
    mp.spawn(_worker, args=(world, port, results), nprocs=world, join=True)
    assert results[0] == results[1] == (2.0, 10.0)      # 2 ranks x 10 units / 2.0 s


def test_single_process_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_value(8.0, 4, 2.0) == 16.0
    peaks, kind = bench.load_peaks()
    assert peaks["hbm_gbs"] > 1000 and kind in ("measured", "fallback")


def test_gpus_flag_without_a_launcher_starts_the_replicas():
    # `bench.py --gpus N` run plainly starts N ranks itself; here through the reference arm, which needs no GPU:
    # rank 0 prints the one JSON line, the other rank exits quietly
    import json
    import subprocess
    code = ("import sys; sys.path.insert(0, %r); import bench; "
            "sys.exit(bench.spawn_replicas(2, ['--impl', 'reference', '--steps', '1', '--warmup', '0', '--gpus', '2']))" % ROOT)
    done = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=300)
    assert done.returncode == 0, done.stderr
    lines = [ln for ln in done.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
