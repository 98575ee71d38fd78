"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (no data-path
collective); the job's time is the slowest rank's and its work the sum over ranks."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2407_21018_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, units = replicas.job_time_and_work(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    thr = replicas.job_throughput(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    dist.barrier()
    out[rank] = (ms, units, thr)
    dist.destroy_process_group()


def test_two_replicas_aggregate():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank, args=(world, 29000 + os.getpid() % 2000, out), nprocs=world, join=True)
        for r in range(world):
            ms, units, thr = out[r]
            assert ms == 15.0            # slowest rank
            assert units == 300.0        # all ranks' work
            assert abs(thr - 300.0 / 15e-3) < 1e-6


def test_single_replica_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2407_21018_b200 import replicas
    assert replicas.job_time_and_work(3.0, 7.0) == (3.0, 7.0)


def test_launch_starts_the_asked_number_of_ranks(tmp_path):
    """The path `bench.py --gpus N` takes when it is started as ONE process: it re-launches itself as N
    ranks through replicas.launch.  Here the ranks are CPU processes on gloo."""
    sys.path.insert(0, ROOT)
    from paper_2407_21018_b200 import replicas
    out = tmp_path / "ranks.txt"
    rc = replicas.launch(2, os.path.join(ROOT, "tests", "_replica_probe.py"), [str(out)],
                         port=31000 + os.getpid() % 2000)
    assert rc == 0
    world, ms, units = out.read_text().split()
    assert int(world) == 2 and float(ms) == 20.0 and float(units) == 2.0
