"""Child of tests/test_replicas_gloo.py: one rank of a CPU job started through replicas.launch."""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import torch.distributed as dist  # noqa: E402

from paper_2407_21018_b200 import replicas  # noqa: E402

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms, units = replicas.job_time_and_work(10.0 * (rank + 1), 1.0)
if rank == 0:
    with open(sys.argv[1], "w") as f:
        f.write(f"{world} {ms} {units}\n")
dist.destroy_process_group()
