"""A stand-in for one rank of a multi-GPU benchmark run, used by the launcher test on CPU: joins a
gloo group from the launcher's environment, feeds fixed per-rank byte counts and times through the
same aggregation the benchmark uses, and lets rank 0 print one JSON line. Launches no kernel."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import torch.distributed as dist                                   # noqa: E402

from paper_2510_00932_b200 import harness                          # noqa: E402

rank, local_rank, world = harness.dist_env()
dist.init_process_group("gloo")
assert dist.get_world_size() == world and dist.get_rank() == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
gbs, ms = harness.whole_job_gbs(1.0e9 * (rank + 1), 10.0 + 5.0 * rank)      # the last rank is the slow one
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": world, "value": gbs, "ms": ms, "argv": sys.argv[1:]}), flush=True)
dist.destroy_process_group()
