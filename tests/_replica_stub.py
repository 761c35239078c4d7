"""A stand-in for bench.py's measurement under the replica launcher: the same bookkeeping (process group from the
launcher's environment, barrier, slowest rank's time, whole-job rate, one JSON line from rank 0) around a stubbed
step, on CPU with the gloo backend."""
import argparse
import json
import os
import sys

import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
from paper_2602_08404_b200 import replicas as R  # noqa: E402

ap = argparse.ArgumentParser()
ap.add_argument("--gpus", type=int, default=1)
ap.add_argument("--steps", type=int, default=1)
args = ap.parse_args()
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
R.barrier()
ms_per_step = R.max_over_ranks(0.040 + 0.010 * rank)      # the stubbed step: rank r "takes" 40 + 10 r microseconds
R.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": R.world_size(), "asked": args.gpus, "steps": args.steps, "ms_per_step": ms_per_step,
                      "value": R.whole_job_rate(4, ms_per_step)}))
dist.destroy_process_group()
