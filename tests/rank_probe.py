"""Child script of test_dp_gloo.py::test_launch_ranks...: started by dp.launch_ranks as one of N CPU ranks,
it joins a gloo group, sums its rank + 1 over the group and writes what it saw to the folder given as argv[1]."""
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2507_19766_b200 import dp  # noqa: E402


def main():
    out_dir, expected = sys.argv[1], int(sys.argv[2])
    world, rank, local_rank = dp.world_from_env(expected)
    dist.init_process_group("gloo")
    t = torch.tensor([rank + 1], dtype=torch.int64)
    dist.all_reduce(t)
    with open(os.path.join(out_dir, f"rank{rank}"), "w") as f:
        f.write(f"{world} {local_rank} {int(t)}")
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
