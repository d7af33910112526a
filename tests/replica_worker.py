"""Worker of test_bench_replicas.py: one rank of a world_size-2 gloo job on CPU."""
import os
import sys
from pathlib import Path

import torch
import torch.distributed as dist

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))
import bench  # noqa: E402


def main():
    rank, world, _ = bench.dist_env()
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{os.environ['MASTER_PORT']}",
                            rank=rank, world_size=world)
    dev = torch.device("cpu")
    # every replica times its own collectives; the job's time is the slowest rank's
    local_total_ms = 10.0 * (rank + 1)
    steps = 5
    total = bench.max_over_ranks(local_total_ms, dev, True)
    assert total == 10.0 * world, total
    value = bench.whole_job_value(world, 256, 65536, total / steps)
    want = world * 2 * 256 * 255 * 65536 / (total / steps * 1e-3) / 1e9
    assert abs(value - want) < 1e-9 * want
    dist.barrier()
    if rank == 0:
        print(f"ok {value:.3f}")
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
