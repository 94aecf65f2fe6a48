"""Worker of the world_size-2 gloo test: exercises bench.py's replica plumbing
(rendezvous on 127.0.0.1, barrier, max-over-ranks, whole-job value) on CPU."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def main():
    rank, _, world = bench._dist_env()
    dist = bench.init_replicas(world, backend="gloo")
    assert dist is not None and dist.get_world_size() == world
    dist.barrier()
    my_ms = 100.0 + 50.0 * rank                      # rank 1 is the slow replica
    ms = bench.max_over_ranks(my_ms, dist)
    value = bench.whole_job_value(world, 8 * 128, ms)
    dist.barrier()
    print(json.dumps({"rank": rank, "ms": ms, "value": value}))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
