"""Run by tests/test_bench_dist.py under torch.distributed.run with two CPU ranks (gloo): exercises the
rendezvous, barrier and max-over-ranks helpers that bench.py uses when it is launched on several GPUs."""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main() -> int:
    world, rank, local = bench.dist_setup(2)
    assert world == 2 and rank in (0, 1) and local == rank
    bench.barrier_and_sync(world)
    # every rank times its own replica; the job's time is that of the slowest one
    mine = 10.0 + 5.0 * rank
    worst = bench.max_over_ranks(mine, world)
    assert worst == 15.0, worst
    # whole-job value: units of all ranks over the slowest rank's time (weak scaling, replicas)
    per_step_units, steps = 3.0, 7
    value = world * per_step_units * steps / (worst / 1e3)
    assert abs(value - 2 * 3.0 * 7 / 0.015) < 1e-9
    bench.barrier_and_sync(world)
    import torch.distributed as dist
    dist.destroy_process_group()
    if rank == 0:
        print("DIST_PROBE_OK")
    return 0


if __name__ == "__main__":
    sys.exit(main())
