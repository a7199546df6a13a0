"""A stand-in for the benchmark's rank path that needs no GPU: every rank "processes" a fixed number
of units per step on the CPU (a short sleep, longer on higher ranks) through the same replica
plumbing bench.py uses (launcher environment, gloo instead of nccl, barriers around the timed region,
maximum over the ranks, whole-job rate).  Rank 0 prints one JSON line.  Started by
tests/test_replicas_gloo.py through replicas.relaunch_under_launcher, as `bench.py --gpus N` starts
itself when it is run as a plain command."""
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2503_17922_b200 import replicas   # noqa: E402


def main() -> None:
    n = int(sys.argv[1])
    if not replicas.launcher_present():
        sys.exit(replicas.relaunch_under_launcher(n, os.path.abspath(__file__), sys.argv[1:]))
    rank, world, local = replicas.rank_env()
    assert world == n and 0 <= rank < n and local == rank
    replicas.init("gloo")
    t = {}
    ms = replicas.timed_region(lambda i: time.sleep(0.002 * (rank + 1)), steps=5, warmup=3,
                               start=lambda: t.__setitem__("t0", time.perf_counter()),
                               stop_ms=lambda: (time.perf_counter() - t["t0"]) * 1e3, sync_cuda=False)
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ms_per_step": ms / 5, "value": replicas.whole_job_rate(1000, world, ms / 5)}))
    replicas.shutdown()


if __name__ == "__main__":
    main()
