"""The benchmark's N > 1 path on CPU: two gloo ranks run the replica plumbing (barrier, maximum of
the per-rank times, whole-job rate) exactly as bench.py does over NCCL."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank: int, world: int, port: int, out_dir: str) -> None:
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2503_17922_b200 import replicas
    assert replicas.rank_env() == (rank, world, rank)
    replicas.init("gloo")
    replicas.barrier(sync_cuda=False)
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
    total_ms = replicas.max_over_ranks(my_ms)
    rate = replicas.whole_job_rate(32768, world, total_ms / 4)
    replicas.barrier(sync_cuda=False)
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{total_ms} {rate}")
    replicas.shutdown()


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    results = [open(tmp_path / f"rank{r}.txt").read().split() for r in range(world)]
    for total_ms, rate in results:
        assert float(total_ms) == 15.0                                   # the maximum over the ranks
        assert abs(float(rate) - 32768 * 2 / (15.0 / 4 * 1e-3)) < 1e-6   # both replicas count


def test_plain_command_starts_its_own_ranks():
    """`bench.py --gpus N` run without a launcher starts N ranks of itself; the same helper is driven
    here by a CPU stand-in for the timed call.  The slowest rank (rank 1 sleeps twice as long) sets
    the time, and both replicas count in the rate."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "replica_stub.py"), "2"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2
    assert rec["ms_per_step"] >= 4.0                         # rank 1's 4 ms per step, not rank 0's 2 ms
    assert abs(rec["value"] - 1000 * 2 / (rec["ms_per_step"] * 1e-3)) < 1e-6


def test_launcher_command_shape():
    sys.path.insert(0, ROOT)
    from paper_2503_17922_b200 import replicas
    cmd = replicas.launcher_command(4, "bench.py", ["--gpus", "4", "--steps", "7"], 29511)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert "--nproc-per-node=4" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-5:] == ["bench.py", "--gpus", "4", "--steps", "7"]


def test_single_process_is_a_noop():
    sys.path.insert(0, ROOT)
    from paper_2503_17922_b200 import replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.rank_env() == (0, 1, 0)
    replicas.init("gloo")
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(100, 1, 1.0) == 100000.0
