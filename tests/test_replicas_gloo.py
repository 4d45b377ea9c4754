"""The N > 1 path of the benchmark on CPU: two gloo ranks run the replica plumbing (barrier, maximum of the per-rank
step times, whole-job throughput) that `bench.py --gpus N` runs over NCCL."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out_dir):
    import torch.distributed as dist
    from paper_2609_29812_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local = 40.0 + 5.0 * rank                 # rank 1 is the slow one
        dist.barrier()
        ms = replicas.max_over_ranks(ms_local, world)
        value = replicas.job_throughput(32768, world, ms)
        with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
            f.write(f"{ms!r} {value!r}")
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_job_total(tmp_path):
    import torch.multiprocessing as mp
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        ms, value = (float(x) for x in open(tmp_path / f"rank{rank}.txt").read().split())
        assert ms == 45.0                            # both ranks agree on the slowest replica's time
        assert value == pytest.approx(2 * 32768 / 45.0e-3)


def test_single_rank_needs_no_process_group():
    from paper_2609_29812_b200 import replicas
    assert replicas.max_over_ranks(12.5, 1) == 12.5
    assert replicas.job_throughput(1000, 1, 10.0) == pytest.approx(1.0e5)
