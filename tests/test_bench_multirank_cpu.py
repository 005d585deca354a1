"""Host logic of the N > 1 benchmark path on CPU (gloo, world_size 2): the path shards by
replication with no data-path collective; the only exchange is the max-over-ranks of the timing,
and the reported value is the whole-job throughput."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    slowest = bench.max_over_ranks(local_ms)
    value = bench.job_value(tokens_per_rank=16384, steps=4, world=world, max_ms_total=slowest)
    dist.barrier()
    if rank == 0:
        torch.save({"slowest": slowest, "value": value}, out)
    dist.destroy_process_group()


def test_two_ranks_report_max_time_and_whole_job_value(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = torch.load(out)
    assert got["slowest"] == 15.0
    assert abs(got["value"] - 2 * 16384 * 4 / 15e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.job_value(100, 2, 1, 1000.0) == 200.0
    work = bench.algorithmic_work(__import__("paper_2506_08373_b200.workloads", fromlist=["x"]).CONFIGS[1], 32, 16384)
    assert abs(work["flops_one_pass"] - 4.12e11) / 4.12e11 < 0.01          # one contraction at config 1
    assert abs(work["gather_bytes"] + work["select_bytes"] - 286e6) / 286e6 < 0.02
