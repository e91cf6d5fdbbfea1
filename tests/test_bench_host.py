"""Host logic of the benchmark, on CPU: the multi-rank aggregation (gloo, world_size 2), the byte model and
the clock-sample parsing."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    dist.barrier()
    # rank 1 is slower: the job's time is the max over ranks, its tokens the sum over ranks
    value, tmax = bench.aggregate(tokens_per_rank=800.0, seconds_this_rank=1.0 + rank, world=world)
    ret[rank] = (value, tmax)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_over_gloo():
    world, port = 2, _free_port()
    ret = mp.Manager().dict()
    mp.spawn(_rank_main, args=(world, port, ret), nprocs=world, join=True)
    for rank in range(world):
        value, tmax = ret[rank]
        assert tmax == 2.0 and value == 2 * 800.0 / 2.0


def test_single_rank_aggregation_and_byte_model():
    assert bench.aggregate(100.0, 0.5, 1) == (200.0, 0.5)
    # K and V bf16 read once + three 4-byte statistics read and written
    assert bench.algorithmic_bytes_per_unit_step(1024, 128, 2) == 4 * 1024 * 128 + 24 * 1024


def test_clock_sample_parsing():
    s = bench.ClockSampler(0)
    s.proc = type("P", (), {"terminate": lambda self: None})()
    row = lambda mhz, cap: ["0", str(mhz), "1965", "700.1", "0x4", "Not Active", "Not Active", "Not Active", cap]
    s.rows = [(1.0, row(1900, "Not Active")), (1.1, row(1700, "Active")), (1.2, row(1800, "Active")), (9.0, row(300, "Not Active"))]
    out = s.stop(0.9, 1.3)
    assert out["sm_mhz"] == 1800 and out["sm_max_mhz"] == 1965 and out["reasons"] == ["sw_power_cap"]
