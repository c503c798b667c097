"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks run independent replicas and the
reported throughput is all ranks' units over the slowest rank's time (no data-path collective)."""

import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)

    def rmax(x):
        t = torch.tensor([x], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def rsum(x):
        t = torch.tensor([x], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    # rank 0 took 10 ms, rank 1 took 25 ms, 512 positions x 100 steps each
    local_ms = 10.0 if rank == 0 else 25.0
    value, total_ms = bench.aggregate_over_ranks(local_ms, 512.0 * 100, world, rmax, rsum)
    dist.barrier()
    out[rank] = (value, total_ms)
    dist.destroy_process_group()


def test_two_rank_aggregation_uses_slowest_rank_and_all_units():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        value, total_ms = out[rank]
        assert total_ms == 25.0
        assert value == pytest.approx(2 * 512 * 100 / 0.025)


def test_single_rank_aggregation_is_identity():
    value, total_ms = bench.aggregate_over_ranks(4.0, 2048.0, 1, lambda x: x, lambda x: x)
    assert total_ms == 4.0 and value == pytest.approx(2048.0 / 0.004)


def test_reference_arm_line_has_the_contract_keys(capsys, monkeypatch):
    """--impl reference prints one JSON line with the keys the contract names (tiny sample)."""
    import json
    monkeypatch.setattr(sys, "argv", ["bench.py", "--impl", "reference", "--steps", "1", "--warmup", "1", "--ref-rows", "1"])
    bench.main()
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "positions/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("chain FSD verify")
