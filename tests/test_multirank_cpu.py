"""The N > 1 path of the benchmark is N independent replicas plus one timing reduction; this covers
the reduction and the rank logic with two gloo ranks on the CPU."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    dist.barrier()
    # whole-job value = units of all ranks / the slowest rank's time
    per_rank_bytes = bench.exchange_bytes(4, 1 << 12, 4, 1000)
    value = world * per_rank_bytes / (ms * 1e-3) / 1e9
    torch.save({"ms": ms, "value": value}, os.path.join(out, "r%d.pt" % rank))
    dist.destroy_process_group()


def test_two_rank_timing_reduction(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = torch.load(tmp_path / "r0.pt")
    r1 = torch.load(tmp_path / "r1.pt")
    assert r0["ms"] == r1["ms"] == 15.0
    assert r0["value"] == r1["value"]


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--impl", "reference", "--steps", "1", "--warmup", "1"])
    bench.main()
    assert capsys.readouterr().out.strip() == ""               # other ranks exit without work or output
