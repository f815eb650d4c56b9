"""Multi-rank host logic of the benchmark ("replicas only": no data-path collective), run as two gloo
ranks on CPU: every rank gets its own seed, the timing is the maximum over ranks, the reported value is the
work of all ranks over that time, and only rank 0 runs the reference arm."""
import importlib.util
import os
import socket
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def load_bench():
    spec = importlib.util.spec_from_file_location("bench_module", ROOT / "bench.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench = load_bench()
    local_ms = 10.0 + 5.0 * rank                         # rank 1 is the slow one
    ms_max = bench.max_over_ranks(local_ms, torch.device("cpu"), world)
    value = bench.whole_job_rate(128, world, ms_max * 1e-3)
    seed = bench.replica_seed(20260711, rank)
    Path(out_dir, f"rank{rank}.txt").write_text(f"{ms_max} {value} {seed}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_time_is_max_and_value_is_whole_job(tmp_path):
    world, port = 2, free_port()
    mp.spawn(worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [Path(tmp_path, f"rank{r}.txt").read_text().split() for r in range(world)]
    for r, (ms_max, value, seed) in enumerate(got):
        assert float(ms_max) == 15.0                     # every rank sees the slowest rank's time
        assert abs(float(value) - 2 * 128 / 15e-3) < 1e-6
        assert int(seed) == 20260711 + 1000 * r          # replicas do not share inputs
    assert got[0][2] != got[1][2]


def test_single_rank_needs_no_process_group():
    bench = load_bench()
    assert bench.max_over_ranks(3.5, torch.device("cpu"), 1) == 3.5
    assert bench.whole_job_rate(10, 1, 2.0) == 5.0


def test_reference_arm_is_silent_on_other_ranks(monkeypatch, capsys):
    bench = load_bench()
    monkeypatch.setenv("RANK", "1")
    args = type("A", (), dict(workload="cfg1", warmup=1, steps=1, gpus=2))()
    bench.run_reference(args)                            # must return without touching the oracle
    assert capsys.readouterr().out == ""
