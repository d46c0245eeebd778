"""World-size-2 check (gloo, CPU) of the rank plumbing the benchmark uses on several GPUs:
every rank draws its own batch, no data is exchanged, the reported throughput is the sum of
the units over the slowest rank's time, and the reference arm leaves the other ranks idle."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2502_00425_b200 import dist as D
    info = D.rank_info_from_env()
    D.init(info, backend="gloo")
    D.barrier()
    seconds = 2.0 if rank == 0 else 4.0          # rank 1 is the slow one
    value, t = D.aggregate_throughput(100.0 * (rank + 1), seconds)
    out.put((rank, info.is_main, D.batch_seed(1, rank), D.max_over_ranks(rank), D.sum_over_ranks(1.0), value, t))
    D.barrier()
    D.shutdown()


def test_two_rank_aggregation_over_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    rows = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in rows] == [True, False]
    assert rows[0][2] != rows[1][2]                       # different batch per rank
    for r in rows:
        assert r[3] == 1.0 and r[4] == 2.0                # max / sum over ranks
        assert r[5] == 300.0 / 4.0 and r[6] == 4.0        # all units / slowest rank


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_single_process_helpers_are_identities():
    sys.path.insert(0, ROOT)
    from paper_2502_00425_b200 import dist as D
    assert D.max_over_ranks(3.5) == 3.5 and D.sum_over_ranks(2.0) == 2.0
    assert D.aggregate_throughput(10.0, 2.0) == (5.0, 2.0)
    assert json.dumps(D.rank_info_from_env().__dict__)
