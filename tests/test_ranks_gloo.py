"""The multi-GPU bookkeeping on two CPU processes (gloo): ownership of sequences, barrier,
max / sum over ranks and the whole-job throughput rule (all units over the slowest rank)."""

import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2602_01901_b200 import workloads as W
    from paper_2602_01901_b200.ranks import RankGroup, owned_sequences

    g = RankGroup(backend="gloo")
    mine = owned_sequences(5, g.rank, g.world)
    g.barrier()
    slow = g.max_over_ranks(1.0 + g.rank)          # rank 1 is the slow one
    total = g.sum_over_ranks(len(mine))
    tput, secs = g.throughput(units_this_rank=10.0 * (g.rank + 1), seconds_this_rank=2.0 + g.rank)
    # every rank draws the inputs of its own global sequences: disjoint data, same generator
    w = W.get_workload("tiny")
    first = W.draw_block_np(w.seed, W.T_DECODE_Q, [0], list(mine), [0], [0], 8)
    out.put((g.rank, list(mine), slow, total, tput, secs, first.tolist()))
    g.close()


def test_two_ranks_on_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, own0, slow0, tot0, tput0, secs0, d0), (r1, own1, slow1, tot1, tput1, secs1, d1) = results
    assert (r0, r1) == (0, 1)
    assert own0 == [0, 1, 2] and own1 == [3, 4]                   # disjoint, covering, sizes differ by <= 1
    assert slow0 == slow1 == 2.0                                   # max over ranks
    assert tot0 == tot1 == 5.0                                     # sum over ranks
    assert secs0 == secs1 == 3.0 and tput0 == tput1 == pytest.approx(30.0 / 3.0)
    assert d0 != d1[: len(d0)]                                      # different sequences, different values


def test_single_process_is_identity():
    from paper_2602_01901_b200.ranks import RankGroup, owned_sequences

    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    g = RankGroup()
    assert (g.rank, g.world) == (0, 1)
    assert g.max_over_ranks(3.5) == 3.5 and g.sum_over_ranks(2.0) == 2.0
    assert list(owned_sequences(7, 0, 1)) == list(range(7))
    parts = [list(owned_sequences(10, r, 4)) for r in range(4)]
    assert sum(parts, []) == list(range(10)) and max(map(len, parts)) - min(map(len, parts)) <= 1
    with pytest.raises(ValueError):
        owned_sequences(4, 2, 2)


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` without torchrun re-launches itself as two ranks; the reference arm
    (the CPU oracle; needs no GPU) answers with the number of ranks that took part."""
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--dist-backend", "gloo", "--workload", "tiny"], capture_output=True, text=True, timeout=600,
                         env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                       # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
