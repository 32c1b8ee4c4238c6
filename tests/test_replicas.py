"""The multi-GPU path is "replicas only": ranks own disjoint sequences and share nothing but the timing
reduction.  These tests run that host logic with two gloo ranks on CPU, and check that the benchmark's
reference arm stays silent on every rank but 0."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_00528_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rep = replicas.replica_from_env()
        ids = replicas.sequence_ids(rep, 3)
        # every rank "measures" its own time; the job's figure is the slowest rank's
        mine = 1.0 + 0.5 * rank
        slowest = replicas.max_over_ranks(mine, dist)
        gathered = [None] * world
        dist.all_gather_object(gathered, ids)
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump({"ids": ids, "all_ids": gathered, "slowest": slowest, "reporter": rep.is_reporter,
                       "rate": replicas.whole_job_rate(10, world, slowest)}, f)
    finally:
        dist.destroy_process_group()


def test_two_ranks_own_disjoint_sequences_and_agree_on_the_slowest_time(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    assert res[0]["ids"] == [0, 1, 2] and res[1]["ids"] == [3, 4, 5]
    flat = sorted(i for ids in res[0]["all_ids"] for i in ids)
    assert flat == list(range(6))                               # disjoint and covering
    assert res[0]["slowest"] == res[1]["slowest"] == 1.5        # max over ranks, identical on both
    assert [r["reporter"] for r in res] == [True, False]
    assert res[0]["rate"] == pytest.approx(2 * 10 / 1.5)        # whole-job aggregate, weak scaling


def test_single_process_is_identity():
    rep = replicas.replica_from_env({})
    assert (rep.rank, rep.local_rank, rep.world) == (0, 0, 1) and rep.is_reporter
    assert replicas.sequence_ids(rep, 4) == [0, 1, 2, 3]
    assert replicas.max_over_ranks(2.5) == 2.5
    with pytest.raises(ValueError):
        replicas.whole_job_rate(1, 1, 0.0)
    with pytest.raises(ValueError):
        replicas.sequence_ids(replicas.Replica(2, 0, 2), 1)


def test_reference_arm_prints_nothing_on_other_ranks():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_product_path_refuses_to_run_without_a_gpu():
    if torch.cuda.is_available():
        pytest.skip("needs a box without a GPU")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1"], capture_output=True,
                       text=True, timeout=300)
    assert p.returncode != 0 and "no CPU fallback" in (p.stderr + p.stdout)
