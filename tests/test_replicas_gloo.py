"""The N > 1 path on CPU: two gloo ranks exercise the host logic that `bench.py --gpus N` runs per GPU
(rank discovery, per-replica seeds, barrier, max over ranks, whole-job throughput).  The data path has no
collective: replicas only."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.multiprocessing as mp

from paper_2508_12801_b200 import replicas, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    info = replicas.rank_info()
    assert (info.rank, info.local_rank, info.world) == (rank, rank, world)
    assert replicas.init_group(info, "gloo")
    replicas.barrier(info)
    ms_local = 5.0 + 3.0 * rank                                   # rank 1 is the slow one
    ms_max = replicas.max_over_ranks(info, ms_local)
    wl = synth.scaled(synth.WORKLOADS["tiny"], T=64)
    H = synth.hidden(wl, replicas.replica_seed(info))
    rec = {"rank": rank, "ms_max": ms_max, "value": replicas.aggregate_tokens_per_s(info, 1000, ms_max),
           "h_sum": float(H.double().sum())}
    replicas.barrier(info)
    replicas.shutdown(info)
    with open(out + f".{rank}", "w") as f:
        json.dump(rec, f)


def test_two_ranks_agree_on_the_slowest_time(tmp_path):
    port, out = _free_port(), str(tmp_path / "rec")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    recs = [json.load(open(out + f".{r}")) for r in range(2)]
    assert recs[0]["ms_max"] == recs[1]["ms_max"] == 8.0          # the max, seen by both
    assert recs[0]["value"] == pytest.approx(2 * 1000 / 8e-3)     # whole job: both batches in the slowest time
    assert recs[0]["h_sum"] != recs[1]["h_sum"]                   # replicas route different batches


def test_single_process_needs_no_group():
    info = replicas.rank_info({})
    assert (info.rank, info.local_rank, info.world) == (0, 0, 1)
    assert replicas.init_group(info, "gloo") is False
    assert replicas.max_over_ranks(info, 3.5) == 3.5
    assert replicas.aggregate_tokens_per_s(info, 65536, 6.4) == pytest.approx(65536 / 6.4e-3)
    replicas.barrier(info); replicas.shutdown(info)
    with pytest.raises(ValueError):
        replicas.rank_info({"RANK": "2", "WORLD_SIZE": "2"})


def test_reference_arm_runs_on_rank_0_only():
    """`bench.py --impl reference` under a 2-rank launch: rank 1 exits 0 without output, rank 0 prints the line."""
    outs = []
    for rank in (0, 1):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2")
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--steps", "1", "--warmup", "0", "--workload", "tiny", "--ref-tokens", "128"],
                           env=env, capture_output=True, text=True, timeout=600, cwd=ROOT)
        assert r.returncode == 0, r.stderr[-2000:]
        outs.append(r.stdout.strip())
    assert outs[1] == ""
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
