"""The N > 1 bookkeeping of the benchmark on CPU: two gloo ranks, one process each.

Checks that ranks own different batches of the same shape, that the time reduction is a max seen by every
rank, that the reference arm prints on rank 0 only, and that token sharding needs no exchange: the
per-rank plans (computed by the oracle here) add up to the plan statistics of the concatenated batch.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import shard, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert shard.env_rank_world() == (rank, rank, world)
        base = synth.WORKLOADS["tiny"]
        w = shard.rank_workload(base, rank)
        idx = synth.make_idx(w)
        counts = orc.plan(idx, None, w.E_tgt)[0]
        # every rank sees the slowest rank's time
        mine = 10.0 + 5.0 * rank
        slowest = shard.max_over_ranks(mine, torch.device("cpu"), world)
        shard.barrier(world)
        # gather the shards on rank 0 to compare with the concatenated batch
        gathered = [None] * world
        dist.all_gather_object(gathered, (idx, counts, slowest, (w.T, w.d, w.ffn, w.k)))
        if rank == 0:
            np.save(os.path.join(out_dir, "ok.npy"), np.array([1]))
            idxs = [g[0] for g in gathered]
            assert not np.array_equal(idxs[0], idxs[1]), "ranks must own different batches"
            assert all(g[3] == gathered[0][3] for g in gathered), "same shapes on every rank (weak scaling)"
            assert all(g[2] == 10.0 + 5.0 * (world - 1) for g in gathered)
            whole = orc.plan(np.concatenate(idxs, axis=0), None, w.E_tgt)[0]
            assert np.array_equal(whole, sum(g[1] for g in gathered))
            assert whole.sum() == world * w.R
            assert shard.job_tokens_per_sec(world, w.T, 2.0) == world * w.T / 2e-3
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_tokens_without_exchange(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert os.path.exists(tmp_path / "ok.npy")


def test_reference_arm_prints_on_rank0_only():
    env = dict(os.environ, WORLD_SIZE="2", LOCAL_RANK="1", RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env.update(LOCAL_RANK="0", RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
