"""The N > 1 path on CPU: two `gloo` ranks.  Units (layer, sequence, KV head) are independent, so
ranks share no data: each draws its own batch (seeds shifted by the rank) and the only
communication is the max-over-ranks of the step time."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2603_00907_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.small_case(3, batch=2, seq_lens=(200, 150), budgets=(80, 60))
        data = wl.make_layer(w, 0, seq_offset=rank)
        digest = torch.tensor([float(data["K"].astype(np.int64).sum() % 1000003)], dtype=torch.float64)
        gathered = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(gathered, digest)
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
        tokens = world * bench.rank_tokens_per_step(w, 1)
        out[rank] = ([float(g.item()) for g in gathered], ms, tokens)
    finally:
        dist.destroy_process_group()


def test_two_ranks_hold_different_shards_and_time_is_the_slowest():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in range(world):
        digests, ms, tokens = res[r]
        assert digests[0] != digests[1]            # every rank generated its own sequences
        assert ms == 15.0                          # the slowest rank's time, on every rank
        assert tokens == 2 * (200 + 150)
    assert res[0][0] == res[1][0]


def test_rank_shards_are_reproducible_and_rank0_is_the_single_gpu_batch():
    w = wl.small_case(4, batch=1, seq_lens=(120,), budgets=(60,))
    a, b = wl.make_layer(w, 0, seq_offset=1), wl.make_layer(w, 0, seq_offset=1)
    assert np.array_equal(a["K"], b["K"]) and np.array_equal(a["V"], b["V"])
    assert np.array_equal(wl.make_layer(w, 0)["K"], wl.make_layer(w, 0, seq_offset=0)["K"])
    assert not np.array_equal(a["K"], wl.make_layer(w, 0)["K"])


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself; in its CPU
    self-check mode they run the sharding arithmetic over gloo: rank -> its own shard, tokens x
    world, time = the slowest rank's."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--shard-check"],
                       capture_output=True, text=True, timeout=300, env=env, cwd=root)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                  # rank 0 alone prints
    d = lines[0]
    assert d["n_gpus"] == 2 and d["ms_per_step"] == 15.0 and d["tokens_per_step"] == 2 * (200 + 150)
    assert len(d["digests"]) == 2 and d["digests"][0] != d["digests"][1]
    # one rank, no launcher: the same path without a process group
    r1 = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "1", "--shard-check"],
                        capture_output=True, text=True, timeout=300, env=env, cwd=root)
    d1 = json.loads([l for l in r1.stdout.splitlines() if l.startswith("{")][0])
    assert d1["n_gpus"] == 1 and d1["tokens_per_step"] == 350 and d1["digests"] == d["digests"][:1]
