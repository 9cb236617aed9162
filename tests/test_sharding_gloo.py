"""N > 1 host logic on CPU: two gloo ranks split a batch of requests, each runs its shard
(through the oracle here, as the CUDA path would on its own GPU), and the union equals the
unsharded result; the timing reduction takes the max over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_26140_b200 import sharding, workloads as wl


def test_shard_range_partitions_exactly():
    for n in (0, 1, 2, 7, 16, 33):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    assert sharding.aggregate_throughput(103, 8, 0.5) == 8 * 103 / 0.5e-3
    assert sharding.max_over_ranks(3.5) == 3.5


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import acache_oracle as orc
        shape = wl.LayerShape(64, 4, 2, 16, 96, 1e-5, True, 1e4, "small")
        lay = wl.make_layout(3, 2, 20, 4, 8, 8, "masked")          # 3 requests over 2 ranks: 2 + 1
        case = wl.make_case(shape, lay, 0.25, cfg_id=21)
        lo, hi = sharding.shard_range(lay.batch, rank, world)
        mine = {}
        for b in range(lo, hi):
            r = orc.layer_step(case.weights, shape, case.x[b], case.cache_k[b], case.cache_v[b], lay.ctx_len,
                               lay.affix_start, lay.affix_len, lay.masked_pos[b], lay.extra_rows[b],
                               case.rope_cos, case.rope_sin, ratio=0.25)
            mine[b] = (r["anchor_idx"], r["y"], r["cache_k"])
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        t = sharding.max_over_ranks(1.0 + rank, dist)              # "step time" differs per rank
        assert t == float(world)
        if rank == 0:
            merged = {}
            for g in gathered:
                assert not (set(g) & set(merged))                  # shards are disjoint
                merged.update(g)
            assert sorted(merged) == list(range(lay.batch))
            for b in range(lay.batch):                             # unsharded run gives the same
                r = orc.layer_step(case.weights, shape, case.x[b], case.cache_k[b], case.cache_v[b], lay.ctx_len,
                                   lay.affix_start, lay.affix_len, lay.masked_pos[b], lay.extra_rows[b],
                                   case.rope_cos, case.rope_sin, ratio=0.25)
                assert np.array_equal(merged[b][0], r["anchor_idx"])
                assert np.array_equal(merged[b][1], r["y"]) and np.array_equal(merged[b][2], r["cache_k"])
            open(os.path.join(out_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_cover_the_batch(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").exists()


def test_launch_plan_and_self_start_command():
    assert sharding.launch_plan(1, {}) == ("run", 1)
    assert sharding.launch_plan(8, {}) == ("spawn", 8)
    assert sharding.launch_plan(8, {"WORLD_SIZE": "8"}) == ("run", 8)
    assert sharding.launch_plan(8, {"WORLD_SIZE": "1"}) == ("refuse", 1)
    assert sharding.launch_plan(1, {"WORLD_SIZE": "2"}) == ("refuse", 2)
    cmd = sharding.torchrun_command("bench.py", ["--gpus", "4", "--steps", "7"], 4, 29511)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-5:] == ["bench.py", "--gpus", "4", "--steps", "7"]


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with no WORLD_SIZE around it starts two ranks of itself (each prints who it is
    and leaves: no GPU here); under a launcher with another rank count it refuses."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--rank-echo"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    seen = sorted(json.loads(l)["rank"] for l in r.stdout.splitlines() if l.startswith("{"))
    assert seen == [0, 1]
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--rank-echo"], env={**env, "WORLD_SIZE": "1"},
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "bench.py starts its own ranks" in r.stderr
