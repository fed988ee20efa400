"""The N > 1 path of the benchmark on CPU (gloo, world size 2): ranks hold disjoint sequences
(seed offset by rank), there is no data-path collective, the reported time is the maximum over
ranks after a barrier, and throughput aggregates the units of all ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2412_02252_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = bench.WORKLOADS["tiny"]
        seed = bench.rank_seed(w["seed"], rank)
        k = synth.gen_kv(seed, synth.TAG_K, 0, 0, 0, 8, w["Hkv"], w["d"])
        mine = torch.tensor([float(k.float().sum())], dtype=torch.float64)
        gathered = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(gathered, mine)
        elapsed = 10.0 + rank                                    # pretend timings: rank 1 is slower
        t = bench.reduce_max(elapsed, dist, torch.device("cpu"))
        agg = bench.aggregate(ms=t, steps=5, layers=w["L"], batch_per_rank=w["B"], world=world)
        ret[rank] = (seed, [float(g) for g in gathered], t, agg)
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_sequences_and_take_max_time():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
    (s0, g0, t0, a0), (s1, g1, t1, a1) = ret[0], ret[1]
    assert s0 != s1                                   # every rank decodes its own sequences
    assert g0 == g1 and g0[0] != g0[1]                # and their K/V really differ
    assert t0 == t1 == 11.0                           # max over ranks on every rank
    assert a0 == a1
    # 5 steps x 4 layers x 2 ranks layer-steps in 11 ms
    assert abs(a0["us_per_layer_step"] - 11.0e3 / (5 * 4 * 2)) < 1e-9
    assert abs(a0["decode_tokens_per_s"] - 2 * 1 / (11.0e-3 / 5)) < 1e-6


def test_single_rank_aggregate_is_plain():
    a = bench.aggregate(ms=2.0, steps=10, layers=32, batch_per_rank=1, world=1)
    assert abs(a["us_per_layer_step"] - 2000.0 / 320) < 1e-12
    assert bench.reduce_max(3.5, None, torch.device("cpu")) == 3.5
