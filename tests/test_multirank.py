"""The N > 1 paths on CPU (gloo, world size 2), driving the library itself through host-only caches
(device = -1: argument checks and bookkeeping, no CUDA call).

Two ways of using several GPUs, neither with a collective on the data path:
  * by sequence: every rank holds its own sequences (seed offset by rank);
  * by KV head (pod_shard_config / pod_shard_block_map): rank r holds KV heads
    [r H_kv / P, (r + 1) H_kv / P) of the same sequences and the query heads that read them; its cache is
    an ordinary cache of those heads, its outputs a disjoint slice of [B][H_q][d].
Checked here: the head -> rank map and the output slices tile the full head range; the ranks' byte
counts add up to the unsplit cache's; head-wise block maps are cut by columns; the call-order rules
hold on every rank's cache; the benchmark's aggregation takes the maximum over ranks and does not
restate a latency as a throughput when the ranks work on the same layer-steps.
"""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth

FULL = dict(n_layers=6, n_q_heads=16, n_kv_heads=4, head_dim=64, group_size=2, n_sink=4, n_recent=16, batch=2)
LENS = [100, 37]
HEAD_WISE = [[0, 0, 0, 0], [0, 1, 0, 1], [0, 1, 2, 1], [3, 1, 2, 1], [3, 4, 2, 1], [3, 4, 2, 5]]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _fill(cache, n_layers, lens):
    for l in range(n_layers):
        for b, n in enumerate(lens):
            assert cache.write(l, b, 0x1000, 0x1000, n) == B.POD_DRY_RUN


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        full = B.make_config(device=-1, **FULL)
        local, kv0, q0 = B.pod_shard_config(full, rank, world)
        # the rank's cache: an ordinary cache of its heads
        cache = B.PodCache(local, LENS)
        _fill(cache, FULL["n_layers"], LENS)
        mine = torch.tensor([cache.bytes(B.POD_BYTES_LIVE), cache.bytes(B.POD_BYTES_DENSE_EQUIV), kv0, local.n_kv_heads,
                             q0, local.n_q_heads], dtype=torch.int64)
        gathered = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(gathered, mine)
        # order rules on the rank's cache: a sharing layer before its block's lowest layer is refused, then accepted
        p = 0x1000
        order = []
        try:
            cache.decode_attn(1, p, p)
            order.append("accepted")
        except B.PodError as e:
            order.append(e.status)
        assert cache.decode_attn(0, p, p) == B.POD_DRY_RUN
        order.append(cache.decode_attn(1, p, p))
        # head-wise blocks: the rank's columns of the map, and a cache built from them
        cols = B.pod_shard_block_map(full, HEAD_WISE, rank, world)
        hw = B.PodCache(local, LENS, lowest_layer=cols)
        _fill(hw, FULL["n_layers"], LENS)
        hw_live = torch.tensor([hw.bytes(B.POD_BYTES_LIVE)], dtype=torch.int64)
        dist.all_reduce(hw_live)
        # by sequence: disjoint seeds, really different K/V
        seed = bench.rank_seed(7, rank)
        k = synth.gen_kv(seed, synth.TAG_K, 0, 0, 0, 8, FULL["n_kv_heads"], FULL["head_dim"])
        ksum = torch.tensor([float(k.float().sum())], dtype=torch.float64)
        ksums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(ksums, ksum)
        # outputs of a KV-head split, gathered: rank r's slice holds query heads r * H_q / P onwards
        Bn, Hl, d = FULL["batch"], local.n_q_heads, FULL["head_dim"]
        whole_out = torch.arange(Bn * FULL["n_q_heads"] * d, dtype=torch.float32).reshape(Bn, FULL["n_q_heads"], d).to(torch.bfloat16)
        mine = whole_out[:, q0:q0 + Hl].contiguous()
        got = bench.heads_from_gathered(bench.gather_outputs(dist, mine, torch.empty(world, Bn, Hl, d, dtype=torch.bfloat16)))
        gather_ok = bool(torch.equal(got, whole_out))
        # timing: the slowest rank counts
        t = bench.reduce_max(10.0 + rank, dist, torch.device("cpu"))
        ret[rank] = dict(gathered=[g.tolist() for g in gathered], order=order, cols=cols, hw_live=int(hw_live.item()),
                         seed=seed, ksums=[float(x) for x in ksums], t=t, gather_ok=gather_ok)
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_by_kv_head_and_by_sequence():
    world = 2
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    r0, r1 = ret[0], ret[1]
    assert r0["gathered"] == r1["gathered"]
    (live0, dense0, kv00, nkv0, q00, nq0), (live1, dense1, kv01, nkv1, q01, nq1) = r0["gathered"]
    # the unsplit cache on the host
    full = B.make_config(device=-1, **FULL)
    whole = B.PodCache(full, LENS)
    _fill(whole, FULL["n_layers"], LENS)
    assert live0 + live1 == whole.bytes(B.POD_BYTES_LIVE) and dense0 + dense1 == whole.bytes(B.POD_BYTES_DENSE_EQUIV)
    # heads: contiguous, disjoint, covering; query heads follow their KV heads
    r = FULL["n_q_heads"] // FULL["n_kv_heads"]
    assert (kv00, nkv0, kv01, nkv1) == (0, 2, 2, 2)
    assert (q00, nq0, q01, nq1) == (0, 2 * r, 2 * r, 2 * r)
    # order rules hold per rank
    assert r0["order"] == r1["order"] == [B.POD_ERR_ORDER, B.POD_DRY_RUN]
    # head-wise map: columns
    assert r0["cols"] == [row[0:2] for row in HEAD_WISE] and r1["cols"] == [row[2:4] for row in HEAD_WISE]
    hw_whole = B.PodCache(full, LENS, lowest_layer=HEAD_WISE)
    _fill(hw_whole, FULL["n_layers"], LENS)
    assert r0["hw_live"] == r1["hw_live"] == hw_whole.bytes(B.POD_BYTES_LIVE)
    # by sequence
    assert r0["seed"] != r1["seed"] and r0["ksums"] == r1["ksums"] and r0["ksums"][0] != r0["ksums"][1]
    assert r0["t"] == r1["t"] == 11.0                            # max over ranks on every rank
    assert r0["gather_ok"] and r1["gather_ok"]                   # gathered slices give the unsplit [B][H_q][d]


def test_shard_config_rejects_what_does_not_divide():
    full = B.make_config(device=-1, **FULL)
    for rank, world in [(0, 3), (2, 2), (-1, 2), (0, 0)]:
        try:
            B.pod_shard_config(full, rank, world)
            assert False, (rank, world)
        except B.PodError as e:
            assert e.status == B.POD_ERR_INVALID
    local, kv0, q0 = B.pod_shard_config(full, 3, 4)
    assert (local.n_kv_heads, local.n_q_heads, kv0, q0) == (1, 4, 3, 12)
    assert (local.n_layers, local.head_dim, local.group_size, local.batch) == (6, 64, 2, 2)


def test_aggregate_by_sequence_and_by_kv_head():
    a = bench.aggregate(ms=2.0, steps=10, layers=32, batch_per_rank=1, world=1)
    assert abs(a["us_per_layer_step"] - 2000.0 / 320) < 1e-12 and a["per_rank_us_per_layer_step"] == a["us_per_layer_step"]
    assert bench.reduce_max(3.5, None, torch.device("cpu")) == 3.5
    # two ranks with their own sequences: twice the work in the same time; the rank's own figure stays beside it
    s = bench.aggregate(ms=11.0, steps=5, layers=4, batch_per_rank=1, world=2)
    assert abs(s["per_rank_us_per_layer_step"] - 11.0e3 / 20) < 1e-9 and abs(s["us_per_layer_step"] - 11.0e3 / 40) < 1e-9
    assert abs(s["decode_tokens_per_s"] - 2 / (11.0e-3 / 5)) < 1e-6
    # two ranks with half of the heads each: the same layer-steps, nothing is divided
    h = bench.aggregate(ms=11.0, steps=5, layers=4, batch_per_rank=1, world=2, shard="kv-head")
    assert abs(h["us_per_layer_step"] - 11.0e3 / 20) < 1e-9 and abs(h["decode_tokens_per_s"] - 1 / (11.0e-3 / 5)) < 1e-6
