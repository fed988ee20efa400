"""Parity at the full sizes of the five configurations, in the launch configuration bench.py times: the CUDA
path runs every layer, and the oracle recomputes EVERY (sequence, layer, head) output of configurations 2 and 4,
of two sequences of configuration 3, and of configuration 5 at its first and last decode step (by default two
seeded KV heads -- eight query heads -- per (sequence, layer); all of them with POD_FULL_PARITY=1), from the
regenerated history (the full history never exists on the host).  A head-wise block map and a gate threshold are
run at the 32K size as well."""
import os

import numpy as np
import pytest
import torch

import bench
from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth
from podtest import Case, KVHeadChecker

pytestmark = pytest.mark.gpu
FULL = os.environ.get("POD_FULL_PARITY", "0") == "1"


def _free_gb():
    free, _ = torch.cuda.mem_get_info()
    return free / 2 ** 30


def _check_everything(case, outs, seqs=None, step=0, lens=None, heads_of=None, tau=None):
    """Every (sequence in seqs, layer, KV head) -- all r query heads of each -- against the oracle."""
    lens = case.lens if lens is None else lens
    chk = KVHeadChecker(case)
    for b in (range(case.B) if seqs is None else seqs):
        for l in range(case.L):
            for kvh in (range(case.Hkv) if heads_of is None else heads_of(b, l)):
                chk.submit(outs, l, b, kvh, lens[b], step=step, tau=tau)
    worst = chk.finish()
    return chk.checked, worst


def test_config2_llama8b_32k_every_head():
    """32 layers, G = 2, 32/8 heads, d = 128, 32768 tokens, S = 16, W = 2048, outlier channels: all 1024 outputs."""
    case = Case(seed=2, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, lens=[32768], outliers=True)
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    assert cache.last_launch()["n_ctas"] == 296                  # one wave of 148 SMs x 2 CTAs
    checked, _ = _check_everything(case, outs)
    assert checked == 32 * 32
    live, dense = cache.bytes(B.POD_BYTES_LIVE), cache.bytes(B.POD_BYTES_DENSE_EQUIV)
    assert dense == 4 << 30 and abs((1 - live / dense) - 0.234252929688) < 1e-9
    assert torch.isfinite(outs.float()).all()


def test_config2_one_launch_steps_every_head():
    """The same configuration through the one-launch form bench.py times (append + attention, launches back to
    back, so that they start optimistically and hand their logits over through the per-head words): three steps,
    every output of the last one."""
    n0, steps = 32768, 3
    case = Case(seed=2, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, lens=[n0], outliers=True, caps=[n0 + steps])
    cache = case.make_cache()
    case.prefill(cache)
    stream = torch.cuda.current_stream().cuda_stream
    outs = torch.empty(case.L, 1, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
    ins = [[(case.kv(synth.TAG_K, l, 0, n0 + s, n0 + s + 1, "cuda"), case.kv(synth.TAG_V, l, 0, n0 + s, n0 + s + 1, "cuda"),
             case.q(l, s + 1, "cuda")) for l in range(case.L)] for s in range(steps)]
    torch.cuda.synchronize()
    for s in range(steps):                                       # nothing but the library's launches in the stream
        for l in range(case.L):
            k, v, q = ins[s][l]
            cache.append_decode_attn(l, k, v, q, outs[l], stream)
    torch.cuda.synchronize()
    assert cache.device_status() == B.POD_OK
    checked, _ = _check_everything(case, outs, step=steps, lens=[n0 + steps])
    assert checked == 32 * 32


def test_config4_long_context_128k_every_head():
    """Batch 1, 131072 tokens, G = 2, S = 16, W = 4096, outlier channels; split-K over the distant segment."""
    if _free_gb() < 20:
        pytest.skip("needs 20 GiB of free device memory")
    case = Case(seed=4, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=4096, lens=[131072], outliers=True)
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    checked, _ = _check_everything(case, outs)
    assert checked == 32 * 32
    assert cache.bytes(B.POD_BYTES_LIVE) == 13019643904
    assert torch.isfinite(outs.float()).all()


def test_config3_batch16_32k_two_sequences_every_head():
    """Batch 16 x 32768 tokens, G = 4, S = 16, W = 1024: every output of the first and the last sequence, and one
    seeded (layer, KV head) of each of the others."""
    if _free_gb() < 60:
        pytest.skip("needs 60 GiB of free device memory")
    case = Case(seed=3, L=32, G=4, Hq=32, Hkv=8, d=128, S=16, W=1024, lens=[32768] * 16)
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    checked, _ = _check_everything(case, outs, seqs=(0, 15))
    assert checked == 2 * 32 * 32
    rng = np.random.default_rng(3)
    chk = KVHeadChecker(case)
    for b in range(1, 15):
        chk.submit(outs, int(rng.integers(32)), b, int(rng.integers(8)), 32768)
    chk.finish()
    live, dense = cache.bytes(B.POD_BYTES_LIVE), cache.bytes(B.POD_BYTES_DENSE_EQUIV)
    assert dense == 64 << 30 and abs((1 - live / dense) - 0.363098144531) < 1e-9
    assert torch.isfinite(outs.float()).all()


def test_config5_ragged_serving_mix():
    """32 sequences of 4096..65536 tokens (seeded), G = 2, S = 16, W = 2048: prefill of every full
    sequence, then 16 decode steps (append one token per sequence and layer, decode every layer),
    alternating between the one-launch form and the two-call form.  Checked: every (sequence, layer) at the
    first and the last step, and four seeded (sequence, step) pairs in between with all their layers."""
    if _free_gb() < 140:
        pytest.skip("needs 140 GiB of free device memory")
    seed, steps = 5, 16
    lens0 = synth.ragged_lengths(seed, 32, 4096, 65536)
    case = Case(seed=seed, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, lens=lens0,
                caps=[n + steps for n in lens0])
    cache = case.make_cache()
    case.prefill(cache, chunk=16384)
    stream = torch.cuda.current_stream().cuda_stream
    rng = np.random.default_rng(seed)
    between = {int(s): int(b) for s, b in zip(rng.choice(np.arange(2, steps), 4, replace=False), rng.integers(32, size=4))}
    outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
    checked = 0
    for step in range(1, steps + 1):
        lens = [n + step for n in lens0]
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            if step % 2:                       # odd steps as one launch per layer, even steps as two calls
                cache.append_decode_attn(l, k, v, case.q(l, step, "cuda"), outs[l], stream)
            else:
                cache.write(l, -1, k, v, 1, stream)
                cache.decode_attn(l, case.q(l, step, "cuda"), outs[l], stream)
        torch.cuda.synchronize()
        assert torch.isfinite(outs.float()).all()
        if step in (1, steps):
            pick = (lambda b, l: range(8)) if FULL else (lambda b, l: sorted({int(x) for x in np.random.default_rng(step * 4099 + b * 37 + l).choice(8, 2, replace=False)}))
            n, _ = _check_everything(case, outs, step=step, lens=lens, heads_of=pick)
            checked += n
        elif step in between:
            n, _ = _check_everything(case, outs, seqs=(between[step],), step=step, lens=lens,
                                     heads_of=lambda b, l: (int((b + l + step) % 8),))
            checked += n
    assert checked == (2 * 32 * 32 * (8 if FULL else 2) + 4 * 32) * 4
    assert cache.device_status() == B.POD_OK
    from oracle import pod_oracle as O
    live, dense = O.pod_cache_bytes([n + steps for n in lens0], n_layers=32, n_kv_heads=8, head_dim=128,
                                    group_size=2, n_s=16, n_r=2048)
    assert cache.bytes(B.POD_BYTES_LIVE) == live and cache.bytes(B.POD_BYTES_DENSE_EQUIV) == dense


def test_head_wise_blocks_at_32k():
    """The seeded head-wise block map of bench.py's llama3-8b-32k-headwise workload (about 70 % of the (layer,
    KV head) pairs share) at full size: layers mix heads that keep their keys, heads that read stored logits and
    heads of different work in one launch.  Two steps of the one-launch form; every layer, three seeded KV heads."""
    w = bench.WORKLOADS["llama3-8b-32k-headwise"]
    low = bench.block_map(w)
    n0, steps = 32768, 2
    case = Case(seed=2, L=32, G=1, Hq=32, Hkv=8, d=128, S=16, W=2048, lens=[n0], outliers=True, caps=[n0 + steps], lowest=low)
    cache = case.make_cache()
    case.prefill(cache)
    stream = torch.cuda.current_stream().cuda_stream
    outs = torch.empty(case.L, 1, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
    for s in range(1, steps + 1):
        for l in range(case.L):
            cache.append_decode_attn(l, case.kv(synth.TAG_K, l, 0, n0 + s - 1, n0 + s, "cuda"), case.kv(synth.TAG_V, l, 0, n0 + s - 1, n0 + s, "cuda"),
                                     case.q(l, s, "cuda"), outs[l], stream)
    torch.cuda.synchronize()
    assert cache.device_status() == B.POD_OK
    pick = lambda b, l: sorted({int(x) for x in np.random.default_rng(977 + l).choice(8, 3, replace=False)})
    checked, _ = _check_everything(case, outs, step=steps, lens=[n0 + steps], heads_of=pick)
    assert checked == 32 * 3 * 4
    from oracle import pod_oracle as O
    live, _ = O.pod_cache_bytes([n0 + steps], n_layers=32, n_kv_heads=8, head_dim=128, lowest=low, n_s=16, n_r=2048)
    assert cache.bytes(B.POD_BYTES_LIVE) == live


def test_gate_threshold_at_32k():
    """The distant-skip approximation (gate threshold 0.5) at the 32K size: sharing layers run as two launches;
    two seeded KV heads of every layer against the oracle's gated result (either candidate within 0.01 of the
    threshold)."""
    tau = 0.5
    case = Case(seed=2, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, lens=[32768], outliers=True)
    cache = case.make_cache()
    cache.set_gate_threshold(tau)
    case.prefill(cache)
    outs = case.decode_all(cache)
    pick = lambda b, l: sorted({int(x) for x in np.random.default_rng(313 + l).choice(8, 2, replace=False)})
    checked, _ = _check_everything(case, outs, heads_of=pick, tau=tau)
    assert checked == 32 * 2 * 4


@pytest.mark.parametrize("T,W,samples", [
    (32768, 2048, [(0, 0), (17, 3), (2063, 1), (2064, 1), (2065, 6), (4095, 2), (4096, 2), (12345, 7), (16383, 0), (16384, 5),
                   (20000, 4), (32511, 3), (32512, 3), (32639, 6), (32640, 6), (32767, 0), (32767, 7)]),
    (131072, 4096, [(4111, 2), (4112, 2), (65535, 0), (65536, 7), (100000, 4), (130815, 1), (130816, 1), (131071, 5)])])
def test_prefill_attention_sampled(T, W, samples):
    """pod_prefill_attn at the size bench.py times (32768 positions, 32/8 heads, S = 16, W = 2048, outlier
    channels) and at the longest context of the configurations (131072 positions, W = 4096): both layers of a
    block; the oracle recomputes sampled (position, KV head) outputs one by one as decode steps on the prefix
    (all four query heads of the KV head)."""
    if T > 65536 and _free_gb() < 12:
        pytest.skip("needs 12 GiB of free device memory")
    from oracle import pod_oracle as O
    Hq, Hkv, d, S, seed = 32, 8, 128, 16, 2
    gen = lambda tag, layer, h, outl: synth.gen_kv(seed, tag, layer, 0, 0, T, h, d, outliers=outl, device="cuda")
    Q = [gen(synth.TAG_Q, l, Hq, False) for l in range(2)]
    K = [gen(synth.TAG_K, l, Hkv, True) for l in range(2)]
    V = [gen(synth.TAG_V, l, Hkv, True) for l in range(2)]
    outs = [torch.zeros(T, Hq, d, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    B.pod_prefill_attn(Q[0], K[0], V[0], outs[0], n_sink=S, n_recent=W)
    B.pod_prefill_attn(Q[1], K[1], V[1], outs[1], n_sink=S, n_recent=W, q_low=Q[0], k_low=K[0])
    torch.cuda.synchronize()
    assert B.pod_prefill_status() == B.POD_OK
    assert all(torch.isfinite(o.float()).all() for o in outs)
    r = Hq // Hkv
    for (i, kh) in samples:
        f = lambda xs, hs: np.stack([x[:i + 1, hs].double().cpu().numpy() for x in xs])
        Kn, Vn = f(K, slice(kh, kh + 1)), f(V, slice(kh, kh + 1))
        qn = np.stack([x[i, kh * r:(kh + 1) * r].double().cpu().numpy() for x in Q])
        vmax = np.abs(Vn).max(axis=(1, 2))                                   # [L][d]
        for l in range(2):
            ref = O.pod_decode_layer(qn, Kn, Vn, l, group_size=2, n_s=S, n_r=W)   # [r][d]
            got = outs[l][i, kh * r:(kh + 1) * r].double().cpu().numpy()
            err = np.abs(got - ref)
            bound = 1e-2 + 2.0 ** -8 * vmax[l][None]                          # as in test_gpu_prefill.py
            rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
            assert (err <= bound).all() and rel <= 5e-3, (i, kh, l, err.max(), rel)
