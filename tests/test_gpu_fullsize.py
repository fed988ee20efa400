"""Parity at the full sizes of the five configurations, in the launch configuration bench.py
times: the CUDA path runs every layer; the oracle recomputes sampled (sequence, layer, head)
outputs one by one from the regenerated history (the full history never exists on the host)."""
import numpy as np
import pytest
import torch

from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth
from podtest import Case, assert_close

pytestmark = pytest.mark.gpu


def _sample_check(case, outs, triples, step=0, lens=None):
    lens = case.lens if lens is None else lens
    worst = [0.0, 0.0]
    for (b, l, h) in triples:
        ref = case.oracle_head(l, b, h, n=lens[b], step=step)
        ma, rl = assert_close(outs[l, b, h], ref, f"seq {b} layer {l} head {h} step {step}")
        worst = [max(worst[0], ma), max(worst[1], rl)]
    return worst


def _free_gb():
    free, _ = torch.cuda.mem_get_info()
    return free / 2 ** 30


def test_config2_llama8b_32k():
    """32 layers, G = 2, 32/8 heads, d = 128, 32768 tokens, S = 16, W = 2048, outlier channels."""
    case = Case(seed=2, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, lens=[32768], outliers=True)
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    geo = cache.last_launch()
    assert geo["n_ctas"] == 296                                  # one wave of 148 SMs x 2 CTAs
    triples = [(0, l, h) for l in (0, 1) for h in range(32)]     # a whole block, every head
    triples += [(0, l, h) for l, h in [(2, 5), (3, 5), (14, 0), (15, 31), (30, 17), (31, 17), (31, 0), (17, 9)]]
    _sample_check(case, outs, triples)
    live, dense = cache.bytes(B.POD_BYTES_LIVE), cache.bytes(B.POD_BYTES_DENSE_EQUIV)
    assert dense == 4 << 30 and abs((1 - live / dense) - 0.234252929688) < 1e-9
    assert torch.isfinite(outs.float()).all()


def test_config4_long_context_128k():
    """Batch 1, 131072 tokens, G = 2, S = 16, W = 4096, outlier channels; split-K over the distant segment."""
    if _free_gb() < 20:
        pytest.skip("needs 20 GiB of free device memory")
    case = Case(seed=4, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=4096, lens=[131072], outliers=True)
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    triples = [(0, l, h) for l, h in [(0, 0), (1, 0), (1, 3), (6, 12), (7, 12), (31, 31), (30, 30), (19, 7)]]
    _sample_check(case, outs, triples)
    assert cache.bytes(B.POD_BYTES_LIVE) == 13019643904
    assert torch.isfinite(outs.float()).all()


def test_config3_batch16_32k():
    """Batch 16 x 32768 tokens, G = 4, S = 16, W = 1024."""
    if _free_gb() < 60:
        pytest.skip("needs 60 GiB of free device memory")
    case = Case(seed=3, L=32, G=4, Hq=32, Hkv=8, d=128, S=16, W=1024, lens=[32768] * 16)
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    triples = [(0, 0, 0), (0, 1, 0), (0, 2, 0), (0, 3, 0), (15, 3, 31), (7, 17, 13), (3, 28, 2), (12, 31, 20),
               (15, 30, 7), (9, 5, 5)]
    _sample_check(case, outs, triples)
    live, dense = cache.bytes(B.POD_BYTES_LIVE), cache.bytes(B.POD_BYTES_DENSE_EQUIV)
    assert dense == 64 << 30 and abs((1 - live / dense) - 0.363098144531) < 1e-9
    assert torch.isfinite(outs.float()).all()


def test_config5_ragged_serving_mix():
    """32 sequences of 4096..65536 tokens (seeded), G = 2, S = 16, W = 2048: prefill of every full
    sequence, then 16 decode steps (append one token per sequence and layer, decode every layer),
    alternating between the one-launch form and the two-call form."""
    if _free_gb() < 140:
        pytest.skip("needs 140 GiB of free device memory")
    seed, steps = 5, 16
    lens0 = synth.ragged_lengths(seed, 32, 4096, 65536)
    case = Case(seed=seed, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, lens=lens0,
                caps=[n + steps for n in lens0])
    cache = case.make_cache()
    case.prefill(cache, chunk=16384)
    stream = torch.cuda.current_stream().cuda_stream
    short, long_ = int(np.argmin(lens0)), int(np.argmax(lens0))
    rng = np.random.default_rng(seed)
    outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
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
        if step in (1, 8, 9, steps):
            triples = [(short, 0, 0), (short, 1, 3), (long_, 30, 8), (long_, 31, 8)]
            triples += [(int(rng.integers(32)), int(rng.integers(32)), int(rng.integers(32))) for _ in range(4)]
            _sample_check(case, outs, triples, step=step, lens=lens)
            assert torch.isfinite(outs.float()).all()
    assert cache.device_status() == B.POD_OK
    from oracle import pod_oracle as O
    live, dense = O.pod_cache_bytes([n + steps for n in lens0], n_layers=32, n_kv_heads=8, head_dim=128,
                                    group_size=2, n_s=16, n_r=2048)
    assert cache.bytes(B.POD_BYTES_LIVE) == live and cache.bytes(B.POD_BYTES_DENSE_EQUIV) == dense


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
