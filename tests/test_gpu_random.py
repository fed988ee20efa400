"""Seeded random configurations of the decode path against the oracle: shapes, block maps, window sizes, batch
mixes, prefill chunkings and call forms drawn together, so that combinations no hand-written case lists are met.
Every (sequence, layer, query head) of the checked steps is compared element by element, and the cache contents
bit for bit with the oracle's layout after the prefill and after the last step."""
from __future__ import annotations

import random

import numpy as np
import pytest
import torch

from oracle import pod_oracle as O
from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth
from podtest import MAX_ABS, REL_L2, Case
from test_gpu_parity import _compare_layout, _oracle_cache

pytestmark = pytest.mark.gpu

N_STEPS = 6
CHECK_STEPS = (1, 3, 6)


def draw_case(seed):
    rng = random.Random(1000 + seed)
    d = rng.choice([64, 128])
    Hkv = rng.choice([1, 2, 3, 4])
    r = rng.choice([1, 2, 3, 4, 8])
    L = rng.randint(2, 6)
    G = rng.choice([1, 2, 3, 4])
    S = rng.choice([0, 1, 4, 16, 20])
    W = rng.choice([1, 8, 16, 64, 100])
    Bn = rng.randint(1, 5)
    kinds = [lambda: rng.randint(0, max(0, S)),                       # inside the sink (or empty)
             lambda: rng.randint(S, S + W),                           # window not full yet
             lambda: rng.randint(S + W + 1, S + W + 40),              # a few distant tokens
             lambda: rng.randint(200, 700)]                           # several tiles and chunks of distant tokens
    lens = [rng.choice(kinds)() for _ in range(Bn)]
    lowest = None
    if rng.random() < 0.35:                                           # head-wise blocks: runs of consecutive layers per head
        lowest = [[0] * Hkv]
        for l in range(1, L):
            lowest.append([lowest[l - 1][h] if rng.random() < 0.6 else l for h in range(Hkv)])
    scale = rng.choice([0.0, 0.0, 0.05, 0.2])
    caps = [n + N_STEPS + rng.randint(0, 9) for n in lens]
    case = Case(seed=500 + seed, L=L, G=G, Hq=Hkv * r, Hkv=Hkv, d=d, S=S, W=W, lens=lens, caps=caps, scale=scale,
                lowest=lowest, outliers=rng.random() < 0.5)
    chunk = rng.choice([7, 64, 1000])
    # per step and layer: one launch (append + attention) or two calls
    fused = [[rng.random() < 0.6 for _ in range(L)] for _ in range(N_STEPS + 1)]
    # some one-launch calls are told that their early copy of the inputs was stale (host-side injection): the head is
    # then recomputed by the plain loop of the CTA that combines it
    stale = [[rng.random() < 0.25 for _ in range(L)] for _ in range(N_STEPS + 1)]
    tau = rng.choice([None, None, 0.3, 0.6, 0.9])                      # gate threshold of the sharing layers
    return case, chunk, fused, stale, tau


def check_group(case, outs, layer, b, kvh, n, step, tau=None):
    """The r query heads of one KV head against the oracle.  Relative L2 as everywhere.  The absolute bound is
    1e-2 plus 2^-8 of the largest value the channel holds: a context of a handful of tokens with an outlier
    channel gives outputs as large as single value rows (tens), and the two bf16 roundings that belong to the
    arithmetic (the probabilities as tensor-core operand, the output) each move such a channel by up to 2^-9 of
    that -- more than 1e-2 by themselves; with long contexts the second term is small against the first."""
    r = case.Hq // case.Hkv
    low = case.lowest[layer][kvh]
    f = lambda tag, l: case.kv(tag, l, b, 0, n, "cpu", heads=[kvh])[:, 0].double().numpy()
    K_l, V_l = f(synth.TAG_K, layer), f(synth.TAG_V, layer)
    K_a = K_l if low == layer else f(synth.TAG_K, low)
    bound = MAX_ABS + 2.0 ** -8 * np.abs(V_l).max(axis=0)
    worst = 0.0
    for h in range(kvh * r, (kvh + 1) * r):
        q_l = case.q(layer, step, "cpu")[b, h].double().numpy()
        q_a = case.q(low, step, "cpu")[b, h].double().numpy()
        ref, _ = O.pod_attention_joint(q_l, q_a, K_l, K_a, V_l, case.S, case.W, scale=(case.scale if case.scale > 0 else None))
        got = outs[layer, b, h].double().cpu().numpy()
        if tau is not None and low != layer:
            # a head of a sharing layer under a gate threshold: the oracle's decision decides, except within 0.01 of
            # the threshold (the device takes it in fp32), where either candidate is a valid result
            alt, g, _ = O.pod_attention_gate_skip(q_l, q_a, K_l, K_a, V_l, case.S, case.W, tau,
                                                  scale=(case.scale if case.scale > 0 else None))
            if abs(g - tau) >= 0.01 or np.abs(got - alt).max() < np.abs(got - ref).max():
                ref = alt
        err = np.abs(got - ref)
        rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
        assert (err <= bound).all() and rel <= REL_L2, (
            f"seq {b} layer {layer} head {h} step {step} n {n}: max_abs={err.max():.3e} (bound {bound[err.argmax()]:.3e}) rel_l2={rel:.3e}")
        worst = max(worst, rel)
    return r


@pytest.mark.parametrize("seed", range(40))
def test_random_configuration_decodes_like_the_oracle(seed):
    case, chunk, fused, stale, tau = draw_case(seed)
    cache = case.make_cache()
    case.prefill(cache, chunk=chunk)
    stream = torch.cuda.current_stream().cuda_stream
    if tau is not None:
        cache.set_gate_threshold(tau)
    # the oracle's layout of every sequence, kept up by plain writes and appends
    ocs = [_oracle_cache(case, b) for b in range(case.B)]
    for b, oc in enumerate(ocs):
        for l in range(case.L):
            if case.lens[b]:
                oc.write(l, synth.bf16_bits(case.kv(synth.TAG_K, l, b, 0, case.lens[b], "cpu")),
                         synth.bf16_bits(case.kv(synth.TAG_V, l, b, 0, case.lens[b], "cpu")))
    _compare_layout(case, cache, ocs)
    checked = 0
    for step in range(1, N_STEPS + 1):
        lens = [n + step for n in case.lens]
        outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            q = case.q(l, step, "cuda")
            if fused[step][l]:
                if stale[step][l]:
                    cache.inject_stale_query()
                cache.append_decode_attn(l, k, v, q, outs[l], stream)
            else:
                cache.write(l, -1, k, v, 1, stream)
                cache.decode_attn(l, q, outs[l], stream)
            kb, vb = synth.bf16_bits(k), synth.bf16_bits(v)
            for b, oc in enumerate(ocs):
                oc.append(l, kb[b], vb[b])
        torch.cuda.synchronize()
        assert [cache.seq_len(b, case.L - 1) for b in range(case.B)] == lens
        if step in CHECK_STEPS:
            host = outs.cpu()
            for l in range(case.L):
                for b in range(case.B):
                    for kvh in range(case.Hkv):
                        checked += check_group(case, host, l, b, kvh, lens[b], step, tau)
    _compare_layout(case, cache, ocs)                          # bit for bit after the appends of both call forms
    assert checked == len(CHECK_STEPS) * case.L * case.B * case.Hq
    assert cache.device_status() == B.POD_OK
    cache.destroy()


def draw_prefill(seed):
    rng = random.Random(7000 + seed)
    d = rng.choice([64, 128])
    Hkv = rng.choice([1, 2, 3])
    r = rng.choice([1, 2, 4])
    T = rng.choice([rng.randint(1, 40), rng.randint(100, 300), rng.randint(250, 530), rng.randint(600, 1300)])
    S = rng.choice([0, 1, 4, 16, 130, 260])
    W = rng.choice([1, 31, 64, 127, 128, 300, 2000])
    sharing = rng.random() < 0.7
    shares = None
    if sharing and rng.random() < 0.5:
        shares = [rng.randint(0, 1) for _ in range(Hkv)]
    scale = rng.choice([0.0, 0.0, 0.1])
    return dict(d=d, Hkv=Hkv, Hq=Hkv * r, T=T, S=S, W=W, sharing=sharing, shares=shares, scale=scale,
                outliers=rng.random() < 0.5)


@pytest.mark.parametrize("seed", range(24))
def test_random_configuration_prefill_like_the_oracle(seed):
    """pod_prefill_attn on drawn lengths (ragged query blocks and key tiles), sinks longer than a tile, windows
    shorter and longer than the sequence, plain and sharing layers, some heads sharing and some not: every
    position, head and channel against the oracle's prefill form."""
    c = draw_prefill(seed)
    d, Hq, Hkv, T, S, W = c["d"], c["Hq"], c["Hkv"], c["T"], c["S"], c["W"]
    gen = lambda tag, layer, h: synth.gen_kv(900 + seed, tag, layer, 0, 0, T, h, d,
                                             outliers=c["outliers"] and tag != synth.TAG_Q, device="cuda")
    Q = [gen(synth.TAG_Q, l, Hq) for l in range(2)]
    K = [gen(synth.TAG_K, l, Hkv) for l in range(2)]
    V = [gen(synth.TAG_V, l, Hkv) for l in range(2)]
    out = torch.zeros(T, Hq, d, dtype=torch.bfloat16, device="cuda")
    kw = dict(q_low=Q[0], k_low=K[0], head_shares=c["shares"]) if c["sharing"] else {}
    B.pod_prefill_attn(Q[1], K[1], V[1], out, n_sink=S, n_recent=W, sm_scale=c["scale"], **kw)
    torch.cuda.synchronize()
    assert B.pod_prefill_status() == B.POD_OK
    f = lambda xs: np.stack([x.double().cpu().numpy() for x in xs])
    takes_low = lambda h: c["sharing"] and (c["shares"] is None or c["shares"][h])
    low = np.array([[0] * Hkv, [0 if takes_low(h) else 1 for h in range(Hkv)]])
    ref = O.pod_prefill_layer(f(Q), f(K), f(V), 1, lowest=low, n_s=S, n_r=W, scale=(c["scale"] if c["scale"] > 0 else None))
    got = out.double().cpu().numpy()
    err = np.abs(got - ref)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    vmax = V[1].double().abs().amax(dim=0).cpu().numpy()                     # [H_kv][d]
    bound = MAX_ABS + 2.0 ** -8 * np.repeat(vmax, Hq // Hkv, axis=0)[None]   # the prefill tests' bound
    assert (err <= bound).all() and rel <= REL_L2, f"{c}: max_abs={err.max():.3e} rel_l2={rel:.3e}"
