"""Pins of the oracle's head-wise blocks: the greedy layer grouping (Algorithm 1) and decode
attention / layout / byte counts under a per-head lowest map.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import pod_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_example():
    sim = np.eye(5)[None].copy()
    blocks = lowest = None
    for line in open(os.path.join(GOLDEN, "greedy_grouping_example.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "sim":
            a, b, v = int(t[1]), int(t[2]), float(t[3])
            sim[0, a, b] = sim[0, b, a] = v
        elif t[0] == "blocks":
            blocks = [[int(x) for x in part.split(",")] for part in line.split(None, 1)[1].split("|")]
        elif t[0] == "lowest":
            lowest = [int(x) for x in t[1:]]
    return sim, blocks, lowest


def test_greedy_grouping_hand_worked_example():
    sim, blocks, lowest = _read_example()
    got = O.greedy_layer_blocks(sim, threshold=0.5)
    assert got == [blocks]
    assert O.lowest_map_from_blocks(got, 5)[:, 0].tolist() == lowest


def test_greedy_grouping_special_cases():
    L, H = 7, 3
    assert O.greedy_layer_blocks(np.ones((H, L, L))) == [[list(range(L))]] * H          # all similar
    assert O.greedy_layer_blocks(np.zeros((H, L, L))) == [[[l] for l in range(L)]] * H  # none similar
    # similar exactly when in the same run of G layers: the uniform partition comes back
    for G in (1, 2, 3, 4):
        sim = np.array([[[1.0 if a // G == b // G else 0.0 for b in range(L)] for a in range(L)]] * H)
        low = O.lowest_map_from_blocks(O.greedy_layer_blocks(sim), L)
        np.testing.assert_array_equal(low, O.uniform_lowest_map(L, H, G))
    # the threshold is inclusive
    sim = np.full((1, 3, 3), 0.5)
    assert O.greedy_layer_blocks(sim, 0.5) == [[[0, 1, 2]]]
    assert O.greedy_layer_blocks(sim, 0.5000001) == [[[0], [1], [2]]]


@pytest.mark.parametrize("seed", range(6))
def test_greedy_grouping_defining_properties(seed):
    """On random similarities: blocks are runs of consecutive layers that partition the layers; all
    pairs inside a block are similar; and a block could not have taken the next layer (greedy):
    the layer that opens a block is dissimilar to some layer of the block before it.  Heads are
    independent of one another."""
    rng = np.random.default_rng(seed)
    H, L, thr = 4, 9, 0.5
    sim = rng.random((H, L, L))
    sim = (sim + sim.transpose(0, 2, 1)) / 2
    res = O.greedy_layer_blocks(sim, thr)
    for h in range(H):
        blocks = res[h]
        assert [l for b in blocks for l in b] == list(range(L))
        for i, b in enumerate(blocks):
            assert all(sim[h, x, y] >= thr for x, y in itertools.combinations(b, 2))
            if i > 0:
                assert any(sim[h, b[0], y] < thr for y in blocks[i - 1])
        assert O.greedy_layer_blocks(sim[h:h + 1], thr) == [blocks]


def test_lowest_map_validation():
    O.check_lowest_map([[0, 0], [0, 1], [2, 1]])
    for bad in ([[0], [0], [1]], [[1], [1]], [[0], [2], [2]], [[0], [0], [0], [2]]):
        with pytest.raises(ValueError):
            O.check_lowest_map(bad)


def _inputs(rng, L, n, Hq, Hkv, d):
    bf = lambda x: (x.astype(np.float32).view(np.uint32) & 0xFFFF0000).view(np.float32).astype(np.float64)
    return (bf(rng.standard_normal((L, Hq, d))), bf(rng.standard_normal((L, n, Hkv, d))),
            bf(rng.standard_normal((L, n, Hkv, d))))


def test_uniform_map_equals_group_size():
    rng = np.random.default_rng(0)
    L, n, Hq, Hkv, d, S, W = 5, 40, 4, 2, 8, 3, 6
    q, K, V = _inputs(rng, L, n, Hq, Hkv, d)
    for G in (1, 2, 3):
        low = O.uniform_lowest_map(L, Hkv, G)
        for l in range(L):
            a = O.pod_decode_layer(q, K, V, l, group_size=G, n_s=S, n_r=W)
            b = O.pod_decode_layer(q, K, V, l, lowest=low, n_s=S, n_r=W)
            np.testing.assert_array_equal(a, b)
        assert (O.pod_cache_bytes([n], n_layers=L, n_kv_heads=Hkv, head_dim=d, group_size=G, n_s=S, n_r=W)
                == O.pod_cache_bytes([n], n_layers=L, n_kv_heads=Hkv, head_dim=d, lowest=low, n_s=S, n_r=W))


def test_head_wise_blocks_against_brute_force_and_per_head_independence():
    """Every query head follows the blocks of its own KV head: pure-Python evaluation of the
    definition, and equality with the uniform-G oracle run of the G that head uses."""
    rng = np.random.default_rng(1)
    L, n, Hq, Hkv, d, S, W = 6, 37, 6, 3, 8, 2, 5
    q, K, V = _inputs(rng, L, n, Hq, Hkv, d)
    low = np.array([O.uniform_lowest_map(L, 1, G)[:, 0] for G in (1, 2, 3)]).T      # head h uses G = h + 1
    r = Hq // Hkv
    for l in range(L):
        got = O.pod_decode_layer(q, K, V, l, lowest=low, n_s=S, n_r=W)
        for h in range(Hq):
            kv = h // r
            ref_g = O.pod_decode_layer(q, K, V, l, group_size=kv + 1, n_s=S, n_r=W)[h]
            np.testing.assert_allclose(got[h], ref_g, rtol=0, atol=1e-14)
            a = int(low[l, kv])
            logits = []
            for p in range(n):
                prox = p < S or p >= n - W
                qq, kk = (q[l, h], K[l, p, kv]) if prox else (q[a, h], K[a, p, kv])
                logits.append(sum(float(x) * float(y) for x, y in zip(qq, kk)) / np.sqrt(d))
            m = max(logits)
            w = [np.exp(x - m) for x in logits]
            z = sum(w)
            ref = [sum(w[p] / z * float(V[l, p, kv, c]) for p in range(n)) for c in range(d)]
            np.testing.assert_allclose(got[h], ref, rtol=0, atol=1e-12)


def _bits(rng, *shape):
    return (rng.standard_normal(shape).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def test_head_wise_layout_incremental_equals_direct_and_attend_equals_definition():
    rng = np.random.default_rng(2)
    L, n, Hq, Hkv, d, S, W = 5, 31, 4, 2, 8, 2, 6
    low = np.array([[0, 0], [0, 1], [0, 1], [3, 1], [3, 4]])
    Kb, Vb = _bits(rng, L, n, Hkv, d), _bits(rng, L, n, Hkv, d)
    inc = O.PodCacheOracle(L, Hkv, d, None, S, W, n + 3, lowest=low)
    for l in range(L):
        inc.write(l, Kb[l], Vb[l])
    direct = O.layout_from_history(Kb, Vb, lowest=low, n_s=S, n_r=W, capacity=n + 3)
    assert inc.blocks == [[0, 3], [0, 1, 4]]
    for name in ("sinkK", "sinkV", "ringK", "ringV", "distK", "distV"):
        count = inc.n_blocks if name == "distK" else L
        for i in range(count):
            for h in range(Hkv):
                a, _ = inc.valid_rows(name, i, h)
                b, _ = direct.valid_rows(name, i, h)
                np.testing.assert_array_equal(a, b)
    # distant keys of head 1, block 1 (layers 1..3) are layer 1's keys
    np.testing.assert_array_equal(inc.valid_rows("distK", 1, 1)[0], Kb[1, S:n - W, 1])
    assert inc.valid_rows("distK", 2, 0)[0].shape[0] == 0           # head 0 has two blocks only
    K, V = O.bits_to_f64(Kb), O.bits_to_f64(Vb)
    q = O.bits_to_f64(_bits(rng, L, Hq, d))
    r = Hq // Hkv
    for l in range(L):
        q_low = np.stack([q[int(low[l, h // r]), h] for h in range(Hq)])
        np.testing.assert_allclose(inc.attend(l, q[l], q_low),
                                   O.pod_decode_layer(q, K, V, l, lowest=low, n_s=S, n_r=W), rtol=0, atol=1e-12)


def test_head_wise_byte_counts():
    """Enumeration of the rows kept against the count, and the closed form with the fraction of
    (layer, head) pairs that share.  A map in which 70 % of the pairs share reproduces the paper's
    35 % in the limit of long contexts (Section 3: about 35 % of the KV cache saved)."""
    L, H, d, S, W, n = 10, 4, 16, 4, 12, 500
    rng = np.random.default_rng(3)
    low = np.zeros((L, H), dtype=np.int64)
    for h in range(H):
        for l in range(1, L):
            low[l, h] = l if rng.random() < 0.4 else low[l - 1, h]
    live, dense = O.pod_cache_bytes([n], n_layers=L, n_kv_heads=H, head_dim=d, lowest=low, n_s=S, n_r=W)
    rows = 0
    for l in range(L):
        for h in range(H):
            for p in range(n):
                prox = p < S or p >= n - W
                rows += 2 if (prox or low[l, h] == l) else 1
    assert live == rows * d * 2 and dense == L * H * n * 2 * d * 2
    shared = float(np.mean(low != np.arange(L)[:, None]))
    assert abs((1 - live / dense) - O.pod_saving_closed_form(n, n_layers=L, n_s=S, n_r=W, shared_fraction=shared)) < 1e-12
    assert abs(O.pod_saving_closed_form(10 ** 9, n_layers=32, n_s=16, n_r=4080, shared_fraction=0.7) - 0.35) < 1e-5


# --------------------------------------------------------------------------- gate threshold (distant skip)
def _one_head(rng, n, d):
    bf = lambda x: (x.astype(np.float32).view(np.uint32) & 0xFFFF0000).view(np.float32).astype(np.float64)
    return (bf(rng.standard_normal(d)), bf(rng.standard_normal(d)), bf(rng.standard_normal((n, d))),
            bf(rng.standard_normal((n, d))), bf(rng.standard_normal((n, d))))


def test_gate_skip_limits_and_identity():
    """tau above 1 never skips and gives the joint softmax; tau = 0 always skips and gives textbook
    attention over the proximal tokens alone (torch SDPA); in between the decision is g >= tau, and
    the two candidate outputs differ by exactly (1 - g)(o^P - o^D)."""
    import torch
    rng = np.random.default_rng(4)
    n, d, S, W = 60, 16, 3, 9
    q_l, q_a, K_l, K_a, V_l = _one_head(rng, n, d)
    full, _ = O.pod_attention_joint(q_l, q_a, K_l, K_a, V_l, S, W)
    o, g, skipped = O.pod_attention_gate_skip(q_l, q_a, K_l, K_a, V_l, S, W, tau=1.5)
    assert not skipped and 0 < g < 1
    np.testing.assert_allclose(o, full, rtol=0, atol=1e-12)
    o0, g0, skipped0 = O.pod_attention_gate_skip(q_l, q_a, K_l, K_a, V_l, S, W, tau=0.0)
    assert skipped0 and g0 == g
    prox = np.array([p < S or p >= n - W for p in range(n)])
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q_l)[None, None], torch.tensor(K_l[prox])[None], torch.tensor(V_l[prox])[None])[0, 0].numpy()
    np.testing.assert_allclose(o0, ref, rtol=0, atol=1e-12)
    # the decision flips exactly at g
    assert O.pod_attention_gate_skip(q_l, q_a, K_l, K_a, V_l, S, W, tau=g)[2]
    assert not O.pod_attention_gate_skip(q_l, q_a, K_l, K_a, V_l, S, W, tau=np.nextafter(g, 1.0))[2]
    # o_full = g o^P + (1 - g) o^D  =>  o^P - o_full = (1 - g)(o^P - o^D)
    dist = ~prox
    a = (K_a[dist] @ q_a) / np.sqrt(d)
    w = np.exp(a - a.max()); w /= w.sum()
    oD = w @ V_l[dist]
    np.testing.assert_allclose(o0 - full, (1 - g) * (o0 - oD), rtol=0, atol=1e-12)
    # no distant tokens: nothing to skip, result is dense attention
    o_s, g_s, sk = O.pod_attention_gate_skip(q_l, q_a, K_l[:10], K_a[:10], V_l[:10], S, W, tau=0.0)
    assert g_s == 1.0 and not sk


def test_gate_skip_applies_to_non_lowest_layers_only_and_is_monotone_in_tau():
    rng = np.random.default_rng(6)
    L, n, Hq, Hkv, d, S, W = 4, 80, 4, 2, 8, 2, 10
    q, K, V = _inputs(rng, L, n, Hq, Hkv, d)
    K[1, S:n - W] *= 0.05                                       # irrelevant: layer 1 scores with layer 0's keys
    q[0] *= 0.2                                                 # weak distant logits for block 0 ...
    q[1] *= 3.0                                                 # ... strong proximal ones at layer 1
    for l in range(L):
        info = []
        got = O.pod_decode_layer(q, K, V, l, group_size=2, n_s=S, n_r=W, tau=0.0, info=info)
        if l % 2 == 0:                                          # lowest layers never skip
            assert all(not sk for _, sk in info)
            np.testing.assert_array_equal(got, O.pod_decode_layer(q, K, V, l, group_size=2, n_s=S, n_r=W))
        else:
            assert all(sk for _, sk in info)
    prev = None
    for tau in (1.1, 0.9, 0.7, 0.5, 0.3, 0.0):
        info = []
        O.pod_decode_layer(q, K, V, 1, group_size=2, n_s=S, n_r=W, tau=tau, info=info)
        skipped = [sk for _, sk in info]
        assert skipped == [g >= tau for g, _ in info]
        if prev is not None:
            assert all(b or not a for a, b in zip(prev, skipped))     # once skipped, skipped for smaller tau
        prev = skipped
    gs = [g for g, _ in info]
    assert max(gs) > 0.5                                              # the construction gives a confident gate


# --------------------------------------------------------------------------- prefill (all positions)
def test_prefill_oracle_against_causal_attention_and_explicit_masks():
    """For a lowest layer the prefill form is ordinary causal attention (torch SDPA, is_causal); for
    another layer it equals a softmax over a matrix of logits assembled with the proximal / distant
    masks of Fig. 2 (middle) written out explicitly; its last row is the decode step."""
    import torch
    rng = np.random.default_rng(8)
    L, n, Hq, Hkv, d, S, W = 2, 45, 4, 2, 8, 3, 7
    bf = lambda x: (x.astype(np.float32).view(np.uint32) & 0xFFFF0000).view(np.float32).astype(np.float64)
    q = bf(rng.standard_normal((L, n, Hq, d)))
    K, V = bf(rng.standard_normal((L, n, Hkv, d))), bf(rng.standard_normal((L, n, Hkv, d)))
    r = Hq // Hkv
    o0 = O.pod_prefill_layer(q, K, V, 0, group_size=2, n_s=S, n_r=W)
    for h in range(Hq):
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.tensor(q[0, :, h])[None], torch.tensor(K[0, :, h // r])[None], torch.tensor(V[0, :, h // r])[None],
            is_causal=True)[0].numpy()
        np.testing.assert_allclose(o0[:, h], ref, rtol=0, atol=1e-12)
    o1 = O.pod_prefill_layer(q, K, V, 1, group_size=2, n_s=S, n_r=W)
    i = np.arange(n)[:, None]
    j = np.arange(n)[None, :]
    causal = j <= i
    prox = (j < S) | (j > i - W)                 # the last W tokens up to and including i
    for h in range(Hq):
        kv = h // r
        own = q[1, :, h] @ K[1, :, kv].T / np.sqrt(d)
        low = q[0, :, h] @ K[0, :, kv].T / np.sqrt(d)
        a = np.where(prox, own, low)
        a = np.where(causal, a, -np.inf)
        w = np.exp(a - a.max(axis=1, keepdims=True))
        w /= w.sum(axis=1, keepdims=True)
        np.testing.assert_allclose(o1[:, h], w @ V[1, :, kv], rtol=0, atol=1e-12)
    np.testing.assert_allclose(o1[-1], O.pod_decode_layer(q[:, -1], K, V, 1, group_size=2, n_s=S, n_r=W), rtol=0, atol=0)
