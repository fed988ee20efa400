"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is independent of the oracle's own
code path: a library routine (torch SDPA in fp64), pure-Python loops, rational numbers
worked by hand, closed forms, or invariants.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import pod_oracle as O
from paper_2412_02252_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_history(rng, L, n, H, d):
    return rng.standard_normal((L, n, H, d)), rng.standard_normal((L, n, H, d))


def _sdpa_dense(q, K, V, scale):
    """Textbook dense attention through a library routine (torch, fp64)."""
    qt = torch.from_numpy(q)[None, None, None, :]
    kt = torch.from_numpy(K)[None, None]
    vt = torch.from_numpy(V)[None, None]
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=scale)
    return o[0, 0, 0].numpy()


# ---------------------------------------------------------------- hand-worked example
def _load_example():
    vals = {}
    with open(os.path.join(GOLDEN, "hand_worked_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, *v = line.split()
                vals[k] = np.array([float(x) for x in v])
    return vals


def test_hand_worked_example():
    ex = _load_example()
    K1 = np.log(np.stack([ex["a"], ex["c"]], axis=1))
    K0 = np.log(np.stack([ex["e"], ex["b"]], axis=1))
    V1, V0 = ex["V1"].reshape(4, 2), ex["V0"].reshape(4, 2)
    q1, q0 = np.array([1.0, 0.0]), np.array([0.0, 1.0])
    o1, w1 = O.pod_attention_joint(q1, q0, K1, K0, V1, 1, 1, scale=1.0)
    np.testing.assert_allclose(o1, ex["expect_o1"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(w1, [0.1, 0.2, 0.4, 0.3], rtol=0, atol=1e-14)
    og, g = O.pod_attention_gate(q1, q0, K1, K0, V1, 1, 1, scale=1.0)
    np.testing.assert_allclose(og, ex["expect_o1"], rtol=0, atol=1e-12)
    assert abs(g - ex["expect_g1"][0]) < 1e-14
    # lowest layer: ordinary attention with its own q, K, V
    o0, _ = O.pod_attention_joint(q0, q0, K0, K0, V0, 1, 1, scale=1.0)
    np.testing.assert_allclose(o0, ex["expect_o0"], rtol=0, atol=1e-12)
    # through the all-heads entry point, blocks of 2 and of 1
    q = np.stack([q0, q1])[:, None, :]
    K = np.stack([K0, K1])[:, :, None, :]
    V = np.stack([V0, V1])[:, :, None, :]
    o = O.pod_decode_layer(q, K, V, 1, group_size=2, n_s=1, n_r=1, scale=1.0)
    np.testing.assert_allclose(o[0], ex["expect_o1"], atol=1e-12)
    o = O.pod_decode_layer(q, K, V, 1, group_size=2, n_s=1, n_r=1, scale=1.0, form="gate")
    np.testing.assert_allclose(o[0], ex["expect_o1"], atol=1e-12)
    o = O.pod_decode_layer(q, K, V, 1, group_size=1, n_s=1, n_r=1, scale=1.0)
    np.testing.assert_allclose(o[0], ex["expect_o1_dense"], atol=1e-12)
    # the two partial outputs of Eq. 1
    a, prox = O.pod_logits(q1, q0, K1, K0, 1, 1, 1.0)
    np.testing.assert_allclose(O._softmax(a[prox]) @ V1[prox], ex["expect_o1P"], atol=1e-12)
    np.testing.assert_allclose(O._softmax(a[~prox]) @ V1[~prox], ex["expect_o1D"], atol=1e-12)


def test_hand_worked_example_layout_form():
    """Same example through the cache layout: K/V rounded to bf16 first, so compare with the
    definition form on the rounded values and with the exact rationals loosely."""
    ex = _load_example()
    K1 = np.log(np.stack([ex["a"], ex["c"]], axis=1))
    K0 = np.log(np.stack([ex["e"], ex["b"]], axis=1))
    V1, V0 = ex["V1"].reshape(4, 2), ex["V0"].reshape(4, 2)
    to_bits = lambda x: synth.bf16_bits(torch.from_numpy(x).to(torch.bfloat16))
    Kb = np.stack([to_bits(K0), to_bits(K1)])[:, :, None, :]
    Vb = np.stack([to_bits(V0), to_bits(V1)])[:, :, None, :]
    c = O.PodCacheOracle(2, 1, 2, 2, 1, 1, capacity=8)
    for l in range(2):
        c.write(l, Kb[l], Vb[l])
    q = np.array([[[0.0, 1.0]], [[1.0, 0.0]]])
    o1 = c.attend(1, q[1], q[0], scale=1.0)
    ref = O.pod_decode_layer(q, O.bits_to_f64(Kb), O.bits_to_f64(Vb), 1, group_size=2,
                             n_s=1, n_r=1, scale=1.0)
    np.testing.assert_allclose(o1, ref, atol=1e-12)
    np.testing.assert_allclose(o1[0], ex["expect_o1"], atol=0.1)


# ---------------------------------------------------------------- definition pins
@pytest.mark.parametrize("n,n_s,n_r", [(1, 2, 3), (5, 2, 3), (6, 2, 3), (17, 2, 3), (40, 4, 8)])
def test_weights_sum_to_one_and_gate_identity(n, n_s, n_r):
    rng = np.random.default_rng(n)
    d = 16
    q_l, q_a = rng.standard_normal(d), rng.standard_normal(d)
    K_l, K_a, V_l = (rng.standard_normal((n, d)) for _ in range(3))
    o, w = O.pod_attention_joint(q_l, q_a, K_l, K_a, V_l, n_s, n_r)
    assert abs(w.sum() - 1.0) < 1e-12 and (w >= 0).all()
    og, g = O.pod_attention_gate(q_l, q_a, K_l, K_a, V_l, n_s, n_r)
    np.testing.assert_allclose(o, og, rtol=0, atol=1e-12)       # Appendix C identity
    assert 0.0 <= g <= 1.0
    if n <= n_s + n_r:
        assert g == 1.0                                         # distant term omitted


def test_block_of_one_layer_is_dense_attention():
    rng = np.random.default_rng(1)
    L, n, H, d, Hq = 3, 50, 2, 32, 4
    K, V = _rand_history(rng, L, n, H, d)
    q = rng.standard_normal((L, Hq, d))
    for layer in range(L):
        o = O.pod_decode_layer(q, K, V, layer, group_size=1, n_s=4, n_r=8)
        for h in range(Hq):
            ref = _sdpa_dense(q[layer, h], K[layer, :, h // 2], V[layer, :, h // 2], 1 / math.sqrt(d))
            np.testing.assert_allclose(o[h], ref, rtol=0, atol=1e-12)


def test_lowest_layer_of_block_is_dense_attention():
    rng = np.random.default_rng(2)
    L, n, H, d = 4, 33, 1, 8
    K, V = _rand_history(rng, L, n, H, d)
    q = rng.standard_normal((L, 2, d))
    for layer in (0, 2):
        o = O.pod_decode_layer(q, K, V, layer, group_size=2, n_s=3, n_r=5)
        for h in range(2):
            ref = _sdpa_dense(q[layer, h], K[layer, :, 0], V[layer, :, 0], 1 / math.sqrt(d))
            np.testing.assert_allclose(o[h], ref, atol=1e-12)


@pytest.mark.parametrize("n", [1, 3, 7, 8])
def test_no_distant_tokens_is_dense_attention(n):
    rng = np.random.default_rng(3)
    L, H, d = 2, 1, 8
    K, V = _rand_history(rng, L, n, H, d)
    q = rng.standard_normal((L, 1, d))
    o = O.pod_decode_layer(q, K, V, 1, group_size=2, n_s=3, n_r=5)       # n <= n_s + n_r
    ref = _sdpa_dense(q[1, 0], K[1, :, 0], V[1, :, 0], 1 / math.sqrt(d))
    np.testing.assert_allclose(o[0], ref, atol=1e-12)


def test_identical_layers_in_block_give_dense():
    """If q and K coincide across a block the shared scores are the layer's own scores."""
    rng = np.random.default_rng(4)
    L, n, H, d = 2, 40, 1, 8
    K, V = _rand_history(rng, L, n, H, d)
    K[1] = K[0]
    q = rng.standard_normal((L, 1, d))
    q[1] = q[0]
    o = O.pod_decode_layer(q, K, V, 1, group_size=2, n_s=2, n_r=6)
    ref = _sdpa_dense(q[1, 0], K[1, :, 0], V[1, :, 0], 1 / math.sqrt(d))
    np.testing.assert_allclose(o[0], ref, atol=1e-12)


def test_distant_weight_ratios_follow_lowest_layer_query():
    rng = np.random.default_rng(5)
    n, d, n_s, n_r = 30, 8, 2, 4
    K_l, K_a, V_l = (rng.standard_normal((n, d)) for _ in range(3))
    q_l, q_a = rng.standard_normal(d), rng.standard_normal(d)
    _, w = O.pod_attention_joint(q_l, q_a, K_l, K_a, V_l, n_s, n_r)
    _, w2 = O.pod_attention_joint(q_l + rng.standard_normal(d), q_a, K_l, K_a, V_l, n_s, n_r)
    dist = slice(n_s, n - n_r)
    np.testing.assert_allclose(w[dist] / w[dist].sum(), w2[dist] / w2[dist].sum(), rtol=1e-12)
    assert not np.allclose(w[dist].sum(), w2[dist].sum())
    _, w3 = O.pod_attention_joint(q_l, q_a + rng.standard_normal(d), K_l, K_a, V_l, n_s, n_r)
    assert not np.allclose(w[dist] / w[dist].sum(), w3[dist] / w3[dist].sum())
    # distant ratios are softmax(q_a . K_a): they ignore layer l's keys altogether
    _, w4 = O.pod_attention_joint(q_l, q_a, K_l + 1.0, K_a, V_l, n_s, n_r)
    np.testing.assert_allclose(w[dist] / w[dist].sum(), w4[dist] / w4[dist].sum(), rtol=1e-12)


def _brute_force(q, K, V, layer, G, n_s, n_r):
    """Pure-Python per-token loops straight from Eq. 1 / Appendix C (one sequence)."""
    n, H, d = len(K[0]), len(K[0][0]), len(K[0][0][0])
    Hq = len(q[0])
    r = Hq // H
    a = layer - layer % G
    out = [[0.0] * d for _ in range(Hq)]
    for h in range(Hq):
        kv = h // r
        logit = []
        for p in range(n):
            if p < n_s or p >= n - n_r:
                s = sum(q[layer][h][c] * K[layer][p][kv][c] for c in range(d))
            else:
                s = sum(q[a][h][c] * K[a][p][kv][c] for c in range(d))
            logit.append(s / math.sqrt(d))
        m = max(logit)
        den = sum(math.exp(x - m) for x in logit)
        for p in range(n):
            w = math.exp(logit[p] - m) / den
            for c in range(d):
                out[h][c] += w * V[layer][p][kv][c]
    return np.array(out)


def test_brute_force_definition_and_layout_all_lengths():
    """Definition form, gate form, layout form and brute force agree for every length from 1
    to 3 (n_s + n_r), covering: inside the sink, partial ring, first distant token, wraps."""
    L, H, Hq, d, G, n_s, n_r = 3, 2, 4, 4, 2, 2, 3
    n_max = 3 * (n_s + n_r)
    Kt = torch.stack([synth.gen_kv(7, synth.TAG_K, l, 0, 0, n_max, H, d) for l in range(L)])
    Vt = torch.stack([synth.gen_kv(7, synth.TAG_V, l, 0, 0, n_max, H, d) for l in range(L)])
    Kb, Vb = synth.bf16_bits(Kt), synth.bf16_bits(Vt)
    K, V = O.bits_to_f64(Kb), O.bits_to_f64(Vb)
    np.testing.assert_array_equal(K, Kt.double().numpy())
    cache = O.PodCacheOracle(L, H, d, G, n_s, n_r, capacity=n_max)
    for n in range(1, n_max + 1):
        q = torch.stack([synth.gen_q(7, l, n, 1, Hq, d)[0] for l in range(L)]).double().numpy()
        for l in range(L):
            cache.append(l, Kb[l, n - 1], Vb[l, n - 1])
        for l in range(L):
            ref = _brute_force(q.tolist(), K[:, :n].tolist(), V[:, :n].tolist(), l, G, n_s, n_r)
            o_def = O.pod_decode_layer(q, K[:, :n], V[:, :n], l, group_size=G, n_s=n_s, n_r=n_r)
            o_gate = O.pod_decode_layer(q, K[:, :n], V[:, :n], l, group_size=G, n_s=n_s,
                                        n_r=n_r, form="gate")
            o_lay = cache.attend(l, q[l], q[l - l % G])
            np.testing.assert_allclose(o_def, ref, rtol=0, atol=1e-12)
            np.testing.assert_allclose(o_gate, ref, rtol=0, atol=1e-12)
            np.testing.assert_allclose(o_lay, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("where", ["first", "last_sink", "first_distant", "last_distant",
                                   "first_recent", "current", "ring_slot0", "ring_last_slot"])
@pytest.mark.parametrize("layer", [0, 1])
def test_planted_key_selects_that_tokens_value(where, layer):
    """A key equal to a large multiple of the query that scores it dominates the softmax, so
    the output is that token's value row (layer's own V) wherever the token sits."""
    rng = np.random.default_rng(11)
    L, n, d, n_s, n_r, G = 2, 41, 8, 4, 8, 2
    pos = {"first": 0, "last_sink": n_s - 1, "first_distant": n_s, "last_distant": n - n_r - 1,
           "first_recent": n - n_r, "current": n - 1,
           "ring_slot0": next(p for p in range(n - n_r, n) if (p - n_s) % n_r == 0),
           "ring_last_slot": next(p for p in range(n - n_r, n) if (p - n_s) % n_r == n_r - 1)}[where]
    K, V = _rand_history(rng, L, n, 1, d)
    q = rng.standard_normal((L, 1, d))
    distant = n_s <= pos < n - n_r
    src = 0 if (distant and layer == 1) else layer        # whose query/key scores this token
    K[src, pos, 0] = 200.0 * q[src, 0] / np.linalg.norm(q[src, 0])
    o = O.pod_decode_layer(q, K, V, layer, group_size=G, n_s=n_s, n_r=n_r)
    np.testing.assert_allclose(o[0], V[layer, pos, 0], atol=1e-6)
    # and through the layout
    to_bits = lambda x: synth.bf16_bits(torch.from_numpy(x).to(torch.bfloat16))
    Kb, Vb = to_bits(K), to_bits(V)
    c = O.PodCacheOracle(L, 1, d, G, n_s, n_r, capacity=n)
    for l in range(L):
        c.write(l, Kb[l], Vb[l])
    qb = O.bits_to_f64(to_bits(q))
    o2 = c.attend(layer, qb[layer], qb[layer - layer % G])
    np.testing.assert_allclose(o2[0], O.bits_to_f64(Vb)[layer, pos, 0], atol=1e-6)


# ---------------------------------------------------------------- layout / update rule
@pytest.mark.parametrize("chunks", [[1] * 30, [30], [7, 1, 1, 13, 8], [2, 9, 19], [5, 25]])
def test_incremental_layout_equals_layout_from_history(chunks):
    L, H, d, G, n_s, n_r = 3, 2, 4, 2, 2, 5
    n = sum(chunks)
    Kb = synth.bf16_bits(torch.stack([synth.gen_kv(3, synth.TAG_K, l, 0, 0, n, H, d) for l in range(L)]))
    Vb = synth.bf16_bits(torch.stack([synth.gen_kv(3, synth.TAG_V, l, 0, 0, n, H, d) for l in range(L)]))
    c = O.PodCacheOracle(L, H, d, G, n_s, n_r, capacity=n)
    at = 0
    for t in chunks:
        for l in range(L):
            c.write(l, Kb[l, at:at + t], Vb[l, at:at + t])
        at += t
        ref = O.layout_from_history(Kb[:, :at], Vb[:, :at], group_size=G, n_s=n_s, n_r=n_r, capacity=n)
        for region, count in (("sinkK", L), ("sinkV", L), ("ringK", L), ("ringV", L),
                              ("distV", L), ("distK", c.n_blocks)):
            for i in range(count):
                for h in range(H):
                    a, _ = c.valid_rows(region, i, h)
                    b, _ = ref.valid_rows(region, i, h)
                    np.testing.assert_array_equal(a, b)
    # distant keys of non-lowest layers are nowhere: block store holds the lowest layer's
    n_d = n - n_s - n_r
    np.testing.assert_array_equal(c.distK[0, :, :n_d], Kb[0, n_s:n - n_r].transpose(1, 0, 2))
    np.testing.assert_array_equal(c.distK[1, :, :n_d], Kb[2, n_s:n - n_r].transpose(1, 0, 2))
    np.testing.assert_array_equal(c.distV[1, :, :n_d], Vb[1, n_s:n - n_r].transpose(1, 0, 2))


def test_capacity_is_enforced():
    c = O.PodCacheOracle(1, 1, 2, 1, 1, 1, capacity=2)
    row = np.zeros((1, 2), dtype=np.uint16)
    c.append(0, row, row)
    c.append(0, row, row)
    with pytest.raises(ValueError):
        c.append(0, row, row)


# ---------------------------------------------------------------- byte accounting
CFG8B = dict(n_layers=32, n_kv_heads=8, head_dim=128)


@pytest.mark.parametrize("lens,kw,live,dense,saving", [
    ([512], dict(n_layers=4, n_kv_heads=2, head_dim=64, group_size=2, n_s=16, n_r=64),
     827392, 1048576, 0.2109375),
    ([32768], dict(CFG8B, group_size=2, n_s=16, n_r=2048), None, 4 << 30, 0.234252929688),
    ([32768] * 16, dict(CFG8B, group_size=4, n_s=16, n_r=1024), None, 64 << 30, 0.363098144531),
    ([131072], dict(CFG8B, group_size=2, n_s=16, n_r=4096), 13019643904, 16 << 30,
     0.242156982422),
])
def test_cache_bytes_closed_form(lens, kw, live, dense, saving):
    lv, dn = O.pod_cache_bytes(lens, **kw)
    assert dn == dense
    if live is not None:
        assert lv == live
    assert abs((1 - lv / dn) - saving) < 1e-9
    cf = O.pod_saving_closed_form(lens[0], n_layers=kw["n_layers"], group_size=kw["group_size"],
                                  n_s=kw["n_s"], n_r=kw["n_r"])
    assert abs((1 - lv / dn) - cf) < 1e-12


def test_cache_bytes_count_the_layout_regions():
    """Byte count == number of valid rows actually held by the layout oracle."""
    L, H, d, G, n_s, n_r, n = 5, 2, 4, 2, 3, 4, 20          # last block is short (G does not divide L)
    c = O.PodCacheOracle(L, H, d, G, n_s, n_r, capacity=n)
    row = np.zeros((H, d), dtype=np.uint16)
    for l in range(L):
        for _ in range(n):
            c.append(l, row, row)
    rows = 0
    for region, count in (("sinkK", L), ("sinkV", L), ("ringK", L), ("ringV", L), ("distV", L),
                          ("distK", c.n_blocks)):
        for i in range(count):
            for h in range(H):
                rows += c.valid_rows(region, i, h)[0].shape[0]
    lv, dn = O.pod_cache_bytes([n], n_layers=L, n_kv_heads=H, head_dim=d, group_size=G, n_s=n_s, n_r=n_r)
    assert lv == rows * d * 2
    assert dn == L * 2 * n * H * d * 2


def test_saving_limits_and_paper_arithmetic():
    vals = {}
    with open(os.path.join(GOLDEN, "paper_saving_arithmetic.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                vals[line[0]] = float(line[1])
    # only keys are shared: below one half for every G, one half in the limit n_d/n -> 1, G -> L
    for G in (1, 2, 3, 4, 8, 32):
        s = O.pod_saving_closed_form(10 ** 9, n_layers=32, group_size=G, n_s=16, n_r=4080)
        assert s < 0.5
        assert abs(s - (1 - math.ceil(32 / G) / 32) / 2) < 1e-5
    assert O.pod_saving_closed_form(4096, n_layers=32, group_size=2, n_s=16, n_r=4080) == 0.0
    # sharing K *and* V between 2 layers (CLA) would be one half exactly
    assert vals["cla_factor2"] == 50.0
    # token selection to 4096 of 32768 tokens and its composition with a flat 35 % saving
    assert abs(100 * (1 - 4096 / 32768) - vals["snapkv"]) < 1e-12
    assert round(100 * (1 - (4096 / 32768) * (1 - vals["pod_flat"] / 100)), 1) == vals["pod_plus_snapkv"]
    # the flat 35 % at n = 32768, n_s + n_r = 4096 means 80 % of (layer, head) distant keys dropped
    frac_dropped = (vals["pod_flat"] / 100) * 2 / ((32768 - 4096) / 32768)
    assert abs(frac_dropped - 0.8) < 1e-12


# ---------------------------------------------------------------- generator sanity
def test_generator_is_addressable_and_normal():
    full = synth.gen_kv(5, synth.TAG_K, 3, 1, 0, 64, 4, 16, outliers=True)
    part = synth.gen_kv(5, synth.TAG_K, 3, 1, 10, 20, 4, 16, outliers=True, heads=[2])
    assert torch.equal(full[10:20, 2:3], part)
    x = synth.gen_kv(0, synth.TAG_V, 0, 0, 0, 4096, 8, 128).float()
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1) < 5e-3
    a = synth.gen_kv(0, synth.TAG_K, 0, 0, 0, 256, 8, 128).float().flatten()
    b = synth.gen_kv(0, synth.TAG_K, 1, 0, 0, 256, 8, 128).float().flatten()
    assert abs(torch.corrcoef(torch.stack([a, b]))[0, 1]) < 0.01
    m = synth.outlier_channels(0, synth.TAG_K, 0, 8, 128)
    assert 0 < m.sum() < 40
    lens = synth.ragged_lengths(5, 32, 4096, 65536)
    assert len(lens) == 32 and min(lens) >= 4096 and max(lens) <= 65536 and len(set(lens)) > 20
