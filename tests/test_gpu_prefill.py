"""GPU parity of pod_prefill_attn (PoD attention for every position, tcgen05 tensor cores) against the
fp64 oracle's prefill form, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import pod_oracle as O
from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth
from podtest import MAX_ABS, REL_L2

pytestmark = pytest.mark.gpu


def _inputs(seed, T, Hq, Hkv, d=128, outliers=False):
    kv = lambda tag, layer: synth.gen_kv(seed, tag, layer, 0, 0, T, Hkv, d, outliers=outliers, device="cuda")
    # queries of every position: the generator's "step" axis is the position
    q = lambda layer: torch.stack([synth.gen_q(seed, layer, t, 1, Hq, d, device="cuda")[0] for t in range(0, T, 1)]) \
        if T <= 64 else synth.gen_kv(seed, synth.TAG_Q, layer, 0, 0, T, Hq, d, device="cuda")
    return q, kv


def _check(got, ref, what, V):
    """Relative L2 as everywhere.  The absolute bound of the decode tests (1e-2) suits outputs that
    average thousands of value rows; the first positions of a prefill attend to a handful of tokens,
    so their outputs are as large as single value rows (up to 35 in an outlier channel).  Two roundings
    to bf16 are part of the method's arithmetic here -- the probabilities fed to the tensor cores and the
    output -- each at most 2^-9 relative, so an output channel c may move by 2^-9 sum_j p_j |v_jc| +
    2^-9 |o_c| <= 2^-8 max_j |v_jc|: that term is added per (KV head, channel)."""
    g = got.double().cpu().numpy()
    err = np.abs(g - ref)
    rel = np.linalg.norm(g - ref) / max(np.linalg.norm(ref), 1e-30)
    vmax = V.double().abs().amax(dim=0).cpu().numpy()                      # [H_kv][d]
    r = got.shape[1] // V.shape[1]
    bound = MAX_ABS + 2.0 ** -8 * np.repeat(vmax, r, axis=0)[None]           # [1][H_q][d]
    assert (err <= bound).all() and rel <= REL_L2, f"{what}: max_abs={err.max():.3e} rel_l2={rel:.3e}"


@pytest.mark.parametrize("T,S,W", [(1, 4, 32), (5, 4, 32), (64, 4, 32), (129, 4, 32), (700, 16, 200), (777, 0, 65),
                                   (1000, 4, 300), (513, 70, 64)])
def test_prefill_lowest_layer_is_causal_attention(T, S, W):
    """A layer that is the lowest of every head's block: ragged tails, several query blocks and key tiles."""
    Hq, Hkv = 4, 2
    q, kv = _inputs(31, T, Hq, Hkv)
    Q, K, V = q(0), kv(synth.TAG_K, 0), kv(synth.TAG_V, 0)
    out = torch.zeros(T, Hq, 128, dtype=torch.bfloat16, device="cuda")
    B.pod_prefill_attn(Q, K, V, out, n_sink=S, n_recent=W)
    torch.cuda.synchronize()
    assert B.pod_prefill_status() == B.POD_OK
    f = lambda x: x.double().cpu().numpy()
    ref = O.pod_prefill_layer(f(Q)[None], f(K)[None], f(V)[None], 0, group_size=1, n_s=S, n_r=W)
    _check(out, ref, f"T={T}", V)


@pytest.mark.parametrize("T,S,W,shares", [(300, 4, 32, None), (700, 16, 200, None), (1000, 4, 300, [1, 0]),
                                          (450, 0, 64, [0, 1]), (200, 130, 10, None), (90, 4, 200, None),
                                          (600, 300, 1, None), (257, 0, 1, None), (256, 128, 128, [1, 1]), (1, 0, 1, None),
                                          (640, 256, 127, None)])
def test_prefill_sharing_layer(T, S, W, shares):
    """A layer whose distant logits come from the block's lowest layer (all heads, or some: head-wise
    blocks); windows that cross tile boundaries, a sink longer than a tile, a window longer than the
    sequence (everything proximal)."""
    Hq, Hkv = 8, 2
    q, kv = _inputs(32, T, Hq, Hkv, outliers=True)
    Q = [q(l) for l in range(2)]
    K = [kv(synth.TAG_K, l) for l in range(2)]
    V = [kv(synth.TAG_V, l) for l in range(2)]
    out = torch.zeros(T, Hq, 128, dtype=torch.bfloat16, device="cuda")
    B.pod_prefill_attn(Q[1], K[1], V[1], out, n_sink=S, n_recent=W, q_low=Q[0], k_low=K[0], head_shares=shares)
    torch.cuda.synchronize()
    assert B.pod_prefill_status() == B.POD_OK
    f = lambda xs: np.stack([x.double().cpu().numpy() for x in xs])
    low = [[0, 0], [0 if (shares is None or shares[0]) else 1, 0 if (shares is None or shares[1]) else 1]]
    ref = O.pod_prefill_layer(f(Q), f(K), f(V), 1, lowest=np.array(low), n_s=S, n_r=W)
    _check(out, ref, f"T={T} shares={shares}", V[1])


def test_prefill_matches_decode_steps():
    """The last rows of a prefill are what the decode path returns for the same tokens fed one by one."""
    T, Hq, Hkv, S, W = 600, 8, 2, 4, 64
    q, kv = _inputs(33, T, Hq, Hkv)
    Q = [q(l) for l in range(2)]
    K = [kv(synth.TAG_K, l) for l in range(2)]
    V = [kv(synth.TAG_V, l) for l in range(2)]
    outs = [torch.zeros(T, Hq, 128, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    B.pod_prefill_attn(Q[0], K[0], V[0], outs[0], n_sink=S, n_recent=W)
    B.pod_prefill_attn(Q[1], K[1], V[1], outs[1], n_sink=S, n_recent=W, q_low=Q[0], k_low=K[0])
    cfg = B.make_config(n_layers=2, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=128, group_size=2, n_sink=S, n_recent=W,
                        batch=1, device=0)
    cache = B.PodCache(cfg, [T])
    first = T - 5
    for l in range(2):
        cache.write(l, 0, K[l][:first], V[l][:first], first)
    dec = torch.zeros(2, 1, Hq, 128, dtype=torch.bfloat16, device="cuda")
    for t in range(first, T):
        for l in range(2):
            cache.append_decode_attn(l, K[l][t:t + 1], V[l][t:t + 1], Q[l][t:t + 1], dec[l])
        torch.cuda.synchronize()
        for l in range(2):
            d = (dec[l, 0].float() - outs[l][t].float()).abs().max().item()
            assert d <= 2e-2, (t, l, d)                 # two bf16 results of the same quantity (averages over 600 tokens)
    assert cache.device_status() == B.POD_OK and B.pod_prefill_status() == B.POD_OK


@pytest.mark.parametrize("T,S,W", [(8192, 16, 2048), (5000, 0, 1000)])
def test_prefill_long_sequence_sampled_rows(T, S, W):
    """A sequence of many query blocks and key tiles (the ring of K/V slots wraps many times, the passes
    with the lowest layer's product are most of the work, Q is exchanged between the two kinds of pass):
    both layers of a block, checked on sampled positions that the oracle computes one by one -- the first
    rows, rows around every boundary of a 256-row block in the middle, rows whose window edge or sink edge
    falls inside a tile, and the last rows."""
    Hq, Hkv = 8, 2
    q, kv = _inputs(34, T, Hq, Hkv, outliers=True)
    Q = [q(l) for l in range(2)]
    K = [kv(synth.TAG_K, l) for l in range(2)]
    V = [kv(synth.TAG_V, l) for l in range(2)]
    outs = [torch.zeros(T, Hq, 128, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    B.pod_prefill_attn(Q[0], K[0], V[0], outs[0], n_sink=S, n_recent=W)
    B.pod_prefill_attn(Q[1], K[1], V[1], outs[1], n_sink=S, n_recent=W, q_low=Q[0], k_low=K[0])
    torch.cuda.synchronize()
    assert B.pod_prefill_status() == B.POD_OK
    rows = sorted({0, 1, S, S + 1, W - 1, W, W + S - 1, W + S, W + S + 1, W + S + 127, W + S + 128, 2047, 2048, 2303, 2304,
                   T // 2 - 1, T // 2, T // 2 + 127, T // 2 + 128, T // 2 + 255, T // 2 + 256, T - 257, T - 256, T - 129,
                   T - 128, T - 2, T - 1} & set(range(T)))
    f = lambda xs: np.stack([x.double().cpu().numpy() for x in xs])
    Qn, Kn, Vn = f(Q), f(K), f(V)
    for l in range(2):
        ref = np.stack([O.pod_decode_layer(Qn[:, i], Kn[:, :i + 1], Vn[:, :i + 1], l, group_size=2, n_s=S, n_r=W)
                        for i in rows])
        _check(outs[l][rows], ref, f"T={T} layer {l} rows {rows[0]}..{rows[-1]}", V[l])


@pytest.mark.parametrize("T,S,W", [(5, 4, 32), (300, 4, 32), (1000, 16, 200)])
def test_prefill_head_dim_64(T, S, W):
    """Heads of 64 channels (one 128-byte sub-tile per operand row): a lowest layer and a sharing layer."""
    Hq, Hkv, d = 8, 2, 64
    q, kv = _inputs(35, T, Hq, Hkv, d=d, outliers=True)
    Q = [q(l) for l in range(2)]
    K = [kv(synth.TAG_K, l) for l in range(2)]
    V = [kv(synth.TAG_V, l) for l in range(2)]
    outs = [torch.zeros(T, Hq, d, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    B.pod_prefill_attn(Q[0], K[0], V[0], outs[0], n_sink=S, n_recent=W)
    B.pod_prefill_attn(Q[1], K[1], V[1], outs[1], n_sink=S, n_recent=W, q_low=Q[0], k_low=K[0])
    torch.cuda.synchronize()
    assert B.pod_prefill_status() == B.POD_OK
    f = lambda xs: np.stack([x.double().cpu().numpy() for x in xs])
    for l in range(2):
        ref = O.pod_prefill_layer(f(Q), f(K), f(V), l, group_size=2, n_s=S, n_r=W)
        _check(outs[l], ref, f"d=64 T={T} layer {l}", V[l])


def test_prefill_rejects_bad_arguments():
    x = torch.zeros(4, 2, 128, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(4, 2, 32, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.PodError):
        B.pod_prefill_attn(y, y, y, y, n_sink=1, n_recent=1)                    # head_dim 32
    with pytest.raises(B.PodError):
        B.pod_prefill_attn(x, x, x, x, n_sink=1, n_recent=0)
    with pytest.raises(B.PodError):
        B.pod_prefill_attn(x, x, x, x, n_sink=1, n_recent=1, q_low=x)           # q_low without k_low


def test_prefill_error_word_stops_launches_until_read():
    """The error path without any failing kernel: the error word is set from the host; launches then return
    without touching their output, pod_prefill_status reports the error once and clears it, and the next
    launch computes again."""
    T, Hq, Hkv = 300, 4, 2
    q, kv = _inputs(36, T, Hq, Hkv)
    Q, K, V = q(0), kv(synth.TAG_K, 0), kv(synth.TAG_V, 0)
    out = torch.zeros(T, Hq, 128, dtype=torch.bfloat16, device="cuda")
    B.pod_prefill_attn(Q, K, V, out, n_sink=4, n_recent=32)
    assert B.pod_prefill_status() == B.POD_OK
    good = out.clone()
    B.pod_prefill_inject_error()
    out.fill_(7.0)
    B.pod_prefill_attn(Q, K, V, out, n_sink=4, n_recent=32)
    torch.cuda.synchronize()
    assert (out == 7.0).all()                                   # nothing was computed
    assert B.pod_prefill_status() == B.POD_ERR_DEVICE
    assert B.pod_prefill_status() == B.POD_OK                   # read once, cleared
    B.pod_prefill_attn(Q, K, V, out, n_sink=4, n_recent=32)
    torch.cuda.synchronize()
    assert B.pod_prefill_status() == B.POD_OK and torch.equal(out, good)
