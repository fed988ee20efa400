"""GPU parity: the CUDA path through the C ABI against the fp64 oracle on the same seeded
inputs.  Layout is compared bit for bit; attention within max-abs 1e-2 and relative L2 5e-3."""
import numpy as np
import pytest
import torch

from oracle import pod_oracle as O
from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth
from podtest import Case, assert_close

pytestmark = pytest.mark.gpu

REGIONS = [("sinkK", B.POD_REGION_SINK_K), ("sinkV", B.POD_REGION_SINK_V),
           ("ringK", B.POD_REGION_RING_K), ("ringV", B.POD_REGION_RING_V),
           ("distK", B.POD_REGION_DIST_K), ("distV", B.POD_REGION_DIST_V)]


def _oracle_cache(case, b):
    return O.PodCacheOracle(case.L, case.Hkv, case.d, case.G, case.S, case.W, case.caps[b], lowest=case.lowest)


def _compare_layout(case, cache, oracles):
    for b, oc in enumerate(oracles):
        for name, rid in REGIONS:
            count = oc.n_blocks if name == "distK" else case.L
            for i in range(count):
                for h in range(case.Hkv):
                    ref, first = oc.valid_rows(name, i, h)
                    if ref.shape[0] == 0:              # nothing valid (or this head has fewer blocks)
                        continue
                    got = cache.read_region(rid, i, b, h, first, ref.shape[0])
                    np.testing.assert_array_equal(got, ref, err_msg=f"{name}[{i}] seq {b} head {h}")


# --------------------------------------------------------------------------- layout
@pytest.mark.parametrize("chunks", [[40], [1] * 40, [3, 17, 1, 1, 9, 9], [25, 15], [6, 30, 4]])
@pytest.mark.parametrize("d", [64, 128])
def test_cache_write_layout_bit_exact(chunks, d):
    """Prefill, chunked prefill (chunks larger than the window too), appends and ring wraps."""
    case = Case(seed=21, L=3, G=2, Hq=4, Hkv=2, d=d, S=3, W=7, lens=[sum(chunks)], caps=[sum(chunks) + 5])
    cache = case.make_cache()
    oc = _oracle_cache(case, 0)
    at = 0
    for t in chunks:
        for l in range(case.L):
            k = case.kv(synth.TAG_K, l, 0, at, at + t, "cuda")
            v = case.kv(synth.TAG_V, l, 0, at, at + t, "cuda")
            cache.write(l, 0, k, v, t)
            oc.write(l, synth.bf16_bits(k), synth.bf16_bits(v))
        at += t
        _compare_layout(case, cache, [oc])
        assert cache.seq_len(0, 0) == at
    live, dense = O.pod_cache_bytes([at], n_layers=3, n_kv_heads=2, head_dim=d, group_size=2, n_s=3, n_r=7)
    assert cache.bytes(B.POD_BYTES_LIVE) == live and cache.bytes(B.POD_BYTES_DENSE_EQUIV) == dense


def test_batched_append_layout_bit_exact():
    """seq = -1 appends one token to every sequence of a ragged batch, across ring wraps."""
    lens = [0, 5, 11, 30]
    case = Case(seed=22, L=2, G=2, Hq=8, Hkv=2, d=64, S=2, W=4, lens=lens, caps=[n + 12 for n in lens])
    cache = case.make_cache()
    ocs = [_oracle_cache(case, b) for b in range(case.B)]
    case.prefill(cache, chunk=7)
    for b, oc in enumerate(ocs):
        for l in range(case.L):
            if lens[b]:
                oc.write(l, synth.bf16_bits(case.kv(synth.TAG_K, l, b, 0, lens[b], "cpu")),
                         synth.bf16_bits(case.kv(synth.TAG_V, l, b, 0, lens[b], "cpu")))
    _compare_layout(case, cache, ocs)
    for step in range(12):
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] + step, lens[b] + step + 1, "cuda")[0]
                             for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] + step, lens[b] + step + 1, "cuda")[0]
                             for b in range(case.B)])
            cache.write(l, -1, k, v, 1)
            kb, vb = synth.bf16_bits(k), synth.bf16_bits(v)
            for b, oc in enumerate(ocs):
                oc.append(l, kb[b], vb[b])
        _compare_layout(case, cache, ocs)
    with pytest.raises(B.PodError) as e:
        cache.write(0, -1, k, v, 1)
    assert e.value.status == B.POD_ERR_CAPACITY


# --------------------------------------------------------------------------- attention, small
def _check_all_heads(case, outs, step=0, lens=None):
    lens = case.lens if lens is None else lens
    worst = (0.0, 0.0)
    for l in range(case.L):
        for b in range(case.B):
            ref = np.stack([case.oracle_head(l, b, h, n=lens[b], step=step) for h in range(case.Hq)])
            ma, rl = assert_close(outs[l, b], ref, f"layer {l} seq {b}")
            worst = (max(worst[0], ma), max(worst[1], rl))
    return worst


def test_config1_tiny_all_heads():
    """Batch 1, 4 layers, G = 2, 8/2 heads, d = 64, 512 tokens, S = 16, W = 64, seed 0."""
    case = Case(seed=0, L=4, G=2, Hq=8, Hkv=2, d=64, S=16, W=64, lens=[512])
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    _check_all_heads(case, outs)
    assert cache.bytes(B.POD_BYTES_LIVE) == 827392
    # the same answer from the layout oracle fed with the same bits
    oc = _oracle_cache(case, 0)
    for l in range(4):
        oc.write(l, synth.bf16_bits(case.kv(synth.TAG_K, l, 0, 0, 512, "cpu")),
                 synth.bf16_bits(case.kv(synth.TAG_V, l, 0, 0, 512, "cpu")))
    for l in range(4):
        q = case.q(l, 0, "cpu")[0].double().numpy()
        ql = case.q(l - l % 2, 0, "cpu")[0].double().numpy()
        assert_close(outs[l, 0], oc.attend(l, q, ql), f"layout oracle layer {l}")


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 2), (64, 8, 2), (128, 4, 4), (128, 4, 2), (64, 16, 2),
                                      (128, 16, 2), (128, 6, 2)])
def test_shapes_and_ragged_batch(d, Hq, Hkv):
    """Several GQA ratios and head sizes on a ragged batch whose lengths cover: empty, inside the
    sink, partial ring, exactly S + W, first distant token, several tiles with a ragged tail."""
    S, W = 4, 24
    lens = [0, 1, 3, 4, 5, 20, 28, 29, 37, 100, 333, 1000]
    case = Case(seed=3, L=3, G=2, Hq=Hq, Hkv=Hkv, d=d, S=S, W=W, lens=lens, caps=[max(n, 1) for n in lens])
    cache = case.make_cache()
    case.prefill(cache, chunk=97)
    outs = case.decode_all(cache)
    _check_all_heads(case, outs)
    assert (outs[:, 0] == 0).all()          # empty sequence: zeros


@pytest.mark.parametrize("G", [1, 3, 4])
def test_group_sizes(G):
    case = Case(seed=4, L=5, G=G, Hq=8, Hkv=2, d=128, S=8, W=32, lens=[700, 64])
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    _check_all_heads(case, outs)


def test_decode_steps_with_window_rollover():
    """Appends and decodes interleaved per layer, as a model runs them, over ring wraps."""
    lens0 = [30, 75, 9]
    case = Case(seed=5, L=4, G=2, Hq=8, Hkv=2, d=128, S=4, W=16, lens=lens0, caps=[n + 40 for n in lens0])
    cache = case.make_cache()
    case.prefill(cache)
    stream = torch.cuda.current_stream().cuda_stream
    for step in range(1, 36):
        lens = [n + step for n in lens0]
        outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            cache.write(l, -1, k, v, 1, stream)
            cache.decode_attn(l, case.q(l, step, "cuda"), outs[l], stream)
        torch.cuda.synchronize()
        if step in (1, 2, 7, 16, 17, 35):
            _check_all_heads(case, outs, step=step, lens=lens)
    assert cache.device_status() == B.POD_OK


@pytest.mark.parametrize("d,G,lens0", [(128, 2, [30, 75, 9, 0, 3]), (64, 3, [19, 20, 21, 150]),
                                       (128, 2, [5 * i for i in range(10)])])
def test_fused_append_decode_steps(d, G, lens0):
    """pod_append_decode_attn over many steps (first tokens, sink fill, ring fill, ring wraps, small
    and large batches): outputs against the oracle, cache contents bit for bit against the
    oracle's layout, which is maintained by plain appends."""
    S, W = 4, 16
    case = Case(seed=15, L=4, G=G, Hq=8, Hkv=2, d=d, S=S, W=W, lens=lens0, caps=[n + 40 for n in lens0])
    cache = case.make_cache()
    case.prefill(cache)
    ocs = [_oracle_cache(case, b) for b in range(case.B)]
    for b, oc in enumerate(ocs):
        for l in range(case.L):
            if lens0[b]:
                oc.write(l, synth.bf16_bits(case.kv(synth.TAG_K, l, b, 0, lens0[b], "cpu")),
                         synth.bf16_bits(case.kv(synth.TAG_V, l, b, 0, lens0[b], "cpu")))
    stream = torch.cuda.current_stream().cuda_stream
    for step in range(1, 40):
        lens = [n + step for n in lens0]
        outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            cache.append_decode_attn(l, k, v, case.q(l, step, "cuda"), outs[l], stream)
            kb, vb = synth.bf16_bits(k), synth.bf16_bits(v)
            for b, oc in enumerate(ocs):
                oc.append(l, kb[b], vb[b])
        torch.cuda.synchronize()
        assert [cache.seq_len(b, 0) for b in range(case.B)] == lens
        if step in (1, 2, 3, 4, 5, 16, 17, 20, 21, 22, 37, 39):
            _check_all_heads(case, outs, step=step, lens=lens)
            _compare_layout(case, cache, ocs)
    assert cache.device_status() == B.POD_OK
    # the two-call form continues from the state the fused form left (device lengths included)
    step = 40
    lens = [n + step for n in lens0]
    outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
    for l in range(case.L):
        k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
        v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
        cache.write(l, -1, k, v, 1, stream)
        cache.decode_attn(l, case.q(l, step, "cuda"), outs[l], stream)
    torch.cuda.synchronize()
    _check_all_heads(case, outs, step=step, lens=lens)
    with pytest.raises(B.PodError) as e:
        cache.append_decode_attn(0, k, v, case.q(0, 0, "cuda"), outs[0], stream)
    assert e.value.status == B.POD_ERR_CAPACITY


def test_shared_logits_fallback_and_mixed_calls():
    """Layers other than a block's lowest reuse the lowest layer's distant logits when the stored
    ones are theirs, and score the block's keys themselves when another block has been decoded in
    between; one-launch and two-call forms may be mixed inside a block.  All against the oracle."""
    lens0 = [90, 41]
    case = Case(seed=16, L=4, G=2, Hq=8, Hkv=2, d=128, S=4, W=16, lens=lens0, caps=[n + 8 for n in lens0])
    cache = case.make_cache()
    case.prefill(cache)
    stream = torch.cuda.current_stream().cuda_stream
    outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
    for l in (0, 2, 1, 3, 1):                 # layer 1 after block 1's lowest layer: fallback; layer 3, then 1 again
        cache.decode_attn(l, case.q(l, 0, "cuda"), outs[l], stream)
    torch.cuda.synchronize()
    _check_all_heads(case, outs, step=0)
    for step, fused_layers in ((1, (0, 2)), (2, (1, 3)), (3, (0, 1, 2, 3)), (4, ())):
        lens = [n + step for n in lens0]
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            if l in fused_layers:
                cache.append_decode_attn(l, k, v, case.q(l, step, "cuda"), outs[l], stream)
            else:
                cache.write(l, -1, k, v, 1, stream)
                cache.decode_attn(l, case.q(l, step, "cuda"), outs[l], stream)
        torch.cuda.synchronize()
        _check_all_heads(case, outs, step=step, lens=lens)
    assert cache.device_status() == B.POD_OK


HEAD_WISE = [[0, 0, 0, 0], [0, 1, 0, 1], [0, 1, 2, 1], [3, 1, 2, 1], [3, 4, 2, 1], [3, 4, 2, 5]]


@pytest.mark.parametrize("d", [128, 64])
def test_head_wise_blocks_layout_and_attention(d):
    """Blocks chosen per KV head (Algorithm 1's output shape): a layer is the lowest of its block for
    some heads and not for others.  Prefill, two-call steps, one-launch steps across ring wraps; cache
    contents bit for bit against the oracle's layout, outputs against the definition."""
    lens0 = [70, 23, 0]
    case = Case(seed=17, L=6, G=1, Hq=8, Hkv=4, d=d, S=4, W=16, lens=lens0, caps=[n + 30 for n in lens0],
                lowest=HEAD_WISE)
    cache = case.make_cache()
    case.prefill(cache, chunk=33)
    ocs = [_oracle_cache(case, b) for b in range(case.B)]
    for b, oc in enumerate(ocs):
        for l in range(case.L):
            if lens0[b]:
                oc.write(l, synth.bf16_bits(case.kv(synth.TAG_K, l, b, 0, lens0[b], "cpu")),
                         synth.bf16_bits(case.kv(synth.TAG_V, l, b, 0, lens0[b], "cpu")))
    _compare_layout(case, cache, ocs)
    _check_all_heads(case, case.decode_all(cache))
    live, dense = O.pod_cache_bytes(lens0, n_layers=6, n_kv_heads=4, head_dim=d, lowest=HEAD_WISE, n_s=4, n_r=16)
    assert cache.bytes(B.POD_BYTES_LIVE) == live and cache.bytes(B.POD_BYTES_DENSE_EQUIV) == dense
    stream = torch.cuda.current_stream().cuda_stream
    outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
    for step in range(1, 26):
        lens = [n + step for n in lens0]
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            if step % 3:
                cache.append_decode_attn(l, k, v, case.q(l, step, "cuda"), outs[l], stream)
            else:
                cache.write(l, -1, k, v, 1, stream)
                cache.decode_attn(l, case.q(l, step, "cuda"), outs[l], stream)
            kb, vb = synth.bf16_bits(k), synth.bf16_bits(v)
            for b, oc in enumerate(ocs):
                oc.append(l, kb[b], vb[b])
        torch.cuda.synchronize()
        if step in (1, 2, 3, 16, 17, 18, 21, 24, 25):
            _check_all_heads(case, outs, step=step, lens=lens)
            _compare_layout(case, cache, ocs)
    assert cache.device_status() == B.POD_OK


def test_head_wise_blocks_from_greedy_grouping_many_tiles():
    """A map produced by the library's greedy grouping from a seeded similarity tensor, on a context
    of several thousand tokens (many tiles and splits per head)."""
    rng = np.random.default_rng(5)
    L, Hkv = 8, 2
    sim = rng.random((Hkv, L, L)) * 0.7 + 0.25
    sim = np.maximum(sim, sim.transpose(0, 2, 1))
    lowest = B.pod_greedy_layer_blocks(sim.tolist(), 0.5)
    assert lowest == O.lowest_map_from_blocks(O.greedy_layer_blocks(sim.astype(np.float32).astype(np.float64), 0.5), L).tolist()
    assert any(lowest[l][0] != lowest[l][1] for l in range(L))         # the heads really differ
    case = Case(seed=18, L=L, G=1, Hq=8, Hkv=Hkv, d=128, S=16, W=256, lens=[5000, 3333], lowest=lowest)
    cache = case.make_cache()
    case.prefill(cache)
    outs = case.decode_all(cache)
    for l in range(L):
        for b in range(2):
            for h in (0, 3, 4, 7):
                assert_close(outs[l, b, h], case.oracle_head(l, b, h), f"layer {l} seq {b} head {h}")


def _gate_case(seed, n, lowest=None, G=2):
    """Inputs for the gate tests: the queries of some heads of the non-lowest layers are scaled up, so
    that their proximal logits dominate (g close to 1), others are left alone (g small)."""
    case = Case(seed=seed, L=4, G=G, Hq=8, Hkv=2, d=128, S=4, W=64, lens=[n], caps=[n + 8], lowest=lowest)
    dev = "cuda"
    K = [case.kv(synth.TAG_K, l, 0, 0, n + 2, dev) for l in range(case.L)]
    V = [case.kv(synth.TAG_V, l, 0, 0, n + 2, dev) for l in range(case.L)]
    gain = torch.tensor([[1, 1, 1, 1, 1, 1, 1, 1], [4, 1, 3, 1, 4, 4, 3, 5], [1, 1, 1, 1, 1, 1, 1, 1],
                         [1, 5, 1, 2.5, 1, 1, 1, 1]], dtype=torch.float32, device=dev)
    qs = [[(case.q(l, step, dev).float() * gain[l][None, :, None]).to(torch.bfloat16) for l in range(case.L)]
          for step in range(2)]
    return case, K, V, qs


def _gate_check(case, K, V, q_step, outs, n, tau, expect_some=True):
    """Every head against the oracle's gated result; a head whose g lies within 0.01 of tau may match
    either candidate (the device takes the decision in fp32 from its own sums)."""
    Kh = torch.stack([k[:n] for k in K]).double().cpu().numpy()
    Vh = torch.stack([v[:n] for v in V]).double().cpu().numpy()
    qh = torch.stack([q[0] for q in q_step]).double().cpu().numpy()
    kinds = set()
    for l in range(case.L):
        info = []
        kw = dict(lowest=np.array(case.lowest), n_s=case.S, n_r=case.W)
        ref = O.pod_decode_layer(qh, Kh, Vh, l, tau=tau, info=info, **kw)
        for h in range(case.Hq):
            g, skipped = info[h]
            if g is not None and abs(g - tau) < 0.01:
                alt = O.pod_decode_layer(qh, Kh, Vh, l, tau=(0.0 if not skipped else 2.0), **kw)[h]
                got = outs[l, 0, h].double().cpu().numpy()
                assert min(np.abs(got - ref[h]).max(), np.abs(got - alt).max()) <= 1e-2
                continue
            assert_close(outs[l, 0, h], ref[h], f"tau {tau} layer {l} head {h} g {g} skipped {skipped}")
            kinds.add(("skip" if skipped else "full") if g is not None else "lowest")
    if expect_some:
        assert kinds == {"skip", "full", "lowest"}, kinds


@pytest.mark.parametrize("head_wise", [False, True])
def test_gate_threshold_skips_distant_tokens(head_wise):
    """pod_cache_set_gate_threshold: heads of non-lowest layers whose gate g reaches tau give the softmax
    over their proximal tokens alone, the others (and all heads of lowest layers) the full result; both
    kinds occur inside one KV head.  Two-call form, then one-launch steps; tau = 0 and tau off."""
    n = 1500
    lowest = [[0, 0], [0, 1], [2, 1], [2, 1]] if head_wise else None
    case, K, V, qs = _gate_case(19, n, lowest=lowest)
    cache = case.make_cache()
    stream = torch.cuda.current_stream().cuda_stream
    for l in range(case.L):
        cache.write(l, 0, K[l][:n], V[l][:n], n, stream)
    outs = torch.empty(case.L, 1, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")

    def decode(q_step):
        for l in range(case.L):
            cache.decode_attn(l, q_step[l], outs[l], stream)
        torch.cuda.synchronize()

    for tau in (0.5, 0.0, 2.0):
        cache.set_gate_threshold(tau)
        decode(qs[0])
        _gate_check(case, K, V, qs[0], outs, n, tau, expect_some=(tau == 0.5))
    assert cache.last_launch()["n_kernels"] == 1                     # gate off: one launch
    cache.set_gate_threshold(0.5)
    for step in (1, 2):                                              # one-launch form with the gate on
        for l in range(case.L):
            cache.append_decode_attn(l, K[l][n + step - 1:n + step], V[l][n + step - 1:n + step], qs[step - 1][l],
                                     outs[l], stream)
        torch.cuda.synchronize()
        _gate_check(case, K, V, qs[step - 1], outs, n + step, 0.5)
    assert cache.last_launch()["n_kernels"] == 2                     # proximal launch + distant launch
    assert cache.device_status() == B.POD_OK
    with pytest.raises(B.PodError):
        cache.set_gate_threshold(-0.1)


def test_custom_scale():
    case = Case(seed=6, L=2, G=2, Hq=4, Hkv=1, d=64, S=2, W=6, lens=[50], scale=0.31)
    cache = case.make_cache()
    case.prefill(cache)
    _check_all_heads(case, case.decode_all(cache))


# --------------------------------------------------------------------------- planted keys
@pytest.mark.parametrize("layer", [0, 1])
def test_planted_key_at_every_boundary(layer):
    """A key aligned with the query that scores it dominates the softmax: the output must be
    that token's value row of the decoded layer.  Planted at the region boundaries and at the edges of the
    kernel's tiles (16 rows; 32 distant rows for a layer that reads stored logits) and chunks (runs of a few
    tiles) in the order the kernel walks a head: sink rows, ring slots, then distant rows."""
    L, G, Hq, Hkv, d, S, W, n = 2, 2, 4, 1, 128, 16, 64, 3000
    seed = 9
    cfg = B.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, group_size=G, n_sink=S,
                        n_recent=W, batch=1, device=0)
    K = [synth.gen_kv(seed, synth.TAG_K, l, 0, 0, n, Hkv, d, device="cuda") for l in range(L)]
    V = [synth.gen_kv(seed, synth.TAG_V, l, 0, 0, n, Hkv, d, device="cuda") for l in range(L)]
    q = [synth.gen_q(seed, l, 0, 1, Hq, d, device="cuda") for l in range(L)]
    # make all four query heads of the group identical so one planted key serves them all
    for l in range(L):
        q[l][:, :] = q[l][:, :1]
    in_slot = lambda slot: next(p for p in range(n - W, n) if (p - S) % W == slot)
    positions = [0, S - 1, S, S + 1, n - W - 1, n - W, n - 1, S + W - 1, S + W]
    positions += [in_slot(x) for x in (0, 15, 16, 31, 32, 47, 48, 63)]     # tile edges among the ring slots
    n_d = n - S - W
    last16, last32 = (n_d - 1) // 16 * 16, (n_d - 1) // 32 * 32
    dist_edges = [0, 15, 16, 31, 32, 33, 47, 48, 63, 64, 95, 96, 511, 512, 527, 528, 1023, 1024, 1471, 1472, 1500,
                  last16 - 1, last16, last32 - 1, last32, n_d - 1]
    positions += [S + t for t in dist_edges]                                 # tile and chunk edges among the distant rows
    cache = B.PodCache(cfg, [n])
    for l in range(L):
        cache.write(l, 0, K[l], V[l], n)
    out = torch.empty(1, Hq, d, dtype=torch.bfloat16, device="cuda")
    tmp = torch.empty(1, Hq, d, dtype=torch.bfloat16, device="cuda")
    for pos in sorted(set(p for p in positions if 0 <= p < n)):
        distant = S <= pos < n - W
        src = 0 if (distant and layer == 1) else layer
        Kp = [k.clone() for k in K]
        qv = q[src][0, 0].float()
        Kp[src][pos, 0] = (60.0 * qv / qv.norm()).to(torch.bfloat16)
        cache.reset()
        for l in range(L):
            cache.write(l, 0, Kp[l], V[l], n)
        cache.decode_attn(0, q[0], tmp)
        cache.decode_attn(1, q[1], out)
        got = tmp if layer == 0 else out
        torch.cuda.synchronize()
        want = V[layer][pos, 0].float()
        for h in range(Hq):
            err = (got[0, h].float() - want).abs().max().item()
            assert err <= 1e-2, f"pos {pos} head {h}: {err}"


def test_shared_scores_follow_lowest_layer_query():
    """At a non-lowest layer, changing the layer's own query leaves an output dominated by a
    distant planted key untouched; the distant scores are the lowest layer's."""
    case = Case(seed=10, L=2, G=2, Hq=4, Hkv=1, d=64, S=4, W=8, lens=[400])
    cache = case.make_cache()
    K = [case.kv(synth.TAG_K, l, 0, 0, 400, "cuda") for l in range(2)]
    V = [case.kv(synth.TAG_V, l, 0, 0, 400, "cuda") for l in range(2)]
    q0, q1 = case.q(0, 0, "cuda"), case.q(1, 0, "cuda")
    q0[:, :] = q0[:, :1]
    K[0][200, 0] = (80.0 * q0[0, 0].float() / q0[0, 0].float().norm()).to(torch.bfloat16)
    for l in range(2):
        cache.write(l, 0, K[l], V[l], 400)
    o0 = torch.empty_like(q0)
    o1 = torch.empty_like(q0)
    o1b = torch.empty_like(q0)
    cache.decode_attn(0, q0, o0)
    cache.decode_attn(1, q1, o1)
    cache.decode_attn(1, -q1, o1b)
    torch.cuda.synchronize()
    want = V[1][200, 0].float()
    assert (o1[0].float() - want).abs().max() <= 1e-2
    assert (o1b[0].float() - want).abs().max() <= 1e-2


# --------------------------------------------------------------------------- error paths on a device cache
def test_error_paths_on_device_cache():
    case = Case(seed=1, L=2, G=2, Hq=4, Hkv=1, d=64, S=2, W=4, lens=[10])
    cache = case.make_cache()
    k = case.kv(synth.TAG_K, 0, 0, 0, 10, "cuda")
    q = case.q(0, 0, "cuda")
    out = torch.empty_like(q)
    cache.write(0, 0, k, k, 10)
    with pytest.raises(B.PodError) as e:
        cache.write(0, 0, k, k, 1)
    assert e.value.status == B.POD_ERR_CAPACITY
    with pytest.raises(B.PodError) as e:
        cache.decode_attn(1, q, out)
    assert e.value.status == B.POD_ERR_ORDER
    arena = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.PodError) as e:
        B.PodCache(case.cfg, case.caps, arena=arena)
    assert e.value.status == B.POD_ERR_ARENA
    need = B.pod_cache_required_bytes(case.cfg, case.caps)
    arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    c2 = B.PodCache(case.cfg, case.caps, arena=arena)      # caller-owned arena works
    c2.write(0, 0, k, k, 10)
    c2.decode_attn(0, q, out)
    torch.cuda.synchronize()
    assert c2.device_status() == B.POD_OK
    assert_close(out[0], np.stack([_dense_head(case, k, q, h) for h in range(4)]), "arena cache")


def _dense_head(case, k, q, h):
    kk = k[:, 0].double().cpu().numpy()
    qq = q[0, h].double().cpu().numpy()
    o, _ = O.pod_attention_joint(qq, qq, kk, kk, kk, case.S, case.W)
    return o


def test_cache_error_word_is_reported_once_and_decoding_goes_on():
    """The decode path's error word without any failing kernel: it is set from the host
    (pod_cache_inject_error), pod_cache_device_status reports POD_ERR_DEVICE once and clears it, and the
    next decode of the same cache is correct."""
    case = Case(seed=41, L=2, G=2, Hq=8, Hkv=2, d=64, S=4, W=32, lens=[700])
    cache = case.make_cache()
    case.prefill(cache)
    assert cache.device_status() == B.POD_OK
    cache.inject_error()
    assert cache.device_status() == B.POD_ERR_DEVICE
    assert cache.device_status() == B.POD_OK
    outs = case.decode_all(cache)                               # asserts POD_OK after the launches
    for l in range(2):
        for h in range(8):
            assert_close(outs[l, 0, h], case.oracle_head(l, 0, h), f"layer {l} head {h} after the injected error")


@pytest.mark.parametrize("d,G,Hq,Hkv", [(128, 2, 8, 2), (64, 3, 8, 1)])
def test_stale_query_path_recomputes_heads_exactly(d, G, Hq, Hkv):
    """Launches that follow a decode launch of another layer stream with an early copy of q and check it
    after waiting for the stream's previous kernel; a head whose copy was stale is recomputed by one CTA.
    The test forces that path from the host (pod_cache_inject_stale_query) for lowest layers (which also
    store the distant logits that the block's next layers then consume) and for sharing layers, over
    steps that fill the sink, fill the ring and wrap it: outputs against the oracle, cache contents bit
    for bit against the oracle's layout."""
    S, W = 4, 16
    lens0 = [70, 3, 21]
    case = Case(seed=23, L=6, G=G, Hq=Hq, Hkv=Hkv, d=d, S=S, W=W, lens=lens0, caps=[n + 24 for n in lens0])
    cache = case.make_cache()
    case.prefill(cache)
    ocs = [_oracle_cache(case, b) for b in range(case.B)]
    for b, oc in enumerate(ocs):
        for l in range(case.L):
            oc.write(l, synth.bf16_bits(case.kv(synth.TAG_K, l, b, 0, lens0[b], "cpu")),
                     synth.bf16_bits(case.kv(synth.TAG_V, l, b, 0, lens0[b], "cpu")))
    stream = torch.cuda.current_stream().cuda_stream
    for step in range(1, 24):
        lens = [n + step for n in lens0]
        outs = torch.empty(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
        for l in range(case.L):
            k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda")[0] for b in range(case.B)])
            if (step + l) % 3 == 0:                     # lowest and sharing layers alike, a different set every step
                cache.inject_stale_query()
            cache.append_decode_attn(l, k, v, case.q(l, step, "cuda"), outs[l], stream)
            kb, vb = synth.bf16_bits(k), synth.bf16_bits(v)
            for b, oc in enumerate(ocs):
                oc.append(l, kb[b], vb[b])
        torch.cuda.synchronize()
        _check_all_heads(case, outs, step=step, lens=lens)
        if step in (1, 2, 13, 14, 23):
            _compare_layout(case, cache, ocs)
    assert cache.device_status() == B.POD_OK


def test_kv_head_shards_reproduce_the_unsplit_attention():
    """The KV-head split for several GPUs, run here on one: the cache of each "rank" is built from
    pod_shard_config / pod_shard_block_map with the rank's slices of k, v and q (contiguous, as column-parallel
    projections produce them); the ranks' outputs, put side by side at their first query head, are the
    unsplit attention -- checked head by head against the oracle -- and the ranks' bytes add up."""
    lens0 = [300, 77]
    case = Case(seed=29, L=6, G=2, Hq=16, Hkv=4, d=64, S=4, W=16, lens=lens0, caps=[n + 4 for n in lens0], lowest=HEAD_WISE)
    world, r = 2, 4
    stream = torch.cuda.current_stream().cuda_stream
    outs = torch.zeros(case.L, case.B, case.Hq, case.d, dtype=torch.bfloat16, device="cuda")
    live = 0
    for rank in range(world):
        local, kv0, q0 = B.pod_shard_config(case.cfg, rank, world)
        heads = list(range(kv0, kv0 + local.n_kv_heads))
        cache = B.PodCache(local, case.caps, lowest_layer=B.pod_shard_block_map(case.cfg, case.lowest, rank, world))
        for l in range(case.L):
            for b in range(case.B):
                k = case.kv(synth.TAG_K, l, b, 0, lens0[b], "cuda", heads=heads)
                v = case.kv(synth.TAG_V, l, b, 0, lens0[b], "cuda", heads=heads)
                cache.write(l, b, k, v, lens0[b], stream)
        for step in (1, 2):                                   # the one-launch form, two steps
            lens = [n + step for n in lens0]
            for l in range(case.L):
                k = torch.stack([case.kv(synth.TAG_K, l, b, lens[b] - 1, lens[b], "cuda", heads=heads)[0] for b in range(case.B)])
                v = torch.stack([case.kv(synth.TAG_V, l, b, lens[b] - 1, lens[b], "cuda", heads=heads)[0] for b in range(case.B)])
                q = case.q(l, step, "cuda")[:, q0:q0 + local.n_q_heads].contiguous()
                o = torch.empty_like(q)
                cache.append_decode_attn(l, k, v, q, o, stream)
                outs[l, :, q0:q0 + local.n_q_heads] = o
        torch.cuda.synchronize()
        assert cache.device_status() == B.POD_OK
        live += cache.bytes(B.POD_BYTES_LIVE)
        cache.destroy()
    _check_all_heads(case, outs, step=2, lens=[n + 2 for n in lens0])
    whole, _ = O.pod_cache_bytes([n + 2 for n in lens0], n_layers=case.L, n_kv_heads=case.Hkv, head_dim=case.d,
                                 group_size=case.G, n_s=case.S, n_r=case.W, lowest=case.lowest)
    assert live == whole
