"""Host-side checks of the C-ABI library that need no GPU: exported symbols, argument
validation, call-order rules and byte accounting on a host-only cache (device = -1)."""
import ctypes
import os
import re

import pytest

from oracle import pod_oracle as O
from paper_2412_02252_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "pod.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pod_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert "pod_cache_create" in names and "pod_decode_attn" in names
    assert "pod_cache_write" in names and "pod_cache_bytes" in names
    raw = ctypes.CDLL(B._build.LIB)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in pod.h but not exported"
    assert sorted(B.EXPORTS) == names


def _cfg(**kw):
    base = dict(n_layers=4, n_q_heads=8, n_kv_heads=2, head_dim=64, group_size=2, n_sink=16,
                n_recent=64, batch=1, device=-1)
    base.update(kw)
    return B.make_config(**base)


def test_strerror_covers_all_codes():
    seen = {B.pod_strerror(s) for s in range(-6, 2)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert B.pod_strerror(-99) == "unknown status"


@pytest.mark.parametrize("bad", [dict(head_dim=96), dict(n_q_heads=7), dict(n_q_heads=32, n_kv_heads=2),
                                 dict(group_size=0), dict(n_recent=0), dict(n_sink=-1), dict(batch=0),
                                 dict(n_layers=0), dict(sm_scale=-1.0)])
def test_invalid_configs_are_rejected(bad):
    cfg = _cfg(**bad)
    caps = [512] * max(1, cfg.batch)
    if cfg.batch >= 1:
        assert B.pod_cache_required_bytes(cfg, caps) == 0
        with pytest.raises(B.PodError) as e:
            B.PodCache(cfg, caps)
        assert e.value.status == B.POD_ERR_INVALID
    else:
        h = ctypes.c_void_p()
        st = B.lib.pod_cache_create(ctypes.byref(cfg), (ctypes.c_int32 * 1)(512), None, 0, ctypes.byref(h))
        assert st == B.POD_ERR_INVALID


def test_required_bytes_covers_regions_at_capacity():
    cfg = _cfg()
    need = B.pod_cache_required_bytes(cfg, [512])
    live, _ = O.pod_cache_bytes([512], n_layers=4, n_kv_heads=2, head_dim=64, group_size=2, n_s=16, n_r=64)
    assert need >= live and need % 256 == 0
    assert B.pod_cache_required_bytes(cfg, [1024]) > need
    # capacity below the proximal window still reserves the whole sink + ring
    assert B.pod_cache_required_bytes(cfg, [8]) >= 4 * 2 * 2 * 80 * 128


def _fake_ptr():
    return 0x1000          # never dereferenced by a host-only cache


def test_bytes_match_closed_form_and_oracle():
    for lens, kw in [([512], dict()),
                     ([100, 80, 512], dict(batch=3)),
                     ([300], dict(n_layers=5, group_size=2)),          # short last block
                     ([300], dict(group_size=1)),
                     ([40], dict())]:
        cfg = _cfg(**kw)
        c = B.PodCache(cfg, [max(lens)] * cfg.batch)
        for l in range(cfg.n_layers):
            for b, n in enumerate(lens):
                assert c.write(l, b, _fake_ptr(), _fake_ptr(), n) == B.POD_DRY_RUN
        live, dense = O.pod_cache_bytes(lens, n_layers=cfg.n_layers, n_kv_heads=2, head_dim=64,
                                        group_size=cfg.group_size, n_s=16, n_r=64)
        assert c.bytes(B.POD_BYTES_LIVE) == live
        assert c.bytes(B.POD_BYTES_DENSE_EQUIV) == dense
        assert c.bytes(B.POD_BYTES_ALLOCATED) == B.pod_cache_required_bytes(cfg, [max(lens)] * cfg.batch)
        assert c.bytes(7) == -1
        for b, n in enumerate(lens):
            assert c.seq_len(b, 0) == n
    cfg = _cfg()
    c = B.PodCache(cfg, [512])
    for l in range(4):
        c.write(l, 0, _fake_ptr(), _fake_ptr(), 512)
    assert c.bytes(B.POD_BYTES_LIVE) == 827392 and c.bytes(B.POD_BYTES_DENSE_EQUIV) == 1048576


def test_write_validation_and_capacity():
    cfg = _cfg(batch=2)
    c = B.PodCache(cfg, [10, 20])
    p = _fake_ptr()
    for args in [(4, 0, p, p, 1), (-1, 0, p, p, 1), (0, 2, p, p, 1), (0, -2, p, p, 1), (0, 0, p, p, 0),
                 (0, -1, p, p, 2), (0, 0, 0, p, 1), (0, 0, p, 0, 1), (0, 0, p + 8, p, 1)]:
        with pytest.raises(B.PodError) as e:
            c.write(*args)
        assert e.value.status == B.POD_ERR_INVALID
    c.write(0, 0, p, p, 10)
    with pytest.raises(B.PodError) as e:
        c.write(0, 0, p, p, 1)
    assert e.value.status == B.POD_ERR_CAPACITY
    with pytest.raises(B.PodError) as e:      # batched append fails if any sequence is full; nothing advances
        c.write(0, -1, p, p, 1)
    assert e.value.status == B.POD_ERR_CAPACITY
    assert c.seq_len(0, 0) == 10 and c.seq_len(1, 0) == 0
    c.reset(0)
    assert c.seq_len(0, 0) == 0
    assert c.write(0, -1, p, p, 1) == B.POD_DRY_RUN
    assert c.seq_len(0, 0) == 1 and c.seq_len(1, 0) == 1


def test_decode_order_rules():
    cfg = _cfg()
    c = B.PodCache(cfg, [512])
    p = _fake_ptr()
    for l in range(4):
        c.write(l, 0, p, p, 100)
    # a non-lowest layer before its block's lowest layer: no stashed query
    with pytest.raises(B.PodError) as e:
        c.decode_attn(1, p, p)
    assert e.value.status == B.POD_ERR_ORDER
    assert c.decode_attn(0, p, p) == B.POD_DRY_RUN
    assert c.decode_attn(1, p, p) == B.POD_DRY_RUN
    with pytest.raises(B.PodError) as e:      # block 1 has its own stash
        c.decode_attn(3, p, p)
    assert e.value.status == B.POD_ERR_ORDER
    # next step, interleaved write/decode per layer as a model would do it
    c.write(0, 0, p, p, 1)
    assert c.decode_attn(0, p, p) == B.POD_DRY_RUN
    with pytest.raises(B.PodError) as e:      # layer 1 not yet appended: block lengths differ
        c.decode_attn(1, p, p)
    assert e.value.status == B.POD_ERR_ORDER
    c.write(1, 0, p, p, 1)
    assert c.decode_attn(1, p, p) == B.POD_DRY_RUN
    # stale stash: lowest layer decoded at an older length
    c.write(0, 0, p, p, 1)
    c.write(1, 0, p, p, 1)
    with pytest.raises(B.PodError) as e:
        c.decode_attn(1, p, p)
    assert e.value.status == B.POD_ERR_ORDER
    for args in [(4, p, p), (-1, p, p), (0, 0, p), (0, p, 0), (0, p + 2, p)]:
        with pytest.raises(B.PodError) as e:
            c.decode_attn(*args)
        assert e.value.status == B.POD_ERR_INVALID


def test_fused_append_decode_order_and_capacity_rules():
    """The one-launch form obeys the rules of write + decode, judged at the lengths after the append."""
    cfg = _cfg(batch=2)
    c = B.PodCache(cfg, [12, 40])
    p = _fake_ptr()
    for l in range(4):
        for b in range(2):
            c.write(l, b, p, p, 10)
    with pytest.raises(B.PodError) as e:      # block's lowest layer has not run this step
        c.append_decode_attn(1, p, p, p, p)
    assert e.value.status == B.POD_ERR_ORDER
    assert c.seq_len(0, 1) == 10              # a refused call changes nothing
    assert c.append_decode_attn(0, p, p, p, p) == B.POD_DRY_RUN
    assert c.seq_len(0, 0) == 11 and c.seq_len(1, 0) == 11
    assert c.append_decode_attn(1, p, p, p, p) == B.POD_DRY_RUN
    assert c.decode_attn(1, p, p) == B.POD_DRY_RUN          # same lengths, same stash: allowed again
    assert c.append_decode_attn(0, p, p, p, p) == B.POD_DRY_RUN
    with pytest.raises(B.PodError) as e:      # sequence 0 is full at 12
        c.append_decode_attn(0, p, p, p, p)
    assert e.value.status == B.POD_ERR_CAPACITY
    assert c.seq_len(0, 0) == 12 and c.seq_len(1, 0) == 12
    for args in [(0, 0, p, p, p), (0, p, 0, p, p), (0, p, p, 0, p), (0, p, p, p, 0), (9, p, p, p, p),
                 (0, p + 2, p, p, p)]:
        with pytest.raises(B.PodError) as e:
            c.append_decode_attn(*args)
        assert e.value.status == B.POD_ERR_INVALID


def test_greedy_layer_blocks_matches_the_oracle():
    """The library's Algorithm 1 against the oracle's on random similarities and on the hand-worked case."""
    import numpy as np
    rng = np.random.default_rng(11)
    for H, L, thr in [(1, 5, 0.5), (4, 9, 0.5), (3, 12, 0.3), (2, 7, 0.8)]:
        sim = rng.random((H, L, L)).astype(np.float32)
        want = O.lowest_map_from_blocks(O.greedy_layer_blocks(sim.astype(np.float64), thr), L)
        got = B.pod_greedy_layer_blocks(sim.tolist(), thr)
        assert got == want.tolist()
    sim = np.eye(5)[None].copy()
    for a, b, v in [(0, 1, .8), (0, 2, .4), (1, 2, .9), (0, 3, .9), (1, 3, .6), (2, 3, .7), (2, 4, .9), (3, 4, .2)]:
        sim[0, a, b] = sim[0, b, a] = v
    assert [row[0] for row in B.pod_greedy_layer_blocks(sim.tolist(), 0.5)] == [0, 0, 2, 2, 4]


def test_head_wise_block_maps_on_a_host_only_cache():
    cfg = _cfg(n_layers=4, n_kv_heads=2, n_q_heads=8, group_size=1)
    p = _fake_ptr()
    low = [[0, 0], [0, 1], [2, 1], [2, 1]]              # head 0: {0,1},{2,3}; head 1: {0},{1,2,3}
    for bad in ([[0, 0], [0, 0], [1, 0], [1, 0]], [[1, 0], [1, 1], [2, 1], [2, 1]], [[0, 0], [0, 2], [2, 2], [2, 2]]):
        with pytest.raises(B.PodError) as e:
            B.PodCache(cfg, [600], lowest_layer=bad)
        assert e.value.status == B.POD_ERR_INVALID
        assert B.pod_cache_required_bytes(cfg, [600], lowest_layer=bad) == 0
    assert B.pod_cache_required_bytes(cfg, [600], lowest_layer=low) > 0
    c = B.PodCache(cfg, [600], lowest_layer=low)
    for l in range(4):
        c.write(l, 0, p, p, 500)
    live, dense = O.pod_cache_bytes([500], n_layers=4, n_kv_heads=2, head_dim=64, lowest=low, n_s=16, n_r=64)
    assert c.bytes(B.POD_BYTES_LIVE) == live and c.bytes(B.POD_BYTES_DENSE_EQUIV) == dense
    # layer 1: head 0 needs layer 0's query of this step, head 1 starts a block here
    with pytest.raises(B.PodError) as e:
        c.decode_attn(1, p, p)
    assert e.value.status == B.POD_ERR_ORDER
    assert c.decode_attn(0, p, p) == B.POD_DRY_RUN
    assert c.decode_attn(1, p, p) == B.POD_DRY_RUN
    assert c.decode_attn(2, p, p) == B.POD_DRY_RUN      # head 0 lowest, head 1 follows layer 1 (decoded)
    assert c.decode_attn(3, p, p) == B.POD_DRY_RUN
    c.write(0, 0, p, p, 1)
    c.write(1, 0, p, p, 1)
    c.write(2, 0, p, p, 1)
    assert c.decode_attn(0, p, p) == B.POD_DRY_RUN
    with pytest.raises(B.PodError) as e:                 # head 1 of layer 2 follows layer 1, not decoded at this length
        c.decode_attn(2, p, p)
    assert e.value.status == B.POD_ERR_ORDER
    assert c.decode_attn(1, p, p) == B.POD_DRY_RUN
    assert c.decode_attn(2, p, p) == B.POD_DRY_RUN
    # a uniform map given explicitly is the same cache as group_size
    cu = B.PodCache(_cfg(n_layers=4, group_size=1), [600], lowest_layer=[[0, 0], [0, 0], [2, 2], [2, 2]])
    cg = B.PodCache(_cfg(n_layers=4, group_size=2), [600])
    assert cu.bytes(B.POD_BYTES_ALLOCATED) == cg.bytes(B.POD_BYTES_ALLOCATED)


def test_largest_cache_is_bounded_by_32_bit_row_indices():
    """Tile coordinates are 32-bit row indices: a cache whose regions would hold 2^31 rows or more is
    refused at creation (and sized 0), the largest one below that is accepted on a host-only cache."""
    cfg = _cfg(n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128, group_size=2, n_sink=16, n_recent=2048)
    # value rows of every layer + key rows of every block + the stored logits of a distant token
    # (two stores per KV head, 4 query heads x 4 bytes each: 8 x 2 x 16 B = one 256-byte row)
    rows_per_token = 32 * 8 + 16 * 8 + 1
    too_many = (2 ** 31) // rows_per_token + 4096
    assert B.pod_cache_required_bytes(cfg, [too_many]) == 0
    with pytest.raises(B.PodError) as e:
        B.PodCache(cfg, [too_many])
    assert e.value.status == B.POD_ERR_INVALID
    ok = (2 ** 31) // rows_per_token - 8192
    need = B.pod_cache_required_bytes(cfg, [ok])
    assert need > ok * rows_per_token * 256
    c = B.PodCache(cfg, [ok])
    assert c.bytes(B.POD_BYTES_ALLOCATED) == need


def test_dense_configuration_needs_no_order():
    cfg = _cfg(group_size=1)
    c = B.PodCache(cfg, [64])
    p = _fake_ptr()
    for l in range(4):
        c.write(l, 0, p, p, 5)
    for l in (3, 1, 0, 2):
        assert c.decode_attn(l, p, p) == B.POD_DRY_RUN


def test_host_only_cache_refuses_device_reads():
    c = B.PodCache(_cfg(), [64])
    with pytest.raises(B.PodError):
        c.read_region(B.POD_REGION_SINK_K, 0, 0, 0, 0, 1)
    assert c.device_status() == B.POD_DRY_RUN


def test_null_handles():
    assert B.lib.pod_cache_destroy(None) == B.POD_ERR_INVALID
    assert B.lib.pod_cache_bytes(None, 0) == -1
    assert B.lib.pod_cache_seq_len(None, 0, 0) == B.POD_ERR_INVALID
    assert B.lib.pod_cache_reset(None, 0) == B.POD_ERR_INVALID
    assert B.lib.pod_decode_attn(None, 0, None, None, None) == B.POD_ERR_INVALID
    assert B.lib.pod_append_decode_attn(None, 0, None, None, None, None, None) == B.POD_ERR_INVALID
    assert B.lib.pod_cache_write(None, 0, 0, None, None, 1, None) == B.POD_ERR_INVALID


def test_prefill_rejects_more_sharing_kv_heads_than_its_mask_holds():
    """Argument checks come before any CUDA call, so they are testable without a GPU: with the lowest layer's
    q, k given, more than 256 KV heads cannot be expressed in the kernel's sharing mask and are refused
    rather than silently computed as ordinary causal attention."""
    p = _fake_ptr()
    call = lambda hq, hkv, ql, kl: B.lib.pod_prefill_attn(8, hq, hkv, 64, 4, 4, 0.0, p, p, p, ql, kl, None, p, None)
    assert call(512, 512, p, p) == B.POD_ERR_INVALID
    assert call(257, 257, p, p) == B.POD_ERR_INVALID
    assert call(4, 2, p, None) == B.POD_ERR_INVALID             # q_low without k_low
    assert call(4, 2, p + 8, p) == B.POD_ERR_INVALID            # misaligned


def test_error_injection_on_a_host_only_cache_is_a_dry_run():
    c = B.PodCache(_cfg(), [64])
    assert c.inject_error() == B.POD_DRY_RUN
    assert c.device_status() == B.POD_DRY_RUN
