"""The allocation-free entry point against the oracle and against the ordinary entry point.

``pod_dense_decode_attn_static`` serves programs that cannot allocate device memory at the moment
they need attention (their memory pool already owns the whole GPU, their host framework forbids
raw allocations, or they cannot afford the device-wide synchronisation an allocation may cause):
its split-K scratch is a fixed array inside the library instead of part of an arena.  Here it is
called through the C ABI twice in a row -- the second call finds the array as the first left it --
and each output is compared with the fp64 oracle (dense attention is the PoD definition with one
layer per block) and with what ``pod_cache_write`` + ``pod_decode_attn`` give for the same keys,
values and queries, within the tolerance of the other parity tests.  This file is collected last
so that a run which stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import pod_oracle as O
from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth
from podtest import MAX_ABS, REL_L2

pytestmark = pytest.mark.gpu


def _existing_path(k, v, q, n, Hq, Hkv, d):
    """Dense attention through the ordinary entry points (one layer, every layer its own block)."""
    cfg = B.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, group_size=1, n_sink=4,
                        n_recent=32, batch=1, device=0)
    cache = B.PodCache(cfg, [max(n, 1)])
    out = torch.empty(1, Hq, d, dtype=torch.bfloat16, device="cuda")
    if n:
        cache.write(0, 0, k[:n], v[:n], n)
    cache.decode_attn(0, q.view(1, Hq, d), out)
    torch.cuda.synchronize()
    assert cache.device_status() == B.POD_OK
    cache.destroy()
    return out[0]


def _oracle(k, v, q, n, Hq, Hkv):
    """fp64 dense attention from the definition: every token proximal (n_s = 0, n_r = n)."""
    r = Hq // Hkv
    kk, vv, qq = k[:n].double().cpu().numpy(), v[:n].double().cpu().numpy(), q.double().cpu().numpy()
    return np.stack([O.pod_attention_joint(qq[h], qq[h], kk[:, h // r], kk[:, h // r], vv[:, h // r], 0, n)[0]
                     for h in range(Hq)])


def _compare(got, ref, what):
    g = got.double().cpu().numpy().ravel()
    r = (ref.double().cpu().numpy() if torch.is_tensor(ref) else np.asarray(ref)).ravel()
    max_abs = np.abs(g - r).max()
    rel = np.linalg.norm(g - r) / max(np.linalg.norm(r), 1e-30)
    assert max_abs <= MAX_ABS and rel <= REL_L2, f"{what}: max_abs={max_abs:.3e} rel_l2={rel:.3e}"


def _dense_buffer(seed, cap, n_real, Hkv, d):
    """Caller-owned [2][Hkv][cap][d] buffer: seeded rows below n_real, zeros (finite) above."""
    k = synth.gen_kv(seed, synth.TAG_K, 0, 0, 0, cap, Hkv, d, device="cuda")      # [cap][Hkv][d]
    v = synth.gen_kv(seed, synth.TAG_V, 0, 0, 0, cap, Hkv, d, device="cuda")
    k[n_real:] = 0
    v[n_real:] = 0
    return k, v, torch.stack([k.permute(1, 0, 2), v.permute(1, 0, 2)]).contiguous()


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 2), (64, 8, 2)])
def test_static_scratch_entry_matches_oracle_and_cache_entry_twice(d, Hq, Hkv):
    cap, seed = 5000, 31
    k, v, kv = _dense_buffer(seed, cap, cap, Hkv, d)             # rows past n_tokens are real rows here
    for call, n in enumerate((4321, 1777)):                      # two calls in a row, different work
        q = synth.gen_q(seed, 0, call, 1, Hq, d, device="cuda")[0].contiguous()
        out = torch.empty(Hq, d, dtype=torch.bfloat16, device="cuda")
        st = B.pod_dense_decode_attn_static(kv, cap, n, q, out, Hq, Hkv, d)
        torch.cuda.synchronize()
        assert st == B.POD_OK
        _compare(out, _oracle(k, v, q, n, Hq, Hkv), f"oracle, call {call} n={n}")
        _compare(out, _existing_path(k, v, q, n, Hq, Hkv, d), f"cache entry, call {call} n={n}")
    # an empty context gives zeros, like the ordinary entry point
    out.fill_(1.0)
    assert B.pod_dense_decode_attn_static(kv, cap, 0, q, out, Hq, Hkv, d) == B.POD_OK
    torch.cuda.synchronize()
    assert (out == 0).all()
    assert B.pod_dense_decode_attn_static_status() == B.POD_OK


@pytest.mark.parametrize("d,Hq,Hkv,cap,n", [
    (128, 8, 2, 640, 640),      # the context fills the buffer: the last value head's last tile ends at the tensor's end
    (64, 4, 4, 333, 333),       # the same with a ragged last tile: rows past the tensor read as zero fill
    (128, 8, 2, 64, 1),         # one token
    (64, 8, 2, 64, 17),         # one tile and one row; the rows after it are zeros
    (128, 2, 2, 900, 899),      # one query head per KV head
    (64, 16, 2, 1200, 1111),    # eight query heads per KV head
    (128, 64, 8, 3000, 2999),   # 64 query heads: the limit of the fixed array
])
def test_static_scratch_entry_edge_shapes_against_oracle(d, Hq, Hkv, cap, n):
    seed = 47
    k, v, kv = _dense_buffer(seed, cap, n, Hkv, d)               # rows at and past n_tokens hold zeros
    for call in range(2):                                        # back to back on one stream
        q = synth.gen_q(seed, 0, call, 1, Hq, d, device="cuda")[0].contiguous()
        out = torch.empty(Hq, d, dtype=torch.bfloat16, device="cuda")
        assert B.pod_dense_decode_attn_static(kv, cap, n, q, out, Hq, Hkv, d) == B.POD_OK
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        _compare(out, _oracle(k, v, q, n, Hq, Hkv), f"call {call} d={d} Hq={Hq} Hkv={Hkv} n={n}/{cap}")
    assert B.pod_dense_decode_attn_static_status() == B.POD_OK


def test_static_scratch_error_word_is_kept_until_read():
    """The error path without any failing kernel: the word is set from the host; calls do not clear it (their
    results would be reported as valid otherwise); the status call reports it once and clears it."""
    Hkv, d, cap, Hq = 2, 64, 256, 8
    k, v, kv = _dense_buffer(53, cap, cap, Hkv, d)
    q = synth.gen_q(53, 0, 0, 1, Hq, d, device="cuda")[0].contiguous()
    out = torch.empty(Hq, d, dtype=torch.bfloat16, device="cuda")
    assert B.pod_dense_decode_attn_static(kv, cap, 200, q, out, Hq, Hkv, d) == B.POD_OK
    assert B.pod_dense_decode_attn_static_status() == B.POD_OK
    B.pod_dense_decode_attn_static_inject_error()
    assert B.pod_dense_decode_attn_static(kv, cap, 200, q, out, Hq, Hkv, d) == B.POD_OK   # the call does not clear the word
    assert B.pod_dense_decode_attn_static_status() == B.POD_ERR_DEVICE
    assert B.pod_dense_decode_attn_static_status() == B.POD_OK
    assert B.pod_dense_decode_attn_static(kv, cap, 200, q, out, Hq, Hkv, d) == B.POD_OK
    torch.cuda.synchronize()
    _compare(out, _oracle(k, v, q, 200, Hq, Hkv), "after the injected error")


def test_static_scratch_entry_rejects_sizes_beyond_its_limits():
    Hkv, d, cap = 2, 64, 64
    kv = torch.zeros(2, Hkv, cap, d, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(128, d, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    for args, status in [((kv, cap, cap + 1, q, out, 8, Hkv, d), B.POD_ERR_CAPACITY),      # more tokens than rows
                         ((kv, cap, 8, q, out, 128, 16, d), B.POD_ERR_CAPACITY),           # more than 64 query heads
                         ((kv, cap, 8, q, out, 8, Hkv, 96), B.POD_ERR_INVALID),
                         ((kv, cap, 8, q, out, 7, Hkv, d), B.POD_ERR_INVALID),
                         ((None, cap, 8, q, out, 8, Hkv, d), B.POD_ERR_INVALID)]:
        with pytest.raises(B.PodError) as e:
            B.pod_dense_decode_attn_static(*args)
        assert e.value.status == status
