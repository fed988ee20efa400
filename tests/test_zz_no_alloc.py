"""The allocation-free entry point against the ordinary one.

``pod_dense_decode_attn_static`` serves programs that cannot allocate device memory at the moment
they need attention (their memory pool already owns the whole GPU, their host framework forbids
raw allocations, or they cannot afford the device-wide synchronisation an allocation may cause):
its split-K scratch is a fixed array inside the library instead of part of an arena.  Here it is
called through the C ABI twice in a row -- the second call finds the array as the first left it --
and each output is compared with what ``pod_cache_write`` + ``pod_decode_attn`` give for the same
keys, values and queries, within the tolerance of the other parity tests.  This file is collected
last so that a run which stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

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


def _compare(got, ref, what):
    g, r = got.double().cpu().numpy().ravel(), ref.double().cpu().numpy().ravel()
    max_abs = np.abs(g - r).max()
    rel = np.linalg.norm(g - r) / max(np.linalg.norm(r), 1e-30)
    assert max_abs <= MAX_ABS and rel <= REL_L2, f"{what}: max_abs={max_abs:.3e} rel_l2={rel:.3e}"


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 2), (64, 8, 2)])
def test_static_scratch_entry_matches_cache_entry_twice(d, Hq, Hkv):
    cap = 5000
    seed = 31
    k = synth.gen_kv(seed, synth.TAG_K, 0, 0, 0, cap, Hkv, d, device="cuda")      # [cap][Hkv][d]
    v = synth.gen_kv(seed, synth.TAG_V, 0, 0, 0, cap, Hkv, d, device="cuda")
    # caller-owned dense buffer [2][Hkv][cap][d]; rows past n_tokens are finite (real rows here)
    kv = torch.stack([k.permute(1, 0, 2), v.permute(1, 0, 2)]).contiguous()
    for call, n in enumerate((4321, 1777)):                      # two calls in a row, different work
        q = synth.gen_q(seed, 0, call, 1, Hq, d, device="cuda")[0].contiguous()
        out = torch.empty(Hq, d, dtype=torch.bfloat16, device="cuda")
        st = B.pod_dense_decode_attn_static(kv, cap, n, q, out, Hq, Hkv, d)
        torch.cuda.synchronize()
        assert st == B.POD_OK
        _compare(out, _existing_path(k, v, q, n, Hq, Hkv, d), f"call {call} n={n}")
    # an empty context gives zeros, like the ordinary entry point
    out.fill_(1.0)
    assert B.pod_dense_decode_attn_static(kv, cap, 0, q, out, Hq, Hkv, d) == B.POD_OK
    torch.cuda.synchronize()
    assert (out == 0).all()


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
