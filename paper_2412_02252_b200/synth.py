"""Seeded synthetic inputs for the PoD decode path (test and bench infrastructure).

This module holds none of the method's arithmetic: it only produces the bf16 tensors
(q, K, V) that the CUDA path and the CPU oracle are both fed.  Every element is a pure
function of ``(seed, tensor tag, layer, sequence, position, head, channel)`` computed with
integer operations only, so the same bits come out on the host and on the device and a
100 GiB cache never has to exist in host memory: the host can regenerate any single
(layer, sequence, head) stream it wants to check.

Recipe
------
* a 32-bit counter hash (two rounds of a multiply/xor-shift mixer) of the element's
  linear index inside its tensor, offset by a key derived from (seed, tag, layer, seq);
* the top 16 bits index a 65 536-entry table of N(0,1) quantiles rounded to bf16
  (``ndtri((i + 0.5) / 65536)`` in fp64 on the host), so values are i.i.d. N(0,1)
  up to the table's resolution and clipped at about +-4.3;
* optional outlier channels: a channel ``c`` of (tag, layer) is an outlier when a hash of
  it is 0 modulo 100 (about 1 % of channels); its values are multiplied by 8, which is
  exact in bf16.  This imitates the few large-magnitude channels seen in LLM K/V caches.
"""
from __future__ import annotations

import functools

import torch

TAG_K = 1
TAG_V = 2
TAG_Q = 3

_M32 = 0xFFFFFFFF
_C1 = 0x7FEB352D
_C2 = 0x846CA68B
_GOLD = 0x9E3779B9


def _mix32_int(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * _C1) & _M32
    x ^= x >> 15
    x = (x * _C2) & _M32
    x ^= x >> 16
    return x


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """Same mixer on an int64 tensor whose values lie in [0, 2**32)."""
    x = x ^ (x >> 16)
    x = (x * _C1) & _M32
    x = x ^ (x >> 15)
    x = (x * _C2) & _M32
    x = x ^ (x >> 16)
    return x


def tensor_key(seed: int, tag: int, layer: int, seq: int) -> int:
    k = _mix32_int(seed * _GOLD + 0x51ED27)
    k = _mix32_int(k + tag * 0x632BE5AB)
    k = _mix32_int(k + layer * 0x85157AF5)
    k = _mix32_int(k + seq * 0x2545F491)
    return k


@functools.lru_cache(maxsize=None)
def _table_cpu() -> torch.Tensor:
    p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
    return torch.special.ndtri(p).to(torch.bfloat16)


_table_dev: dict = {}


def normal_table(device="cpu") -> torch.Tensor:
    """bf16 [65536] table of N(0,1) quantiles; always computed on the host, then copied."""
    device = torch.device(device)
    if device.type == "cpu":
        return _table_cpu()
    key = (device.type, device.index)
    if key not in _table_dev:
        _table_dev[key] = _table_cpu().to(device)
    return _table_dev[key]


def outlier_channels(seed: int, tag: int, layer: int, n_heads: int, head_dim: int) -> torch.Tensor:
    """bool [n_heads * head_dim] (host): True where the channel is scaled by 8."""
    key = _mix32_int(tensor_key(seed, tag, layer, 0x7FFF) ^ 0xA5A5A5A5)
    c = torch.arange(n_heads * head_dim, dtype=torch.int64)
    h = _mix32((_mix32(c) + key) & _M32)
    return (h % 100) == 0


def _generate(key: int, counters: torch.Tensor) -> torch.Tensor:
    h = _mix32((_mix32(counters) + key) & _M32)
    return normal_table(counters.device)[h >> 16]


def gen_kv(seed: int, tag: int, layer: int, seq: int, pos0: int, pos1: int,
           n_kv_heads: int, head_dim: int, *, outliers: bool = False, heads=None,
           device="cpu") -> torch.Tensor:
    """bf16 ``[pos1 - pos0][n_heads_out][head_dim]`` slice of K (``TAG_K``) or V (``TAG_V``)
    of one (layer, sequence), token-major like a projection output.

    ``heads``: optional list of KV-head indices; only those heads are generated (in the
    order given), with the values they have in the full tensor.
    """
    device = torch.device(device)
    hd = n_kv_heads * head_dim
    head_ix = torch.arange(n_kv_heads, dtype=torch.int64, device=device) if heads is None \
        else torch.tensor(list(heads), dtype=torch.int64, device=device)
    pos = torch.arange(pos0, pos1, dtype=torch.int64, device=device)
    chan = torch.arange(head_dim, dtype=torch.int64, device=device)
    inner = head_ix[:, None] * head_dim + chan[None, :]            # [h][d]
    counters = pos[:, None, None] * hd + inner[None]               # [t][h][d]
    x = _generate(tensor_key(seed, tag, layer, seq), counters)
    if outliers:
        mask = outlier_channels(seed, tag, layer, n_kv_heads, head_dim).to(device)[inner]
        x = torch.where(mask[None], x * 8.0, x)
    return x.contiguous()


def gen_q(seed: int, layer: int, step: int, batch: int, n_q_heads: int, head_dim: int,
          *, device="cpu") -> torch.Tensor:
    """bf16 ``[batch][n_q_heads][head_dim]`` queries of one layer at one decode step."""
    device = torch.device(device)
    n = batch * n_q_heads * head_dim
    counters = torch.arange(n, dtype=torch.int64, device=device)
    x = _generate(tensor_key(seed, TAG_Q, layer, step), counters)
    return x.view(batch, n_q_heads, head_dim).contiguous()


def ragged_lengths(seed: int, batch: int, lo: int, hi: int) -> list:
    """``batch`` sequence lengths drawn uniformly from [lo, hi] (inclusive), seeded."""
    key = tensor_key(seed, 0x4C, 0, 0)
    return [lo + _mix32_int(_mix32_int(i) + key) % (hi - lo + 1) for i in range(batch)]


def bf16_bits(x: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its bit patterns (host)."""
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
