"""Shared helpers of the GPU parity tests: fill a cache with seeded inputs through the C ABI
and compute oracle outputs for selected (sequence, layer, head) triples on the host."""
from __future__ import annotations

import numpy as np
import torch

from oracle import pod_oracle as O
from paper_2412_02252_b200 import binding as B
from paper_2412_02252_b200 import synth

MAX_ABS, REL_L2 = 1e-2, 5e-3      # bf16 inputs, fp32 accumulation, bf16 output


class Case:
    def __init__(self, *, seed, L, G, Hq, Hkv, d, S, W, lens, outliers=False, caps=None, scale=0.0, lowest=None):
        self.seed, self.L, self.G, self.Hq, self.Hkv, self.d = seed, L, G, Hq, Hkv, d
        self.S, self.W, self.lens, self.outliers, self.scale = S, W, list(lens), outliers, scale
        self.B = len(self.lens)
        self.caps = list(caps) if caps is not None else [max(1, n) for n in self.lens]
        # per-head blocks: lowest[l][h]; None = runs of G layers for every head
        self.lowest = O.uniform_lowest_map(L, Hkv, G).tolist() if lowest is None else [list(r) for r in lowest]
        self.head_wise = lowest is not None
        self.cfg = B.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, group_size=G,
                                 n_sink=S, n_recent=W, batch=self.B, sm_scale=scale, device=0)

    # ---- inputs ------------------------------------------------------------------------------
    def kv(self, tag, layer, seq, p0, p1, device, heads=None):
        return synth.gen_kv(self.seed, tag, layer, seq, p0, p1, self.Hkv, self.d,
                            outliers=self.outliers, heads=heads, device=device)

    def q(self, layer, step, device):
        return synth.gen_q(self.seed, layer, step, self.B, self.Hq, self.d, device=device)

    # ---- CUDA path ---------------------------------------------------------------------------
    def make_cache(self):
        return B.PodCache(self.cfg, self.caps, lowest_layer=self.lowest if self.head_wise else None)

    def prefill(self, cache, upto=None, chunk=8192, layers=None):
        """Writes positions [len so far, upto[b]) of every sequence, layer by layer."""
        upto = self.lens if upto is None else upto
        stream = torch.cuda.current_stream().cuda_stream
        for l in (range(self.L) if layers is None else layers):
            for b in range(self.B):
                at = cache.seq_len(b, l)
                while at < upto[b]:
                    t = min(chunk, upto[b] - at)
                    k = self.kv(synth.TAG_K, l, b, at, at + t, "cuda")
                    v = self.kv(synth.TAG_V, l, b, at, at + t, "cuda")
                    cache.write(l, b, k, v, t, stream)
                    at += t

    def decode_all(self, cache, step=0):
        """One decode call per layer in order; returns bf16 [L][B][Hq][d] on the device."""
        stream = torch.cuda.current_stream().cuda_stream
        outs = torch.empty(self.L, self.B, self.Hq, self.d, dtype=torch.bfloat16, device="cuda")
        for l in range(self.L):
            q = self.q(l, step, "cuda")
            cache.decode_attn(l, q, outs[l], stream)
        torch.cuda.synchronize()
        assert cache.device_status() == B.POD_OK
        return outs

    # ---- oracle ------------------------------------------------------------------------------
    def oracle_head(self, layer, b, h, n=None, step=0):
        """fp64 output of query head h of (layer, sequence b) from the uncompressed history."""
        n = self.lens[b] if n is None else n
        if n == 0:
            return np.zeros(self.d)
        kvh = h // (self.Hq // self.Hkv)
        low = self.lowest[layer][kvh]
        f = lambda tag, l: self.kv(tag, l, b, 0, n, "cpu", heads=[kvh])[:, 0].double().numpy()
        K_l, V_l = f(synth.TAG_K, layer), f(synth.TAG_V, layer)
        K_a = K_l if low == layer else f(synth.TAG_K, low)
        q_l = self.q(layer, step, "cpu")[b, h].double().numpy()
        q_a = self.q(low, step, "cpu")[b, h].double().numpy()
        o, _ = O.pod_attention_joint(q_l, q_a, K_l, K_a, V_l, self.S, self.W,
                                     scale=(self.scale if self.scale > 0 else None))
        return o


def assert_close(got_bf16, ref_f64, what=""):
    got = got_bf16.double().cpu().numpy().reshape(-1)
    ref = np.asarray(ref_f64).reshape(-1)
    max_abs = np.abs(got - ref).max()
    denom = np.linalg.norm(ref)
    rel = np.linalg.norm(got - ref) / denom if denom > 0 else np.linalg.norm(got - ref)
    assert max_abs <= MAX_ABS and rel <= REL_L2, f"{what}: max_abs={max_abs:.3e} rel_l2={rel:.3e}"
    return max_abs, rel
