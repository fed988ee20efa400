"""Shared helpers of the GPU parity tests: fill a cache with seeded inputs through the C ABI
and compute oracle outputs for selected (sequence, layer, head) triples on the host."""
from __future__ import annotations

import concurrent.futures as cf
import os

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


class KVHeadChecker:
    """Oracle comparison of whole KV-head groups at sizes where every (sequence, layer, head) is checked.

    The r query heads of a KV head share K_l, K_a and V_l, so these are regenerated once per group (on the
    GPU, by the seeded generator, and copied to the host as fp32, which holds bf16 exactly); the oracle
    function itself runs unchanged, once per query head, in fp64 on the host.  Groups are computed by a
    pool of host threads (numpy releases the interpreter lock) while the main thread regenerates inputs.
    """

    def __init__(self, case, workers=None, max_pending=24):
        self.case = case
        self.pool = cf.ThreadPoolExecutor(max_workers=workers or max(2, min(16, (os.cpu_count() or 4))))
        try:                                   # one BLAS thread per pool thread instead of a pool of pools
            from threadpoolctl import threadpool_limits
            self._blas = threadpool_limits(limits=1)
        except Exception:
            self._blas = None
        self.pending, self.max_pending = [], max_pending
        self.worst = [0.0, 0.0]
        self.checked = 0

    def _inputs(self, layer, b, kvh, n, step):
        c = self.case
        r = c.Hq // c.Hkv
        low = c.lowest[layer][kvh]
        f = lambda tag, l: c.kv(tag, l, b, 0, n, "cuda", heads=[kvh])[:, 0].float().cpu().numpy()
        K_l, V_l = f(synth.TAG_K, layer), f(synth.TAG_V, layer)
        K_a = K_l if low == layer else f(synth.TAG_K, low)
        q_l = c.q(layer, step, "cpu")[b, kvh * r:(kvh + 1) * r].double().numpy()
        q_a = c.q(low, step, "cpu")[b, kvh * r:(kvh + 1) * r].double().numpy()
        return K_l, K_a, V_l, q_l, q_a, low != layer

    def _work(self, inp, got, what, tau):
        K_l, K_a, V_l, q_l, q_a, shares = inp
        c = self.case
        K_l64, V_l64 = K_l.astype(np.float64), V_l.astype(np.float64)
        K_a64 = K_l64 if K_a is K_l else K_a.astype(np.float64)
        scale = c.scale if c.scale > 0 else None
        res = []
        for i in range(q_l.shape[0]):
            ref, _ = O.pod_attention_joint(q_l[i], q_a[i], K_l64, K_a64, V_l64, c.S, c.W, scale=scale)
            ok = _close(got[i], ref)
            if tau is not None and shares:
                # a head of a sharing layer under a gate threshold: the oracle's decision decides, except within
                # 0.01 of the threshold (the device takes it in fp32), where either candidate is a valid result
                alt, g, skipped = O.pod_attention_gate_skip(q_l[i], q_a[i], K_l64, K_a64, V_l64, c.S, c.W, tau, scale=scale)
                ok_alt = _close(got[i], alt)
                if abs(g - tau) >= 0.01:
                    ok = ok_alt
                elif ok_alt[0]:
                    ok = ok_alt
            res.append((ok, f"{what} head {i}"))
        return res

    def submit(self, outs, layer, b, kvh, n, step=0, tau=None):
        """outs: bf16 device tensor [L][B][Hq][d] (or the same on the host)."""
        r = self.case.Hq // self.case.Hkv
        got = outs[layer, b, kvh * r:(kvh + 1) * r].double().cpu().numpy()
        inp = self._inputs(layer, b, kvh, n, step)
        self.pending.append(self.pool.submit(self._work, inp, got, f"seq {b} layer {layer} kv head {kvh} step {step}", tau))
        if len(self.pending) >= self.max_pending:
            self._drain(self.max_pending // 2)

    def _drain(self, keep):
        while len(self.pending) > keep:
            for (ok, max_abs, rel), what in self.pending.pop(0).result():
                assert ok, f"{what}: max_abs={max_abs:.3e} rel_l2={rel:.3e}"
                self.worst = [max(self.worst[0], max_abs), max(self.worst[1], rel)]
                self.checked += 1

    def finish(self):
        self._drain(0)
        self.pool.shutdown()
        if self._blas is not None:
            self._blas.restore_original_limits()
        return self.worst


def _close(got, ref):
    g, r = np.asarray(got).reshape(-1), np.asarray(ref).reshape(-1)
    max_abs = float(np.abs(g - r).max())
    denom = np.linalg.norm(r)
    rel = float(np.linalg.norm(g - r) / denom) if denom > 0 else float(np.linalg.norm(g - r))
    return (max_abs <= MAX_ABS and rel <= REL_L2), max_abs, rel
