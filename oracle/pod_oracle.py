"""fp64 CPU oracle for PoD decode attention over the compressed KV cache.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the decode path
computes, written from the paper.  It shares no code with the CUDA library and must never
be imported by it: only the tests, the smoke check and the bench's CPU-baseline leg may
call it.  Everything is numpy in float64; inputs are the exact values of the bf16 inputs.

Notation (paper, Section 2.2): layer l lies in a block of consecutive layers whose lowest
layer is l_a; n_s = number of initial ("start"/sink) tokens, n_r = number of most recent
tokens; those two groups are the proximal tokens, everything in between is distant.
Positions here are 0-based and the token being decoded is the last one (i = n), its K/V
already appended: sink = [0, min(n, n_s)), recent = [max(n_s, n - n_r), n),
distant = [n_s, n - n_r) (empty unless n > n_s + n_r).

Pins (tests/test_oracle_pins.py): textbook dense attention when a block has one layer or
when there are no distant tokens; Appendix C identity (gate form == one softmax); weights
sum to one; pure-Python brute force; hand-worked rational example; planted-key cases;
shared-score invariance; incremental layout == layout built from the history; byte counts
against the closed form and the paper's own saving arithmetic.

Blocks are per head (Section 2.1, Algorithm 1: every head gets its own partition of the
layers into runs of consecutive similar layers).  A partition is carried as a "lowest map"
low[l][h] = lowest layer of the block that holds layer l for KV head h; ``group_size`` is the
special case in which every head uses runs of G layers.  greedy_layer_blocks is Algorithm 1.
Pins of these: hand-worked grouping example, the algorithm's defining properties checked by
brute force, uniform maps == group_size, per-head independence, byte counts by enumeration.

Readings of points the paper leaves open are listed next to the code that takes them.
"""
from __future__ import annotations

import math

import numpy as np


# --------------------------------------------------------------------------------------
# helpers that are not part of the method
# --------------------------------------------------------------------------------------
def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def lowest_layer(layer: int, group_size: int) -> int:
    """Blocks are runs of ``group_size`` consecutive layers (0-based); the last may be short."""
    return layer - layer % group_size


def uniform_lowest_map(n_layers: int, n_kv_heads: int, group_size: int) -> np.ndarray:
    """low[l][h] for blocks of ``group_size`` consecutive layers, the same for every head."""
    return np.array([[lowest_layer(l, group_size)] * n_kv_heads for l in range(n_layers)], dtype=np.int64)


def check_lowest_map(low) -> np.ndarray:
    """A lowest map describes, per head, a partition of the layers into runs of consecutive
    layers: low[0][h] = 0 and low[l][h] is either l (a new block starts) or low[l-1][h]."""
    low = np.asarray(low, dtype=np.int64)
    L, H = low.shape
    for h in range(H):
        for l in range(L):
            ok = low[l, h] == l or (l > 0 and low[l, h] == low[l - 1, h])
            if not ok:
                raise ValueError(f"not a partition into consecutive runs at layer {l}, head {h}")
    return low


def greedy_layer_blocks(sim, threshold=0.5):
    """Greedy grouping of consecutive similar layers, per head (Section 2.1, Algorithm 1).

    sim: [H][L][L], sim[h][a][b] = similarity of layers a and b for head h (1 = identical).
    The rule of the algorithm: walking up from layer 0, a layer stays in the block of the layer
    below it exactly when it is similar (>= threshold) to every layer that block holds so far;
    otherwise it starts a block of its own.  Written here through each layer's "reach": the lowest
    layer m such that the layer is similar to all of m .. l-1.  A layer then continues the block
    below it iff its reach is at or below that block's first layer.
    Returns, per head, the list of blocks, each a list of 0-based layers.
    """
    similar = np.asarray(sim, dtype=np.float64) >= threshold
    H, L, _ = similar.shape
    result = []
    for h in range(H):
        reach = np.arange(L)
        for l in range(L):
            below = similar[h, l, :l][::-1]                    # l-1, l-2, ..., 0
            run = int(np.argmin(below)) if not below.all() else l   # similar layers directly below l
            reach[l] = l - run
        first = np.zeros(L, dtype=np.int64)                    # first layer of the block of each layer
        for l in range(1, L):
            first[l] = first[l - 1] if reach[l] <= first[l - 1] else l
        result.append([[int(l) for l in np.flatnonzero(first == f)] for f in np.unique(first)])
    return result


def lowest_map_from_blocks(head_wise_layer_blocks, n_layers: int) -> np.ndarray:
    """low[l][h] from the per-head block lists of greedy_layer_blocks."""
    H = len(head_wise_layer_blocks)
    low = np.full((n_layers, H), -1, dtype=np.int64)
    for h, blocks in enumerate(head_wise_layer_blocks):
        for block in blocks:
            for l in block:
                low[l, h] = block[0]
    return check_lowest_map(low)


def _resolve_map(n_layers, n_kv_heads, group_size, lowest):
    if lowest is not None:
        low = check_lowest_map(lowest)
        if low.shape != (n_layers, n_kv_heads):
            raise ValueError("lowest map must be [n_layers][n_kv_heads]")
        return low
    return uniform_lowest_map(n_layers, n_kv_heads, group_size)


def is_proximal(p: int, n: int, n_s: int, n_r: int) -> bool:
    """Section 2.2: the first n_s and the last n_r tokens (including the current one)."""
    return p < n_s or p >= n - n_r


# --------------------------------------------------------------------------------------
# single head, full (uncompressed) history: the definition
# --------------------------------------------------------------------------------------
def pod_logits(q_l, q_a, K_l, K_a, n_s, n_r, scale):
    """Eq. 1 rows 1 and 3 for one head at the decode position.

    q_l: [d] query of layer l; q_a: [d] query of the block's lowest layer l_a;
    K_l, K_a: [n][d] keys of layer l and of layer l_a.  Returns (logits [n], prox mask [n]).
    Proximal logits pair layer l's query with layer l's keys; distant logits are the ones
    the lowest layer computes: its query with its keys.
    """
    n = K_l.shape[0]
    p = np.arange(n)
    prox = (p < n_s) | (p >= n - n_r)
    a_own = (K_l @ q_l) * scale
    a_low = (K_a @ q_a) * scale
    return np.where(prox, a_own, a_low), prox


def pod_attention_joint(q_l, q_a, K_l, K_a, V_l, n_s, n_r, scale=None):
    """Appendix C: the output is one softmax over the proximal and distant logits together,
    applied to layer l's own values (Eq. 1 rows 2 and 4 use V_l in both).
    Returns (o [d], weights [n])."""
    d = q_l.shape[0]
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    a, _ = pod_logits(q_l, q_a, K_l, K_a, n_s, n_r, scale)
    e = np.exp(a - a.max())
    w = e / e.sum()
    return w @ V_l, w


def pod_attention_gate(q_l, q_a, K_l, K_a, V_l, n_s, n_r, scale=None):
    """Eq. 1 then Eq. 2, as printed: a softmax over the proximal logits, a softmax over
    the distant logits, and the parameter-free gate g blending the two outputs.  With no
    distant tokens the distant term is omitted (footnote to Eq. 1).
    Returns (o [d], g)."""
    d = q_l.shape[0]
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    a, prox = pod_logits(q_l, q_a, K_l, K_a, n_s, n_r, scale)
    aP, VP = a[prox], V_l[prox]
    aD, VD = a[~prox], V_l[~prox]
    oP = _softmax(aP) @ VP
    if aD.size == 0:
        return oP, 1.0
    oD = _softmax(aD) @ VD
    # g = sum exp aP / (sum exp aP + sum exp aD); a common shift keeps the exps finite
    shift = max(aP.max(), aD.max())
    sP = np.exp(aP - shift).sum()
    sD = np.exp(aD - shift).sum()
    g = sP / (sP + sD)
    return g * oP + (1.0 - g) * oD, g


def pod_attention_gate_skip(q_l, q_a, K_l, K_a, V_l, n_s, n_r, tau, scale=None):
    """Appendix "Computation Optimization for Distant Tokens": for a layer that is not the lowest of
    its block the gate g of Eq. 2 is evaluated first (the distant logits are the lowest layer's, so
    their sum is known before any distant value is read); if g >= tau the attention to the distant
    tokens is omitted.  Reading of "omitted": the output is then the proximal output o^P alone (the
    gate is treated as 1); otherwise Eq. 2 is applied unchanged.  The caller applies this to layers
    other than a block's lowest only.  Returns (o [d], g, skipped)."""
    d = q_l.shape[0]
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    a, prox = pod_logits(q_l, q_a, K_l, K_a, n_s, n_r, scale)
    aP, VP = a[prox], V_l[prox]
    aD, VD = a[~prox], V_l[~prox]
    oP = _softmax(aP) @ VP
    if aD.size == 0:                      # no distant tokens: nothing to omit
        return oP, 1.0, False
    shift = max(aP.max(), aD.max())
    sP = np.exp(aP - shift).sum()
    sD = np.exp(aD - shift).sum()
    g = sP / (sP + sD)
    if g >= tau:
        return oP, g, True
    oD = _softmax(aD) @ VD
    return g * oP + (1.0 - g) * oD, g, False


def _softmax(a):
    e = np.exp(a - a.max())
    return e / e.sum()


# --------------------------------------------------------------------------------------
# all heads of one layer, full history
# --------------------------------------------------------------------------------------
def pod_decode_layer(q, K, V, layer, *, group_size=None, lowest=None, n_s, n_r, scale=None, form="joint",
                     tau=None, info=None):
    """One layer's decode attention for one sequence from the uncompressed history.

    q: [L][H_q][d] queries of every layer at this step (only rows ``layer`` and its blocks'
    lowest layers are read); K, V: [L][n][H_kv][d].  Blocks: ``group_size`` (runs of G layers for
    every head) or ``lowest`` (a per-head lowest map [L][H_kv]).  Query head h reads KV head h // r,
    r = H_q / H_kv (grouped-query attention).  Returns o [H_q][d] (float64).
    An empty history (n == 0) gives zeros (convention of this build; the paper is silent).
    ``tau``: gate threshold of the distant-skip optimisation (None = off); heads for which ``layer``
    is not the lowest layer of their block skip the distant tokens when g >= tau.  ``info``, if a
    list, receives (g, skipped) per query head.
    """
    L, n, H_kv, d = K.shape
    H_q = q.shape[1]
    r = H_q // H_kv
    low = _resolve_map(L, H_kv, group_size, lowest)
    out = np.zeros((H_q, d))
    if n == 0:
        return out
    fn = pod_attention_joint if form == "joint" else pod_attention_gate
    for h in range(H_q):
        kv = h // r
        a = int(low[layer, kv])                 # lowest layer of this head's block
        if tau is not None and a != layer:
            out[h], g, skipped = pod_attention_gate_skip(q[layer, h], q[a, h], K[layer, :, kv], K[a, :, kv],
                                                         V[layer, :, kv], n_s, n_r, tau, scale)
            if info is not None:
                info.append((g, skipped))
            continue
        if info is not None:
            info.append((None, False))
        out[h], _ = fn(q[layer, h], q[a, h], K[layer, :, kv], K[a, :, kv], V[layer, :, kv],
                       n_s, n_r, scale)
    return out


def pod_prefill_layer(q, K, V, layer, *, group_size=None, lowest=None, n_s, n_r, scale=None):
    """PoD attention of one layer for EVERY position of a sequence (prefill; Section 2.2 and the
    masks of Fig. 2, middle): position i attends to the tokens up to and including itself, the
    proximal ones being the first n_s and the last n_r of those, exactly as the decode step of a
    sequence that ends at i does.

    q: [L][n][H_q][d] queries of every layer and position; K, V: [L][n][H_kv][d].
    Returns o [n][H_q][d] (float64).  Written as n independent decode steps on prefixes.
    """
    L, n, H_kv, d = K.shape
    H_q = q.shape[2]
    out = np.zeros((n, H_q, d))
    for i in range(n):
        out[i] = pod_decode_layer(q[:, i], K[:, :i + 1], V[:, :i + 1], layer, group_size=group_size,
                                  lowest=lowest, n_s=n_s, n_r=n_r, scale=scale)
    return out


# --------------------------------------------------------------------------------------
# the PoD cache layout, maintained token by token (layout form)
# --------------------------------------------------------------------------------------
class PodCacheOracle:
    """The compressed cache of one sequence as plain arrays of bf16 bit patterns.

    Regions (logical content is the contract; each row is one head's d-vector):
      sinkK/sinkV[l][h][j]          position j < n_s
      ringK/ringV[l][h][s]          position p in the recent window, slot s = (p - n_s) mod n_r
      distV[l][h][p - n_s]          distant position p, layer l's own value
      distK[g][h][p - n_s]          distant position p, key of the lowest layer of block g

    Update rule on appending the token at position p = n (reading of the paper's missing
    cache-update figure): if p < n_s it is a sink row; otherwise it takes ring slot
    (p - n_s) mod n_r, and the token that held that slot, position p - n_r (if >= n_s),
    has just left the recent window: its value moves to distV[l], its key moves to distK[g]
    only when l is the lowest layer of its block and is discarded otherwise.
    """

    def __init__(self, n_layers, n_kv_heads, head_dim, group_size, n_s, n_r, capacity, lowest=None):
        self.L, self.H, self.d = n_layers, n_kv_heads, head_dim
        self.G, self.S, self.W = group_size, n_s, n_r
        self.cap = capacity
        self.cap_d = max(0, capacity - n_s - n_r)
        self.low = _resolve_map(n_layers, n_kv_heads, group_size, lowest)
        # blocks of a head in layer order; block_of[l][h] = index of (l, h)'s block in that list
        self.blocks = [sorted(set(int(x) for x in self.low[:, h])) for h in range(n_kv_heads)]
        self.block_of = np.array([[self.blocks[h].index(int(self.low[l, h])) for h in range(n_kv_heads)]
                                  for l in range(n_layers)])
        self.n_blocks = max(len(b) for b in self.blocks)      # most blocks any head has
        z = lambda *s: np.zeros(s, dtype=np.uint16)
        self.sinkK = z(self.L, self.H, n_s, head_dim)
        self.sinkV = z(self.L, self.H, n_s, head_dim)
        self.ringK = z(self.L, self.H, n_r, head_dim)
        self.ringV = z(self.L, self.H, n_r, head_dim)
        self.distV = z(self.L, self.H, self.cap_d, head_dim)
        self.distK = z(self.n_blocks, self.H, self.cap_d, head_dim)
        self.len = [0] * self.L

    # -- write ---------------------------------------------------------------------------
    def append(self, layer, k_row, v_row):
        """k_row, v_row: uint16 [H_kv][d], the new token's key and value at ``layer``."""
        S, W = self.S, self.W
        p = self.len[layer]
        if p >= self.cap:
            raise ValueError("capacity exceeded")
        if p < S:
            self.sinkK[layer, :, p] = k_row
            self.sinkV[layer, :, p] = v_row
        else:
            slot = (p - S) % W
            old = p - W
            if old >= S:                                   # leaves the recent window
                self.distV[layer, :, old - S] = self.ringV[layer, :, slot]
                for h in range(self.H):
                    if self.low[layer, h] == layer:        # keys survive once per block
                        self.distK[self.block_of[layer, h], h, old - S] = self.ringK[layer, h, slot]
            self.ringK[layer, :, slot] = k_row
            self.ringV[layer, :, slot] = v_row
        self.len[layer] = p + 1

    def write(self, layer, k, v):
        """k, v: uint16 [T][H_kv][d]; a prefill or chunk is T appends in order."""
        for t in range(k.shape[0]):
            self.append(layer, k[t], v[t])

    # -- read ----------------------------------------------------------------------------
    def valid_rows(self, region, index, head):
        """Valid rows of a region for one head, in region order, as uint16 [count][d],
        together with the first region index they start at."""
        if region == "distK" and index >= len(self.blocks[head]):
            return self.distK[index, head, :0], 0          # this head has fewer blocks
        n = self.len[self.blocks[head][index] if region == "distK" else index]
        S, W = self.S, self.W
        n_d = max(0, n - S - W)
        if region in ("sinkK", "sinkV"):
            return getattr(self, region)[index, head, :min(n, S)], 0
        if region in ("ringK", "ringV"):
            return getattr(self, region)[index, head, :min(W, max(0, n - S))], 0
        if region in ("distK", "distV"):
            return getattr(self, region)[index, head, :n_d], 0
        raise KeyError(region)

    def attend(self, layer, q, q_low, scale=None):
        """Decode attention of ``layer`` computed from the regions.

        q: [H_q][d] float64 queries of this layer; q_low: [H_q][d], row h = the query of head h
        at the lowest layer of that head's block at the same step.  Token order inside the softmax is sink, ring slots,
        distant; the softmax does not depend on it.  Returns o [H_q][d] float64.
        """
        S, W, G = self.S, self.W, self.G
        n = self.len[layer]
        H_q = q.shape[0]
        r = H_q // self.H
        scale = 1.0 / math.sqrt(self.d) if scale is None else scale
        out = np.zeros((H_q, self.d))
        if n == 0:
            return out
        for kv in range(self.H):
            if self.len[int(self.low[layer, kv])] != n:
                raise ValueError("layers of a block must hold the same number of tokens")
        n_sink, n_ring, n_d = min(n, S), min(W, max(0, n - S)), max(0, n - S - W)
        for h in range(H_q):
            kv = h // r
            Kp = bits_to_f64(np.concatenate([self.sinkK[layer, kv, :n_sink],
                                             self.ringK[layer, kv, :n_ring]]))
            Vp = bits_to_f64(np.concatenate([self.sinkV[layer, kv, :n_sink],
                                             self.ringV[layer, kv, :n_ring]]))
            Kd = bits_to_f64(self.distK[self.block_of[layer, kv], kv, :n_d])
            Vd = bits_to_f64(self.distV[layer, kv, :n_d])
            a = np.concatenate([(Kp @ q[h]) * scale, (Kd @ q_low[h]) * scale])
            e = np.exp(a - a.max())
            w = e / e.sum()
            out[h] = w @ np.concatenate([Vp, Vd])
        return out


def layout_from_history(K_bits, V_bits, *, group_size=None, lowest=None, n_s, n_r, capacity):
    """The regions as a function of the full history, written out directly (no appends):
    K_bits, V_bits uint16 [L][n][H_kv][d].  Used to check the incremental update rule."""
    L, n, H, d = K_bits.shape
    c = PodCacheOracle(L, H, d, group_size, n_s, n_r, capacity, lowest=lowest)
    for l in range(L):
        for p in range(n):
            kr, vr = K_bits[l, p], V_bits[l, p]
            if p < n_s:
                c.sinkK[l, :, p], c.sinkV[l, :, p] = kr, vr
            elif p >= n - n_r:
                s = (p - n_s) % n_r
                c.ringK[l, :, s], c.ringV[l, :, s] = kr, vr
            else:
                c.distV[l, :, p - n_s] = vr
                for h in range(H):
                    if c.low[l, h] == l:
                        c.distK[c.block_of[l, h], h, p - n_s] = kr[h]
        c.len[l] = n
    return c


# --------------------------------------------------------------------------------------
# byte accounting
# --------------------------------------------------------------------------------------
def pod_cache_bytes(lens, *, n_layers, n_kv_heads, head_dim, group_size=None, lowest=None, n_s, n_r,
                    elem_bytes=2):
    """(live PoD bytes, dense-equivalent bytes) for sequences of the given lengths.

    Proximal tokens keep K and V in every layer; distant tokens keep V in every layer and K
    once per block (abstract; Section 2.2).  Dense keeps K and V of all tokens in all layers.
    """
    row = head_dim * elem_bytes
    low = _resolve_map(n_layers, n_kv_heads, group_size, lowest)
    # (layer, head) pairs that are the lowest layer of their block keep their distant keys
    n_key_stores = int(sum(low[l, h] == l for l in range(n_layers) for h in range(n_kv_heads)))
    live = dense = 0
    for n in lens:
        n_p = min(n, n_s + n_r)
        n_d = n - n_p
        live += row * (n_kv_heads * n_layers * (2 * n_p + n_d) + n_key_stores * n_d)
        dense += n_kv_heads * row * n_layers * 2 * n
    return live, dense


def pod_saving_closed_form(n, *, n_layers, group_size=None, n_s, n_r, shared_fraction=None):
    """Fraction of dense KV bytes saved at length n: half of the bytes are keys, a fraction
    n_d/n of them belongs to distant tokens, and of those only one layer per block remains.
    ``shared_fraction``: fraction of (layer, head) pairs that are not the lowest layer of their
    block, for head-wise blocks; with ``group_size`` it is 1 - ceil(L/G)/L."""
    n_d = max(0, n - n_s - n_r)
    if shared_fraction is None:
        n_blocks = (n_layers + group_size - 1) // group_size
        shared_fraction = 1.0 - n_blocks / n_layers
    return (n_d / n) * shared_fraction / 2.0
