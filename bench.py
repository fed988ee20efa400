#!/usr/bin/env python
"""Benchmark of the PoD decode hot path (cache append + decode attention for every layer).

One "step" is one decode step of the whole model's attention: for each layer, append the new
token's K/V to the PoD cache and attend over it (``pod_append_decode_attn``: the work of
``pod_cache_write`` + ``pod_decode_attn`` in one launch; the two-call form is timed beside it).  The
headline workload is the LLaMA-3-8B-shaped single-sequence decode at 32K context (32 layers, G = 2,
32/8 heads, d = 128, S = 16, W = 2048, seeded synthetic bf16 K/V with outlier channels); the 128K,
batch-16 and ragged serving workloads are measured in the same run and reported under ``workloads``.

    python bench.py --gpus 1 --steps 50 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # the fp64 CPU oracle on the host cores

Prints ONE JSON line (rank 0).  With several GPUs the ranks hold independent sequences (no data-path
collective, weak scaling), or -- ``--shard kv-head`` -- each rank holds H_kv / N KV heads of the same
sequences (strong scaling; outputs stay sharded by query head, as a row-parallel output projection
takes them).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: batch, context, layers, G, Hq, Hkv, d, S, W, outliers, seed
    "llama3-8b-32k": dict(B=1, n=32768, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, outliers=True, seed=2),
    "llama3-8b-128k": dict(B=1, n=131072, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=4096, outliers=True, seed=4),
    "llama3-8b-32k-b16": dict(B=16, n=32768, L=32, G=4, Hq=32, Hkv=8, d=128, S=16, W=1024, outliers=False, seed=3),
    # serving mix: 32 sequences of seeded lengths in [4096, 65536], prefill of each, then decode steps
    "ragged-serving": dict(B=32, n=None, ragged=(4096, 65536), L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048,
                           outliers=False, seed=5, steps=16),
    # the 32K workload with head-wise blocks (Algorithm 1's output shape): every (layer, head) past layer 0
    # opens a new block with probability 0.3 (seeded), so about 70 % of the pairs share, the fraction
    # behind the paper's 35 % saving
    "llama3-8b-32k-headwise": dict(B=1, n=32768, L=32, G=1, Hq=32, Hkv=8, d=128, S=16, W=2048, outliers=True, seed=2,
                                   head_wise_new_block_p=0.3),
    "tiny": dict(B=1, n=512, L=4, G=2, Hq=8, Hkv=2, d=64, S=16, W=64, outliers=False, seed=0),
}
EXTRA_WORKLOADS = ("llama3-8b-128k", "llama3-8b-32k-b16", "ragged-serving")
METRIC = "pod_decode_attn_us_per_layer_step"
UNIT = "us/layer-step"
KERNEL_SOURCES = ("paper_2412_02252_b200/csrc/pod_decode.cu", "paper_2412_02252_b200/csrc/pod_common.h")
L2_FLUSH_BYTES = 512 << 20


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _bf16_peak(key="bf16_tflops"):
    fallback = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}[key]
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f).get(key, fallback))
    return fallback


def kernel_source_hash():
    """sha256 over the decode kernel's sources: a profile records it, so that counters taken from an
    older kernel are not quoted for the current one."""
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def profile_traffic(workload):
    """(DRAM bytes per launch of the split-K kernel from the committed ncu summary or None, where it came from).
    None when there is no capture for the workload or when the kernel has changed since the capture."""
    rel = os.path.join("profiles", f"pod_decode_splitk_{workload}.md")
    src = {"file": rel, "kernel_sources_now": kernel_source_hash()}
    traffic, recorded, commit = None, None, None
    try:
        with open(os.path.join(ROOT, rel)) as f:
            for line in f:
                if line.startswith("traffic_bytes_per_launch:"):
                    traffic = float(line.split(":")[1].split()[0])
                elif line.startswith("kernel_sources_sha256:"):
                    recorded = line.split(":")[1].split()[0]
                elif line.startswith("captured_at_commit:"):
                    commit = line.split(":")[1].split()[0]
    except OSError:
        src["note"] = "no ncu capture of this workload (12-41 GiB on the device is not a small case); see DESIGN.md"
        return None, src
    src.update(kernel_sources_at_capture=recorded, captured_at_commit=commit)
    if recorded != src["kernel_sources_now"]:
        src["note"] = "the decode kernel has changed since the counters were taken: traffic withheld"
        return None, src
    return traffic, src


def seq_lengths(w):
    if w.get("ragged"):
        from paper_2412_02252_b200 import synth
        lo, hi = w["ragged"]
        return synth.ragged_lengths(w["seed"], w["B"], lo, hi)
    return [w["n"]] * w["B"]


def block_map(w, heads=None):
    """lowest[l][h] of a workload: runs of G layers for every head, or the seeded head-wise map."""
    L, Hkv, G = w["L"], w["Hkv"], w["G"]
    p_new = w.get("head_wise_new_block_p")
    if p_new is None:
        low = [[l - l % G] * Hkv for l in range(L)]
    else:
        import random
        rng = random.Random(w["seed"] * 7919 + 13)
        low = [[0] * Hkv for _ in range(L)]
        for h in range(Hkv):
            for l in range(1, L):
                low[l][h] = l if rng.random() < p_new else low[l - 1][h]
    if heads is not None:
        low = [[row[h] for h in heads] for row in low]
    return low


def launch_bytes(low, l, *, lens, S, W, row, r):
    """Algorithmic bytes of the decode launch of layer l.  A head for which l is the lowest layer of its
    block reads one key and one value row per token and, when the block goes on, stores the distant
    logits (4 bytes per query head and distant token); a head whose block started lower reads the
    value rows, the proximal key rows and those logits."""
    total = 0.0
    L = len(low)
    for n in lens:
        n_p = min(n, S + W)
        n_d = n - n_p
        for h in range(len(low[l])):
            if low[l][h] == l:
                goes_on = l + 1 < L and low[l + 1][h] == l
                total += 2 * n * row + (n_d * r * 4 if goes_on else 0)
            else:
                total += n * row + n_p * row + n_d * r * 4
    return total


def layer_kind(low, l):
    """'lowest' if every head's block starts at l, 'sharing' if none does, else 'mixed'."""
    k = sum(low[l][h] == l for h in range(len(low[l])))
    return "lowest" if k == len(low[l]) else ("sharing" if k == 0 else "mixed")


def rank_seed(seed, rank):
    """Every rank decodes its own sequences: disjoint seeds, no data-path collective."""
    return seed + 1000 * rank


def reduce_max(x, dist, device):
    """Maximum of a per-rank timing over all ranks (identity without a process group)."""
    if dist is None:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_outputs(dist, local, gathered):
    """KV-head split, for a consumer that wants every head on every rank: one all-gather of the ranks'
    output slices.  local: this rank's [B][H_q / P][d]; gathered: [P][B][H_q / P][d], slice r = rank r's heads
    (query heads r * H_q / P onwards).  8 KiB per sequence and layer at the 8B shapes."""
    # as bytes (every backend moves uint8), the ranks' slices one after the other along the first dimension
    dist.all_gather_into_tensor(gathered.view(torch.uint8).flatten(0, 1), local.view(torch.uint8))
    return gathered


def heads_from_gathered(gathered):
    """[P][B][H_q / P][d] as gather_outputs leaves it -> [B][H_q][d] in the order of the unsplit call."""
    P, Bn, Hl, d = gathered.shape
    return gathered.permute(1, 0, 2, 3).reshape(Bn, P * Hl, d)


def aggregate(*, ms, steps, layers, batch_per_rank, world, shard="sequence"):
    """Whole-job figures from the slowest rank's time for `steps` steps.  Ranks that hold their own
    sequences (shard = "sequence") multiply the work: the job's time per layer-step is the rank's divided
    by the number of ranks, printed beside the rank's own.  Ranks that hold KV heads of the same sequences
    (shard = "kv-head") work on the same layer-steps: nothing is divided."""
    per_rank = ms * 1e3 / (steps * layers)
    if shard == "kv-head":
        return {"us_per_layer_step": per_rank, "per_rank_us_per_layer_step": per_rank,
                "decode_tokens_per_s": batch_per_rank / (ms * 1e-3 / steps)}
    return {"us_per_layer_step": per_rank / world, "per_rank_us_per_layer_step": per_rank,
            "decode_tokens_per_s": world * batch_per_rank / (ms * 1e-3 / steps)}


def med_min(xs):
    return None if not xs else {"median": round(statistics.median(xs), 3), "min": round(min(xs), 3), "n": len(xs)}


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        return self

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 6:
                    continue
                try:
                    sm.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[2:6]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------ one workload on this rank
class Runner:
    """Cache + resident step inputs of one workload on this rank, and the ways of timing its steps."""

    def __init__(self, name, w, *, B, synth, dev, local, seed, dist, heads=None, n_in=4, reserve_steps=0):
        self.name, self.w, self.B, self.synth, self.dev, self.local, self.dist = name, w, B, synth, dev, local, dist
        self.seed = seed
        self.heads = heads                                      # KV heads this rank holds (None = all)
        self.L, self.S, self.W, self.d = w["L"], w["S"], w["W"], w["d"]
        self.Hkv = w["Hkv"] if heads is None else len(heads)
        self.r = w["Hq"] // w["Hkv"]
        self.Hq = self.Hkv * self.r
        self.lens0 = seq_lengths(w)
        self.Bn = len(self.lens0)
        self.low_map = block_map(w, heads)
        self.head_wise = "head_wise_new_block_p" in w
        self.n_in = n_in
        self.reserve = reserve_steps
        self.stream = torch.cuda.current_stream().cuda_stream
        self.gathered = None                                    # [L][P][B][H_q / P][d] when the ranks' outputs are gathered
        self.launches = 0
        self.cache = None
        self.step_no = 0
        self._inputs()

    def _gen(self, tag, layer, b, p0, p1):
        return self.synth.gen_kv(self.seed, tag, layer, b, p0, p1, self.w["Hkv"], self.d, outliers=self.w["outliers"],
                                 heads=self.heads, device=self.dev)

    def _inputs(self):
        """per-step inputs, resident in HBM: [step][layer] -> k, v [B][Hkv][d], q [B][Hq][d]"""
        s_, L, Bn = self.synth, self.L, self.Bn
        self.ks = torch.stack([torch.stack([torch.stack([self._gen(s_.TAG_K, l, b, self.lens0[b] + s, self.lens0[b] + s + 1)[0]
                                                          for b in range(Bn)]) for l in range(L)]) for s in range(self.n_in)])
        self.vs = torch.stack([torch.stack([torch.stack([self._gen(s_.TAG_V, l, b, self.lens0[b] + s, self.lens0[b] + s + 1)[0]
                                                          for b in range(Bn)]) for l in range(L)]) for s in range(self.n_in)])
        q0 = 0 if self.heads is None else self.heads[0] * self.r
        self.qs = torch.stack([torch.stack([s_.gen_q(self.seed, l, s, Bn, self.w["Hq"], self.d, device=self.dev)[:, q0:q0 + self.Hq].contiguous()
                                            for l in range(L)]) for s in range(self.n_in)])
        self.outs = torch.empty(L, Bn, self.Hq, self.d, dtype=torch.bfloat16, device=self.dev)
        # raw device pointers, so that the timed loop is the C-ABI calls and nothing else
        self.kp = [[self.ks[i, l].data_ptr() for l in range(L)] for i in range(self.n_in)]
        self.vp = [[self.vs[i, l].data_ptr() for l in range(L)] for i in range(self.n_in)]
        self.qp = [[self.qs[i, l].data_ptr() for l in range(L)] for i in range(self.n_in)]
        self.op = [self.outs[l].data_ptr() for l in range(L)]

    def build(self, group=None):
        """Creates the cache (G = group, or the workload's blocks) and writes every sequence's context."""
        B, w = self.B, self.w
        G = w["G"] if group is None else group
        cfg = B.make_config(n_layers=self.L, n_q_heads=self.Hq, n_kv_heads=self.Hkv, head_dim=self.d, group_size=G,
                            n_sink=self.S, n_recent=self.W, batch=self.Bn, device=self.local)
        use_map = self.head_wise and group is None
        self.cache = B.PodCache(cfg, [n + self.reserve for n in self.lens0], lowest_layer=(self.low_map if use_map else None))
        self.G_now = G
        s_ = self.synth
        for l in range(self.L):
            for b in range(self.Bn):
                at = 0
                while at < self.lens0[b]:
                    t = min(16384, self.lens0[b] - at)
                    self.cache.write(l, b, self._gen(s_.TAG_K, l, b, at, at + t), self._gen(s_.TAG_V, l, b, at, at + t), t, self.stream)
                    at += t
        torch.cuda.synchronize()
        self.step_no = 0
        return self.cache

    def destroy(self):
        if self.cache is not None:
            self.cache.destroy()
            self.cache = None
            torch.cuda.empty_cache()

    def kinds(self):
        low = self.low_map if self.G_now == self.w["G"] else [[l - l % self.G_now] * self.Hkv for l in range(self.L)]
        return [layer_kind(low, l) for l in range(self.L)]

    # ---- steps -------------------------------------------------------------------------------
    def step(self, two_calls=False, events=None, flush=None):
        c, i = self.cache, self.step_no % self.n_in
        kpi, vpi, qpi, op, st = self.kp[i], self.vp[i], self.qp[i], self.op, self.stream
        if two_calls:
            for l in range(self.L):
                c.write(l, -1, kpi[l], vpi[l], 1, st)
                c.decode_attn(l, qpi[l], op[l], st)
            self.launches += self.L * (1 + c.last_launch()["n_kernels"])
        elif events is None:
            for l in range(self.L):
                c.append_decode_attn(l, kpi[l], vpi[l], qpi[l], op[l], st)
                if self.gathered is not None:       # every rank gets every head of this layer's output
                    gather_outputs(self.dist, self.outs[l], self.gathered[l])
            self.launches += self.L
        else:                                       # an event pair around every launch: the launches are serialised
            for l in range(self.L):
                if flush is not None:
                    flush.fill_(l & 1)              # a write larger than L2 between launches
                events[l][0].record()
                c.append_decode_attn(l, kpi[l], vpi[l], qpi[l], op[l], st)
                events[l][1].record()
        self.step_no += 1

    def barrier(self):
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            torch.cuda.synchronize()

    def region(self, steps, two_calls=False):
        """ms of exactly `steps` steps: CUDA events on the launching stream, barrier + synchronize on both sides."""
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        self.launches = 0
        t0.record()
        for _ in range(steps):
            self.step(two_calls)
        t1.record()
        self.barrier()
        return reduce_max(t0.elapsed_time(t1), self.dist, self.dev)

    def per_step(self, steps):
        """us per layer-step of each of `steps` steps (an event pair per step, steps back to back)."""
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        torch.cuda.synchronize()
        for a, b in evs:
            a.record()
            self.step()
            b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) * 1e3 / self.L for a, b in evs]

    def isolated(self, steps, flush=None):
        """us of single launches by kind: an event pair around each launch (which serialises them; with `flush`
        a write larger than L2 runs between launches)."""
        out = {}
        kinds = self.kinds()
        for _ in range(steps):
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(self.L)]
            self.step(events=evs, flush=flush)
            torch.cuda.synchronize()
            for l in range(self.L):
                out.setdefault(kinds[l], []).append(evs[l][0].elapsed_time(evs[l][1]) * 1e3)
        return out

    def pipelined(self, steps):
        """us from the end of the previous launch to the end of this one, by kind, inside back-to-back steps:
        from the library's launch trace (the GPU's own timer; events between launches would serialise them)."""
        n = steps * self.L
        buf = torch.zeros(2 * n, dtype=torch.int64, device=self.dev)
        self.cache.set_trace(buf, n)
        for _ in range(steps):
            self.step()
        torch.cuda.synchronize()
        got = self.cache.trace_count()
        self.cache.set_trace(None, 0)
        t = buf.view(n, 2).cpu().tolist()
        kinds = self.kinds()
        out, overlap = {}, {}
        for i in range(1, min(got, n)):
            k = kinds[i % self.L]
            out.setdefault(k, []).append((t[i][1] - t[i - 1][1]) / 1e3)
            overlap.setdefault(k, []).append((t[i - 1][1] - t[i][0]) / 1e3)
        return out, overlap


def measure(run, args, *, steps, warmup, regions, primary, hbm_peak, clocks_index, dist_world):
    """Times one workload: `regions` regions of `steps` steps (median = the figure), per-step events, single launches
    by kind (warm and after an L2 flush), the pipelined cost of a launch by kind, and the same kernels on a
    per-layer K+V cache (G = 1)."""
    B, w = run.B, run.w
    row, r = run.d * 2, run.r
    out = {}
    sampler = ClockSampler(clocks_index).start() if clocks_index is not None else None
    time.sleep(0.25 if sampler else 0)
    run.build()
    for _ in range(warmup):
        run.step()
    torch.cuda.synchronize()
    if run.cache.device_status() != B.POD_OK:
        raise SystemExit("bench.py: the decode kernel reported a device-side wait limit during warm-up")
    ms = [run.region(steps) for _ in range(regions)]
    n_launch = run.launches
    geo = run.cache.last_launch()
    ms_med = statistics.median(ms)
    out["regions_us_per_layer_step"] = [round(x * 1e3 / (steps * run.L * (1 if args.shard == "kv-head" else dist_world)), 3) for x in ms]
    n_mid = [n + warmup + regions * steps / 2.0 for n in run.lens0]         # lengths in the middle of the timed steps
    per_layer = [launch_bytes(run.low_map, l, lens=n_mid, S=run.S, W=run.W, row=row, r=r) for l in range(run.L)]
    alg = sum(per_layer) / run.L
    per_us = ms_med * 1e3 / (steps * run.L)                                 # this rank's us per launch
    achieved = alg / (per_us * 1e-6) / 1e9
    dense_bytes = sum(2 * n * run.Hkv * row for n in n_mid)
    kinds = run.kinds()
    by_kind = {k: sum(per_layer[l] for l in range(run.L) if kinds[l] == k) / max(1, kinds.count(k)) for k in set(kinds)}
    out.update({
        "us_per_layer_step": round(per_us, 3), "ms_per_step": round(ms_med / steps, 4), "steps": steps, "regions": regions,
        "launches_per_region": n_launch,
        "algorithmic_bytes_per_launch": int(alg), "algorithmic_bytes_by_kind": {k: int(v) for k, v in by_kind.items()},
        "achieved_gbs": round(achieved, 1), "frac": round(achieved / hbm_peak, 4), "frac_of_8TBs": round(achieved / 8000.0, 4),
        "dense_equivalent_gbs": round(dense_bytes / (per_us * 1e-6) / 1e9, 1),
        "context": run.cache.seq_len(0, 0) if run.Bn == 1 else {"min": min(run.lens0), "max": max(run.lens0), "sum": sum(run.lens0)},
        "batch": run.Bn, "split_tokens": geo["split_tokens"], "ctas": geo["n_ctas"],
        "step_reads_gib": round(run.L * alg / 2 ** 30, 2),
    })
    ps = run.per_step(max(steps, 50) if primary else steps)
    out["per_step_us_per_layer_step"] = med_min(ps)
    iso_steps = 4 if primary else 2
    warm = run.isolated(iso_steps)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=run.dev)
    cold = run.isolated(iso_steps, flush=flush)
    del flush
    pipe, overlap = run.pipelined(iso_steps)
    out["launch_kinds"] = {
        k: {"bytes": int(by_kind[k]),
            "isolated_us": med_min(warm.get(k, [])), "isolated_after_l2_flush_us": med_min(cold.get(k, [])),
            "pipelined_us": med_min(pipe.get(k, [])), "overlap_with_previous_us": med_min(overlap.get(k, []))}
        for k in sorted(set(kinds))}
    out["launch_kinds_note"] = ("isolated: CUDA events around one launch (events between launches serialise them; the second "
                                "figure has a %d MiB write between launches); pipelined: end of the previous launch to end of "
                                "this one inside back-to-back steps, from the library's launch trace on the GPU timer" % (L2_FLUSH_BYTES >> 20))
    if primary:
        ms_two = statistics.median([run.region(steps, two_calls=True) for _ in range(3)])
        out["two_call_us_per_layer_step"] = round(ms_two * 1e3 / (steps * run.L), 3)
    out["cache_bytes"] = {"pod_live": run.cache.bytes(B.POD_BYTES_LIVE), "dense_equiv": run.cache.bytes(B.POD_BYTES_DENSE_EQUIV)}
    out["cache_bytes"]["saving"] = round(1 - out["cache_bytes"]["pod_live"] / out["cache_bytes"]["dense_equiv"], 5)
    assert run.cache.device_status() == B.POD_OK
    out["clocks"] = sampler.stop() if sampler else None      # sampled during everything above
    return out, ms_med, n_launch


def dense_leg(run, steps, warmup, regions):
    """The same kernels on a cache in which every layer is its own block (a per-layer K+V cache)."""
    run.destroy()
    run.build(group=1)
    for _ in range(warmup):
        run.step()
    ms = statistics.median([run.region(steps) for _ in range(regions)])
    run.destroy()
    return round(ms * 1e3 / (steps * run.L), 3)


# ------------------------------------------------------------------------------ our arm
def run_ours(args):
    from paper_2412_02252_b200 import binding as B
    from paper_2412_02252_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the PoD library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    hbm_peak, peak_kind = _peaks()
    stream = torch.cuda.current_stream().cuda_stream

    w = dict(WORKLOADS[args.workload])
    Hq, Hkv, d, S, W, L = (w[k] for k in ("Hq", "Hkv", "d", "S", "W", "L"))
    heads = None
    seed = w["seed"]
    if world > 1 and args.shard == "kv-head":
        cfg_full = B.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, group_size=w["G"], n_sink=S,
                                 n_recent=W, batch=w["B"], device=local)
        local_cfg, kv0, _ = B.pod_shard_config(cfg_full, rank, world)       # raises if world does not divide H_kv
        heads = list(range(kv0, kv0 + local_cfg.n_kv_heads))
    elif world > 1:
        seed = rank_seed(seed, rank)
    elif args.one_shard_of > 1:
        # one GPU doing the work of one rank of a KV-head split (rank 0 of --one-shard-of ranks): what a rank's
        # launches cost, without the other ranks -- not a multi-GPU measurement
        cfg_full = B.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, group_size=w["G"], n_sink=S,
                                 n_recent=W, batch=w["B"], device=local)
        local_cfg, kv0, _ = B.pod_shard_config(cfg_full, 0, args.one_shard_of)
        heads = list(range(kv0, kv0 + local_cfg.n_kv_heads))

    if args.only == "prefill-attn":
        if rank == 0:
            print(json.dumps({"prefill_attn": time_prefill_attn(B, synth, w, seed, dev, stream, args)}), flush=True)
        return
    if args.only == "prefill-write":
        if rank == 0:
            print(json.dumps({"prefill_write": time_prefill_write(B, synth, w, seed, dev, local, stream)}), flush=True)
        return
    if args.only == "decode-steps":
        # warm-up and one region of the headline steps, nothing else: the command profilers are pointed at
        run = Runner(args.workload, w, B=B, synth=synth, dev=dev, local=local, seed=seed, dist=dist, heads=heads,
                     reserve_steps=args.warmup + args.steps + 8)
        run.build()
        for _ in range(args.warmup):
            run.step()
        ms = run.region(args.steps)
        assert run.cache.device_status() == B.POD_OK
        if rank == 0:
            print(json.dumps({"decode_steps": {"us_per_layer_step": round(ms * 1e3 / (args.steps * L), 3), "steps": args.steps,
                                               "launches": run.launches}}), flush=True)
        run.destroy()
        return

    steps = w.get("steps", args.steps)
    regions = max(1, args.regions)
    e2e_steps = max(3, min(steps, 20))
    reserve = args.warmup + regions * steps + max(steps, 50) + 3 * (steps + 3) + e2e_steps + 64
    run = Runner(args.workload, w, B=B, synth=synth, dev=dev, local=local, seed=seed, dist=dist, heads=heads, reserve_steps=reserve)
    if args.gate_tau is not None:
        raise SystemExit("bench.py: --gate-tau is timed by tests and DESIGN.md's table, not by this line")
    if args.gather_outputs:
        if not (world > 1 and args.shard == "kv-head"):
            raise SystemExit("bench.py: --gather-outputs goes with --shard kv-head on more than one GPU")
        run.gathered = torch.empty(L, world, run.Bn, run.Hq, d, dtype=torch.bfloat16, device=dev)
    res, ms, n_launch = measure(run, args, steps=steps, warmup=args.warmup, regions=regions, primary=True, hbm_peak=hbm_peak,
                                clocks_index=local if rank == 0 else None, dist_world=world)

    # ---- e2e: host buffers, H2D of k/v/q and D2H of the outputs inside the timed region -----------
    hk, hv, hq = (x.cpu().pin_memory() for x in (run.ks, run.vs, run.qs))
    dk, dv, dq = torch.empty_like(run.ks[0]), torch.empty_like(run.vs[0]), torch.empty_like(run.qs[0])
    hout = torch.empty(L, run.Bn, run.Hq, d, dtype=torch.bfloat16).pin_memory()
    dkp, dvp, dqp = ([x[l].data_ptr() for l in range(L)] for x in (dk, dv, dq))

    def e2e_step(s):
        """One step through the public call with host buffers: the step's k, v, q of every layer go up
        in three copies from pinned memory, one launch per layer, the outputs come back."""
        i = s % run.n_in
        dk.copy_(hk[i], non_blocking=True)
        dv.copy_(hv[i], non_blocking=True)
        dq.copy_(hq[i], non_blocking=True)
        for l in range(L):
            run.cache.append_decode_attn(l, dkp[l], dvp[l], dqp[l], run.op[l], stream)
        hout.copy_(run.outs, non_blocking=True)
        torch.cuda.current_stream().synchronize()      # the caller needs the outputs on the host

    for s in range(3):
        e2e_step(s)
    run.barrier()
    t0 = time.perf_counter()
    for s in range(e2e_steps):
        e2e_step(3 + s)
    torch.cuda.synchronize()
    e2e_ms = reduce_max((time.perf_counter() - t0) * 1e3, dist, dev)   # wall clock: the host waits for every step's output
    run.barrier()
    h2d = L * run.Bn * (2 * run.Hkv + run.Hq) * d * 2
    d2h = L * run.Bn * run.Hq * d * 2
    assert run.cache.device_status() == B.POD_OK
    run.destroy()

    dense_us = None
    if world == 1 and not args.no_dense:
        dense_us = dense_leg(run, steps, args.warmup, min(regions, 3))
    del run
    torch.cuda.empty_cache()

    prefill = time_prefill_write(B, synth, w, seed, dev, local, stream) if rank == 0 else None
    prefill_attn = time_prefill_attn(B, synth, w, seed, dev, stream, args) if rank == 0 and d == 128 else None

    # ---- the other configurations of the scope table, one after the other (each frees its cache) ----
    others = {}
    if world == 1 and not args.no_extra and args.workload == "llama3-8b-32k" and args.one_shard_of <= 1:
        for name in EXTRA_WORKLOADS:
            free_gib = torch.cuda.mem_get_info()[0] / 2 ** 30
            wx = dict(WORKLOADS[name])
            lens = seq_lengths(wx)
            need_gib = sum(lens) * wx["L"] * 2 * wx["Hkv"] * wx["d"] * 2 / 2 ** 30 * 1.05 + 2      # the G = 1 cache is the larger one
            if free_gib < need_gib:
                others[name] = {"skipped": "needs %.0f GiB of device memory, %.0f free" % (need_gib, free_gib)}
                continue
            sx = wx.get("steps", min(args.steps, 20))
            rx = max(1, min(args.regions, 5))
            rsv = 3 + rx * sx + sx + 8 + 32
            rr = Runner(name, wx, B=B, synth=synth, dev=dev, local=local, seed=wx["seed"], dist=None, reserve_steps=rsv)
            ox, _, _ = measure(rr, args, steps=sx, warmup=3, regions=rx, primary=False, hbm_peak=hbm_peak, clocks_index=local, dist_world=1)
            rr.destroy()
            ox["dense_kv_baseline_us_per_layer_step"] = None if args.no_dense else dense_leg(rr, sx, 3, min(rx, 3))
            ox["roofline_peak_gbs"] = hbm_peak
            tr, src = profile_traffic(name)
            ox["traffic"], ox["traffic_source"] = tr, src
            others[name] = ox
            del rr
            torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    agg = aggregate(ms=ms, steps=steps, layers=L, batch_per_rank=len(seq_lengths(w)), world=world, shard=args.shard)
    traffic, traffic_src = profile_traffic(args.workload)
    low_map = block_map(w)
    n_low_pairs = sum(low_map[l][h] == l for l in range(L) for h in range(Hkv))
    line = {
        "metric": METRIC, "value": round(agg["us_per_layer_step"], 3), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": args.warmup, "ms_per_step": res["ms_per_step"],
        "higher_is_better": False, "scaling": "strong" if (world > 1 and args.shard == "kv-head") else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch_per_gpu": res["batch"], "context": res["context"], "layers": L,
                   "group_size": w["G"], "q_heads": Hq, "kv_heads": Hkv, "head_dim": d, "n_sink": S, "n_recent": W,
                   "l2": "inputs larger than L2 (a step reads %.1f GiB)" % res["step_reads_gib"],
                   "blocks": ("head-wise, seeded" if "head_wise_new_block_p" in w else "runs of %d layers" % w["G"]) +
                             ": %d of %d (layer, KV head) pairs keep their own distant keys" % (n_low_pairs, L * Hkv),
                   "shard": args.shard if world > 1 else None,
                   "gather_outputs": bool(args.gather_outputs),
                   "split_tokens": res["split_tokens"], "ctas": res["ctas"],
                   "timing": "value = median of %d regions of %d steps, each bracketed by barrier + synchronize" % (regions, steps)},
        "per_rank_us_per_layer_step": round(agg["per_rank_us_per_layer_step"], 3),
        "decode_tokens_per_s": round(agg["decode_tokens_per_s"], 1),
        "regions_us_per_layer_step": res["regions_us_per_layer_step"],
        "per_step_us_per_layer_step": res["per_step_us_per_layer_step"],
        "hbm_gbs_step": round(L * res["algorithmic_bytes_per_launch"] / (res["ms_per_step"] * 1e-3) / 1e9, 1),
        "roofline": {"bound": "hbm", "achieved": res["achieved_gbs"], "peak": hbm_peak, "unit": "GB/s",
                     "frac": res["frac"], "traffic": traffic, "traffic_source": traffic_src, "peak_kind": peak_kind,
                     "kernel": "pod_decode_splitk_kernel (append + split-K + combine in one launch)",
                     "us_per_launch": res["us_per_layer_step"],
                     "algorithmic_bytes_per_launch": res["algorithmic_bytes_per_launch"],
                     "algorithmic_bytes_by_kind": res["algorithmic_bytes_by_kind"],
                     "frac_of_8TBs": res["frac_of_8TBs"],
                     "dense_equivalent_gbs": res["dense_equivalent_gbs"]},
        "launch_kinds": res["launch_kinds"], "launch_kinds_note": res["launch_kinds_note"],
        "e2e": {"value": round(e2e_ms * 1e3 / (e2e_steps * L * (1 if args.shard == "kv-head" else world)), 3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": n_launch,
        "clocks": res["clocks"],
        "cache_bytes": res["cache_bytes"],
        "workloads": others,
        "prefill_write": prefill,
        "prefill_attn": prefill_attn,
        "two_call_us_per_layer_step": res.get("two_call_us_per_layer_step"),
        "dense_kv_baseline_us_per_layer_step": dense_us,
    }
    if args.one_shard_of > 1:
        line["config"]["shard"] = "rank 0 of a %d-way KV-head split, alone on one GPU (%d of %d KV heads)" % (
            args.one_shard_of, len(heads), Hkv)
    if not args.no_cpu and world == 1 and "head_wise_new_block_p" not in w and not w.get("ragged") and args.one_shard_of <= 1:
        line["cpu_baseline"] = cpu_baseline(args.workload, budget_s=args.cpu_budget)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def time_prefill_write(B, synth, w, seed, dev, local, stream, reps=6):
    """pod_cache_write of one sequence's whole context (n tokens, one call per layer) into a
    two-layer cache with blocks of two layers: layer 0 keeps its distant keys, layer 1 drops them.
    Calls are issued back to back (each appends n more tokens) and timed with CUDA events."""
    Hq, Hkv, d, S, W = (w[k] for k in ("Hq", "Hkv", "d", "S", "W"))
    n = w["n"] or 32768
    T_ = min(n, 32768)
    cfg = B.make_config(n_layers=2, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, group_size=2,
                        n_sink=S, n_recent=W, batch=1, device=local)
    pc = B.PodCache(cfg, [T_ * (reps + 2)])
    k = synth.gen_kv(seed, synth.TAG_K, 0, 0, 0, T_, Hkv, d, outliers=w["outliers"], device=dev)
    v = synth.gen_kv(seed, synth.TAG_V, 0, 0, 0, T_, Hkv, d, outliers=w["outliers"], device=dev)
    out, row = {}, d * 2
    for l, name in ((0, "lowest_layer"), (1, "other_layer")):
        pc.write(l, 0, k, v, T_, stream)                      # fills the window; untimed
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            pc.write(l, 0, k, v, T_, stream)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / reps
        keeps = Hkv if l == 0 else 0                          # heads whose distant keys this layer keeps
        # read: every value row, the key rows that are kept (all for layer 0, the last W for layer 1),
        # and the W rows per head and kind that leave the ring; written: the same rows at their new places
        rows = T_ * Hkv + T_ * keeps + W * (Hkv - keeps) + W * (Hkv + keeps)
        out[name] = {"us": round(us, 2), "gbs": round(2 * rows * row / (us * 1e-6) / 1e9, 1)}
        # yardstick: a plain device-to-device copy of as many bytes, issued the same way (the copy rate the
        # roofline uses is that of much larger buffers; at this size a launch's ramp and tail weigh more)
        nb = rows * row
        srcs = [torch.empty(nb, dtype=torch.uint8, device=dev).fill_(i) for i in range(2)]
        dsts = [torch.empty(nb, dtype=torch.uint8, device=dev) for _ in range(reps)]
        dsts[0].copy_(srcs[0])
        torch.cuda.synchronize()
        e0.record()
        for i in range(reps):
            dsts[i].copy_(srcs[i % 2])
        e1.record()
        torch.cuda.synchronize()
        cus = e0.elapsed_time(e1) * 1e3 / reps
        out[name]["device_copy_same_bytes"] = {"us": round(cus, 2), "gbs": round(2 * nb / (cus * 1e-6) / 1e9, 1)}
        del srcs, dsts
    pc.destroy()
    out["tokens_per_call"] = T_
    out["note"] = "bytes read + written per call over the mean of back-to-back calls"
    return out


def time_prefill_attn(B, synth, w, seed, dev, stream, args, reps=4):
    """pod_prefill_attn over one sequence's whole context for one layer: once as the lowest layer of
    its block (plain causal attention) and once as a layer whose heads all take their distant logits
    from the lowest layer.  FLOPs counted: the causal half of the two products, 4 d per (query, key)
    pair and head; masked pairs inside a tile and the second pass over edge tiles are not counted."""
    Hq, Hkv, d, S, W = (w[k] for k in ("Hq", "Hkv", "d", "S", "W"))
    T_ = min(w["n"] or 32768, args.prefill_tokens)
    gen = lambda tag, layer, h: synth.gen_kv(seed, tag, layer, 0, 0, T_, h, d, outliers=w["outliers"] and tag != synth.TAG_Q, device=dev)
    q, k, v = gen(synth.TAG_Q, 1, Hq), gen(synth.TAG_K, 1, Hkv), gen(synth.TAG_V, 1, Hkv)
    ql, kl = gen(synth.TAG_Q, 0, Hq), gen(synth.TAG_K, 0, Hkv)
    o = torch.empty(T_, Hq, d, device=dev, dtype=torch.bfloat16)
    flops = 4.0 * d * Hq * (T_ * (T_ + 1) / 2)
    out = {}
    kinds = (("lowest_layer", False), ("sharing_layer", True))
    call = lambda share: B.pod_prefill_attn(q, k, v, o, n_sink=S, n_recent=W, q_low=ql if share else None,
                                            k_low=kl if share else None, stream=stream)
    for _, share in kinds:                                    # warm-up
        call(share)
    torch.cuda.synchronize()
    # The peak this leg is set against is a burst figure (a GEMM timed from an idle GPU, before the power cap
    # bites), so the leg starts the same way: idle for a moment, one untimed call to bring the clocks up, then
    # the timed calls.  The two kinds take turns, so that a drifting clock weighs on both alike.
    if not args.no_idle:
        time.sleep(1.5)
    call(False)
    evs = {name: [] for name, _ in kinds}
    for _ in range(reps):
        for name, share in kinds:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            call(share)
            e1.record()
            evs[name].append((e0, e1))
    torch.cuda.synchronize()
    for name, _ in kinds:
        times = [a.elapsed_time(b) for a, b in evs[name]]
        ms = sum(times) / reps
        out[name] = {"ms": round(ms, 3), "tflops": round(flops / ms / 1e9, 1), "ms_min": round(min(times), 3),
                     "tflops_best": round(flops / min(times) / 1e9, 1)}
    # the same call back to back for over a second: what the kernel holds once the power cap has settled,
    # against the GEMM figure taken the same way
    if args.prefill_sustained_calls > 0 and T_ >= 16384:
        n_sus = args.prefill_sustained_calls
        sampler = ClockSampler(dev.index or 0).start()
        evs_s = []
        for i in range(n_sus):
            tail = i >= n_sus - max(4, n_sus // 4)
            if tail:
                e0 = torch.cuda.Event(enable_timing=True)
                e0.record()
            call(False)
            if tail:
                e1 = torch.cuda.Event(enable_timing=True)
                e1.record()
                evs_s.append((e0, e1))
        torch.cuda.synchronize()
        clocks = sampler.stop()
        ms_s = statistics.mean(a.elapsed_time(b) for a, b in evs_s)
        peak_s = _bf16_peak("bf16_tflops_sustained")
        out["sustained"] = {"calls": n_sus, "timed": "mean of the last %d calls" % len(evs_s), "ms": round(ms_s, 3),
                            "tflops": round(flops / ms_s / 1e9, 1), "peak_tflops_sustained": peak_s,
                            "frac_of_sustained": round(flops / ms_s / 1e9 / peak_s, 4), "clocks": clocks}
    assert B.pod_prefill_status() == 0
    out["tokens"] = T_
    out["peak_tflops"] = _bf16_peak()
    out["roofline"] = {"bound": "tensor", "achieved": out["lowest_layer"]["tflops"], "peak": out["peak_tflops"],
                       "unit": "TFLOP/s", "frac": round(out["lowest_layer"]["tflops"] / out["peak_tflops"], 4),
                       "frac_sharing_layer": round(out["sharing_layer"]["tflops"] / out["peak_tflops"], 4)}
    out["note"] = ("causal FLOPs (2 products x 2 d per visible pair) over the mean of the calls of a kind (the kinds alternate, "
                   "started from an idle GPU like the burst peak they are set against); peak = measured cuBLAS bf16 burst")
    return out


# ------------------------------------------------------------------------------ CPU oracle legs
def _oracle_block_inputs(workload, block=0, n=None):
    """fp64 history of one block of layers for sequence 0 (host), and the step's queries."""
    from paper_2412_02252_b200 import synth
    w = WORKLOADS[workload]
    n = w["n"] if n is None else n
    G, Hkv, d, Hq = w["G"], w["Hkv"], w["d"], w["Hq"]
    layers = list(range(block * G, min(w["L"], (block + 1) * G)))
    K = torch.stack([synth.gen_kv(w["seed"], synth.TAG_K, l, 0, 0, n, Hkv, d, outliers=w["outliers"]) for l in layers])
    V = torch.stack([synth.gen_kv(w["seed"], synth.TAG_V, l, 0, 0, n, Hkv, d, outliers=w["outliers"]) for l in layers])
    q = torch.stack([synth.gen_q(w["seed"], l, 0, w["B"], Hq, d)[0] for l in layers])
    return K.double().numpy(), V.double().numpy(), q.double().numpy(), layers


def _oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        ts = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(ts) if ts else 1
    except Exception:
        return 1


def cpu_baseline(workload, budget_s=15.0):
    """The fp64 oracle, as it stands, on a bounded sample: whole layer-steps (all query heads of
    one sequence) of the first block of layers, repeated until the budget is used."""
    from oracle import pod_oracle as O
    w = WORKLOADS[workload]
    K, V, q, layers = _oracle_block_inputs(workload)
    done, t_used = 0, 0.0
    while t_used < budget_s and done < 64:
        li = done % len(layers)
        t0 = time.perf_counter()
        O.pod_decode_layer(q, K, V, li, group_size=w["G"], n_s=w["S"], n_r=w["W"])
        t_used += time.perf_counter() - t0
        done += 1
    return {"value": round(t_used * 1e6 / done / 1.0, 1), "unit": UNIT, "cores": _oracle_threads(),
            "host_cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{done} layer-steps (layers {layers}, all {w['Hq']} query heads, 1 sequence of "
                      f"{w['n']} tokens) of the {workload} workload; batch scales linearly"}


def run_reference(args):
    """The reference arm of this build is the fp64 CPU oracle (the paper ships no code)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import pod_oracle as O
    w = WORKLOADS[args.workload]
    K, V, q, layers = _oracle_block_inputs(args.workload)
    steps = max(1, min(args.steps, 8))
    warm = max(0, min(args.warmup, 1))

    def one(i):
        O.pod_decode_layer(q, K, V, i % len(layers), group_size=w["G"], n_s=w["S"], n_r=w["W"])

    for i in range(warm):
        one(i)
    t0 = time.perf_counter()
    for i in range(steps):
        one(i)
    dt = time.perf_counter() - t0
    us = dt * 1e6 / steps * w["B"]
    sample = (f"each step = one layer-step of sequence 0 (all {w['Hq']} query heads, {w['n']} tokens), "
              f"scaled by batch {w['B']}; {steps} steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(us, 1), "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": warm,
        "ms_per_step": round(dt * 1e3 / steps, 3), "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload},
        "cpu_baseline": {"value": round(us, 1), "unit": UNIT, "kind": "oracle", "cores": _oracle_threads(),
                         "host_cores": os.cpu_count(), "sample": sample},
        "e2e": {"value": round(us, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--regions", type=int, default=5, help="timed regions of --steps steps; the figure is their median")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3-8b-32k", choices=sorted(WORKLOADS))
    ap.add_argument("--shard", default="sequence", choices=["sequence", "kv-head"],
                    help="with several GPUs: independent sequences per rank, or H_kv / N KV heads of the same sequences per rank")
    ap.add_argument("--gather-outputs", action="store_true",
                    help="with --shard kv-head: all-gather every layer's output slices (NCCL) inside the timed steps, "
                         "for a consumer that needs all heads on every rank; default: outputs stay sharded")
    ap.add_argument("--one-shard-of", type=int, default=1,
                    help="on one GPU: run rank 0's share of a KV-head split over this many ranks (what one rank's launches cost)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense-KV baseline legs")
    ap.add_argument("--no-extra", action="store_true", help="skip the 128K, batch-16 and ragged workloads")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--gate-tau", type=float, default=None, help=argparse.SUPPRESS)
    ap.add_argument("--prefill-tokens", type=int, default=32768,
                    help="positions of the prefill-attention leg (capped at the workload's context)")
    ap.add_argument("--prefill-sustained-calls", type=int, default=150,
                    help="back-to-back calls of the prefill-attention leg's sustained figure (0 = skip it)")
    ap.add_argument("--no-idle", action="store_true", help="prefill-attention leg: do not idle before the timed calls")
    ap.add_argument("--only", default=None, choices=["prefill-attn", "prefill-write", "decode-steps"],
                    help="run one side leg alone and print its object (for profiling)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
