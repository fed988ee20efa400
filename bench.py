#!/usr/bin/env python
"""Benchmark of the PoD decode hot path (cache append + decode attention for every layer).

One "step" is one decode step of the whole model's attention: for each layer, append the new
token's K/V to the PoD cache and attend over it (``pod_append_decode_attn``: the work of
``pod_cache_write`` + ``pod_decode_attn`` in one launch; the two-call form is timed beside it).  The workload
is the LLaMA-3-8B-shaped single-sequence decode at 32K context (32 layers, G = 2, 32/8 heads,
d = 128, S = 16, W = 2048, seeded synthetic bf16 K/V with outlier channels).

    python bench.py --gpus 1 --steps 50 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # the fp64 CPU oracle on the host cores

Prints ONE JSON line (rank 0).  Ranks hold independent sequences (no data-path collective):
weak scaling.
"""
from __future__ import annotations

import argparse
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
    # name: (batch, context, layers, G, Hq, Hkv, d, S, W, outliers, seed)
    "llama3-8b-32k": dict(B=1, n=32768, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=2048, outliers=True, seed=2),
    "llama3-8b-128k": dict(B=1, n=131072, L=32, G=2, Hq=32, Hkv=8, d=128, S=16, W=4096, outliers=True, seed=4),
    "llama3-8b-32k-b16": dict(B=16, n=32768, L=32, G=4, Hq=32, Hkv=8, d=128, S=16, W=1024, outliers=False, seed=3),
    # the 32K workload with head-wise blocks (Algorithm 1's output shape): every (layer, head) past layer 0
    # opens a new block with probability 0.3 (seeded), so about 70 % of the pairs share, the fraction
    # behind the paper's 35 % saving
    "llama3-8b-32k-headwise": dict(B=1, n=32768, L=32, G=1, Hq=32, Hkv=8, d=128, S=16, W=2048, outliers=True, seed=2,
                                   head_wise_new_block_p=0.3),
    "tiny": dict(B=1, n=512, L=4, G=2, Hq=8, Hkv=2, d=64, S=16, W=64, outliers=False, seed=0),
}
METRIC = "pod_decode_attn_us_per_layer_step"
UNIT = "us/layer-step"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _bf16_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f).get("bf16_tflops", 1590.0))
    return 1590.0


def _profile_traffic(workload):
    """DRAM bytes per launch of the split-K kernel from the committed ncu summary, or None."""
    path = os.path.join(ROOT, "profiles", f"pod_decode_splitk_{workload}.md")
    try:
        with open(path) as f:
            for line in f:
                if line.startswith("traffic_bytes_per_launch:"):
                    return float(line.split(":")[1].split()[0])
    except OSError:
        pass
    return None


def block_map(w):
    """lowest[l][h] of a workload: runs of G layers for every head, or the seeded head-wise map."""
    L, Hkv, G = w["L"], w["Hkv"], w["G"]
    p_new = w.get("head_wise_new_block_p")
    if p_new is None:
        return [[l - l % G] * Hkv for l in range(L)]
    import random
    rng = random.Random(w["seed"] * 7919 + 13)
    low = [[0] * Hkv for _ in range(L)]
    for h in range(Hkv):
        for l in range(1, L):
            low[l][h] = l if rng.random() < p_new else low[l - 1][h]
    return low


def launch_bytes(low, l, *, n, n_p, n_d, row, r, batch):
    """Algorithmic bytes of the decode launch of layer l.  A head for which l is the lowest layer of its
    block reads one key and one value row per token and, when the block goes on, stores the distant
    logits (4 bytes per query head and distant token); a head whose block started lower reads the
    value rows, the proximal key rows and those logits."""
    total = 0.0
    L = len(low)
    for h in range(len(low[l])):
        if low[l][h] == l:
            goes_on = l + 1 < L and low[l + 1][h] == l
            total += 2 * n * row + (n_d * r * 4 if goes_on else 0)
        else:
            total += n * row + n_p * row + n_d * r * 4
    return batch * total


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


def aggregate(*, ms, steps, layers, batch_per_rank, world):
    """Whole-job figures from the slowest rank's time for `steps` steps."""
    return {"us_per_layer_step": ms * 1e3 / (steps * layers * world),
            "decode_tokens_per_s": world * batch_per_rank / (ms * 1e-3 / steps)}


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

    w = dict(WORKLOADS[args.workload])
    Bn, n, L, G, Hq, Hkv, d, S, W = (w[k] for k in ("B", "n", "L", "G", "Hq", "Hkv", "d", "S", "W"))
    seed = rank_seed(w["seed"], rank)
    low_map = block_map(w)
    head_wise = "head_wise_new_block_p" in w
    total_steps = args.warmup + args.steps
    e2e_steps = max(3, min(args.steps, 20))
    extra = 2 * total_steps + 2 * (e2e_steps + 3) + 12    # headroom for every timed pass
    dev = torch.device("cuda", local)
    stream = torch.cuda.current_stream().cuda_stream

    def time_prefill_write(reps=6):
        """pod_cache_write of one sequence's whole context (n tokens, one call per layer) into a
        two-layer cache with blocks of two layers: layer 0 keeps its distant keys, layer 1 drops them.
        Calls are issued back to back (each appends n more tokens) and timed with CUDA events."""
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
        pc.destroy()
        out["tokens_per_call"] = T_
        out["note"] = "bytes read + written per call over the mean of back-to-back calls"
        return out

    def time_prefill_attn(reps=4):
        """pod_prefill_attn over one sequence's whole context for one layer: once as the lowest layer of
        its block (plain causal attention) and once as a layer whose heads all take their distant logits
        from the lowest layer.  FLOPs counted: the causal half of the two products, 4 d per (query, key)
        pair and head; masked pairs inside a tile and the second pass over edge tiles are not counted."""
        T_ = min(n, args.prefill_tokens)
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
        # the two kinds take turns, so that a drifting clock (the power cap) weighs on both alike
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
            ms = sum(a.elapsed_time(b) for a, b in evs[name]) / reps
            out[name] = {"ms": round(ms, 3), "tflops": round(flops / ms / 1e9, 1)}
        assert B.pod_prefill_status() == 0
        out["tokens"] = T_
        out["peak_tflops"] = _bf16_peak()
        out["roofline"] = {"bound": "tensor", "achieved": out["lowest_layer"]["tflops"], "peak": out["peak_tflops"],
                           "unit": "TFLOP/s", "frac": round(out["lowest_layer"]["tflops"] / out["peak_tflops"], 4),
                           "frac_sharing_layer": round(out["sharing_layer"]["tflops"] / out["peak_tflops"], 4)}
        out["note"] = "causal FLOPs (2 products x 2 d per visible pair) over the mean of the calls of a kind (the kinds alternate); peak = measured cuBLAS bf16 burst"
        return out

    if args.only == "prefill-attn":
        if rank == 0:
            print(json.dumps({"prefill_attn": time_prefill_attn()}), flush=True)
        return

    def build_cache(group, use_map=False):
        cfg = B.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, group_size=group,
                            n_sink=S, n_recent=W, batch=Bn, device=local)
        cache = B.PodCache(cfg, [n + extra] * Bn, lowest_layer=(low_map if use_map else None))
        for l in range(L):
            for b in range(Bn):
                at = 0
                while at < n - 1:
                    t = min(8192, n - 1 - at)
                    k = synth.gen_kv(seed, synth.TAG_K, l, b, at, at + t, Hkv, d, outliers=w["outliers"], device=dev)
                    v = synth.gen_kv(seed, synth.TAG_V, l, b, at, at + t, Hkv, d, outliers=w["outliers"], device=dev)
                    cache.write(l, b, k, v, t, stream)
                    at += t
        torch.cuda.synchronize()
        return cache

    # per-step inputs, resident in HBM: [step][layer] -> k, v [B][Hkv][d], q [B][Hq][d]
    n_in = 8
    def step_inputs(device):
        ks = torch.stack([torch.stack([torch.stack([
            synth.gen_kv(seed, synth.TAG_K, l, b, n - 1 + s, n + s, Hkv, d, outliers=w["outliers"], device=device)[0]
            for b in range(Bn)]) for l in range(L)]) for s in range(n_in)])
        vs = torch.stack([torch.stack([torch.stack([
            synth.gen_kv(seed, synth.TAG_V, l, b, n - 1 + s, n + s, Hkv, d, outliers=w["outliers"], device=device)[0]
            for b in range(Bn)]) for l in range(L)]) for s in range(n_in)])
        qs = torch.stack([torch.stack([synth.gen_q(seed, l, s, Bn, Hq, d, device=device) for l in range(L)])
                          for s in range(n_in)])
        return ks, vs, qs

    ks, vs, qs = step_inputs(dev)
    outs = torch.empty(L, Bn, Hq, d, dtype=torch.bfloat16, device=dev)
    launches = [0]
    # raw device pointers, so that the timed loop is the C-ABI calls and nothing else
    kp = [[ks[i, l].data_ptr() for l in range(L)] for i in range(n_in)]
    vp = [[vs[i, l].data_ptr() for l in range(L)] for i in range(n_in)]
    qp = [[qs[i, l].data_ptr() for l in range(L)] for i in range(n_in)]
    op = [outs[l].data_ptr() for l in range(L)]

    def step(cache, s, two_calls=False):
        i = s % n_in
        kpi, vpi, qpi = kp[i], vp[i], qp[i]
        if two_calls:
            for l in range(L):
                cache.write(l, -1, kpi[l], vpi[l], 1, stream)
                cache.decode_attn(l, qpi[l], op[l], stream)
            launches[0] += L * (1 + cache.last_launch()["n_kernels"])
        else:
            for l in range(L):
                cache.append_decode_attn(l, kpi[l], vpi[l], qpi[l], op[l], stream)
            launches[0] += launches_per_step

    launches_per_step = L          # one launch per layer; set after the first step if the gate adds launches

    def count_launches_per_step(cache):
        """Kernels one step launches (a gated layer is two launches), counted on one untimed step."""
        i, total = 0, 0
        for l in range(L):
            cache.append_decode_attn(l, kp[i][l], vp[i][l], qp[i][l], op[l], stream)
            total += cache.last_launch()["n_kernels"]
        return total

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(cache, steps, warmup, first_step, two_calls=False):
        """ms for `steps` steps, CUDA events on the launching stream around the whole region."""
        for s in range(warmup):
            step(cache, first_step + s, two_calls)
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        # a kernel whose bounded waits gave up in the warm-up would make every timed launch last seconds: stop here
        if cache.device_status() != B.POD_OK:
            raise SystemExit("bench.py: the decode kernel reported a device-side wait limit during warm-up")
        launches[0] = 0
        t0.record()
        for s in range(steps):
            step(cache, first_step + warmup + s, two_calls)
        t1.record()
        barrier()
        return t0.elapsed_time(t1)

    def rmax(x):
        return reduce_max(x, dist, dev)

    cache = build_cache(G, use_map=head_wise)
    if args.gate_tau is not None:
        cache.set_gate_threshold(args.gate_tau)
        launches_per_step = count_launches_per_step(cache)
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    # ---- headline: K steps, device-resident inputs ------------------------------------------------
    ms = timed(cache, args.steps, args.warmup, 0)
    n_launch = launches[0]
    ms = rmax(ms)
    # ---- the same steps as two calls per layer (pod_cache_write, then pod_decode_attn) -----------
    ms_two = rmax(timed(cache, args.steps, 3, total_steps, two_calls=True))
    clocks = sampler.stop() if sampler else None
    geo = cache.last_launch()
    # ---- e2e: host buffers, H2D of k/v/q and D2H of the outputs inside the timed region -----------
    hk, hv, hq = (x.cpu().pin_memory() for x in (ks, vs, qs))
    dk, dv, dq = torch.empty_like(ks[0]), torch.empty_like(vs[0]), torch.empty_like(qs[0])
    hout = torch.empty(L, Bn, Hq, d, dtype=torch.bfloat16).pin_memory()

    dkp = [dk[l].data_ptr() for l in range(L)]
    dvp = [dv[l].data_ptr() for l in range(L)]
    dqp = [dq[l].data_ptr() for l in range(L)]

    def e2e_step(s):
        """One step through the public call with host buffers: the step's k, v, q of every layer go up
        in three copies from pinned memory, one launch per layer, the outputs come back."""
        i = s % n_in
        dk.copy_(hk[i], non_blocking=True)
        dv.copy_(hv[i], non_blocking=True)
        dq.copy_(hq[i], non_blocking=True)
        for l in range(L):
            cache.append_decode_attn(l, dkp[l], dvp[l], dqp[l], op[l], stream)
        hout.copy_(outs, non_blocking=True)
        torch.cuda.current_stream().synchronize()      # the caller needs the outputs on the host

    for s in range(3):
        e2e_step(s)
    barrier()
    t0 = time.perf_counter()
    for s in range(e2e_steps):
        e2e_step(3 + s)
    torch.cuda.synchronize()
    e2e_ms = rmax((time.perf_counter() - t0) * 1e3)   # wall clock: the host waits for every step's output
    barrier()
    h2d = L * Bn * (2 * Hkv + Hq) * d * 2
    d2h = L * Bn * Hq * d * 2
    live = cache.bytes(B.POD_BYTES_LIVE)
    dense_equiv = cache.bytes(B.POD_BYTES_DENSE_EQUIV)
    n_now = cache.seq_len(0, 0)
    assert cache.device_status() == B.POD_OK
    cache.destroy()
    del cache
    torch.cuda.empty_cache()

    prefill = time_prefill_write() if rank == 0 else None
    prefill_attn = time_prefill_attn() if rank == 0 and d == 128 else None
    # ---- dense-KV baseline: the same kernels with every layer its own block (G = 1) ---------------
    dense_us = None
    if world == 1 and not args.no_dense:
        dcache = build_cache(1)
        dms = timed(dcache, args.steps, args.warmup, 0)
        dense_us = dms * 1e3 / (args.steps * L)
        dcache.destroy()
        del dcache

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    agg = aggregate(ms=ms, steps=args.steps, layers=L, batch_per_rank=Bn, world=world)
    us_layer = agg["us_per_layer_step"]
    hbm_peak, peak_kind = _peaks()
    n_avg = n + args.warmup + args.steps / 2.0
    row = d * 2
    n_p = min(n_avg, S + W)
    n_d = n_avg - n_p
    per_layer = [launch_bytes(low_map, l, n=n_avg, n_p=n_p, n_d=n_d, row=row, r=Hq // Hkv, batch=Bn) for l in range(L)]
    alg_bytes = sum(per_layer) / L
    n_low_pairs = sum(low_map[l][h] == l for l in range(L) for h in range(Hkv))
    dense_bytes = Bn * 2 * n_avg * Hkv * row              # what a per-layer K+V cache would read
    # the timed region holds nothing but launches of the one kernel: its average duration
    per_us = ms * 1e3 / n_launch
    achieved = alg_bytes / (per_us * 1e-6) / 1e9
    traffic = _profile_traffic(args.workload)
    line = {
        "metric": METRIC, "value": round(us_layer, 3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4),
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "batch_per_gpu": Bn, "context": n_now, "layers": L,
                   "group_size": G, "q_heads": Hq, "kv_heads": Hkv, "head_dim": d, "n_sink": S,
                   "n_recent": W, "l2": "inputs larger than L2 (a step reads %.1f GiB)" % (L * alg_bytes / 2**30),
                   "blocks": ("head-wise, seeded" if head_wise else "runs of %d layers" % G) +
                             ": %d of %d (layer, KV head) pairs keep their own distant keys" % (n_low_pairs, L * Hkv),
                   "gate_tau": args.gate_tau,
                   "split_tokens": geo["split_tokens"], "ctas": geo["n_ctas"]},
        "decode_tokens_per_s": round(agg["decode_tokens_per_s"], 1),
        "hbm_gbs_step": round(L * alg_bytes / (ms * 1e-3 / args.steps) / 1e9, 1),
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": hbm_peak, "unit": "GB/s",
                     "frac": round(achieved / hbm_peak, 4), "traffic": traffic, "peak_kind": peak_kind,
                     "kernel": "pod_decode_splitk_kernel (append + split-K + combine in one launch)",
                     "us_per_launch": round(per_us, 3),
                     "algorithmic_bytes_per_launch": int(alg_bytes),
                     "algorithmic_bytes_max_launch": int(max(per_layer)),
                     "algorithmic_bytes_min_launch": int(min(per_layer)),
                     "frac_of_8TBs": round(achieved / 8000.0, 4),
                     "dense_equivalent_gbs": round(dense_bytes / (per_us * 1e-6) / 1e9, 1)},
        "e2e": {"value": round(e2e_ms * 1e3 / (e2e_steps * L * world), 3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": n_launch,
        "clocks": clocks,
        "cache_bytes": {"pod_live": live, "dense_equiv": dense_equiv, "saving": round(1 - live / dense_equiv, 5)},
        "prefill_write": prefill,
        "prefill_attn": prefill_attn,
        "two_call_us_per_layer_step": round(ms_two * 1e3 / (args.steps * L * world), 3),
        "dense_kv_baseline_us_per_layer_step": None if dense_us is None else round(dense_us, 3),
    }
    if not args.no_cpu and world == 1 and not head_wise:
        line["cpu_baseline"] = cpu_baseline(args.workload, budget_s=args.cpu_budget)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


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
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3-8b-32k", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense-KV baseline leg")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--gate-tau", type=float, default=None,
                    help="gate threshold of the distant-skip approximation (default: off, exact attention)")
    ap.add_argument("--prefill-tokens", type=int, default=32768,
                    help="positions of the prefill-attention leg (capped at the workload's context)")
    ap.add_argument("--only", default=None, choices=["prefill-attn"],
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
