"""Host arithmetic of bench.py that the reported roofline rests on (no GPU): algorithmic bytes per launch against
figures worked out by hand from the per-token byte counts, the kinds of layers, and the rule that DRAM traffic from
a profile is only quoted for the kernel sources it was captured with."""
import json
import os

import bench


def test_launch_bytes_at_the_8b_shapes():
    # 32 query / 8 KV heads, d = 128: a row is 256 B; per token a lowest layer reads 8 key + 8 value rows = 4096 B
    # and stores 32 x 4 B of logits per distant token; a sharing layer reads 2048 B of values per token, 2048 B of
    # keys per proximal token and 128 B of logits per distant token.
    S, W, row, r, Hkv = 16, 2048, 256, 4, 8
    n = 32768 + 3
    n_p, n_d = S + W, n - S - W
    low = [[l - l % 2] * Hkv for l in range(4)]
    lowest = bench.launch_bytes(low, 0, lens=[n], S=S, W=W, row=row, r=r)
    sharing = bench.launch_bytes(low, 1, lens=[n], S=S, W=W, row=row, r=r)
    assert lowest == n * 4096 + n_d * 128
    assert sharing == n * 2048 + n_p * 2048 + n_d * 128
    # G = 1: every layer is a block of its own, nothing is stored
    dense = [[l] * Hkv for l in range(4)]
    assert bench.launch_bytes(dense, 2, lens=[n], S=S, W=W, row=row, r=r) == n * 4096
    # the last layer of the model cannot be followed by a sharing layer: no logits stored
    odd = [[0] * Hkv, [0] * Hkv, [2] * Hkv]
    assert bench.launch_bytes(odd, 2, lens=[n], S=S, W=W, row=row, r=r) == n * 4096
    # a context inside the window has no distant token; a batch adds up
    assert bench.launch_bytes(low, 1, lens=[100, n], S=S, W=W, row=row, r=r) == 100 * 4096 + sharing
    assert [bench.layer_kind(low, l) for l in range(4)] == ["lowest", "sharing", "lowest", "sharing"]
    assert bench.layer_kind([[0, 0], [0, 1]], 1) == "mixed"


def test_workload_table_matches_the_scope_table():
    w = bench.WORKLOADS
    for name, (Bn, G, n, W) in {"llama3-8b-32k": (1, 2, 32768, 2048), "llama3-8b-128k": (1, 2, 131072, 4096),
                                "llama3-8b-32k-b16": (16, 4, 32768, 1024)}.items():
        assert (w[name]["B"], w[name]["G"], w[name]["n"], w[name]["W"]) == (Bn, G, n, W), name
        assert (w[name]["L"], w[name]["Hq"], w[name]["Hkv"], w[name]["d"], w[name]["S"]) == (32, 32, 8, 128, 16), name
    lens = bench.seq_lengths(w["ragged-serving"])
    assert len(lens) == 32 and min(lens) >= 4096 and max(lens) <= 65536
    assert lens == bench.seq_lengths(w["ragged-serving"])                   # seeded: the same draw every time


def test_traffic_is_withheld_when_the_kernel_changed(tmp_path, monkeypatch):
    traffic, src = bench.profile_traffic("llama3-8b-32k")
    assert src["file"] == os.path.join("profiles", "pod_decode_splitk_llama3-8b-32k.md")
    if traffic is not None:                                                 # the committed capture is of these sources
        assert src["kernel_sources_at_capture"] == src["kernel_sources_now"] and traffic > 50e6
    # a workload without a capture
    none, src2 = bench.profile_traffic("llama3-8b-128k")
    assert none is None and "no ncu capture" in src2["note"]
    # a capture of other sources: the figure is not quoted
    prof = tmp_path / "profiles"
    prof.mkdir()
    (prof / "pod_decode_splitk_llama3-8b-32k.md").write_text(
        "captured_at_commit: abc1234\nkernel_sources_sha256: 0000000000000000\ntraffic_bytes_per_launch: 1.0e8\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "kernel_source_hash", lambda: "1111111111111111")
    stale, src3 = bench.profile_traffic("llama3-8b-32k")
    assert stale is None and "changed" in src3["note"] and src3["captured_at_commit"] == "abc1234"
    monkeypatch.setattr(bench, "kernel_source_hash", lambda: "0000000000000000")
    fresh, _ = bench.profile_traffic("llama3-8b-32k")
    assert fresh == 1.0e8
    json.dumps(src3)                                                        # goes into the JSON line as it is
