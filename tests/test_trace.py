"""The trace tool: span formatting / summary on the CPU, and one traced decode on the GPU (in a process of its own,
because a process holds either the product library or the traced build)."""
import json
import os
import subprocess
import sys

import pytest

from paper_2608_11688_b200 import trace

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_summary_and_format_of_hand_made_spans():
    spans = [(1, 1000, 6000), (3, 2000, 8000), (4, 8000, 12000), (5, 12500, 25000), (1, 25000, 30000)]
    s = trace.summarize(spans)
    assert s[trace.KERNEL_NAMES[1]] == {"launches": 2, "mean_us": 5.0, "max_us": 5.0}
    assert s[trace.KERNEL_NAMES[5]]["mean_us"] == 12.5
    # union of the spans: [1000, 12000] + [12500, 30000] = 28500 of 29000 ns
    assert s["_all"]["spans"] == 5 and abs(s["_all"]["wall_us"] - 29.0) < 1e-9
    assert abs(s["_all"]["busy_fraction"] - 28500 / 29000) < 1e-12
    text = trace.format_spans(spans, limit=4).splitlines()
    assert len(text) == 1 + 4 + 1 and text[-1].startswith("... 1 more")
    gate = text[3].split()
    assert gate[0] == "gate" and float(gate[1]) == 7.0 and float(gate[3]) == 4.0 and float(gate[4]) == 0.0
    assert float(text[4].split()[-1]) == 0.5     # the FFN starts 0.5 us after the gate's end
    assert trace.format_spans([]) == "(no spans recorded)"
    assert trace.summarize([]) == {}


def test_persistent_kernel_phase_summary_of_hand_made_stamps():
    import numpy as np
    st = np.zeros((2, 4, 16), np.int64)
    for cta in range(2):
        for l in range(4):
            t0 = 1000 + 20000 * l + 100 * cta
            st[cta, l, 0] = t0
            st[cta, l, 5] = t0 + 4000 + 1000 * cta          # gate logits complete: 4 and 5 us
            st[cta, l, 8] = t0 + 15000
    ph = trace.decode_phase_medians(st)
    assert ph[trace.DECODE_STAMPS[5]] == 4.5 and ph[trace.DECODE_STAMPS[8]] == 15.0 and ph["layer period"] == 20.0
    assert trace.DECODE_STAMPS[1] not in ph                  # never stamped
    assert "gate logits complete" in trace.format_decode_phases(ph)
    assert trace.decode_phase_medians(st[:, :2]) == {}


@pytest.mark.gpu
def test_traced_persistent_decode_records_one_kernel_per_token_and_its_phases():
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import harness
    if not harness.token_kernel_expected():
        pytest.skip("launch calls may block here: apex_decode_token keeps to per-layer launches")
    r = subprocess.run([sys.executable, "bench.py", "--trace", "--config", "1", "--layers", "4", "--resident", "--warmup", "3"],
                       cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    t = line["trace"]
    assert t[trace.KERNEL_NAMES[10]]["launches"] == line["tokens_traced"] and t["_all"]["spans"] == line["tokens_traced"]
    ph = line["persistent_kernel_phase_median_us"]
    order = [trace.DECODE_STAMPS[i] for i in (5, 6, 7, 8, 13)]   # gate -> plan -> first row -> last row -> y added
    assert all(k in ph for k in order) and all(ph[a] <= ph[b] for a, b in zip(order[:-1], order[1:])), ph
    assert 1.0 < ph["layer period"] < 500.0


@pytest.mark.gpu
def test_traced_decode_records_every_kernel_in_order():
    r = subprocess.run([sys.executable, "bench.py", "--trace", "--config", "0", "--resident", "--warmup", "3", "--layer-launches"],
                       cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    t = line["trace"]
    n = line["tokens_traced"] * line["layers"]
    for kid in (1, 3, 4, 5):     # prefetch router (+ selection), attention stand-in, gate, expert FFN: one launch per layer-step
        assert t[trace.KERNEL_NAMES[kid]]["launches"] == n, t
        assert 0.5 < t[trace.KERNEL_NAMES[kid]]["mean_us"] < 500.0
    assert t["_all"]["spans"] == 4 * n and 0.0 < t["_all"]["busy_fraction"] <= 1.0
    ph = line["ffn_cta_phase_median_cycles"]
    assert len(ph) == 7 and all(v >= 0 for v in ph.values())
    # the table printed beside it lists the kernels of a layer-step in launch order
    rows = [l for l in r.stderr.splitlines() if l[:6] in ("prefet", "attent", "gate  ", "expert")]
    assert rows[0].startswith("prefetch router") and rows[1].startswith("attention") and rows[2].startswith("gate")
    assert rows[3].startswith("expert FFN")


@pytest.mark.gpu
def test_bench_line_carries_the_contract_keys():
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import harness
    if not harness.token_kernel_expected():
        pytest.skip("launch calls may block here: apex_decode_token keeps to per-layer launches")
    # a short run of the default workload (config 1, 32 layers): one JSON line with the metric, the end-to-end figure
    # through host buffers, the roofline record of the dominant kernel, the CPU oracle baseline and the clock record
    r = subprocess.run([sys.executable, "bench.py", "--steps", "6", "--warmup", "3", "--no-policies", "--no-other-configs",
                        "--cpu-baseline-tokens", "1"], cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["metric"] == "moe_decode_tokens_per_s" and d["unit"] == "tokens/s" and d["n_gpus"] == 1 and d["steps"] == 6
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["config"]["workload"].startswith("config1") and "model" not in d["config"]
    assert 5.0 < d["value"] < 1000.0 and abs(d["ms_per_step"] * d["value"] - 1000.0) < 1.0
    assert d["gpu_launches"] == 6                                  # one token kernel per timed token
    e = d["e2e"]
    assert 5.0 < e["value"] < 1000.0 and e["h2d_bytes_per_step"] == 2 * 32 * 1536 * 4 and e["d2h_bytes_per_step"] == 32 * 1536 * 4
    rf = d["roofline"]
    assert rf["bound"] == "hbm" and rf["kernel"] == "decode_token_kernel" and rf["unit"] == "GB/s"
    assert abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9 and 0.05 < rf["frac"] < 1.2 and "traffic" in rf
    assert rf["per_layer_ffn_kernel_alone"]["kernel"] == "moe_ffn_stream_kernel" and rf["per_layer_ffn_kernel_alone"]["traffic"] > 3.7e7
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and "sample" in c
    k = d["clocks"]
    assert k["sm_mhz"] > 0 and k["sm_max_mhz"] >= k["sm_mhz"] and isinstance(k["reasons"], list)
