"""The benchmark's output contract: the LAST line printed is one short JSON object with the headline
(metric, value, roofline, cpu_baseline, e2e, clocks, launches); everything else comes before it, one
JSON object per line.  A line of many kilobytes cannot be read back by a caller that keeps only the
tail of the output."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, timeout=600):
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, capture_output=True,
                       text=True, timeout=timeout)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.strip()]
    assert lines, "nothing printed"
    return [json.loads(l) for l in lines], lines


def test_reference_arm_prints_one_short_line_with_the_contract_keys():
    objs, lines = _run(["--impl", "reference", "--workload", "tiny", "--T", "64", "--k", "2", "--steps", "2",
                        "--warmup", "1", "--ref-tokens", "16"])
    assert len(lines) == 1 and len(lines[0]) < 2048
    d = objs[0]
    assert d["impl"] == "reference" and d["value"] > 0 and d["unit"] == "tokens/s" and d["higher_is_better"] is True
    assert d["steps"] == 2 and d["warmup"] == 1 and d["vs_baseline"] is None and d["dtype"] == "f64"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


@pytest.mark.gpu
def test_headline_is_the_last_line_and_short(tmp_path):
    side = tmp_path / "detail.jsonl"
    objs, lines = _run(["--workload", "tiny", "--T", "64", "--k", "2", "--steps", "3", "--warmup", "3", "--stacks=",
                        "--cpu-seconds", "0.5", "--min-seconds", "0.05", "--detail-file", str(side)])
    head = objs[-1]
    assert len(lines[-1]) < 2048, "the headline line must stay short"
    assert all("detail" in o for o in objs[:-1]) and "detail" not in head
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in head, key
    assert head["value"] > 0 and head["n_gpus"] == 1 and head["steps"] == 3 and head["warmup"] == 3
    assert head["dtype"] == "bf16" and head["vs_baseline"] is None and "workload" in head["config"]
    assert head["gpu_launches"] > 0
    roof = head["roofline"]
    assert roof["bound"] in ("hbm", "tensor") and roof["unit"] in ("GB/s", "TFLOP/s")
    assert roof["achieved"] > 0 and roof["peak"] > 0 and abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-6
    e2e = head["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] == 64 * 256 * 2 == e2e["d2h_bytes_per_step"]
    cpu = head["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["value"] > 0 and cpu["cores"] >= 1 and cpu["sample"]
    # the side file holds every line, the headline included
    kept = [json.loads(l) for l in side.read_text().splitlines() if l.strip()]
    assert kept[-1]["value"] == head["value"] and len(kept) == len(objs)


def test_work_model_gives_the_hand_computed_figures():
    """The roofline numerators, against figures worked out by hand for the Qwen1.5-MoE-shaped layer
    (d 2048, E 60, I 1408, gated shared expert of 5632): 17.3 MB per routed expert and 69.2 MB for the
    shared expert in bf16, 138.7 MB for a one-token call that touches four experts; 1.136e12 flop
    for 8192 tokens at k = 4, of which 7.559e11 in the gate/up GEMM."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    from paper_2509_02753_b200 import synth
    wl = synth.WORKLOADS["qwen15"]
    per_expert = 3 * 2048 * 1408 * 2
    shared = 3 * 2048 * 5632 * 2
    assert per_expert == 17_301_504 and shared == 69_206_016
    assert bench.layer_bytes(wl, 1, 4) == 4 * per_expert + shared + (2048 * 60 + 2048) * 2 + 2 * 2048 * 2 == 138_670_080
    assert bench.layer_flops(wl, 8192, 4) == 8192 * (4 * 6 * 2048 * 1408 + 6 * 2048 * 5632 + 2 * 2048 * 60)
    assert abs(bench.layer_flops(wl, 8192, 4) / 1.136e12 - 1) < 2e-3
    assert abs(bench.ffn1_flops(wl, 8192, 4) / 7.559e11 - 1) < 1e-3
    # phase 1 at 8192 tokens with all 60 experts touched: 738 MB of gate/up weights + activations = 1090 MB
    assert abs(bench.ffn1_bytes(wl, 8192, 4, 60) / 1.0905e9 - 1) < 2e-3
