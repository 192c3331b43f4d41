"""Host-side checks of bench.py's output contract that need no GPU: the reference arm (the CPU oracle)
prints one JSON line with the keys the contract names, and the flop / score counts the roofline uses
match their definitions."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "C1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"].startswith("4-bit attention prefill TFLOPS")
    for key in ("value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["e2e"]["value"] == d["value"] and d["vs_baseline"] is None and d["steps"] == 1


def test_flop_count_matches_the_metric_definition():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2607_04302_b200 import synth
    c2 = synth.config("C2")
    assert bench.attn_flops(c2) == 4 * 1 * 32 * 4096 * 4096 * 128 / 2          # causal: halved
    assert bench.attn_flops(synth.config("C2", causal=False)) == 4 * 32 * 4096 * 4096 * 128
    assert bench.whole_job_tflops(c2, 2, 10, 1000.0) == 2 * bench.attn_flops(c2) * 10 / 1.0 / 1e12
