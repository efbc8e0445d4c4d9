"""The benchmark's output contract, as far as it can be checked without a GPU: the reference arm
(the CPU oracle timed on the host cores) prints one JSON line with the agreed keys, and the traffic
table is keyed to kernel sources in a way that a reworded comment does not disturb."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_agreed_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in j, key
    assert j["impl"] == "reference" and j["steps"] == 2 and j["warmup"] >= 3 and j["value"] > 0
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] >= 1
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in j["config"] and "model" not in j["config"]


def test_traffic_table_is_keyed_to_statements_not_comments():
    sys.path.insert(0, ROOT)
    import bench
    a = "int f(int x) { return x + 1; }   // add one\n"
    b = "/* increments */\nint f(int x)\n{\n    return x + 1;\n}\n"
    c = "int f(int x) { return x + 2; }\n"
    assert bench.source_digest(a) == bench.source_digest(b) != bench.source_digest(c)
    for name, kernel in (("c2", 1), ("c3", 2), ("c4", 3), ("c5", 4), ("c2t", 5)):
        assert len(bench.NCU_TRAFFIC[name]["sha"]) == 16 == len(bench.kernel_source_hash(kernel))
