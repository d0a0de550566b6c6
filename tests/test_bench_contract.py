"""The benchmark's reference arm (the CPU oracle on a bounded sample) runs without a GPU: its one
JSON line carries the keys the measurement contract asks for, with the same metric, unit and
workload description as the CUDA arm prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    sys.path.insert(0, ROOT)
    import bench
    env = dict(os.environ, PYTHONPATH=ROOT)
    # the arm as it is, but with a sample of 128 query rows: a few tenths of a second of oracle work
    code = ("import sys, bench; bench.cpu_baseline.__defaults__ = (128,); "
            "sys.argv = ['bench.py', '--impl', 'reference', '--steps', '2', '--warmup', '1']; bench.main()")
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["steps"] == 2 and d["warmup"] == 1 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["value"] > 0 and d["gpu_launches"] == 0 and d["dtype"] == "f64" and d["data"] == "synthetic"
    assert d["config"]["workload"] == bench.WORKLOAD and d["config"]["chunk"] == 32768
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


def test_work_model_matches_the_closed_forms():
    """Flops and bytes the roofline uses: 4 Hq d (Lc n_cache + Lc (Lc + 1) / 2) per chunk step, and
    Q + K + V + O bytes per launch."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2506_01215_b200 import synth
    w = synth.WORKLOADS["llama8b_128k"]
    assert bench.attn_flops(w, 0) == 4 * 32 * 128 * (32768 * 32769 // 2)
    assert bench.attn_flops(w, 1) == 4 * 32 * 128 * (32768 * 8192 + 32768 * 32769 // 2)
    assert abs(sum(bench.attn_flops(w, s) for s in range(4)) / 1e12 - 48.38) < 0.01
    assert bench.attn_bytes(w) == 2 * 128 * (2 * 32 * 32768 + 2 * 8 * 40960)
    assert bench.retrieval_gather_bytes(w) == 131072 * 1024 * 2 + 2 * 4096 * 4096 * 2
    assert bench.job_throughput(w, 2, 10.0) == 2 * 131072 / 10e-3
