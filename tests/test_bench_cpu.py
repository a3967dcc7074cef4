"""bench.py pieces that need no GPU: the reference arm prints one well-formed JSON line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line(oracle):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, check=True)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "dlion_step_param_worker_updates_per_s"
    assert d["value"] > 0 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["config"]["workload"] == "c1"


def test_other_ranks_of_the_reference_arm_do_nothing(oracle):
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_algorithmic_bytes():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2404_00438_b200 import inputs
    w = inputs.workload("c5")
    assert bench.bytes_per_param_worker_k1(w) == 10.125 and bench.bytes_per_param_worker_k1(w, 2) == 6.125
    assert bench.bytes_per_param_k2(w) == 10.0
    assert bench.bytes_per_param_worker_k1(inputs.workload("c1")) == 12.125
    assert bench.host_memory_available() > 0


def test_traffic_record_matches_the_committed_kernel_sources():
    """profiles/ncu_traffic.json is keyed by a hash of the worker-side kernel's sources: the
    record in the tree must be the one captured from the sources in the tree, and close to the
    algorithmic bytes (a capture with wasted re-reads would show here)."""
    sys.path.insert(0, ROOT)
    import bench
    f32 = bench.ncu_traffic("worker_step_kernel", "grads_bf16_momentum_f32")
    b16 = bench.ncu_traffic("worker_step_kernel", "grads_bf16_momentum_bf16")
    assert f32 is not None and b16 is not None, "kernel sources changed since the ncu capture: capture again"
    assert 0.97 * 10.125 <= f32 <= 1.03 * 10.125 and 0.97 * 6.125 <= b16 <= 1.03 * 6.125
    assert bench.ncu_traffic("worker_step_kernel", "no_such_variant") is None
