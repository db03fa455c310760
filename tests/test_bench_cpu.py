"""CPU checks of bench.py: the reference arm's JSON line, the loud failure of the product arm
without a GPU, and the FLOP accounting the roofline figures rest on."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2609_27547_b200 import synth


def _run(*args):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, timeout=600)


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    p = _run("--impl", "reference", "--config", "0", "--steps", "1", "--warmup", "0")
    assert p.returncode == 0, p.stderr
    lines = [l for l in p.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "env_action_chunks_per_sec" and d["unit"] == "chunks/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["n_gpus"] == 1 and d["steps"] == 1
    assert d["value"] > 0 and d["config"]["workload"].startswith("configs[0]")
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and "envs" in cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "chunks/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["gpu_launches"] == 0


def test_product_arm_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        return
    p = _run("--config", "0", "--steps", "1")
    assert p.returncode != 0
    assert "no CPU fallback" in (p.stderr + p.stdout)
    assert not [l for l in p.stdout.splitlines() if l.startswith("{")]     # and prints no result line


def test_flop_accounting():
    import bench
    w = synth.WORKLOADS[4]
    # K [L (28 H d^2 + 4 H P d + 4 H^2 d) + 4 H A d] per chunk
    H, A, d, L, K, P = w.H, w.A, w.d, w.L, w.K, 768
    per_chunk = K * (L * (28 * H * d * d + 4 * H * P * d + 4 * H * H * d) + 4 * H * A * d)
    env = synth.EnvInputs(0, None, None, P, 0)
    assert bench.workload_flops(w, [env]) == per_chunk
    assert abs(per_chunk - 158.56e9) / 158.56e9 < 1e-3
    late = synth.EnvInputs(1, None, None, P, 7)           # an environment that starts at step 7 runs 3 steps
    assert bench.workload_flops(w, [late]) == per_chunk * 3 // 10
    wh = synth.scaled(w, d_ctx=1024)
    assert bench.workload_flops(wh, [env]) == per_chunk + 4 * L * d * 1024 * P
