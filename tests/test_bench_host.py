"""Host side of bench.py that needs no GPU: the reference arm (the CPU oracle timed over exactly K steps on a
bounded token sample, printed by rank 0 alone) and the refusal of the product arm to run without a GPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench(*argv, **env):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], cwd=ROOT,
                          env=dict(os.environ, **env), capture_output=True, text=True, timeout=600)


def test_reference_arm_times_exactly_k_steps_of_the_oracle():
    out = _bench("--impl", "reference", "--workload", "tiny_fp32", "--steps", "3", "--warmup", "2")
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["steps"] == 3 and line["warmup"] == 2
    assert line["metric"] == "moe_layer_fwd_bwd_tokens_per_s" and line["unit"] == "tokens/s"
    assert line["higher_is_better"] is True and line["vs_baseline"] is None
    assert line["config"]["workload"] == "tiny_fp32"
    cpu = line["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] == line["value"] > 0
    assert line["e2e"] == {"value": line["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
    assert abs(line["ms_per_step"] * 1e-3 * line["value"] - 512) < 1e-6 * 512    # the sample: all 512 tokens of this workload


def test_reference_arm_halves_its_sample_to_fit_the_time_budget():
    out = _bench("--impl", "reference", "--workload", "182m_slice", "--steps", "2", "--warmup", "1",
                 "--ref-tokens", "2048", "--ref-budget-s", "0.001")
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert "over 256 of the 4096 tokens" in line["cpu_baseline"]["sample"]
    assert line["steps"] == 2


def test_reference_arm_prints_on_rank_zero_only():
    out = _bench("--impl", "reference", "--workload", "tiny_fp32", "--steps", "1", "--warmup", "1",
                 RANK="1", WORLD_SIZE="2")
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_product_arm_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        return
    out = _bench("--workload", "tiny_fp32", "--steps", "1", "--warmup", "1")
    assert out.returncode != 0
    assert "impl" not in out.stdout and "NVIDIA" in out.stderr
