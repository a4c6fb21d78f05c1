"""Host-only checks of bench.py: the reference arm (the CPU oracle) prints one JSON line with the contract's keys,
and the product arm refuses to run without a CUDA device instead of falling back to the CPU."""
import json
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                          cwd=ROOT, timeout=600)


def test_reference_arm_prints_the_contract_line():
    out = _run("--impl", "reference", "--config", "1", "--steps", "2", "--warmup", "1")
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in j, key
    assert j["impl"] == "reference" and j["metric"] == "nlr_iterations_per_second" and j["unit"] == "iterations/s"
    assert j["steps"] == 2 and j["warmup"] == 1 and j["n_gpus"] == 1 and j["higher_is_better"] is True
    assert j["vs_baseline"] is None and j["gpu_launches"] == 0 and j["value"] > 0
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["value"] == j["value"]
    assert j["e2e"] == {"value": j["value"], "unit": j["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in j["config"] and "model" not in j["config"]
    assert j["cpu_baseline"]["extrapolated"] is False and j["config"]["config_index"] == 1


def _bench_module():
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_roofline_object_names_the_longer_phase_and_keeps_the_other():
    b = _bench_module()
    n, d, r = 1_000_000, 128, 16
    # first phase longer than the second product: it must be the one described at the top level
    o = b.roofline_objects(n, d, r, "mma.tf32x3", ms_first=0.1208, ms_second=0.1123, it_s=0.2450e-3)
    assert o["kernel"].startswith("first phase") and o["other"]["kernel"].startswith("second product")
    assert o["bound"] == "hbm" and o["unit"] == "GB/s"
    assert abs(o["achieved"] - b.first_phase_bytes(n, d, r) / 0.1208e-3 / 1e9) < 1e-6 * o["achieved"]
    assert abs(o["frac"] - o["achieved"] / o["peak"]) < 1e-12
    it = o["iteration"]
    for key in ("frac", "bound", "frac_of_hbm_B_alg", "frac_of_hbm_B_min", "useful_tflops", "ms_between_phases",
                "algorithmic_bytes", "minimal_bytes"):
        assert key in it, key
    assert it["algorithmic_bytes"] == 8 * n * d + 12 * n * r + 16 * n and it["minimal_bytes"] == 8 * n * d + 8 * n * r
    assert abs(it["frac"] - it["frac_of_hbm_B_alg"]) < 1e-12 and it["frac_of_hbm_B_min"] < it["frac_of_hbm_B_alg"]
    assert o["traffic"] is not None and o["traffic_source"].startswith("profiles/")
    # the other order
    o2 = b.roofline_objects(n, d, r, "mma.tf32x3", ms_first=0.10, ms_second=0.12, it_s=0.23e-3)
    assert o2["kernel"].startswith("second product")
    # a tensor-bound shape reports the three issued products and the useful rate beside them
    o4 = b.roofline_objects(2_000_000, 768, 1000, "f16x3.tiled", ms_first=10.4, ms_second=9.3, it_s=20.0e-3)
    assert o4["bound"] == "tensor" and o4["unit"] == "TFLOP/s" and o4["iteration"]["bound"] == "tensor"
    assert abs(o4["flops_per_launch"] - 3 * 2.0 * 2_000_000 * 768 * 1000) < 1.0
    assert abs(o4["iteration"]["useful_tflops"] * 3 - o4["iteration"]["achieved_tflops"]) < 1e-9
    # a shape with no capture reports null traffic instead of a stale number
    assert b.roofline_objects(12345, 64, 100, "f16x3", 1.0, 1.0, 2.1e-3)["traffic"] is None


def test_cpu_sample_is_bounded_and_marked():
    b = _bench_module()
    assert b.oracle_sample_rows(2000, 16, 4) == 2000
    assert b.oracle_sample_rows(1_000_000, 128, 16) == 1_000_000
    m4 = b.oracle_sample_rows(2_000_000, 768, 1000)
    assert 4096 <= m4 < 2_000_000 and 4.0 * m4 * 768 * 1000 <= b.CPU_SAMPLE_FLOPS * 1.01
    import synth
    spec = synth.config(1)
    X, _, _ = synth.make_mixture(spec)
    leg = b.cpu_baseline_leg(spec, X, synth.make_u0(spec.n, spec.K, spec.K), synth.default_hparams(spec.K))
    for key in ("value", "unit", "cores", "kind", "sample", "extrapolated"):
        assert key in leg
    assert leg["kind"] == "oracle" and leg["extrapolated"] is False and leg["value"] > 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="needs a machine without a GPU")
def test_product_arm_has_no_cpu_fallback():
    out = _run("--config", "1", "--steps", "1", "--warmup", "1")
    assert out.returncode != 0
    assert "no CPU fallback" in (out.stderr + out.stdout)
