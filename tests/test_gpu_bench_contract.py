"""bench.py's one-line JSON contract, checked on the tiny config (seconds): every key the driver reads is there
with a sensible type, for the GPU arm and for the oracle ("reference") arm."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    r = subprocess.run([sys.executable, "bench.py", "--workload", "c1", "--steps", "3", "--warmup", "3", *extra],
                       cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # exactly one JSON line on stdout
    return json.loads(lines[0])


def test_gpu_arm_line():
    d = _run("--ref-rows", "64", "--sweep-plan", "fused=c1:3;dense=c1:2;fwdchunk=c1:2")
    assert d["unit"] == "tokens/s" and d["higher_is_better"] is True and d["scaling"] == "weak"
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] >= 3
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["ms_per_step_min"] <= d["ms_per_step_median"]
    assert abs(d["value"] - 256 / (d["ms_per_step"] * 1e-3)) <= 1e-6 * d["value"]          # whole-job tokens / time
    assert d["vs_baseline"] is None and d["dtype"] == "bf16" and d["data"] == "synthetic"
    assert "workload" in d["config"] and "model" not in d["config"]
    assert d["gpu_launches"] > 0 and d["gpu_launches"] % d["steps"] == 0
    c = d["clocks"]
    assert c["sm_max_mhz"] >= c["sm_mhz"] > 0 and isinstance(c["reasons"], list)
    e = d["e2e"]
    assert e["value"] > 0 and e["unit"] == "tokens/s" and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"] * 1.05                    # copies inside the timed region cannot make it faster
    rec = d["e2e_record_from_host"]
    assert rec["h2d_bytes_per_step"] == 256 * 16 * 8 and rec["d2h_bytes_per_step"] == 4
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and "traffic" in r
    b = d["cpu_baseline"]
    assert b["kind"] == "oracle" and b["cores"] >= 1 and b["value"] > 0 and b["unit"] == "tokens/s" and b["sample"]
    f = d["feature_loss"]
    assert 0 < f["mse"]["frac_of_hbm_copy"] < 1.3 and 0 < f["cosine"]["frac_of_hbm_copy"] < 1.3
    assert set(d["stages"]) >= {"fwd_gemm_lse", "bwd_gemm_dlogits", "dhidden_gemm", "dweight_gemm"}
    assert d["stage_clocks"]["sm_mhz"] > 0 and d["stage_check"]["sum_of_stage_ms"] > 0
    assert all(v["ms_x_mhz_per_launch"] > 0 for k, v in d["stages"].items() if v["launches_per_step"])
    rows = d["context_sweep"]["rows"]
    assert [r["method"] for r in rows] == ["fused", "dense", "fwdchunk"]
    for r in rows:                                           # measured, in a process of its own, same loss
        assert r["ms_per_iter"] > 0 and r["peak_gb"] > 0 and r["driver_delta_gb"] >= 0 and r["steps"] >= 2
        assert abs(r["loss"] - d["loss"]) <= 1e-3 * abs(d["loss"])
    assert rows[0]["status"] == 0 and 0 < rows[0]["frac_of_bf16_burst_peak"] < 1.2
    assert d["collective"] is None and d["config"]["parallelism"].startswith("independent")


def test_reference_arm_line():
    d = _run("--impl", "reference", "--ref-rows", "32")
    assert d["impl"] == "reference" and d["unit"] == "tokens/s" and d["value"] > 0
    assert d["dtype"] == "f64" and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"]["value"] == d["value"] and d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in d["config"]


def test_sharded_modes_on_one_rank_give_the_same_loss():
    """--parallel tokens / vocab with a single rank: the same batch through the data-parallel and the
    tensor-parallel call sequences (count kernel + device-side divisor; shard statistics + finish) must give the
    loss of the plain two calls, and the line must say what crosses ranks per step."""
    base = _run("--no-sweep", "--no-e2e", "--no-cpu-baseline")
    for mode, scaling in (("tokens", "weak"), ("vocab", "strong")):
        d = _run("--no-sweep", "--no-e2e", "--no-cpu-baseline", "--parallel", mode)
        assert abs(d["loss"] - base["loss"]) <= 1e-6 * abs(base["loss"])
        assert d["scaling"] == scaling and d["collective"]["bytes_per_step"] > 0 and d["gpu_launches"] > 0
        assert d["value"] > 0 and d["single_pass"] is None
        assert (d["roofline"] is not None and d["stages"]["dweight_gemm"]["tflops"] > 0) if mode == "tokens" \
            else (d["roofline"] is None and d["stages"] is None)
