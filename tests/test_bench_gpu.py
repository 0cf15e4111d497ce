"""bench.py end to end on the GPU (smallest workload): one JSON line with every key the measurement contract asks for."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, timeout=600,
                         cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_bench_line_has_the_contract_keys():
    d = run_bench("--workload", "tiny", "--steps", "5", "--warmup", "3")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] == 3 and d["scaling"] == "weak" and d["data"] == "synthetic"
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["config"]["workload"] == "tiny" and "model" not in d["config"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["matches_device_path"] is True
    assert d["gpu_launches"] == 2 * d["steps"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_default_line_covers_every_configuration_and_headlines_the_largest():
    d = run_bench("--steps", "3", "--warmup", "3", "--repeats", "3", "--no-cpu-baseline", "--sharded")
    c = d["config"]
    assert c["workload"] == "opt30b" and d["dtype"] == "f32"
    names = [r["workload"] for r in c["workloads"]]
    assert sorted(names) == sorted(["tiny", "opt13b", "opt30b", "llama70b", "ragged"])
    for r in c["workloads"]:
        assert r["ms_per_step"] > 0 and r["partial_us"] > 0 and r["merge_us"] > 0 and r["e2e"]["matches_device_path"] is True
        rp = r["repeats_ms_per_step"]
        assert len(rp["all"]) == 3 and rp["min"] <= rp["median"] <= rp["max"] and len(rp["sm_mhz"]) == 3
        assert set(r["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
        if r["workload"] == "tiny":
            assert "step_frac_of_8000" not in r and r["us_per_step"] > 0
        else:
            ro = r["roofline"]
            assert 0.3 < r["step_frac_of_8000"] < 1.05 and ro["traffic"] > 0.98 * ro["alg_bytes_per_launch"]     # (partials that stay in the L2 never reach DRAM)
            assert abs(ro["frac"] - ro["achieved"] / ro["peak"]) < 1e-9
            assert r["probe_us"] > 0 and 0.3 < r["step_frac_of_probe"] < 1.5     # the bare loads are the ceiling
    head = [r for r in c["workloads"] if r["workload"] == "opt30b"][0]
    assert d["ms_per_step"] == head["ms_per_step"] and d["value"] == head["kv_tokens_per_s"]
    assert d["roofline"] == head["roofline"] and d["e2e"] == head["e2e"]
    assert c["min_step_frac_of_8000"] == min(r["step_frac_of_8000"] for r in c["workloads"] if r["workload"] != "tiny")
    assert [h["shape"] for h in c["handoff"]] == ["mha", "gqa8", "mha_c512", "gqa8_c512"] and all(h["gbs"] > 1000 for h in c["handoff"])
    s = d["sharded"]
    assert s["ranks"] == 1 and s["gpu_tokens_total"] == 419430 and s["tokens_this_rank"] == 419430 and s["ms_per_step"] > 0
