"""bench.py end to end on a GPU: one short run, then the JSON line is checked against the
measurement contract (keys, units, launch count, sane roofline fractions)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys(bq):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "4", "--warmup", "3", "--e2e-steps", "1", "--no-cpu-baseline"],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads(r.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 4 and d["higher_is_better"] is True
    assert d["data"] == "synthetic" and "workload" in d["config"] and d["vs_baseline"] is None
    assert d["gpu_launches"] == 4 * 12
    rf = d["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and 0.3 < rf["frac"] < 1.1 and abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-3
    assert rf["traffic"] is None or 0.9 < rf["traffic"] / d["kernels"][rf["kernel"]]["algorithmic_bytes"] < 1.1
    e = d["e2e"]
    assert e["unit"] == "GB/s" and 0 < e["value"] < d["value"] and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert len(d["kernels"]) == 12 and all(0.2 < k["frac_of_measured"] < 1.1 for k in d["kernels"].values())
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    for q in d["quality"].values():
        assert 1.8 < q["compression_ratio"] < 2.0 and 0.003 < q["rel_rms_error"] < 0.03
    for v in d["bq4"].values():
        assert 0.2 < v["quantize_frac_of_measured"] < 1.1 and 0.5 < v["dequantize_frac_of_measured"] < 1.1
        assert 3.5 < v["compression_ratio"] < 4.0 and 0.05 < v["rel_rms_error"] < 0.3
    assert set(d["bq4"]) == {"b64", "b1024", "b64_scale16"} and d["bq4"]["b64_scale16"]["compression_ratio"] > d["bq4"]["b64"]["compression_ratio"]
    t = d["autotune"]
    assert 0.3 < t["frac_of_measured"] < 1.1 and t["picked_for_rel_rms_0.01"] in t["blocks"] and len(t["rel_rms_error"]) == len(t["blocks"])
    assert all(abs(a - q["rel_rms_error"]) < 2e-5 for a, q in zip(t["rel_rms_error"], d["quality"].values()))
    sc = d["small_configs"]
    assert set(sc) == {"tiny", "decode70b", "prefill7b", "moe_prefill"}
    for v in sc.values():
        assert all(0 < v[op]["warm_us"] < 1000 and 0 < v[op]["frac_of_measured"] < 1.1 for op in ("quantize", "dequantize", "roundtrip"))
        assert ("cold_us" in v["roundtrip"]) == v["fits_l2"]
    assert sc["moe_prefill"]["roundtrip"]["frac_of_measured"] > 0.5 and not sc["moe_prefill"]["fits_l2"]
    # the decomposed linear layer: its own roofline object, no kernel error (its full-size parity is tests/test_gpu_mmd.py's)
    m = d["mmd"]
    mr = m["roofline"]
    assert mr["bound"] == "tensor" and mr["unit"] == "TOP/s" and 0.3 < mr["frac"] < 1.1 and abs(mr["frac"] - mr["achieved"] / mr["peak"]) < 1e-3
    assert m["kernel_status"] == 0 and 0.001 < m["quality"]["weight_rel_rms_error"] < 0.1
    assert 0 < m["e2e"]["tops"] < m["tops"] and m["e2e"]["h2d_bytes_per_call"] > 0 and m["cpu_baseline"]["kind"] == "oracle"
    assert 1.9 < m["quality"]["weight_bytes_ratio"] < 2.0 and m["gpu_launches"] > 0
    dec = m["decode"]
    assert dec["kernel_status"] == 0 and 0.2 < dec["frac_of_measured_hbm"] < 1.1
    wide = m["decode_wide"]
    assert wide["kernel_status"] == 0 and 0.3 < wide["frac_of_measured_hbm"] < 1.1 and wide["algorithmic_bytes"] > 3 * dec["algorithmic_bytes"]
    assert abs(mr["ms"] - m["ms_per_call"]) < 1e-6 and mr["product_kernel_estimate"]["frac"] >= mr["frac"]      # the roofline is the whole call's
    # the input's fingerprint, the host-buffer calls behind e2e, finished sections on stderr as they complete
    assert len(d["config"]["input_sha256"]) == 64 and "bq_roundtrip_host" in e["api"]
    sections = [json.loads(line)["section"] for line in r.stderr.splitlines() if line.startswith('{"section"')]
    assert sections[:3] == ["kernels", "e2e", "quality"] and {"bq4", "autotune", "small_configs", "mmd", "transport"} <= set(sections)
    # the boundary transport, loop-back: what arrives is the fused roundtrip's bytes; about half the bytes cross
    tr = d["transport"]
    assert tr["bit_identical_to_roundtrip"] is True and "loop-back" in tr["link"] and 1.9 < tr["bytes_ratio"] < 2.0
    assert 0 < tr["store"]["ms"] < 5 and 0 < tr["copy"]["ms"] < 5 and tr["pieces"] == 16
    mt = d["mtpp"]
    assert mt["orders_per_s"] > 1000 * mt["cpu_baseline"]["value"] > 0 and 0 < mt["best_bottleneck"] <= mt["worst_bottleneck"]


def test_bench_on_another_config(bq):
    """--config runs the step on one of the other workloads; a tensor that fits in L2 is flushed out before every launch."""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "3", "--warmup", "3", "--e2e-steps", "1", "--config", "prefill7b"],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert "prefill7b" in d["config"]["workload"] and "256 MiB buffer is written before every launch" in d["config"]["l2"]
    assert d["gpu_launches"] == 3 * 3 and set(d["kernels"]) == {"quantize_b256", "dequantize_b256", "roundtrip_b256"}
    assert d["cpu_baseline"]["kind"] == "oracle" and d["mmd"] is None and d["roofline"]["traffic"] is None
    assert 0 < d["e2e"]["value"] < d["value"]
