"""The bench's reference arm (the oracle on host cores) prints one JSON line with the contract's keys; runs without a GPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["impl"] == "reference" and d["metric"] == "fp8_kv_decode_attn_achieved_hbm_gbs_64k_ctx" and d["unit"] == "GB/s"
    for key in ("value", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline", "dtype",
                "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["steps"] == 1 and d["value"] > 0 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in d["config"] and "sample" in d["config"]


def test_traffic_is_tied_to_the_kernel_sources():
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    a = argparse.Namespace(ncu_traffic=None, config=3, kernel="mma", splits=0, contiguous=False)
    t = bench.ncu_traffic(a)
    assert t is None or t == bench.NCU_CAPTURE["dram_bytes_per_launch"]
    a.kernel = "tcgen05"
    assert bench.ncu_traffic(a) is None          # the capture is of the default kernel only
    a.kernel, a.ncu_traffic = "mma", 123.0
    assert bench.ncu_traffic(a) == 123.0         # an explicit figure is reported as given
