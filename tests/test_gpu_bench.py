"""The benchmark's contract, on the smallest workload: `bench.py` prints one JSON line that carries
the metric, the per-operation figures, the roofline and CPU-baseline objects, the end-to-end leg with
its declared copy sizes, the clock record and a non-zero count of this library's kernel launches."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_bench_line_on_config0():
    d = _run("--workload", "cfg0", "--steps", "5", "--warmup", "3", "--also", "")
    assert d["unit"] == "GB/s" and d["value"] > 0 and d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] == 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["config"]["workload"].startswith("cfg0:") and "fit the 126 MB L2" in d["config"]["l2"]
    assert d["gpu_launches"] == 5 * 4 and d["self_check"] == "ok"
    assert set(d["ops"]) == {"pack", "checksum", "unpack", "shard", "pack+checksum+shard"}
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    assert r["traffic"] is None or r["traffic"] > 0
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0 and c["sample"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] == 25_790_464 and e["d2h_bytes_per_step"] > 25_790_464
    assert e["self_check"] == "ok" and e["path"] in e["paths"]
    assert d["clocks"]["sm_max_mhz"] and isinstance(d["clocks"]["reasons"], list)
    for key in ("fused_send", "fused_receive", "shard_one_shot", "graph_step", "transfer"):
        assert d[key] and all(v for k, v in d[key].items() if k.endswith("_match")), key


def test_bench_profiling_case_is_small_and_kernels_only():
    d = _run("--workload", "cfg3", "--layers", "1", "--shard", "0,2", "--steps", "1", "--warmup", "3", "--kernels-only")
    assert d["config"]["workload"].endswith("1layers") and d["config"]["state_bytes"] == 1_497_595_904
    assert d["e2e"] is None and d["cpu_baseline"] is None and d["transfer"] is None and d["also"] == {}
    assert d["self_check"] == "ok" and d["gpu_launches"] == 4
