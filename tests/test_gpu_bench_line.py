"""bench.py on a GPU: the JSON line carries the keys of the measurement contract, on the default code path and
on the one-layer-over-the-ranks path forced onto one rank (every shard on this GPU, the all-reduce a no-op)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench(*flags):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "cfg4", "--steps", "3",
                          "--warmup", "3", *flags], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_default_line_has_the_contract_keys():
    d = _bench("--ref-rows", "64")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["config"]["workload"] == "cfg4" and d["scaling"] == "weak" and d["higher_is_better"] is False
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["kernel_launches"] == 3 * 8 and 0.0 < r["frac"] < 1.2
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-12 and r["accumulate_stage"]["achieved"] <= r["achieved"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 2 * 32896 * 1024 * 4 + 4096 * 1024 * 4 and d["e2e"]["value"] > d["value"]
    assert d["gpu_launches"] > 0 and d["value"] > 0


def test_one_layer_over_the_ranks_path_on_one_rank():
    d = _bench("--shard-layer", "--no-cpu-baseline", "--no-e2e")
    assert d["scaling"] == "strong" and d["n_gpus"] == 1 and d["value"] > 0
    assert "one layer over 1 GPUs" in d["config"]["parallelism"]
