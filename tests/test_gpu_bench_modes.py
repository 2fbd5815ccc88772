"""The benchmark's other workloads run and print one well-formed JSON line each (small sizes; numbers are not checked)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, timeout=600,
                         cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout[-2000:]
    return json.loads(lines[0])


@pytest.mark.parametrize("args,keys", [
    (["--config", "3", "--layers", "2", "--steps", "3", "--warmup", "3", "--no-cpu-baseline"], ["e2e", "e2e_all_layers_per_call", "kernels", "decode_all_layers_one_launch"]),
    (["--config", "4", "--steps", "16", "--warmup", "3"], []),
    (["--config", "5", "--layers", "2", "--steps", "2", "--warmup", "3"], ["kernels"]),
    (["--workload", "overlap", "--layers", "2", "--steps", "3", "--warmup", "3"], ["kernels"]),
    (["--workload", "qkv", "--layers", "2", "--steps", "2", "--warmup", "3"], ["points", "decode_projection", "decode_layer_chain"]),
    (["--workload", "sweep", "--layers", "1"], ["sweep"]),
    (["--workload", "drift", "--layers", "2", "--chunks", "80"], ["drift"]),
    (["--workload", "drift", "--config", "5", "--layers", "2", "--chunks", "40"], ["drift"]),
    (["--workload", "decode-trace", "--layers", "2"], ["trace"]),
])
def test_bench_workloads_print_one_json_line(args, keys):
    d = _run(*args)
    for k in ("metric", "value", "unit", "n_gpus", "ms_per_step", "higher_is_better", "scaling", "dtype", "data", "config", "roofline"):
        assert k in d, k
    assert d["value"] > 0 and (d["roofline"]["frac"] is None or d["roofline"]["frac"] > 0)
    for k in keys:
        assert d.get(k) is not None, k


def test_sweep_has_the_policy_arms():
    d = _run("--workload", "sweep", "--layers", "1")
    arms = {r["axis"]: r for r in d["sweep"]}
    assert "policy:native_rope" in arms and "policy:sink_any_type" in arms and "deployed" in arms
    assert arms["policy:native_rope"]["contiguous"] is False and arms["deployed"]["contiguous"] is True
    # native positions: the eviction re-rotates nothing, so it must be much cheaper than the deployed policy's
    assert arms["policy:native_rope"]["evict_ms"] < arms["deployed"]["evict_ms"]
