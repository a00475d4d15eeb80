"""The benchmark's reference arm (the CPU oracle timed on the host cores) and its host logic.

Runs without a GPU: the arm touches neither the library nor a device.
"""

import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402

REQUIRED = ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
            "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches")


def _run(extra_env, *flags):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env.update(extra_env)
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", *flags], env=env,
                          capture_output=True, text=True, timeout=600)


def test_reference_arm_prints_one_line_with_the_contract_keys():
    res = _run({}, "--steps", "1", "--warmup", "1", "--gpus", "1")
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in REQUIRED:
        assert k in d, k
    assert d["impl"] == "reference" and d["steps"] == 1 and d["warmup"] == 1 and d["n_gpus"] == 1
    assert d["value"] > 0 and d["unit"] == "TFLOP/s" and d["higher_is_better"] is True
    assert d["dtype"] == "f64" and d["gpu_launches"] == 0 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["cpu_baseline"]["cores"] >= 1 and "2340 of 4680" in d["cpu_baseline"]["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == bench.WORKLOAD and "model" not in d["config"]


def test_other_ranks_of_a_launcher_leave_without_work_or_output():
    res = _run({"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1", "MASTER_ADDR": "127.0.0.1",
                "MASTER_PORT": "29999"}, "--steps", "1", "--warmup", "0", "--gpus", "2")
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_sample_shrinks_with_the_number_of_steps():
    sizes = [bench.reference_sample_size(k, w) for k, w in ((1, 0), (3, 1), (20, 5), (40, 10), (100, 5))]
    work = [h * r for h, r in sizes]
    assert sizes[0] == (2, 2340) and sizes[-1] == (1, 256)
    assert all(a >= b for a, b in zip(work, work[1:]))
    for (k, w), (h, r) in zip(((1, 0), (3, 1), (20, 5), (40, 10), (100, 5)), sizes):
        assert 1 <= h <= 12 and 1 <= r <= 4680
