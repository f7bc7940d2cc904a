"""The benchmark's one-line contract.

CPU: the reference arm (the oracle on the host cores) prints one JSON line with the same metric, unit and config
keys as the GPU arm, rank 0 alone prints it, and the default arm fails loudly without a GPU.
GPU: the default arm on a small workload prints the line with every key a reader of it relies on.
"""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent

BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches"}
CONFIG_KEYS = {"workload", "d", "k", "N_nodes", "M", "S", "layers", "qsgd_levels", "l2", "parallelism"}


def _run(args, env_extra=None, timeout=600):
    env = dict(os.environ)
    env.update(env_extra or {})
    return subprocess.run([sys.executable, str(ROOT / "bench.py")] + args, cwd=ROOT, env=env, capture_output=True,
                          text=True, timeout=timeout)


def _one_line(stdout):
    lines = [x for x in stdout.strip().splitlines() if x.strip()]
    assert len(lines) == 1, lines
    return json.loads(lines[0])


def test_reference_arm_prints_the_line_on_the_host():
    r = _run(["--impl", "reference", "--workload", "tiny", "--steps", "2", "--warmup", "1"])
    assert r.returncode == 0, r.stderr[-2000:]
    line = _one_line(r.stdout)
    assert BASE_KEYS <= set(line) and line["impl"] == "reference"
    assert CONFIG_KEYS <= set(line["config"]) and line["config"]["workload"] == "tiny"
    assert line["unit"] == "GB/s" and line["higher_is_better"] is True and line["value"] > 0
    assert line["steps"] == 2 and line["warmup"] == 1 and line["gpu_launches"] == 0
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] and "slices" in cb["sample"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_reference_arm_is_silent_on_the_other_ranks():
    r = _run(["--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0", "--gpus", "2"],
             env_extra={"RANK": "1", "LOCAL_RANK": "1", "WORLD_SIZE": "2"})
    assert r.returncode == 0, r.stderr[-2000:]
    assert r.stdout.strip() == ""


def test_reference_arm_of_the_quantizing_workload_names_its_levels():
    """The largest configuration quantizes the compressed vectors: its reference line carries the levels, and its
    sample is a bounded part of the workload (the whole of it would take the oracle about ten seconds a step)."""
    r = _run(["--impl", "reference", "--workload", "large", "--steps", "1", "--warmup", "0", "--reference-seconds", "2"])
    assert r.returncode == 0, r.stderr[-2000:]
    line = _one_line(r.stdout)
    assert line["config"]["workload"] == "large" and line["config"]["qsgd_levels"] == 7
    assert "quantize" in line["cpu_baseline"]["sample"]


def test_default_arm_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    r = _run(["--workload", "tiny", "--steps", "3", "--warmup", "3"])
    assert r.returncode != 0
    assert r.stdout.strip() == ""     # no line, hence no number, from a machine that cannot run the kernels


@pytest.mark.gpu
def test_default_arm_prints_every_key_on_a_small_workload():
    r = _run(["--workload", "resnet32", "--steps", "5", "--warmup", "3", "--no-nested"])
    assert r.returncode == 0, r.stderr[-2000:]
    line = _one_line(r.stdout)
    assert BASE_KEYS <= set(line) and line.get("impl", "ours") == "ours"
    assert CONFIG_KEYS <= set(line["config"])
    assert line["gpu_launches"] > 0 and line["value"] > 0
    rf = line["roofline"]
    assert {"bound", "achieved", "peak", "unit", "frac", "traffic"} <= set(rf)
    assert abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1
    e = line["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < line["value"]       # the copies are inside its timed region
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(line["clocks"])
