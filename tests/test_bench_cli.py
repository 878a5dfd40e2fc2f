"""Host-only checks of bench.py's launch logic (no GPU): the rank count asked for and the launcher's must agree,
and more ranks than devices is an error, not a silent single-GPU run."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, env=None, timeout=600):
    e = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, env=e, cwd=ROOT,
                          capture_output=True, text=True, timeout=timeout)


def test_gpus_flag_must_match_the_launchers_world_size():
    r = _run(["--gpus", "1"], env={"WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0"})
    assert r.returncode != 0 and "does not match WORLD_SIZE=2" in r.stderr


def test_more_ranks_than_devices_is_refused():
    import torch
    n = torch.cuda.device_count() + 1
    r = _run(["--gpus", str(max(2, n))])
    assert r.returncode != 0 and "CUDA device(s) visible" in r.stderr


def test_reference_arm_prints_one_line_with_the_same_config_keys():
    r = _run(["--impl", "reference", "--workload", "tiny_top3", "--steps", "1", "--warmup", "0",
              "--ref-tokens-per-thread", "16"])
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["gpu_launches"] == 0 and line["value"] > 0
    assert set(line["config"]) == {"workload", "T", "H", "E", "K", "L", "controller", "parallelism", "l2"}
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"
    # ranks other than 0 print nothing and exit 0
    r1 = _run(["--impl", "reference", "--workload", "tiny_top3", "--steps", "1", "--warmup", "0", "--gpus", "2"],
              env={"WORLD_SIZE": "2", "RANK": "1", "LOCAL_RANK": "1"})
    assert r1.returncode == 0 and r1.stdout.strip() == ""


@pytest.mark.gpu
def test_bench_line_has_the_contract_keys_on_a_small_workload():
    r = _run(["--workload", "tiny_top3", "--steps", "5", "--warmup", "3", "--no-all-configs", "--min-region-s", "0.05",
              "--ref-tokens-per-thread", "32"])
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks",
                "near_tie", "all_configs", "repeats"):
        assert key in line, key
    assert line["n_gpus"] == 1 and line["steps"] == 5 and line["value"] > 0 and line["gpu_launches"] >= 10
    assert line["config"]["workload"] == "tiny_top3" and line["vs_baseline"] is None
    assert set(line["roofline"]) >= {"bound", "achieved", "peak", "unit", "frac", "traffic"}
    assert line["e2e"]["h2d_bytes_per_step"] > 0 and line["e2e"]["d2h_bytes_per_step"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["near_tie"]["differing_with_clear_gap"] == 0
