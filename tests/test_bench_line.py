"""The JSON line bench.py prints: keys and types of both arms (the reference arm needs no GPU)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric": str, "value": float, "unit": str, "n_gpus": int, "steps": int, "warmup": int,
             "ms_per_step": float, "higher_is_better": bool, "scaling": str, "dtype": str, "data": str,
             "config": dict, "e2e": dict, "cpu_baseline": dict, "gpu_launches": int}


def run_bench(*flags):
    env = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], cwd=ROOT, env=env,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                    # exactly one JSON line
    return json.loads(lines[0])


def check_base(line):
    for k, t in BASE_KEYS.items():
        assert k in line, k
        assert isinstance(line[k], t) or (t is float and isinstance(line[k], int)), (k, line[k])
    assert "vs_baseline" in line and line["vs_baseline"] is None
    assert line["value"] > 0 and line["ms_per_step"] > 0 and "workload" in line["config"]
    assert set(line["e2e"]) >= {"value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"}
    assert set(line["cpu_baseline"]) >= {"value", "unit", "cores", "kind", "sample"}
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1


def test_reference_arm_line():
    line = run_bench("--impl", "reference", "--workload", "cfg1", "--steps", "2", "--warmup", "1", "--cpu-sample", "64")
    check_base(line)
    assert line["impl"] == "reference" and line["dtype"] == "f64" and line["gpu_launches"] == 0
    assert line["steps"] == 2 and line["warmup"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]


def test_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` with no launcher around it starts two ranks itself (CPU ranks over gloo in
    the reference arm); rank 0 prints the one line, which says how many ranks reported in."""
    line = run_bench("--impl", "reference", "--gpus", "2", "--workload", "cfg1", "--steps", "1", "--warmup", "0",
                     "--cpu-sample", "32")
    check_base(line)
    assert line["n_gpus"] == 2 and line["ranks_reported"] == 2


@pytest.mark.gpu
def test_gpu_arm_line():
    line = run_bench("--workload", "cfg1", "--steps", "3", "--warmup", "3", "--hbm-log2", "20", "--cpu-sample", "64")
    check_base(line)
    # the step's result comes back to the host: 4 bytes of log-prob per token besides the loss record
    assert line["e2e"]["d2h_bytes_per_step"] > 4 * 1000
    assert "impl" not in line and line["dtype"] == "bf16" and line["n_gpus"] == 1 and line["scaling"] == "weak"
    assert line["gpu_launches"] > 0 and line["e2e"]["h2d_bytes_per_step"] > 0 and line["e2e"]["d2h_bytes_per_step"] > 0
    roof = line["roofline"]
    assert set(roof) >= {"bound", "achieved", "peak", "unit", "frac", "traffic"}
    assert roof["bound"] == "tensor" and roof["unit"] == "TFLOP/s" and roof["achieved"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    clocks = line["clocks"]
    assert set(clocks) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert set(line["hbm_kernels"]) >= {"pack_microbatch", "policy_loss", "grpo_advantage", "controller_get"}
    assert line["step_ms_rank0"]["min"] <= line["step_ms_rank0"]["median"] <= line["step_ms_rank0"]["max"]


@pytest.mark.gpu
def test_data_parallel_code_path_with_a_process_group_of_one_rank():
    """The exchanges of the data-parallel step -- NCCL all-gather of rewards, advantages by group id, the
    dW all-reduce started by the backward's "d_W ready" event on a second stream -- run on one GPU
    through a process group of one rank (where they change no value)."""
    import math
    line = run_bench("--workload", "cfg4_mini", "--dp-single-rank", "--steps", "3", "--warmup", "3", "--hbm-log2", "20",
                     "--cpu-sample", "64")
    check_base(line)
    dp = line["data_parallel"]
    assert dp["ranks"] == 1 and dp["responses_per_rank"] == 32 and sum(dp["tokens_per_rank"]) == 1024
    assert line["config"]["parallelism"].startswith("dp1")
    assert math.isfinite(line["loss"]) and math.isfinite(line["fused_update"]["loss"])
    assert line["backward"]["ms"] > 0
