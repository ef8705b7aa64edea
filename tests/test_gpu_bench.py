"""bench.py on small cases, in-process: every leg prints one JSON line with the keys the
measurement contract names, and its figures hang together."""
import json

import pytest

from gpu_util import require_gpu

pytestmark = pytest.mark.gpu

COMMON = ["--steps", "3", "--repeats", "2", "--warmup", "3", "--no-cpu-baseline"]


def run_bench(capsys, argv):
    import bench
    require_gpu()
    bench.run_ours(bench.parse_args(argv + COMMON))
    lines = [l for l in capsys.readouterr().out.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def check_common(line, units):
    assert line["metric"] == "DPPF consensus rounds/s" and line["unit"] == "rounds/s"
    assert line["value"] > 0 and line["ms_per_step"] > 0 and line["higher_is_better"] is True
    assert line["steps"] == 3 and line["repeats"] == 2 and line["warmup"] == 3
    assert line["dtype"] == "f32" and line["data"] == "synthetic" and line["vs_baseline"] is None
    assert abs(line["value"] - 1e3 / line["ms_per_step"]) <= 1e-6 * line["value"]
    lo, hi = line["ms_per_step_min_max"]
    assert lo <= line["ms_per_step"] <= hi
    roof = line["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 1000
    assert roof["algorithmic_bytes_per_launch"] == units * line["config"]["replica_bytes"]
    assert 0 < roof["frac"] < 2.0 and abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert "sm_mhz" in line["clocks"] and isinstance(line["clocks"]["reasons"], list)
    assert line["gpu_launches"] >= line["steps"] * line["repeats"]
    assert "workload" in line["config"] and "model" not in line["config"]


def test_plain_round_line_with_multi_round_and_end_to_end(capsys):
    line = run_bench(capsys, ["--workload", "C4", "--d", "3000003", "--rounds-per-call", "7", "--multi-round-calls", "2",
                              "--e2e-steps", "2"])
    check_common(line, 3)
    assert line["scaling"] == "weak" and line["n_gpus"] == 1 and line["config"]["variant"] == "plain"
    mr = line["multi_round"]
    B = line["config"]["replica_bytes"]
    assert mr["rounds_per_call"] == 7 and mr["algorithmic_bytes_per_call"] == 15 * B and mr["value"] > 0
    assert abs(mr["frac"] - mr["achieved"] / mr["peak"]) < 1e-9
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] == B and e2e["d2h_bytes_per_step"] == B + 16
    assert e2e["value"] < line["value"]                     # the copies are inside its timed region
    assert len(line["norms_last_round"]) == 4


@pytest.mark.parametrize("argv,units,variant", [
    (["--workload", "C3", "--d", "2000003"], 7, "plain"),
    (["--workload", "C2", "--d", "1000003", "--variant", "general"], 3, "general"),
    (["--workload", "C4", "--d", "2000003", "--variant", "adamw"], 9, "adamw"),
])
def test_fused_general_and_adamw_lines(capsys, argv, units, variant):
    line = run_bench(capsys, argv)
    check_common(line, units)
    assert line["config"]["variant"] == variant and "multi_round" not in line


def test_column_shard_line_on_one_gpu(capsys):
    line = run_bench(capsys, ["--workload", "C4", "--d", "2000003", "--shard", "columns"])
    check_common(line, 3)
    assert line["scaling"] == "strong" and "column shards" in line["parallelism"]
    assert line["gpu_launches"] == 3 * 2 * 3                # distance, sum, update per step


def test_worker_per_gpu_line_on_one_gpu(capsys):
    line = run_bench(capsys, ["--workload", "C4", "--d", "2000003", "--shard", "workers"])
    assert line["roofline"]["algorithmic_bytes_per_launch"] == 5 * 2000003 * 4
    assert line["scaling"] == "strong" and "one replica" in line["parallelism"]
    assert line["gpu_launches"] == 3 * 2 and 0 < line["roofline"]["frac"] < 2.0 and len(line["norms_last_round"]) == 1
