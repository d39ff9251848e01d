"""The batched-workload runner end to end on a few-block cut of each shape (GPU)."""
import json
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("args", [["c3", "--layers", "4"], ["c4", "--layers", "2", "--exec", "tensor"],
                                  ["c5", "--layers", "2", "--rows", "1", "--exec", "fused"]],
                         ids=["c3", "c4-tensor", "c5-single-row-fused"])
def test_workload_runner_prints_a_consistent_line(args):
    out = subprocess.run([sys.executable, "-m", "paper_2503_08524_b200.workloads", *args, "--steps", "3",
                          "--profile"], capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["workload"] == args[0] and line["steps"] == 3
    assert line["ms_per_step"] > 0 and line["tokens_per_s"] > 0
    assert abs(line["achieved_gbs"] - line["algorithmic_gb_per_step"] * 1e3 / line["ms_per_step"]) < 1.0
    assert 0 < line["frac_of_hbm_peak"] < 1.5
    layers = int(args[2])
    assert 0 < line["layers_touched_per_step"] <= layers
    assert line["rows_layers_per_step"] <= line["rows"] * layers
    assert line["kernel_classes"]
    if "fused" in args:
        assert line["launches_per_step"] == 1 and "fused_step" in line["kernel_classes"]
    else:
        assert line["launches_per_step"] > 1 and "attention" in line["kernel_classes"]
