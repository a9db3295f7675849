"""Host-side logic of bench.py that needs no GPU: interval arithmetic of the overlap fraction, the
clock-sample parser, the algorithmic byte counts and the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_1906_12043_b200 import workloads as W  # noqa: E402


def test_overlap_fraction_is_the_share_of_mean_time_inside_local_steps():
    by = {"local_step": [(0.0, 1.0), (1.5, 2.5)], "mean": [(0.5, 1.75)]}
    # mean lives 1.25; inside steps: [0.5, 1.0] + [1.5, 1.75] = 0.75
    assert bench.overlap_fraction(by) == pytest.approx(0.6)
    assert bench.overlap_fraction({"local_step": [(0, 1)], "mean": [(2, 3)]}) == 0.0
    assert bench.overlap_fraction({"local_step": [(0, 4)], "mean": [(1, 2), (3, 3.5)]}) == 1.0
    assert bench.overlap_fraction({"local_step": [(0, 1)]}) is None


def test_profile_records_are_grouped_by_kernel_name():
    names = {0: "local_step", 2: "mean", 3: "merge"}
    by = bench.summarize_profile([(2, 0.0, 0.1), (0, 0.0, 0.5), (0, 0.5, 1.0), (3, 1.0, 1.3)], names)
    assert by == {"mean": [(0.0, 0.1)], "local_step": [(0.0, 0.5), (0.5, 1.0)], "merge": [(1.0, 1.3)]}


def test_algorithmic_bytes_of_a_round():
    wl = W.WORKLOADS["resnet18"]
    n = wl.K * wl.P
    # k local steps of 20 B, mean 4 (1 + 1/K) B, merge 12 + 4/K B per worker-parameter; + 8 B with a copy
    assert wl.bytes_per_round() == (20 * wl.k + 16) * n + 8 * wl.P
    assert wl.bytes_per_round(snapshot_copy=True) - wl.bytes_per_round() == 8 * n
    assert W.bytes_mean(16) * n + W.bytes_merge(16) * n == pytest.approx(16 * n + 8 * wl.P)
    assert W.WORKLOADS["vgg16"].K * W.WORKLOADS["vgg16"].P > 2 ** 31


def test_clock_sampler_parses_nvidia_smi_lines(monkeypatch):
    class FakeProc:
        def terminate(self):
            pass

        def communicate(self, timeout=None):
            return ("1965, 1965, 412.5, 0x0000000000000000, Not Active, Not Active, Not Active, Not Active\n"
                    "1687, 1965, 998.1, 0x0000000000000004, Not Active, Not Active, Not Active, Active\n"
                    "1650, 1965, 1001.3, 0x0000000000000004, Not Active, Not Active, Not Active, Active\n"
                    "garbage line\n", "")

    s = bench.ClockSampler.__new__(bench.ClockSampler)
    s.proc = FakeProc()
    out = s.stop()
    assert out["sm_mhz"] == 1687.0 and out["sm_max_mhz"] == 1965.0 and out["samples"] == 3
    assert out["reasons"] == ["sw_power_cap"]


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` times the CPU oracle on a bounded column sample (tiny here)."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "3", "--warmup", "1", "--cpu-sample-cols", "4096"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "updates/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"] == {"value": line["value"], "unit": "updates/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"] == "tiny" and line["higher_is_better"] is True


def test_reference_arm_of_the_mlp_workload_prints_the_contract_line():
    """The MLP workload's reference arm: rounds of the oracle on a sample of two workers."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "mlp",
                          "--steps", "1", "--warmup", "0", "--k", "1"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["config"]["workload"] == "mlp" and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"] > 0
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
