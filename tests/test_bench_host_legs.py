"""The host-only legs of bench.py (the oracle timed beside a workload, the global autoscaler
simulation on an instance model) run without a GPU: their output must carry what the bench line
promises, so that a change in the library's host API cannot silently cost the line at the end of
a long GPU run."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


@pytest.fixture(scope="module")
def bench():
    from paper_2501_08090_b200 import build
    build.build()
    import bench as b
    return b


def test_oracle_beside_reports_a_bounded_sample(bench):
    out = bench.oracle_beside("mixed_sweep", batch=8, max_tokens=3000, passes=1)
    assert out["kind"] == "oracle" and out["unit"] == "TB/s" and out["cores"] >= 1
    assert out["value"] > 0 and out["us_per_step_extrapolated"] > 0
    assert "of 8 requests" in out["sample"] and "tokens" in out["sample"]
    long_one = bench.oracle_beside("skewed_long", max_tokens=2000, passes=1)      # one request far above the bound
    assert long_one["value"] > 0 and "of 8 requests" in long_one["sample"]


def test_global_simulation_leg_runs_on_an_instance_model(bench):
    local = {"runs": [{"itl_slo_ms": 200.0, "peak_batch": 400, "trough_batch": 200, "max_itl_ms": 190.0},
                      {"itl_slo_ms": 2000.0, "peak_batch": 4000, "trough_batch": 2000, "max_itl_ms": 1900.0}]}
    out = bench.run_global_simulation(local)
    assert out["requests"] == 4000 and len(out["policies"]) == 2
    chiron, immediate = out["policies"]
    assert chiron["interactive_ttft_met"] == 1.0 and chiron["batch_ttft_met"] == 1.0
    assert chiron["instance_hours"][2] <= immediate["instance_hours"][2]
    assert chiron["events"] > 4000 * 3
