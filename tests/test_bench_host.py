"""Host-side pieces of bench.py that need no GPU: the algorithmic-byte formulas against the
per-index counts of the state layout, and the reference arm's JSON line."""
import json
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
import bench  # noqa: E402


@pytest.mark.parametrize("M", [1, 2, 4, 8, 16])
def test_algorithmic_bytes(M):
    # every state word read once and written once; fp32 = 4 B, bf16 = 2 B
    assert bench.outer_bytes_per_param(2, M, 0) == 32 * M + 8       # theta, start, stale local, momentum + stale mean
    assert bench.outer_bytes_per_param(1, M, 0) == 24 * M + 8
    assert bench.outer_bytes_per_param(0, M, 0) == 24 * M
    assert bench.outer_bytes_per_param(2, M, 1) == 28 * M + 8       # bf16 theta
    assert bench.outer_bytes_per_param(2, M, 2) == 34 * M + 8       # master read, master + bf16 copy written
    assert bench.adamw_bytes_per_param(M, 0, 0) == 28 * M
    assert bench.adamw_bytes_per_param(M, 1, 1) == 22 * M
    assert bench.adamw_bytes_per_param(M, 2, 1) == 28 * M


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1",
                          "--P", "200000"], capture_output=True, text=True, timeout=300, check=True).stdout
    lines = [l for l in out.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["value"] > 0 and d["gpu_launches"] == 0


def test_both_arms_describe_the_workload_identically():
    """The GPU arm and the CPU reference arm must print the same `config` for the same command
    line, so that a reader (or a driver) comparing the two lines sees one workload."""
    import argparse
    from paper_2502_12996_b200 import inputs
    args = argparse.Namespace(workload=bench.DEFAULT_WORKLOAD, variant="eager", outer_only=False, strong=False, kernel=0,
                              comm="f32", M=0)
    w = inputs.WORKLOADS[bench.DEFAULT_WORKLOAD]
    cfg = bench.config_dict(args, w, w.P)
    assert cfg["workload"] == "cfg4a" and cfg["M"] == 2 and cfg["P_per_gpu"] == 2_400_000_000
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "1",
                          "--workload", "cfg0"], capture_output=True, text=True, timeout=300, check=True).stdout
    d = json.loads(out.strip().splitlines()[-1])
    args.workload = "cfg0"
    assert d["config"] == bench.config_dict(args, inputs.WORKLOADS["cfg0"], inputs.WORKLOADS["cfg0"].P)
    assert "cold-L2" in d["config"]["l2"]                         # 37.7 MB of state: smaller than L2
    assert "state >> 126 MB L2" in cfg["l2"]


def test_traffic_table_parses():
    table = bench.load_traffic()
    assert ("outer", "eager", 4, 0) in table
    for (kernel, variant, M, kind), (bpp, source) in table.items():
        assert kernel in ("outer", "adamw") and 1 <= M <= 64 and kind in (0, 1, 2) and bpp > 0
        assert (ROOT / "profiles" / source).exists(), source


def test_oracle_sample_is_bounded():
    from paper_2502_12996_b200 import inputs
    for w in inputs.WORKLOADS.values():
        n = bench.oracle_sample_size(w, w.P)
        assert n <= w.P and n * w.M <= 140_000_000
