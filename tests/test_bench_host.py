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
