"""Host logic of bench.py that needs no GPU: the recall measures against hand-made answers, the
algorithmic-byte formula, the tracked DRAM-traffic table, the workload strings both arms share, and
the reference arm under a launcher (rank 0 prints the line, other ranks do nothing)."""
import json
import os
import subprocess
import sys

import numpy as np

import bench

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_recall_measures_on_hand_made_rows():
    gt = np.array([[1, 2, 3, 4], [5, 6, -1, -1], [-1, -1, -1, -1]], dtype=np.int32)
    ids = np.array([[4, 9, 1, 8], [6, 5, -1, -1], [-1, -1, -1, -1]], dtype=np.int32)
    # row 0: 2 of 4; row 1: 2 of 2; row 2 has no true neighbour and does not count
    assert bench.recall_at_k(ids, gt) == (0.5 + 1.0) / 2
    gt_d = np.array([[1.0, 2.0, 2.0, 3.0], [1.0, np.inf, np.inf, np.inf]], dtype=np.float32)
    d = np.array([[1.0, 2.0, 3.0, 3.5], [2.0, np.inf, np.inf, np.inf]], dtype=np.float32)
    # row 0: three distances within the 4th true one (3.0) of four; row 1: none within 1.0 of one
    assert bench.recall_tie_aware(d, gt_d) == (0.75 + 0.0) / 2


def test_algorithmic_bytes_formula():
    # two queries: 3 and 5 ENC rows scanned, 10 and 20 distances; n = 1024, d = 96 (row 384 B), m = 16, k = 10
    st = np.array([[7, 3, 0, 10], [9, 5, 0, 20]], dtype=np.uint32)
    per_query = 4 * 96 + 8 * 10 + 8 * 10
    assert bench.algorithmic_bytes(st, 1024, 96, 96, 16, 10) == 2 * per_query + 64 * 8 + 384 * 30


def test_traffic_table_is_read_by_exact_operating_point():
    assert os.path.exists(bench.TRAFFIC_TABLE)
    rows = [ln.split() for ln in open(bench.TRAFFIC_TABLE) if ln.strip() and not ln.startswith("#")]
    assert rows and all(len(r) >= 8 for r in rows)
    for r in rows:
        name, ranges = r[0].split(":")
        assert ranges == "mixed"
        got = bench.ncu_traffic(name, int(r[1]), int(r[2]), int(r[3]), int(r[4]))
        assert got == float(r[5])
        assert bench.ncu_traffic(name, int(r[1]), int(r[2]), int(r[3]), int(r[4]) + 1) is None
        assert bench.ncu_traffic(name, int(r[1]), int(r[2]), int(r[3]), int(r[4]), fraction=2.0 ** -7) is None
        assert os.path.exists(os.path.join(ROOT, "profiles", r[7]))      # the summary that holds the command


def test_workload_strings():
    import datagen
    wl = datagen.make_workload("tiny", n=500, nq=3)
    assert bench.workload_text(wl) == "tiny: n=500 d=32 nq=3 k=10 mixed selectivity (width fraction log-uniform 2^-8..1)"
    assert bench.workload_text(wl, 2.0 ** -4).endswith("fixed width fraction 2^-4")


def test_reference_arm_prints_one_line_on_rank_0_only(libs, tmp_path):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny", "--n", "3000",
           "--nq", "40", "--steps", "2", "--warmup", "1", "--builder", "cpu", "--cache-dir", str(tmp_path)]
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["unit"] == "queries/s" and j["value"] > 0 and j["steps"] == 2
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["value"] == j["value"]
    assert j["e2e"] == {"value": j["value"], "unit": "queries/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert j["config"]["workload"].startswith("tiny: n=3000")
    env["RANK"] = env["LOCAL_RANK"] = "1"
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and out.stdout.strip() == ""
