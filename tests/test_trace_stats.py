"""Trace statistics on hand-made traces with known answers (CPU only)."""
import numpy as np

from paper_2609_22335_b200 import trace_stats as TS
from paper_2609_22335_b200.api import TRACE_DTYPE


def _trace(rows):
    """rows: (sm, worker, cls, node, t_start, t_end[, inst, frame])"""
    t = np.zeros(len(rows), dtype=TRACE_DTYPE)
    for i, r in enumerate(rows):
        t[i]["sm"], t[i]["worker"], t[i]["cls"], t[i]["node"], t[i]["t_start"], t[i]["t_end"] = r[:6]
        if len(r) > 6:
            t[i]["inst"], t[i]["frame"] = r[6], r[7]
    return t


def test_union_and_intersection_lengths():
    s = np.array([0, 5, 20, 22], dtype=np.int64)
    e = np.array([10, 8, 25, 30], dtype=np.int64)
    assert TS._union_length(s, e) == 10 + 10
    assert TS._union_length(s[:0], e[:0]) == 0
    # set A covers [0,10) u [20,30); set B covers [5,22): both = [5,10) u [20,22) = 7
    assert TS._both_length(s, e, np.array([5], dtype=np.int64), np.array([22], dtype=np.int64)) == 7


def test_busy_fraction_and_class_shares():
    # two SMs x one worker, wall 100 ns; SM0 busy 100 (VLM GEMM 60 + head GEMM 40), SM1 busy 50 (VLM attention)
    tr = _trace([(0, 0, 0, 0, 0, 60), (0, 0, 4, 1, 60, 100), (1, 0, 2, 2, 10, 60)])
    assert TS.wall_ns(tr) == 100
    assert abs(TS.busy_fraction(tr) - 150 / 200) < 1e-12
    assert abs(TS.busy_fraction(tr, n_workers=6) - 150 / 600) < 1e-12        # idle worker groups counted
    sh = TS.class_shares(tr)
    assert abs(sh["vlm_gemm"] - 0.4) < 1e-12 and abs(sh["head_gemm"] - 40 / 150) < 1e-12
    assert abs(sh["vlm_attention"] - 50 / 150) < 1e-12 and "head_attention" not in sh


def test_concurrency_fraction_hand_case():
    # overlap window: both phases have started at t=20 (head starts at 20), either has finished at t=100 -> [20,100]
    # SM0: VLM [0,100) on worker 0, head [20,60) on worker 1 -> both for 40 of 80
    # SM1: VLM [0,50) then head [50,100): never both -> 0
    # SM2: head [90,120) worker 0, VLM [80,100) worker 1 -> clipped to the window: both for [90,100) = 10 of 80
    tr = _trace([(0, 0, 0, 0, 0, 100), (0, 1, 4, 1, 20, 60), (1, 0, 0, 0, 0, 50), (1, 0, 5, 1, 50, 100),
                 (2, 0, 6, 1, 90, 120), (2, 1, 1, 0, 80, 100)])
    assert TS.overlap_window(tr) == (20, 100)
    c = TS.concurrency_fraction(tr)
    assert c["window_ns"] == 80
    assert abs(c["mean"] - (0.5 + 0.0 + 0.125) / 3) < 1e-12 and c["max"] == 0.5 and c["min"] == 0.0
    # SMs that never ran a tile pull the mean down when the SM count is given
    assert abs(TS.concurrency_fraction(tr, n_sms=6)["mean"] - (0.5 + 0.125) / 6) < 1e-12
    # one phase only -> no overlap window
    assert TS.concurrency_fraction(_trace([(0, 0, 0, 0, 0, 10)]))["mean"] == 0.0


def test_admission_markers_are_not_tiles():
    tr = _trace([(0, 0, 0, TS.ADMIT_NODE, 0, 0), (0, 0, 0, 0, 5, 15)])
    assert len(TS.tiles_only(tr)) == 1 and TS.wall_ns(tr) == 10


def test_per_class_rates_and_pairs():
    program = [dict(n_tiles=2, flops=4e6, weight_bytes=2e3, phase=0), dict(n_tiles=1, flops=1e3, weight_bytes=5e4, phase=1)]
    # node 0 (VLM GEMM): two tiles of 1000 ns, 2e6 FLOP each -> 2e6 / 1e-6 s = 2 TFLOP/s per worker
    # node 1 (head GEMM): one tile of 500 ns streaming 5e4 bytes -> 100 GB/s per worker
    tr = _trace([(0, 0, 0, 0, 0, 1000, 0, 0), (1, 0, 0, 0, 0, 1000, 0, 0), (0, 1, 4, 1, 200, 700, 1, 0)])
    r = TS.per_class_rates(tr, program, n_workers=4)
    assert abs(r["vlm_gemm"]["tflops_all_workers"] - 8.0) < 1e-9 and r["vlm_gemm"]["tiles"] == 2
    assert abs(r["head_gemm"]["weight_gbs_all_workers"] - 400.0) < 1e-9
    assert abs(r["head_gemm"]["mean_tile_us"] - 0.5) < 1e-12
    p = TS.smaller_side_of_concurrent_pairs(tr, program)
    assert p["pairs"] == 1 and p["one_tile"] == 1.0 and p["median"] == 1.0
    s = TS.summary(tr, program, n_sms=2, workers_per_sm=2)
    assert s["tiles"] == 3 and abs(s["sm_busy_frac"] - 2500 / (4 * 1000)) < 1e-12


def test_gap_stats():
    # worker (0,0): VLM GEMM [0,10), head GEMM [14,20), VLM GEMM [20,30): gaps 4 (before a head tile) and 0 (before a VLM tile)
    # worker (1,0): head GEMM [0,5), head GEMM [11,12): gap 6
    tr = _trace([(0, 0, 0, 0, 0, 10), (0, 0, 4, 1, 14, 20), (0, 0, 0, 0, 20, 30), (1, 0, 4, 1, 0, 5), (1, 0, 4, 1, 11, 12)])
    g = TS.gap_stats(tr)
    assert g["all"]["gaps"] == 3 and abs(g["all"]["mean_us"] - 10 / 3 * 1e-3) < 1e-12
    assert g["head_gemm"]["gaps"] == 2 and abs(g["head_gemm"]["mean_us"] - 5e-3) < 1e-12 and g["head_gemm"]["share_of_idle"] == 1.0
    assert g["vlm_gemm"]["gaps"] == 1 and g["vlm_gemm"]["mean_us"] == 0.0


def test_backlog_stats_hand_case():
    # node 0 (two tiles) -> node 1 (one tile); the frame is admitted at t = 0
    program = [{"n_tiles": 2, "phase": 0, "succ": [1]}, {"n_tiles": 1, "phase": 1, "succ": []}]
    tr = _trace([(0, 0, 0, TS.ADMIT_NODE, 0, 0, 0, 0),
                 (0, 0, 0, 0, 10, 50, 0, 0), (0, 1, 0, 0, 10, 30, 0, 0),     # node 0: ready at 0, both tiles start at 10
                 (0, 1, 4, 1, 60, 80, 0, 0)])                                # node 1: ready at 50 (last end of node 0), starts at 60
    b = TS.backlog_stats(tr, program, n_workers=2)
    assert b["wait_ready_to_start_us"]["vlm"]["mean"] == 10e-3 and b["wait_ready_to_start_us"]["head"]["mean"] == 10e-3
    # backlog: 2 tiles over [0,10), none over [10,50), 1 over [50,60) -> (20 + 10) / 60
    assert abs(b["mean_backlog_tiles"] - 30 / 60) < 1e-12
    # the one idle interval, worker (0,1) from 30 to 60: nothing was ready until 50 (three of the four sample points)
    idle = b["idle_between_tiles"]
    assert abs(idle["share_with_empty_backlog"] - 0.75) < 1e-12 and abs(idle["share_with_deep_backlog"] - 0.25) < 1e-12
    # and the summary carries it when the program lists successors
    s = TS.summary(tr, [dict(p, flops=0.0, weight_bytes=0.0) for p in program], n_sms=1, workers_per_sm=2)
    assert "backlog" in s
