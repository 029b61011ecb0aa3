"""Tag derivation from a profiling log (CPU only): the ncu CSV reader and the quantisation of Section 3.2.2."""
import os

import pytest

from paper_2609_22335_b200 import auto_tags as AT
from oracle.admission_oracle import quantise_tau

HEADER = '"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"'


def _row(i, kernel, grid, metric, value):
    return f'"{i}","1","python","h","{kernel}","1","7","(128, 1, 1)","({grid}, 1, 1)","0","10.0","Command line profiler metrics","{metric}","%","{value}"'


def _csv(tmp_path, launches):
    lines = ["==PROF== Connected to process 1", HEADER]
    for i, (kernel, grid, vals) in enumerate(launches):
        for m, v in zip(AT.METRICS, vals):
            lines.append(_row(i, kernel, grid, m, v))
    p = tmp_path / "l.csv"
    p.write_text("\n".join(lines) + "\n")
    return str(p)


def test_quantise_matches_the_oracles_rule():
    for u in (0.0, 0.03, 0.0334, 0.374, 0.5, 0.97, 1.0, 1.7):
        assert AT.quantise(u) == quantise_tau(u)


def test_derive_from_a_hand_made_log(tmp_path):
    node = "vla_node_kernel(DeviceCtx, const NodeDesc *, int, int)"
    launches = [("vla_fold_gain_kernel(...)", 592, (0, 0, 50)),      # other kernels are ignored
                (node, 1, (0, 0, 0)),                                  # load-time constant program: before the frame
                (node, 148, (40.0, 10.0, 20.0)),                       # node 0: VLM GEMM, a tile on every SM
                (node, 296, (60.0, 10.0, 40.0)),                       # node 1: VLM GEMM, two waves
                (node, 37, (4.0, 16.0, 10.0))]                         # node 2: head GEMM on 37 of 148 SMs
    program = [dict(cls=0, n_tiles=148), dict(cls=0, n_tiles=296), dict(cls=4, n_tiles=37)]
    tags, detail = AT.derive(AT.read_launches(_csv(tmp_path, launches)), program, n_sms=148)
    # class 0: tile-weighted means u_tc = (148*0.4 + 296*0.6)/444 = 0.5333, u_alu = 0.1, u_mem = (148*0.2 + 296*0.4)/444 = 0.3333
    assert tags[0] == [8, 2, 5] and abs(detail[0]["u_tc"] - 0.53333) < 1e-4
    # class 4: DRAM share scaled from 37 to 148 SMs: 0.10 * 4 = 0.4 -> 6; tensor 0.04 -> 1; alu 0.16 -> 2
    assert tags[4] == [1, 2, 6]
    assert tags[1] is None and tags[7] is None                         # classes the frame does not exercise
    rel = AT.relative_tags(detail)                                     # heaviest class per pipeline -> 15
    assert rel[0] == [15, 9, 12] and rel[4] == [1, 15, 15] and rel[1] is None
    with pytest.raises(ValueError):                                    # a window that does not line up is refused
        AT.derive(AT.read_launches(_csv(tmp_path, launches)), [dict(cls=0, n_tiles=5)] * 3, n_sms=148)


def test_command_line_names_the_metrics_and_keeps_the_clocks():
    cmd = AT.ncu_command("cfg2")
    assert "--clock-control none" in cmd and all(m in cmd for m in AT.METRICS) and "regex:vla_node_kernel" in cmd
