"""The trace checker itself, on a hand-made program and trace: accepts a valid trace, rejects each violation."""
import numpy as np
import pytest

from paper_2609_22335_b200.api import TRACE_DTYPE
from trace_check import check_trace, ADMIT_NODE

# a -> b (2 tiles) -> emit
PROGRAM = [dict(name="a", op=0, n_tiles=1, succ=[1]), dict(name="b", op=0, n_tiles=2, succ=[2]),
           dict(name="emit", op=8, n_tiles=1, succ=[])]


def _valid(n_frames=3, depth=2):
    rows = []
    for f in range(n_frames):
        t0 = 1000 * f
        inst = f % depth
        rows += [(inst, ADMIT_NODE, 0, f, t0, t0), (inst, 0, 0, f, t0 + 10, t0 + 20), (inst, 1, 0, f, t0 + 20, t0 + 30),
                 (inst, 1, 1, f, t0 + 25, t0 + 40), (inst, 2, 0, f, t0 + 40, t0 + 50)]
    t = np.zeros(len(rows), dtype=TRACE_DTYPE)
    for i, r in enumerate(rows):
        t[i]["inst"], t[i]["node"], t[i]["tile"], t[i]["frame"], t[i]["t_start"], t[i]["t_end"] = r
    return t


def test_valid_trace_passes():
    t = _valid()
    assert check_trace(t, len(t), PROGRAM, 1, 3) == {"tiles": 12, "admissions": 3}


@pytest.mark.parametrize("what", ["twice", "missing", "edge", "admission", "ring", "slot", "overflow"])
def test_violations_are_caught(what):
    t = _valid()
    total = len(t)
    if what == "twice":
        t[3]["tile"] = 0                      # tile 0 of b ran twice, tile 1 never
    elif what == "missing":
        t = np.delete(t, 3)
        total = len(t)
    elif what == "edge":
        t[2]["t_start"] = 15                  # b starts before a ended
    elif what == "admission":
        t[6]["t_start"] = 999                 # a tile of frame 1 starts before the frame's admission at 1000
    elif what == "ring":
        t[11]["t_start"] = 45                 # first tile of frame 2 before frame 0's emit ended (slot 0 reused)
        t[10]["t_start"] = t[10]["t_end"] = 40
    elif what == "slot":
        t[6]["inst"] = 0                      # a tile of frame 1 ran in slot 0
    elif what == "overflow":
        total = len(t) + 5
    with pytest.raises(AssertionError):
        check_trace(t, total, PROGRAM, 1, 3)
