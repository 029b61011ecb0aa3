"""The pick of the persistent kernel (csrc/pick.cuh), compiled for the host, against the Algorithm 1 oracle.

With one class per group it must be the paper's listing exactly (Section 3.3, Algorithm 1); with several classes
per group Phase 1 is decided per group (a group = the tiles of one phase, the paper's "kernel").
"""
import ctypes as C
import os
import random
import subprocess

import pytest

from oracle.admission_oracle import SMState, admission_decision

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def pick_lib(tmp_path_factory):
    out = tmp_path_factory.mktemp("pick") / "libpick_host.so"
    subprocess.run(["g++", "-O1", "-shared", "-fPIC", "-x", "c++", os.path.join(HERE, "pick_host_shim.cc"), "-o", str(out)],
                   check=True)
    lib = C.CDLL(str(out))
    lib.pick_host.argtypes = [C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_uint, C.c_uint, C.POINTER(C.c_int),
                              C.POINTER(C.c_int), C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int),
                              C.POINTER(C.c_int)]
    lib.pick_host.restype = C.c_int
    return lib


def _call(lib, taus, group, pending, feasible, cta, u, rr, policy, u_max, grid=None, res=None):
    n = len(taus)
    tau = (C.c_int * (3 * n))(*[x for t in taus for x in t])
    grp = (C.c_int * n)(*group)
    cc = (C.c_int * n)(*cta)
    uu = (C.c_int * 3)(*u)
    pm = sum(1 << k for k in range(n) if pending[k])
    fm = sum(1 << k for k in range(n) if feasible[k])
    phase = C.c_int(0)
    gg = (C.c_int * n)(*grid) if grid is not None else None
    rs = (C.c_int * n)(*res) if res is not None else None
    k = lib.pick_host(n, tau, grp, pm, fm, cc, uu, rr, policy, u_max, C.byref(phase), gg, rs)
    return k, phase.value, list(cc), list(uu)


def test_one_class_per_group_is_algorithm_1(pick_lib):
    rnd = random.Random(5)
    for _ in range(400):
        n = rnd.randint(1, 8)
        taus = [tuple(rnd.randint(0, 15) for _ in range(3)) for _ in range(n)]
        st = SMState(n)
        st.cta_count = [rnd.randint(0, 2) for _ in range(n)]
        st.u = [sum(st.cta_count[k] * taus[k][x] for k in range(n)) for x in range(3)]
        pending = [rnd.random() < 0.7 for _ in range(n)]
        feas = [rnd.random() < 0.7 for _ in range(n)]
        rr = rnd.randint(0, n - 1)
        u_max = rnd.choice([255, 45, 30])
        k, ph, cc, uu = _call(pick_lib, taus, list(range(n)), pending, feas, st.cta_count, st.u, rr, 0, u_max)
        ko, pho = admission_decision(st, taus, pending, feas, rr_start=rr, u_max=u_max)
        assert k == (-1 if ko is None else ko) and ph == pho
        assert cc == st.cta_count and [min(v, u_max) for v in uu] == [min(v, u_max) for v in st.u]


def test_phase_1_is_decided_per_group(pick_lib):
    # classes 0..3 = group 0 (VLM), 4..7 = group 1 (action head); a VLM GEMM is resident, nothing of the head is
    taus = [(15, 2, 3), (15, 4, 3), (8, 8, 2), (0, 4, 10), (2, 3, 12), (2, 4, 12), (1, 8, 4), (0, 3, 6)]
    group = [0, 0, 0, 0, 1, 1, 1, 1]
    cta = [1, 0, 0, 0, 0, 0, 0, 0]
    u = list(taus[0])
    pending = [True, False, True, False, False, False, True, False]     # VLM GEMM, VLM attention, head attention
    feas = [True] * 8
    # Phase 1: the head's group is not represented on this SM -> its pending class wins although its tags score lowest
    k, ph, _, _ = _call(pick_lib, taus, group, pending, feas, cta, u, 0, 0, 45)
    assert (k, ph) == (6, 1)
    # VLM attention (class 2) has no tile resident, but its GROUP has: it is not a Phase-1 candidate
    pending2 = [True, False, True, False, False, False, False, False]
    k, ph, _, _ = _call(pick_lib, taus, group, pending2, feas, cta, u, 0, 0, 45)
    assert ph == 2 and k == 2          # Phase 2: complementary to the resident tensor-heavy tile
    # with the hardware's 255 the headroom hardly moves and the tensor-heavy class keeps winning
    k, ph, _, _ = _call(pick_lib, taus, group, pending2, feas, cta, u, 0, 0, 255)
    assert ph == 2 and k == 0
    # an infeasible class is never picked; nothing pending -> nothing
    k, ph, _, _ = _call(pick_lib, taus, group, pending, [True] * 6 + [False, True], cta, u, 0, 0, 45)
    assert k in (0, 2) and ph == 2
    assert _call(pick_lib, taus, group, [False] * 8, feas, cta, u, 0, 0, 45)[:2] == (-1, 0)


def test_other_policies(pick_lib):
    taus = [(1, 1, 1)] * 4
    group = [0, 1, 2, 3]
    pending = [False, True, True, True]
    feas = [True, True, False, True]
    assert _call(pick_lib, taus, group, pending, feas, [0] * 4, [0] * 3, 2, 1, 45)[0] == 1     # class order
    assert _call(pick_lib, taus, group, pending, feas, [0] * 4, [0] * 3, 2, 2, 45)[0] == 3     # round robin from 2: 2 is infeasible


def test_score_variants_match_the_oracle(pick_lib):
    """-G (policy 3) and -R (policy 4): exact agreement with the oracle's rational comparison, ties included."""
    rnd = random.Random(21)
    for _ in range(600):
        n = rnd.randint(1, 8)
        taus = [tuple(rnd.randint(0, 15) for _ in range(3)) for _ in range(n)]
        st = SMState(n)
        st.cta_count = [rnd.randint(0, 3) for _ in range(n)]
        st.u = [sum(st.cta_count[k] * taus[k][x] for k in range(n)) for x in range(3)]
        pending = [rnd.random() < 0.8 for _ in range(n)]
        feas = [rnd.random() < 0.8 for _ in range(n)]
        rr = rnd.randint(0, n - 1)
        u_max = rnd.choice([255, 45])
        grid = [rnd.choice([1, 2, 5, 30, 444, 100000]) for _ in range(n)]
        res = [rnd.choice([1, 12, 16, 18, 36]) for _ in range(n)]
        for policy, variant in ((3, "G"), (4, "R")):
            k, ph, cc, uu = _call(pick_lib, taus, list(range(n)), pending, feas, st.cta_count, st.u, rr, policy, u_max, grid, res)
            so = st.copy()
            ko, pho = admission_decision(so, taus, pending, feas, rr_start=rr, u_max=u_max, variant=variant, grid=grid, regs=res)
            assert k == (-1 if ko is None else ko) and ph == pho, (variant, taus, st.cta_count, grid, res)
            assert cc == so.cta_count
    # the hand-derived cases of the oracle's pins, through the device header
    taus = [(15, 2, 3), (0, 4, 9)]
    assert _call(pick_lib, taus, [0, 1], [1, 1], [1, 1], [1, 1], [15, 6, 12], 0, 3, 255, [2, 30], [1, 1])[:2] == (1, 2)
    assert _call(pick_lib, taus, [0, 1], [1, 1], [1, 1], [1, 1], [15, 6, 12], 0, 3, 255, [8, 8], [1, 1])[:2] == (0, 2)
    assert _call(pick_lib, taus, [0, 1], [1, 1], [1, 1], [1, 1], [15, 6, 12], 0, 4, 255, [1, 1], [64, 32])[:2] == (1, 2)
    assert _call(pick_lib, taus, [0, 1], [1, 1], [1, 1], [1, 1], [15, 6, 12], 0, 4, 255, [1, 1], [48, 48])[:2] == (0, 2)
