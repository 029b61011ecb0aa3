"""Pins of the admission-decision oracle (paper Algorithm 1, Section 3.3) on hand-derived cases."""
import random

from fractions import Fraction

from oracle.admission_oracle import (SMState, admission_decision, admit, complete, score, quantise_tau, variant_score,
                                     U_MAX, TAU_MAX)


def test_hand_derived_sequence():
    # kernels A tau=(15,2,3), B tau=(0,4,9), both pending and feasible, empty SM
    taus = [(15, 2, 3), (0, 4, 9)]
    st = SMState(2)
    assert admission_decision(st, taus, [True, True], [True, True]) == (0, 1)     # Phase 1 admits A
    assert admission_decision(st, taus, [True, True], [True, True]) == (1, 1)     # Phase 1 admits B
    assert st.u == [15, 6, 12]
    # Phase 2: s_A = 240*15 + 249*2 + 243*3 = 4827 ; s_B = 249*4 + 243*9 = 3183
    assert score(st, taus[0]) == 4827 and score(st, taus[1]) == 3183
    assert admission_decision(st, taus, [True, True], [True, True]) == (0, 2)
    assert st.cta_count == [2, 1] and st.u == [30, 8, 15]


def test_paper_arithmetic_identities():
    # 17 co-resident CTAs at tau = 15 reach the cap exactly (Section 3.3.2)
    st = SMState(1)
    for _ in range(17):
        admit(st, 0, (15, 0, 0))
    assert st.u[0] == 17 * 15 == U_MAX
    admit(st, 0, (15, 0, 0))
    assert st.u[0] == U_MAX                                                        # saturates
    # 3 x 8-bit registers + 2 x 6-bit counters = 36 bits; 170 SMs -> 765 bytes (Section 3.4.2)
    assert 3 * 8 + 2 * 6 == 36 and 170 * 36 // 8 == 765


def test_ties_keep_first_seen_and_infeasible_never_admitted():
    taus = [(5, 5, 5), (5, 5, 5), (15, 15, 15)]
    st = SMState(3)
    st.cta_count = [1, 1, 1]                                                        # everyone resident -> Phase 2
    k, ph = admission_decision(st, taus, [True, True, True], [True, True, False])
    assert (k, ph) == (0, 2)                                                        # tie -> first seen; kernel 2 infeasible
    st2 = SMState(3)
    assert admission_decision(st2, taus, [True] * 3, [False] * 3) == (None, 0)
    assert st2.cta_count == [0, 0, 0] and st2.u == [0, 0, 0]
    # not pending -> never admitted even if feasible
    assert admission_decision(SMState(3), taus, [False, False, True], [True, True, True]) == (2, 1)


def test_phase1_before_phase2_and_round_robin_start():
    taus = [(15, 0, 0), (0, 1, 1)]
    st = SMState(2)
    st.cta_count = [3, 0]
    st.u = [45, 0, 0]
    # kernel 1 scores far lower but is unrepresented -> Phase 1 picks it
    assert score(st, taus[1]) < score(st, taus[0])
    assert admission_decision(st, taus, [True, True], [True, True]) == (1, 1)
    # rotated Phase-1 scan start
    st = SMState(3)
    assert admission_decision(st, [(1, 1, 1)] * 3, [True] * 3, [True] * 3, rr_start=2) == (2, 1)
    assert admission_decision(st, [(1, 1, 1)] * 3, [True] * 3, [True] * 3, rr_start=2) == (0, 1)


def test_phase2_prefers_complementary_pipeline():
    # SM busy on the tensor pipe: a memory-heavy kernel outscores a tensor-heavy one of equal total intensity
    taus = [(12, 1, 1), (1, 1, 12)]
    st = SMState(2)
    st.cta_count = [1, 1]
    st.u = [200, 10, 10]
    assert admission_decision(st, taus, [True, True], [True, True]) == (1, 2)


def test_random_invariants():
    rnd = random.Random(7)
    for _ in range(200):
        n = rnd.randint(1, 5)
        taus = [tuple(rnd.randint(0, TAU_MAX) for _ in range(3)) for _ in range(n)]
        st = SMState(n)
        resident = []
        for _ in range(12):                      # stays below saturation: 12 * 15 < 255
            pending = [rnd.random() < 0.7 for _ in range(n)]
            feas = [rnd.random() < 0.7 for _ in range(n)]
            before = st.copy()
            k, ph = admission_decision(st, taus, pending, feas)
            if k is None:
                assert not any(p and f for p, f in zip(pending, feas))
                assert st.u == before.u and st.cta_count == before.cta_count
                continue
            assert pending[k] and feas[k]
            assert sum(st.cta_count) == sum(before.cta_count) + 1                  # at most one admission
            if ph == 2:                          # Phase 2 only when no unrepresented feasible pending kernel exists
                assert not any(pending[j] and feas[j] and before.cta_count[j] == 0 for j in range(n))
                best = max(score(before, taus[j]) for j in range(n) if pending[j] and feas[j])
                assert score(before, taus[k]) == best
            resident.append(k)
        for k in resident:
            complete(st, k, taus[k])
        assert st.u == [0, 0, 0] and st.cta_count == [0] * n                        # returns to empty


def test_quantise_tau():
    assert [quantise_tau(x) for x in (0.0, 0.03, 0.374, 1.0, 1.7)] == [0, 0, 6, 15, 15]


def test_grid_progress_variant_hand_derived():
    # the state of test_hand_derived_sequence before its third call: U = (15, 6, 12), one CTA of A and of B resident,
    # s_A = 4827, s_B = 3183 (the base policy admits A)
    taus = [(15, 2, 3), (0, 4, 9)]

    def fresh():
        st = SMState(2)
        st.cta_count = [1, 1]
        st.u = [15, 6, 12]
        return st
    # -G: s * G_k / (c_k + 1).  A has a 2-CTA grid, B a 30-CTA grid: 4827*2/2 = 4827 < 3183*30/2 = 47745 -> B
    st = fresh()
    assert variant_score(st, 0, taus[0], "G", grid=[2, 30]) == 4827
    assert variant_score(st, 1, taus[1], "G", grid=[2, 30]) == 47745
    assert admission_decision(st, taus, [True, True], [True, True], variant="G", grid=[2, 30]) == (1, 2)
    # equal grids: the factor G/(c+1) is common and the base order stands
    assert admission_decision(fresh(), taus, [True, True], [True, True], variant="G", grid=[8, 8]) == (0, 2)
    # the score decays as a kernel accumulates CTAs: with 3 CTAs of A resident, 4 * s_B > 2 * s_A flips the order
    st = fresh()
    st.cta_count = [3, 1]
    assert variant_score(st, 0, taus[0], "G", grid=[8, 8]) == Fraction(4827 * 8, 4)
    assert variant_score(st, 1, taus[1], "G", grid=[8, 8]) == Fraction(3183 * 8, 2)
    assert admission_decision(st, taus, [True, True], [True, True], variant="G", grid=[8, 8]) == (1, 2)
    # Phase 1 is untouched by the variants
    st = SMState(2)
    assert admission_decision(st, taus, [True, True], [True, True], variant="G", grid=[1, 1000]) == (0, 1)


def test_register_variant_hand_derived():
    taus = [(15, 2, 3), (0, 4, 9)]

    def fresh():
        st = SMState(2)
        st.cta_count = [1, 1]
        st.u = [15, 6, 12]
        return st
    # -R: s / (c_k * R_k + 1).  A uses 64 registers per CTA, B 32: 4827/65 = 74.3 < 3183/33 = 96.5 -> B
    st = fresh()
    assert variant_score(st, 0, taus[0], "R", regs=[64, 32]) == Fraction(4827, 65)
    assert variant_score(st, 1, taus[1], "R", regs=[64, 32]) == Fraction(3183, 33)
    assert admission_decision(st, taus, [True, True], [True, True], variant="R", regs=[64, 32]) == (1, 2)
    # equal register counts: the base order stands
    assert admission_decision(fresh(), taus, [True, True], [True, True], variant="R", regs=[48, 48]) == (0, 2)
    # a kernel with no CTA resident is not penalised at all (denominator 1) -- but then Phase 1 takes it anyway
    st = fresh()
    st.cta_count = [1, 0]
    assert admission_decision(st, taus, [True, True], [True, True], variant="R", regs=[64, 32]) == (1, 1)
    # exact ties keep the first seen: s_0/(1*1+1) == s_1/(1*3+1) with s_1 = 2 s_0
    taus2 = [(1, 0, 0), (2, 0, 0)]
    st = SMState(2)
    st.cta_count = [1, 1]
    assert admission_decision(st, taus2, [True, True], [True, True], variant="R", regs=[1, 3]) == (0, 2)
