"""CPU oracle of the single-admission decision (paper Algorithm 1) and the per-SM
utilisation registers (paper Section 3.3).  TEST INFRASTRUCTURE ONLY: the GPU
library never imports or calls this.

The steps follow the algorithm in the paper's order and notation:

  state per SM j : CTA_count(k, j), U_TC[j], U_ALU[j], U_MEM[j]   (8-bit, cap U_max = 255)
  per kernel k   : tau(k) = (tau_TC, tau_ALU, tau_MEM), each 0..15; pending(k); Feasible(k, j)

  Phase 1: the first pending kernel, in dispatcher order, that has no CTA on SM j
           and is feasible, is admitted; return.
  Phase 2: otherwise, among pending feasible kernels, the one with the largest
           s = sum_x (U_max - U_x[j]) * tau_x(k), strict '>' so ties keep the
           first seen; admit it (or nothing when none is feasible).
  Admit  : CTA_count += 1, U_x += tau_x (capped at U_max).
  Completion: CTA_count -= 1, U_x -= tau_x.

Reading of an ambiguity: the listing scans "in dispatcher order" while the prose
of Section 3.4.1 says Phase 1 "picks one by round-robin".  ``rr_start`` lets the
caller rotate the start of the Phase-1 scan; rr_start = 0 is the listing as
printed.

Two variants of the Phase-2 score (paper Section 4, "Implementations"):

  -G  s_GRID = s * G_k / (c_k(j) + 1)      G_k = full grid size of kernel k, c_k(j) = its CTAs on SM j
  -R  s_REG  = s / (c_k(j) * R_k + 1)      R_k = registers per CTA of kernel k

Both are ratios of integers; they are compared exactly (Fraction), so a caller
that compares them by integer cross-multiplication takes the same decisions.
Phase 1, the strict '>' and the admit / completion rules are unchanged.

Pins: tests/test_admission_oracle.py (hand-derived decision sequence, the
paper's arithmetic identities 17 x 15 = 255 and 24 + 12 = 36 bits, invariants,
hand-derived -G / -R cases).
"""
from __future__ import annotations

from fractions import Fraction

U_MAX = 255
TAU_MAX = 15


class SMState:
    def __init__(self, n_kernels: int):
        self.cta_count = [0] * n_kernels
        self.u = [0, 0, 0]                  # U_TC, U_ALU, U_MEM

    def copy(self):
        s = SMState(len(self.cta_count))
        s.cta_count = list(self.cta_count)
        s.u = list(self.u)
        return s


def score(state: SMState, tau, u_max: int = U_MAX) -> int:
    """s = sum over pipelines of headroom times intensity (headroom never negative)."""
    return sum((u_max - min(u_max, state.u[x])) * tau[x] for x in range(3))


def admit(state: SMState, k: int, tau, u_max: int = U_MAX) -> None:
    state.cta_count[k] += 1
    for x in range(3):
        state.u[x] = min(u_max, state.u[x] + tau[x])


def complete(state: SMState, k: int, tau) -> None:
    state.cta_count[k] -= 1
    for x in range(3):
        state.u[x] = max(0, state.u[x] - tau[x])


def variant_score(state: SMState, k: int, tau, variant: str = "base", grid=None, regs=None, u_max: int = U_MAX):
    """Phase-2 score of kernel k under the base policy or one of its two variants, as an exact ratio."""
    s = score(state, tau, u_max)
    c = state.cta_count[k]
    if variant == "base":
        return Fraction(s)
    if variant == "G":
        return Fraction(s * grid[k], c + 1)
    if variant == "R":
        return Fraction(s, c * regs[k] + 1)
    raise ValueError(variant)


def admission_decision(state: SMState, taus, pending, feasible, rr_start: int = 0, u_max: int = U_MAX,
                       variant: str = "base", grid=None, regs=None):
    """One invocation: returns (kernel admitted or None, phase 1|2|0) and updates ``state``.

    taus[k] = (tau_TC, tau_ALU, tau_MEM); pending[k], feasible[k] booleans.  ``u_max`` is the
    saturation value of the utilisation registers (Section 3.3: 8-bit, 255); a caller whose SM
    holds fewer, larger units of work passes the value its counters reach on a full SM.
    ``variant`` "G" needs grid[k] (G_k), "R" needs regs[k] (R_k).
    """
    n = len(taus)
    # Phase 1
    for i in range(n):
        k = (rr_start + i) % n
        if not pending[k]:
            continue
        if state.cta_count[k] == 0 and feasible[k]:
            admit(state, k, taus[k], u_max)
            return k, 1
    # Phase 2
    best_score, best_kernel = -1, None
    for k in range(n):
        if not pending[k]:
            continue
        if not feasible[k]:
            continue
        s = variant_score(state, k, taus[k], variant, grid, regs, u_max)
        if s > best_score:
            best_score, best_kernel = s, k
    if best_kernel is None:
        return None, 0
    admit(state, best_kernel, taus[best_kernel], u_max)
    return best_kernel, 2


def quantise_tau(fraction: float) -> int:
    """Utilisation fraction of peak -> 4-bit intensity field (Section 3.2.2)."""
    return max(0, min(TAU_MAX, int(round(TAU_MAX * fraction))))
