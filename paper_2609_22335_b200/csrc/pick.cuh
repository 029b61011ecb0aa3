// The pick: which tile class a free worker on SM j admits next.
//
// Software analogue of the paper's single-admission decision (Algorithm 1) with
// its per-SM utilisation registers (Section 3.3): a tile class plays the role of
// a kernel, a worker group running a tile plays the role of a resident CTA,
// Feasible(k, j) is "the class's shared-memory and tensor-memory need fits what
// this SM has free right now".  One call chooses at most one class.
//
//   Phase 1  a pending, feasible class whose GROUP has no tile resident on this SM
//            wins, scanning from a rotating start (co-residency priority: a short
//            action-head tile is never stuck behind resident VLM tiles).  A group
//            is what the paper calls a kernel of one stream: the engine groups the
//            tile classes by phase (VLM stream, action-head stream: K = 2, as in
//            the paper's evaluation); with one class per group this is the
//            paper's listing exactly;
//   Phase 2  otherwise the pending feasible class with the largest
//            s = sum_x (U_max - U_x[j]) * tau_x(k); strict '>' keeps the first seen.
//
// Counters are 32-bit and exact; headroom is clamped at U_max when scoring.  U_max is the value a
// utilisation counter reaches on a full SM: 255 for the paper's 8-bit registers with up to 32 resident
// CTAs, 15 x (worker groups per SM) here, where an SM holds that many tiles.  With the hardware's 255
// and three tiles the headroom would never move and Phase 2 would degenerate to a fixed class order.
#pragma once
#include <stdint.h>

#ifndef __CUDACC__
#define VLA_HD
#else
#define VLA_HD __host__ __device__
#endif

namespace vla {

constexpr int PICK_MAX_CLASSES = 8;
constexpr int PICK_U_MAX = 255;

struct PickState {
  int cta_count[PICK_MAX_CLASSES];   // tiles of class k resident on this SM
  int u[3];                          // U_TC, U_ALU, U_MEM
  int rr;                            // start of the next Phase-1 scan
};

enum PickPolicy : int { POLICY_TWO_PHASE = 0, POLICY_CLASS_ORDER = 1, POLICY_ROUND_ROBIN = 2 };

// Returns the chosen class or -1; *phase = 1 or 2 (0 when nothing was chosen).
VLA_HD inline int pick_choose(int n_cls, const int* tau /*[n_cls][3]*/, const int* group /*[n_cls]*/, unsigned pending,
                              unsigned feasible, const PickState& st, int rr_start, int policy, int u_max, int* phase) {
  *phase = 0;
  unsigned ok = pending & feasible;
  if (ok == 0) return -1;
  if (policy == POLICY_CLASS_ORDER) {
    for (int k = 0; k < n_cls; ++k)
      if (ok & (1u << k)) { *phase = 1; return k; }
    return -1;
  }
  if (policy == POLICY_ROUND_ROBIN) {
    for (int i = 0; i < n_cls; ++i) {
      int k = (rr_start + i) % n_cls;
      if (ok & (1u << k)) { *phase = 1; return k; }
    }
    return -1;
  }
  int resident[PICK_MAX_CLASSES];                         // tiles resident per group
  for (int g = 0; g < PICK_MAX_CLASSES; ++g) resident[g] = 0;
  for (int k = 0; k < n_cls; ++k) resident[group[k]] += st.cta_count[k];
  for (int i = 0; i < n_cls; ++i) {                       // Phase 1
    int k = (rr_start + i) % n_cls;
    if ((ok & (1u << k)) && resident[group[k]] == 0) { *phase = 1; return k; }
  }
  int best = -1, best_score = -1;                         // Phase 2
  for (int k = 0; k < n_cls; ++k) {
    if (!(ok & (1u << k))) continue;
    int s = 0;
    for (int x = 0; x < 3; ++x) {
      int used = st.u[x] > u_max ? u_max : st.u[x];
      s += (u_max - used) * tau[k * 3 + x];
    }
    if (s > best_score) { best_score = s; best = k; }
  }
  if (best >= 0) *phase = 2;
  return best;
}

VLA_HD inline void pick_commit(PickState& st, int k, const int* tau) {
  st.cta_count[k] += 1;
  for (int x = 0; x < 3; ++x) st.u[x] += tau[k * 3 + x];
}

VLA_HD inline void pick_release(PickState& st, int k, const int* tau) {
  st.cta_count[k] -= 1;
  for (int x = 0; x < 3; ++x) st.u[x] -= tau[k * 3 + x];
}

}  // namespace vla
