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
// Two variants of the Phase-2 score (paper Section 4): -G multiplies s by G_k / (c_k + 1), where G_k is the
// class's grid still to place (its queue depth here) and c_k its tiles resident on this SM; -R divides s by
// c_k * R_k + 1, where R_k is the per-tile footprint of the class in the resource that varies between tiles
// (shared-memory units here: registers are fixed per worker group).  Both are ratios of integers and are compared
// exactly by cross-multiplication in 64 bits.
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

enum PickPolicy : int { POLICY_TWO_PHASE = 0, POLICY_CLASS_ORDER = 1, POLICY_ROUND_ROBIN = 2, POLICY_TWO_PHASE_G = 3,
                        POLICY_TWO_PHASE_R = 4 };
VLA_HD inline bool pick_is_two_phase(int policy) {
  return policy == POLICY_TWO_PHASE || policy == POLICY_TWO_PHASE_G || policy == POLICY_TWO_PHASE_R;
}

VLA_HD inline int pick_lowest_bit(unsigned m) {           // m != 0
#ifdef __CUDA_ARCH__
  return __ffs((int)m) - 1;
#else
  return __builtin_ctz(m);
#endif
}
// First set bit of `m` (n_cls bits) scanning upwards from position `start`, wrapping around.
VLA_HD inline int pick_first_from(unsigned m, int start, int n_cls) {
  const unsigned all = (1u << n_cls) - 1u;
  const unsigned rot = ((m >> start) | (m << (n_cls - start))) & all;
  const int k = start + pick_lowest_bit(rot);
  return k >= n_cls ? k - n_cls : k;
}
// group_mask[k] = bit mask of the classes in k's group (k's own bit included), from the group ids.
VLA_HD inline void pick_group_masks(int n_cls, const int* group, unsigned* group_mask) {
  for (int k = 0; k < n_cls; ++k) {
    unsigned m = 0;
    for (int j = 0; j < n_cls; ++j)
      if (group[j] == group[k]) m |= 1u << j;
    group_mask[k] = m;
  }
}

// Returns the chosen class or -1; *phase = 1 or 2 (0 when nothing was chosen).
// group_mask: see pick_group_masks.  grid[k] (G_k, for POLICY_TWO_PHASE_G) and res[k] (R_k, for POLICY_TWO_PHASE_R)
// may be null for the other policies.  Every array is read at loop-constant positions only, so a caller that inlines
// this with a constant n_cls keeps them in registers (the persistent kernel calls it on every tile hand-over).
VLA_HD inline int pick_choose(int n_cls, const int* tau /*[n_cls][3]*/, const unsigned* group_mask /*[n_cls]*/, unsigned pending,
                              unsigned feasible, const PickState& st, int rr_start, int policy, int u_max, int* phase,
                              const int* grid = nullptr, const int* res = nullptr) {
  *phase = 0;
  const unsigned ok = pending & feasible & ((1u << n_cls) - 1u);
  if (ok == 0) return -1;
  if (rr_start >= n_cls || rr_start < 0) rr_start = 0;
  if (policy == POLICY_CLASS_ORDER) { *phase = 1; return pick_lowest_bit(ok); }
  if (policy == POLICY_ROUND_ROBIN) { *phase = 1; return pick_first_from(ok, rr_start, n_cls); }
  // Phase 1: classes whose group has no tile resident on this SM
  unsigned occupied = 0, unrep = 0;
#pragma unroll
  for (int k = 0; k < PICK_MAX_CLASSES; ++k)
    if (k < n_cls && st.cta_count[k] > 0) occupied |= 1u << k;
#pragma unroll
  for (int k = 0; k < PICK_MAX_CLASSES; ++k)
    if (k < n_cls && (group_mask[k] & occupied) == 0u) unrep |= 1u << k;
  if (ok & unrep) { *phase = 1; return pick_first_from(ok & unrep, rr_start, n_cls); }
  // Phase 2: headroom per pipeline, then the largest score, strict '>' (first seen wins ties)
  int head[3];
#pragma unroll
  for (int x = 0; x < 3; ++x) head[x] = u_max - (st.u[x] > u_max ? u_max : st.u[x]);
  int best = -1;
  if (policy == POLICY_TWO_PHASE || (policy == POLICY_TWO_PHASE_G && !grid) || (policy == POLICY_TWO_PHASE_R && !res)) {
    int best_score = -1;                                  // Algorithm 1 as printed: integer scores
#pragma unroll
    for (int k = 0; k < PICK_MAX_CLASSES; ++k) {
      if (k >= n_cls || !(ok & (1u << k))) continue;
      const int s = head[0] * tau[k * 3] + head[1] * tau[k * 3 + 1] + head[2] * tau[k * 3 + 2];
      if (s > best_score) { best_score = s; best = k; }
    }
  } else {
    long long best_num = -1, best_den = 1;                // the variants: ratios num/den compared by cross-multiplication
#pragma unroll
    for (int k = 0; k < PICK_MAX_CLASSES; ++k) {
      if (k >= n_cls || !(ok & (1u << k))) continue;
      const int s = head[0] * tau[k * 3] + head[1] * tau[k * 3 + 1] + head[2] * tau[k * 3 + 2];
      long long num = s, den = 1;
      if (policy == POLICY_TWO_PHASE_G) { num = (long long)s * grid[k]; den = st.cta_count[k] + 1; }
      else den = (long long)st.cta_count[k] * res[k] + 1;
      if (num * best_den > best_num * den) { best_num = num; best_den = den; best = k; }
    }
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
