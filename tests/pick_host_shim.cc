// Host build of the pick (the same header the persistent kernel compiles) for the CPU tests.
#include "../paper_2609_22335_b200/csrc/pick.cuh"

extern "C" int pick_host(int n_cls, const int* tau, const int* group, unsigned pending, unsigned feasible,
                         int* cta_count /*[n_cls], updated*/, int* u /*[3], updated*/, int rr_start, int policy,
                         int u_max, int* phase, const int* grid /*[n_cls] or null*/, const int* res /*[n_cls] or null*/) {
  vla::PickState st;
  for (int k = 0; k < vla::PICK_MAX_CLASSES; ++k) st.cta_count[k] = k < n_cls ? cta_count[k] : 0;
  for (int x = 0; x < 3; ++x) st.u[x] = u[x];
  st.rr = rr_start;
  unsigned group_mask[vla::PICK_MAX_CLASSES];
  vla::pick_group_masks(n_cls, group, group_mask);
  const int k = vla::pick_choose(n_cls, tau, group_mask, pending, feasible, st, rr_start, policy, u_max, phase, grid, res);
  if (k >= 0) vla::pick_commit(st, k, tau);
  for (int i = 0; i < n_cls; ++i) cta_count[i] = st.cta_count[i];
  for (int x = 0; x < 3; ++x) u[x] = st.u[x];
  return k;
}
