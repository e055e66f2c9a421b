// Layout search over the cost counts of Table 1 (the paper lists the automated search for a
// computation layout as future work, Section 11, and gives the model it would use: per processor the
// multiply-adds of the local einsums and the values that enter Allreduces, Sections 8.1-8.3).
// Exhaustive: every assignment of the candidate tensor dimensions to a mesh dimension or to none is
// planned with the host planner (which decides legality exactly as for a real call) and scored by
//     cost = sum over the workload's einsums of  macs_per_proc + comm_weight * allreduce_values,
// ties going to the smaller memory footprint (sum of slice elements), then to the assignment that
// comes first when candidates are enumerated in the given order, "unsplit" before mesh dimension 0, 1, ...
#include <cstring>
#include <memory>

#include "mtf_internal.h"

using mtf::fail;

extern "C" mtf_status mtf_layout_search(const mtf_mesh_t* mesh, int32_t n_einsums, const mtf_tensor* in0, const mtf_tensor* in1, const mtf_tensor* out,
                                        int32_t n_names, const char* const* names, double comm_weight, int32_t* chosen_mesh_dim, double* cost,
                                        int64_t* footprint) {
  if (!mesh || !in0 || !in1 || !out || !names || !chosen_mesh_dim || n_einsums < 1 || n_names < 0 || n_names > 12)
    return fail(MTF_ERR_INVALID_ARG, "layout_search: bad argument");
  const int R = (int)mesh->dims.size();
  std::vector<int> pick(n_names, -1), best;
  double best_cost = 0;
  int64_t best_foot = 0;
  bool have = false;
  // odometer over assignments: the FIRST name varies slowest, each digit runs -1 (unsplit), 0, 1, ...
  while (true) {
    mtf_layout_t L;
    L.mesh = mesh->dims;
    for (int i = 0; i < n_names; ++i)
      if (pick[i] >= 0) L.rules.emplace_back(names[i], pick[i]);
    double c = 0;
    int64_t foot = 0;
    bool legal = true;
    for (int e = 0; e < n_einsums && legal; ++e) {
      const mtf_tensor ins[2] = {in0[e], in1[e]};
      std::unique_ptr<mtf_plan_t> P;
      mtf_status st = mtf::make_plan(&L, 2, ins, &out[e], nullptr, MTF_KERNEL_SIMT, -1, &P);     // (family irrelevant: only legality and counts are read)
      if (st == MTF_ERR_ILLEGAL_LAYOUT || st == MTF_ERR_NOT_DIVISIBLE) { legal = false; break; }
      if (st != MTF_OK) return st;
      c += (double)P->macs_per_proc + comm_weight * (double)P->allreduce_values;
      foot += P->slice_elems;
    }
    if (legal && (!have || c < best_cost || (c == best_cost && foot < best_foot))) {
      have = true; best = pick; best_cost = c; best_foot = foot;
    }
    int i = n_names - 1;
    while (i >= 0 && ++pick[i] == R) { pick[i] = -1; --i; }
    if (i < 0) break;
  }
  if (!have) return fail(MTF_ERR_ILLEGAL_LAYOUT, "layout_search: no legal layout");
  for (int i = 0; i < n_names; ++i) chosen_mesh_dim[i] = best[i];
  if (cost) *cost = best_cost;
  if (footprint) *footprint = best_foot;
  return MTF_OK;
}
