// One mesh dimension mapped onto several GPUs, one process per GPU (the paper's own setting: Section 2,
// a mesh is a naming abstraction over the physical processors; Algorithm 1 line 2 and Section 8.1 /
// 8.2 say where the sums across processors are).  A rank-bound layout describes the virtual processors
// one rank owns; tensors under it are the rank's boxes of the global tensors; einsums whose reduced-out
// dimensions are split over the rank-spanning mesh dimension leave partial sums, which the caller's
// collective hooks add up behind the producing launch.  Host logic only: no communication library here.
#include <cstring>

#include "mtf_internal.h"

using mtf::fail;

namespace mtf {

bool rank_sum_needed(const mtf_layout_t* L, const std::vector<std::string>& reduced) {
  if (!L || L->bound_dim < 0 || L->world <= 1) return false;
  for (auto& n : reduced)
    if (L->mesh_dim_of(n) == L->bound_dim) return true;
  return false;
}

mtf_status rank_allreduce_start(const mtf_layout_t* L, void* data, int64_t count, mtf_dtype dtype, void* stream) {
  if (!L || !L->ar_start || L->world <= 1) return MTF_OK;
  mtf_status st = L->ar_start(L->ar_user, data, count, dtype, stream);
  if (st != MTF_OK) return fail(st, "the rank collective hook (start) returned status %d", (int)st);
  return MTF_OK;
}

mtf_status rank_wait(const mtf_layout_t* L, void* stream) {
  if (!L || !L->ar_wait || L->world <= 1) return MTF_OK;
  mtf_status st = L->ar_wait(L->ar_user, stream);
  if (st != MTF_OK) return fail(st, "the rank collective hook (wait) returned status %d", (int)st);
  return MTF_OK;
}

}  // namespace mtf

extern "C" {

mtf_status mtf_layout_bind_ranks(const mtf_layout_t* layout, const char* mesh_dim, int32_t world, int32_t rank,
                                 mtf_rank_allreduce_fn start, mtf_rank_wait_fn wait, void* user, mtf_layout_t** out) {
  if (!out) return fail(MTF_ERR_INVALID_ARG, "layout_bind_ranks: out is NULL");
  *out = nullptr;
  if (!layout || !mesh_dim) return fail(MTF_ERR_INVALID_ARG, "layout_bind_ranks: NULL argument");
  if (world < 1 || rank < 0 || rank >= world) return fail(MTF_ERR_INVALID_ARG, "layout_bind_ranks: rank %d of %d", rank, world);
  if ((start == nullptr) != (wait == nullptr)) return fail(MTF_ERR_INVALID_ARG, "layout_bind_ranks: give both collective hooks or neither");
  if (layout->bound_dim >= 0) return fail(MTF_ERR_UNSUPPORTED, "layout_bind_ranks: the layout is already bound to ranks (one rank-spanning mesh dimension)");
  int j = -1;
  for (size_t m = 0; m < layout->mesh.size(); ++m)
    if (layout->mesh[m].name == mesh_dim) j = (int)m;
  if (j < 0) return fail(MTF_ERR_UNKNOWN_DIM, "layout_bind_ranks: mesh has no dimension '%s'", mesh_dim);
  if (layout->mesh[j].size % world != 0)
    return fail(MTF_ERR_NOT_DIVISIBLE, "layout_bind_ranks: mesh dimension '%s' of size %lld is not divisible by %d ranks", mesh_dim, (long long)layout->mesh[j].size, world);
  mtf_layout_t* L = new mtf_layout_t();
  L->mesh = layout->mesh;
  L->rules = layout->rules;
  L->bound_dim = j;
  L->world = world;
  L->rank = rank;
  L->bound_global = layout->mesh[j].size;
  L->mesh[j].size = layout->mesh[j].size / world;
  L->ar_start = start; L->ar_wait = wait; L->ar_user = user;
  *out = L;
  return MTF_OK;
}

mtf_status mtf_rank_box(const mtf_layout_t* L, int32_t ndim, const mtf_dim* global_dims, int64_t* offsets, int64_t* sizes) {
  if (!L || (ndim > 0 && (!offsets || !sizes))) return fail(MTF_ERR_INVALID_ARG, "rank_box: NULL argument");
  std::vector<mtf::Dim> d;
  mtf_status st = mtf::read_dims(ndim, global_dims, &d, "tensor");
  if (st != MTF_OK) return st;
  int seen = -1;
  for (int i = 0; i < ndim; ++i) {
    offsets[i] = 0;
    sizes[i] = d[i].size;
    if (L->bound_dim >= 0 && L->mesh_dim_of(d[i].name) == L->bound_dim) {
      if (seen >= 0) return fail(MTF_ERR_ILLEGAL_LAYOUT, "dimensions '%s' and '%s' are both split over the rank-spanning mesh dimension", d[seen].name.c_str(), d[i].name.c_str());
      seen = i;
      if (d[i].size % L->bound_global != 0)
        return fail(MTF_ERR_NOT_DIVISIBLE, "dimension '%s' of size %lld is not divisible by mesh dimension '%s' of size %lld", d[i].name.c_str(),
                    (long long)d[i].size, L->mesh[L->bound_dim].name.c_str(), (long long)L->bound_global);
      sizes[i] = d[i].size / L->world;
      offsets[i] = sizes[i] * L->rank;
    }
  }
  return MTF_OK;
}

mtf_status mtf_plan_needs_rank_sum(const mtf_plan_t* plan, int32_t* flags) {
  if (!plan || !flags) return fail(MTF_ERR_INVALID_ARG, "plan_needs_rank_sum: NULL argument");
  *flags = (plan->rank_sum ? 1 : 0) | (plan->rsum_rank_sum ? 2 : 0);
  return MTF_OK;
}

mtf_status mtf_rank_wait(const mtf_layout_t* L, void* stream) {
  if (!L) return fail(MTF_ERR_INVALID_ARG, "rank_wait: layout is NULL");
  return mtf::rank_wait(L, stream);
}

}  // extern "C"
