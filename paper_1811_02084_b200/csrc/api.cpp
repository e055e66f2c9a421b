// The C ABI (include/mtf.h): argument checking, plan caching and the block compositions.  Every
// numerical step runs in the CUDA kernels; this file only validates, plans and launches.
#include <algorithm>
#include <cstring>

#include "mtf_internal.h"

namespace mtf {
mtf_status ffn_forward_impl(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* bias, const mtf_tensor* v,
                            mtf_tensor* h_saved, mtf_tensor* y, const mtf_tensor* y_residual, void* workspace, size_t workspace_bytes, void* stream);
mtf_status ffn_backward_impl(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* v, const mtf_tensor* h_saved,
                             const mtf_tensor* dy, mtf_tensor* dx, const mtf_tensor* dx_residual, mtf_tensor* dw, mtf_tensor* dbias, mtf_tensor* dv,
                             void* workspace, size_t workspace_bytes, void* stream);
const char* last_error();
int64_t launch_count();
mtf_status read_device_status(int* code);
mtf_status read_bad_index(int* seen);
mtf_status read_row_status(int* code);
mtf_status debug_wait_test(long long limit_cycles, int skip_first_commit);
mtf_status read_attention_status(int* code);
mtf_status launch_permute_copy(const void* src, void* dst, int elem_bytes, int ndim, const int64_t* sizes, const int64_t* sstr, const int64_t* dstr, void* stream);
mtf_status read_attention_bwd_status(int* code);
}  // namespace mtf

using mtf::Dim;
using mtf::fail;

namespace {

thread_local int g_force_kernel = -1;
thread_local bool g_next_independent = false;
thread_local int g_force_reduce = -1;

int elem_bytes(int dt) { return dt == MTF_BF16 ? 2 : 4; }

int64_t numel(const mtf_tensor& t) {
  int64_t n = 1;
  for (int i = 0; i < t.ndim; ++i) n *= t.dims[i].size;
  return n;
}

bool dims_match(const std::vector<Dim>& want, const mtf_tensor& t) {
  if ((int)want.size() != t.ndim) return false;
  for (int i = 0; i < t.ndim; ++i)
    if (!t.dims[i].name || want[i].name != t.dims[i].name || want[i].size != t.dims[i].size) return false;
  return true;
}

mtf_status exec_plan(const mtf_plan_t* P, const mtf_tensor* in, mtf_tensor* out, const mtf_epilogue* epi,
                     void* workspace, size_t workspace_bytes, void* stream, int n_terms = 1, const void* const* extra_operands = nullptr,
                     int row_softmax = 0, int n_groups = 1, const void* const* group_operands = nullptr) {
  if (!P || !in || !out) return fail(MTF_ERR_INVALID_ARG, "einsum exec: NULL argument");
  if (!dims_match(P->dimsA, in[0]) || (P->has_B && !dims_match(P->dimsB, in[1])) || !dims_match(P->dimsC, *out))
    return fail(MTF_ERR_SIZE_MISMATCH, "einsum exec: operand dims differ from the planned ones");
  if (in[0].dtype != P->dtA || (P->has_B && in[1].dtype != P->dtB) || out->dtype != P->dtC)
    return fail(MTF_ERR_INVALID_ARG, "einsum exec: operand dtypes differ from the planned ones");
  if (!in[0].data || (P->has_B && !in[1].data) || !out->data) return fail(MTF_ERR_INVALID_ARG, "einsum exec: NULL data pointer");
  const void* bias = nullptr;
  const void* mask = nullptr;
  const void* resid = nullptr;
  if (P->epi.on) {
    if (!epi) return fail(MTF_ERR_INVALID_ARG, "einsum exec: the plan has an epilogue, none was passed");
    if (P->epi.has_bias) {
      if (!epi->bias || !epi->bias->data || !dims_match(P->epi.bias_dims, *epi->bias) || epi->bias->dtype != P->epi.dtBias)
        return fail(MTF_ERR_INVALID_ARG, "einsum exec: bias differs from the planned one");
      bias = epi->bias->data;
    }
    if (P->epi.has_mask) {
      if (!epi->relu_mask || !epi->relu_mask->data || !dims_match(P->dimsC, *epi->relu_mask) || epi->relu_mask->dtype != P->epi.dtMask)
        return fail(MTF_ERR_INVALID_ARG, "einsum exec: relu_mask differs from the planned one");
      mask = epi->relu_mask->data;
    }
    if (P->epi.has_res) {
      if (!epi->residual || !epi->residual->data || !dims_match(P->dimsC, *epi->residual) || epi->residual->dtype != P->epi.dtRes)
        return fail(MTF_ERR_INVALID_ARG, "einsum exec: residual differs from the planned one");
      resid = epi->residual->data;
      if (P->rank_sum && P->rank != 0) resid = nullptr;      // a partial sum across ranks: rank 0 alone adds the residual
    }
  }
  float* rsum = nullptr;
  int64_t rsum_elems = 1;
  if (P->epi.on && P->epi.has_rsum) {
    if (!epi->reduce_sum_out || !epi->reduce_sum_out->data || !dims_match(P->epi.rsum_dims, *epi->reduce_sum_out) || epi->reduce_sum_out->dtype != MTF_F32)
      return fail(MTF_ERR_INVALID_ARG, "einsum exec: reduce_sum_out differs from the planned one");
    rsum = reinterpret_cast<float*>(epi->reduce_sum_out->data);
    for (auto& d : P->epi.rsum_dims) rsum_elems *= d.size;
  }
  const float scale = P->epi.on ? epi->scale : 1.f;
  const int relu = P->epi.on ? (epi->relu != 0) : 0;
  if (row_softmax && P->rank_sum) return fail(MTF_ERR_UNSUPPORTED, "a row softmax cannot follow a sum that is split across ranks");
  mtf_status st;
  if (P->kernel_kind == MTF_KERNEL_TCGEN05) {
    st = mtf::launch_tc(*P, in[0].data, in[1].data, out->data, bias, P->epi.dtBias, mask, P->epi.dtMask, resid,
                        P->epi.dtRes, scale, relu, rsum, workspace, workspace_bytes, stream, n_terms, extra_operands, row_softmax, n_groups, group_operands);
  } else {
    if (n_terms != 1 || row_softmax || n_groups != 1) return fail(MTF_ERR_UNSUPPORTED, "multi-term, grouped or fused-softmax contraction on the generic kernel");
    SimtParams s = P->simt;
    s.A = in[0].data;
    s.B = P->has_B ? in[1].data : nullptr;
    s.C = out->data;
    s.bias = bias; s.mask = mask; s.resid = resid;
    s.scale = scale; s.relu = relu;
    s.rsum = rsum;
    st = mtf::launch_simt(s, rsum_elems, stream);
  }
  if (st != MTF_OK) return st;
  // one mesh dimension across ranks: the result is a partial sum; the caller's hook adds the ranks' parts up behind this launch
  if (P->ar_start && (P->rank_sum || (P->rsum_rank_sum && rsum))) {
    if (P->rank_sum) {
      mtf_status hs = P->ar_start(P->ar_user, out->data, numel(*out), out->dtype, stream);
      if (hs != MTF_OK) return fail(hs, "the rank collective hook (start) returned status %d", (int)hs);
      for (int g = 1; g < n_groups; ++g) {       // grouped launch: the other problems' outputs (same shape and type)
        hs = P->ar_start(P->ar_user, const_cast<void*>(group_operands[3 * (g - 1) + 2]), numel(*out), out->dtype, stream);
        if (hs != MTF_OK) return fail(hs, "the rank collective hook (start) returned status %d", (int)hs);
      }
    }
    if (P->rsum_rank_sum && rsum) {
      mtf_status hs = P->ar_start(P->ar_user, rsum, rsum_elems, MTF_F32, stream);
      if (hs != MTF_OK) return fail(hs, "the rank collective hook (start) returned status %d", (int)hs);
    }
  }
  return MTF_OK;
}

// Plan through the layout's cache.  The returned pointer stays valid for the layout's lifetime.
mtf_status cached_plan(const mtf_layout_t* L, int n_in, const mtf_tensor* in, const mtf_tensor* out,
                       const mtf_epilogue* epi, const mtf_plan_t** plan) {
  if (!L || !in || !out) return fail(MTF_ERR_INVALID_ARG, "einsum: NULL argument");
  if (n_in < 1 || n_in > 2) return fail(MTF_ERR_UNSUPPORTED, "einsum: the GPU path takes 1 or 2 inputs, got %d", n_in);
  for (int q = 0; q < n_in; ++q)
    if (in[q].ndim < 0 || in[q].ndim > mtf::kMaxTensorDims || (in[q].ndim && !in[q].dims)) return fail(MTF_ERR_INVALID_ARG, "einsum: bad input descriptor");
  if (out->ndim < 0 || out->ndim > mtf::kMaxTensorDims || (out->ndim && !out->dims)) return fail(MTF_ERR_INVALID_ARG, "einsum: bad output descriptor");
  mtf_layout_t* Lm = const_cast<mtf_layout_t*>(L);
  const std::string key = mtf::plan_key(n_in, in, out, epi, g_force_kernel, g_force_reduce);
  std::lock_guard<std::mutex> lock(Lm->mu);
  auto it = Lm->cache.find(key);
  if (it == Lm->cache.end()) {
    std::unique_ptr<mtf_plan_t> P;
    mtf_status st = mtf::make_plan(L, n_in, in, out, epi, g_force_kernel, g_force_reduce, &P);
    if (st != MTF_OK) return st;
    P->key = key;
    it = Lm->cache.emplace(key, std::move(P)).first;
  }
  *plan = it->second.get();
  return MTF_OK;
}

// "batch io, io hidden -> batch hidden" must agree with the descriptors' names.
mtf_status check_equation(const char* eq, int n_in, const mtf_tensor* in, const mtf_tensor* out) {
  std::vector<std::vector<std::string>> groups(1);
  std::string tok;
  auto flush = [&] { if (!tok.empty()) { groups.back().push_back(tok); tok.clear(); } };
  for (const char* c = eq; *c; ++c) {
    if (*c == ',') { flush(); groups.emplace_back(); }
    else if (*c == '-' && c[1] == '>') { flush(); groups.emplace_back(); ++c; }
    else if (*c == ' ' || *c == '\t') flush();
    else tok.push_back(*c);
  }
  flush();
  if ((int)groups.size() != n_in + 1) return fail(MTF_ERR_INVALID_ARG, "equation '%s' does not have %d inputs and one output", eq, n_in);
  for (int q = 0; q <= n_in; ++q) {
    const mtf_tensor& t = q < n_in ? in[q] : *out;
    if ((int)groups[q].size() != t.ndim) return fail(MTF_ERR_INVALID_ARG, "equation '%s': operand %d has %d dims, descriptor has %d", eq, q, (int)groups[q].size(), t.ndim);
    for (int i = 0; i < t.ndim; ++i)
      if (groups[q][i] != t.dims[i].name) return fail(MTF_ERR_INVALID_ARG, "equation '%s': operand %d dim %d is '%s' in the descriptor", eq, q, i, t.dims[i].name);
  }
  return MTF_OK;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct FfnShapes {
  std::vector<mtf_dim> tok_hidden, hidden_only;
};

mtf_status ffn_check(const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* v) {
  if (!x || !w || !v) return fail(MTF_ERR_INVALID_ARG, "ffn: NULL tensor");
  if (x->ndim < 2 || x->ndim > mtf::kMaxTensorDims - 1 || w->ndim != 2 || v->ndim != 2 || !x->dims || !w->dims || !v->dims)
    return fail(MTF_ERR_INVALID_ARG, "ffn: x must be [*tokens, d_in], w [d_in, hidden], v [hidden, d_out]");
  for (int i = 0; i < x->ndim; ++i) if (!x->dims[i].name) return fail(MTF_ERR_INVALID_ARG, "ffn: unnamed dimension");
  if (!w->dims[0].name || !w->dims[1].name || !v->dims[0].name || !v->dims[1].name) return fail(MTF_ERR_INVALID_ARG, "ffn: unnamed dimension");
  if (strcmp(x->dims[x->ndim - 1].name, w->dims[0].name) != 0) return fail(MTF_ERR_UNKNOWN_DIM, "ffn: x's last dim '%s' is not w's first dim '%s'", x->dims[x->ndim - 1].name, w->dims[0].name);
  if (strcmp(w->dims[1].name, v->dims[0].name) != 0) return fail(MTF_ERR_UNKNOWN_DIM, "ffn: w's second dim '%s' is not v's first dim '%s'", w->dims[1].name, v->dims[0].name);
  return MTF_OK;
}

}  // namespace

extern "C" {

mtf_status mtf_mesh_create(int32_t ndim, const mtf_dim* mesh_dims, mtf_mesh_t** out) {
  if (!out) return fail(MTF_ERR_INVALID_ARG, "mesh_create: out is NULL");
  *out = nullptr;
  if (ndim < 1 || ndim > mtf::kMaxMeshDims) return fail(MTF_ERR_INVALID_ARG, "mesh_create: ndim %d outside [1, %d]", ndim, mtf::kMaxMeshDims);
  std::vector<Dim> d;
  mtf_status st = mtf::read_dims(ndim, mesh_dims, &d, "mesh");
  if (st != MTF_OK) return st;
  mtf_mesh_t* m = new mtf_mesh_t();
  m->dims = d;
  for (auto& x : d) m->P *= x.size;
  *out = m;
  return MTF_OK;
}

mtf_status mtf_mesh_destroy(mtf_mesh_t* mesh) {
  delete mesh;
  return MTF_OK;
}

mtf_status mtf_mesh_size(const mtf_mesh_t* mesh, int64_t* n) {
  if (!mesh || !n) return fail(MTF_ERR_INVALID_ARG, "mesh_size: NULL argument");
  *n = mesh->P;
  return MTF_OK;
}

mtf_status mtf_mesh_coords(const mtf_mesh_t* mesh, int64_t p, int64_t* coords) {
  if (!mesh || !coords) return fail(MTF_ERR_INVALID_ARG, "mesh_coords: NULL argument");
  if (p < 0 || p >= mesh->P) return fail(MTF_ERR_INVALID_ARG, "mesh_coords: processor %lld outside mesh of %lld", (long long)p, (long long)mesh->P);
  for (int j = (int)mesh->dims.size() - 1; j >= 0; --j) {
    coords[j] = p % mesh->dims[j].size;
    p /= mesh->dims[j].size;
  }
  return MTF_OK;
}

mtf_status mtf_layout(const mtf_mesh_t* mesh, int32_t nrules, const char* const* tensor_dim, const char* const* mesh_dim,
                      mtf_layout_t** out) {
  if (!out) return fail(MTF_ERR_INVALID_ARG, "layout: out is NULL");
  *out = nullptr;
  if (!mesh) return fail(MTF_ERR_INVALID_ARG, "layout: mesh is NULL");
  if (nrules < 0 || nrules > 64 || (nrules > 0 && (!tensor_dim || !mesh_dim))) return fail(MTF_ERR_INVALID_ARG, "layout: bad rule list");
  std::unique_ptr<mtf_layout_t> L(new mtf_layout_t());
  L->mesh = mesh->dims;
  for (int i = 0; i < nrules; ++i) {
    if (!tensor_dim[i] || !tensor_dim[i][0] || !mesh_dim[i]) return fail(MTF_ERR_INVALID_ARG, "layout: rule %d has an empty name", i);
    int j = -1;
    for (size_t m = 0; m < mesh->dims.size(); ++m)
      if (mesh->dims[m].name == mesh_dim[i]) j = (int)m;
    if (j < 0) return fail(MTF_ERR_UNKNOWN_DIM, "layout: mesh has no dimension '%s'", mesh_dim[i]);
    for (auto& r : L->rules)
      if (r.first == tensor_dim[i]) return fail(MTF_ERR_INVALID_ARG, "layout: tensor dimension '%s' is mapped twice", tensor_dim[i]);
    L->rules.emplace_back(tensor_dim[i], j);
  }
  *out = L.release();
  return MTF_OK;
}

mtf_status mtf_layout_destroy(mtf_layout_t* layout) {
  delete layout;
  return MTF_OK;
}

mtf_status mtf_layout_check_tensor(const mtf_layout_t* layout, int32_t ndim, const mtf_dim* dims) {
  if (!layout) return fail(MTF_ERR_INVALID_ARG, "layout_check_tensor: layout is NULL");
  std::vector<Dim> d;
  mtf_status st = mtf::read_dims(ndim, dims, &d, "tensor");
  if (st != MTF_OK) return st;
  return mtf::check_tensor(layout, d);
}

mtf_status mtf_slice_map(const mtf_layout_t* layout, int32_t ndim, const mtf_dim* dims, int64_t processor,
                         int64_t* offsets, int64_t* sizes) {
  if (!layout || (ndim > 0 && (!offsets || !sizes))) return fail(MTF_ERR_INVALID_ARG, "slice_map: NULL argument");
  std::vector<Dim> d;
  mtf_status st = mtf::read_dims(ndim, dims, &d, "tensor");
  if (st != MTF_OK) return st;
  return mtf::slice_box(layout, d, processor, offsets, sizes);
}

mtf_status mtf_slice_gather(const mtf_layout_t* layout, const mtf_tensor* global, int64_t processor, void* out_slice,
                            void* stream) {
  if (!layout || !global || !global->data || !out_slice) return fail(MTF_ERR_INVALID_ARG, "slice_gather: NULL argument");
  if (global->dtype != MTF_F32 && global->dtype != MTF_BF16) return fail(MTF_ERR_INVALID_ARG, "slice_gather: unknown dtype");
  std::vector<Dim> d;
  mtf_status st = mtf::read_dims(global->ndim, global->dims, &d, "tensor");
  if (st != MTF_OK) return st;
  int64_t offs[mtf::kMaxTensorDims], sizes[mtf::kMaxTensorDims];
  if ((st = mtf::slice_box(layout, d, processor, offs, sizes)) != MTF_OK) return st;
  auto gs = mtf::row_major_strides(d);
  const int eb = elem_bytes(global->dtype), nd = global->ndim;
  // a box whose rows are whole 16-byte pieces on both sides goes through the vectorised row copy
  if (nd >= 1) {
    const int64_t vec = 16 / eb;
    int64_t base = 0, total = 1, sstr[mtf::kMaxTensorDims], dstr[mtf::kMaxTensorDims];
    for (int i = nd - 1; i >= 0; --i) { dstr[i] = total; total *= sizes[i]; }
    bool ok = total > 0 && total < 0x7fffffffLL && sizes[nd - 1] % vec == 0;
    for (int i = 0; i < nd; ++i) { sstr[i] = gs[i]; base += offs[i] * gs[i]; }
    for (int i = 0; ok && i + 1 < nd; ++i) ok = sstr[i] % vec == 0 && dstr[i] % vec == 0;
    const uint8_t* src = reinterpret_cast<const uint8_t*>(global->data) + base * eb;
    ok = ok && !(reinterpret_cast<uintptr_t>(src) & 15) && !(reinterpret_cast<uintptr_t>(out_slice) & 15);
    if (ok) return mtf::launch_permute_copy(src, out_slice, eb, nd, sizes, sstr, dstr, stream);
  }
  return mtf::launch_slice_gather(global->data, out_slice, eb, nd, sizes, offs, gs.data(), stream);
}

mtf_status mtf_einsum_plan(const mtf_layout_t* layout, int32_t n_in, const mtf_tensor* in_desc, const mtf_tensor* out_desc,
                           const mtf_epilogue* epilogue, mtf_plan_t** out) {
  if (!out) return fail(MTF_ERR_INVALID_ARG, "einsum_plan: out is NULL");
  *out = nullptr;
  std::unique_ptr<mtf_plan_t> P;
  mtf_status st = mtf::make_plan(layout, n_in, in_desc, out_desc, epilogue, g_force_kernel, g_force_reduce, &P);
  if (st != MTF_OK) return st;
  *out = P.release();
  return MTF_OK;
}

mtf_status mtf_plan_destroy(mtf_plan_t* plan) {
  delete plan;
  return MTF_OK;
}

mtf_status mtf_plan_workspace_bytes(const mtf_plan_t* plan, size_t* bytes) {
  if (!plan || !bytes) return fail(MTF_ERR_INVALID_ARG, "plan_workspace_bytes: NULL argument");
  *bytes = plan->workspace_bytes;
  return MTF_OK;
}

mtf_status mtf_plan_cost(const mtf_plan_t* plan, int64_t* macs, int64_t* allreduce_values, int64_t* slice_elems, int32_t* n_reduce) {
  if (!plan) return fail(MTF_ERR_INVALID_ARG, "plan_cost: plan is NULL");
  if (macs) *macs = plan->macs_per_proc;
  if (allreduce_values) *allreduce_values = plan->allreduce_values;
  if (slice_elems) *slice_elems = plan->slice_elems;
  if (n_reduce) *n_reduce = plan->n_reduce_mesh_dims;
  return MTF_OK;
}

mtf_status mtf_plan_info(const mtf_plan_t* plan, int32_t* kernel_kind, int32_t* reduce_mode, int64_t* n_slices,
                         int64_t* group_size, uint32_t* reduce_mask) {
  if (!plan) return fail(MTF_ERR_INVALID_ARG, "plan_info: plan is NULL");
  if (kernel_kind) *kernel_kind = plan->kernel_kind;
  if (reduce_mode) *reduce_mode = plan->reduce_mode;
  if (n_slices) *n_slices = plan->n_slices;
  if (group_size) *group_size = plan->group_size;
  if (reduce_mask) *reduce_mask = plan->reduce_mask;
  return MTF_OK;
}

mtf_status mtf_einsum_exec(const mtf_plan_t* plan, const mtf_tensor* in, mtf_tensor* out, const mtf_epilogue* epilogue,
                           void* workspace, size_t workspace_bytes, void* stream) {
  const bool independent = mtf::take_independent_hint();     // (cleared whatever happens below)
  if (independent && plan && plan->kernel_kind == MTF_KERNEL_TCGEN05) mtf::hint_next_launch_independent();
  const mtf_status st = exec_plan(plan, in, out, epilogue, workspace, workspace_bytes, stream);
  (void)mtf::take_independent_hint();
  return st;
}

mtf_status mtf_einsum(const mtf_layout_t* layout, const char* equation, int32_t n_in, const mtf_tensor* in, mtf_tensor* out,
                      const mtf_epilogue* epilogue, void* workspace, size_t workspace_bytes, void* stream) {
  const bool independent = mtf::take_independent_hint();     // (cleared whatever happens below)
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, n_in, in, out, epilogue, &P);
  if (st != MTF_OK) return st;
  if (equation && (st = check_equation(equation, n_in, in, out)) != MTF_OK) return st;
  if (independent && P->kernel_kind == MTF_KERNEL_TCGEN05) mtf::hint_next_launch_independent();
  st = exec_plan(P, in, out, epilogue, workspace, workspace_bytes, stream);
  (void)mtf::take_independent_hint();
  return st;
}

mtf_status mtf_einsum_builtin_scratch(const mtf_layout_t* layout, const char* equation, int32_t n_in, const mtf_tensor* in,
                                      mtf_tensor* out, const mtf_epilogue* epilogue, void* stream) {
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, n_in, in, out, epilogue, &P);
  if (st != MTF_OK) return st;
  if (equation && (st = check_equation(equation, n_in, in, out)) != MTF_OK) return st;
  if (P->kernel_kind != MTF_KERNEL_TCGEN05 || P->reduce_mode != MTF_REDUCE_WORKSPACE)
    return exec_plan(P, in, out, epilogue, nullptr, 0, stream);      // this plan needs no scratch at all
  if (P->workspace_bytes > mtf::builtin_scratch_capacity())
    return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "this einsum needs %zu scratch bytes, the built-in scratch holds %zu; use mtf_einsum with a caller-provided workspace",
                P->workspace_bytes, mtf::builtin_scratch_capacity());
  // the regular execution path (one validator for both entry points), on the library's own scratch: the
  // tile counters inside it are cleared on the stream before the launch and partial tiles are written
  // before they are read, so what the previous call left there does not matter
  void* ws = nullptr;
  if ((st = mtf::builtin_scratch_ptr(&ws)) != MTF_OK) return st;
  return exec_plan(P, in, out, epilogue, ws, mtf::builtin_scratch_capacity(), stream);
}

mtf_status mtf_einsum_workspace_bytes(const mtf_layout_t* layout, int32_t n_in, const mtf_tensor* in, const mtf_tensor* out,
                                      const mtf_epilogue* epilogue, size_t* bytes) {
  if (!bytes) return fail(MTF_ERR_INVALID_ARG, "einsum_workspace_bytes: bytes is NULL");
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, n_in, in, out, epilogue, &P);
  if (st != MTF_OK) return st;
  *bytes = P->workspace_bytes;
  return MTF_OK;
}

mtf_status mtf_hint_independent(void) {
  g_next_independent = true;
  return MTF_OK;
}

mtf_status mtf_plan_force(int32_t kernel_kind, int32_t reduce_mode) {
  if (kernel_kind < -1 || kernel_kind > 4 || reduce_mode < -1 || reduce_mode > 3)
    return fail(MTF_ERR_INVALID_ARG, "plan_force: value out of range");
  g_force_kernel = kernel_kind;
  g_force_reduce = reduce_mode;
  return MTF_OK;
}

mtf_status mtf_reduce_sum(const mtf_layout_t* layout, const mtf_tensor* in, mtf_tensor* out, void* stream) {
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, 1, in, out, nullptr, &P);
  if (st != MTF_OK) return st;
  return exec_plan(P, in, out, nullptr, nullptr, 0, stream);
}

// ---- feed-forward block --------------------------------------------------------------------------------

mtf_status mtf_ffn_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* bias,
                           const mtf_tensor* v, mtf_tensor* h_saved, mtf_tensor* y, void* workspace, size_t workspace_bytes,
                           void* stream) {
  mtf_status st = mtf::ffn_forward_impl(layout, x, w, bias, v, h_saved, y, nullptr, workspace, workspace_bytes, stream);
  return st != MTF_OK ? st : mtf::rank_wait(layout, stream);
}

}  // extern "C"

// y_residual (NULL or a tensor with y's dims) is added to y in the second einsum's epilogue.
mtf_status mtf::ffn_forward_impl(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* bias,
                                 const mtf_tensor* v, mtf_tensor* h_saved, mtf_tensor* y, const mtf_tensor* y_residual, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  mtf_status st = ffn_check(x, w, v);
  if (st != MTF_OK) return st;
  if (!h_saved || !y) return fail(MTF_ERR_INVALID_ARG, "ffn_forward: NULL output");
  // h = relu(x.w + bias): bias add and relu ride in the first einsum's epilogue
  mtf_epilogue e1;
  e1.scale = 1.f; e1.relu = 1; e1.bias = bias; e1.relu_mask = nullptr; e1.residual = nullptr; e1.reduce_sum_out = nullptr;
  mtf_tensor in1[2] = {*x, *w};
  if ((st = mtf_einsum(layout, nullptr, 2, in1, h_saved, &e1, workspace, workspace_bytes, stream)) != MTF_OK) return st;
  mtf_tensor in2[2] = {*h_saved, *v};
  mtf_epilogue e2;
  e2.scale = 1.f; e2.relu = 0; e2.bias = nullptr; e2.relu_mask = nullptr; e2.residual = y_residual; e2.reduce_sum_out = nullptr;
  return mtf_einsum(layout, nullptr, 2, in2, y, y_residual ? &e2 : nullptr, workspace, workspace_bytes, stream);
}

extern "C" {

static void ffn_dhp_desc(const mtf_tensor* h_like_dims_from_x, const mtf_tensor* w, mtf_dtype dt, mtf_dim* storage, mtf_tensor* out) {
  const mtf_tensor* x = h_like_dims_from_x;
  for (int i = 0; i < x->ndim - 1; ++i) storage[i] = x->dims[i];
  storage[x->ndim - 1] = w->dims[1];
  out->data = nullptr;
  out->dtype = dt;
  out->ndim = x->ndim;
  out->dims = storage;
}

mtf_status mtf_ffn_workspace_bytes(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, size_t* bytes) {
  if (!bytes) return fail(MTF_ERR_INVALID_ARG, "ffn_workspace_bytes: bytes is NULL");
  if (!layout || !x || !w || x->ndim < 2 || w->ndim != 2 || !x->dims || !w->dims) return fail(MTF_ERR_INVALID_ARG, "ffn_workspace_bytes: bad argument");
  mtf_dim hd[mtf::kMaxTensorDims];
  mtf_tensor dhp;
  ffn_dhp_desc(x, w, x->dtype, hd, &dhp);
  // dhp buffer + room for the largest per-einsum scratch (workspace-mode partials are bounded by
  // tiles * group * 128 * 256 * 4 bytes with tiles <= 74; 256 MiB covers every shape that picks it)
  size_t scratch = 0;
  {
    // the four backward einsums and the two forward ones, planned with these shapes
    mtf_dim vd[2] = {w->dims[1], w->dims[0]};
    mtf_tensor v = {nullptr, w->dtype, 2, vd};
    mtf_tensor hs = dhp;
    mtf_tensor xin = *x;
    mtf_dim yd[mtf::kMaxTensorDims];
    for (int i = 0; i < x->ndim; ++i) yd[i] = x->dims[i];
    mtf_tensor dy = {nullptr, x->dtype, x->ndim, yd};
    struct Case { mtf_tensor a, b, c; } cases[6] = {
        {xin, *w, hs}, {hs, v, dy}, {dy, v, dhp}, {hs, dy, {nullptr, MTF_F32, 2, vd}}, {xin, dhp, {nullptr, MTF_F32, 2, w->dims}}, {dhp, *w, xin}};
    int idx = 0;
    for (auto& c : cases) {
      mtf_tensor in[2] = {c.a, c.b};
      size_t b = 0;
      // (the dhp launch carries the fused column sum for dbias: its fixed-order finish wants scratch too)
      mtf_dim bd[1] = {w->dims[1]};
      mtf_tensor dbias = {nullptr, MTF_F32, 1, bd};
      mtf_epilogue e;
      e.scale = 1.f; e.relu = 0; e.bias = nullptr; e.relu_mask = &hs; e.residual = nullptr; e.reduce_sum_out = &dbias;
      mtf_status st = mtf_einsum_workspace_bytes(layout, 2, in, &c.c, idx == 2 ? &e : nullptr, &b);
      if (st != MTF_OK) return st;
      scratch = std::max(scratch, b);
      ++idx;
    }
  }
  *bytes = align256((size_t)numel(dhp) * elem_bytes(dhp.dtype)) + align256(scratch) + 256;
  return MTF_OK;
}

mtf_status mtf_ffn_backward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* v,
                            const mtf_tensor* h_saved, const mtf_tensor* dy, mtf_tensor* dx, mtf_tensor* dw, mtf_tensor* dbias,
                            mtf_tensor* dv, void* workspace, size_t workspace_bytes, void* stream) {
  mtf_status st = mtf::ffn_backward_impl(layout, x, w, v, h_saved, dy, dx, nullptr, dw, dbias, dv, workspace, workspace_bytes, stream);
  return st != MTF_OK ? st : mtf::rank_wait(layout, stream);
}

}  // extern "C"

mtf_status mtf::einsum_terms(const mtf_layout_t* layout, int n_terms, const mtf_tensor (*terms)[2], mtf_tensor* out,
                             const mtf_epilogue* epilogue, void* workspace, size_t workspace_bytes, void* stream) {
  if (!layout || !terms || !out || n_terms < 1 || n_terms > 3) return fail(MTF_ERR_INVALID_ARG, "einsum_terms: bad argument");
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, 2, terms[0], out, epilogue, &P);
  if (st != MTF_OK) return st;
  if (n_terms == 1) return exec_plan(P, terms[0], out, epilogue, workspace, workspace_bytes, stream);
  if (P->kernel_kind != MTF_KERNEL_TCGEN05 || P->reduce_mode == MTF_REDUCE_WORKSPACE)
    return fail(MTF_ERR_UNSUPPORTED, "einsum_terms: this plan takes one product per launch");
  const void* extra[4] = {nullptr, nullptr, nullptr, nullptr};
  for (int i = 1; i < n_terms; ++i)
    for (int q = 0; q < 2; ++q) {
      const mtf_tensor& a = terms[0][q];
      const mtf_tensor& b = terms[i][q];
      bool same = a.ndim == b.ndim && a.dtype == b.dtype && b.data != nullptr;
      for (int d = 0; same && d < a.ndim; ++d) same = a.dims[d].size == b.dims[d].size;
      if (!same) return fail(MTF_ERR_SIZE_MISMATCH, "einsum_terms: term %d operand %d differs in shape or type from term 0", i, q);
      extra[2 * (i - 1) + q] = b.data;
    }
  return exec_plan(P, terms[0], out, epilogue, workspace, workspace_bytes, stream, n_terms, extra);
}

void mtf::hint_next_launch_independent() { g_next_independent = true; }
int mtf::swap_force_reduce(int mode) { const int was = g_force_reduce; g_force_reduce = mode; return was; }
bool mtf::take_independent_hint() {
  const bool v = g_next_independent;
  g_next_independent = false;
  return v;
}

mtf_status mtf::einsum_group(const mtf_layout_t* layout, int n_groups, const mtf_tensor (*ins)[2], mtf_tensor* const* outs,
                             void* workspace, size_t workspace_bytes, void* stream) {
  if (!layout || !ins || !outs || n_groups < 1 || n_groups > 3) return fail(MTF_ERR_INVALID_ARG, "einsum_group: bad argument");
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, 2, ins[0], outs[0], nullptr, &P);
  if (st != MTF_OK) return st;
  if (n_groups == 1) return exec_plan(P, ins[0], outs[0], nullptr, workspace, workspace_bytes, stream);
  if (P->kernel_kind != MTF_KERNEL_TCGEN05) return fail(MTF_ERR_UNSUPPORTED, "einsum_group: this plan runs one problem per launch");
  const void* ops[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  for (int g = 1; g < n_groups; ++g) {
    const mtf_tensor* cand[3] = {&ins[g][0], &ins[g][1], outs[g]};
    const mtf_tensor* ref[3] = {&ins[0][0], &ins[0][1], outs[0]};
    for (int q = 0; q < 3; ++q) {
      bool same = cand[q] && cand[q]->ndim == ref[q]->ndim && cand[q]->dtype == ref[q]->dtype && cand[q]->data != nullptr;
      for (int d = 0; same && d < ref[q]->ndim; ++d) same = cand[q]->dims[d].size == ref[q]->dims[d].size;
      if (!same) return fail(MTF_ERR_SIZE_MISMATCH, "einsum_group: problem %d tensor %d differs in shape or type from problem 0", g, q);
      ops[3 * (g - 1) + q] = cand[q]->data;
    }
  }
  return exec_plan(P, ins[0], outs[0], nullptr, workspace, workspace_bytes, stream, 1, nullptr, 0, n_groups, ops);
}

mtf_status mtf::einsum_row_softmax(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, mtf_tensor* weights, float scale,
                                   int causal, void* workspace, size_t workspace_bytes, void* stream) {
  if (!layout || !a || !b || !weights) return fail(MTF_ERR_INVALID_ARG, "einsum_row_softmax: NULL argument");
  mtf_epilogue e;
  e.scale = scale; e.relu = 0; e.bias = nullptr; e.relu_mask = nullptr; e.residual = nullptr; e.reduce_sum_out = nullptr;
  const mtf_tensor in[2] = {*a, *b};
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, 2, in, weights, &e, &P);
  if (st != MTF_OK) return st;
  if (P->kernel_kind != MTF_KERNEL_TCGEN05 || P->tc.swapped) return fail(MTF_ERR_UNSUPPORTED, "einsum_row_softmax: not on this plan");
  // the causal limit compares a row's position with the column: the rows of the contraction must be one dimension
  if (causal && (weights->ndim < 2 || weights->dims[weights->ndim - 2].size != P->tc.M || weights->dims[weights->ndim - 1].size != P->tc.N))
    return fail(MTF_ERR_UNSUPPORTED, "einsum_row_softmax: a causal mask needs the two last output dimensions to be the rows and columns of the contraction");
  return exec_plan(P, in, weights, &e, workspace, workspace_bytes, stream, 1, nullptr, causal ? 2 : 1);
}

// out = a . b (plain, bf16) with the per-row statistics of a log-sum-exp left at the head of the workspace by the
// epilogue: float2 [rows][*parts] (maximum, sum of exp(value - maximum)) of the stored values of every column part.
mtf_status mtf::einsum_row_lse(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, mtf_tensor* out, void* workspace, size_t workspace_bytes,
                               void* stream, int* parts) {
  if (!layout || !a || !b || !out || !parts) return fail(MTF_ERR_INVALID_ARG, "einsum_row_lse: NULL argument");
  const mtf_tensor in[2] = {*a, *b};
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, 2, in, out, nullptr, &P);
  if (st != MTF_OK) return st;
  if (P->kernel_kind != MTF_KERNEL_TCGEN05 || P->tc.swapped || P->rank_sum || P->reduce_mode == MTF_REDUCE_WORKSPACE)
    return fail(MTF_ERR_UNSUPPORTED, "einsum_row_lse: not on this plan");
  const int64_t ns = P->tc.N / P->tc.sn;
  *parts = (int)(P->tc.sn * ((ns + P->tc.block_n - 1) / P->tc.block_n) * 2);
  return exec_plan(P, in, out, nullptr, workspace, workspace_bytes, stream, 1, nullptr, 5);
}

mtf_status mtf::einsum_row_softmax_bwd(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, const mtf_tensor* weights,
                                       mtf_tensor* dlogits, int causal, void* workspace, size_t workspace_bytes, void* stream) {
  if (!layout || !a || !b || !weights || !dlogits) return fail(MTF_ERR_INVALID_ARG, "einsum_row_softmax_bwd: NULL argument");
  mtf_epilogue e;
  e.scale = 1.f; e.relu = 0; e.bias = nullptr; e.relu_mask = weights; e.residual = nullptr; e.reduce_sum_out = nullptr;
  const mtf_tensor in[2] = {*a, *b};
  const mtf_plan_t* P = nullptr;
  mtf_status st = cached_plan(layout, 2, in, dlogits, &e, &P);
  if (st != MTF_OK) return st;
  if (P->kernel_kind != MTF_KERNEL_TCGEN05 || P->tc.swapped) return fail(MTF_ERR_UNSUPPORTED, "einsum_row_softmax_bwd: not on this plan");
  return exec_plan(P, in, dlogits, &e, workspace, workspace_bytes, stream, 1, nullptr, causal ? 4 : 3);
}

// dx_residual (NULL or a tensor with dx's dims) is added to dx in the last einsum's epilogue.
mtf_status mtf::ffn_backward_impl(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* v,
                                  const mtf_tensor* h_saved, const mtf_tensor* dy, mtf_tensor* dx, const mtf_tensor* dx_residual,
                                  mtf_tensor* dw, mtf_tensor* dbias, mtf_tensor* dv, void* workspace, size_t workspace_bytes, void* stream) {
  mtf_status st = ffn_check(x, w, v);
  if (st != MTF_OK) return st;
  if (!h_saved || !dy || !dx || !dw || !dv) return fail(MTF_ERR_INVALID_ARG, "ffn_backward: NULL tensor");
  if (h_saved->ndim != x->ndim) return fail(MTF_ERR_SIZE_MISMATCH, "ffn_backward: h_saved must be [*tokens, hidden]");
  // dhp lives at the head of the workspace
  mtf_dim hd[mtf::kMaxTensorDims];
  mtf_tensor dhp;
  ffn_dhp_desc(x, w, h_saved->dtype, hd, &dhp);
  const size_t dhp_bytes = align256((size_t)numel(dhp) * elem_bytes(dhp.dtype));
  if (!workspace || workspace_bytes < dhp_bytes) return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "ffn_backward needs at least %zu workspace bytes, got %zu", dhp_bytes, workspace_bytes);
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return fail(MTF_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  dhp.data = workspace;
  void* rest = reinterpret_cast<uint8_t*>(workspace) + dhp_bytes;
  const size_t rest_bytes = workspace_bytes - dhp_bytes;

  // dhp = (dy . v^T) * [h > 0]   (relu'(0) = 0)
  mtf_epilogue e1;
  // dbias = sum over tokens of dhp rides in the same launch when it is an f32 tensor
  const bool fuse_dbias = dbias && dbias->dtype == MTF_F32;
  e1.scale = 1.f; e1.relu = 0; e1.bias = nullptr; e1.relu_mask = h_saved; e1.residual = nullptr;
  e1.reduce_sum_out = fuse_dbias ? dbias : nullptr;
  mtf_tensor in1[2] = {*dy, *v};
  if ((st = mtf_einsum(layout, nullptr, 2, in1, &dhp, &e1, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = mtf::tap("dhp", dhp, stream)) != MTF_OK) return st;
  // dv = h^T . dy  and  dw = x^T . dhp  reduce out the token dims (Section 8.1)
  mtf_tensor in2[2] = {*h_saved, *dy};
  mtf::hint_next_launch_independent();        // dv reads h and dy, which the dhp launch only reads, and writes dv
  if ((st = mtf_einsum(layout, nullptr, 2, in2, dv, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  mtf_tensor in3[2] = {*x, dhp};
  if ((st = mtf_einsum(layout, nullptr, 2, in3, dw, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  if (dbias && !fuse_dbias && (st = mtf_reduce_sum(layout, &dhp, dbias, stream)) != MTF_OK) return st;
  // dx = dhp . w^T reduces out hidden (Section 8.2)
  mtf_tensor in4[2] = {dhp, *w};
  mtf_epilogue e4;
  e4.scale = 1.f; e4.relu = 0; e4.bias = nullptr; e4.relu_mask = nullptr; e4.residual = dx_residual; e4.reduce_sum_out = nullptr;
  if (!(dbias && !fuse_dbias)) mtf::hint_next_launch_independent();      // dx reads dhp and w and writes dx; the dw launch before it reads x and dhp and writes dw
  return mtf_einsum(layout, nullptr, 2, in4, dx, dx_residual ? &e4 : nullptr, rest, rest_bytes, stream);
}

extern "C" {

const char* mtf_status_string(mtf_status s) {
  switch (s) {
    case MTF_OK: return "MTF_OK";
    case MTF_ERR_INVALID_ARG: return "MTF_ERR_INVALID_ARG";
    case MTF_ERR_DUPLICATE_DIM: return "MTF_ERR_DUPLICATE_DIM";
    case MTF_ERR_UNKNOWN_DIM: return "MTF_ERR_UNKNOWN_DIM";
    case MTF_ERR_SIZE_MISMATCH: return "MTF_ERR_SIZE_MISMATCH";
    case MTF_ERR_ILLEGAL_LAYOUT: return "MTF_ERR_ILLEGAL_LAYOUT";
    case MTF_ERR_NOT_DIVISIBLE: return "MTF_ERR_NOT_DIVISIBLE";
    case MTF_ERR_UNSUPPORTED: return "MTF_ERR_UNSUPPORTED";
    case MTF_ERR_WORKSPACE_TOO_SMALL: return "MTF_ERR_WORKSPACE_TOO_SMALL";
    case MTF_ERR_CUDA: return "MTF_ERR_CUDA";
    case MTF_ERR_TIMEOUT: return "MTF_ERR_TIMEOUT";
  }
  return "MTF_ERR_?";
}

const char* mtf_last_error(void) { return mtf::last_error(); }

mtf_status mtf_device_status(int32_t* code) {
  int c = 0;
  mtf_status st = mtf::read_device_status(&c);
  if (code) *code = c;
  if (st != MTF_OK) return st;
  int rc = 0;
  if ((st = mtf::read_attention_status(&rc)) != MTF_OK) return st;
  if (!rc && (st = mtf::read_attention_bwd_status(&rc)) != MTF_OK) return st;
  if (!rc && (st = mtf::read_row_status(&rc)) != MTF_OK) return st;
  if (rc) {
    if (code) *code = rc;
    return fail(MTF_ERR_TIMEOUT, "a bounded device-side wait gave up (code 0x%x)", rc);
  }
  int bad = 0;
  if ((st = mtf::read_bad_index(&bad)) != MTF_OK) return st;
  if (bad) return fail(MTF_ERR_INVALID_ARG, "a token id or target outside [0, vocab) was seen by the vocab kernels");
  return MTF_OK;
}

int64_t mtf_launch_count(void) { return mtf::launch_count(); }

mtf_status mtf_debug_wait_test(int64_t limit_cycles, int32_t withhold_one_signal) { return mtf::debug_wait_test(limit_cycles, withhold_one_signal); }

mtf_status mtf_stage_tap_begin(void* device_buffer, size_t bytes) { return mtf::tap_begin(device_buffer, bytes); }
mtf_status mtf_stage_tap_end(int32_t* n_entries) { return mtf::tap_end(n_entries); }
mtf_status mtf_stage_tap_entry(int32_t index, const char** name, size_t* offset, size_t* bytes) { return mtf::tap_entry(index, name, offset, bytes); }

}  // extern "C"
