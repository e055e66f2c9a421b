// Host planner: named dimensions, mesh, computation layout, slice boxes and einsum planning.
//
// Follows the paper's rules: a tensor's layout is the restriction of the computation layout to its
// dimensions and must be injective, split sizes must divide (Section 5); a processor's slice is the
// contiguous block selected by its mesh coordinate (Section 5); an einsum is a local einsum per
// processor followed by a sum over the mesh dimensions of reduced-out split dimensions (Section 6).
// On one GPU the plan turns that into: which distinct slices exist, which of them form a reduce
// group, and how the grouped kernel walks them.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <set>

#include "mtf_internal.h"

namespace mtf {

static thread_local char g_err[512] = "";

// bf16 contractions above this many multiply-adds are not sent to the generic kernel unasked (2^30: ~0.1 s there)
constexpr double kGenericKernelMacLimit = 1073741824.0;

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

mtf_status fail(mtf_status s, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return s;
}

const char* last_error() { return g_err; }

mtf_status read_dims(int32_t ndim, const mtf_dim* dims, std::vector<Dim>* out, const char* what) {
  out->clear();
  if (ndim < 0 || ndim > kMaxTensorDims) return fail(MTF_ERR_INVALID_ARG, "%s: ndim %d outside [0, %d]", what, ndim, kMaxTensorDims);
  if (ndim > 0 && !dims) return fail(MTF_ERR_INVALID_ARG, "%s: dims is NULL", what);
  for (int i = 0; i < ndim; ++i) {
    if (!dims[i].name || !dims[i].name[0]) return fail(MTF_ERR_INVALID_ARG, "%s: dimension %d has no name", what, i);
    if (dims[i].size <= 0) return fail(MTF_ERR_INVALID_ARG, "%s: dimension '%s' has size %lld", what, dims[i].name, (long long)dims[i].size);
    for (auto& d : *out)
      if (d.name == dims[i].name) return fail(MTF_ERR_DUPLICATE_DIM, "%s: dimension name '%s' appears twice", what, dims[i].name);
    out->push_back({dims[i].name, dims[i].size});
  }
  return MTF_OK;
}

std::vector<int64_t> row_major_strides(const std::vector<Dim>& dims) {
  std::vector<int64_t> s(dims.size(), 1);
  for (int i = (int)dims.size() - 2; i >= 0; --i) s[i] = s[i + 1] * dims[i + 1].size;
  return s;
}

// Section 5: restriction of the layout to one tensor must be injective; sizes must divide.
mtf_status check_tensor(const mtf_layout_t* L, const std::vector<Dim>& dims) {
  int owner[kMaxMeshDims];
  for (int j = 0; j < kMaxMeshDims; ++j) owner[j] = -1;
  for (size_t i = 0; i < dims.size(); ++i) {
    int j = L->mesh_dim_of(dims[i].name);
    if (j < 0) continue;
    if (owner[j] >= 0)
      return fail(MTF_ERR_ILLEGAL_LAYOUT, "dimensions '%s' and '%s' are both split over mesh dimension '%s'",
                  dims[owner[j]].name.c_str(), dims[i].name.c_str(), L->mesh[j].name.c_str());
    owner[j] = (int)i;
    if (dims[i].size % L->mesh[j].size != 0)
      return fail(MTF_ERR_NOT_DIVISIBLE, "dimension '%s' of size %lld is not divisible by mesh dimension '%s' of size %lld",
                  dims[i].name.c_str(), (long long)dims[i].size, L->mesh[j].name.c_str(), (long long)L->mesh[j].size);
  }
  return MTF_OK;
}

static void mesh_coords(const std::vector<Dim>& mesh, int64_t p, int64_t* c) {
  for (int j = (int)mesh.size() - 1; j >= 0; --j) {   // last mesh dimension varies fastest
    c[j] = p % mesh[j].size;
    p /= mesh[j].size;
  }
}

mtf_status slice_box(const mtf_layout_t* L, const std::vector<Dim>& dims, int64_t p, int64_t* offs, int64_t* sizes) {
  mtf_status st = check_tensor(L, dims);
  if (st != MTF_OK) return st;
  int64_t P = 1;
  for (auto& m : L->mesh) P *= m.size;
  if (p < 0 || p >= P) return fail(MTF_ERR_INVALID_ARG, "processor %lld outside mesh of %lld", (long long)p, (long long)P);
  int64_t c[kMaxMeshDims];
  mesh_coords(L->mesh, p, c);
  for (size_t i = 0; i < dims.size(); ++i) {
    int j = L->mesh_dim_of(dims[i].name);
    if (j < 0) {
      offs[i] = 0;
      sizes[i] = dims[i].size;
    } else {
      int64_t t = dims[i].size / L->mesh[j].size;
      offs[i] = c[j] * t;
      sizes[i] = t;
    }
  }
  return MTF_OK;
}

static const char* dt_name(int dt) { return dt == MTF_BF16 ? "bf16" : "f32"; }

std::string plan_key(int n_in, const mtf_tensor* in, const mtf_tensor* out, const mtf_epilogue* epi, int fk, int fr) {
  std::string k;
  auto add_t = [&](const mtf_tensor* t) {
    k += dt_name(t->dtype);
    k += '[';
    for (int i = 0; i < t->ndim; ++i) {
      k += t->dims[i].name ? t->dims[i].name : "?";
      k += ':';
      k += std::to_string((long long)t->dims[i].size);
      k += ',';
    }
    k += ']';
  };
  for (int q = 0; q < n_in; ++q) add_t(&in[q]);
  k += "->";
  add_t(out);
  if (epi) {
    k += "|e";
    k += epi->relu ? 'r' : '-';
    k += (epi->scale != 1.f) ? 's' : '-';
    if (epi->bias) { k += 'b'; add_t(epi->bias); }
    if (epi->relu_mask) { k += 'm'; k += dt_name(epi->relu_mask->dtype); }
    if (epi->residual) { k += 'a'; k += dt_name(epi->residual->dtype); }
    if (epi->reduce_sum_out) { k += 'S'; add_t(epi->reduce_sum_out); }
  }
  k += "|f" + std::to_string(fk) + "," + std::to_string(fr);
  return k;
}

static bool same_dims(const std::vector<Dim>& a, const std::vector<Dim>& b) {
  if (a.size() != b.size()) return false;
  for (size_t i = 0; i < a.size(); ++i)
    if (a[i].name != b[i].name || a[i].size != b[i].size) return false;
  return true;
}

// Merge the iteration dims of one category into a single (size, stride) per operand.  `idx` lists
// the dims; they are ordered by descending stride in the first operand that has them and must nest
// contiguously, in the same order, in every operand that carries the category.
struct Merged {
  bool ok = false;
  int64_t size = 1;
  int64_t sA = 0, sB = 0, sC = 0;
  int64_t nsplit = 1;
  int split_mesh_dim = -1;
};

static Merged merge_category(const std::vector<IterDim>& it, std::vector<int> idx, bool useA, bool useB, bool useC) {
  Merged m;
  if (idx.empty()) { m.ok = true; return m; }
  auto stride_of = [&](int i, int which) { return which == 0 ? it[i].sA : which == 1 ? it[i].sB : it[i].sC; };
  int first = useA ? 0 : (useB ? 1 : 2);
  std::sort(idx.begin(), idx.end(), [&](int a, int b) { return stride_of(a, first) > stride_of(b, first); });
  for (int which = 0; which < 3; ++which) {
    if ((which == 0 && !useA) || (which == 1 && !useB) || (which == 2 && !useC)) continue;
    for (size_t j = 0; j + 1 < idx.size(); ++j)
      if (stride_of(idx[j], which) != it[idx[j + 1]].size * stride_of(idx[j + 1], which)) return m;
  }
  for (int i : idx) m.size *= it[i].size;
  int inner = idx.back();
  m.sA = useA ? it[inner].sA : 0;
  m.sB = useB ? it[inner].sB : 0;
  m.sC = useC ? it[inner].sC : 0;
  // a split is expressible as equal contiguous blocks only on the outermost component
  for (size_t j = 0; j < idx.size(); ++j) {
    if (it[idx[j]].nsplit > 1) {
      if (j != 0) return m;
      m.nsplit = it[idx[j]].nsplit;
      m.split_mesh_dim = it[idx[j]].mesh_dim;
    }
  }
  m.ok = true;
  return m;
}

static bool plan_tc(mtf_plan_t* P, std::string* why, int force_single_cta) {
  const auto& it = P->iter;
  if (!P->has_B) { *why = "one operand"; return false; }
  if (P->dtA != MTF_BF16 || P->dtB != MTF_BF16) { *why = "operands are not bf16"; return false; }
  std::vector<int> cb, cm, cn, ck;
  for (int i = 0; i < (int)it.size(); ++i) {
    const IterDim& d = it[i];
    if (d.inA && d.inB && d.inC) cb.push_back(i);
    else if (d.inA && !d.inB && d.inC) cm.push_back(i);
    else if (!d.inA && d.inB && d.inC) cn.push_back(i);
    else if (d.inA && d.inB && !d.inC) ck.push_back(i);
    else { *why = "a reduced dimension belongs to one operand only"; return false; }
  }
  if (cm.empty() || cn.empty() || ck.empty()) { *why = "no M, N or K dimension"; return false; }
  if ((int)cb.size() > kMaxOuter) { *why = "more than three batch dimensions"; return false; }
  Merged mm = merge_category(it, cm, true, false, true);
  Merged mn = merge_category(it, cn, false, true, true);
  Merged mk = merge_category(it, ck, true, true, false);
  if (!mm.ok || !mn.ok || !mk.ok) { *why = "a dimension group does not merge into one strided dimension"; return false; }

  TcParams t;
  // batch dims ordered by descending stride in C
  std::sort(cb.begin(), cb.end(), [&](int a, int b) { return it[a].sC > it[b].sC; });
  t.n_outer = (int)cb.size();
  for (int j = 0; j < t.n_outer; ++j) {
    t.outer_size[j] = it[cb[j]].size;
    t.outer_split[j] = it[cb[j]].nsplit;
    t.outer_sA[j] = it[cb[j]].sA;
    t.outer_sB[j] = it[cb[j]].sB;
    t.outer_sC[j] = it[cb[j]].sC;
  }
  // C must have N contiguous; if M is contiguous instead, exchange the operands' roles.
  bool swap = false;
  if (mn.sC != 1) {
    if (mm.sC == 1) swap = true;
    else { *why = "neither M nor N is contiguous in the output"; return false; }
  }
  Merged a_m = swap ? mn : mm, b_n = swap ? mm : mn;
  // strides of the "A" role operand: over its M-like dim and over K
  int64_t a_sM = swap ? mn.sB : mm.sA, a_sK = swap ? mk.sB : mk.sA;
  int64_t b_sN = swap ? mm.sA : mn.sB, b_sK = swap ? mk.sA : mk.sB;
  if (swap)
    for (int j = 0; j < t.n_outer; ++j) std::swap(t.outer_sA[j], t.outer_sB[j]);
  t.swapped = swap ? 1 : 0;
  t.M = a_m.size; t.N = b_n.size; t.K = mk.size;
  t.sm = a_m.nsplit; t.sn = b_n.nsplit; t.sk = mk.nsplit;
  t.ldc = swap ? mn.sC : mm.sC;
  auto major = [&](int64_t s_mn, int64_t s_k, int64_t ext_mn, int64_t ext_k, int* mn_major, int64_t* ld) {
    if (s_k == 1 && (s_mn % 8 == 0 || ext_mn == 1)) { *mn_major = 0; *ld = s_mn; return true; }
    if (s_mn == 1 && (s_k % 8 == 0 || ext_k == 1)) { *mn_major = 1; *ld = s_k; return true; }
    return false;
  };
  if (!major(a_sM, a_sK, t.M, t.K, &t.a_mn_major, &t.a_ld) || !major(b_sN, b_sK, t.N, t.K, &t.b_mn_major, &t.b_ld)) {
    *why = "an operand has no unit-stride M/N or K dimension with 16-byte aligned rows";
    return false;
  }
  for (int j = 0; j < t.n_outer; ++j)
    if (t.outer_sA[j] % 8 || t.outer_sB[j] % 8) { *why = "batch stride not 16-byte aligned"; return false; }
  // A tensor-map copy must start on a 16-byte boundary along the contiguous dimension.  For an operand
  // whose M / N dimension is the contiguous one the first column of a slice is a multiple of the slice
  // extent, so that extent must be a multiple of 8 bf16 elements (k offsets are always multiples of a 64-element k-block:
  // the slices of a split K are contiguous and walked as one range).
  if (t.a_mn_major && t.sm > 1 && (t.M / t.sm) % 8) { *why = "M slices of an M-contiguous operand do not start on 16-byte boundaries"; return false; }
  if (t.b_mn_major && t.sn > 1 && (t.N / t.sn) % 8) { *why = "N slices of an N-contiguous operand do not start on 16-byte boundaries"; return false; }
  // vectorised epilogue stores: rows of C must start 16-byte aligned
  int64_t cvec = P->dtC == MTF_BF16 ? 8 : 4;
  if (t.ldc % cvec) { *why = "output rows not 16-byte aligned"; return false; }
  for (int j = 0; j < t.n_outer; ++j)
    if (t.outer_sC[j] % cvec) { *why = "output batch stride not 16-byte aligned"; return false; }
  if ((t.N / t.sn) % cvec) { *why = "N slice extent not a multiple of the store vector"; return false; }
  // epilogue operands
  if (P->epi.has_bias) {
    // bias must vary along exactly the N group (or the M group after a swap), matching its merge
    const auto& bd = P->epi.bias_dims;
    const std::vector<int>& want = swap ? cm : cn;    // the kernel's N group
    const std::vector<int>& other = swap ? cn : cm;   // the kernel's M group
    auto covers = [&](const std::vector<int>& grp) {
      if (bd.size() != grp.size()) return false;
      std::vector<int> g = grp;
      std::sort(g.begin(), g.end(), [&](int a, int b) { return it[a].sC > it[b].sC; });
      for (size_t j = 0; j < g.size(); ++j)
        if (bd[j].name != it[g[j]].name) return false;
      return true;
    };
    if (covers(want)) t.bias_along_m = 0;
    else if (covers(other)) t.bias_along_m = 1;
    else { *why = "bias dims are not exactly the N (or M) group in storage order"; return false; }
  }
  if (P->epi.has_rsum && P->epi.has_res) { *why = "reduce_sum_out together with a residual"; return false; }
  if (P->epi.has_rsum) {
    const auto& rd = P->epi.rsum_dims;
    std::vector<int> g = swap ? cm : cn;              // the kernel's N group
    std::sort(g.begin(), g.end(), [&](int a, int b) { return it[a].sC > it[b].sC; });
    bool same = rd.size() == g.size();
    for (size_t j = 0; same && j < g.size(); ++j) same = rd[j].name == it[g[j]].name;
    if (!same) { *why = "reduce_sum_out dims are not exactly the contiguous output group"; return false; }
  }
  int64_t Ns = t.N / t.sn;
  t.block_n = Ns > 128 ? 256 : (Ns > 64 ? 128 : 64);
  // CTA pairs need a B half of at least one 64-wide swizzle block and pay off on tall slices
  t.cta_pair = (t.block_n >= 128 && t.M / t.sm > 128 && force_single_cta == 0) ? 1 : 0;
  P->tc = t;
  return true;
}

mtf_status make_plan(const mtf_layout_t* L, int n_in, const mtf_tensor* in, const mtf_tensor* out,
                     const mtf_epilogue* epi, int force_kernel, int force_reduce, std::unique_ptr<mtf_plan_t>* result) {
  if (!L || !in || !out) return fail(MTF_ERR_INVALID_ARG, "einsum: NULL argument");
  if (n_in < 1 || n_in > 2) return fail(MTF_ERR_UNSUPPORTED, "einsum: the GPU path takes 1 or 2 inputs, got %d", n_in);
  std::unique_ptr<mtf_plan_t> P(new mtf_plan_t());
  P->mesh = L->mesh;
  mtf_status st;
  if ((st = read_dims(in[0].ndim, in[0].dims, &P->dimsA, "einsum input 0")) != MTF_OK) return st;
  P->has_B = n_in == 2;
  if (P->has_B && (st = read_dims(in[1].ndim, in[1].dims, &P->dimsB, "einsum input 1")) != MTF_OK) return st;
  if ((st = read_dims(out->ndim, out->dims, &P->dimsC, "einsum output")) != MTF_OK) return st;
  auto dt_ok = [](int d) { return d == MTF_F32 || d == MTF_BF16; };
  if (!dt_ok(in[0].dtype) || (P->has_B && !dt_ok(in[1].dtype)) || !dt_ok(out->dtype)) return fail(MTF_ERR_INVALID_ARG, "einsum: unknown dtype");
  P->dtA = in[0].dtype; P->dtB = P->has_B ? in[1].dtype : MTF_F32; P->dtC = out->dtype;

  // iteration space = union of the input dims (Section 6); sizes must agree by name
  auto sA = row_major_strides(P->dimsA), sB = row_major_strides(P->dimsB), sC = row_major_strides(P->dimsC);
  auto find = [&](const std::string& n) -> IterDim* {
    for (auto& d : P->iter) if (d.name == n) return &d;
    return nullptr;
  };
  for (size_t i = 0; i < P->dimsA.size(); ++i) {
    IterDim d; d.name = P->dimsA[i].name; d.size = P->dimsA[i].size; d.inA = true; d.sA = sA[i];
    P->iter.push_back(d);
  }
  for (size_t i = 0; i < P->dimsB.size(); ++i) {
    IterDim* e = find(P->dimsB[i].name);
    if (e) {
      if (e->size != P->dimsB[i].size) return fail(MTF_ERR_SIZE_MISMATCH, "dimension '%s' has sizes %lld and %lld", e->name.c_str(), (long long)e->size, (long long)P->dimsB[i].size);
      e->inB = true; e->sB = sB[i];
    } else {
      IterDim d; d.name = P->dimsB[i].name; d.size = P->dimsB[i].size; d.inB = true; d.sB = sB[i];
      P->iter.push_back(d);
    }
  }
  for (size_t i = 0; i < P->dimsC.size(); ++i) {
    IterDim* e = find(P->dimsC[i].name);
    if (!e) return fail(MTF_ERR_UNKNOWN_DIM, "output dimension '%s' is in no input", P->dimsC[i].name.c_str());
    if (e->size != P->dimsC[i].size) return fail(MTF_ERR_SIZE_MISMATCH, "output dimension '%s' has size %lld, inputs have %lld", e->name.c_str(), (long long)P->dimsC[i].size, (long long)e->size);
    e->inC = true; e->sC = sC[i];
  }
  if ((int)P->iter.size() > kMaxIterDims) return fail(MTF_ERR_UNSUPPORTED, "more than %d distinct dimensions", kMaxIterDims);

  // legality: every operand, and the whole iteration space (two different split dims of one
  // operation on one mesh dim would give each processor only matching blocks)
  if ((st = check_tensor(L, P->dimsA)) != MTF_OK) return st;
  if (P->has_B && (st = check_tensor(L, P->dimsB)) != MTF_OK) return st;
  if ((st = check_tensor(L, P->dimsC)) != MTF_OK) return st;
  {
    std::vector<Dim> all;
    for (auto& d : P->iter) all.push_back({d.name, d.size});
    if ((st = check_tensor(L, all)) != MTF_OK) return st;
  }
  for (auto& d : P->iter) {
    d.mesh_dim = L->mesh_dim_of(d.name);
    d.nsplit = d.mesh_dim >= 0 ? L->mesh[d.mesh_dim].size : 1;
  }

  // epilogue
  if (epi) {
    P->epi.on = true;
    P->epi.scale = epi->scale;
    P->epi.relu = epi->relu != 0;
    if (epi->bias) {
      P->epi.has_bias = true;
      if (!dt_ok(epi->bias->dtype)) return fail(MTF_ERR_INVALID_ARG, "bias: unknown dtype");
      P->epi.dtBias = epi->bias->dtype;
      if ((st = read_dims(epi->bias->ndim, epi->bias->dims, &P->epi.bias_dims, "bias")) != MTF_OK) return st;
      for (auto& b : P->epi.bias_dims) {
        IterDim* e = find(b.name);
        if (!e || !e->inC) return fail(MTF_ERR_UNKNOWN_DIM, "bias dimension '%s' is not an output dimension", b.name.c_str());
        if (e->size != b.size) return fail(MTF_ERR_SIZE_MISMATCH, "bias dimension '%s' has size %lld, output has %lld", b.name.c_str(), (long long)b.size, (long long)e->size);
      }
    }
    if (epi->reduce_sum_out) {
      P->epi.has_rsum = true;
      if (epi->reduce_sum_out->dtype != MTF_F32) return fail(MTF_ERR_UNSUPPORTED, "reduce_sum_out must be f32");
      if ((st = read_dims(epi->reduce_sum_out->ndim, epi->reduce_sum_out->dims, &P->epi.rsum_dims, "reduce_sum_out")) != MTF_OK) return st;
      for (auto& b : P->epi.rsum_dims) {
        IterDim* e = find(b.name);
        if (!e || !e->inC) return fail(MTF_ERR_UNKNOWN_DIM, "reduce_sum_out dimension '%s' is not an output dimension", b.name.c_str());
        if (e->size != b.size) return fail(MTF_ERR_SIZE_MISMATCH, "reduce_sum_out dimension '%s' has size %lld, output has %lld", b.name.c_str(), (long long)b.size, (long long)e->size);
      }
    }
    for (int which = 0; which < 2; ++which) {
      const mtf_tensor* t = which == 0 ? epi->relu_mask : epi->residual;
      if (!t) continue;
      std::vector<Dim> td;
      if ((st = read_dims(t->ndim, t->dims, &td, which == 0 ? "relu_mask" : "residual")) != MTF_OK) return st;
      if (!same_dims(td, P->dimsC)) return fail(MTF_ERR_SIZE_MISMATCH, "%s must have exactly the output's dims and order", which == 0 ? "relu_mask" : "residual");
      if (!dt_ok(t->dtype)) return fail(MTF_ERR_INVALID_ARG, "epilogue operand: unknown dtype");
      if (which == 0) { P->epi.has_mask = true; P->epi.dtMask = t->dtype; }
      else { P->epi.has_res = true; P->epi.dtRes = t->dtype; }
    }
  }

  // reduce group = mesh dims of reduced-out split dims (Section 6); distinct slices = product of
  // the mesh dims any dimension of the iteration space is split over (replicas computed once)
  bool used[kMaxMeshDims] = {false, false, false, false};
  P->reduce_mask = 0;
  P->group_size = 1;
  int64_t macs = 1;
  for (auto& d : P->iter) {
    macs *= d.size / d.nsplit;
    if (d.mesh_dim >= 0) {
      used[d.mesh_dim] = true;
      if (!d.inC) {
        P->reduce_mask |= 1u << d.mesh_dim;
        P->group_size *= d.nsplit;
      }
    }
  }
  P->n_slices = 1;
  for (size_t j = 0; j < L->mesh.size(); ++j)
    if (used[j]) P->n_slices *= L->mesh[j].size;
  P->n_reduce_mesh_dims = 0;
  for (int j = 0; j < kMaxMeshDims; ++j)
    if (P->reduce_mask & (1u << j)) ++P->n_reduce_mesh_dims;
  auto local_elems = [&](const std::vector<Dim>& dims) {
    int64_t n = 1;
    for (auto& d : dims) {
      int j = L->mesh_dim_of(d.name);
      n *= j >= 0 ? d.size / L->mesh[j].size : d.size;
    }
    return n;
  };
  P->macs_per_proc = macs;
  int64_t out_slice = local_elems(P->dimsC);
  P->allreduce_values = P->reduce_mask ? out_slice : 0;
  P->slice_elems = out_slice + local_elems(P->dimsA) + (P->has_B ? local_elems(P->dimsB) : 0);

  // ---- rank binding: which results are partial sums that the ranks still have to add up ----
  if (L->bound_dim >= 0 && L->world > 1) {
    P->rank = L->rank;
    P->ar_start = L->ar_start;
    P->ar_user = L->ar_user;
    for (auto& d : P->iter)
      if (!d.inC && L->mesh_dim_of(d.name) == L->bound_dim) P->rank_sum = true;
    if (P->epi.has_rsum)
      for (auto& d : P->iter) {
        if (!d.inC || L->mesh_dim_of(d.name) != L->bound_dim) continue;
        bool kept = false;
        for (auto& r : P->epi.rsum_dims) kept = kept || r.name == d.name;
        if (!kept) P->rsum_rank_sum = true;
      }
    if (P->rank_sum && (P->epi.has_bias || P->epi.relu || P->epi.has_mask || P->epi.has_rsum))
      return fail(MTF_ERR_UNSUPPORTED, "this einsum sums out a dimension that is split across ranks: its result on one rank is a partial sum, "
                  "which bias, relu, relu_mask and a fused reduce_sum cannot be applied to");
  }

  // ---- generic strided kernel parameters (always built: it is the fallback family) ----
  SimtParams& s = P->simt;
  s.n_out = (int)P->dimsC.size();
  for (int i = 0; i < s.n_out; ++i) {
    IterDim* e = find(P->dimsC[i].name);
    s.out_size[i] = e->size;
    s.out_sA[i] = e->sA; s.out_sB[i] = e->sB; s.out_sC[i] = e->sC;
    s.out_sBias[i] = 0;
    s.out_sRsum[i] = 0;
  }
  if (P->epi.has_rsum) {
    auto rs = row_major_strides(P->epi.rsum_dims);
    for (size_t b = 0; b < P->epi.rsum_dims.size(); ++b)
      for (int i = 0; i < s.n_out; ++i)
        if (P->dimsC[i].name == P->epi.rsum_dims[b].name) s.out_sRsum[i] = rs[b];
  }
  if (P->epi.has_bias) {
    auto bs = row_major_strides(P->epi.bias_dims);
    for (size_t b = 0; b < P->epi.bias_dims.size(); ++b)
      for (int i = 0; i < s.n_out; ++i)
        if (P->dimsC[i].name == P->epi.bias_dims[b].name) s.out_sBias[i] = bs[b];
  }
  s.total_out = 1;
  for (int i = 0; i < s.n_out; ++i) s.total_out *= s.out_size[i];
  {
    std::vector<int> red;
    for (int i = 0; i < (int)P->iter.size(); ++i) if (!P->iter[i].inC) red.push_back(i);
    std::vector<int> split = red;
    split.erase(std::remove_if(split.begin(), split.end(), [&](int i) { return P->iter[i].nsplit <= 1; }), split.end());
    std::sort(split.begin(), split.end(), [&](int a, int b) { return P->iter[a].mesh_dim < P->iter[b].mesh_dim; });
    int n = 0;
    for (int i : split) {   // group levels: ascending processor order = lower mesh-dim index outermost
      const IterDim& d = P->iter[i];
      int64_t blk = d.size / d.nsplit;
      s.lvl_extent[n] = d.nsplit; s.lvl_sA[n] = blk * d.sA; s.lvl_sB[n] = blk * d.sB; ++n;
    }
    s.n_group = n;
    for (int i : red) {
      const IterDim& d = P->iter[i];
      s.lvl_extent[n] = d.size / d.nsplit; s.lvl_sA[n] = d.sA; s.lvl_sB[n] = d.sB; ++n;
    }
    s.n_levels = n;
  }
  s.dtA = P->dtA; s.dtB = P->dtB; s.dtC = P->dtC;
  s.dtBias = P->epi.dtBias; s.dtMask = P->epi.dtMask; s.dtRes = P->epi.dtRes;
  s.has_B = P->has_B ? 1 : 0;
  s.scale = P->epi.on ? P->epi.scale : 1.f;
  s.relu = P->epi.relu ? 1 : 0;

  // ---- kernel family and reduce mode ----
  std::string why;
  const int force_single_cta = force_kernel == 2 ? 1 : 0;     // testing hook: tensor cores without CTA pairs
  const int wide_pref = force_kernel == 3 ? 1 : (force_kernel == 4 ? 0 : -1);   // testing hook: wide pair tiles always / never
  if (force_kernel >= 2) force_kernel = MTF_KERNEL_TCGEN05;
  bool tc_ok = plan_tc(P.get(), &why, force_single_cta);
  if (tc_ok) P->tc.wide_pref = wide_pref;
  if (!P->has_B && force_kernel == MTF_KERNEL_TCGEN05) force_kernel = -1;   // forcing concerns contractions only
  if (!P->has_B && force_reduce == MTF_REDUCE_WORKSPACE) force_reduce = -1;
  if (force_kernel == MTF_KERNEL_TCGEN05 && !tc_ok) return fail(MTF_ERR_UNSUPPORTED, "tensor-core path cannot run this einsum: %s", why.c_str());
  P->kernel_kind = (tc_ok && force_kernel != MTF_KERNEL_SIMT) ? MTF_KERNEL_TCGEN05 : MTF_KERNEL_SIMT;
  // A large bf16 contraction the tensor-core path declines would run ~100x slower on the generic
  // kernel (one thread per output element): refuse it with the reason instead of a silent cliff.
  // mtf_plan_force(MTF_KERNEL_SIMT, ..) is the opt-in for running it there all the same.
  if (P->kernel_kind == MTF_KERNEL_SIMT && P->has_B && !tc_ok && force_kernel != MTF_KERNEL_SIMT && P->dtA == MTF_BF16 && P->dtB == MTF_BF16) {
    double total_macs = 1.0;
    for (auto& d : P->iter) total_macs *= (double)d.size;
    if (total_macs > kGenericKernelMacLimit)
      return fail(MTF_ERR_UNSUPPORTED, "this bf16 einsum (%.3g multiply-adds) cannot run on the tensor-core path (%s) and is too large for the generic kernel; "
                  "change the shapes, or opt in with mtf_plan_force(MTF_KERNEL_SIMT, -1)", total_macs, why.c_str());
  }
  P->reduce_mode = P->group_size > 1 ? MTF_REDUCE_CHAINED : MTF_REDUCE_NONE;
  P->workspace_bytes = 0;
  if (P->kernel_kind == MTF_KERNEL_TCGEN05) {
    TcParams& t = P->tc;
    bool ws_possible = t.sk > 1 && (t.K / t.sk) % 64 == 0;
    int mode = t.sk > 1 ? MTF_REDUCE_CHAINED : MTF_REDUCE_NONE;
    if (force_reduce == MTF_REDUCE_WORKSPACE) {
      if (!ws_possible) return fail(MTF_ERR_UNSUPPORTED, "workspace reduction needs a split K with slices that are multiples of 64");
      mode = MTF_REDUCE_WORKSPACE;
    } else if (force_reduce < 0 && ws_possible) {
      // few output tiles and a long, split K: spread the group's slices over CTAs instead
      const int64_t rows = t.cta_pair ? 256 : 128;
      int64_t tiles = ((t.M / t.sm + rows - 1) / rows) * t.sm * ((t.N / t.sn + t.block_n - 1) / t.block_n) * t.sn;
      for (int j = 0; j < t.n_outer; ++j) tiles *= t.outer_size[j];
      // measured: a workspace launch costs ~22 us beyond its (shorter) main loop (clearing the counters,
      // writing and adding the fragments), the chained one ~7 us, and a k-block takes ~0.33 us, so the
      // k-blocks taken off the critical path must be worth the difference
      const int64_t kb_total = t.K / 64, kb_saved = kb_total - kb_total / t.sk;
      if (tiles * (t.cta_pair ? 4 : 2) <= device_sm_count() && t.K / t.sk >= 256 && kb_saved >= 64) mode = MTF_REDUCE_WORKSPACE;
    }
    t.reduce_mode = mode;
    P->reduce_mode = mode;
    // tail balancing: few whole waves of tiles with a large idle remainder and a long K
    t.balance = 0;
    if (mode != MTF_REDUCE_WORKSPACE && t.cta_pair && t.K >= 32 * 64) {
      int64_t tiles = ((t.M / t.sm + 255) / 256) * t.sm * ((t.N / t.sn + t.block_n - 1) / t.block_n) * t.sn;
      for (int j = 0; j < t.n_outer; ++j) tiles *= t.outer_size[j];
      const int64_t workers = device_sm_count() / 2;     // CTA pairs of the device; the launcher re-checks
      const int64_t rounds = (tiles + workers - 1) / workers;
      // Measured on the FFN shapes the fragment traffic costs more than the idle tail it removes,
      // so the schedule is only taken when asked for (mtf_plan_force reduce_mode 3).
      if (force_reduce == 3 && tiles >= workers && (double)tiles / (double)(rounds * workers) <= 0.92) t.balance = 1;
    }
    P->workspace_bytes = tc_workspace_bytes(t);
    if (P->epi.has_rsum && mode != MTF_REDUCE_WORKSPACE && !t.balance) P->workspace_bytes = std::max(P->workspace_bytes, tc_rsum_partial_bytes(t));
  } else if (force_reduce == MTF_REDUCE_WORKSPACE) {
    return fail(MTF_ERR_UNSUPPORTED, "workspace reduction exists only on the tensor-core path");
  }
  *result = std::move(P);
  return MTF_OK;
}

}  // namespace mtf
