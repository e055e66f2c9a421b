// Block compositions above the einsum: softmax, layer normalisation, multi-head attention and the
// Transformer decoder layer, forward and backward.  Every contraction goes through mtf_einsum (so it
// is planned under the layout and runs in the grouped tensor-core kernel); the row kernels do the
// reductions.  The paper gives the layout of these blocks (Section 9: batch, heads and d_ff are the
// split dimensions) and defers their maths to the Transformer of Vaswani et al.; the formulas are
// restated next to each function.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <initializer_list>

#include "mtf_internal.h"

namespace mtf {
mtf_status launch_softmax_fwd(const float* logits, void* weights, int64_t rows, int n, int L, int causal, void* stream);
mtf_status launch_softmax_bwd(const void* P, const float* dP, void* dlg, int64_t rows, int n, void* stream);
mtf_status launch_layernorm_fwd(const void* x, const float* gamma, const float* beta, void* y, float* stats, int64_t rows, int n, float eps, void* stream);
mtf_status launch_layernorm_bwd(const void* dy, const void* x, const float* stats, const float* gamma, const void* residual, void* dx,
                                float* dgamma, float* dbeta, int64_t rows, int n, void* scratch, size_t scratch_bytes, void* stream);
size_t layernorm_bwd_scratch_bytes(int n);
bool attention_fused_supported(int64_t L, int64_t d_k, int64_t d_v);
bool attention_bwd_fused_supported(int64_t L, int64_t d_k, int64_t d_v);
mtf_status launch_attention_bwd_fused(const void* q, const void* kk, const void* vv, const void* weights, const void* dout, void* dq, void* dkk, void* dvv,
                                      void* dlogits_dump, int64_t B, int64_t H, int64_t L, float scale, int causal, void* stream);
bool tap_is_open();
mtf_status launch_attention_fwd_fused(const void* q, const void* kk, const void* vv, void* weights, void* o, int64_t B, int64_t H, int64_t L, float scale,
                                      int causal, void* stream);
mtf_status ffn_forward_impl(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* bias, const mtf_tensor* v,
                            mtf_tensor* h_saved, mtf_tensor* y, const mtf_tensor* y_residual, void* workspace, size_t workspace_bytes, void* stream);
mtf_status ffn_backward_impl(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w, const mtf_tensor* v, const mtf_tensor* h_saved,
                             const mtf_tensor* dy, mtf_tensor* dx, const mtf_tensor* dx_residual, mtf_tensor* dw, mtf_tensor* dbias, mtf_tensor* dv,
                             void* workspace, size_t workspace_bytes, void* stream);
}  // namespace mtf

using mtf::fail;

namespace {

// A tensor descriptor that owns its dims array.
struct TD {
  mtf_dim d[mtf::kMaxTensorDims];
  mtf_tensor t;
  TD() { t.data = nullptr; t.dtype = MTF_BF16; t.ndim = 0; t.dims = d; }
  TD(const TD& o) { *this = o; }
  TD& operator=(const TD& o) {
    for (int i = 0; i < o.t.ndim; ++i) d[i] = o.d[i];
    t = o.t;
    t.dims = d;
    return *this;
  }
  static TD make(mtf_dtype dt, std::initializer_list<mtf_dim> dims, void* data = nullptr) {
    TD r;
    int i = 0;
    for (auto& x : dims) r.d[i++] = x;
    r.t.ndim = i;
    r.t.dtype = dt;
    r.t.data = data;
    return r;
  }
  int64_t numel() const {
    int64_t n = 1;
    for (int i = 0; i < t.ndim; ++i) n *= d[i].size;
    return n;
  }
  size_t bytes() const { return (size_t)numel() * (t.dtype == MTF_BF16 ? 2 : 4); }
};

// same memory, one dimension renamed (Section 6.1: a reshape that changes only a name)
TD renamed(const mtf_tensor& src, const char* from, const char* to) {
  TD r;
  for (int i = 0; i < src.ndim; ++i) {
    r.d[i] = src.dims[i];
    if (strcmp(src.dims[i].name, from) == 0) r.d[i].name = to;
  }
  r.t = src;
  r.t.dims = r.d;
  return r;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct Arena {
  uint8_t* base;
  size_t size, used;
  bool overflow;
  Arena(void* b, size_t s) : base(reinterpret_cast<uint8_t*>(b)), size(s), used(0), overflow(false) {}
  void* take(size_t bytes) {
    const size_t a = align256(bytes);
    if (!base || used + a > size) { overflow = true; used += a; return nullptr; }
    void* p = base + used;
    used += a;
    return p;
  }
};

bool same_shape(const mtf_tensor& a, const mtf_tensor& b) {
  if (a.ndim != b.ndim) return false;
  for (int i = 0; i < a.ndim; ++i)
    if (a.dims[i].size != b.dims[i].size || strcmp(a.dims[i].name, b.dims[i].name) != 0) return false;
  return true;
}

int64_t numel(const mtf_tensor& t) {
  int64_t n = 1;
  for (int i = 0; i < t.ndim; ++i) n *= t.dims[i].size;
  return n;
}

const char* kMemory = "memory_length";

struct AttShapes {
  mtf_dim b, l, d, h, k, v, m;
  double scale;
};

mtf_status attention_shapes(const mtf_tensor* x, const mtf_tensor* wq, const mtf_tensor* wk, const mtf_tensor* wv, const mtf_tensor* wo, AttShapes* s) {
  if (!x || !wq || !wk || !wv || !wo) return fail(MTF_ERR_INVALID_ARG, "attention: NULL tensor");
  if (x->ndim != 3 || wq->ndim != 3 || wk->ndim != 3 || wv->ndim != 3 || wo->ndim != 3)
    return fail(MTF_ERR_INVALID_ARG, "attention: x must be [batch, length, d_model], wq/wk [d_model, heads, d_k], wv [d_model, heads, d_v], wo [heads, d_v, d_model]");
  for (const mtf_tensor* t : {x, wq, wk, wv, wo})
    for (int i = 0; i < 3; ++i)
      if (!t->dims || !t->dims[i].name) return fail(MTF_ERR_INVALID_ARG, "attention: unnamed dimension");
  s->b = x->dims[0]; s->l = x->dims[1]; s->d = x->dims[2];
  s->h = wq->dims[1]; s->k = wq->dims[2]; s->v = wv->dims[2];
  s->m = s->l; s->m.name = kMemory;
  if (strcmp(s->l.name, kMemory) == 0) return fail(MTF_ERR_INVALID_ARG, "attention: the query length dimension may not be called '%s'", kMemory);
  auto is = [](const mtf_dim& a, const mtf_dim& b) { return strcmp(a.name, b.name) == 0 && a.size == b.size; };
  if (!is(wq->dims[0], s->d) || !is(wk->dims[0], s->d) || !is(wv->dims[0], s->d) || !is(wo->dims[2], s->d) || !is(wk->dims[1], s->h) ||
      !is(wv->dims[1], s->h) || !is(wo->dims[0], s->h) || !is(wk->dims[2], s->k) || !is(wo->dims[1], s->v))
    return fail(MTF_ERR_SIZE_MISMATCH, "attention: projection shapes do not fit x / each other");
  s->scale = 1.0 / std::sqrt((double)s->k.size);
  return MTF_OK;
}

mtf_epilogue epi_none() {
  mtf_epilogue e;
  e.scale = 1.f; e.relu = 0; e.bias = nullptr; e.relu_mask = nullptr; e.residual = nullptr; e.reduce_sum_out = nullptr;
  return e;
}

mtf_status ein(const mtf_layout_t* L, const mtf_tensor& a, const mtf_tensor& b, mtf_tensor* out, const mtf_epilogue* e, void* ws, size_t wsb, void* stream) {
  mtf_tensor in[2] = {a, b};
  return mtf_einsum(L, nullptr, 2, in, out, e, ws, wsb, stream);
}

size_t ein_ws(const mtf_layout_t* L, const mtf_tensor& a, const mtf_tensor& b, const mtf_tensor& out, mtf_status* st) {
  mtf_tensor in[2] = {a, b};
  size_t bytes = 0;
  mtf_status s = mtf_einsum_workspace_bytes(L, 2, in, &out, nullptr, &bytes);
  if (s != MTF_OK && *st == MTF_OK) *st = s;
  return bytes;
}

}  // namespace

extern "C" {

// ---- softmax over the last dimension -----------------------------------------------------------------
// weights = exp(logits - max) / sum exp(logits - max) along the last dimension; with `causal` the
// entries whose last index exceeds the second-to-last index are excluded (weight exactly 0).
mtf_status mtf_softmax_forward(const mtf_layout_t* layout, const mtf_tensor* logits, int32_t causal, mtf_tensor* weights, void* stream) {
  if (!layout || !logits || !weights || !logits->data || !weights->data) return fail(MTF_ERR_INVALID_ARG, "softmax: NULL argument");
  if (logits->ndim < 2 || !same_shape(*logits, *weights)) return fail(MTF_ERR_SIZE_MISMATCH, "softmax: logits and weights must have the same dims (at least two)");
  if (logits->dtype != MTF_F32 || weights->dtype != MTF_BF16) return fail(MTF_ERR_UNSUPPORTED, "softmax: logits must be f32 and weights bf16");
  mtf_status st = mtf_layout_check_tensor(layout, logits->ndim, logits->dims);
  if (st != MTF_OK) return st;
  const int n = (int)logits->dims[logits->ndim - 1].size, L = (int)logits->dims[logits->ndim - 2].size;
  if (causal && n != L) return fail(MTF_ERR_SIZE_MISMATCH, "softmax: a causal mask needs equal query and memory lengths");
  return mtf::launch_softmax_fwd(reinterpret_cast<const float*>(logits->data), weights->data, numel(*logits) / n, n, L, causal ? 1 : 0, stream);
}

// dlogits = weights * (dweights - sum_last(dweights * weights))
mtf_status mtf_softmax_backward(const mtf_layout_t* layout, const mtf_tensor* weights, const mtf_tensor* dweights, mtf_tensor* dlogits, void* stream) {
  if (!layout || !weights || !dweights || !dlogits || !weights->data || !dweights->data || !dlogits->data) return fail(MTF_ERR_INVALID_ARG, "softmax backward: NULL argument");
  if (weights->ndim < 1 || !same_shape(*weights, *dweights) || !same_shape(*weights, *dlogits)) return fail(MTF_ERR_SIZE_MISMATCH, "softmax backward: all three tensors must have the same dims");
  if (weights->dtype != MTF_BF16 || dweights->dtype != MTF_F32 || dlogits->dtype != MTF_BF16) return fail(MTF_ERR_UNSUPPORTED, "softmax backward: weights bf16, dweights f32, dlogits bf16");
  mtf_status st = mtf_layout_check_tensor(layout, weights->ndim, weights->dims);
  if (st != MTF_OK) return st;
  const int n = (int)weights->dims[weights->ndim - 1].size;
  return mtf::launch_softmax_bwd(weights->data, reinterpret_cast<const float*>(dweights->data), dlogits->data, numel(*weights) / n, n, stream);
}

// ---- layer normalisation over the last dimension ------------------------------------------------------
// mu = mean(x), var = mean((x - mu)^2), rstd = (var + eps)^-1/2, y = gamma * (x - mu) * rstd + beta;
// stats (f32, two values per row: mu, rstd) is kept for the backward pass.
mtf_status mtf_layernorm_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* gamma, const mtf_tensor* beta, float eps,
                                 mtf_tensor* y, mtf_tensor* stats, void* stream) {
  if (!layout || !x || !gamma || !beta || !y || !stats || !x->data || !gamma->data || !beta->data || !y->data || !stats->data)
    return fail(MTF_ERR_INVALID_ARG, "layernorm: NULL argument");
  if (x->ndim < 2 || !same_shape(*x, *y)) return fail(MTF_ERR_SIZE_MISMATCH, "layernorm: x and y must have the same dims (at least two)");
  const int n = (int)x->dims[x->ndim - 1].size;
  const int64_t rows = numel(*x) / n;
  if (gamma->ndim != 1 || beta->ndim != 1 || gamma->dims[0].size != n || beta->dims[0].size != n) return fail(MTF_ERR_SIZE_MISMATCH, "layernorm: gamma and beta must be [last dim of x]");
  if (x->dtype != MTF_BF16 || y->dtype != MTF_BF16 || gamma->dtype != MTF_F32 || beta->dtype != MTF_F32 || stats->dtype != MTF_F32)
    return fail(MTF_ERR_UNSUPPORTED, "layernorm: x, y bf16; gamma, beta, stats f32");
  if (numel(*stats) != 2 * rows) return fail(MTF_ERR_SIZE_MISMATCH, "layernorm: stats must hold two values per row");
  mtf_status st = mtf_layout_check_tensor(layout, x->ndim, x->dims);
  if (st != MTF_OK) return st;
  return mtf::launch_layernorm_fwd(x->data, reinterpret_cast<const float*>(gamma->data), reinterpret_cast<const float*>(beta->data), y->data,
                                   reinterpret_cast<float*>(stats->data), rows, n, eps, stream);
}

// g = dy * gamma; dx = rstd * (g - mean(g) - xh * mean(g * xh)) (+ residual); dgamma = sum_rows dy * xh; dbeta = sum_rows dy
mtf_status mtf_layernorm_workspace_bytes(int64_t row_length, size_t* bytes) {
  if (!bytes || row_length <= 0 || row_length > 0x7fffffff) return fail(MTF_ERR_INVALID_ARG, "layernorm_workspace_bytes: bad argument");
  *bytes = mtf::layernorm_bwd_scratch_bytes((int)row_length);
  return MTF_OK;
}

mtf_status mtf_layernorm_backward(const mtf_layout_t* layout, const mtf_tensor* dy, const mtf_tensor* x, const mtf_tensor* stats, const mtf_tensor* gamma,
                                  const mtf_tensor* residual, mtf_tensor* dx, mtf_tensor* dgamma, mtf_tensor* dbeta, void* workspace,
                                  size_t workspace_bytes, void* stream) {
  if (!layout || !dy || !x || !stats || !gamma || !dx || !dy->data || !x->data || !stats->data || !gamma->data || !dx->data) return fail(MTF_ERR_INVALID_ARG, "layernorm backward: NULL argument");
  if (x->ndim < 2 || !same_shape(*x, *dy) || !same_shape(*x, *dx) || (residual && !same_shape(*x, *residual))) return fail(MTF_ERR_SIZE_MISMATCH, "layernorm backward: dy, x, dx (and residual) must have the same dims");
  const int n = (int)x->dims[x->ndim - 1].size;
  const int64_t rows = numel(*x) / n;
  if (x->dtype != MTF_BF16 || dy->dtype != MTF_BF16 || dx->dtype != MTF_BF16 || gamma->dtype != MTF_F32 || stats->dtype != MTF_F32 || (residual && residual->dtype != MTF_BF16))
    return fail(MTF_ERR_UNSUPPORTED, "layernorm backward: activations bf16; gamma, stats f32");
  if ((dgamma == nullptr) != (dbeta == nullptr)) return fail(MTF_ERR_INVALID_ARG, "layernorm backward: give both dgamma and dbeta or neither");
  if (dgamma && (dgamma->dtype != MTF_F32 || dbeta->dtype != MTF_F32 || numel(*dgamma) != n || numel(*dbeta) != n || !dgamma->data || !dbeta->data))
    return fail(MTF_ERR_INVALID_ARG, "layernorm backward: dgamma and dbeta must be f32 [last dim of x]");
  if (residual && !residual->data) return fail(MTF_ERR_INVALID_ARG, "layernorm backward: residual has no data");
  mtf_status st = mtf_layout_check_tensor(layout, x->ndim, x->dims);
  if (st != MTF_OK) return st;
  st = mtf::launch_layernorm_bwd(dy->data, x->data, reinterpret_cast<const float*>(stats->data), reinterpret_cast<const float*>(gamma->data),
                                 residual ? residual->data : nullptr, dx->data, dgamma ? reinterpret_cast<float*>(dgamma->data) : nullptr,
                                 dbeta ? reinterpret_cast<float*>(dbeta->data) : nullptr, rows, n, workspace, workspace_bytes, stream);
  if (st != MTF_OK || !dgamma) return st;
  // the parameter gradients sum over the token dimensions: with one of them split across ranks they are partial sums
  std::vector<std::string> reduced;
  for (int i = 0; i + 1 < x->ndim; ++i) reduced.push_back(x->dims[i].name);
  if (mtf::rank_sum_needed(layout, reduced)) {
    if ((st = mtf::rank_allreduce_start(layout, dgamma->data, n, MTF_F32, stream)) != MTF_OK) return st;
    if ((st = mtf::rank_allreduce_start(layout, dbeta->data, n, MTF_F32, stream)) != MTF_OK) return st;
  }
  return MTF_OK;
}

// ---- multi-head attention -----------------------------------------------------------------------------
// q[b,l,h,k] = sum_d x wq; kk[b,m,h,k] = sum_d xm wk; vv[b,m,h,v] = sum_d xm wv (xm = x with `length`
// renamed memory_length); logits[b,h,l,m] = d_k^-1/2 sum_k q kk; weights = softmax_m (causal: m <= l);
// o[b,l,h,v] = sum_m weights vv; y[b,l,d] = sum_{h,v} o wo (+ residual).
mtf_status mtf_einsum_softmax(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, float scale, int32_t causal,
                              mtf_tensor* weights, void* workspace, size_t workspace_bytes, void* stream) {
  return mtf::einsum_row_softmax(layout, a, b, weights, scale, causal ? 1 : 0, workspace, workspace_bytes, stream);
}

mtf_status mtf_einsum_softmax_backward(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, const mtf_tensor* weights,
                                       mtf_tensor* dlogits, void* workspace, size_t workspace_bytes, void* stream) {
  return mtf::einsum_row_softmax_bwd(layout, a, b, weights, dlogits, 0, workspace, workspace_bytes, stream);
}

mtf_status mtf_attention_workspace_bytes(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* wq, const mtf_tensor* wv, size_t* bytes) {
  if (!layout || !x || !wq || !wv || !bytes || x->ndim != 3 || wq->ndim != 3 || wv->ndim != 3) return fail(MTF_ERR_INVALID_ARG, "attention_workspace_bytes: bad argument");
  const int64_t B = x->dims[0].size, L = x->dims[1].size, H = wq->dims[1].size, K = wq->dims[2].size, V = wv->dims[2].size;
  const size_t lg32 = align256((size_t)B * H * L * L * 4), lg16 = align256((size_t)B * H * L * L * 2);
  const size_t qk = align256((size_t)B * L * H * K * 2), vv = align256((size_t)B * L * H * V * 2);
  const size_t fwd = lg32;
  const size_t bwd = vv /*do*/ + lg32 /*dP*/ + lg16 /*dlogits*/ + 2 * qk /*dq, dkk*/ + vv /*dvv*/ + align256((size_t)numel(*x) * 4) /*dx in fp32*/;
  // room for a workspace-mode group sum of any of the projection-gradient einsums
  *bytes = std::max(fwd, bwd) + (64u << 20) + 256;
  return MTF_OK;
}

mtf_status mtf_attention_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* wq, const mtf_tensor* wk, const mtf_tensor* wv,
                                 const mtf_tensor* wo, int32_t causal, const mtf_tensor* residual, mtf_tensor* q, mtf_tensor* kk, mtf_tensor* vv,
                                 mtf_tensor* weights, mtf_tensor* o, mtf_tensor* y, void* workspace, size_t workspace_bytes, void* stream) {
  AttShapes s;
  mtf_status st = attention_shapes(x, wq, wk, wv, wo, &s);
  if (st != MTF_OK) return st;
  if (!layout || !q || !kk || !vv || !weights || !o || !y) return fail(MTF_ERR_INVALID_ARG, "attention_forward: NULL output");
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return fail(MTF_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  Arena ar(workspace, workspace_bytes);
  TD lg = TD::make(MTF_F32, {s.b, s.h, s.l, s.m});
  lg.t.data = ar.take(lg.bytes());
  if (ar.overflow) return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "attention_forward needs %zu workspace bytes, got %zu", ar.used, workspace_bytes);
  void* rest = ar.base + ar.used;
  const size_t rest_bytes = ar.size - ar.used;
  TD xm = renamed(*x, s.l.name, kMemory);
  {
    // the three projections are problems of one shape: one grouped launch where the plan allows it
    const mtf_tensor gin[3][2] = {{*x, *wq}, {xm.t, *wk}, {xm.t, *wv}};
    mtf_tensor* const gout[3] = {q, kk, vv};
    st = (s.k.size == s.v.size) ? mtf::einsum_group(layout, 3, gin, gout, rest, rest_bytes, stream) : MTF_ERR_UNSUPPORTED;
    if (st == MTF_ERR_UNSUPPORTED) {
      if ((st = ein(layout, *x, *wq, q, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
      if ((st = ein(layout, xm.t, *wk, kk, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
      st = ein(layout, xm.t, *wv, vv, nullptr, rest, rest_bytes, stream);
    }
    if (st != MTF_OK) return st;
  }
  // The whole core - logits, softmax, weights . v - in one launch when the shapes allow it (d_k = d_v = 64, rows of at most
  // 512 logits, only batch and heads split, tensors in the canonical dimension orders): every (batch, head) pair is an
  // independent problem on the processor that owns it, so the layout only decides who computes which pair.
  {
    auto unsplit = [&](const mtf_dim& d) { const int j = layout->mesh_dim_of(d.name); return j < 0 || layout->mesh[j].size == 1; };
    auto order = [](const mtf_tensor* t, std::initializer_list<mtf_dim> want) {
      if (t->ndim != (int)want.size() || t->dtype != MTF_BF16 || !t->data) return false;
      int i = 0;
      for (auto& w : want) { if (strcmp(t->dims[i].name, w.name) != 0 || t->dims[i].size != w.size) return false; ++i; }
      return true;
    };
    const bool canonical = order(q, {s.b, s.l, s.h, s.k}) && order(kk, {s.b, s.m, s.h, s.k}) && order(vv, {s.b, s.m, s.h, s.v}) &&
                           order(weights, {s.b, s.h, s.l, s.m}) && order(o, {s.b, s.l, s.h, s.v});
    // (legality and divisibility of the batch and heads splits were checked by the projections' plans above)
    if (canonical && mtf::attention_fused_supported(s.l.size, s.k.size, s.v.size) && unsplit(s.l) && unsplit(s.m) && unsplit(s.k) && unsplit(s.v)) {
      if ((st = mtf::launch_attention_fwd_fused(q->data, kk->data, vv->data, weights->data, o->data, s.b.size, s.h.size, s.l.size, (float)s.scale, causal ? 1 : 0,
                                                stream)) != MTF_OK)
        return st;
      mtf_epilogue er2 = epi_none();
      er2.residual = residual;
      if ((st = ein(layout, *o, *wo, y, residual ? &er2 : nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
      return mtf::rank_wait(layout, stream);
    }
  }
  mtf_epilogue es = epi_none();
  es.scale = (float)s.scale;
  // logits and softmax in one launch where a row of logits fits a tile (the fp32 logits then never
  // leave the tensor memory); otherwise the logits go through the workspace and the row kernel
  st = mtf::einsum_row_softmax(layout, q, kk, weights, (float)s.scale, causal, rest, rest_bytes, stream);
  if (st == MTF_ERR_UNSUPPORTED) {
    if ((st = ein(layout, *q, *kk, &lg.t, &es, rest, rest_bytes, stream)) != MTF_OK) return st;
    st = mtf_softmax_forward(layout, &lg.t, causal, weights, stream);
  }
  if (st != MTF_OK) return st;
  if ((st = ein(layout, *weights, *vv, o, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  mtf_epilogue er = epi_none();
  er.residual = residual;
  if ((st = ein(layout, *o, *wo, y, residual ? &er : nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  return mtf::rank_wait(layout, stream);        // heads split across ranks: y is summed over them before anyone reads it
}

// dwo = sum_{b,l} o dy; do = sum_d dy wo; dP = sum_v do vv; dvv = sum_l P do; dlogits = P (dP - sum_m dP P);
// dq = s sum_m dlogits kk; dkk = s sum_l dlogits q; dwq = sum_{b,l} x dq; dwk = sum_{b,m} xm dkk;
// dwv = sum_{b,m} xm dvv; dx = sum_{h,k} dq wq + sum_{h,k} dkk wk + sum_{h,v} dvv wv (+ dx_residual).
mtf_status mtf_attention_backward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* wq, const mtf_tensor* wk, const mtf_tensor* wv,
                                  const mtf_tensor* wo, int32_t causal, const mtf_tensor* q, const mtf_tensor* kk, const mtf_tensor* vv, const mtf_tensor* weights,
                                  const mtf_tensor* o, const mtf_tensor* dy, const mtf_tensor* dx_residual, mtf_tensor* dx, mtf_tensor* dwq,
                                  mtf_tensor* dwk, mtf_tensor* dwv, mtf_tensor* dwo, void* workspace, size_t workspace_bytes, void* stream) {
  AttShapes s;
  mtf_status st = attention_shapes(x, wq, wk, wv, wo, &s);
  if (st != MTF_OK) return st;
  if (!layout || !q || !kk || !vv || !weights || !o || !dy || !dx || !dwq || !dwk || !dwv || !dwo) return fail(MTF_ERR_INVALID_ARG, "attention_backward: NULL tensor");
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return fail(MTF_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  Arena ar(workspace, workspace_bytes);
  TD dob = TD::make(MTF_BF16, {s.b, s.l, s.h, s.v});
  TD dP = TD::make(MTF_F32, {s.b, s.h, s.l, s.m});
  TD dlg = TD::make(MTF_BF16, {s.b, s.h, s.l, s.m});
  TD dq = TD::make(MTF_BF16, {s.b, s.l, s.h, s.k});
  TD dkk = TD::make(MTF_BF16, {s.b, s.m, s.h, s.k});
  TD dvv = TD::make(MTF_BF16, {s.b, s.m, s.h, s.v});
  TD dx32 = TD::make(MTF_F32, {s.b, s.l, s.d});     // dx is accumulated in fp32 and rounded once
  for (TD* t : {&dob, &dP, &dlg, &dq, &dkk, &dvv, &dx32}) t->t.data = ar.take(t->bytes());
  if (ar.overflow) return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "attention_backward needs %zu workspace bytes, got %zu", ar.used, workspace_bytes);
  void* rest = ar.base + ar.used;
  const size_t rest_bytes = ar.size - ar.used;
  TD xm = renamed(*x, s.l.name, kMemory);
  // The whole core - dP, the softmax backward, dvv, dq, dkk - in one launch under the conditions of the forward core
  // (d_k = d_v = 64, rows of at most 512, only batch and heads split, canonical dimension orders): the weights are read
  // once and the gradient of the logits never leaves the chip.
  bool core_ok = false;
  {
    auto unsplit = [&](const mtf_dim& d) { const int j = layout->mesh_dim_of(d.name); return j < 0 || layout->mesh[j].size == 1; };
    auto order = [](const mtf_tensor* t, std::initializer_list<mtf_dim> want) {
      if (t->ndim != (int)want.size() || t->dtype != MTF_BF16 || !t->data) return false;
      int i = 0;
      for (auto& w : want) { if (strcmp(t->dims[i].name, w.name) != 0 || t->dims[i].size != w.size) return false; ++i; }
      return true;
    };
    const bool canonical = order(q, {s.b, s.l, s.h, s.k}) && order(kk, {s.b, s.m, s.h, s.k}) && order(vv, {s.b, s.m, s.h, s.v}) &&
                           order(weights, {s.b, s.h, s.l, s.m}) && order(o, {s.b, s.l, s.h, s.v});
    core_ok = canonical && mtf::attention_bwd_fused_supported(s.l.size, s.k.size, s.v.size) && unsplit(s.l) && unsplit(s.m) && unsplit(s.k) && unsplit(s.v);
  }
  // dWo reads o and dy and nothing the core touches.  Behind the one-launch core it is issued as an independent launch
  // with the group sum chained in its accumulators (no cleared counters in front of it), so its tiles start on the SMs
  // that the core's last round of (batch, head) pairs leaves idle; otherwise it goes first.
  const bool dwo_late = core_ok;
  if (!dwo_late && (st = ein(layout, *o, *dy, dwo, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = ein(layout, *dy, *wo, &dob.t, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = mtf::tap("do", dob.t, stream)) != MTF_OK) return st;
  bool core_done = false;
  {
    if (core_ok) {
      // (with the stage tap open the gradient of the logits is written out as well, as the contractions consume it)
      void* dump = mtf::tap_is_open() ? dlg.t.data : nullptr;
      if ((st = mtf::launch_attention_bwd_fused(q->data, kk->data, vv->data, weights->data, dob.t.data, dq.t.data, dkk.t.data, dvv.t.data, dump, s.b.size, s.h.size,
                                                s.l.size, (float)s.scale, causal ? 1 : 0 /* a hint: the zeros of a causal P give zero gradients anyway */, stream)) != MTF_OK)
        return st;
      if (dump && (st = mtf::tap("dlogits", dlg.t, stream)) != MTF_OK) return st;
      core_done = true;
      if (dwo_late) {
        const int was = mtf::swap_force_reduce(MTF_REDUCE_CHAINED);
        mtf::hint_next_launch_independent();
        st = ein(layout, *o, *dy, dwo, nullptr, rest, rest_bytes, stream);
        mtf::swap_force_reduce(was);
        if (st != MTF_OK) return st;
      }
    }
  }
  if (!core_done) {
  // dP and the softmax backward in one launch where a row fits a tile (dP then stays in tensor
  // memory); otherwise dP goes through the workspace in fp32 and the row kernel follows
  st = mtf::einsum_row_softmax_bwd(layout, &dob.t, vv, weights, &dlg.t, 0 /* zeros of a causal P give zeros here without being told */, rest, rest_bytes, stream);
  const bool fused_bwd = st == MTF_OK;
  if (st != MTF_OK && st != MTF_ERR_UNSUPPORTED) return st;
  if (!fused_bwd && (st = ein(layout, dob.t, *vv, &dP.t, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = ein(layout, *weights, dob.t, &dvv.t, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  if (!fused_bwd && (st = mtf_softmax_backward(layout, weights, &dP.t, &dlg.t, stream)) != MTF_OK) return st;
  if ((st = mtf::tap("dvv", dvv.t, stream)) != MTF_OK || (st = mtf::tap("dlogits", dlg.t, stream)) != MTF_OK) return st;
  mtf_epilogue es = epi_none();
  es.scale = (float)s.scale;
  if ((st = ein(layout, dlg.t, *kk, &dq.t, &es, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = ein(layout, dlg.t, *q, &dkk.t, &es, rest, rest_bytes, stream)) != MTF_OK) return st;
  } else if ((st = mtf::tap("dvv", dvv.t, stream)) != MTF_OK) {
    return st;
  }
  if ((st = mtf::tap("dq", dq.t, stream)) != MTF_OK || (st = mtf::tap("dkk", dkk.t, stream)) != MTF_OK) return st;
  {
    // the three weight gradients are problems of one shape (few output tiles each): one grouped launch
    const mtf_tensor gin[3][2] = {{*x, dq.t}, {xm.t, dkk.t}, {xm.t, dvv.t}};
    mtf_tensor* const gout[3] = {dwq, dwk, dwv};
    st = (s.k.size == s.v.size && dwq->dtype == dwk->dtype && dwq->dtype == dwv->dtype) ? mtf::einsum_group(layout, 3, gin, gout, rest, rest_bytes, stream)
                                                                                      : MTF_ERR_UNSUPPORTED;
    if (st == MTF_ERR_UNSUPPORTED) {
      if ((st = ein(layout, *x, dq.t, dwq, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
      if ((st = ein(layout, xm.t, dkk.t, dwk, nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
      st = ein(layout, xm.t, dvv.t, dwv, nullptr, rest, rest_bytes, stream);
    }
    if (st != MTF_OK) return st;
  }
  // the three contributions to dx are accumulated through the residual stage, in an fp32 buffer
  // (viewed with the memory_length name for the two that come from the key / value side); the
  // last einsum adds the running sum and writes dx once
  mtf_epilogue er = epi_none();
  er.residual = dx_residual;
  {
    // one launch where the plan allows it: the k loop runs through dq.wq, then dkk.wk, then dvv.wv
    // into one accumulator (same shapes; the key / value side carries the memory_length name)
    const mtf_tensor terms[3][2] = {{dq.t, *wq}, {dkk.t, *wk}, {dvv.t, *wv}};
    // (it reads what the weight-gradient launch before it only reads and writes dx: an independent launch, whose tiles
    //  start on the SMs that launch's few tiles leave idle)
    mtf::hint_next_launch_independent();
    st = mtf::einsum_terms(layout, 3, terms, dx, dx_residual ? &er : nullptr, rest, rest_bytes, stream);
    (void)mtf::take_independent_hint();
    if (st == MTF_OK) return mtf::rank_wait(layout, stream);
    if (st != MTF_ERR_UNSUPPORTED) return st;
  }
  if (layout->bound_dim >= 0 && layout->world > 1 && mtf::rank_sum_needed(layout, {s.h.name, s.k.name, s.v.name}))
    return fail(MTF_ERR_UNSUPPORTED, "attention_backward: with heads split across ranks dx needs the single three-term launch, which this plan cannot run");
  if ((st = ein(layout, dq.t, *wq, &dx32.t, dx_residual ? &er : nullptr, rest, rest_bytes, stream)) != MTF_OK) return st;
  TD dx32m = renamed(dx32.t, s.l.name, kMemory);
  mtf_epilogue ea = epi_none();
  ea.residual = &dx32m.t;
  if ((st = ein(layout, dkk.t, *wk, &dx32m.t, &ea, rest, rest_bytes, stream)) != MTF_OK) return st;
  TD dxm = renamed(*dx, s.l.name, kMemory);
  if ((st = ein(layout, dvv.t, *wv, &dxm.t, &ea, rest, rest_bytes, stream)) != MTF_OK) return st;
  return mtf::rank_wait(layout, stream);
}

// ---- decoder layer: a = LN1(x + Attention(x)); out = LN2(a + FFN(a)) ------------------------------------
mtf_status mtf_decoder_layer_workspace_bytes(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_decoder_params* p, size_t* bytes) {
  if (!layout || !x || !p || !bytes || !p->wq || !p->wv || !p->w) return fail(MTF_ERR_INVALID_ARG, "decoder_layer_workspace_bytes: bad argument");
  size_t att = 0, ffn = 0;
  mtf_status st = mtf_attention_workspace_bytes(layout, x, p->wq, p->wv, &att);
  if (st != MTF_OK) return st;
  if ((st = mtf_ffn_workspace_bytes(layout, x, p->w, &ffn)) != MTF_OK) return st;
  const size_t act = align256((size_t)numel(*x) * 2);
  *bytes = std::max(att, ffn) + 2 * act + 256;     // + the two gradient streams that cross the residual sums
  return MTF_OK;
}

mtf_status mtf_decoder_layer_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_decoder_params* p, int32_t causal, float eps,
                                     const mtf_decoder_saved* sv, mtf_tensor* out, void* workspace, size_t workspace_bytes, void* stream) {
  if (!layout || !x || !p || !sv || !out) return fail(MTF_ERR_INVALID_ARG, "decoder_layer_forward: NULL argument");
  for (const mtf_tensor* t : {p->wq, p->wk, p->wv, p->wo, p->ln1_gamma, p->ln1_beta, p->w, p->v, p->ln2_gamma, p->ln2_beta})
    if (!t) return fail(MTF_ERR_INVALID_ARG, "decoder_layer_forward: a parameter tensor is NULL");
  for (const mtf_tensor* t : {sv->q, sv->kk, sv->vv, sv->weights, sv->o, sv->s1, sv->stats1, sv->a, sv->h, sv->s2, sv->stats2})
    if (!t) return fail(MTF_ERR_INVALID_ARG, "decoder_layer_forward: a saved-activation tensor is NULL");
  mtf_status st;
  // s1 = x + Attention(x) (the residual rides in the output projection's epilogue); a = LN1(s1)
  if ((st = mtf_attention_forward(layout, x, p->wq, p->wk, p->wv, p->wo, causal, x, sv->q, sv->kk, sv->vv, sv->weights, sv->o, sv->s1, workspace, workspace_bytes, stream)) != MTF_OK) return st;
  if ((st = mtf_layernorm_forward(layout, sv->s1, p->ln1_gamma, p->ln1_beta, eps, sv->a, sv->stats1, stream)) != MTF_OK) return st;
  // s2 = a + FFN(a); out = LN2(s2)
  if ((st = mtf::ffn_forward_impl(layout, sv->a, p->w, p->bias, p->v, sv->h, sv->s2, sv->a, workspace, workspace_bytes, stream)) != MTF_OK) return st;
  if ((st = mtf::rank_wait(layout, stream)) != MTF_OK) return st;        // d_ff split across ranks: s2 is summed before the layer norm reads it
  return mtf_layernorm_forward(layout, sv->s2, p->ln2_gamma, p->ln2_beta, eps, out, sv->stats2, stream);
}

mtf_status mtf_decoder_layer_backward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_decoder_params* p, int32_t causal,
                                      const mtf_decoder_saved* sv, const mtf_tensor* dout, mtf_tensor* dx, const mtf_decoder_grads* g, void* workspace, size_t workspace_bytes,
                                      void* stream) {
  if (!layout || !x || !p || !sv || !dout || !dx || !g) return fail(MTF_ERR_INVALID_ARG, "decoder_layer_backward: NULL argument");
  for (const mtf_tensor* t : {g->dwq, g->dwk, g->dwv, g->dwo, g->dln1_gamma, g->dln1_beta, g->dw, g->dv, g->dln2_gamma, g->dln2_beta})
    if (!t) return fail(MTF_ERR_INVALID_ARG, "decoder_layer_backward: a gradient tensor is NULL");
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return fail(MTF_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  Arena ar(workspace, workspace_bytes);
  TD ds2, da;                                   // gradients on (a + FFN(a)) and on a
  ds2 = renamed(*x, "", "");
  da = renamed(*x, "", "");
  ds2.t.dtype = MTF_BF16; da.t.dtype = MTF_BF16;
  ds2.t.data = ar.take(ds2.bytes());
  da.t.data = ar.take(da.bytes());
  if (ar.overflow) return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "decoder_layer_backward needs more than %zu workspace bytes", workspace_bytes);
  void* rest = ar.base + ar.used;
  const size_t rest_bytes = ar.size - ar.used;
  mtf_status st;
  if ((st = mtf_layernorm_backward(layout, dout, sv->s2, sv->stats2, p->ln2_gamma, nullptr, &ds2.t, g->dln2_gamma, g->dln2_beta, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = mtf::tap("ds2", ds2.t, stream)) != MTF_OK) return st;
  // da = ds2 + dFFN/da
  if ((st = mtf::ffn_backward_impl(layout, sv->a, p->w, p->v, sv->h, &ds2.t, &da.t, &ds2.t, g->dw, g->dbias, g->dv, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = mtf::rank_wait(layout, stream)) != MTF_OK) return st;        // da (and the parameter gradients) summed across ranks
  if ((st = mtf::tap("da", da.t, stream)) != MTF_OK) return st;
  // ds1 (reusing ds2's buffer) = LN1 backward; dx = ds1 + dAttention/dx
  if ((st = mtf_layernorm_backward(layout, &da.t, sv->s1, sv->stats1, p->ln1_gamma, nullptr, &ds2.t, g->dln1_gamma, g->dln1_beta, rest, rest_bytes, stream)) != MTF_OK) return st;
  if ((st = mtf::tap("ds1", ds2.t, stream)) != MTF_OK) return st;
  return mtf_attention_backward(layout, x, p->wq, p->wk, p->wv, p->wo, causal, sv->q, sv->kk, sv->vv, sv->weights, sv->o, &ds2.t, &ds2.t, dx, g->dwq, g->dwk,
                                g->dwv, g->dwo, rest, rest_bytes, stream);
}

}  // extern "C"
