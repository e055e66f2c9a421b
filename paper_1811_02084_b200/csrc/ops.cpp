// Entry points beside the einsum and the blocks: the parameter update of Algorithm 1 line 3, the
// reshape / transposing copies of Section 6.1, and the vocab-dimension operations of the Section 9
// layout (embedding, logits + cross-entropy).  Validation and composition only; the arithmetic runs in
// update.cu, relayout.cu, vocab.cu and, for the contractions, through mtf_einsum.
#include <algorithm>
#include <cstring>

#include "mtf_internal.h"

namespace mtf {
mtf_status launch_sgd_update(float* master, void* param, const void* grad, int grad_bf16, float* mom, int64_t n, float lr, float mu, float wd, void* stream);
mtf_status launch_xent_combine(const void* partial, int parts, const void* logits, const int32_t* targets, float* lse, float* loss, int64_t n_rows, int64_t vocab,
                               void* stream);
mtf_status launch_permute_copy(const void* src, void* dst, int elem_bytes, int ndim, const int64_t* sizes, const int64_t* sstr, const int64_t* dstr, void* stream);
mtf_status launch_embedding_gather(const int32_t* ids, const void* table, void* x, int64_t n_tokens, int64_t d, int elem_bytes, int64_t vocab, void* stream);
mtf_status launch_embedding_scatter_add(const int32_t* ids, const void* dx, int dx_bf16, float* dtable, int64_t n_tokens, int64_t d, int64_t vocab, void* stream);
mtf_status launch_xent_rows(const void* logits, const int32_t* targets, float* lse, float* loss, int64_t n_rows, int64_t vocab, void* stream);
mtf_status launch_xent_backward(void* logits, const int32_t* targets, const float* lse, const float* dloss, int64_t n_rows, int64_t vocab, void* stream);
}  // namespace mtf

using mtf::Dim;
using mtf::fail;

namespace {

int64_t numel(const mtf_tensor& t) {
  int64_t n = 1;
  for (int i = 0; i < t.ndim; ++i) n *= t.dims[i].size;
  return n;
}

bool same_dims(const mtf_tensor& a, const mtf_tensor& b) {
  if (a.ndim != b.ndim) return false;
  for (int i = 0; i < a.ndim; ++i)
    if (!a.dims[i].name || !b.dims[i].name || strcmp(a.dims[i].name, b.dims[i].name) != 0 || a.dims[i].size != b.dims[i].size) return false;
  return true;
}

mtf_status legal(const mtf_layout_t* L, const mtf_tensor& t, const char* what) {
  std::vector<Dim> d;
  mtf_status st = mtf::read_dims(t.ndim, t.dims, &d, what);
  if (st != MTF_OK) return st;
  return mtf::check_tensor(L, d);
}

}  // namespace

extern "C" {

// ---- Algorithm 1 line 3 -------------------------------------------------------------------------------------
mtf_status mtf_update(const mtf_layout_t* layout, const mtf_tensor* grad, mtf_tensor* master, mtf_tensor* momentum, mtf_tensor* param,
                      const mtf_update_params* hp, void* stream) {
  if (!layout || !grad || !master || !hp || !grad->data || !master->data) return fail(MTF_ERR_INVALID_ARG, "update: NULL argument");
  mtf_status st = legal(layout, *master, "update: master");
  if (st != MTF_OK) return st;
  if (master->dtype != MTF_F32) return fail(MTF_ERR_UNSUPPORTED, "update: the master copy must be f32");
  if (!same_dims(*grad, *master) || (momentum && !same_dims(*momentum, *master)) || (param && !same_dims(*param, *master)))
    return fail(MTF_ERR_SIZE_MISMATCH, "update: gradient, momentum and working copy must have the master copy's dims");
  if (grad->dtype != MTF_F32 && grad->dtype != MTF_BF16) return fail(MTF_ERR_INVALID_ARG, "update: unknown gradient dtype");
  if (momentum && (momentum->dtype != MTF_F32 || !momentum->data)) return fail(MTF_ERR_INVALID_ARG, "update: momentum must be an f32 tensor with data");
  if (param && (param->dtype != MTF_BF16 || !param->data)) return fail(MTF_ERR_INVALID_ARG, "update: the working copy must be a bf16 tensor with data");
  for (const mtf_tensor* t : {(const mtf_tensor*)master, grad, (const mtf_tensor*)momentum, (const mtf_tensor*)param})
    if (t && (reinterpret_cast<uintptr_t>(t->data) & 15)) return fail(MTF_ERR_INVALID_ARG, "update: tensors must be 16-byte aligned");
  if (hp->momentum != 0.f && !momentum) return fail(MTF_ERR_INVALID_ARG, "update: momentum %g needs a momentum tensor", (double)hp->momentum);
  return mtf::launch_sgd_update(reinterpret_cast<float*>(master->data), param ? param->data : nullptr, grad->data, grad->dtype == MTF_BF16,
                                momentum ? reinterpret_cast<float*>(momentum->data) : nullptr, numel(*master), hp->lr, hp->momentum, hp->weight_decay, stream);
}

// ---- Section 6.1: reshape that changes names (host: what the lowering would communicate) ----------------------
mtf_status mtf_reshape_plan(const mtf_layout_t* layout, int32_t ndim, const mtf_dim* in_dims, const char* const* out_names, int32_t* pattern,
                            int64_t* received_per_proc) {
  if (!layout || !out_names || !pattern || !received_per_proc) return fail(MTF_ERR_INVALID_ARG, "reshape_plan: NULL argument");
  std::vector<Dim> din, dout;
  mtf_status st = mtf::read_dims(ndim, in_dims, &din, "reshape input");
  if (st != MTF_OK) return st;
  std::vector<mtf_dim> od(ndim);
  for (int i = 0; i < ndim; ++i) { od[i].name = out_names[i]; od[i].size = in_dims[i].size; }
  if ((st = mtf::read_dims(ndim, od.data(), &dout, "reshape output")) != MTF_OK) return st;
  if ((st = mtf::check_tensor(layout, din)) != MTF_OK || (st = mtf::check_tensor(layout, dout)) != MTF_OK) return st;
  const int R = (int)layout->mesh.size();
  int64_t local = 1;                                   // elements of one processor's input slice
  for (auto& d : din) {
    const int j = layout->mesh_dim_of(d.name);
    local *= j >= 0 ? d.size / layout->mesh[j].size : d.size;
  }
  // the gathers of all changed mesh dimensions run first (ascending mesh dimension), each multiplying the local extent
  for (int j = 0; j < R; ++j) {
    int pin = -1, pout = -1;
    for (int i = 0; i < ndim; ++i) {
      if (layout->mesh_dim_of(din[i].name) == j) pin = i;
      if (layout->mesh_dim_of(dout[i].name) == j) pout = i;
    }
    const int64_t m = layout->mesh[j].size;
    pattern[j] = MTF_RESHAPE_NONE;
    received_per_proc[j] = 0;
    if (pin == pout) continue;
    if (pin >= 0 && pout < 0) { pattern[j] = MTF_RESHAPE_ALLGATHER; received_per_proc[j] = local * (m - 1); local *= m; }
    else if (pin < 0) { pattern[j] = MTF_RESHAPE_SLICE; }
    else { pattern[j] = MTF_RESHAPE_ALLTOALL; received_per_proc[j] = local * (m - 1) / m; local *= m; }
  }
  return MTF_OK;
}

// out = in with its dimensions in another storage order (out's names are a permutation of in's)
mtf_status mtf_transpose(const mtf_layout_t* layout, const mtf_tensor* in, mtf_tensor* out, void* stream) {
  if (!layout || !in || !out || !in->data || !out->data) return fail(MTF_ERR_INVALID_ARG, "transpose: NULL argument");
  if (in->dtype != out->dtype || in->ndim != out->ndim) return fail(MTF_ERR_INVALID_ARG, "transpose: input and output must agree in type and number of dims");
  mtf_status st = legal(layout, *in, "transpose input");
  if (st != MTF_OK || (st = legal(layout, *out, "transpose output")) != MTF_OK) return st;
  int64_t istr[mtf::kMaxTensorDims], ostr[mtf::kMaxTensorDims], sizes[mtf::kMaxTensorDims], sstr[mtf::kMaxTensorDims];
  int64_t s = 1;
  for (int i = in->ndim - 1; i >= 0; --i) { istr[i] = s; s *= in->dims[i].size; }
  s = 1;
  for (int i = out->ndim - 1; i >= 0; --i) { ostr[i] = s; s *= out->dims[i].size; }
  for (int i = 0; i < out->ndim; ++i) {
    int src = -1;
    for (int k = 0; k < in->ndim; ++k)
      if (strcmp(in->dims[k].name, out->dims[i].name) == 0) src = k;
    if (src < 0) return fail(MTF_ERR_UNKNOWN_DIM, "transpose: output dimension '%s' is not an input dimension", out->dims[i].name);
    if (in->dims[src].size != out->dims[i].size) return fail(MTF_ERR_SIZE_MISMATCH, "transpose: dimension '%s' changes size", out->dims[i].name);
    sizes[i] = out->dims[i].size;
    sstr[i] = istr[src];
  }
  return mtf::launch_permute_copy(in->data, out->data, in->dtype == MTF_BF16 ? 2 : 4, out->ndim, sizes, sstr, ostr, stream);
}

// one processor's dense slice written back into its box of the global tensor (the inverse of mtf_slice_gather)
mtf_status mtf_slice_scatter(const mtf_layout_t* layout, const void* slice, int64_t processor, mtf_tensor* global, void* stream) {
  if (!layout || !slice || !global || !global->data) return fail(MTF_ERR_INVALID_ARG, "slice_scatter: NULL argument");
  std::vector<Dim> d;
  mtf_status st = mtf::read_dims(global->ndim, global->dims, &d, "tensor");
  if (st != MTF_OK) return st;
  int64_t offs[mtf::kMaxTensorDims], sizes[mtf::kMaxTensorDims], sstr[mtf::kMaxTensorDims];
  if ((st = mtf::slice_box(layout, d, processor, offs, sizes)) != MTF_OK) return st;
  auto gs = mtf::row_major_strides(d);
  int64_t s = 1, base = 0;
  for (int i = global->ndim - 1; i >= 0; --i) { sstr[i] = s; s *= sizes[i]; base += offs[i] * gs[i]; }
  const int eb = global->dtype == MTF_BF16 ? 2 : 4;
  return mtf::launch_permute_copy(slice, reinterpret_cast<uint8_t*>(global->data) + base * eb, eb, global->ndim, sizes, sstr, gs.data(), stream);
}

// ---- vocab (Section 9) -----------------------------------------------------------------------------------------
static mtf_status vocab_not_across_ranks(const mtf_layout_t* L, const char* vocab_name, const char* what) {
  if (L->bound_dim >= 0 && L->world > 1 && L->mesh_dim_of(vocab_name) == L->bound_dim)
    return fail(MTF_ERR_UNSUPPORTED, "%s: the vocab dimension is split across ranks; the row statistics / the lookup would need a combine across ranks, which is not built", what);
  return MTF_OK;
}

mtf_status mtf_embedding_forward(const mtf_layout_t* layout, const int32_t* ids, const mtf_tensor* table, mtf_tensor* x, void* stream) {
  if (!layout || !ids || !table || !x || !table->data || !x->data) return fail(MTF_ERR_INVALID_ARG, "embedding_forward: NULL argument");
  if (table->ndim != 2 || x->ndim < 2 || table->dtype != x->dtype) return fail(MTF_ERR_INVALID_ARG, "embedding_forward: table [vocab, d], x [*tokens, d] of the same type");
  if (strcmp(table->dims[1].name, x->dims[x->ndim - 1].name) != 0 || table->dims[1].size != x->dims[x->ndim - 1].size)
    return fail(MTF_ERR_SIZE_MISMATCH, "embedding_forward: the table's second dim must be x's last dim");
  mtf_status st = legal(layout, *table, "embedding table");
  if (st != MTF_OK || (st = legal(layout, *x, "embedding output")) != MTF_OK) return st;
  if ((st = vocab_not_across_ranks(layout, table->dims[0].name, "embedding_forward")) != MTF_OK) return st;
  const int64_t d = table->dims[1].size;
  return mtf::launch_embedding_gather(ids, table->data, x->data, numel(*x) / d, d, x->dtype == MTF_BF16 ? 2 : 4, table->dims[0].size, stream);
}

mtf_status mtf_embedding_backward(const mtf_layout_t* layout, const int32_t* ids, const mtf_tensor* dx, mtf_tensor* dtable, void* stream) {
  if (!layout || !ids || !dx || !dtable || !dx->data || !dtable->data) return fail(MTF_ERR_INVALID_ARG, "embedding_backward: NULL argument");
  if (dtable->ndim != 2 || dx->ndim < 2 || dtable->dtype != MTF_F32) return fail(MTF_ERR_INVALID_ARG, "embedding_backward: dtable f32 [vocab, d], dx [*tokens, d]");
  if (strcmp(dtable->dims[1].name, dx->dims[dx->ndim - 1].name) != 0 || dtable->dims[1].size != dx->dims[dx->ndim - 1].size)
    return fail(MTF_ERR_SIZE_MISMATCH, "embedding_backward: dtable's second dim must be dx's last dim");
  mtf_status st = legal(layout, *dtable, "embedding table gradient");
  if (st != MTF_OK || (st = legal(layout, *dx, "embedding output gradient")) != MTF_OK) return st;
  const int64_t d = dtable->dims[1].size;
  st = mtf::launch_embedding_scatter_add(ids, dx->data, dx->dtype == MTF_BF16, reinterpret_cast<float*>(dtable->data), numel(*dx) / d, d, dtable->dims[0].size, stream);
  if (st != MTF_OK) return st;
  // the sum runs over the token dimensions: with one of them split across ranks every rank holds a partial table gradient
  std::vector<std::string> reduced;
  for (int i = 0; i + 1 < dx->ndim; ++i) reduced.push_back(dx->dims[i].name);
  if (mtf::rank_sum_needed(layout, reduced)) {
    if ((st = mtf::rank_allreduce_start(layout, dtable->data, numel(*dtable), MTF_F32, stream)) != MTF_OK) return st;
    return mtf::rank_wait(layout, stream);
  }
  return MTF_OK;
}

// the row part alone, on stored logits: lse and loss per token
mtf_status mtf_softmax_xent_forward(const mtf_layout_t* layout, const mtf_tensor* logits, const int32_t* targets, mtf_tensor* lse, mtf_tensor* loss, void* stream) {
  if (!layout || !logits || !targets || !lse || !loss || !logits->data || !lse->data || !loss->data) return fail(MTF_ERR_INVALID_ARG, "softmax_xent_forward: NULL argument");
  if (logits->ndim < 2 || logits->dtype != MTF_BF16 || lse->dtype != MTF_F32 || loss->dtype != MTF_F32) return fail(MTF_ERR_UNSUPPORTED, "softmax_xent_forward: logits bf16 [*tokens, vocab]; lse and loss f32");
  const int64_t V = logits->dims[logits->ndim - 1].size, rows = numel(*logits) / V;
  if (numel(*lse) != rows || numel(*loss) != rows) return fail(MTF_ERR_SIZE_MISMATCH, "softmax_xent_forward: lse and loss hold one value per token");
  mtf_status st = legal(layout, *logits, "logits");
  if (st != MTF_OK || (st = vocab_not_across_ranks(layout, logits->dims[logits->ndim - 1].name, "softmax_xent_forward")) != MTF_OK) return st;
  return mtf::launch_xent_rows(logits->data, targets, reinterpret_cast<float*>(lse->data), reinterpret_cast<float*>(loss->data), rows, V, stream);
}

// dlogits = (exp(logits - lse) - onehot(target)) * dloss, written over the logits
mtf_status mtf_softmax_xent_backward(const mtf_layout_t* layout, mtf_tensor* logits, const int32_t* targets, const mtf_tensor* lse, const mtf_tensor* dloss, void* stream) {
  if (!layout || !logits || !targets || !lse || !dloss || !logits->data || !lse->data || !dloss->data) return fail(MTF_ERR_INVALID_ARG, "softmax_xent_backward: NULL argument");
  if (logits->ndim < 2 || logits->dtype != MTF_BF16 || lse->dtype != MTF_F32 || dloss->dtype != MTF_F32) return fail(MTF_ERR_UNSUPPORTED, "softmax_xent_backward: logits bf16 [*tokens, vocab]; lse and dloss f32");
  const int64_t V = logits->dims[logits->ndim - 1].size, rows = numel(*logits) / V;
  if (numel(*lse) != rows || numel(*dloss) != rows) return fail(MTF_ERR_SIZE_MISMATCH, "softmax_xent_backward: lse and dloss hold one value per token");
  if (V % 8 || (reinterpret_cast<uintptr_t>(logits->data) & 15)) return fail(MTF_ERR_UNSUPPORTED, "cross-entropy: vocab must be a multiple of 8 and the logits 16-byte aligned");
  mtf_status st = legal(layout, *logits, "logits");
  if (st != MTF_OK || (st = vocab_not_across_ranks(layout, logits->dims[logits->ndim - 1].name, "softmax_xent_backward")) != MTF_OK) return st;
  return mtf::launch_xent_backward(logits->data, targets, reinterpret_cast<const float*>(lse->data), reinterpret_cast<const float*>(dloss->data), rows, V, stream);
}

mtf_status mtf_xent_forward(const mtf_layout_t* layout, const mtf_tensor* h, const mtf_tensor* wout, const int32_t* targets, mtf_tensor* logits,
                            mtf_tensor* lse, mtf_tensor* loss, void* workspace, size_t workspace_bytes, void* stream) {
  if (!layout || !h || !wout || !targets || !logits || !lse || !loss || !logits->data || !lse->data || !loss->data) return fail(MTF_ERR_INVALID_ARG, "xent_forward: NULL argument");
  if (wout->ndim != 2 || h->ndim < 2 || logits->ndim != h->ndim) return fail(MTF_ERR_INVALID_ARG, "xent_forward: h [*tokens, d], wout [d, vocab], logits [*tokens, vocab]");
  if (logits->dtype != MTF_BF16 || lse->dtype != MTF_F32 || loss->dtype != MTF_F32) return fail(MTF_ERR_UNSUPPORTED, "xent_forward: logits bf16; lse and loss f32");
  const int64_t V = wout->dims[1].size, rows = numel(*logits) / V;
  if (numel(*lse) != rows || numel(*loss) != rows) return fail(MTF_ERR_SIZE_MISMATCH, "xent_forward: lse and loss hold one value per token");
  mtf_status st = vocab_not_across_ranks(layout, wout->dims[1].name, "xent_forward");
  if (st != MTF_OK) return st;
  const mtf_tensor in[2] = {*h, *wout};
  // With room in the workspace the logits contraction takes the local maximum and sum of exponentials of every column
  // part of every row in its epilogue (Section 6 "Reduction": the local reduction), and a small launch combines the
  // parts (the group combine): the logits are not read back for the log-sum-exp.
  if (workspace && !(reinterpret_cast<uintptr_t>(workspace) & 255)) {
    int parts = 0;
    st = mtf::einsum_row_lse(layout, h, wout, logits, workspace, workspace_bytes, stream, &parts);
    if (st == MTF_OK)
      return mtf::launch_xent_combine(workspace, parts, logits->data, targets, reinterpret_cast<float*>(lse->data), reinterpret_cast<float*>(loss->data), rows, V, stream);
    if (st != MTF_ERR_UNSUPPORTED && st != MTF_ERR_WORKSPACE_TOO_SMALL) return st;
  }
  if ((st = mtf_einsum(layout, nullptr, 2, in, logits, nullptr, workspace, workspace_bytes, stream)) != MTF_OK) return st;
  return mtf_softmax_xent_forward(layout, logits, targets, lse, loss, stream);
}

mtf_status mtf_xent_backward(const mtf_layout_t* layout, const mtf_tensor* h, const mtf_tensor* wout, const int32_t* targets, mtf_tensor* logits,
                             const mtf_tensor* lse, const mtf_tensor* dloss, mtf_tensor* dh, mtf_tensor* dwout, void* workspace, size_t workspace_bytes,
                             void* stream) {
  if (!layout || !h || !wout || !targets || !logits || !lse || !dloss || !dh || !dwout || !logits->data || !lse->data || !dloss->data)
    return fail(MTF_ERR_INVALID_ARG, "xent_backward: NULL argument");
  if (wout->ndim != 2 || logits->dtype != MTF_BF16 || lse->dtype != MTF_F32 || dloss->dtype != MTF_F32) return fail(MTF_ERR_UNSUPPORTED, "xent_backward: logits bf16; lse and dloss f32");
  const int64_t V = wout->dims[1].size, rows = numel(*logits) / V;
  if (numel(*lse) != rows || numel(*dloss) != rows) return fail(MTF_ERR_SIZE_MISMATCH, "xent_backward: lse and dloss hold one value per token");
  mtf_status st = vocab_not_across_ranks(layout, wout->dims[1].name, "xent_backward");
  if (st != MTF_OK) return st;
  // dlogits = (softmax - onehot) * dloss, written over the logits; then the two contractions that read it
  if ((st = mtf_softmax_xent_backward(layout, logits, targets, lse, dloss, stream)) != MTF_OK) return st;
  if ((st = mtf::tap("dlogits", *logits, stream)) != MTF_OK) return st;
  const mtf_tensor in1[2] = {*logits, *wout};
  if ((st = mtf_einsum(layout, nullptr, 2, in1, dh, nullptr, workspace, workspace_bytes, stream)) != MTF_OK) return st;
  const mtf_tensor in2[2] = {*h, *logits};
  if ((st = mtf_einsum(layout, nullptr, 2, in2, dwout, nullptr, workspace, workspace_bytes, stream)) != MTF_OK) return st;
  return mtf::rank_wait(layout, stream);
}

}  // extern "C"
