// Internal declarations shared by the host planner, the kernels' launchers and the C ABI.
// Nothing here is visible to users of include/mtf.h.
#pragma once

#include <cstdint>
#include <map>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/mtf.h"

namespace mtf {

constexpr int kMaxMeshDims = 4;
constexpr int kMaxTensorDims = 8;
constexpr int kMaxIterDims = 12;
constexpr int kMaxOuter = 3;     // batch-like dims the tensor-core kernel keeps as separate coordinates

struct Dim {
  std::string name;
  int64_t size;
};

void set_error(const char* fmt, ...);
mtf_status fail(mtf_status s, const char* fmt, ...);

// ---- dims helpers --------------------------------------------------------------------------------
mtf_status read_dims(int32_t ndim, const mtf_dim* dims, std::vector<Dim>* out, const char* what);
std::vector<int64_t> row_major_strides(const std::vector<Dim>& dims);

}  // namespace mtf

struct mtf_mesh_s {
  std::vector<mtf::Dim> dims;
  int64_t P = 1;
};

// One dimension of an einsum's iteration space (the union of all operand dimensions).
struct IterDim {
  std::string name;
  int64_t size = 0;
  int mesh_dim = -1;     // mesh dimension this tensor dimension is split over, -1 = not split
  int64_t nsplit = 1;    // size of that mesh dimension (1 when not split)
  int64_t sA = 0, sB = 0, sC = 0;   // element strides in in[0], in[1], out (0 = operand lacks it)
  bool inA = false, inB = false, inC = false;
};

// ---- parameters of the generic strided kernel (any dtype mix, any dimension structure) ------------
struct SimtParams {
  int n_out = 0;                       // output dims, in the output's storage order
  int64_t out_size[mtf::kMaxTensorDims];
  int64_t out_sA[mtf::kMaxTensorDims], out_sB[mtf::kMaxTensorDims], out_sC[mtf::kMaxTensorDims];
  int64_t out_sBias[mtf::kMaxTensorDims];
  int64_t out_sRsum[mtf::kMaxTensorDims];
  // reduction loop nest: first n_group levels walk the members of the reduce group in ascending
  // processor order (one level per split reduced dim, lower mesh-dim index outermost); the rest walk
  // the local extents of the reduced dims.  A partial sum is closed after each group member.
  int n_levels = 0, n_group = 0;
  int64_t lvl_extent[mtf::kMaxIterDims + mtf::kMaxMeshDims];
  int64_t lvl_sA[mtf::kMaxIterDims + mtf::kMaxMeshDims], lvl_sB[mtf::kMaxIterDims + mtf::kMaxMeshDims];
  int64_t total_out = 0;
  int dtA = 0, dtB = 0, dtC = 0, dtBias = 0, dtMask = 0, dtRes = 0;
  int has_B = 1;
  float scale = 1.f;
  int relu = 0;
  const void* A = nullptr;
  const void* B = nullptr;
  void* C = nullptr;
  const void* bias = nullptr;
  const void* mask = nullptr;
  const void* resid = nullptr;
  float* rsum = nullptr;                // fused reduce_sum output (fp32, pre-zeroed)
};

// ---- parameters of the tcgen05 grouped GEMM ---------------------------------------------------------
// Canonical form: C[o0,o1,o2][m][n] = sum_k A[o..][m][k] * B[o..][k][n], each of M, N, K one merged
// strided dimension, up to three outer (batch) dimensions.  Every extent may be split into equal
// contiguous blocks (the virtual processors' slices).
struct TcParams {
  int64_t M = 1, N = 1, K = 1;
  int64_t sm = 1, sn = 1, sk = 1;            // number of slices along M, N, K
  int n_outer = 0;
  int64_t outer_size[mtf::kMaxOuter] = {1, 1, 1};
  int64_t outer_split[mtf::kMaxOuter] = {1, 1, 1};
  int64_t outer_sC[mtf::kMaxOuter] = {0, 0, 0};
  int64_t outer_sA[mtf::kMaxOuter] = {0, 0, 0}, outer_sB[mtf::kMaxOuter] = {0, 0, 0};
  int a_mn_major = 0, b_mn_major = 0;        // 0: K contiguous in smem rows, 1: M/N contiguous
  int64_t a_ld = 0, b_ld = 0;                // element stride of the non-contiguous one of (M|N, K)
  int64_t ldc = 0;                           // element stride of M in C (N is contiguous)
  int block_n = 256;
  int wide_pref = -1;                        // 256 x 512 pair tiles: -1 = launcher's wave heuristic, 0 = never, 1 = wherever the shape allows
  int balance = 0;                           // tiles leave a partly filled last wave: balanced k-range schedule (needs workspace)
  int cta_pair = 0;                          // two CTAs (a cluster) own a 256-row tile, tcgen05 cta_group::2
  int swapped = 0;                           // in[0] and in[1] exchanged so that N is contiguous in C
  int reduce_mode = MTF_REDUCE_NONE;
  int bias_along_m = 0;                      // bias varies with m (after a swap) instead of n
};

struct EpilogueDesc {
  bool on = false;
  float scale = 1.f;
  bool relu = false;
  bool has_bias = false, has_mask = false, has_res = false, has_rsum = false;
  std::vector<mtf::Dim> bias_dims, rsum_dims;
  int dtBias = 0, dtMask = 0, dtRes = 0;
};

struct mtf_plan_s {
  // problem
  std::vector<mtf::Dim> mesh;
  std::vector<mtf::Dim> dimsA, dimsB, dimsC;
  int dtA = 0, dtB = 0, dtC = 0;
  bool has_B = true;
  std::vector<IterDim> iter;
  EpilogueDesc epi;
  // decisions
  int kernel_kind = MTF_KERNEL_SIMT;
  int reduce_mode = MTF_REDUCE_NONE;
  int64_t n_slices = 1, group_size = 1;
  uint32_t reduce_mask = 0;
  size_t workspace_bytes = 0;
  // one mesh dimension mapped onto ranks (mtf_layout_bind_ranks): the on-device result is a partial sum
  // that the ranks still have to add up when a reduced-out dimension is split over that mesh dimension
  bool rank_sum = false;          // ... of the einsum's output
  bool rsum_rank_sum = false;     // ... of the fused reduce_sum output
  int rank = 0;
  mtf_rank_allreduce_fn ar_start = nullptr;
  void* ar_user = nullptr;
  // cost counts
  int64_t macs_per_proc = 0, allreduce_values = 0, slice_elems = 0;
  int n_reduce_mesh_dims = 0;
  // kernel parameters (pointers filled in at exec time)
  SimtParams simt;
  TcParams tc;
  std::string key;
};

struct mtf_layout_s {
  std::vector<mtf::Dim> mesh;
  std::vector<std::pair<std::string, int>> rules;   // tensor-dim name -> mesh-dim index
  // rank binding: mesh dimension `bound_dim` (of global size bound_global) is spread over `world` ranks;
  // this handle describes rank `rank`'s part, its mesh carries bound_global / world processors there
  int bound_dim = -1;
  int world = 1, rank = 0;
  int64_t bound_global = 0;
  mtf_rank_allreduce_fn ar_start = nullptr;
  mtf_rank_wait_fn ar_wait = nullptr;
  void* ar_user = nullptr;
  std::mutex mu;
  std::map<std::string, std::unique_ptr<mtf_plan_t>> cache;
  int mesh_dim_of(const std::string& tdim) const {
    for (auto& r : rules)
      if (r.first == tdim) return r.second;
    return -1;
  }
};

namespace mtf {

// host planner
mtf_status check_tensor(const mtf_layout_t* L, const std::vector<Dim>& dims);
mtf_status slice_box(const mtf_layout_t* L, const std::vector<Dim>& dims, int64_t p, int64_t* offs, int64_t* sizes);
mtf_status make_plan(const mtf_layout_t* L, int n_in, const mtf_tensor* in, const mtf_tensor* out,
                     const mtf_epilogue* epi, int force_kernel, int force_reduce, std::unique_ptr<mtf_plan_t>* plan);
std::string plan_key(int n_in, const mtf_tensor* in, const mtf_tensor* out, const mtf_epilogue* epi, int fk, int fr);

// rank binding (ranks.cpp): does summing out `reduced` (dimension names) leave a sum across ranks to do?
bool rank_sum_needed(const mtf_layout_t* L, const std::vector<std::string>& reduced);
// start the sum across ranks of `count` values at `data` behind what is queued on `stream`; no-op without hooks
mtf_status rank_allreduce_start(const mtf_layout_t* L, void* data, int64_t count, mtf_dtype dtype, void* stream);
// make `stream` wait for every sum across ranks started so far; no-op without hooks
mtf_status rank_wait(const mtf_layout_t* L, void* stream);

// launchers (defined in the .cu files)
mtf_status launch_simt(const SimtParams& p, int64_t rsum_elems, void* stream);
mtf_status launch_tc(const mtf_plan_t& plan, const void* A, const void* B, void* C, const void* bias, int dtBias,
                     const void* mask, int dtMask, const void* resid, int dtRes, float scale, int relu, float* rsum,
                     void* workspace, size_t workspace_bytes, void* stream, int n_terms = 1,
                     const void* const* extra_operands = nullptr,    // A_1, B_1 (, A_2, B_2) of a multi-term launch
                     int row_softmax = 0,                            // 1 / 2 (causal): softmax over each row of scale * (A . B) in the epilogue;
                                                                     // 3 / 4 (causal): its backward, P (A . B - rowsum(P A . B)), P = the mask operand
                     int n_groups = 1,                               // grouped launch: up to 3 independent problems of this plan's shape
                     const void* const* group_operands = nullptr);   // A_1, B_1, C_1 (, A_2, B_2, C_2)
// Hint for the next tensor-core launch of this thread: it neither reads nor writes anything the launch
// before it on the same stream touches (set by the block compositions, consumed by the launch).
void hint_next_launch_independent();
// Sets the reduce mode that plans made on this thread are forced to (-1: the planner's choice); returns the old one.
int swap_force_reduce(int mode);
bool take_independent_hint();
// n_groups (1..3) independent einsums with the dims of group 0 (names may differ, sizes and types may
// not) in one launch, so that contractions with few output tiles fill the GPU together.
// MTF_ERR_UNSUPPORTED when the plan cannot (generic kernel): the caller then runs them one by one.
mtf_status einsum_group(const mtf_layout_t* layout, int n_groups, const mtf_tensor (*ins)[2], mtf_tensor* const* outs,
                        void* workspace, size_t workspace_bytes, void* stream);
// Sum of n_terms (1..3) products of operand pairs with the dims of terms[0] (names may differ, sizes
// and types may not) in one launch, one accumulator.  MTF_ERR_UNSUPPORTED when this plan cannot
// (generic kernel, workspace reduce mode): the caller then chains einsums through the residual stage.
mtf_status einsum_terms(const mtf_layout_t* layout, int n_terms, const mtf_tensor (*terms)[2], mtf_tensor* out,
                        const mtf_epilogue* epilogue, void* workspace, size_t workspace_bytes, void* stream);
// weights[.., l, m] = softmax_m(scale * sum_k a b (causal: only m <= l)) in one launch, bf16 result.
// MTF_ERR_UNSUPPORTED when the plan cannot (rows longer than a tile, generic kernel, split rows).
// dlogits[.., l, m] = P (dP - sum_m dP P) with dP = sum_v a b, in one launch (same conditions, whole 32 x 64 boxes only).
mtf_status einsum_row_softmax_bwd(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, const mtf_tensor* weights,
                                  mtf_tensor* dlogits, int causal, void* workspace, size_t workspace_bytes, void* stream);
// a . b (plain, bf16) whose epilogue also leaves float2 [rows][*parts] row statistics (maximum, sum of exponentials of
// the stored values per column part) at the head of the workspace
mtf_status einsum_row_lse(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, mtf_tensor* out, void* workspace, size_t workspace_bytes,
                          void* stream, int* parts);
mtf_status einsum_row_softmax(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, mtf_tensor* weights, float scale,
                              int causal, void* workspace, size_t workspace_bytes, void* stream);
// Sum of n_terms (1..3) products of operand pairs with the dims of terms[0] (names may differ, sizes
// and types may not) in one launch, one accumulator.  MTF_ERR_UNSUPPORTED when this plan cannot
// (generic kernel, workspace reduce mode): the caller then chains einsums through the residual stage.
mtf_status einsum_terms(const mtf_layout_t* layout, int n_terms, const mtf_tensor (*terms)[2], mtf_tensor* out,
                        const mtf_epilogue* epilogue, void* workspace, size_t workspace_bytes, void* stream);
size_t tc_workspace_bytes(const TcParams& t);
size_t tc_rsum_partial_bytes(const TcParams& t);
// out0[c] (and out1[c] when planes = 2) = sum over g = 0 .. groups-1, in that order, of partial[g][plane][c]
mtf_status launch_colsum_finalize(const float* partial, int groups, int planes, int n, float* out0, float* out1, void* stream);
size_t builtin_scratch_capacity();
// SM count of the current device; 148 (a B200) when no device can be asked, so that planning works without one.
int device_sm_count();
// Device address of the library's own scratch array on the current device (resolved once per device).
mtf_status builtin_scratch_ptr(void** out);
mtf_status launch_slice_gather(const void* src, void* dst, int elem_bytes, int ndim, const int64_t* sizes,
                               const int64_t* offs, const int64_t* gstrides, void* stream);
void count_launch(int n = 1);
// stage tap (mtf_stage_tap_*): while a tap is open on this thread, `tap` copies the named intermediate
// into the caller's buffer on the stream, right behind the launch that produced it
mtf_status tap_begin(void* device_buffer, size_t bytes);
mtf_status tap_end(int32_t* n_entries);
mtf_status tap_entry(int32_t i, const char** name, size_t* offset, size_t* bytes);
mtf_status tap(const char* name, const mtf_tensor& t, void* stream);

}  // namespace mtf
