// Generic strided named-dimension einsum kernel (any dimension structure, f32 / bf16 operands) and
// the slice-gather kernel.  One thread owns one global output element.  The reduction runs as the
// paper's lowering does (Section 6): for every member of the element's reduce group, in ascending
// processor order, a local partial sum over that processor's block of the reduced dimensions; the
// partials are then added in that order (the Allreduce, realised on the device).  Component-wise
// work (Section 6, Section 7 broadcasting) is applied to the sum before the store.
//
// This family is the fp32 path and the fallback for shapes the tensor-core family does not take;
// it is plain FFMA code and makes no attempt at tiling.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>

#include <string>
#include <vector>

#include "mtf_internal.h"

namespace {

__device__ __forceinline__ float ld_as_float(const void* p, int dt, int64_t off) {
  if (dt == MTF_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[off]);
  return reinterpret_cast<const float*>(p)[off];
}

__global__ void __launch_bounds__(256) einsum_simt_kernel(const SimtParams p) {
  const int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= p.total_out) return;
  int64_t offA = 0, offB = 0, offC = 0, offBias = 0, offRsum = 0, rem = o;
  for (int d = p.n_out - 1; d >= 0; --d) {
    const int64_t i = rem % p.out_size[d];
    rem /= p.out_size[d];
    offA += i * p.out_sA[d];
    offB += i * p.out_sB[d];
    offC += i * p.out_sC[d];
    offBias += i * p.out_sBias[d];
    offRsum += i * p.out_sRsum[d];
  }
  int64_t n_group = 1, n_local = 1;
  for (int l = 0; l < p.n_group; ++l) n_group *= p.lvl_extent[l];
  for (int l = p.n_group; l < p.n_levels; ++l) n_local *= p.lvl_extent[l];

  float total = 0.f;
  for (int64_t g = 0; g < n_group; ++g) {          // members of the reduce group, ascending processor order
    int64_t gA = offA, gB = offB, gr = g;
    for (int l = p.n_group - 1; l >= 0; --l) {
      const int64_t i = gr % p.lvl_extent[l];
      gr /= p.lvl_extent[l];
      gA += i * p.lvl_sA[l];
      gB += i * p.lvl_sB[l];
    }
    float partial = 0.f;                           // this processor's local einsum
    int64_t idx[mtf::kMaxIterDims];
    for (int l = 0; l < p.n_levels - p.n_group; ++l) idx[l] = 0;
    int64_t a = gA, b = gB;
    for (int64_t r = 0; r < n_local; ++r) {
      const float va = ld_as_float(p.A, p.dtA, a);
      const float vb = p.has_B ? ld_as_float(p.B, p.dtB, b) : 1.f;
      partial = fmaf(va, vb, partial);
      for (int l = p.n_levels - 1; l >= p.n_group; --l) {   // odometer over the local reduced extents
        const int k = l - p.n_group;
        a += p.lvl_sA[l];
        b += p.lvl_sB[l];
        if (++idx[k] < p.lvl_extent[l]) break;
        a -= idx[k] * p.lvl_sA[l];
        b -= idx[k] * p.lvl_sB[l];
        idx[k] = 0;
      }
    }
    total += partial;                              // the group sum
  }
  float t = total * p.scale;
  if (p.bias) t += ld_as_float(p.bias, p.dtBias, offBias);
  if (p.relu) t = fmaxf(t, 0.f);
  if (p.mask && !(ld_as_float(p.mask, p.dtMask, offC) > 0.f)) t = 0.f;
  if (p.rsum) atomicAdd(p.rsum + offRsum, t);      // fused reduction output (Section 6 "Reduction")
  if (p.resid) t += ld_as_float(p.resid, p.dtRes, offC);
  if (p.dtC == MTF_BF16) reinterpret_cast<__nv_bfloat16*>(p.C)[offC] = __float2bfloat16_rn(t);
  else reinterpret_cast<float*>(p.C)[offC] = t;
}

struct GatherParams {
  int ndim;
  int64_t sizes[mtf::kMaxTensorDims], offs[mtf::kMaxTensorDims], gstr[mtf::kMaxTensorDims];
  int64_t total;
  int elem_bytes;
};

__global__ void __launch_bounds__(256) slice_gather_kernel(const void* __restrict__ src, void* __restrict__ dst, const GatherParams g) {
  const int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= g.total) return;
  int64_t rem = o, off = 0;
  for (int d = g.ndim - 1; d >= 0; --d) {
    const int64_t i = rem % g.sizes[d];
    rem /= g.sizes[d];
    off += (g.offs[d] + i) * g.gstr[d];
  }
  if (g.elem_bytes == 2) reinterpret_cast<uint16_t*>(dst)[o] = reinterpret_cast<const uint16_t*>(src)[off];
  else reinterpret_cast<uint32_t*>(dst)[o] = reinterpret_cast<const uint32_t*>(src)[off];
}

std::atomic<int64_t> g_launches{0};

}  // namespace

namespace mtf {

void count_launch(int n) { g_launches.fetch_add(n); }
int64_t launch_count() { return g_launches.load(); }

static mtf_status check_launch(const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  return MTF_OK;
}

mtf_status launch_simt(const SimtParams& p, int64_t rsum_elems, void* stream) {
  if (p.total_out <= 0) return MTF_OK;
  if (p.rsum) {
    cudaError_t e = cudaMemsetAsync(p.rsum, 0, (size_t)rsum_elems * sizeof(float), (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
  }
  const int64_t blocks = (p.total_out + 255) / 256;
  if (blocks > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "output too large for the generic kernel's grid");
  einsum_simt_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(p);
  count_launch();
  return check_launch("einsum_simt_kernel");
}

mtf_status launch_slice_gather(const void* src, void* dst, int elem_bytes, int ndim, const int64_t* sizes,
                               const int64_t* offs, const int64_t* gstrides, void* stream) {
  GatherParams g;
  g.ndim = ndim;
  g.total = 1;
  g.elem_bytes = elem_bytes;
  for (int i = 0; i < ndim; ++i) {
    g.sizes[i] = sizes[i];
    g.offs[i] = offs[i];
    g.gstr[i] = gstrides[i];
    g.total *= sizes[i];
  }
  if (g.total <= 0) return MTF_OK;
  const int64_t blocks = (g.total + 255) / 256;
  if (blocks > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "slice too large for the gather kernel's grid");
  slice_gather_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(src, dst, g);
  count_launch();
  return check_launch("slice_gather_kernel");
}

// ---- stage tap: copies of scratch-resident intermediates for verification -----------------------------
namespace {
struct TapEntry { std::string name; size_t offset, bytes; };
struct TapState {
  uint8_t* base = nullptr;
  size_t size = 0, used = 0;
  bool active = false, overflow = false;
  std::vector<TapEntry> entries;
};
thread_local TapState g_tap;
}  // namespace

bool tap_is_open() { return g_tap.active; }

mtf_status tap_begin(void* device_buffer, size_t bytes) {
  if (!device_buffer || (reinterpret_cast<uintptr_t>(device_buffer) & 255)) return fail(MTF_ERR_INVALID_ARG, "stage tap: the buffer must be a 256-byte aligned device pointer");
  g_tap.base = reinterpret_cast<uint8_t*>(device_buffer);
  g_tap.size = bytes; g_tap.used = 0; g_tap.active = true; g_tap.overflow = false;
  g_tap.entries.clear();
  return MTF_OK;
}

mtf_status tap_end(int32_t* n_entries) {
  g_tap.active = false;
  if (n_entries) *n_entries = (int32_t)g_tap.entries.size();
  if (g_tap.overflow) return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "stage tap: the buffer of %zu bytes was too small (needed %zu)", g_tap.size, g_tap.used);
  return MTF_OK;
}

mtf_status tap_entry(int32_t i, const char** name, size_t* offset, size_t* bytes) {
  if (i < 0 || i >= (int32_t)g_tap.entries.size()) return fail(MTF_ERR_INVALID_ARG, "stage tap: entry %d of %d", i, (int)g_tap.entries.size());
  if (name) *name = g_tap.entries[i].name.c_str();
  if (offset) *offset = g_tap.entries[i].offset;
  if (bytes) *bytes = g_tap.entries[i].bytes;
  return MTF_OK;
}

// Called by the block compositions right after the launch that produced `t`; does nothing unless a tap is open.
mtf_status tap(const char* name, const mtf_tensor& t, void* stream) {
  if (!g_tap.active || !t.data) return MTF_OK;
  size_t n = t.dtype == MTF_BF16 ? 2 : 4;
  for (int i = 0; i < t.ndim; ++i) n *= (size_t)t.dims[i].size;
  const size_t off = g_tap.used;
  g_tap.used += (n + 255) / 256 * 256;
  if (g_tap.used > g_tap.size) { g_tap.overflow = true; return MTF_OK; }
  cudaError_t e = cudaMemcpyAsync(g_tap.base + off, t.data, n, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "stage tap copy: %s", cudaGetErrorString(e));
  g_tap.entries.push_back({name, off, n});
  return MTF_OK;
}

}  // namespace mtf
