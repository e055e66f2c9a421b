// The `vocab` dimension of the Transformer layout (Section 9: vocab, d_ff and heads are the split
// dimensions): the memory-bound kernels around the logits einsum.
//
//   embedding_gather_kernel      x[t, :] = E[ids[t], :]             the einsum onehot(ids) . E that reduces
//                                                                   `vocab`: exactly one slice of a vocab-split
//                                                                   table contributes a non-zero row, and since
//                                                                   the table is stored once the group sum is a
//                                                                   row lookup
//   embedding_scatter_add_kernel dE[ids[t], :] += dx[t, :]          reduces the token dimensions (fp32 atomics)
//   xent_rows_kernel             per token: max, sum of exponentials and picked logit over the WHOLE row
//                                (Section 6 "Reduction": local reduction per vocab slice + the group combine,
//                                done here by one block that walks all slices of the row), lse and loss
//   xent_backward_kernel         dlogits = (exp(logits - lse) - onehot(target)) * dloss, in place
// Bound: HBM.  Rows are read in 16-byte pieces, coalesced.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "mtf_internal.h"

namespace {

__device__ __forceinline__ void bf16x8(const uint4& u, float* f) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    f[2 * e] = __uint_as_float(w[e] << 16);
    f[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
  }
}

__global__ void __launch_bounds__(256) embedding_gather_kernel(const int32_t* __restrict__ ids, const uint4* __restrict__ table, uint4* __restrict__ x,
                                                               long long n_tokens, int pieces, int vocab, int* __restrict__ bad) {
  const long long total = n_tokens * pieces;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / pieces;
    const int p = (int)(i - t * pieces);
    const int id = ids[t];
    if (id < 0 || id >= vocab) { if (p == 0) atomicExch(bad, 1); x[i] = make_uint4(0u, 0u, 0u, 0u); continue; }
    x[i] = table[(long long)id * pieces + p];
  }
}

// dtable (f32, zeroed by the launcher) += rows of dx (bf16 or f32) at ids
template <bool kBf16>
__global__ void __launch_bounds__(256) embedding_scatter_add_kernel(const int32_t* __restrict__ ids, const void* __restrict__ dx, float* __restrict__ dtable,
                                                                    long long n_tokens, int d, int vocab) {
  const long long total = n_tokens * d;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / d;
    const int c = (int)(i - t * d);
    const int id = ids[t];
    if (id < 0 || id >= vocab) continue;
    const float v = kBf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(dx)[i]) : reinterpret_cast<const float*>(dx)[i];
    atomicAdd(dtable + (long long)id * d + c, v);
  }
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One block per token row of bf16 logits (vocab a multiple of 8).  One pass over the row: every thread keeps a running
// maximum and the sum of exponentials relative to it (rescaled when the maximum moves); the threads' pairs are then
// combined - the local reduction of each part of the row followed by the combine of Section 6's "Reduction".
// The picked logit is read directly.
__device__ __forceinline__ void lse_combine(float& m, float& s, float m2, float s2) {
  const float mx = fmaxf(m, m2);
  s = (m == -INFINITY ? 0.f : s * __expf(m - mx)) + (m2 == -INFINITY ? 0.f : s2 * __expf(m2 - mx));
  m = mx;
}

__global__ void __launch_bounds__(256) xent_rows_kernel(const __nv_bfloat16* __restrict__ logits, const int32_t* __restrict__ targets, float* __restrict__ lse,
                                                        float* __restrict__ loss, int vocab, int* __restrict__ bad) {
  __shared__ float red_m[8], red_s[8];
  const long long row = blockIdx.x;
  const uint4* r = reinterpret_cast<const uint4*>(logits + row * vocab);
  const int pieces = vocab / 8;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float m = -INFINITY, s = 0.f;
  for (int p = threadIdx.x; p < pieces; p += 256) {
    float f[8];
    bf16x8(r[p], f);
    float pm = f[0];
#pragma unroll
    for (int e = 1; e < 8; ++e) pm = fmaxf(pm, f[e]);
    if (pm > m) { s *= __expf(m - pm); m = pm; }          // (m = -inf: s is 0 and stays 0)
#pragma unroll
    for (int e = 0; e < 8; ++e) s += __expf(f[e] - m);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    lse_combine(m, s, m2, s2);
  }
  if (lane == 0) { red_m[warp] = m; red_s[warp] = s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float mm = red_m[0], ss = red_s[0];
    for (int w = 1; w < 8; ++w) lse_combine(mm, ss, red_m[w], red_s[w]);
    const float l = mm + logf(ss);
    lse[row] = l;
    const int tg = targets[row];
    if (tg < 0 || tg >= vocab) { atomicExch(bad, 1); loss[row] = 0.f; }
    else loss[row] = l - __bfloat162float(logits[row * vocab + tg]);
  }
}

// The group combine of Section 6's "Reduction" for row statistics that the logits contraction left per column part
// (its epilogue took the local maximum and sum of exponentials of every part of every row while the tile was still
// on the chip): one warp per row combines the parts in a fixed order, then lse and loss as above.
__global__ void __launch_bounds__(256) xent_combine_kernel(const float2* __restrict__ partial, int parts, const __nv_bfloat16* __restrict__ logits,
                                                           const int32_t* __restrict__ targets, float* __restrict__ lse, float* __restrict__ loss,
                                                           long long n_rows, int vocab, int* __restrict__ bad) {
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const int lane = threadIdx.x & 31;
  float m = -INFINITY, s = 0.f;
  for (int p = lane; p < parts; p += 32) {
    const float2 ps = partial[row * parts + p];
    lse_combine(m, s, ps.x, ps.y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    lse_combine(m, s, m2, s2);
  }
  if (lane == 0) {
    const float l = m + logf(s);
    lse[row] = l;
    const int tg = targets[row];
    if (tg < 0 || tg >= vocab) { atomicExch(bad, 1); loss[row] = 0.f; }
    else loss[row] = l - __bfloat162float(logits[row * vocab + tg]);
  }
}

// dlogits[t, v] = (exp(logits[t, v] - lse[t]) - [v == target[t]]) * dloss[t], written over the logits
__global__ void __launch_bounds__(256) xent_backward_kernel(__nv_bfloat16* __restrict__ logits, const int32_t* __restrict__ targets, const float* __restrict__ lse,
                                                            const float* __restrict__ dloss, long long n_rows, int vocab) {
  const int pieces = vocab / 8;
  const long long total = n_rows * pieces;
  uint4* lg = reinterpret_cast<uint4*>(logits);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / pieces;
    const int c0 = (int)(i - t * pieces) * 8;
    const float l = lse[t], g = dloss[t];
    const int tg = targets[t] - c0;
    float f[8];
    bf16x8(lg[i], f);
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = (__expf(f[2 * e] - l) - (tg == 2 * e ? 1.f : 0.f)) * g;
      const float b = (__expf(f[2 * e + 1] - l) - (tg == 2 * e + 1 ? 1.f : 0.f)) * g;
      __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
      w[e] = *reinterpret_cast<uint32_t*>(&h);
    }
    lg[i] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

__device__ int g_bad_index = 0;

}  // namespace

namespace mtf {

static mtf_status after(const char* what) {
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  return MTF_OK;
}

static int* bad_flag() {
  int* p = nullptr;
  cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_bad_index);
  return p;
}

mtf_status launch_embedding_gather(const int32_t* ids, const void* table, void* x, int64_t n_tokens, int64_t d, int elem_bytes, int64_t vocab, void* stream) {
  if (n_tokens <= 0) return MTF_OK;
  if ((d * elem_bytes) % 16 || (reinterpret_cast<uintptr_t>(table) & 15) || (reinterpret_cast<uintptr_t>(x) & 15))
    return fail(MTF_ERR_UNSUPPORTED, "embedding: rows must be multiples of 16 bytes and 16-byte aligned");
  const int pieces = (int)(d * elem_bytes / 16);
  const long long blocks = std::min<long long>((n_tokens * pieces + 255) / 256, (long long)device_sm_count() * 16);
  embedding_gather_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(ids, reinterpret_cast<const uint4*>(table), reinterpret_cast<uint4*>(x), n_tokens, pieces, (int)vocab, bad_flag());
  return after("embedding_gather_kernel");
}

mtf_status launch_embedding_scatter_add(const int32_t* ids, const void* dx, int dx_bf16, float* dtable, int64_t n_tokens, int64_t d, int64_t vocab, void* stream) {
  cudaError_t e = cudaMemsetAsync(dtable, 0, (size_t)vocab * d * sizeof(float), (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
  if (n_tokens <= 0) return MTF_OK;
  const long long blocks = std::min<long long>((n_tokens * d + 255) / 256, (long long)device_sm_count() * 16);
  if (dx_bf16) embedding_scatter_add_kernel<true><<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(ids, dx, dtable, n_tokens, (int)d, (int)vocab);
  else embedding_scatter_add_kernel<false><<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(ids, dx, dtable, n_tokens, (int)d, (int)vocab);
  return after("embedding_scatter_add_kernel");
}

mtf_status launch_xent_rows(const void* logits, const int32_t* targets, float* lse, float* loss, int64_t n_rows, int64_t vocab, void* stream) {
  if (n_rows <= 0) return MTF_OK;
  if (vocab % 8 || (reinterpret_cast<uintptr_t>(logits) & 15)) return fail(MTF_ERR_UNSUPPORTED, "cross-entropy: vocab must be a multiple of 8 and the logits 16-byte aligned");
  if (n_rows > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "cross-entropy: too many rows");
  xent_rows_kernel<<<(unsigned)n_rows, 256, 0, (cudaStream_t)stream>>>(reinterpret_cast<const __nv_bfloat16*>(logits), targets, lse, loss, (int)vocab, bad_flag());
  return after("xent_rows_kernel");
}

mtf_status launch_xent_combine(const void* partial, int parts, const void* logits, const int32_t* targets, float* lse, float* loss, int64_t n_rows, int64_t vocab,
                               void* stream) {
  if (n_rows <= 0) return MTF_OK;
  if (parts <= 0 || n_rows > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "cross-entropy combine: bad sizes");
  xent_combine_kernel<<<(unsigned)((n_rows + 7) / 8), 256, 0, (cudaStream_t)stream>>>(reinterpret_cast<const float2*>(partial), parts,
                                                                                   reinterpret_cast<const __nv_bfloat16*>(logits), targets, lse, loss, n_rows, (int)vocab,
                                                                                   bad_flag());
  return after("xent_combine_kernel");
}

mtf_status launch_xent_backward(void* logits, const int32_t* targets, const float* lse, const float* dloss, int64_t n_rows, int64_t vocab, void* stream) {
  if (n_rows <= 0) return MTF_OK;
  const long long blocks = std::min<long long>((n_rows * (vocab / 8) + 255) / 256, (long long)device_sm_count() * 16);
  xent_backward_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(reinterpret_cast<__nv_bfloat16*>(logits), targets, lse, dloss, n_rows, (int)vocab);
  return after("xent_backward_kernel");
}

// 1 when a token id or a target outside [0, vocab) was seen since the last call (synchronises the device); resets the flag
mtf_status read_bad_index(int* seen) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaDeviceSynchronize: %s", cudaGetErrorString(e));
  int v = 0;
  e = cudaMemcpyFromSymbol(&v, g_bad_index, sizeof(int));
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemcpyFromSymbol: %s", cudaGetErrorString(e));
  if (v) { int z = 0; cudaMemcpyToSymbol(g_bad_index, &z, sizeof(int)); }
  *seen = v;
  return MTF_OK;
}

}  // namespace mtf
