// Algorithm 1, line 3: W(t+1) = Update(W(t), gradient), as one fused memory-bound pass per parameter.
// The paper leaves Update open; the reading taken here is stochastic gradient descent with optional
// momentum and decoupled weight decay on an fp32 master copy, which also refreshes the bf16 working
// copy the contractions read:
//     m <- momentum * m + g   (no momentum buffer: m = g);   W <- W - lr * (m + weight_decay * W);   Wb <- bf16(W)
// The update is component-wise (Section 6), so it is local under every layout: every virtual
// processor updates its own slice, and since a tensor is stored once on the GPU the union of those
// slices is one pass over the whole tensor (replicas are logical).  Bound: HBM.  Bytes per element:
// read g (4 or 2) + W (4) [+ m (4)], write W (4) [+ m (4)] [+ Wb (2)].
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "mtf_internal.h"

namespace {

template <bool kMom, bool kGradBf16, bool kParam>
__global__ void __launch_bounds__(256) sgd_update_kernel(float* __restrict__ master, __nv_bfloat16* __restrict__ param, const void* __restrict__ grad,
                                                         float* __restrict__ mom, long long n, float lr, float mu, float wd) {
  const long long n4 = n / 4;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    float4 w = reinterpret_cast<const float4*>(master)[i];
    float g[4];
    if (kGradBf16) {
      const uint2 u = reinterpret_cast<const uint2*>(grad)[i];
      g[0] = __uint_as_float(u.x << 16); g[1] = __uint_as_float(u.x & 0xFFFF0000u);
      g[2] = __uint_as_float(u.y << 16); g[3] = __uint_as_float(u.y & 0xFFFF0000u);
    } else {
      const float4 v = reinterpret_cast<const float4*>(grad)[i];
      g[0] = v.x; g[1] = v.y; g[2] = v.z; g[3] = v.w;
    }
    float m[4] = {g[0], g[1], g[2], g[3]};
    if (kMom) {
      const float4 mo = reinterpret_cast<const float4*>(mom)[i];
      m[0] = fmaf(mu, mo.x, g[0]); m[1] = fmaf(mu, mo.y, g[1]); m[2] = fmaf(mu, mo.z, g[2]); m[3] = fmaf(mu, mo.w, g[3]);
      reinterpret_cast<float4*>(mom)[i] = make_float4(m[0], m[1], m[2], m[3]);
    }
    w.x = fmaf(-lr, fmaf(wd, w.x, m[0]), w.x);
    w.y = fmaf(-lr, fmaf(wd, w.y, m[1]), w.y);
    w.z = fmaf(-lr, fmaf(wd, w.z, m[2]), w.z);
    w.w = fmaf(-lr, fmaf(wd, w.w, m[3]), w.w);
    reinterpret_cast<float4*>(master)[i] = w;
    if (kParam) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
      reinterpret_cast<uint2*>(param)[i] = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    }
  }
  // ragged tail (fewer than four elements): one thread each
  const long long t = n4 * 4 + (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) {
    const float g = kGradBf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(grad)[t]) : reinterpret_cast<const float*>(grad)[t];
    float m = g;
    if (kMom) { m = fmaf(mu, mom[t], g); mom[t] = m; }
    const float w = fmaf(-lr, fmaf(wd, master[t], m), master[t]);
    master[t] = w;
    if (kParam) param[t] = __float2bfloat16_rn(w);
  }
}

}  // namespace

namespace mtf {

mtf_status launch_sgd_update(float* master, void* param, const void* grad, int grad_bf16, float* mom, int64_t n, float lr, float mu, float wd, void* stream) {
  if (n <= 0) return MTF_OK;
  const long long blocks = std::min<long long>((n / 4 + 255) / 256 + 1, (long long)device_sm_count() * 8);
  cudaStream_t st = (cudaStream_t)stream;
  __nv_bfloat16* pb = reinterpret_cast<__nv_bfloat16*>(param);
#define MTF_UPD(M, G, P) sgd_update_kernel<M, G, P><<<(unsigned)blocks, 256, 0, st>>>(master, pb, grad, mom, n, lr, mu, wd)
  if (mom) {
    if (grad_bf16) { if (param) MTF_UPD(true, true, true); else MTF_UPD(true, true, false); }
    else { if (param) MTF_UPD(true, false, true); else MTF_UPD(true, false, false); }
  } else {
    if (grad_bf16) { if (param) MTF_UPD(false, true, true); else MTF_UPD(false, true, false); }
    else { if (param) MTF_UPD(false, false, true); else MTF_UPD(false, false, false); }
  }
#undef MTF_UPD
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "sgd_update_kernel: %s", cudaGetErrorString(e));
  return MTF_OK;
}

}  // namespace mtf
