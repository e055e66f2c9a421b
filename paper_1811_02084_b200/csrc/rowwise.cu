// Memory-bound row kernels of the attention block and the decoder layer: softmax over the last
// dimension (forward and backward) and layer normalisation over the last dimension (forward,
// backward, and the column sums for the gain / offset gradients).
//
// In the paper's terms these are the "Reduction" lowering of Section 6 (reduce_max / reduce_sum over
// memory_length, reduce_sum over d_model) with component-wise work around it.  A row is handled by
// one warp and never leaves the GPU, so the group sum over a split reduced dimension is the warp's
// own shuffle reduction over the whole row.  The column sums (reduce out the token dims, i.e. the
// gradient Allreduce of Algorithm 1 under a batch split) accumulate per block and finish with fp32
// atomics.  All loads and stores are 16-byte vectors, coalesced along the row.
#include <algorithm>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "mtf_internal.h"

namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ void bf16x8_to_float(const uint4& u, float* f) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    f[2 * e] = __uint_as_float(w[e] << 16);
    f[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint4 float_to_bf16x8(const float* f) {
  uint32_t w[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
    w[e] = *reinterpret_cast<uint32_t*>(&h);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// weights[row, :] = softmax(logits[row, :]) with columns > (row % L) masked when causal.
// logits fp32, weights bf16, n a multiple of 8.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
softmax_fwd_kernel(const float* __restrict__ logits, __nv_bfloat16* __restrict__ weights, int64_t rows, int n, int L, int causal) {
  const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const float* x = logits + row * n;
  const int limit = causal ? (int)(row % L) + 1 : n;     // columns [0, limit) take part
  float mx = -INFINITY;
  for (int c = lane * 4; c < limit; c += 128) {
    const float4 v = *reinterpret_cast<const float4*>(x + c);
    mx = fmaxf(mx, v.x);
    if (c + 1 < limit) mx = fmaxf(mx, v.y);
    if (c + 2 < limit) mx = fmaxf(mx, v.z);
    if (c + 3 < limit) mx = fmaxf(mx, v.w);
  }
  mx = warp_max(mx);
  float sum = 0.f;
  for (int c = lane * 4; c < limit; c += 128) {
    const float4 v = *reinterpret_cast<const float4*>(x + c);
    sum += __expf(v.x - mx);
    if (c + 1 < limit) sum += __expf(v.y - mx);
    if (c + 2 < limit) sum += __expf(v.z - mx);
    if (c + 3 < limit) sum += __expf(v.w - mx);
  }
  sum = warp_sum(sum);
  const float inv = 1.f / sum;
  __nv_bfloat16* w = weights + row * n;
  for (int c = lane * 8; c < n; c += 256) {
    float f[8];
    const float4 a = *reinterpret_cast<const float4*>(x + c);
    const float4 b = *reinterpret_cast<const float4*>(x + c + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = (c + e < limit) ? __expf(v[e] - mx) * inv : 0.f;
    *reinterpret_cast<uint4*>(w + c) = float_to_bf16x8(f);
  }
}

// dlogits[row, :] = P * (dP - sum_j dP_j P_j);  P bf16, dP fp32, dlogits bf16.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
softmax_bwd_kernel(const __nv_bfloat16* __restrict__ P, const float* __restrict__ dP, __nv_bfloat16* __restrict__ dlg, int64_t rows, int n) {
  const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const __nv_bfloat16* p = P + row * n;
  const float* d = dP + row * n;
  float dot = 0.f;
  for (int c = lane * 8; c < n; c += 256) {
    float pf[8];
    bf16x8_to_float(*reinterpret_cast<const uint4*>(p + c), pf);
    const float4 a = *reinterpret_cast<const float4*>(d + c);
    const float4 b = *reinterpret_cast<const float4*>(d + c + 4);
    dot += pf[0] * a.x + pf[1] * a.y + pf[2] * a.z + pf[3] * a.w + pf[4] * b.x + pf[5] * b.y + pf[6] * b.z + pf[7] * b.w;
  }
  dot = warp_sum(dot);
  __nv_bfloat16* o = dlg + row * n;
  for (int c = lane * 8; c < n; c += 256) {
    float pf[8], f[8];
    bf16x8_to_float(*reinterpret_cast<const uint4*>(p + c), pf);
    const float4 a = *reinterpret_cast<const float4*>(d + c);
    const float4 b = *reinterpret_cast<const float4*>(d + c + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = pf[e] * (v[e] - dot);
    *reinterpret_cast<uint4*>(o + c) = float_to_bf16x8(f);
  }
}

// y = gamma * (x - mu) * rstd + beta over the last dim (biased variance, eps inside the root);
// stats[row] = (mu, rstd).  x, y bf16; gamma, beta fp32; n a multiple of 8.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
layernorm_fwd_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                     __nv_bfloat16* __restrict__ y, float* __restrict__ stats, int64_t rows, int n, float eps) {
  const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const __nv_bfloat16* xr = x + row * n;
  float s = 0.f;
  for (int c = lane * 8; c < n; c += 256) {
    float f[8];
    bf16x8_to_float(*reinterpret_cast<const uint4*>(xr + c), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) s += f[e];
  }
  const float mu = warp_sum(s) / (float)n;
  float q = 0.f;
  for (int c = lane * 8; c < n; c += 256) {
    float f[8];
    bf16x8_to_float(*reinterpret_cast<const uint4*>(xr + c), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) q += (f[e] - mu) * (f[e] - mu);
  }
  const float rstd = rsqrtf(warp_sum(q) / (float)n + eps);
  if (lane == 0) { stats[2 * row] = mu; stats[2 * row + 1] = rstd; }
  __nv_bfloat16* yr = y + row * n;
  for (int c = lane * 8; c < n; c += 256) {
    float f[8], o[8];
    bf16x8_to_float(*reinterpret_cast<const uint4*>(xr + c), f);
    const float4 g0 = *reinterpret_cast<const float4*>(gamma + c), g1 = *reinterpret_cast<const float4*>(gamma + c + 4);
    const float4 b0 = *reinterpret_cast<const float4*>(beta + c), b1 = *reinterpret_cast<const float4*>(beta + c + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) o[e] = g[e] * (f[e] - mu) * rstd + b[e];
    *reinterpret_cast<uint4*>(yr + c) = float_to_bf16x8(o);
  }
}

// dx = rstd * (g - mean(g) - xh * mean(g * xh)) (+ residual), g = dy * gamma, xh = (x - mu) * rstd.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
layernorm_bwd_dx_kernel(const __nv_bfloat16* __restrict__ dy, const __nv_bfloat16* __restrict__ x, const float* __restrict__ stats,
                        const float* __restrict__ gamma, const __nv_bfloat16* __restrict__ residual, __nv_bfloat16* __restrict__ dx,
                        int64_t rows, int n) {
  const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const __nv_bfloat16* xr = x + row * n;
  const __nv_bfloat16* dr = dy + row * n;
  const float mu = stats[2 * row], rstd = stats[2 * row + 1];
  float s1 = 0.f, s2 = 0.f;
  for (int c = lane * 8; c < n; c += 256) {
    float xf[8], df[8];
    bf16x8_to_float(*reinterpret_cast<const uint4*>(xr + c), xf);
    bf16x8_to_float(*reinterpret_cast<const uint4*>(dr + c), df);
    const float4 g0 = *reinterpret_cast<const float4*>(gamma + c), g1 = *reinterpret_cast<const float4*>(gamma + c + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float gg = df[e] * g[e];
      s1 += gg;
      s2 += gg * (xf[e] - mu) * rstd;
    }
  }
  const float m1 = warp_sum(s1) / (float)n, m2 = warp_sum(s2) / (float)n;
  for (int c = lane * 8; c < n; c += 256) {
    float xf[8], df[8], o[8], rf[8];
    bf16x8_to_float(*reinterpret_cast<const uint4*>(xr + c), xf);
    bf16x8_to_float(*reinterpret_cast<const uint4*>(dr + c), df);
    if (residual) bf16x8_to_float(*reinterpret_cast<const uint4*>(residual + row * n + c), rf);
    const float4 g0 = *reinterpret_cast<const float4*>(gamma + c), g1 = *reinterpret_cast<const float4*>(gamma + c + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float xh = (xf[e] - mu) * rstd;
      o[e] = rstd * (df[e] * g[e] - m1 - xh * m2) + (residual ? rf[e] : 0.f);
    }
    *reinterpret_cast<uint4*>(dx + row * n + c) = float_to_bf16x8(o);
  }
}

// Rows of exactly NCH * 256 columns: a lane keeps its NCH pieces of 8 columns in registers, so the row
// is read from memory once and all its loads are in flight together.
template <int NCH>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
layernorm_fwd_rows_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                          __nv_bfloat16* __restrict__ y, float* __restrict__ stats, int64_t rows, float eps) {
  constexpr int n = NCH * 256;
  const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const __nv_bfloat16* xr = x + row * n + lane * 8;
  uint4 xv[NCH];
#pragma unroll
  for (int i = 0; i < NCH; ++i) xv[i] = *reinterpret_cast<const uint4*>(xr + i * 256);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    float f[8];
    bf16x8_to_float(xv[i], f);
#pragma unroll
    for (int e = 0; e < 8; ++e) s += f[e];
  }
  const float mu = warp_sum(s) / (float)n;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    float f[8];
    bf16x8_to_float(xv[i], f);
#pragma unroll
    for (int e = 0; e < 8; ++e) q += (f[e] - mu) * (f[e] - mu);
  }
  const float rstd = rsqrtf(warp_sum(q) / (float)n + eps);
  if (lane == 0) { stats[2 * row] = mu; stats[2 * row + 1] = rstd; }
  __nv_bfloat16* yr = y + row * n + lane * 8;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int c = i * 256 + lane * 8;
    float f[8], o[8];
    bf16x8_to_float(xv[i], f);
    const float4 g0 = *reinterpret_cast<const float4*>(gamma + c), g1 = *reinterpret_cast<const float4*>(gamma + c + 4);
    const float4 b0 = *reinterpret_cast<const float4*>(beta + c), b1 = *reinterpret_cast<const float4*>(beta + c + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) o[e] = g[e] * (f[e] - mu) * rstd + b[e];
    *reinterpret_cast<uint4*>(yr + i * 256) = float_to_bf16x8(o);
  }
}

// Backward for rows of NCH * 256 columns, dx and the parameter gradients in one pass over dy and x:
// a persistent grid of 8-warp blocks, every warp walks rows with both rows in registers and keeps
// its lanes' partial dgamma / dbeta sums in registers; at the end the block adds them up in shared
// memory and issues one fp32 atomic per column and block.
// kSmemAcc (the 2048-column case, whose 128 partial sums per lane do not fit the registers next to
// the two rows): every warp keeps its partial sums in a shared-memory strip of its own instead.
template <int NCH, bool kSmemAcc>
__global__ void __launch_bounds__(kWarpsPerBlock * 32, 1)
layernorm_bwd_rows_kernel(const __nv_bfloat16* __restrict__ dy, const __nv_bfloat16* __restrict__ x, const float* __restrict__ stats,
                          const float* __restrict__ gamma, const __nv_bfloat16* __restrict__ residual, __nv_bfloat16* __restrict__ dx,
                          float* __restrict__ dgamma, float* __restrict__ dbeta, float* __restrict__ partial, int64_t rows) {
  constexpr int n = NCH * 256;
  constexpr int kAccRegs = kSmemAcc ? 1 : NCH;
  extern __shared__ float4 sh_dyn[];
  float* const sh = reinterpret_cast<float*>(sh_dyn);                 // [2][n] block sums, then (kSmemAcc) [warps][2][n] strips
  const int n_sh = 2 * n * (kSmemAcc ? 1 + kWarpsPerBlock : 1);
  for (int i = threadIdx.x; i < n_sh; i += kWarpsPerBlock * 32) sh[i] = 0.f;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  float* const strip = sh + 2 * n * (1 + (threadIdx.x >> 5));           // this warp's strip: [2][n]
  const int64_t wid = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5), nw = (int64_t)gridDim.x * kWarpsPerBlock;
  float ag[kAccRegs][8], ab[kAccRegs][8];
#pragma unroll
  for (int i = 0; i < kAccRegs; ++i)
#pragma unroll
    for (int e = 0; e < 8; ++e) { ag[i][e] = 0.f; ab[i][e] = 0.f; }
  for (int64_t row = wid; row < rows; row += nw) {
    const __nv_bfloat16* xr = x + row * n + lane * 8;
    const __nv_bfloat16* dr = dy + row * n + lane * 8;
    uint4 xv[NCH], dv[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) { xv[i] = *reinterpret_cast<const uint4*>(xr + i * 256); dv[i] = *reinterpret_cast<const uint4*>(dr + i * 256); }
    const float mu = stats[2 * row], rstd = stats[2 * row + 1];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int c = i * 256 + lane * 8;
      float xf[8], df[8];
      bf16x8_to_float(xv[i], xf);
      bf16x8_to_float(dv[i], df);
      const float4 g0 = *reinterpret_cast<const float4*>(gamma + c), g1 = *reinterpret_cast<const float4*>(gamma + c + 4);
      const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
      if (kSmemAcc) {
        float4* pg = reinterpret_cast<float4*>(strip + c);
        float4* pb = reinterpret_cast<float4*>(strip + n + c);
        float4 a0 = pg[0], a1 = pg[1], b0 = pb[0], b1 = pb[1];
        float ga[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w}, be[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float xh = (xf[e] - mu) * rstd;
          const float gg = df[e] * g[e];
          s1 += gg;
          s2 += gg * xh;
          ga[e] += df[e] * xh;
          be[e] += df[e];
        }
        pg[0] = make_float4(ga[0], ga[1], ga[2], ga[3]); pg[1] = make_float4(ga[4], ga[5], ga[6], ga[7]);
        pb[0] = make_float4(be[0], be[1], be[2], be[3]); pb[1] = make_float4(be[4], be[5], be[6], be[7]);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float xh = (xf[e] - mu) * rstd;
          const float gg = df[e] * g[e];
          s1 += gg;
          s2 += gg * xh;
          ag[kSmemAcc ? 0 : i][e] += df[e] * xh;
          ab[kSmemAcc ? 0 : i][e] += df[e];
        }
      }
    }
    const float m1 = warp_sum(s1) / (float)n, m2 = warp_sum(s2) / (float)n;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int c = i * 256 + lane * 8;
      float xf[8], df[8], o[8], rf[8];
      bf16x8_to_float(xv[i], xf);
      bf16x8_to_float(dv[i], df);
      if (residual) bf16x8_to_float(*reinterpret_cast<const uint4*>(residual + row * n + c), rf);
      const float4 g0 = *reinterpret_cast<const float4*>(gamma + c), g1 = *reinterpret_cast<const float4*>(gamma + c + 4);
      const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float xh = (xf[e] - mu) * rstd;
        o[e] = rstd * (df[e] * g[e] - m1 - xh * m2) + (residual ? rf[e] : 0.f);
      }
      *reinterpret_cast<uint4*>(dx + row * n + c) = float_to_bf16x8(o);
    }
  }
  // Block sums in warp order (a fixed order), then either into this block's row of `partial` ([gridDim.x][2][n];
  // colsum_finalize_kernel adds the blocks up in block order, so the result repeats bit for bit) or, without
  // a partial buffer, onto the zeroed outputs with fp32 atomics.
  if (dgamma && dbeta) {
    if (kSmemAcc) {
      __syncthreads();
      for (int c = threadIdx.x; c < 2 * n; c += kWarpsPerBlock * 32) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kWarpsPerBlock; ++w) t += sh[2 * n * (1 + w) + c];
        if (partial) partial[(size_t)blockIdx.x * 2 * n + c] = t;
        else atomicAdd((c < n ? dgamma : dbeta) + (c < n ? c : c - n), t);
      }
    } else {
      for (int w = 0; w < kWarpsPerBlock; ++w) {
        if ((int)(threadIdx.x >> 5) == w) {
#pragma unroll
          for (int i = 0; i < kAccRegs; ++i)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              sh[i * 256 + lane * 8 + e] += ag[i][e];
              sh[n + i * 256 + lane * 8 + e] += ab[i][e];
            }
        }
        __syncthreads();
      }
      for (int c = threadIdx.x; c < 2 * n; c += kWarpsPerBlock * 32) {
        if (partial) partial[(size_t)blockIdx.x * 2 * n + c] = sh[c];
        else atomicAdd((c < n ? dgamma : dbeta) + (c < n ? c : c - n), sh[c]);
      }
    }
  }
}

// Fixed-order finish of column sums whose partial sums were left by `groups` producers: partial is [groups][planes][n].
// A block owns 32 columns; its eight warps each add up one contiguous eighth of the groups in ascending order (loads
// issued four ahead), and the eight sums are then added in warp order.  The order depends on `groups` only, never on
// timing, so the result repeats bit for bit.  planes = 2: out0 from plane 0, out1 from plane 1.
__global__ void __launch_bounds__(256) colsum_finalize_kernel(const float* __restrict__ partial, int groups, int planes, int n, float* __restrict__ out0,
                                                              float* __restrict__ out1) {
  __shared__ float sh[2][8][32];
  const int tx = threadIdx.x & 31, seg = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + tx;
  const int g0 = (int)((long long)groups * seg / 8), g1 = (int)((long long)groups * (seg + 1) / 8);
  float s0 = 0.f, s1 = 0.f;
  if (c < n) {
    const size_t stride = (size_t)planes * n;
    const float* p = partial + (size_t)g0 * stride + c;
    int g = g0;
    for (; g + 4 <= g1; g += 4, p += 4 * stride) {
      const float a0 = p[0], a1 = p[stride], a2 = p[2 * stride], a3 = p[3 * stride];
      float b0 = 0.f, b1 = 0.f, b2 = 0.f, b3 = 0.f;
      if (planes > 1) { b0 = p[n]; b1 = p[stride + n]; b2 = p[2 * stride + n]; b3 = p[3 * stride + n]; }
      s0 = ((s0 + a0) + a1) + a2 + a3;
      s1 = ((s1 + b0) + b1) + b2 + b3;
    }
    for (; g < g1; ++g, p += stride) {
      s0 += p[0];
      if (planes > 1) s1 += p[n];
    }
  }
  sh[0][seg][tx] = s0;
  sh[1][seg][tx] = s1;
  __syncthreads();
  if (seg == 0 && c < n) {
    float t0 = sh[0][0][tx], t1 = sh[1][0][tx];
#pragma unroll
    for (int w = 1; w < 8; ++w) { t0 += sh[0][w][tx]; t1 += sh[1][w][tx]; }
    out0[c] = t0;
    if (planes > 1 && out1) out1[c] = t1;
  }
}

// dgamma[c] += sum_rows dy * xh,  dbeta[c] += sum_rows dy.  Block = 32 x 8 threads: 64 columns
// (two per thread), the 8 thread rows interleave over a chunk of token rows; fp32 atomics finish.
__global__ void __launch_bounds__(256)
layernorm_bwd_params_kernel(const __nv_bfloat16* __restrict__ dy, const __nv_bfloat16* __restrict__ x, const float* __restrict__ stats,
                            float* __restrict__ dgamma, float* __restrict__ dbeta, int64_t rows, int n, int rows_per_block) {
  __shared__ float sh[2][8][64];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int c = blockIdx.x * 64 + tx * 2;
  const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
  const int64_t r1 = r0 + rows_per_block < rows ? r0 + rows_per_block : rows;
  float ag0 = 0.f, ag1 = 0.f, ab0 = 0.f, ab1 = 0.f;
  if (c < n) {
    for (int64_t r = r0 + ty; r < r1; r += 8) {
      const uint32_t dv = *reinterpret_cast<const uint32_t*>(dy + r * n + c);
      const uint32_t xv = *reinterpret_cast<const uint32_t*>(x + r * n + c);
      const float mu = stats[2 * r], rstd = stats[2 * r + 1];
      const float d0 = __uint_as_float(dv << 16), d1 = __uint_as_float(dv & 0xFFFF0000u);
      const float x0 = __uint_as_float(xv << 16), x1 = __uint_as_float(xv & 0xFFFF0000u);
      ag0 += d0 * (x0 - mu) * rstd;
      ag1 += d1 * (x1 - mu) * rstd;
      ab0 += d0;
      ab1 += d1;
    }
  }
  sh[0][ty][tx * 2] = ag0; sh[0][ty][tx * 2 + 1] = ag1;
  sh[1][ty][tx * 2] = ab0; sh[1][ty][tx * 2 + 1] = ab1;
  __syncthreads();
  if (threadIdx.x < 128) {
    const int which = threadIdx.x >> 6, col = threadIdx.x & 63;
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) s += sh[which][j][col];
    const int cc = blockIdx.x * 64 + col;
    if (cc < n) atomicAdd((which == 0 ? dgamma : dbeta) + cc, s);
  }
}

cudaError_t last_error() { return cudaGetLastError(); }

}  // namespace

namespace mtf {

static mtf_status check(const char* what) {
  cudaError_t e = last_error();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  return MTF_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

mtf_status launch_softmax_fwd(const float* logits, void* weights, int64_t rows, int n, int L, int causal, void* stream) {
  if (n % 8 || !aligned16(logits) || !aligned16(weights)) return fail(MTF_ERR_UNSUPPORTED, "softmax: row length must be a multiple of 8 and pointers 16-byte aligned");
  if (rows <= 0) return MTF_OK;
  const int64_t blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (blocks > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "softmax: too many rows");
  softmax_fwd_kernel<<<(unsigned)blocks, kWarpsPerBlock * 32, 0, (cudaStream_t)stream>>>(logits, reinterpret_cast<__nv_bfloat16*>(weights), rows, n, L, causal);
  count_launch();
  return check("softmax_fwd_kernel");
}

mtf_status launch_softmax_bwd(const void* P, const float* dP, void* dlg, int64_t rows, int n, void* stream) {
  if (n % 8 || !aligned16(P) || !aligned16(dP) || !aligned16(dlg)) return fail(MTF_ERR_UNSUPPORTED, "softmax backward: row length must be a multiple of 8 and pointers 16-byte aligned");
  if (rows <= 0) return MTF_OK;
  const int64_t blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (blocks > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "softmax backward: too many rows");
  softmax_bwd_kernel<<<(unsigned)blocks, kWarpsPerBlock * 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<const __nv_bfloat16*>(P), dP, reinterpret_cast<__nv_bfloat16*>(dlg), rows, n);
  count_launch();
  return check("softmax_bwd_kernel");
}

mtf_status launch_layernorm_fwd(const void* x, const float* gamma, const float* beta, void* y, float* stats, int64_t rows, int n, float eps, void* stream) {
  if (n % 8 || !aligned16(x) || !aligned16(y) || !aligned16(gamma) || !aligned16(beta)) return fail(MTF_ERR_UNSUPPORTED, "layernorm: row length must be a multiple of 8 and pointers 16-byte aligned");
  if (rows <= 0) return MTF_OK;
  const int64_t blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (blocks > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "layernorm: too many rows");
  const __nv_bfloat16* xb = reinterpret_cast<const __nv_bfloat16*>(x);
  __nv_bfloat16* yb = reinterpret_cast<__nv_bfloat16*>(y);
  cudaStream_t st = (cudaStream_t)stream;
  // rows of 256, 512, 1024 or 2048 columns stay in registers; other lengths re-read the row per pass
  switch (n) {
    case 256: layernorm_fwd_rows_kernel<1><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, st>>>(xb, gamma, beta, yb, stats, rows, eps); break;
    case 512: layernorm_fwd_rows_kernel<2><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, st>>>(xb, gamma, beta, yb, stats, rows, eps); break;
    case 1024: layernorm_fwd_rows_kernel<4><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, st>>>(xb, gamma, beta, yb, stats, rows, eps); break;
    case 2048: layernorm_fwd_rows_kernel<8><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, st>>>(xb, gamma, beta, yb, stats, rows, eps); break;
    default: layernorm_fwd_kernel<<<(unsigned)blocks, kWarpsPerBlock * 32, 0, st>>>(xb, gamma, beta, yb, stats, rows, n, eps);
  }
  count_launch();
  return check("layernorm_fwd_kernel");
}

// Bytes of scratch with which the parameter gradients are summed in a fixed order (0: this row length always uses atomics)
size_t layernorm_bwd_scratch_bytes(int n) {
  if (n != 256 && n != 512 && n != 1024 && n != 2048) return 0;
  return (size_t)device_sm_count() * 2 * 2 * n * sizeof(float);
}

mtf_status launch_colsum_finalize(const float* partial, int groups, int planes, int n, float* out0, float* out1, void* stream) {
  colsum_finalize_kernel<<<(unsigned)((n + 31) / 32), 256, 0, (cudaStream_t)stream>>>(partial, groups, planes, n, out0, out1);
  count_launch();
  return check("colsum_finalize_kernel");
}

mtf_status launch_layernorm_bwd(const void* dy, const void* x, const float* stats, const float* gamma, const void* residual, void* dx,
                                float* dgamma, float* dbeta, int64_t rows, int n, void* scratch, size_t scratch_bytes, void* stream) {
  if (n % 8 || !aligned16(x) || !aligned16(dy) || !aligned16(dx) || !aligned16(gamma) || (residual && !aligned16(residual)))
    return fail(MTF_ERR_UNSUPPORTED, "layernorm backward: row length must be a multiple of 8 and pointers 16-byte aligned");
  if (rows <= 0) return MTF_OK;
  cudaStream_t st = (cudaStream_t)stream;
  if (n == 256 || n == 512 || n == 1024 || n == 2048) {
    // one pass over dy and x for dx and the parameter gradients (persistent grid)
    const int sms = device_sm_count();
    unsigned grid = (unsigned)std::min<int64_t>((rows + kWarpsPerBlock - 1) / kWarpsPerBlock, 2 * (int64_t)sms);
    if (n == 2048) grid = std::min(grid, (unsigned)sms);
    const bool want = dgamma && dbeta;
    float* partial = nullptr;
    if (want && scratch && !(reinterpret_cast<uintptr_t>(scratch) & 15) && scratch_bytes >= (size_t)grid * 2 * n * sizeof(float)) partial = reinterpret_cast<float*>(scratch);
    if (want && !partial) {
      cudaError_t e = cudaMemsetAsync(dgamma, 0, (size_t)n * sizeof(float), st);
      if (e == cudaSuccess) e = cudaMemsetAsync(dbeta, 0, (size_t)n * sizeof(float), st);
      if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    }
    const __nv_bfloat16* db = reinterpret_cast<const __nv_bfloat16*>(dy);
    const __nv_bfloat16* xb = reinterpret_cast<const __nv_bfloat16*>(x);
    const __nv_bfloat16* rb = reinterpret_cast<const __nv_bfloat16*>(residual);
    __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(dx);
    float* dg = want ? dgamma : nullptr;
    float* dbp = want ? dbeta : nullptr;
    const size_t sm_small = 2 * (size_t)n * sizeof(float), sm_big = sm_small * (1 + kWarpsPerBlock);       // 144 KB for 2048 columns
    switch (n) {
      case 256: layernorm_bwd_rows_kernel<1, false><<<grid, kWarpsPerBlock * 32, sm_small, st>>>(db, xb, stats, gamma, rb, ob, dg, dbp, partial, rows); break;
      case 512: layernorm_bwd_rows_kernel<2, false><<<grid, kWarpsPerBlock * 32, sm_small, st>>>(db, xb, stats, gamma, rb, ob, dg, dbp, partial, rows); break;
      case 1024: layernorm_bwd_rows_kernel<4, false><<<grid, kWarpsPerBlock * 32, sm_small, st>>>(db, xb, stats, gamma, rb, ob, dg, dbp, partial, rows); break;
      default: {
        static cudaError_t attr = cudaFuncSetAttribute(layernorm_bwd_rows_kernel<8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(2 * 2048 * sizeof(float) * (1 + kWarpsPerBlock)));
        if (attr != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(attr));
        layernorm_bwd_rows_kernel<8, true><<<grid, kWarpsPerBlock * 32, sm_big, st>>>(db, xb, stats, gamma, rb, ob, dg, dbp, partial, rows);
      }
    }
    count_launch();
    mtf_status s2 = check("layernorm_bwd_rows_kernel");
    if (s2 != MTF_OK || !partial) return s2;
    return launch_colsum_finalize(partial, (int)grid, 2, n, dgamma, dbeta, stream);
  }
  const int64_t blocks = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (blocks > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "layernorm backward: too many rows");
  layernorm_bwd_dx_kernel<<<(unsigned)blocks, kWarpsPerBlock * 32, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(dy), reinterpret_cast<const __nv_bfloat16*>(x), stats, gamma,
                                                                          reinterpret_cast<const __nv_bfloat16*>(residual), reinterpret_cast<__nv_bfloat16*>(dx), rows, n);
  count_launch();
  mtf_status s = check("layernorm_bwd_dx_kernel");
  if (s != MTF_OK) return s;
  if (dgamma && dbeta) {
    cudaError_t e = cudaMemsetAsync(dgamma, 0, (size_t)n * sizeof(float), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(dbeta, 0, (size_t)n * sizeof(float), st);
    if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    const int rows_per_block = 256;
    dim3 grid((unsigned)((n + 63) / 64), (unsigned)((rows + rows_per_block - 1) / rows_per_block));
    layernorm_bwd_params_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(dy), reinterpret_cast<const __nv_bfloat16*>(x), stats, dgamma, dbeta, rows, n, rows_per_block);
    count_launch();
    s = check("layernorm_bwd_params_kernel");
  }
  return s;
}

// (no row kernel has a bounded wait today: the status word of this family stays 0)
mtf_status read_row_status(int* code) {
  *code = 0;
  return MTF_OK;
}

}  // namespace mtf
