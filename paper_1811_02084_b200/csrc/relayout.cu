// Data movement of Section 6.1 (reshape with a change of layout) on one GPU.
//
// A tensor is stored once, globally; a virtual processor's slice is a box view of it.  A reshape that
// only changes dimension names therefore moves NO data on one GPU - whatever Allgather, slicing or
// Alltoall the paper's per-processor representation would need is already "done" by every slice being
// a view of the one stored tensor - and the library reports the pattern and the element counts the
// paper's lowering would have communicated (host planner, api).  What does move data:
//   * a change of storage order (the block transpose of an Alltoall, [b, l, h, k] <-> [b, h, l, k]):
//     permute_copy_kernel / permute_transpose_kernel below, bound by HBM (2 bytes in, 2 bytes out
//     per bf16 element);
//   * copying one processor's slice out of / into the global tensor (the per-processor view of an
//     Allgather or of a slice): the same row-copy kernel on a box.
// Index arithmetic uses multiply-high divisions with host-made constants: one divmod per dimension
// per 16-byte piece would otherwise cost more issue slots than the copy has bandwidth for.
#include <cuda_runtime.h>

#include <algorithm>

#include "mtf_internal.h"

namespace {

struct FastDiv32 {
  uint32_t d, mul, shr;
};
FastDiv32 make_fd(long long divisor) {
  FastDiv32 f;
  f.d = (uint32_t)(divisor < 1 ? 1 : divisor);
  f.mul = 0; f.shr = 0;
  if (f.d > 1) {
    uint32_t l = 0;
    while ((1ull << l) < f.d) ++l;
    const unsigned p = 31 + l;
    f.mul = (uint32_t)(((1ull << p) + f.d - 1) / f.d);
    f.shr = p - 32;
  }
  return f;
}
__device__ __forceinline__ uint32_t fd_divmod(uint32_t n, const FastDiv32& f, uint32_t* rem) {
  const uint32_t q = f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr);
  *rem = n - q * f.d;
  return q;
}

constexpr int kMaxD = mtf::kMaxTensorDims;

// Copy of an n-d box, iterated in the DESTINATION's dimension order; the innermost dimension is
// contiguous on both sides and moves in 16-byte pieces.
struct RowCopy {
  int ndim;                       // outer dimensions (without the innermost one)
  FastDiv32 size[kMaxD];          // extents of the outer dimensions, destination order
  long long sstr[kMaxD], dstr[kMaxD];   // strides in 16-byte pieces... of elements scaled: see launcher (in pieces)
  FastDiv32 pieces;               // 16-byte pieces per innermost row
  long long total;                // rows * pieces
};

__global__ void __launch_bounds__(256) permute_copy_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, const RowCopy c) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < c.total; i += (long long)gridDim.x * blockDim.x) {
    uint32_t piece, rem;
    uint32_t row = fd_divmod((uint32_t)i, c.pieces, &piece);
    long long so = piece, d_o = piece;
#pragma unroll 1
    for (int d = c.ndim - 1; d >= 0; --d) {
      row = fd_divmod(row, c.size[d], &rem);
      so += (long long)rem * c.sstr[d];
      d_o += (long long)rem * c.dstr[d];
    }
    dst[d_o] = src[so];
  }
}

// Permutation that changes the innermost dimension: 64 x 64 element tiles through shared memory over
// (the source's innermost dimension, the destination's innermost dimension); everything else is batch.
struct TileTranspose {
  int nbatch;
  FastDiv32 bsize[kMaxD];
  long long bs_src[kMaxD], bs_dst[kMaxD];     // element strides of the batch dimensions
  int n_a, n_b;                               // extents: a = source-innermost dim, b = destination-innermost dim
  long long sa_dst, sb_src;                   // element stride of a in the destination, of b in the source
  FastDiv32 tiles_a, tiles_b;
  long long total_tiles;
};

template <typename T>
__global__ void __launch_bounds__(256) permute_transpose_kernel(const T* __restrict__ src, T* __restrict__ dst, const TileTranspose c) {
  __shared__ T tile[64][64 + 2];
  for (long long t = blockIdx.x; t < c.total_tiles; t += gridDim.x) {
    uint32_t ta, tb, rem;
    uint32_t w = fd_divmod((uint32_t)t, c.tiles_a, &ta);
    w = fd_divmod(w, c.tiles_b, &tb);
    long long so = 0, d_o = 0;
    for (int d = c.nbatch - 1; d >= 0; --d) {
      w = fd_divmod(w, c.bsize[d], &rem);
      so += (long long)rem * c.bs_src[d];
      d_o += (long long)rem * c.bs_dst[d];
    }
    const int a0 = (int)ta * 64, b0 = (int)tb * 64;
    const int lx = threadIdx.x & 63, ly = threadIdx.x >> 6;       // 64 x 4 threads
    for (int r = ly; r < 64; r += 4)                                   // rows along b, contiguous along a
      if (b0 + r < c.n_b && a0 + lx < c.n_a) tile[r][lx] = src[so + (long long)(b0 + r) * c.sb_src + a0 + lx];
    __syncthreads();
    for (int r = ly; r < 64; r += 4)                                   // rows along a, contiguous along b
      if (a0 + r < c.n_a && b0 + lx < c.n_b) dst[d_o + (long long)(a0 + r) * c.sa_dst + b0 + lx] = tile[lx][r];
    __syncthreads();
  }
}

// The same for 2-byte elements with whole 64 x 64 tiles and 16-byte aligned rows on both sides: 16-byte loads along
// the source's contiguous dimension, 16-byte stores along the destination's.  The tile is kept as 32-bit words (two
// neighbouring source columns each) with a row stride of 33 words: the four word stores of a loaded piece and the
// eight word reads of an output piece are both free of bank conflicts (a warp covers 4 pieces x 8 word columns), and
// a thread turns its eight words into two output pieces (the low halves and the high halves) with byte permutes.
__global__ void __launch_bounds__(256) permute_transpose16_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, const TileTranspose c) {
  __shared__ uint32_t tile[64][33];
  const int lp = threadIdx.x & 7, lr = threadIdx.x >> 3;                      // load: piece of 8 elements, row (and row + 32)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int px = (warp & 1) * 4 + (lane & 3), rr = (warp >> 1) * 8 + (lane >> 2);      // store: piece of 8 output columns, pair of output rows
  for (long long t = blockIdx.x; t < c.total_tiles; t += gridDim.x) {
    uint32_t ta, tb, rem;
    uint32_t w = fd_divmod((uint32_t)t, c.tiles_a, &ta);
    w = fd_divmod(w, c.tiles_b, &tb);
    long long so = 0, d_o = 0;
    for (int d = c.nbatch - 1; d >= 0; --d) {
      w = fd_divmod(w, c.bsize[d], &rem);
      so += (long long)rem * c.bs_src[d];
      d_o += (long long)rem * c.bs_dst[d];
    }
    const int a0 = (int)ta * 64, b0 = (int)tb * 64;
    uint4 in[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) in[k] = *reinterpret_cast<const uint4*>(src + so + (long long)(b0 + lr + 32 * k) * c.sb_src + a0 + lp * 8);
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      uint32_t* row = &tile[lr + 32 * k][lp * 4];
      row[0] = in[k].x; row[1] = in[k].y; row[2] = in[k].z; row[3] = in[k].w;
    }
    __syncthreads();
    uint32_t v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = tile[px * 8 + e][rr];
    uint4 lo, hi;
    lo.x = __byte_perm(v[0], v[1], 0x5410); lo.y = __byte_perm(v[2], v[3], 0x5410); lo.z = __byte_perm(v[4], v[5], 0x5410); lo.w = __byte_perm(v[6], v[7], 0x5410);
    hi.x = __byte_perm(v[0], v[1], 0x7632); hi.y = __byte_perm(v[2], v[3], 0x7632); hi.z = __byte_perm(v[4], v[5], 0x7632); hi.w = __byte_perm(v[6], v[7], 0x7632);
    uint16_t* out = dst + d_o + (long long)(a0 + 2 * rr) * c.sa_dst + b0 + px * 8;
    *reinterpret_cast<uint4*>(out) = lo;
    *reinterpret_cast<uint4*>(out + c.sa_dst) = hi;
    __syncthreads();
  }
}

}  // namespace

namespace mtf {

// dst[...] = src[...] for a box described in the destination's dimension order: sizes[i], element strides
// sstr[i] / dstr[i]; the last dimension must be contiguous on both sides.  Falls back to the tile
// transpose when it is not (then the source's contiguous dimension is `src_inner`).
mtf_status launch_permute_copy(const void* src, void* dst, int elem_bytes, int ndim, const int64_t* sizes, const int64_t* sstr, const int64_t* dstr, void* stream) {
  int64_t total = 1;
  for (int i = 0; i < ndim; ++i) total *= sizes[i];
  if (total <= 0) return MTF_OK;
  if (total >= 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "copy of more than 2^31 elements");
  cudaStream_t st = (cudaStream_t)stream;
  const int vec = 16 / elem_bytes;
  const bool inner_same = ndim >= 1 && sstr[ndim - 1] == 1 && dstr[ndim - 1] == 1;
  bool vec_ok = inner_same && sizes[ndim - 1] % vec == 0 && !(reinterpret_cast<uintptr_t>(src) & 15) && !(reinterpret_cast<uintptr_t>(dst) & 15);
  for (int i = 0; vec_ok && i + 1 < ndim; ++i) vec_ok = sstr[i] % vec == 0 && dstr[i] % vec == 0;
  if (vec_ok) {
    RowCopy c;
    c.ndim = ndim - 1;
    for (int i = 0; i + 1 < ndim; ++i) { c.size[i] = make_fd(sizes[i]); c.sstr[i] = sstr[i] / vec; c.dstr[i] = dstr[i] / vec; }
    c.pieces = make_fd(sizes[ndim - 1] / vec);
    c.total = total / vec;
    const long long blocks = std::min<long long>((c.total + 255) / 256, (long long)device_sm_count() * 16);
    permute_copy_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), c);
  } else {
    // a = the source's contiguous dimension, b = the destination's contiguous dimension
    int ia = -1, ib = ndim - 1;
    for (int i = 0; i < ndim; ++i) if (sstr[i] == 1 && sizes[i] > 1) ia = i;
    if (dstr[ib] != 1) return fail(MTF_ERR_UNSUPPORTED, "permuting copy: the destination's last dimension must be contiguous");
    if (ia < 0 || ia == ib) {
      // no distinct contiguous source dimension (or an unaligned same-inner copy): element-wise row copy with one "piece" per element
      ia = -1;
    }
    TileTranspose c;
    c.nbatch = 0;
    if (ia < 0) {
      // degenerate: treat the innermost dimension as b and a dimension of extent 1 as a
      c.n_a = 1; c.sa_dst = 0;
    } else { c.n_a = (int)sizes[ia]; c.sa_dst = dstr[ia]; }
    c.n_b = (int)sizes[ib]; c.sb_src = sstr[ib];
    for (int i = 0; i < ndim; ++i) {
      if (i == ia || i == ib) continue;
      c.bsize[c.nbatch] = make_fd(sizes[i]); c.bs_src[c.nbatch] = sstr[i]; c.bs_dst[c.nbatch] = dstr[i]; ++c.nbatch;
    }
    const long long ta = (c.n_a + 63) / 64, tb = (c.n_b + 63) / 64;
    c.tiles_a = make_fd(ta); c.tiles_b = make_fd(tb);
    c.total_tiles = ta * tb;
    for (int i = 0; i < c.nbatch; ++i) c.total_tiles *= c.bsize[i].d;
    const long long blocks = std::min<long long>(c.total_tiles, (long long)device_sm_count() * 8);
    bool fast16 = elem_bytes == 2 && ia >= 0 && c.n_a % 64 == 0 && c.n_b % 64 == 0 && c.sb_src % 8 == 0 && c.sa_dst % 8 == 0 &&
                  !(reinterpret_cast<uintptr_t>(src) & 15) && !(reinterpret_cast<uintptr_t>(dst) & 15);
    for (int i = 0; fast16 && i < c.nbatch; ++i) fast16 = c.bs_src[i] % 8 == 0 && c.bs_dst[i] % 8 == 0;
    if (fast16) permute_transpose16_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), c);
    else if (elem_bytes == 2) permute_transpose_kernel<uint16_t><<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(dst), c);
    else permute_transpose_kernel<uint32_t><<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(src), reinterpret_cast<uint32_t*>(dst), c);
  }
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "permute copy kernel: %s", cudaGetErrorString(e));
  return MTF_OK;
}

}  // namespace mtf
