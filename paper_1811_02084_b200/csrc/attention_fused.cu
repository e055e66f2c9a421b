// Attention core of the Transformer layout (Section 9: batch and heads are the split dimensions, so every
// (batch, head) pair is an independent problem on whichever virtual processor owns it) in ONE launch:
//     logits[l, m] = scale * sum_k q[l, k] kk[m, k]   (causal: m <= l only)
//     P = softmax over m                               (bf16, written once for the backward pass)
//     o[l, v] = sum_m P[l, m] vv[m, v]
// The fp32 logits live in tensor memory only; the weights go from the softmax warps' registers into a
// shared-memory tile that is at the same time the source of the store to HBM and the A operand of the
// second contraction, so P is never read back.  d_k = d_v = 64, length = memory_length in {128, 256, 384,
// 512} (a whole row of logits fits the 512 columns of tensor memory); other shapes take the launch-per-
// einsum path.
//
// A persistent CTA (one per SM) walks a contiguous, balanced range of (pair, query tile of 128 rows) items; K and V
// of a (batch, head) pair stay in shared memory for all of the pair's tiles in the range, K of the next pair is
// fetched as soon as the last logits of this one are complete, V as soon as its last weights . v is.
// Warp roles (576 threads):
//   warp 0     TMA producer: K, V once per pair; Q per tile
//   warp 1     MMA issuer:   S = Q K^T (tcgen05.mma kind::f16, N up to 256 per instruction), then
//                            O += P_c V_c for every 64-key chunk c of P as it arrives in shared memory
//   warps 2-17 softmax:      four warps per tensor-memory lane quarter; warp part p owns the 64-key chunks c with
//                            c mod 4 = p and the chunk buffer p; row maximum and row sum are exchanged through
//                            shared memory at a named barrier of the quarter's 128 threads; the normalised weights
//                            are written as swizzled 32-row boxes (TMA store + MMA operand)
// O is accumulated in the tensor-memory columns of the first chunk of S, which are dead by then.
// Every mbarrier wait is bounded; on expiry a code is recorded in the status word, a CTA-wide abort flag is raised,
// the remaining waits return at once, work is skipped, and all roles leave through the teardown.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "mtf_internal.h"

namespace {

constexpr int kSoftmaxWarps = 16;                 // four per tensor-memory lane quarter
constexpr int kThreads = 64 + 32 * kSoftmaxWarps;
constexpr int kQBytes = 128 * 64 * 2;            // one query tile
constexpr int kPBufBytes = 128 * 64 * 2;         // one 64-key chunk of the weights for 128 rows
constexpr int kPBufs = 4;                         // one chunk buffer per softmax part: a buffer is written by the same four warps every time
constexpr int kMaxL = 512;
constexpr long long kWaitCycles = 4000000000LL;

__device__ int g_att_status = 0;

struct AttArgs {
  int B, H, L;
  int causal;
  float scale;
  __nv_bfloat16* o;              // [B, L, H, 64]
  long long units;               // B * H
};

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mb_init(uint32_t bar, uint32_t count) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory"); }
__device__ __forceinline__ void mb_expect(uint32_t bar, uint32_t bytes) { asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory"); }
__device__ __forceinline__ void mb_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ bool mb_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __noinline__ bool mb_wait_slow(uint32_t bar, uint32_t parity, int code, volatile int* abort_flag) {
  const long long t0 = clock64();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (mb_try(bar, parity)) return true;
    if (*abort_flag) return false;
    __nanosleep(64);
    if (clock64() - t0 > kWaitCycles) {
      atomicCAS(&g_att_status, 0, code);
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ bool mb_wait(uint32_t bar, uint32_t parity, int code, volatile int* abort_flag) {
  for (int i = 0; i < 16; ++i)
    if (mb_try(bar, parity)) return true;
  return mb_wait_slow(bar, parity, code, abort_flag);
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma(uint32_t tmem_c, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_c), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
      ::"r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]),
        "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]),
        "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Shared-memory matrix descriptor of a 128B-swizzled bf16 tile (rows of 128 bytes, 8-row groups 1024 bytes apart):
// K-major (a row holds 64 k-elements) or MN-major (a row holds 64 m/n-elements of one k).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, int mn_major) {
  const uint64_t lbo = mn_major ? (8192u >> 4) : 1u;
  const uint64_t sbo = 1024u >> 4;
  return (uint64_t)((addr & 0x3FFFF) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h2);
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

// live 64-key chunks of query tile qt: all of them, or under the causal limit those that hold a key <= the tile's last row
__device__ __forceinline__ int live_chunks(const AttArgs& a, int qt) { return a.causal ? min(a.L / 64, 2 * (qt + 1)) : a.L / 64; }

__global__ void __launch_bounds__(kThreads, 1)
attention_fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const __grid_constant__ CUtensorMap map_p, const AttArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = s_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int L = a.L, nc = L / 64, q_tiles = L / 128;
  // layout: Q | K (L rows) | V (L rows) | P chunk buffers | zero box | exchange slots | barriers
  const uint32_t sQ = base, sK = sQ + kQBytes, sV = sK + (uint32_t)L * 128u, sP = sV + (uint32_t)L * 128u;
  const uint32_t sZero = sP + kPBufs * kPBufBytes;
  const uint32_t sX = sZero + 4096u;                          // [2 slots][16 warps][32 lanes] floats
  const uint32_t bar0 = sX + 2u * kSoftmaxWarps * 32u * 4u;
  uint64_t* bars_gen = reinterpret_cast<uint64_t*>(gen + (bar0 - base));
  // barriers: 0 q_full; 1 q_empty; 2 v_full; 3 v_empty; 4 k_full; 5 k_empty; 6 s_full; 7 o_full; 8 o_empty; 9..12 p_full (the four quarter boxes of
  // a chunk buffer are written); 13..16 p_free (the MMAs that read a chunk buffer have retired).  Every barrier has one set of
  // waiters that see each of its phases in order, so a parity wait can never be a phase behind.
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_gen + 24);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this CTA's query tiles: a contiguous, balanced range of all (pair, tile) items
  const long long total_tiles = a.units * q_tiles;
  const long long g0 = total_tiles * blockIdx.x / gridDim.x, g1 = total_tiles * (blockIdx.x + 1) / gridDim.x;

  if (threadIdx.x == 0) {
    mb_init(bar(0), 1); mb_init(bar(1), 1); mb_init(bar(2), 1); mb_init(bar(3), 1);
    mb_init(bar(4), 1); mb_init(bar(5), 1); mb_init(bar(6), 1); mb_init(bar(7), 1); mb_init(bar(8), 4);
    for (int i = 0; i < kPBufs; ++i) { mb_init(bar(9 + i), 4); mb_init(bar(13 + i), 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_p) : "memory");
  }
  for (int i = threadIdx.x; i < 4096 / 16; i += kThreads) sts_v4(sZero + 16u * i, 0u, 0u, 0u, 0u);
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the zero box is read by TMA stores
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      long long tile_seq = 0, unit_seq = -1;
      bool ok = true;
      for (long long g = g0; ok && g < g1; ++g, ++tile_seq) {
        const long long u = g / q_tiles;
        const int qt = (int)(g % q_tiles);
        const int b = (int)(u / a.H), h = (int)(u % a.H);
        const bool new_unit = g == g0 || qt == 0;
        if (new_unit) {
          ++unit_seq;
          if (!(ok = mb_wait(bar(5), ((uint32_t)unit_seq & 1u) ^ 1u, 0x901, abort_flag))) break;      // K of the previous pair is no longer read
          mb_expect(bar(4), (uint32_t)L * 128u);
          for (int r = 0; r < L; r += 128) tma_load_4d(sK + (uint32_t)r * 128u, &map_k, bar(4), 0, r, h, b);
        }
        if (!(ok = mb_wait(bar(1), ((uint32_t)tile_seq & 1u) ^ 1u, 0x902, abort_flag))) break;        // the logits of the previous tile are complete
        mb_expect(bar(0), kQBytes);
        tma_load_4d(sQ, &map_q, bar(0), 0, qt * 128, h, b);
        if (new_unit) {
          // V is wanted only after the softmax of the pair's first tile: its load waits for the previous pair's last MMA
          // without holding up K and Q
          if (!(ok = mb_wait(bar(3), ((uint32_t)unit_seq & 1u) ^ 1u, 0x903, abort_flag))) break;
          mb_expect(bar(2), (uint32_t)L * 128u);
          for (int r = 0; r < L; r += 64) tma_load_4d(sV + (uint32_t)r * 128u, &map_v, bar(2), 0, r, h, b);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer ---------------------------------
    if (lane == 0) {
      long long tile_seq = 0, unit_seq = -1;
      uint32_t pu[kPBufs] = {0u, 0u, 0u, 0u};          // uses of every chunk buffer so far
      const uint64_t dP0 = smem_desc(sP, 0), dV0 = smem_desc(sV, 1), dQ0 = smem_desc(sQ, 0), dK0 = smem_desc(sK, 0);
      bool ok = true;
      {
        for (long long g = g0; ok && g < g1; ++g, ++tile_seq) {
          const int qt = (int)(g % q_tiles);
          const bool new_unit = g == g0 || qt == 0;
          const bool last_of_unit = qt == q_tiles - 1 || g == g1 - 1;
          if (new_unit) {
            ++unit_seq;
            if (!(ok = mb_wait(bar(4), (uint32_t)unit_seq & 1u, 0x911, abort_flag))) break;
          }
          const int live = live_chunks(a, qt);
          const int keys = live * 64 > L ? L : ((live * 64 + 127) / 128) * 128;      // logits columns to compute (whole 128-key blocks)
          if (!(ok = mb_wait(bar(0), (uint32_t)tile_seq & 1u, 0x912, abort_flag))) break;
          if (!(ok = mb_wait(bar(8), ((uint32_t)tile_seq & 1u) ^ 1u, 0x913, abort_flag))) break;       // O of the previous tile has been read out
          fence_after();
          // S = Q K^T: up to two instructions shapes of N <= 256 columns
          for (int n0 = 0; n0 < keys; n0 += 256) {
            const int nn = min(256, keys - n0);
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nn >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma(tmem + (uint32_t)n0, dQ0 + 2u * k, dK0 + (uint64_t)(((uint32_t)n0 * 128u) >> 4) + 2u * k, idesc, k != 0);
          }
          umma_commit(bar(6));               // logits complete
          umma_commit(bar(1));               // ... and the Q buffer may be refilled
          if (last_of_unit) umma_commit(bar(5));           // ... and so may K
          if (new_unit && !(ok = mb_wait(bar(2), (uint32_t)unit_seq & 1u, 0x915, abort_flag))) break;
          // O += P_c V_c, chunk by chunk in the order the softmax warps deliver them
          const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
          for (int c = 0; c < live && ok; ++c) {
            const int buf = c & 3;
            if (!(ok = mb_wait(bar(9 + buf), pu[buf] & 1u, 0x914, abort_flag))) break;
            fence_after();
            const uint64_t da = dP0 + (uint64_t)((uint32_t)buf * (kPBufBytes >> 4));
            const uint64_t db = dV0 + (uint64_t)((uint32_t)c * (8192u >> 4));
            umma(tmem, da, db, idesc_pv, (uint32_t)c);
            umma(tmem, da + 2u, db + (2048u >> 4), idesc_pv, 1u);
            umma(tmem, da + 4u, db + 2u * (2048u >> 4), idesc_pv, 1u);
            umma(tmem, da + 6u, db + 3u * (2048u >> 4), idesc_pv, 1u);
            umma_commit(bar(13 + buf));      // the chunk's buffer may be rewritten
            ++pu[buf];
          }
          if (!ok) break;
          umma_commit(bar(7));               // O complete
          if (last_of_unit) umma_commit(bar(3));           // V of this pair is no longer read
        }
      }
    }
  } else {
    // ------------------------------- softmax warps ------------------------------
    const int q = warp & 3;                        // tensor-memory lane quarter this warp may access
    const int part = (warp - 2) >> 2;              // which of the four warps of the quarter: owns chunks c with c % 4 == part
    const int slot_id = part * 4 + q;              // 0..15
    const float sl2 = a.scale * 1.4426950408889634f;
    const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16);
    long long tile_seq = 0;
    uint32_t pu = 0;                               // uses of this part's chunk buffer so far
    bool ok = true;
    // row statistics of the four warps that share a row: every warp publishes its value, the 128 threads of the lane quarter
    // meet at a named barrier (the waiting warps take no issue slots), and each reads its three peers'.  The two exchanges
    // of a tile use different slots, so a slot is rewritten only after the other slot's barrier.  Every softmax warp
    // reaches every barrier, also after a failed wait (it skips the work, not the meeting).
    auto exchange = [&](int slot, float mine, bool take_max) -> float {
      const uint32_t off = sX + (uint32_t)slot * (4u * kSoftmaxWarps * 32u);
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(off + 4u * (uint32_t)(slot_id * 32 + lane)), "r"(__float_as_uint(mine)) : "memory");
      asm volatile("bar.sync %0, 128;" ::"r"(1 + q) : "memory");
      float r = mine;
#pragma unroll
      for (int pp = 1; pp < 4; ++pp) {
        uint32_t vb;
        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(vb) : "r"(off + 4u * (uint32_t)((((part + pp) & 3) * 4 + q) * 32 + lane)) : "memory");
        const float other = __uint_as_float(vb);
        r = take_max ? fmaxf(r, other) : r + other;
      }
      return r;
    };
    auto wait_all = [&](int b, uint32_t parity, int code) -> bool {      // all lanes wait (lane 0 polls first)
      int w_ok = 1;
      if (lane == 0) w_ok = mb_wait(bar(b), parity, code, abort_flag) ? 1 : 0;
      w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
      if (!w_ok) return false;
      bool mine_ok = lane == 0 ? true : mb_wait(bar(b), parity, code, abort_flag);
      return __all_sync(0xffffffffu, mine_ok);
    };
    // The trip counts below depend on the arguments alone: after a failed wait a warp keeps going through the tiles (waits
    // then return at once, work is skipped) so that its peers never wait for it at a named barrier.
    {
      for (long long g = g0; g < g1; ++g, ++tile_seq) {
        const long long u = g / q_tiles;
        const int qt = (int)(g % q_tiles);
        const int b = (int)(u / a.H), h = (int)(u % a.H);
        const int live = live_chunks(a, qt);
        const int row = qt * 128 + q * 32 + lane;                 // query position of this thread's row
        const int lim = a.causal ? min(L, row + 1) : L;            // columns [0, lim) take part
        const int lim_warp = __shfl_sync(0xffffffffu, lim, 31);    // the warp's widest row
        const int lim_all = __shfl_sync(0xffffffffu, lim, 0);      // columns below it take part in every row of the warp
        if (ok) ok = wait_all(6, (uint32_t)tile_seq & 1u, 0x921);
        fence_after();
        // pass 1: row maximum over this warp's live columns (chunks part, part + 4, ...)
        float mx = -INFINITY;
        if (ok) {
#pragma unroll 1
          for (int c = part; c < live; c += 4) {
            const int c0 = c * 64;
            if (c0 + 64 <= lim_all) {
              uint32_t rawv[64];
              tmem_ld32(taddr + (uint32_t)c0, rawv);
              tmem_ld32(taddr + (uint32_t)c0 + 32u, rawv + 32);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 64; ++j) mx = fmaxf(mx, __uint_as_float(rawv[j]));
            } else {
#pragma unroll 1
              for (int cc = c0; cc < c0 + 64 && cc < lim_warp; cc += 32) {
                uint32_t rawv[32];
                tmem_ld32(taddr + (uint32_t)cc, rawv);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (cc + j < lim) mx = fmaxf(mx, __uint_as_float(rawv[j]));
              }
            }
          }
        }
        mx = exchange(0, mx, true) * sl2;
        // pass 2: exponentials (kept in tensor memory in place of the logits) and their sum
        float sum = 0.f;
        if (ok) {
#pragma unroll 1
          for (int c = part; c < live; c += 4) {
#pragma unroll 1
            for (int c0 = c * 64; c0 < c * 64 + 64 && c0 < lim_warp; c0 += 32) {
              uint32_t rawv[32];
              tmem_ld32(taddr + (uint32_t)c0, rawv);
              tmem_ld_wait();
              if (c0 + 32 <= lim_all) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  const float e = ex2(fmaf(__uint_as_float(rawv[j]), sl2, -mx));
                  sum += e;
                  rawv[j] = __float_as_uint(e);
                }
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  const float e = (c0 + j < lim) ? ex2(fmaf(__uint_as_float(rawv[j]), sl2, -mx)) : 0.f;
                  sum += e;
                  rawv[j] = __float_as_uint(e);
                }
              }
              tmem_st32(taddr + (uint32_t)c0, rawv);
            }
          }
          tmem_st_wait();
        }
        sum = exchange(1, sum, false);
        const float inv = 1.f / sum;
        if (*abort_flag) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        // pass 3: normalised weights of this warp's chunks: live ones into this part's chunk buffer (source of the store to
        // HBM and A operand of O += P_c V_c), chunks wholly beyond the tile's causal limit straight from the zero box
        const int row0 = qt * 128 + q * 32;
        const uint32_t box = sP + (uint32_t)part * kPBufBytes + (uint32_t)q * 4096u;        // this warp's 32 rows of the buffer
        const uint32_t rowaddr = box + (uint32_t)lane * 128u;
        const uint32_t swz = (uint32_t)(lane & 7);
        for (int c = part; c < nc && ok; c += 4) {
          if (c >= live) {
            if (lane == 0) tma_store_4d(&map_p, sZero, c * 64, row0, h, b);
            continue;
          }
          // the values first (tensor-memory reads and arithmetic depend on nobody) ...
          uint32_t pk[32];
          if (c * 64 + 64 <= lim_warp) {
            uint32_t rawv[64];
            tmem_ld32(taddr + (uint32_t)(c * 64), rawv);
            tmem_ld32(taddr + (uint32_t)(c * 64) + 32u, rawv + 32);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) pk[j] = pack2(__uint_as_float(rawv[2 * j]) * inv, __uint_as_float(rawv[2 * j + 1]) * inv);
          } else {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              const int c0 = c * 64 + hh * 32;
              if (c0 < lim_warp) {
                uint32_t rawv[32];
                tmem_ld32(taddr + (uint32_t)c0, rawv);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[hh * 16 + j] = pack2(__uint_as_float(rawv[2 * j]) * inv, __uint_as_float(rawv[2 * j + 1]) * inv);
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[hh * 16 + j] = 0u;
              }
            }
          }
          // ... then the box: free when this warp's previous store from it has read it and the MMAs that read the buffer's
          // previous contents have retired
          {
            int w_ok = 1;
            if (lane == 0) {
              asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
              w_ok = mb_wait(bar(13 + part), (pu & 1u) ^ 1u, 0x922, abort_flag) ? 1 : 0;
            }
            w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
            if (!w_ok) { ok = false; break; }
          }
#pragma unroll
          for (int pc = 0; pc < 8; ++pc)
            sts_v4(rowaddr + ((((uint32_t)pc) ^ swz) << 4), pk[pc * 4], pk[pc * 4 + 1], pk[pc * 4 + 2], pk[pc * 4 + 3]);
          fence_before();
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            mb_arrive(bar(9 + part));                                  // one of the four quarter boxes of the chunk is in place: the MMAs may read it
            tma_store_4d(&map_p, box, c * 64, row0, h, b);             // ... and so does the store (both only read)
          }
          ++pu;
        }
        ok = __all_sync(0xffffffffu, ok);
        // the part-0 warps read O (64 columns, accumulated over the first chunk's columns) and write it out
        if (part == 0 && ok) {
          ok = wait_all(7, (uint32_t)tile_seq & 1u, 0x923);
          fence_after();
          if (ok) {
            uint32_t r0[32], r1[32];
            tmem_ld32(taddr, r0);
            tmem_ld32(taddr + 32u, r1);
            tmem_ld_wait();
            uint4* dst = reinterpret_cast<uint4*>(a.o + (((long long)b * L + row) * a.H + h) * 64);
#pragma unroll
            for (int qq = 0; qq < 4; ++qq)
              dst[qq] = make_uint4(pack2(__uint_as_float(r0[qq * 8]), __uint_as_float(r0[qq * 8 + 1])), pack2(__uint_as_float(r0[qq * 8 + 2]), __uint_as_float(r0[qq * 8 + 3])),
                                   pack2(__uint_as_float(r0[qq * 8 + 4]), __uint_as_float(r0[qq * 8 + 5])), pack2(__uint_as_float(r0[qq * 8 + 6]), __uint_as_float(r0[qq * 8 + 7])));
#pragma unroll
            for (int qq = 0; qq < 4; ++qq)
              dst[4 + qq] = make_uint4(pack2(__uint_as_float(r1[qq * 8]), __uint_as_float(r1[qq * 8 + 1])), pack2(__uint_as_float(r1[qq * 8 + 2]), __uint_as_float(r1[qq * 8 + 3])),
                                       pack2(__uint_as_float(r1[qq * 8 + 4]), __uint_as_float(r1[qq * 8 + 5])), pack2(__uint_as_float(r1[qq * 8 + 6]), __uint_as_float(r1[qq * 8 + 7])));
            fence_before();
            __syncwarp();
            if (lane == 0) mb_arrive(bar(8));
          }
        }
      }
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");      // the stores of the weights have landed
  }

  // ------------------------------- teardown --------------------------------------
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);      // copies and MMAs in flight get time to land
  }
  fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encoder() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// bf16 tensor [d3][d2][d1][d0] (d0 contiguous) as a 4-d tensor map with 128B swizzle; strides in elements
mtf_status map4(CUtensorMap* m, const void* base, const int64_t dims[4], const int64_t strides[3], int box0, int box1) {
  EncodeTiledFn enc = encoder();
  if (!enc) return mtf::fail(MTF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  cuuint64_t d[4] = {(cuuint64_t)dims[0], (cuuint64_t)dims[1], (cuuint64_t)dims[2], (cuuint64_t)dims[3]};
  cuuint64_t s[3] = {(cuuint64_t)strides[0] * 2, (cuuint64_t)strides[1] * 2, (cuuint64_t)strides[2] * 2};
  cuuint32_t box[4] = {(cuuint32_t)box0, (cuuint32_t)box1, 1, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), d, s, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return mtf::fail(MTF_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
  return MTF_OK;
}

}  // namespace

namespace mtf {

bool attention_fused_supported(int64_t L, int64_t d_k, int64_t d_v) { return d_k == 64 && d_v == 64 && L % 128 == 0 && L >= 128 && L <= kMaxL; }

// q, kk [B, L, H, 64]; vv [B, L, H, 64]; weights [B, H, L, L]; o [B, L, H, 64]; all bf16, dense, 16-byte aligned device pointers
mtf_status launch_attention_fwd_fused(const void* q, const void* kk, const void* vv, void* weights, void* o, int64_t B, int64_t H, int64_t L, float scale,
                                      int causal, void* stream) {
  if (!attention_fused_supported(L, 64, 64)) return fail(MTF_ERR_UNSUPPORTED, "fused attention: length %lld", (long long)L);
  if (!(scale > 0.f)) return fail(MTF_ERR_UNSUPPORTED, "fused attention needs a positive scale");
  for (const void* p : {q, kk, vv, (const void*)weights, (const void*)o})
    if (!p || (reinterpret_cast<uintptr_t>(p) & 15)) return fail(MTF_ERR_INVALID_ARG, "fused attention: NULL or misaligned tensor");
  if (B * H <= 0) return MTF_OK;
  CUtensorMap mq, mk, mv, mp;
  const int64_t qd[4] = {64, L, H, B}, qs[3] = {H * 64, 64, L * H * 64};
  const int64_t pd[4] = {L, L, H, B}, ps[3] = {L, L * L, H * L * L};
  mtf_status st;
  if ((st = map4(&mq, q, qd, qs, 64, 128)) != MTF_OK || (st = map4(&mk, kk, qd, qs, 64, 128)) != MTF_OK || (st = map4(&mv, vv, qd, qs, 64, 64)) != MTF_OK ||
      (st = map4(&mp, weights, pd, ps, 64, 32)) != MTF_OK)
    return st;
  AttArgs a;
  a.B = (int)B; a.H = (int)H; a.L = (int)L; a.causal = causal ? 1 : 0; a.scale = scale;
  a.o = reinterpret_cast<__nv_bfloat16*>(o);
  a.units = B * H;
  const size_t smem = 1024 + kQBytes + (size_t)L * 256 + kPBufs * kPBufBytes + 4096 + 2 * kSoftmaxWarps * 32 * 4 + 24 * 8 + 64;
  cudaError_t e = cudaFuncSetAttribute(attention_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  const long long grid = std::min<long long>(a.units * (L / 128), device_sm_count());
  cfg.gridDim = dim3((unsigned)grid, 1, 1); cfg.blockDim = dim3(kThreads, 1, 1); cfg.dynamicSmemBytes = smem; cfg.stream = (cudaStream_t)stream;
  cfg.attrs = at; cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, attention_fwd_kernel, mq, mk, mv, mp, a);
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "attention_fwd_kernel: %s", cudaGetErrorString(e));
  count_launch();
  return MTF_OK;
}

mtf_status read_attention_status(int* code) {
  int v = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&v, g_att_status, sizeof(int));
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemcpyFromSymbol: %s", cudaGetErrorString(e));
  if (v) { int z = 0; cudaMemcpyToSymbol(g_att_status, &z, sizeof(int)); }
  *code = v;
  return MTF_OK;
}

}  // namespace mtf
