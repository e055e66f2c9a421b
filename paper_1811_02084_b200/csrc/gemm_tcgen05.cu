// Grouped bf16 contraction on the 5th-generation tensor cores (sm_100a): the per-slice local einsum
// of Section 6 for every virtual processor of a call in ONE persistent launch, with the sum over a
// reduce group (the paper's Allreduce within a mesh group) fused in:
//   CHAINED   - the worker that owns an output tile runs the K loops of the group's slices back to back
//               (ascending processor order) into one TMEM accumulator;
//   WORKSPACE - every (tile, slice) pair is its own work item; all but the last to arrive leave an fp32
//               fragment in the workspace, the last one adds them in ascending processor order.
// Component-wise work (scale, bias, relu, relu mask, residual, cast), a fused column sum, and for
// attention a whole-row softmax (forward and backward) are applied on the way out.  One launch can
// also sum up to three operand pairs into one accumulator, or run up to three independent problems
// of one shape.
//
// Structure of a CTA (320 threads, one CTA per SM, persistent over work items; by default two CTAs
// form a pair that owns a 256-row tile through tcgen05 cta_group::2):
//   warp 0   : TMA producer   - cp.async.bulk.tensor loads (128B swizzle) into a shared-memory ring
//                               (16 KB of A plus this CTA's part of B per stage, as many stages as fit)
//   warp 1   : MMA issuer     - tcgen05.mma kind::f16 (bf16 x bf16 -> fp32), accumulators in TMEM,
//                               two 128 x 256 accumulators so the epilogue of tile i overlaps tile i+1
//                               (one 128 x 512 accumulator for the wide tiles)
//   warps 2-9: epilogue       - two warps per TMEM lane quarter, alternate 64-column boxes: tcgen05.ld,
//                               the fused stages, 32-row x 128-byte swizzled staging boxes, TMA stores
// Every wait is bounded: after ~2 s it records a code in the device status word, raises a CTA-wide
// abort flag, and all roles fall through to the common teardown (TMEM is freed).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <atomic>
#include <mutex>

#include "mtf_internal.h"

// MTF_CLUSTER_SHARE: defined only by a header that the optional single-GPU build force-includes
// (operand tiles shared between the CTA pairs of a cluster).  The regular library is compiled
// without that header; nothing in this file issues or names such a load.

namespace {

constexpr int BM = 128;
constexpr int kEpilogueWarps = 8;                  // two per TMEM lane quarter, interleaved over the column boxes
constexpr int BK = 64;
constexpr int kMaxBN = 256;
constexpr int kAStageBytes = BM * BK * 2;        // 16 KB
constexpr int kBStageBytes = kMaxBN * BK * 2;    // 32 KB (a CTA of a pair stages half of it)
constexpr int kRingBytes = 5 * (kAStageBytes + kBStageBytes / 2);   // pairs: 5 x (16 KB + 16 KB); single CTAs: 3 x 48 KB fit too
constexpr int kStagingBytes = kEpilogueWarps * 2 * 4096;   // per epilogue warp: two 32-row x 128-byte boxes for TMA stores
constexpr int kMaxStages = 8;                      // ring slots with barriers; a launch uses as many as fit its stage size
constexpr int kSchedSlots = 4;                      // ring of drawn tile numbers that a CTA's roles read in turn
constexpr int kSmemBytes = kRingBytes + kStagingBytes + 1024 /*alignment slack*/ + 320 /*barriers*/ + 96 /*drawn tiles: 2 x 4 barriers, 4 numbers*/;
constexpr int kThreads = 64 + 32 * kEpilogueWarps;
constexpr int kTmemCols = 512;
constexpr long long kTimeoutCycles = 4000000000LL;

__device__ int g_status = 0;
// Testing hooks (mtf_debug_wait_test): the limit of the bounded waits in cycles, and a switch that makes the MMA
// issuer leave out the "accumulator complete" signal of its first tile, so that the epilogue's wait for it runs out.
__device__ long long g_wait_limit = kTimeoutCycles;
__device__ int g_skip_first_commit = 0;

// Division by a run-time constant as a multiply-high and a shift (exact for dividends below 2^31):
// the tile decoder runs once per tile in every warp role and 64-bit divisions made it cost more
// instructions than a tile's whole epilogue.
struct FastDiv {
  uint32_t d, mul, shr;
};
static FastDiv make_fastdiv(long long divisor) {
  FastDiv f;
  f.d = (uint32_t)(divisor < 1 ? 1 : divisor);
  f.mul = 0; f.shr = 0;
  if (f.d > 1) {
    uint32_t l = 0;
    while ((1ull << l) < f.d) ++l;                    // smallest l with 2^l >= d
    const unsigned p = 31 + l;
    f.mul = (uint32_t)(((1ull << p) + f.d - 1) / f.d);
    f.shr = p - 32;
  }
  return f;
}
__device__ __forceinline__ uint32_t fd_div(uint32_t n, const FastDiv& f) { return f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr); }
__device__ __forceinline__ uint32_t fd_divmod(uint32_t n, const FastDiv& f, uint32_t* rem) {
  const uint32_t q = fd_div(n, f);
  *rem = n - q * f.d;
  return q;
}

struct TcArgs {
  int M, N, K;
  int sm, sn, sk;
  int Ms, Ns, Ks;
  int n_outer;
  int outer_local[3];      // extent of each outer dim inside one slice
  int outer_split[3];
  long long outer_sC[3];
  int a_mn_major, b_mn_major;
  int block_n;
  long long ldc;
  int k_sliced;            // walk K slice by slice (slice length is a multiple of BK)
  int reduce_mode;
  int m_tiles, n_tiles;    // per slice
  int n_fastest;           // tile order inside a slice: 1 = walk the n tiles of one m tile first
  long long tiles_per_slice, total_tiles, total_work;
  int balanced;            // workers take equal contiguous ranges of (tile, k-block) units instead of whole tiles
  int late_wait;           // programmatic dependent launch: wait for the previous launch at the end instead of the start
  unsigned* sched;         // not NULL: the workers draw their tiles from this counter pair (next ticket, workers done) instead of
                           // taking every W-th one; zero before the launch, zero again when its last worker has finished
  int reverse;             // walk the tiles from the last to the first (see launch_tc)
  int n_stages, stage_bytes;   // operand ring: 16 KB of A plus this CTA's part of B per stage, as many stages as fit
  int kb_tile;             // k-blocks of one whole tile (all terms)
  int softmax_causal;      // row-softmax epilogue: columns beyond the row's own position are masked out
  int n_groups;            // grouped launch: n_groups (1..3) independent problems of identical shape, tiles of problem g follow those of g - 1
  void* C_group[2];        // outputs of problems 1 and 2
  int n_terms;             // sum of n_terms products A_i . B_i of identical shape in one accumulator (1..3)
  int kb_term;             // k-blocks of one term
  int slots;               // partial-tile slots per tile in the workspace (sk, or 2 when balanced)
  void* C;
  int c_bf16;
  const void* bias;
  int bias_bf16, bias_along_m;
  const void* mask;
  int mask_bf16;
  int mask_tma;            // bf16 mask boxes are loaded by TMA into the output staging buffers (bf16 output only)
  int resid_tma;           // residual boxes (same type as the output) are loaded the same way when there is no mask
  const void* resid;
  int resid_bf16;
  float scale;
  int relu;
  float2* lse_partial;     // EPI_ROW_LSE_BF16: [row][lse_parts] (maximum, sum of exp(value - maximum)) of the row's stored values in every column part
  int lse_parts;           // column parts per row: slices along N x tiles per slice x 2 warps
  float* rsum;             // fused reduce_sum over M of the epilogue value (fp32, pre-zeroed), indexed by n
  float* rsum_partial;     // not NULL: every 32-row group leaves its column sums here ([row group][N]) instead of adding them to rsum with
                           // atomics; a finishing launch adds the groups up in index order, so the sums repeat bit for bit
  float* ws_partials;
  unsigned* ws_counters;     // per (tile, 32-row group, column part): arrivals, then as many again: fragments written
  long long ws_ncounters;
  FastDiv fd_tiles_per_slice, fd_n_tiles, fd_m_tiles, fd_outer_local[3], fd_sn, fd_sm, fd_outer_split[3], fd_sk;
};

// Operand maps of the second and third product of a multi-term launch, or of the second and third
// problem of a grouped launch (A_1, B_1, A_2, B_2).
struct ExtraMaps {
  CUtensorMap m[4];
  CUtensorMap c[2];       // grouped launch: the outputs of problems 1 and 2
};

struct Tile {
  int m0, m_end, n0, n_end;
  int o[3];
  long long c_off;         // element offset of the outer coordinates in C
  long long row_id;        // index of the tile's block of rows among all blocks of rows of the launch (every index but the n tile's)
};

__device__ __forceinline__ Tile decode_tile(const TcArgs& a, long long tile, int tile_rows, int tile_cols) {
  Tile r;
  uint32_t w, rem;
  uint32_t slice = fd_divmod((uint32_t)tile, a.fd_tiles_per_slice, &w);
  uint32_t mt, nt;
  if (a.n_fastest) { w = fd_divmod(w, a.fd_n_tiles, &nt); w = fd_divmod(w, a.fd_m_tiles, &mt); }
  else { w = fd_divmod(w, a.fd_m_tiles, &mt); w = fd_divmod(w, a.fd_n_tiles, &nt); }
  int ol[3] = {0, 0, 0};
  for (int j = a.n_outer - 1; j >= 0; --j) { w = fd_divmod(w, a.fd_outer_local[j], &rem); ol[j] = (int)rem; }
  uint32_t in, im;
  slice = fd_divmod(slice, a.fd_sn, &in);
  slice = fd_divmod(slice, a.fd_sm, &im);
  r.c_off = 0;
  r.o[0] = r.o[1] = r.o[2] = 0;
  long long so_lin = slice, ol_lin = 0;      // (what is left of `slice` is the linear index of the outer split coordinates)
  for (int j = 0; j < a.n_outer; ++j) ol_lin = ol_lin * a.outer_local[j] + ol[j];
  for (int j = a.n_outer - 1; j >= 0; --j) {
    slice = fd_divmod(slice, a.fd_outer_split[j], &rem);
    r.o[j] = (int)rem * a.outer_local[j] + ol[j];
    r.c_off += (long long)r.o[j] * a.outer_sC[j];
  }
  long long OL = 1;
  for (int j = 0; j < a.n_outer; ++j) OL *= a.outer_local[j];
  r.row_id = ((so_lin * a.sm + im) * OL + ol_lin) * a.m_tiles + mt;
  r.m0 = (int)im * a.Ms + (int)mt * tile_rows;
  r.m_end = ((int)im + 1) * a.Ms;
  r.n0 = (int)in * a.Ns + (int)nt * tile_cols;
  r.n_end = ((int)in + 1) * a.Ns;
  return r;
}

// One piece of work for a worker (a CTA, a pair, or a cluster of pairs): k-blocks [kb_begin,
// kb_begin + kb_count) of one output tile.  nfrag > 1: the tile is shared by nfrag workers; this is
// fragment `frag`, it leaves through the workspace and whoever arrives last adds the fragments in order.
struct Seg {
  long long tile;
  int kb_begin, kb_count, frag, nfrag;
  int group;               // problem of a grouped launch
};

// The sequence of segments of worker `w` of `W`.  Three schedules:
//   whole tiles, round robin (tile = w, w + W, ...);
//   WORKSPACE reduce mode: (tile, slice of the reduce group) pairs, round robin;
//   balanced: the (tile, k-block) units are numbered tile-major and cut into W equal contiguous
//   ranges, so that a last, partly filled wave of tiles does not leave SMs idle.  A tile that
//   straddles a range boundary becomes two fragments.
struct SegIter {
  const TcArgs& a;
  long long w, W, work, u, u_end, total_units;
  int kb_per_slice;
  __device__ SegIter(const TcArgs& args, long long worker, long long workers) : a(args), w(worker), W(workers), work(worker) {
    kb_per_slice = a.Ks / BK;
    total_units = a.total_tiles * a.kb_tile;
    u = a.balanced ? (w * total_units) / W : 0;
    u_end = a.balanced ? ((w + 1) * total_units) / W : 0;
  }
  __device__ long long owner(long long unit) const { return ((unit + 1) * W - 1) / total_units; }
  __device__ bool next(Seg& s) {
    s.group = 0;
    if (a.balanced) {
      if (u >= u_end) return false;
      s.tile = u / a.kb_tile;
      s.kb_begin = (int)(u - s.tile * a.kb_tile);
      const long long tile_end = (s.tile + 1) * a.kb_tile;
      const long long e = u_end < tile_end ? u_end : tile_end;
      s.kb_count = (int)(e - u);
      const long long first = owner(s.tile * a.kb_tile), last = owner(tile_end - 1);
      s.nfrag = (int)(last - first + 1);
      s.frag = (int)(w - first);
      u = e;
      return true;
    }
    if (work >= a.total_work) return false;
    if (a.reduce_mode == MTF_REDUCE_WORKSPACE) {
      uint32_t frag;
      s.tile = fd_divmod((uint32_t)work, a.fd_sk, &frag);
      s.frag = (int)frag;
      s.nfrag = a.sk;
      s.kb_begin = s.frag * kb_per_slice;
      s.kb_count = kb_per_slice;
    } else {
      long long w2 = a.reverse ? a.total_work - 1 - work : work;
      if (a.n_groups > 1) { s.group = (int)(w2 / a.total_tiles); w2 -= (long long)s.group * a.total_tiles; }
      s.tile = w2;
      s.frag = 0;
      s.nfrag = 1;
      s.kb_begin = 0;
      s.kb_count = a.kb_tile;
    }
    work += W;
    return true;
  }
  // the same for a tile number drawn from the launch's counter (whole tiles only)
  __device__ bool take(Seg& s, long long drawn_work) {
    work = drawn_work;
    return next(s);
  }
};

// ---- PTX wrappers -----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false after the time limit (recording `code`) or when another role aborted.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, int code, volatile int* abort_flag) {
  const long long t0 = clock64();
  while (true) {
    for (int i = 0; i < 128; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > g_wait_limit) {
      atomicCAS(&g_status, 0, code);
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int code, volatile int* abort_flag) {
  for (int i = 0; i < 32; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, code, abort_flag);
}

// Warp-wide wait for the epilogue warps: lane 0 polls with a pause between polls (so that eight
// waiting warps do not take issue slots from the MMA and TMA threads), the others sleep at the
// warp barrier and then confirm the phase themselves.  Same time limit and abort rule as mbar_wait.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, int code, volatile int* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) {
    if (!mbar_try_wait(bar, parity)) {
      const long long t0 = clock64();
      while (true) {
        __nanosleep(100);
        if (mbar_try_wait(bar, parity)) break;
        if (*abort_flag) { ok = 0; break; }
        if (clock64() - t0 > g_wait_limit) {
          atomicCAS(&g_status, 0, code);
          *abort_flag = 1;
          ok = 0;
          break;
        }
      }
    }
  }
  ok = __shfl_sync(0xffffffffu, ok, 0);
  if (!ok) return false;
  return mbar_wait(bar, parity, code, abort_flag);
}

// kPair: the completion may count on the partner CTA's barrier (cta_group::2 form); never multicast.
template <bool kPair>
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  if (kPair)
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
  else
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}

__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Arrive on the barrier at the same offset in the even CTA of the pair (own barrier when !kPair).
template <bool kPair>
__device__ __forceinline__ void mbar_arrive_pair(uint32_t bar, uint32_t leader_rank) {
  if (kPair)
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}"
        ::"r"(bar), "r"(leader_rank) : "memory");
  else
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Drawn tiles (TcArgs::sched): the producer thread of a worker's first CTA draws tickets from the launch's counter and
// publishes each tile number in a small ring in the shared memory of the worker's CTAs; every other role reads the ring
// in order (its n-th read is slot n mod kSchedSlots).  Slot s: full barrier at ring + 8 s (one arrival: the drawing
// thread), empty barrier at ring + 32 + 8 s in the first CTA (one arrival per reading role of every CTA), number at
// ring + 64 + 4 s.  A number >= total_work ends the sequence; the drawing thread then counts its worker as done, and
// the last worker of the launch clears the counter pair for the next launch that is given it.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool sched_wait(uint32_t bar, uint32_t parity, int code, volatile int* abort_flag) {
  const long long t0 = clock64();
  while (!mbar_try_wait_cluster(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > g_wait_limit) { atomicCAS(&g_status, 0, code); *abort_flag = 1; return false; }
  }
  return true;
}
// The drawing thread: number `t` into slot seq mod kSchedSlots of every CTA of the worker.
__device__ __forceinline__ bool sched_publish(uint32_t ring, uint32_t seq, unsigned t, int n_ctas, volatile int* abort_flag) {
  const uint32_t slot = seq % kSchedSlots, phase = (seq / kSchedSlots) & 1u;
  const uint32_t full = ring + 8u * slot, empty = ring + 32u + 8u * slot, num = ring + 64u + 4u * slot;
  if (seq >= (uint32_t)kSchedSlots && !sched_wait(empty, phase ^ 1u, 0x900 + (int)slot, abort_flag)) return false;
  if (n_ctas == 1) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(num), "r"(t) : "memory");
    asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(full) : "memory");
  } else {
    for (int c = 0; c < n_ctas; ++c)
      asm volatile(
          "{\n\t.reg .b32 ra, rb;\n\t"
          "mapa.shared::cluster.u32 ra, %0, %2;\n\t"
          "mapa.shared::cluster.u32 rb, %1, %2;\n\t"
          "st.shared::cluster.u32 [ra], %3;\n\t"
          "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [rb];\n\t}"
          ::"r"(num), "r"(full), "r"(c), "r"(t) : "memory");
  }
  return true;
}
// A reading role's seq-th number; `arrive`: this thread hands the slot back (one thread per role).
template <bool kPair>
__device__ __forceinline__ bool sched_read(uint32_t ring, uint32_t seq, bool warp_role, bool arrive, volatile int* abort_flag, unsigned* t) {
  const uint32_t slot = seq % kSchedSlots, phase = (seq / kSchedSlots) & 1u;
  const uint32_t full = ring + 8u * slot, empty = ring + 32u + 8u * slot, num = ring + 64u + 4u * slot;
  if (!sched_wait(full, phase, 0x910 + (int)slot, abort_flag)) return false;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(*t) : "r"(num) : "memory");
  if (warp_role) __syncwarp();
  if (arrive) mbar_arrive_pair<kPair>(empty, 0u);
  return true;
}
// The drawing thread has its worker's last ticket: count the worker as done; the last one clears the pair.
__device__ __forceinline__ void sched_worker_done(unsigned* sched, unsigned workers) {
  __threadfence();
  if (atomicAdd(sched + 1, 1u) == workers - 1u) {
    sched[0] = 0u; sched[1] = 0u;
    __threadfence();
  }
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

template <bool kPair>
__device__ __forceinline__ void umma_bf16(uint32_t tmem_c, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  if (kPair)
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_c), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_c), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives on `bar` when every MMA issued so far has retired; for a pair, on the barrier at that
// offset in both CTAs (completion multicast, not a load).
template <bool kPair>
__device__ __forceinline__ void umma_commit(uint32_t bar, uint16_t cta_mask) {
  if (kPair) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(cta_mask) : "memory");
  } else {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
  }
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
      : "r"(taddr)
      : "memory");
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
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor for a 128B-swizzled bf16 tile (descriptor version 1).
//   K-major  (rows of 64 K-elements = 128 B; 8-row groups 1024 B apart): LBO unused (1), SBO = 1024 B
//   MN-major (rows of 64 M/N-elements = 128 B, one row per k; 64-wide column blocks 8 KB apart):
//             LBO = 8192 B (next 64 M/N), SBO = 1024 B (next 8 k)
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, int mn_major) {
  const uint64_t lbo = mn_major ? (8192u >> 4) : 1u;
  const uint64_t sbo = 1024u >> 4;
  return (uint64_t)((addr & 0x3FFFF) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t lo16) { return __uint_as_float(lo16 << 16); }

// Sum over the 32 lanes (rows) of each of 32 columns: lane j ends with column j's total.  Each step
// halves the number of values a lane holds and exchanges the other half with its partner.
__device__ __forceinline__ float warp_column_sums(float* v, int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < off; ++i) {
      const float send = upper ? v[i] : v[i + off];
      const float keep = upper ? v[i + off] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  return v[0];
}

__device__ __forceinline__ void unpack_bf16x8(const uint4& m, float* f) {
  const uint32_t w[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    f[2 * e] = bf16_bits_to_float(w[e] & 0xFFFFu);
    f[2 * e + 1] = bf16_bits_to_float(w[e] >> 16);
  }
}

// Which component-wise stages a launch runs.  EPI_GENERIC reads them from the arguments; the other
// kinds fix them at compile time, so that the common epilogues carry no branches on them and need
// far fewer registers and instructions per chunk.
enum { EPI_GENERIC = 0, EPI_PLAIN_BF16 = 1, EPI_PLAIN_F32 = 2, EPI_BIAS_RELU_BF16 = 3, EPI_MASK_RSUM_BF16 = 4, EPI_ROW_SOFTMAX = 5, EPI_ROW_SOFTMAX_BWD = 6,
       EPI_ROW_LSE_BF16 = 7 /* plain bf16 result + per row and column part the maximum and the sum of exponentials of what was stored */, EPI_KINDS = 8 };
struct EpiFlags {
  bool scale, bias, bias_m, relu, relu_in_pack, mask, mask_bf16, mask_tma, resid, resid_tma, rsum, c_bf16, shared_tiles;
};
template <int EPI>
__device__ __forceinline__ EpiFlags epi_flags(const TcArgs& a) {
  EpiFlags f;
  if (EPI == EPI_GENERIC) {
    f.scale = a.scale != 1.f; f.bias = a.bias != nullptr; f.bias_m = a.bias_along_m != 0; f.relu = a.relu != 0;
    f.mask = a.mask != nullptr; f.mask_bf16 = a.mask_bf16 != 0; f.mask_tma = a.mask_tma != 0; f.resid = a.resid != nullptr; f.resid_tma = a.resid_tma != 0;
    f.rsum = a.rsum != nullptr; f.c_bf16 = a.c_bf16 != 0; f.shared_tiles = true; f.relu_in_pack = false;
  } else {
    f.scale = false; f.bias = EPI == EPI_BIAS_RELU_BF16; f.bias_m = false; f.relu = EPI == EPI_BIAS_RELU_BF16;
    f.mask = f.mask_bf16 = f.mask_tma = f.rsum = EPI == EPI_MASK_RSUM_BF16; f.resid = f.resid_tma = false;
    f.c_bf16 = EPI != EPI_PLAIN_F32;
    f.relu_in_pack = EPI == EPI_BIAS_RELU_BF16;      // relu is the last stage there: it rides in the conversion to bf16
    if (EPI == EPI_ROW_SOFTMAX) f.scale = true;
    if (EPI == EPI_PLAIN_BF16 || EPI == EPI_PLAIN_F32) f.scale = a.scale != 1.f;      // one uniform branch: s . (a . b) stays on the fast kinds
    if (EPI == EPI_ROW_SOFTMAX_BWD) f.mask = f.mask_bf16 = true;      // the weights P arrive like a mask, by TMA
    f.shared_tiles = EPI == EPI_PLAIN_BF16 || EPI == EPI_PLAIN_F32;     // the other fixed kinds never split a tile
  }
  return f;
}

// Fetch the relu mask of one 32-column chunk of this thread's row (bf16 mask: four 16-byte loads).
__device__ __forceinline__ void mask_fetch(const TcArgs& a, long long off, bool on, int n_valid, uint4* mk) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    mk[q] = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);   // 1.0: keeps the value
    if (on && q * 8 < n_valid) mk[q] = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.mask) + off + q * 8);
  }
}

// The component-wise stages on one 32-column chunk of one row, in registers (Section 6, Section 7):
// scale, bias (broadcast), relu, relu mask; the value then feeds the fused reduce_sum; residual last.
//   bias_lane : bias of column (n_first + lane), handed to every lane by shuffle (bias along n)
//   bias_row  : bias of this thread's row (bias along m)
// Keeps a (b) where the lower (upper) bf16 of m is greater than zero, else makes it zero: one packed
// compare for two mask values (ordered: a NaN mask keeps nothing, like the scalar comparison).
__device__ __forceinline__ void keep_where_positive(uint32_t m, float& a, float& b) {
  asm("{\n\t.reg .pred p, q;\n\t"
      "setp.gt.bf16x2 p|q, %2, %3;\n\t"
      "selp.f32 %0, %0, 0f00000000, p;\n\t"
      "selp.f32 %1, %1, 0f00000000, q;\n\t}"
      : "+f"(a), "+f"(b) : "r"(m), "r"(0u));
}

__device__ __forceinline__ void epilogue_math(const TcArgs& a, const EpiFlags& f, float* v, float bias_lane, float bias_row,
                                              const uint4* mk, long long off, bool live, int n_valid) {
  if (f.scale) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] *= a.scale;
  }
  if (f.bias) {
    if (f.bias_m) {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += bias_row;
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += __shfl_sync(0xffffffffu, bias_lane, j);
    }
  }
  if (f.relu && !f.relu_in_pack) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
  }
  if (f.mask) {
    if (f.mask_bf16) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t w[4] = {mk[q].x, mk[q].y, mk[q].z, mk[q].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) keep_where_positive(w[e], v[q * 8 + 2 * e], v[q * 8 + 2 * e + 1]);
      }
    } else if (live) {
      const float* mp = reinterpret_cast<const float*>(a.mask) + off;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j < n_valid && !(mp[j] > 0.f)) v[j] = 0.f;
    }
  }
}

__device__ __forceinline__ void epilogue_residual(const TcArgs& a, const EpiFlags& f, float* v, long long off, bool live, int n_valid) {
  if (!f.resid || !live) return;
  if (a.resid_bf16) {
    const uint4* rp = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.resid) + off);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (q * 8 < n_valid) {
        float f[8];
        unpack_bf16x8(rp[q], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) v[q * 8 + e] += f[e];
      }
  } else {
    const float* rp = reinterpret_cast<const float*>(a.resid) + off;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < n_valid) v[j] += rp[j];
  }
}

__device__ __forceinline__ uint32_t pack_bf16x2_relu(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h2);
}

// 16-byte stores of one chunk straight from registers (ragged tiles and the workspace mode).
__device__ __forceinline__ uint32_t pack_out(const EpiFlags& f, float lo, float hi) {
  return f.relu_in_pack ? pack_bf16x2_relu(lo, hi) : pack_bf16x2(lo, hi);
}

__device__ __forceinline__ void store_direct(const TcArgs& a, const EpiFlags& f, const float* v, long long off, int n_valid, void* c_base = nullptr) {
  if (!c_base) c_base = a.C;
  if (f.c_bf16) {
    uint4* cp = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(c_base) + off);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (q * 8 < n_valid)
        cp[q] = make_uint4(pack_out(f, v[q * 8], v[q * 8 + 1]), pack_out(f, v[q * 8 + 2], v[q * 8 + 3]),
                           pack_out(f, v[q * 8 + 4], v[q * 8 + 5]), pack_out(f, v[q * 8 + 6], v[q * 8 + 7]));
  } else {
    float4* cp = reinterpret_cast<float4*>(reinterpret_cast<float*>(c_base) + off);
#pragma unroll
    for (int q = 0; q < 8; ++q)
      if (q * 4 < n_valid) cp[q] = make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
  }
}

__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 r;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr) : "memory");
  return r;
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

// One chunk of this thread's row into the warp's staging box (32 rows x 128 B, 128B-swizzled as
// the output tensor map expects): 16-byte piece p of row r lives at r*128 + ((p ^ (r & 7)) * 16).
__device__ __forceinline__ void store_staged(const EpiFlags& f, const float* v, uint32_t box, int lane, int half) {
  const uint32_t row = box + (uint32_t)lane * 128u;
  const uint32_t sw = (uint32_t)(lane & 7);
  if (f.c_bf16) {
#pragma unroll
    for (int q = 0; q < 4; ++q)
      st_shared_v4(row + ((((uint32_t)(half * 4 + q)) ^ sw) << 4), pack_out(f, v[q * 8], v[q * 8 + 1]),
                   pack_out(f, v[q * 8 + 2], v[q * 8 + 3]), pack_out(f, v[q * 8 + 4], v[q * 8 + 5]),
                   pack_out(f, v[q * 8 + 6], v[q * 8 + 7]));
  } else {
#pragma unroll
    for (int q = 0; q < 8; ++q)
      st_shared_v4(row + (((uint32_t)q ^ sw) << 4), __float_as_uint(v[q * 4]), __float_as_uint(v[q * 4 + 1]),
                   __float_as_uint(v[q * 4 + 2]), __float_as_uint(v[q * 4 + 3]));
  }
}

__device__ __forceinline__ void tma_store_5d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3, int c4) {
  asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// kPair = false: one CTA owns a 128 x block_n tile (tcgen05 cta_group::1); 3 stages of 48 KB at block_n = 256.
// kPair = true : a cluster of two CTAs owns a 256 x block_n tile (tcgen05 cta_group::2).  Each CTA
//   stages its own 128 rows of A and its own half of the N columns of B (32 KB per stage, 5 stages at block_n = 256),
//   the even CTA of the pair issues every MMA for both, each CTA's TMEM receives its own 128 rows of
//   the result, and each CTA runs the epilogue on its own rows.  Compared with kPair = false a CTA
//   pulls 2/3 of the bytes through L2 per flop and holds 1.5x as many k-blocks in flight.
//   The loads of both CTAs report to the even CTA's "full" barrier; MMA completion is multicast to
//   both CTAs' "empty" and "accumulator full" barriers; the epilogue warps of both CTAs report to
//   the even CTA's "accumulator empty" barrier.  No load uses cluster multicast.
//
// CM x CN > 1 (optional single-GPU build only): a cluster of CM x CN CTA pairs owns a (CM * 256) x
// (CN * block_n) super-tile.  Pairs in one row of the cluster need the same rows of A, pairs in one
// column the same columns of B; each CTA loads only its 1/CN share of its A rows and its 1/CM share
// of its B columns and the load writes it into every CTA that needs it, so a CTA pulls
// 16 KB / CN + 16 KB / CM per k-block through L2 instead of 32 KB.  A stage may be refilled when
// every pair that reads what this CTA writes has retired its MMAs: CM + CN - 1 pair leaders signal
// each CTA's "empty" barrier.
template <bool kPair, int CM, int CN, int EPI, bool kWide, bool kDrawn = false>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_m,
                    const __grid_constant__ CUtensorMap map_w, const __grid_constant__ ExtraMaps extra, const TcArgs a) {
  // kWide (pairs only): the pair owns a 256 x 512 tile, which fills the tensor memory: one accumulator,
  // so a tile's epilogue is not overlapped with the next tile's MMAs, but a CTA pulls 48 KB per
  // k-block through L2 for twice the flops (24 KB per 256 x 256 x 64 instead of 32 KB).  For long K,
  // where the contraction is bound by the L2-to-SM traffic and the exposed epilogue is small.
  static_assert(!kWide || (kPair && CM == 1 && CN == 1), "wide tiles: plain CTA pairs only");
  // The ring has a.n_stages stages of a.stage_bytes (32 KB for a pair with 256-column tiles: 5 stages;
  // 48 KB for wide and single-CTA 256-column tiles: 3 stages; narrower tiles get deeper rings).  The
  // row-softmax kinds leave 2 KB at the end of the ring for the exchange of row statistics.
  const int kStages = a.n_stages;
  const int kStageBytes = a.stage_bytes;
  constexpr int kPairRows = kPair ? 2 * BM : BM;       // rows of C owned by one CTA pair (or single CTA)
  constexpr int kTileRows = kPairRows * CM;            // rows of C owned by a work item
  constexpr bool kCluster = CM * CN > 1;
  static_assert(!kCluster || kPair, "clusters of pairs only");
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte aligned tile ring (the 128B swizzle pattern repeats every 1024 B)
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (tiles_base - raw);
  // after the ring: per epilogue warp two 4 KB staging boxes for the output stores, then the barriers
  const uint32_t staging_base = tiles_base + kRingBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + kRingBytes + kStagingBytes);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty  (S = kMaxStages slots)
  const uint32_t bar_base = staging_base + kStagingBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int i) { return bar_base + 8u * (2 * kMaxStages + i); };
  auto tempty_bar = [&](int i) { return bar_base + 8u * (2 * kMaxStages + 2 + i); };
  // then [2S+4..2S+20): per epilogue warp two barriers for relu-mask boxes loaded into its staging buffers
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 4 + 2 * kEpilogueWarps);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // then the ring of drawn tile numbers (launches with a.sched): 4 full barriers, 4 empty barriers, 4 numbers
  const uint32_t sched_ring = bar_base + 8u * (2 * kMaxStages + 4 + 2 * kEpilogueWarps) + 8u;
  constexpr bool drawn = kDrawn;       // a variant of its own: launches with the fixed tile assignment carry none of this
  static_assert(!kDrawn || !kCluster, "drawn tiles: plain pairs and single CTAs only");

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  constexpr int kClusterCtas = (kPair ? 2 : 1) * CM * CN;
  const int cluster_rank = (int)(blockIdx.x % kClusterCtas);   // 1-D clusters: rank = position in the cluster
  const int cta_rank = kPair ? (cluster_rank & 1) : 0;         // position in the CTA pair
  const int pair_idx = cluster_rank >> 1;                      // which pair of the cluster
  const int pm = pair_idx / CN, pn = pair_idx % CN;            // the pair's row / column in the cluster
  const bool leader = cta_rank == 0;
  const long long work_first = (long long)(blockIdx.x / kClusterCtas);
  const long long work_step = (long long)(gridDim.x / kClusterCtas);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), CM + CN - 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tfull_bar(i), 1); mbar_init(tempty_bar(i), (kPair ? 2 : 1) * kEpilogueWarps); }
    for (int i = 0; i < 2 * kEpilogueWarps; ++i) mbar_init(bar_base + 8u * (2 * kMaxStages + 4 + i), 1);
    for (int i = 0; i < kSchedSlots; ++i) { mbar_init(sched_ring + 8u * i, 1); mbar_init(sched_ring + 32u + 8u * i, (kPair ? 2 : 1) * (1 + kEpilogueWarps)); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
  }
  const uint32_t xchg_base = tiles_base + (uint32_t)(kStages * kStageBytes);     // [2 slots][8 warps][32 lanes] x 8 bytes
  if (EPI == EPI_ROW_SOFTMAX || EPI == EPI_ROW_SOFTMAX_BWD)
    for (int i = threadIdx.x; i < 2 * kEpilogueWarps * 32; i += kThreads)
      asm volatile("st.shared.v2.b32 [%0], {%1, %1};" ::"r"(xchg_base + 8u * i), "r"(0u) : "memory");
  if (warp == 1) {   // TMEM allocation is a warp-wide operation (the same warp of both CTAs of a pair)
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (kPair) cluster_sync();      // the partner's barriers must exist before anything signals them
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Programmatic dependent launch: everything above (barriers, TMEM, tensor-map prefetch) may overlap
  // the tail of the previous kernel on the stream; nothing below touches global memory before that
  // kernel has completed.  The next kernel on the stream may start its own set-up right away.
  // (late_wait: this launch reads and writes nothing that the launch before it on the stream touches, so it
  // starts at once and fills the SMs that launch's last tiles leave idle; it waits for it before exiting
  // instead, so that whatever follows on the stream still sees every earlier launch complete.)
  if (!a.late_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int n_local = kPair ? a.block_n / 2 : a.block_n;       // N columns of B this CTA stages (wide: two runs of 128)
  const uint32_t b_bytes = (uint32_t)n_local * BK * 2;

  if (warp == 0) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      SegIter it(a, work_first, work_step);
      Seg sg;
      // drawn tiles: the first CTA's producer asks for its next ticket a few k-blocks before it has issued the last loads
      // of its tile: early enough to hide the round trip to the counter, late enough that a worker does not hold a tile it
      // will only start much later while other workers run out of work
      uint32_t dseq = 0;
      unsigned pending = 0;
      bool have_pending = false;
      if (drawn && leader) { pending = (unsigned)work_first; have_pending = true; }      // (the first tile needs no ticket: worker w starts with tile w, ticket n is tile W + n)
      auto next_tile = [&]() -> bool {
        if (!drawn) return it.next(sg);
        unsigned t;
        if (leader) {
          if (!have_pending) pending = (unsigned)work_step + atomicAdd(a.sched, 1u);
          have_pending = false;
          t = pending;
          if (!sched_publish(sched_ring, dseq, t, kPair ? 2 : 1, abort_flag)) { ok = false; return false; }
          if ((long long)t >= a.total_work) { sched_worker_done(a.sched, (unsigned)work_step); return false; }
        } else {
          if (!sched_read<kPair>(sched_ring, dseq, false, true, abort_flag, &t)) { ok = false; return false; }
        }
        ++dseq;
        return it.take(sg, (long long)t);
      };
      while (ok && next_tile()) {
        const int kb_first = sg.kb_begin, kb_count = sg.kb_count;
        const Tile tl = decode_tile(a, sg.tile, kTileRows, a.block_n * CN);
        const int m0 = tl.m0 + pm * kPairRows + cta_rank * BM;
        const int n0 = tl.n0 + pn * a.block_n + cta_rank * n_local;
        int term = kb_first / a.kb_term, kt = kb_first - term * a.kb_term;
        for (int kb = 0; kb < kb_count; ++kb) {
          if (drawn && leader && !have_pending && kb == (kb_count > 4 ? kb_count - 4 : 0)) { pending = (unsigned)work_step + atomicAdd(a.sched, 1u); have_pending = true; }
          // slices of the reduce group are walked in ascending order: k0 runs through slice 0's
          // block of K, then slice 1's, ... (the blocks are contiguous in the global tensor); a
          // multi-term launch then goes on with the next product's operands
          const int k0 = kt * BK;
          const int sel = a.n_groups > 1 ? sg.group : term;          // operand pair: the problem of a grouped launch, else the term
          const CUtensorMap* const pa = sel == 0 ? &map_a : &extra.m[2 * (sel - 1)];
          const CUtensorMap* const pb = sel == 0 ? &map_b : &extra.m[2 * (sel - 1) + 1];
          if (++kt == a.kb_term) { kt = 0; ++term; }
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, 0x100 + stage, abort_flag))) break;
          // a pair's loads all count on the even CTA's barrier, which expects both CTAs' bytes
          if (!kPair) mbar_expect_tx(full_bar(stage), kAStageBytes + b_bytes);
          else if (leader) mbar_expect_tx(full_bar(stage), 2u * (kAStageBytes + b_bytes));
          const uint32_t fb = kPair ? (full_bar(stage) & 0xFEFFFFFFu) : full_bar(stage);
          const uint32_t sa = tiles_base + stage * kStageBytes;
          const uint32_t sb = sa + kAStageBytes;
#if defined(MTF_CLUSTER_SHARE)
          if (CN > 1) cluster_share_load_a(sa, pa, fb, pm, pn, CN, cta_rank, a.a_mn_major, BM / CN, m0, k0, tl.o[2], tl.o[1], tl.o[0]);
          else
#endif
          if (a.a_mn_major) {
            tma_load_5d<kPair>(sa, pa, fb, m0, k0, tl.o[2], tl.o[1], tl.o[0]);
            tma_load_5d<kPair>(sa + 8192, pa, fb, m0 + 64, k0, tl.o[2], tl.o[1], tl.o[0]);
          } else {
            tma_load_5d<kPair>(sa, pa, fb, k0, m0, tl.o[2], tl.o[1], tl.o[0]);
          }
#if defined(MTF_CLUSTER_SHARE)
          if (CM > 1) cluster_share_load_b(sb, pb, fb, pm, pn, CM, CN, cta_rank, a.b_mn_major, n_local / CM, n0, k0, tl.o[2], tl.o[1], tl.o[0]);
          else
#endif
          if (kWide) {
            // columns [256 j + 128 rank, + 128) of the tile for MMA j = 0, 1: two runs of 128, 16 KB each
            for (int h2 = 0; h2 < 2; ++h2) {
              const int nh = tl.n0 + 256 * h2 + cta_rank * 128;
              if (a.b_mn_major) {
                tma_load_5d<kPair>(sb + 16384 * h2, pb, fb, nh, k0, tl.o[2], tl.o[1], tl.o[0]);
                tma_load_5d<kPair>(sb + 16384 * h2 + 8192, pb, fb, nh + 64, k0, tl.o[2], tl.o[1], tl.o[0]);
              } else {
                tma_load_5d<kPair>(sb + 16384 * h2, pb, fb, k0, nh, tl.o[2], tl.o[1], tl.o[0]);
              }
            }
          } else if (a.b_mn_major) {
            for (int j = 0; j < n_local / 64; ++j)
              tma_load_5d<kPair>(sb + 8192 * j, pb, fb, n0 + 64 * j, k0, tl.o[2], tl.o[1], tl.o[0]);
          } else {
            tma_load_5d<kPair>(sb, pb, fb, k0, n0, tl.o[2], tl.o[1], tl.o[0]);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (even CTA of a pair only) -------
    if (lane == 0 && leader) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a.a_mn_major << 15) |
                             ((uint32_t)a.b_mn_major << 16) | ((uint32_t)((kWide ? 256 : a.block_n) >> 3) << 17) | ((uint32_t)(kPairRows >> 4) << 24);
      // completion signals: this pair's two CTAs, and every CTA whose loads land in this pair's tiles
      // (the pairs of this pair's cluster row and column)
      const uint16_t pair_mask = (uint16_t)(3u << (2 * pair_idx));
      uint16_t empty_mask = 0;
      for (int i = 0; i < CM; ++i)
        for (int j = 0; j < CN; ++j)
          if (i == pm || j == pn) empty_mask |= (uint16_t)(3u << (2 * (i * CN + j)));
      const uint32_t a_kstep = a.a_mn_major ? 2048u : 32u;   // bytes per 16 k-elements
      const uint32_t b_kstep = a.b_mn_major ? 2048u : 32u;
      int stage = 0;
      uint32_t phase = 0;
      int iter = 0;
      bool ok = true;
      SegIter it(a, work_first, work_step);
      Seg sg;
      auto next_tile = [&]() -> bool {
        if (!drawn) return it.next(sg);
        unsigned t;
        if (!sched_read<kPair>(sched_ring, (uint32_t)iter, false, true, abort_flag, &t)) { ok = false; return false; }
        return it.take(sg, (long long)t);
      };
      for (; ok && next_tile(); ++iter) {
        const int kb_count = sg.kb_count;
        const int acc = kWide ? 0 : (iter & 1);
        const uint32_t acc_phase = kWide ? ((uint32_t)iter & 1u) : ((uint32_t)(iter >> 1) & 1u);
        if (!(ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, 0x200 + acc, abort_flag))) break;
        tcgen05_fence_after();
        const uint32_t tmem_c = tmem_base + (uint32_t)acc * kMaxBN;
        for (int kb = 0; kb < kb_count; ++kb) {
          if (!(ok = mbar_wait(full_bar(stage), phase, 0x300 + stage, abort_flag))) break;
          tcgen05_fence_after();
          const uint32_t sa = tiles_base + stage * kStageBytes;
          const uint32_t sb = sa + kAStageBytes;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = make_smem_desc(sa + k * a_kstep, a.a_mn_major);
            const uint64_t db = make_smem_desc(sb + k * b_kstep, a.b_mn_major);
            umma_bf16<kPair>(tmem_c, da, db, idesc, (kb | k) != 0);
            if (kWide) umma_bf16<kPair>(tmem_c + 256u, da, make_smem_desc(sb + 16384u + k * b_kstep, a.b_mn_major), idesc, (kb | k) != 0);
          }
          umma_commit<kPair>(empty_bar(stage), empty_mask);   // frees the stage in every CTA that writes into this pair's tiles
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok && !(iter == 0 && g_skip_first_commit)) umma_commit<kPair>(tfull_bar(acc), pair_mask);   // accumulator complete (in both CTAs of the pair)
      }
    }
  } else {
    // ------------------------------- epilogue -----------------------------------
    const EpiFlags f = epi_flags<EPI>(a);
    const int q = warp & 3;                        // TMEM lane quarter this warp may read
    const int col_half = (warp - 2) >> 2;          // which of the two warps of this lane quarter
    const uint32_t stg = staging_base + (uint32_t)(warp - 2) * 8192u;      // this warp's two staging boxes
    uint32_t buf = 0;                              // staging box the next output box goes through
    uint32_t mask_phase = 0;                       // bit b: phase of this warp's mask barrier b
    auto mfull_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kMaxStages + 4 + (uint32_t)(warp - 2) * 2 + b); };
    int iter = 0;
    bool ok = true;
    SegIter it(a, work_first, work_step);
    Seg sg;
    auto next_tile = [&]() -> bool {
      if (!drawn) return it.next(sg);
      unsigned t;
      if (!sched_read<kPair>(sched_ring, (uint32_t)iter, true, lane == 0, abort_flag, &t)) { ok = false; return false; }
      return it.take(sg, (long long)t);
    };
    for (; ok && next_tile(); ++iter) {
      const long long t = sg.tile;
      const int ks = sg.frag;
      const bool ws_mode = f.shared_tiles && sg.nfrag > 1;       // this tile is assembled from fragments in the workspace
      Tile tl = decode_tile(a, t, kTileRows, a.block_n * CN);
      tl.m0 += pm * kPairRows;            // this pair's 256 x block_n part of the cluster's super-tile
      tl.n0 += pn * a.block_n;
      const int acc = kWide ? 0 : (iter & 1);
      const uint32_t acc_phase = kWide ? ((uint32_t)iter & 1u) : ((uint32_t)(iter >> 1) & 1u);
      const int pair_row = cta_rank * BM + q * 32 + lane;       // row inside the pair's part of the tile
      const int tile_row = pm * kPairRows + pair_row;            // row inside the work item's tile
      const int row = tl.m0 + pair_row;
      const bool row_ok = row < tl.m_end;
      const long long row_off = tl.c_off + (long long)row * a.ldc;
      // what the epilogue needs from memory is requested before the accumulator is waited for:
      // the tile's bias (lane l keeps columns l, l+32, ...) and the first chunk's relu mask
      const bool bias_n = f.bias && !f.bias_m;
      auto bias_at = [&](int col) -> float {       // bias of one column, 0 outside the slice
        if (!bias_n || col >= tl.n_end) return 0.f;
        return a.bias_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.bias)[col]) : reinterpret_cast<const float*>(a.bias)[col];
      };
      float bias_row = 0.f;
      if (f.bias && f.bias_m && row_ok)
        bias_row = a.bias_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.bias)[row]) : reinterpret_cast<const float*>(a.bias)[row];
      const int row0 = tl.m0 + cta_rank * BM + q * 32;           // first row of this warp
      const bool rows_full = row0 + 32 <= tl.m_end;
      // an epilogue operand that arrives box by box in the staging buffers and is consumed in place:
      // the bf16 relu mask, or the residual
      const bool mask_tma = f.mask_tma && !ws_mode && rows_full;
      const bool resid_tma = f.resid_tma && !ws_mode && rows_full;
      const bool in_tma = (mask_tma || resid_tma) && EPI != EPI_ROW_SOFTMAX_BWD;
      const int box_cols = f.c_bf16 ? 64 : 32;
      // softmax backward: the boxes of P this warp visits (twice: row dot products, then the result);
      // under the causal limit the boxes right of the warp's widest row hold zeros and are not read
      int sb_lim = 0, sb_lim_warp = 0, sb_nbox = 0;
      if (EPI == EPI_ROW_SOFTMAX_BWD) {
        const int ncols = min(a.block_n, tl.n_end - tl.n0);
        sb_lim = a.softmax_causal ? min(ncols, row + 1) : ncols;
        sb_lim_warp = __shfl_sync(0xffffffffu, sb_lim, 31);
        if (rows_full)                     // (a warp is inside its slice with all 32 rows or with none)
          for (int b = col_half * 64; b < sb_lim_warp; b += 128) ++sb_nbox;
        if (sb_nbox > 0 && lane == 0) {
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          mbar_expect_tx(mfull_bar(buf), 4096u);
          tma_load_5d<false>(stg + buf * 4096u, &map_m, mfull_bar(buf), tl.n0 + col_half * 64, row0, tl.o[2], tl.o[1], tl.o[0]);
        }
      }
      if (in_tma && lane == 0) {
        // request the first box into the staging box it will be processed in (free once all but the latest
        // store have been read out); asking for the later boxes to be brought to L2 here measured slower
        if (col_half * box_cols < a.block_n && tl.n0 + col_half * box_cols + box_cols <= tl.n_end) {
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          mbar_expect_tx(mfull_bar(buf), 4096u);
          tma_load_5d<false>(stg + buf * 4096u, &map_m, mfull_bar(buf), tl.n0 + col_half * box_cols, row0, tl.o[2], tl.o[1], tl.o[0]);
        }
      }
      ok = mbar_wait_warp(tfull_bar(acc), acc_phase, 0x400 + acc, abort_flag, lane);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t)acc * kMaxBN + ((uint32_t)(q * 32) << 16);
      if (EPI == EPI_ROW_SOFTMAX_BWD) {
        // The accumulator holds whole rows of dP = do . vv^T; with the weights P of the same rows
        // (64-column boxes by TMA into the staging buffers, one box ahead) the result is
        // dlogits = P (dP - sum_m dP P): a first visit of every box for the row sums, the two warps of
        // a lane quarter exchange their parts, a second visit writes the result over the box and stores it.
        // (exchange slots alternate with the tile, so a warp that runs ahead cannot overwrite what its partner has not read)
        const uint32_t slot_off = (uint32_t)(iter & 1) * (8u * kEpilogueWarps * 32u);
        const uint32_t my_slot = xchg_base + slot_off + 8u * (uint32_t)((warp - 2) * 32 + lane);
        const uint32_t peer_slot = xchg_base + slot_off + 8u * (uint32_t)((((warp - 2) ^ 4)) * 32 + lane);
        const uint32_t seq = (uint32_t)iter + 1u;
        float dot = 0.f;
        auto exchange_dot = [&]() {
          asm volatile("st.volatile.shared.v2.b32 [%0], {%1, %2};" ::"r"(my_slot), "r"(__float_as_uint(dot)), "r"(seq) : "memory");
          uint32_t vb = 0, sq = 0;
          int tries = 0;
          do {
            asm volatile("ld.volatile.shared.v2.b32 {%0, %1}, [%2];" : "=r"(vb), "=r"(sq) : "r"(peer_slot) : "memory");
          } while (sq != seq && ++tries < (1 << 24) && !*abort_flag);
          if (sq != seq) { atomicCAS(&g_status, 0, 0x710); *abort_flag = 1; }
          dot += __uint_as_float(vb);
        };
        if (sb_nbox == 0) exchange_dot();                // no box of its own: the partner still needs a zero from this warp
        const int first_visits = sb_nbox;
        const int visits = 2 * sb_nbox;
#pragma unroll 1
        for (int vis = 0; vis < visits; ++vis) {
          const bool second = vis >= first_visits;
          const int bc = col_half * 64 + 128 * (second ? vis - first_visits : vis);     // first column of the box inside the tile
          const uint32_t box = stg + buf * 4096u;
          if (!mbar_wait(mfull_bar(buf), (mask_phase >> buf) & 1u, 0x500 + (int)buf, abort_flag)) { ok = false; break; }
          mask_phase ^= 1u << buf;
          if (vis + 1 < visits && lane == 0) {           // next visit's box into the other staging box, while this one is worked on
            const int nv = vis + 1;
            const int nbc = col_half * 64 + 128 * (nv >= first_visits ? nv - first_visits : nv);
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            mbar_expect_tx(mfull_bar(buf ^ 1u), 4096u);
            tma_load_5d<false>(stg + (buf ^ 1u) * 4096u, &map_m, mfull_bar(buf ^ 1u), tl.n0 + nbc, row0, tl.o[2], tl.o[1], tl.o[0]);
          }
          const uint32_t srow = box + (uint32_t)lane * 128u;
          const uint32_t sw = (uint32_t)(lane & 7);
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t raw[32];
            tmem_ld32(taddr + bc + 32 * half, raw);
            float pw[32];
#pragma unroll
            for (int i = 0; i < 4; ++i) unpack_bf16x8(ld_shared_v4(srow + ((((uint32_t)(half * 4 + i)) ^ sw) << 4)), pw + 8 * i);
            tmem_ld_wait();
            float* v = reinterpret_cast<float*>(raw);
            if (!second) {
#pragma unroll
              for (int j = 0; j < 32; ++j) dot = fmaf(v[j], pw[j], dot);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = pw[j] * (v[j] - dot);
              store_staged(f, v, box, lane, half);
            }
          }
          if (second) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) tma_store_5d(&map_c, box, tl.n0 + bc, row0, tl.o[2], tl.o[1], tl.o[0]);
          }
          __syncwarp();
          buf ^= 1u;
          if (vis == first_visits - 1) exchange_dot();   // all first visits done: the row's dot product
        }
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        // boxes right of every row's causal limit: zeros
#pragma unroll 1
        for (int bc = col_half * 64 + 128 * sb_nbox; rows_full && bc < a.block_n && tl.n0 + bc + 64 <= tl.n_end; bc += 128) {
          const uint32_t box = stg + buf * 4096u;
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 8; ++i) st_shared_v4(box + (uint32_t)lane * 128u + 16u * i, 0u, 0u, 0u, 0u);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) tma_store_5d(&map_c, box, tl.n0 + bc, row0, tl.o[2], tl.o[1], tl.o[0]);
          buf ^= 1u;
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_pair<kPair>(tempty_bar(acc), (uint32_t)(2 * pair_idx));
        continue;
      }
      if (EPI == EPI_ROW_SOFTMAX) {
        // The tile holds whole rows of logits (one tile column per slice).  Softmax over each row in
        // three passes over the accumulator, which stays in tensor memory: maximum, sum of
        // exponentials, normalised weights (bf16).  A row lives in one lane; the two warps of a lane
        // quarter own alternate 64-column boxes and exchange their partial maximum and sum through
        // shared memory (value + sequence number, bounded wait).
        const float sl2 = a.scale * 1.4426950408889634f;                   // logits in units of log 2
        const int ncols = min(a.block_n, tl.n_end - tl.n0);
        const int lim = a.softmax_causal ? min(ncols, row + 1) : ncols;    // columns [0, lim) take part (row = position in `length`)
        const int lim_warp = __shfl_sync(0xffffffffu, lim, 31);            // rows ascend with the lane: the warp's widest row
        const uint32_t my_slot = xchg_base + 8u * (uint32_t)((warp - 2) * 32 + lane);
        const uint32_t peer_slot = xchg_base + 8u * (uint32_t)((((warp - 2) ^ 4)) * 32 + lane);
        const uint32_t seq = (uint32_t)iter + 1u;
        auto exchange = [&](int slot, float mine, bool take_max) -> float {
          const uint32_t off = (uint32_t)slot * (8u * kEpilogueWarps * 32u);
          asm volatile("st.volatile.shared.v2.b32 [%0], {%1, %2};" ::"r"(my_slot + off), "r"(__float_as_uint(mine)), "r"(seq) : "memory");
          uint32_t vb = 0, sq = 0;
          int tries = 0;
          do {
            asm volatile("ld.volatile.shared.v2.b32 {%0, %1}, [%2];" : "=r"(vb), "=r"(sq) : "r"(peer_slot + off) : "memory");
          } while (sq != seq && ++tries < (1 << 24) && !*abort_flag);
          if (sq != seq) { atomicCAS(&g_status, 0, 0x700 + slot); *abort_flag = 1; }
          const float other = __uint_as_float(vb);
          return take_max ? fmaxf(mine, other) : mine + other;
        };
        const int lim_all = __shfl_sync(0xffffffffu, lim, 0);             // columns below it take part in every row of the warp
        float mx = -INFINITY;
#pragma unroll 1
        for (int c0 = col_half * 64; c0 < lim_warp; c0 += (c0 & 32) ? 96 : 32) {
          uint32_t raw[32];
          tmem_ld32(taddr + c0, raw);
          tmem_ld_wait();
          if (c0 + 32 <= lim_all) {
#pragma unroll
            for (int j = 0; j < 32; ++j) mx = fmaxf(mx, __uint_as_float(raw[j]));
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c0 + j < lim) mx = fmaxf(mx, __uint_as_float(raw[j]));
          }
        }
        // (the maximum is taken over the raw accumulator: scale > 0 keeps the order; a negative scale would need the minimum)
        mx = exchange(0, mx, true) * sl2;
        float sum = 0.f;
#pragma unroll 1
        for (int c0 = col_half * 64; c0 < lim_warp; c0 += (c0 & 32) ? 96 : 32) {
          uint32_t raw[32];
          tmem_ld32(taddr + c0, raw);
          tmem_ld_wait();
          if (c0 + 32 <= lim_all) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float e = ex2_approx(fmaf(__uint_as_float(raw[j]), sl2, -mx));
              sum += e;
              raw[j] = __float_as_uint(e);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float e = (c0 + j < lim) ? ex2_approx(fmaf(__uint_as_float(raw[j]), sl2, -mx)) : 0.f;
              sum += e;
              raw[j] = __float_as_uint(e);
            }
          }
          tmem_st32(taddr + c0, raw);                 // the exponentials replace the logits: the last pass only scales them
        }
        tmem_st_wait();
        sum = exchange(1, sum, false);
        const float inv = 1.f / sum;
#pragma unroll 1
        for (int c0 = col_half * 64; c0 < a.block_n; c0 += (c0 & 32) ? 96 : 32) {
          const int n_first = tl.n0 + c0;
          int n_valid = tl.n_end - n_first;
          n_valid = n_valid > 32 ? 32 : n_valid;
          const bool live = row_ok && n_valid > 0;
          const int box_n0 = tl.n0 + (c0 & ~63);
          const bool staged = rows_full && box_n0 + 64 <= tl.n_end;
          const int half = (c0 >> 5) & 1;
          const uint32_t box = stg + buf * 4096u;
          float v[32];
          if (c0 < lim_warp) {
            uint32_t raw[32];
            tmem_ld32(taddr + c0, raw);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(raw[j]) * inv;
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0.f;
          }
          if (staged && half == 0) {
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            __syncwarp();
          }
          if (staged) store_staged(f, v, box, lane, half);
          else if (live) store_direct(a, f, v, row_off + n_first, n_valid);
          if (staged && half == 1) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) tma_store_5d(&map_c, box, box_n0, row0, tl.o[2], tl.o[1], tl.o[0]);
            buf ^= 1u;
          }
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_pair<kPair>(tempty_bar(acc), (uint32_t)(2 * pair_idx));
        continue;
      }
      // A tile shared by several workers: every worker but the last to arrive (per 32-row group and
      // column part) leaves its fragment in the workspace; the last one keeps its own in registers,
      // adds the others in ascending order of the fragments (= of the processors of the group) and
      // runs the regular epilogue.  It may have to wait for a fragment that is still being written:
      // its writer is already running and waits for nobody.
      const int warp_tile_row = pm * kPairRows + cta_rank * BM + q * 32;      // first row of this warp inside the tile
      const long long ws_ci = (t * (kTileRows / 32) + warp_tile_row / 32) * 2 + col_half;
      bool finisher = true;
      if (ws_mode) {
        unsigned old = 0;
        if (lane == 0) old = atomicAdd(&a.ws_counters[ws_ci], 1u);
        old = __shfl_sync(0xffffffffu, old, 0);
        finisher = old == (unsigned)sg.nfrag - 1;
        if (finisher) {
          int good = 1;
          if (lane == 0) {
            const volatile unsigned* written = a.ws_counters + a.ws_ncounters + ws_ci;
            const long long t0 = clock64();
            while (*written < (unsigned)sg.nfrag - 1) {
              __nanosleep(64);
              if (*abort_flag) { good = 0; break; }
              if (clock64() - t0 > g_wait_limit) { atomicCAS(&g_status, 0, 0x600); *abort_flag = 1; good = 0; break; }
            }
            __threadfence();
          }
          ok = __shfl_sync(0xffffffffu, good, 0) != 0;
          if (!ok) break;
        }
      }
      if (EPI == EPI_MASK_RSUM_BF16 && rows_full && tl.n0 + a.block_n <= tl.n_end) {
        // A tile that lies wholly inside its slice, for the kind whose epilogue sets the pace of its
        // contraction (dhp): a box (two 32-column chunks) at a time, both tensor-memory loads in flight
        // together and the two chunks' arithmetic interleaved (3 us of 117; the same for bias + relu lost 1 us).
#pragma unroll 1
        for (int c0 = col_half * 64; c0 < a.block_n; c0 += 128) {
          uint32_t r0[32], r1[32];
          tmem_ld32(taddr + c0, r0);
          tmem_ld32(taddr + c0 + 32, r1);
          const uint32_t box = stg + buf * 4096u;
          const uint32_t srow = box + (uint32_t)lane * 128u;
          const uint32_t sw = (uint32_t)(lane & 7);
          uint4 mk[8];
          mbar_wait(mfull_bar(buf), (mask_phase >> buf) & 1u, 0x500 + (int)buf, abort_flag);   // its relu mask, requested a box ago
          mask_phase ^= 1u << buf;
          if (lane == 0 && c0 + 128 < a.block_n) {                                             // the next box's mask into the other staging box
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            mbar_expect_tx(mfull_bar(buf ^ 1u), 4096u);
            tma_load_5d<false>(stg + (buf ^ 1u) * 4096u, &map_m, mfull_bar(buf ^ 1u), tl.n0 + c0 + 128, row0, tl.o[2], tl.o[1], tl.o[0]);
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) mk[i] = ld_shared_v4(srow + (((uint32_t)i ^ sw) << 4));
          tmem_ld_wait();
          float* v0 = reinterpret_cast<float*>(r0);
          float* v1 = reinterpret_cast<float*>(r1);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t w0[4] = {mk[i].x, mk[i].y, mk[i].z, mk[i].w}, w1[4] = {mk[4 + i].x, mk[4 + i].y, mk[4 + i].z, mk[4 + i].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              keep_where_positive(w0[e], v0[i * 8 + 2 * e], v0[i * 8 + 2 * e + 1]);
              keep_where_positive(w1[e], v1[i * 8 + 2 * e], v1[i * 8 + 2 * e + 1]);
            }
          }
          store_staged(f, v0, box, lane, 0);
          store_staged(f, v1, box, lane, 1);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) tma_store_5d(&map_c, box, tl.n0 + c0, row0, tl.o[2], tl.o[1], tl.o[0]);
          buf ^= 1u;
          const float s0 = warp_column_sums(v0, lane);      // the column sums while the store drains (v0, v1 are destroyed)
          const float s1 = warp_column_sums(v1, lane);
          if (a.rsum_partial) {
            float* const pr = a.rsum_partial + (size_t)(tl.row_id * (kTileRows / 32) + warp_tile_row / 32) * a.N + tl.n0 + c0 + lane;
            pr[0] = s0;
            pr[32] = s1;
          } else {
            atomicAdd(a.rsum + tl.n0 + c0 + lane, s0);
            atomicAdd(a.rsum + tl.n0 + c0 + 32 + lane, s1);
          }
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_pair<kPair>(tempty_bar(acc), (uint32_t)(2 * pair_idx));
      } else if (finisher) {
        // whole boxes of 32 rows x 128 B that lie inside the slice leave through the staging
        // buffers and TMA stores (a bf16 relu mask of such a box arrives the same way, in place);
        // ragged edges are read and stored from registers
        const CUtensorMap* const pc = sg.group == 0 ? &map_c : &extra.c[sg.group - 1];       // (grouped launch: this problem's output)
        void* const c_base = sg.group == 0 ? a.C : a.C_group[sg.group - 1];
        float bias_cur = bias_at(tl.n0 + col_half * box_cols + lane);      // lane l keeps column l of the current chunk
        float lse_m = -INFINITY, lse_s = 0.f;      // (EPI_ROW_LSE_BF16) running maximum and sum of exponentials of this row's stored values
#pragma unroll 1
        for (int c0 = 0; c0 < a.block_n; c0 += 32) {
          if (((c0 / box_cols) & 1) != col_half) continue;    // the other warp of this lane quarter owns that box
          uint32_t raw[32];
          tmem_ld32(taddr + c0, raw);
          const int n_first = tl.n0 + c0;
          int n_valid = tl.n_end - n_first;
          n_valid = n_valid > 32 ? 32 : n_valid;
          const bool live = row_ok && n_valid > 0;
          const int box_n0 = tl.n0 + (c0 & ~(box_cols - 1));
          const bool staged = rows_full && box_n0 + box_cols <= tl.n_end;
          const int half = (c0 >> 5) & 1;
          const uint32_t box = stg + buf * 4096u;
          if (staged && (c0 & (box_cols - 1)) == 0) {           // first chunk of a box
            if (in_tma) {                                       // its mask / residual was requested a box ago, in place
              mbar_wait(mfull_bar(buf), (mask_phase >> buf) & 1u, 0x500 + (int)buf, abort_flag);
              mask_phase ^= 1u << buf;
              // the operand of this warp's next box of the tile into the other staging box (free once the
              // store issued from it a box ago has been read out), so that it arrives while this box is worked on
              const int next_n0 = box_n0 + 2 * box_cols;
              if (lane == 0 && next_n0 < tl.n0 + a.block_n && next_n0 + box_cols <= tl.n_end) {
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                mbar_expect_tx(mfull_bar(buf ^ 1u), 4096u);
                tma_load_5d<false>(stg + (buf ^ 1u) * 4096u, &map_m, mfull_bar(buf ^ 1u), next_n0, row0, tl.o[2], tl.o[1], tl.o[0]);
              }
            } else {                                            // the box must be free: all but the latest store read out
              if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
              __syncwarp();
            }
          }
          uint4 mk[4];
          if (f.mask && f.mask_bf16) {
            if (staged && mask_tma) {
#pragma unroll
              for (int i = 0; i < 4; ++i) mk[i] = ld_shared_v4(box + (uint32_t)lane * 128u + ((((uint32_t)(half * 4 + i)) ^ (uint32_t)(lane & 7)) << 4));
            } else {
              mask_fetch(a, row_off + n_first, row_ok, n_valid, mk);
            }
          }
          // bias of the chunk this warp handles next (the next chunk of the box, or two boxes on)
          const int next_c0 = (half == 0 && box_cols == 64) ? c0 + 32 : c0 + 32 + box_cols;
          const float bias_next = bias_at(tl.n0 + next_c0 + lane);
          tmem_ld_wait();
          float* v = reinterpret_cast<float*>(raw);
          if (ws_mode) {
            // fragment layout: per 32-row x 32-column chunk 4 KB, piece j of lane l at j * 512 + l * 16 bytes,
            // so that every 16-byte access of a warp covers 512 contiguous bytes
            const float* prow = a.ws_partials + (((size_t)(t * a.slots) * (kTileRows / 32) + (size_t)(warp_tile_row / 32)) * (a.block_n / 32) + (size_t)(c0 / 32)) * 1024 + lane * 4;
            const size_t slot_stride = (size_t)kTileRows * a.block_n;
            float pre[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) pre[j] = 0.f;
            for (int s2 = 0; s2 < sg.nfrag; ++s2) {
              if (s2 == ks) {
#pragma unroll
                for (int j = 0; j < 32; ++j) pre[j] += v[j];
              } else {
                const float4* sp = reinterpret_cast<const float4*>(prow + (size_t)s2 * slot_stride);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const float4 x4 = __ldcg(sp + 32 * j);
                  pre[4 * j] += x4.x; pre[4 * j + 1] += x4.y; pre[4 * j + 2] += x4.z; pre[4 * j + 3] += x4.w;
                }
              }
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = pre[j];
          }
          epilogue_math(a, f, v, bias_cur, bias_row, mk, row_off + n_first, live, n_valid);
          bias_cur = bias_next;
          if (staged && resid_tma) {                 // this lane's part of the residual box, where the result will go
            const uint32_t srow = box + (uint32_t)lane * 128u;
            const uint32_t sw = (uint32_t)(lane & 7);
            if (f.c_bf16) {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                float r8[8];
                unpack_bf16x8(ld_shared_v4(srow + ((((uint32_t)(half * 4 + i)) ^ sw) << 4)), r8);
#pragma unroll
                for (int e = 0; e < 8; ++e) v[i * 8 + e] += r8[e];
              }
            } else {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const uint4 r4 = ld_shared_v4(srow + (((uint32_t)i ^ sw) << 4));
                v[4 * i] += __uint_as_float(r4.x); v[4 * i + 1] += __uint_as_float(r4.y);
                v[4 * i + 2] += __uint_as_float(r4.z); v[4 * i + 3] += __uint_as_float(r4.w);
              }
            }
          } else {
            epilogue_residual(a, f, v, row_off + n_first, live, n_valid);
          }
          if (EPI == EPI_ROW_LSE_BF16 && live) {
            // row statistics of the values as they are stored (rounded to bf16), so that they describe the tensor in memory
            float cm = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              v[j] = __bfloat162float(__float2bfloat16_rn(v[j]));
              if (j < n_valid) cm = fmaxf(cm, v[j]);
            }
            const float nm = fmaxf(lse_m, cm);
            float cs = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (j < n_valid) cs += exp2f((v[j] - nm) * 1.4426950408889634f);
            lse_s = lse_s * exp2f((lse_m - nm) * 1.4426950408889634f) + cs;
            lse_m = nm;
          }
          if (staged) store_staged(f, v, box, lane, half);
          else if (live) store_direct(a, f, v, row_off + n_first, n_valid, c_base);
          if (staged && ((c0 + 32) & (box_cols - 1)) == 0) {     // box complete: hand it to the TMA
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) tma_store_5d(pc, box, box_n0, row0, tl.o[2], tl.o[1], tl.o[0]);
            buf ^= 1u;
          }
          if (f.rsum && n_valid > 0) {       // fused reduce_sum (never combined with a residual): v may be destroyed now
            if (!(rows_full && n_valid == 32)) {       // ragged chunk: rows and columns outside the slice add nothing
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = (live && j < n_valid) ? v[j] : 0.f;
            }
            const float col = warp_column_sums(v, lane);
            if (lane < n_valid) {
              if (a.rsum_partial) a.rsum_partial[(size_t)(tl.row_id * (kTileRows / 32) + warp_tile_row / 32) * a.N + n_first + lane] = col;
              else atomicAdd(a.rsum + n_first + lane, col);
            }
          }
        }
        if (EPI == EPI_ROW_LSE_BF16 && row_ok) {
          const int slice_n = tl.n_end / a.Ns - 1, tile_n = (tl.n0 - slice_n * a.Ns) / a.block_n;
          a.lse_partial[(long long)row * a.lse_parts + (slice_n * a.n_tiles + tile_n) * 2 + col_half] = make_float2(lse_m, lse_s);
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_pair<kPair>(tempty_bar(acc), (uint32_t)(2 * pair_idx));
      } else {
        // fragment `ks` of the tile -> workspace, straight from registers in the chunk layout described
        // at the reading side (the chunks this warp owns in the regular epilogue, so that the finisher
        // finds them under the same counter)
        float* pbase = a.ws_partials + (((size_t)(t * a.slots + ks) * (kTileRows / 32) + (size_t)(warp_tile_row / 32)) * (a.block_n / 32)) * 1024 + lane * 4;
#pragma unroll 1
        for (int c0 = 0; c0 < a.block_n; c0 += 32) {
          if (((c0 / box_cols) & 1) != col_half) continue;
          uint32_t raw[32];
          tmem_ld32(taddr + c0, raw);
          float4* pp = reinterpret_cast<float4*>(pbase + (size_t)(c0 / 32) * 1024);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            __stcg(pp + 32 * j, make_float4(__uint_as_float(raw[4 * j]), __uint_as_float(raw[4 * j + 1]), __uint_as_float(raw[4 * j + 2]), __uint_as_float(raw[4 * j + 3])));
        }
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_pair<kPair>(tempty_bar(acc), (uint32_t)(2 * pair_idx));
        }
        __threadfence();                                   // every lane's part of the fragment, then the flag
        __syncwarp();
        if (lane == 0) atomicAdd(&a.ws_counters[a.ws_ncounters + ws_ci], 1u);
        __syncwarp();
      }
    }
  }

  if (warp >= 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // staged output stores have landed

  // ------------------------------- teardown --------------------------------------
  if (*abort_flag) {
    // failure path: give copies and MMAs in flight time to land before the CTA's resources go away
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tcgen05_fence_before();
  __syncthreads();
  if (kPair) cluster_sync();      // the partner may still signal this CTA's barriers or read its tiles
  if (a.late_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---- host side -----------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// One tensor as a 5-D tensor map: (contiguous dim, second dim, outer2, outer1, outer0), 128B swizzle.
//   dim0 / dim1 : extents of the contiguous and of the strided dimension; ld = element stride of dim1
//   box0 / box1 : box extents in elements (box0 * elem_bytes = 128)
mtf_status make_map(CUtensorMap* map, const void* base, int elem_bytes, int64_t dim0, int64_t dim1, int64_t ld,
                    int box0, int box1, const TcParams& t, const int64_t* outer_stride) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return mtf::fail(MTF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  if (reinterpret_cast<uintptr_t>(base) & 15) return mtf::fail(MTF_ERR_INVALID_ARG, "tensor-core path needs 16-byte aligned tensors");
  const int64_t align = 16 / elem_bytes;     // strides must be multiples of 16 bytes
  cuuint64_t dims[5];
  cuuint64_t strides[4];
  cuuint32_t box[5] = {(cuuint32_t)box0, (cuuint32_t)box1, 1, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  dims[0] = dim0;
  dims[1] = dim1;
  // a dimension of extent 1 may carry any stride, give it a legal one
  int64_t s1 = ld;
  if (dims[1] == 1 || s1 % align != 0 || s1 <= 0) s1 = (dim0 + align - 1) / align * align;
  strides[0] = (cuuint64_t)s1 * elem_bytes;
  const int64_t dummy = (s1 * dim1 + align - 1) / align * align;   // legal stride for extent-1 dimensions
  for (int d = 2; d < 5; ++d) {
    const int src = 4 - d;   // map dim 4 = outer dim 0 ... map dim 2 = outer dim 2 (coordinates o[0..2])
    if (src < t.n_outer && t.outer_size[src] > 1 && outer_stride[src] > 0) {
      dims[d] = t.outer_size[src];
      strides[d - 1] = (cuuint64_t)outer_stride[src] * elem_bytes;
    } else {
      dims[d] = 1;
      strides[d - 1] = (cuuint64_t)dummy * elem_bytes;
    }
  }
  CUresult r = enc(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<void*>(base),
                   dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return mtf::fail(MTF_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d (dims %llu %llu %llu %llu %llu, strides %llu %llu %llu %llu)", (int)r,
                     (unsigned long long)dims[0], (unsigned long long)dims[1], (unsigned long long)dims[2], (unsigned long long)dims[3],
                     (unsigned long long)dims[4], (unsigned long long)strides[0], (unsigned long long)strides[1],
                     (unsigned long long)strides[2], (unsigned long long)strides[3]);
  return MTF_OK;
}

constexpr int kMaxDevices = 64;

int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
  return dev;
}

// SM count of the current device (looked up once per device).
int sm_count() {
  static std::atomic<int> cached[kMaxDevices];
  const int dev = current_device();
  int n = cached[dev].load(std::memory_order_relaxed);
  if (!n) {
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

// ---- counters for launches that draw their tiles ----------------------------------------------------------
// A launch that starts while the launch before it still runs (late_wait) finds some SMs free at once and the
// others later, so its workers draw tiles from a counter instead of owning every W-th one.  A counter pair must
// be zero when its launch starts and is cleared by that launch's last worker, so two launches that may overlap
// need different pairs: every stream has kSchedPerStream pairs, taken in turn by consecutive late launches, and
// after that many in a row the next launch is made an ordinary one (it waits for everything before it, after
// which all pairs are clear again).  Streams beyond kSchedStreams keep the fixed assignment.
constexpr int kSchedStreams = 16, kSchedPerStream = 3;
static __device__ unsigned g_sched_words[kSchedStreams * kSchedPerStream * 2];

struct DeviceSched {
  std::mutex mu;
  unsigned* base = nullptr;
  bool looked_up = false;
  cudaStream_t stream[kSchedStreams];
  int late_run[kSchedStreams];
  int n = 0;
};
static DeviceSched g_dev_sched[kMaxDevices];

// Called once per contraction launch: `late` is whether the launch may skip the wait at its start.  Returns the
// counter pair the launch draws from (NULL: fixed assignment); clears *late when the chain of late launches on
// this stream has used every pair.
static unsigned* sched_for_launch(cudaStream_t st, bool drawable, int* late) {
  DeviceSched& d = g_dev_sched[current_device()];
  std::lock_guard<std::mutex> lock(d.mu);
  if (!d.looked_up) {
    d.looked_up = true;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_sched_words) == cudaSuccess) d.base = reinterpret_cast<unsigned*>(p);
    else (void)cudaGetLastError();
  }
  int idx = -1;
  for (int i = 0; i < d.n; ++i)
    if (d.stream[i] == st) { idx = i; break; }
  if (idx < 0 && d.n < kSchedStreams) { idx = d.n++; d.stream[idx] = st; d.late_run[idx] = 0; }
  if (idx < 0 || !d.base) return nullptr;
  if (!*late) { d.late_run[idx] = 0; return nullptr; }
  if (d.late_run[idx] >= kSchedPerStream) { *late = 0; d.late_run[idx] = 0; return nullptr; }
  const int slot = d.late_run[idx]++;
  return drawable ? d.base + 2 * (idx * kSchedPerStream + slot) : nullptr;
}

static void sched_clear_all() {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_sched_words) == cudaSuccess) cudaMemset(p, 0, sizeof(unsigned) * kSchedStreams * kSchedPerStream * 2);
  else (void)cudaGetLastError();
}

// Clears 32-bit words (the fused reduce_sum output, the arrival counters of shared tiles).  A kernel
// rather than a memset so that it can sit in a chain of programmatically dependent launches: it
// waits for the kernel before it, and the contraction after it overlaps its set-up with this one.
__global__ void zero_words_kernel(uint32_t* p, long long n) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) p[i] = 0u;
}

mtf_status zero_words(void* p, long long n, cudaStream_t st) {
  if (n <= 0) return MTF_OK;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  const long long blocks = std::min<long long>((n + 255) / 256, 4 * sm_count());
  cfg.gridDim = dim3((unsigned)blocks, 1, 1); cfg.blockDim = dim3(256, 1, 1); cfg.stream = st; cfg.attrs = at; cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, zero_words_kernel, reinterpret_cast<uint32_t*>(p), n);
  if (e != cudaSuccess) return mtf::fail(MTF_ERR_CUDA, "zero_words_kernel: %s", cudaGetErrorString(e));
  mtf::count_launch();
  return MTF_OK;
}

// One kernel variant: shared-memory opt-in and the number of clusters that can be resident at once
// are looked up on first use; the grid is that many clusters (persistent) or fewer.
template <bool kPair, int CM, int CN, int EPI, bool kWide, bool kDrawn>
mtf_status launch_variant_impl(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_c, const CUtensorMap& map_m,
                               const CUtensorMap& map_w, const ExtraMaps& extra, const TcArgs& a, cudaStream_t st) {
  constexpr int kCtas = (kPair ? 2 : 1) * CM * CN;
  // the shared-memory opt-in and the number of resident clusters are properties of a device: one set-up per device
  struct PerDevice { std::once_flag once; cudaError_t attr_err = cudaSuccess; int max_clusters = 0; };
  static PerDevice per_device[kMaxDevices];
  PerDevice& pd = per_device[current_device()];
  std::call_once(pd.once, [&pd] {
    cudaError_t& attr_err = pd.attr_err;
    int& max_clusters = pd.max_clusters;
    attr_err = cudaFuncSetAttribute(gemm_tcgen05_kernel<kPair, CM, CN, EPI, kWide, kDrawn>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (attr_err != cudaSuccess) return;
    if (kCtas > 8) attr_err = cudaFuncSetAttribute(gemm_tcgen05_kernel<kPair, CM, CN, EPI, kWide, kDrawn>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (attr_err != cudaSuccess) return;
    if (kCtas == 1) { max_clusters = sm_count(); return; }
    cudaLaunchConfig_t q = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kCtas; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    q.gridDim = dim3(kCtas * sm_count(), 1, 1); q.blockDim = dim3(kThreads, 1, 1); q.dynamicSmemBytes = kSmemBytes;
    q.attrs = at; q.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tcgen05_kernel<kPair, CM, CN, EPI, kWide, kDrawn>, &q) == cudaSuccess && n > 0) max_clusters = n;
    else { max_clusters = sm_count() / kCtas; (void)cudaGetLastError(); }
  });
  const cudaError_t attr_err = pd.attr_err;
  const int max_clusters = pd.max_clusters;
  if (attr_err != cudaSuccess) return mtf::fail(MTF_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(attr_err));
  // balanced schedule: every resident cluster takes an equal share of the k-block units
  const long long clusters = a.balanced ? std::min<long long>(a.total_tiles, max_clusters) : std::min<long long>(a.total_work, max_clusters);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // set-up may overlap the previous kernel's tail
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = kCtas; at[1].val.clusterDim.y = 1; at[1].val.clusterDim.z = 1;
  cfg.gridDim = dim3((unsigned)(kCtas * clusters), 1, 1); cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = st; cfg.attrs = at; cfg.numAttrs = kCtas > 1 ? 2 : 1;
  cudaError_t le = cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<kPair, CM, CN, EPI, kWide, kDrawn>, map_a, map_b, map_c, map_m, map_w, extra, a);
  if (le != cudaSuccess) return mtf::fail(MTF_ERR_CUDA, "gemm_tcgen05_kernel<%d,%d,%d,%d>: %s", (int)kPair, CM, CN, EPI, cudaGetErrorString(le));
  return MTF_OK;
}

// The variant whose workers draw their tiles exists for the kinds an independent launch can have (plain and generic
// epilogues of plain pairs and single CTAs); every other launch ignores TcArgs::sched and leaves its counter untouched.
template <bool kPair, int CM, int CN, int EPI, bool kWide = false>
mtf_status launch_variant(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_c, const CUtensorMap& map_m,
                          const CUtensorMap& map_w, const ExtraMaps& extra, const TcArgs& a, cudaStream_t st) {
  constexpr bool kCanDraw = CM * CN == 1 && (EPI == EPI_GENERIC || EPI == EPI_PLAIN_BF16 || EPI == EPI_PLAIN_F32);
  if constexpr (kCanDraw) {
    if (a.sched) return launch_variant_impl<kPair, CM, CN, EPI, kWide, true>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
  }
  return launch_variant_impl<kPair, CM, CN, EPI, kWide, false>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
}

// Picks the epilogue kind of a launch.  kAllKinds = false leaves out the relu-mask kind (cluster
// shapes that are never used with a mask).
template <bool kPair, int CM, int CN, bool kAllKinds>
mtf_status launch_kind(int epi, const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_c, const CUtensorMap& map_m,
                       const CUtensorMap& map_w, const ExtraMaps& extra, const TcArgs& a, cudaStream_t st) {
  switch (epi) {
    case EPI_PLAIN_BF16: return launch_variant<kPair, CM, CN, EPI_PLAIN_BF16>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    case EPI_PLAIN_F32: return launch_variant<kPair, CM, CN, EPI_PLAIN_F32>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    case EPI_BIAS_RELU_BF16: return launch_variant<kPair, CM, CN, EPI_BIAS_RELU_BF16>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    case EPI_ROW_LSE_BF16:
      if (kAllKinds) return launch_variant<kPair, CM, CN, kAllKinds ? EPI_ROW_LSE_BF16 : EPI_GENERIC>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
      return mtf::fail(MTF_ERR_UNSUPPORTED, "row log-sum-exp partials: no kernel for this cluster shape");
    case EPI_MASK_RSUM_BF16:
      if (kAllKinds) return launch_variant<kPair, CM, CN, kAllKinds ? EPI_MASK_RSUM_BF16 : EPI_GENERIC>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    default: return launch_variant<kPair, CM, CN, EPI_GENERIC>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
  }
}

}  // namespace

namespace mtf {

static int tc_tile_rows(const TcParams& t) { return t.cta_pair ? 2 * BM : BM; }

static int64_t tc_total_tiles(const TcParams& t) {
  const int rows = tc_tile_rows(t);
  int64_t tiles = ((t.M / t.sm + rows - 1) / rows) * ((t.N / t.sn + t.block_n - 1) / t.block_n) * t.sm * t.sn;
  for (int j = 0; j < t.n_outer; ++j) tiles *= t.outer_size[j];
  return tiles;
}

// Scratch for a fused reduce_sum whose column sums are finished in a fixed order: one fp32 row of N per 32-row group
size_t tc_rsum_partial_bytes(const TcParams& t) {
  const int rows = tc_tile_rows(t);
  int64_t groups = ((t.M / t.sm + rows - 1) / rows) * (rows / 32) * t.sm;
  for (int j = 0; j < t.n_outer; ++j) groups *= t.outer_size[j];
  return (size_t)groups * t.N * sizeof(float);
}

size_t tc_workspace_bytes(const TcParams& t) {
  if (t.reduce_mode != MTF_REDUCE_WORKSPACE) {
    if (!t.balance) return 0;
    // two fp32 fragments per tile plus counters, for tiles of up to 512 rows (upper bound over the tile shapes)
    int64_t area = ((t.M / t.sm + 511) / 512 * 512) * t.sm * (((t.N / t.sn + t.block_n - 1) / t.block_n) * t.block_n) * t.sn;
    for (int j = 0; j < t.n_outer; ++j) area *= t.outer_size[j];
    return (size_t)area * 2 * sizeof(float) + (size_t)(area / (32 * 64)) * 4 * sizeof(unsigned) + 1024;
  }
  const int64_t tiles = tc_total_tiles(t);
  return (size_t)tiles * t.sk * tc_tile_rows(t) * t.block_n * sizeof(float) + (size_t)tiles * (tc_tile_rows(t) / 32) * 4 * sizeof(unsigned) + 256;
}

mtf_status launch_tc(const mtf_plan_t& plan, const void* A, const void* B, void* C, const void* bias, int dtBias,
                     const void* mask, int dtMask, const void* resid, int dtRes, float scale, int relu, float* rsum,
                     void* workspace, size_t workspace_bytes, void* stream, int n_terms, const void* const* extra_operands,
                     int row_softmax, int n_groups, const void* const* group_operands) {
  const TcParams& t = plan.tc;
  if (t.swapped) std::swap(A, B);
  if (n_terms < 1 || n_terms > 3 || (n_terms > 1 && !extra_operands)) return fail(MTF_ERR_INVALID_ARG, "1 to 3 terms");
  if (n_terms > 1 && t.reduce_mode == MTF_REDUCE_WORKSPACE) return fail(MTF_ERR_UNSUPPORTED, "a multi-term contraction cannot use the workspace reduce mode");
  if (n_groups < 1 || n_groups > 3 || (n_groups > 1 && (!group_operands || n_terms != 1 || row_softmax || bias || mask || resid || rsum || relu)))
    return fail(MTF_ERR_INVALID_ARG, "a grouped launch takes 1 to 3 plain problems");
  if (t.M > 0x7fffffffLL || t.N > 0x7fffffffLL || t.K > 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "extent beyond 2^31");
  if (reinterpret_cast<uintptr_t>(C) & 15) return fail(MTF_ERR_INVALID_ARG, "tensor-core path needs a 16-byte aligned output");
  if (bias && !t.bias_along_m && (reinterpret_cast<uintptr_t>(bias) & 15)) return fail(MTF_ERR_INVALID_ARG, "tensor-core path needs a 16-byte aligned bias");
  if ((mask && (reinterpret_cast<uintptr_t>(mask) & 15)) || (resid && (reinterpret_cast<uintptr_t>(resid) & 15)))
    return fail(MTF_ERR_INVALID_ARG, "tensor-core path needs 16-byte aligned epilogue operands");

  TcArgs a;
  a.M = (int)t.M; a.N = (int)t.N; a.K = (int)t.K;
  a.sm = (int)t.sm; a.sn = (int)t.sn; a.sk = (int)t.sk;
  a.Ms = a.M / a.sm; a.Ns = a.N / a.sn; a.Ks = a.K / a.sk;
  a.n_outer = t.n_outer;
  for (int j = 0; j < 3; ++j) {
    a.outer_split[j] = (int)t.outer_split[j];
    a.outer_local[j] = (int)(t.outer_size[j] / t.outer_split[j]);
    a.outer_sC[j] = t.outer_sC[j];
  }
  a.a_mn_major = t.a_mn_major; a.b_mn_major = t.b_mn_major;
  a.block_n = t.block_n;
  a.ldc = t.ldc;
  a.reduce_mode = (n_groups > 1 && t.reduce_mode == MTF_REDUCE_WORKSPACE) ? MTF_REDUCE_CHAINED : t.reduce_mode;     // a group has tiles enough: no fragments
  a.k_sliced = (t.sk > 1 && a.Ks % BK == 0) ? 1 : 0;
  // Wide tiles (256 x 512 per pair) for long contractions with a plain epilogue: per tile about 1.5x
  // the time of a 256 x 256 one (twice the MMAs at 3/4 of the L2 traffic each, epilogue exposed), so
  // they win when they halve the number of waves.
  bool wide = false;
  // row_softmax == 5: a plain bf16 contraction that also leaves, per row and column part, the maximum and the sum of
  // exponentials of the stored values at the head of the workspace (float2 [rows][parts]; the caller combines them)
  const bool row_lse = row_softmax == 5;
  if (row_lse) row_softmax = 0;
  const bool plain_epi = scale == 1.f && !resid && !bias && !relu && !mask && !rsum && !row_softmax;
  if (row_lse && (!plain_epi || plan.dtC != MTF_BF16 || t.n_outer != 0 || t.ldc != t.N || t.reduce_mode == MTF_REDUCE_WORKSPACE || n_terms != 1 || n_groups != 1))
    return fail(MTF_ERR_UNSUPPORTED, "row log-sum-exp partials need a plain bf16 contraction with dense rows and no workspace reduction");
  if (row_softmax) {
    // whole rows in one tile: the N slice is the whole dimension and fits a tile (256 columns, or 512 with a wide pair tile)
    const bool fits = a.sn == 1 && (a.Ns <= a.block_n || (a.Ns == 512 && t.cta_pair && t.block_n == 256));
    const bool bwd = row_softmax >= 3;      // backward: the weights come in as the mask operand, whole boxes only
    if (!bwd && !(scale > 0.f)) return fail(MTF_ERR_UNSUPPORTED, "row softmax in the epilogue needs a positive scale");
    if (!fits || plan.dtC != MTF_BF16 || resid || bias || relu || rsum || t.reduce_mode == MTF_REDUCE_WORKSPACE || n_terms != 1 ||
        (bwd ? (!mask || dtMask != MTF_BF16 || scale != 1.f || a.Ms % 32 != 0 || a.Ns % 64 != 0) : mask != nullptr))
      return fail(MTF_ERR_UNSUPPORTED, "row softmax in the epilogue needs a bf16 result whose rows fit one tile (N <= 256, or 512 with CTA pairs) and no other stage");
    wide = a.Ns == 512;
  }
  // (wide tiles also with a residual as the only stage - the contractions whose result is added to a stream of the
  //  decoder layer - through the generic epilogue kind)
  const bool resid_only_epi = scale == 1.f && resid && !bias && !relu && !mask && !rsum && !row_softmax && n_terms == 1;
  const bool wide_legal = t.cta_pair && t.block_n == 256 && t.reduce_mode != MTF_REDUCE_WORKSPACE && (plain_epi || resid_only_epi) && !row_lse && a.Ns % 512 == 0;
  if (t.wide_pref == 1 && !wide_legal)
    return fail(MTF_ERR_UNSUPPORTED, "wide tiles need CTA pairs, a plain or residual-only epilogue, no workspace reduction and an N slice that is a multiple of 512");
  if (wide_legal && t.wide_pref != 0) {
    long long tiles = (long long)((a.Ms + 2 * BM - 1) / (2 * BM)) * (a.Ns / 256) * a.sm * a.sn;
    for (int j = 0; j < t.n_outer; ++j) tiles *= t.outer_size[j];
    const long long workers = sm_count() / 2;
    const long long waves_narrow = (tiles + workers - 1) / workers, waves_wide = (tiles / 2 + workers - 1) / workers;
    wide = t.wide_pref == 1 || (t.K * n_terms >= 64 * BK && 3 * waves_wide < 2 * waves_narrow);
  }
  if (wide) a.block_n = 512;
  // optional single-GPU build: clusters of CTA pairs that share operand tiles
  int cm = 1, cn = 1;
#if defined(MTF_CLUSTER_SHARE)
  if (!wide && !row_softmax && !row_lse && t.cta_pair && t.block_n == 256 && t.reduce_mode != MTF_REDUCE_WORKSPACE && n_terms == 1 && n_groups == 1 &&
      cluster_share_operands_local(A, B)) {      // both operands are allocations of the GPU this launch runs on
    // measured on the FFN shapes: sharing B between two pairs that are neighbours along M is worth
    // 5-10 % on the contractions whose epilogue is light; with a relu mask or a fused reduction in the
    // epilogue the coupling of the two pairs costs more than the saved traffic; 2 x 2 clusters lose
    if (!mask && !rsum) {
      if (a.Ms % 512 == 0) cm = 2;
      else if (a.Ns % 512 == 0) cn = 2;
    }
  }
#endif
  const int tile_rows = tc_tile_rows(t) * cm;
  a.m_tiles = (a.Ms + tile_rows - 1) / tile_rows;
  a.n_tiles = (a.Ns + a.block_n * cn - 1) / (a.block_n * cn);
  a.n_fastest = 0;   // m tiles of one n tile run together: they share the B tile, which measured fastest
  a.tiles_per_slice = (long long)a.m_tiles * a.n_tiles;
  for (int j = 0; j < a.n_outer; ++j) a.tiles_per_slice *= a.outer_local[j];
  long long out_slices = (long long)a.sm * a.sn;
  for (int j = 0; j < a.n_outer; ++j) out_slices *= a.outer_split[j];
  a.total_tiles = a.tiles_per_slice * out_slices;
  a.total_work = a.reduce_mode == MTF_REDUCE_WORKSPACE ? a.total_tiles * a.sk : a.total_tiles * n_groups;
  a.n_groups = n_groups;
  a.C_group[0] = a.C_group[1] = nullptr;
  if (a.total_work >= 0x7fffffffLL) return fail(MTF_ERR_UNSUPPORTED, "more than 2^31 tiles");
  a.fd_tiles_per_slice = make_fastdiv(a.tiles_per_slice);
  a.fd_n_tiles = make_fastdiv(a.n_tiles); a.fd_m_tiles = make_fastdiv(a.m_tiles);
  a.fd_sn = make_fastdiv(a.sn); a.fd_sm = make_fastdiv(a.sm); a.fd_sk = make_fastdiv(a.sk);
  for (int j = 0; j < 3; ++j) { a.fd_outer_local[j] = make_fastdiv(a.outer_local[j]); a.fd_outer_split[j] = make_fastdiv(a.outer_split[j]); }
  a.C = C; a.c_bf16 = plan.dtC == MTF_BF16;
  a.bias = bias; a.bias_bf16 = dtBias == MTF_BF16; a.bias_along_m = t.bias_along_m;
  a.mask = mask; a.mask_bf16 = dtMask == MTF_BF16;
  a.mask_tma = (mask && a.mask_bf16 && a.c_bf16) ? 1 : 0;
  a.resid = resid; a.resid_bf16 = dtRes == MTF_BF16;
  a.resid_tma = (resid && !a.mask_tma && a.resid_bf16 == a.c_bf16) ? 1 : 0;
  a.scale = scale; a.relu = relu;
  a.rsum = rsum;
  a.rsum_partial = nullptr;
  a.lse_partial = nullptr; a.lse_parts = 0;
  if (row_lse) {
    a.lse_parts = a.sn * a.n_tiles * 2;
    const size_t need = (size_t)t.M * a.lse_parts * sizeof(float2);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15) || workspace_bytes < need)
      return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "row log-sum-exp partials need %zu workspace bytes, got %zu", need, workspace_bytes);
    a.lse_partial = reinterpret_cast<float2*>(workspace);
  }
  a.ws_partials = nullptr; a.ws_counters = nullptr; a.ws_ncounters = 0;
  {
    const int b_cols = (t.cta_pair ? a.block_n / 2 : a.block_n);          // B columns staged by one CTA (wide: two runs of 128)
    a.stage_bytes = kAStageBytes + b_cols * BK * 2;
    const int ring = kRingBytes - (row_softmax ? 2048 : 0);
    a.n_stages = std::min(kMaxStages, ring / a.stage_bytes);
  }
  a.kb_term = a.k_sliced ? a.sk * (a.Ks / BK) : (a.K + BK - 1) / BK;
  a.n_terms = n_terms;
  a.softmax_causal = (row_softmax == 2 || row_softmax == 4) ? 1 : 0;
  a.kb_tile = a.kb_term * n_terms;
  // the caller's word that this launch is independent of the one before it (consumed here); only honoured
  // for launches that clear nothing beforehand and use no workspace
  a.late_wait = (take_independent_hint() && !rsum && t.reduce_mode != MTF_REDUCE_WORKSPACE && !t.balance) ? 1 : 0;
  // such a launch draws its tiles (plain pairs and single CTAs; see sched_for_launch)
  a.sched = sched_for_launch((cudaStream_t)stream, cm * cn == 1, &a.late_wait);
  // Successive launches walk their tiles in opposite directions: a contraction that reads what the launch
  // before it wrote (h then y, the attention weights then P.v) starts with the part that is still in L2.
  static std::atomic<unsigned> launch_parity{0};
  a.reverse = a.reduce_mode != MTF_REDUCE_WORKSPACE ? (int)(launch_parity.fetch_add(1) & 1u) : 0;     // (measured: under 1 % of a step)
  a.slots = a.reduce_mode == MTF_REDUCE_WORKSPACE ? a.sk : 2;
  a.balanced = 0;
  if (a.total_work <= 0) return MTF_OK;

  cudaStream_t st = (cudaStream_t)stream;
  if (t.balance && cn == 1 && !wide && n_terms == 1 && n_groups == 1 && !row_softmax && !row_lse && workspace && !(reinterpret_cast<uintptr_t>(workspace) & 255)) {
    // Tail balancing: the tiles do not fill a whole number of waves, so the workers take equal ranges
    // of (tile, k-block) units; a tile cut by a range boundary is assembled from two fp32 fragments in
    // the workspace by whichever worker finishes last (arrive, never wait).
    const long long workers = sm_count() / ((t.cta_pair ? 2 : 1) * cm);
    const long long rounds = (a.total_tiles + workers - 1) / workers;
    const bool worth = a.total_tiles >= workers && (double)a.total_tiles / (double)(rounds * workers) <= 0.92;
    const size_t part_bytes = (size_t)a.total_tiles * 2 * tile_rows * a.block_n * sizeof(float);
    a.ws_ncounters = a.total_tiles * (tile_rows / 32) * 2;
    const size_t cnt_bytes = (size_t)a.ws_ncounters * 2 * sizeof(unsigned);     // arrivals, fragments written
    if (worth && workspace_bytes >= ((part_bytes + 255) / 256) * 256 + cnt_bytes) {
      a.balanced = 1;
      a.ws_partials = reinterpret_cast<float*>(workspace);
      a.ws_counters = reinterpret_cast<unsigned*>(reinterpret_cast<uint8_t*>(workspace) + ((part_bytes + 255) / 256) * 256);
      mtf_status zs = zero_words(a.ws_counters, (long long)(cnt_bytes / sizeof(unsigned)), st);
      if (zs != MTF_OK) return zs;
    }
  }
  if (a.reduce_mode == MTF_REDUCE_WORKSPACE) {
    const size_t need = tc_workspace_bytes(t);
    if (!workspace || workspace_bytes < need) return fail(MTF_ERR_WORKSPACE_TOO_SMALL, "einsum needs %zu workspace bytes, got %zu", need, workspace_bytes);
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return fail(MTF_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    const size_t part_bytes = (size_t)a.total_tiles * a.sk * tile_rows * a.block_n * sizeof(float);
    a.ws_partials = reinterpret_cast<float*>(workspace);
    a.ws_counters = reinterpret_cast<unsigned*>(reinterpret_cast<uint8_t*>(workspace) + ((part_bytes + 255) / 256) * 256);
    a.ws_ncounters = a.total_tiles * (tile_rows / 32) * 2;
    mtf_status zs = zero_words(a.ws_counters, a.ws_ncounters * 2, st);
    if (zs != MTF_OK) return zs;
  }

  long long rsum_groups = 0;
  if (rsum) {
    // with room in the workspace the column sums are left per 32-row group and finished in group order by a small
    // launch behind this one (repeatable bit for bit); otherwise they are added to the zeroed output with atomics
    rsum_groups = (a.total_tiles / ((long long)a.n_tiles * a.sn)) * (tile_rows / 32);
    const size_t need = (size_t)rsum_groups * t.N * sizeof(float);
    if (!a.ws_partials && workspace && !(reinterpret_cast<uintptr_t>(workspace) & 15) && workspace_bytes >= need) {
      a.rsum_partial = reinterpret_cast<float*>(workspace);
    } else {
      mtf_status zs = zero_words(rsum, t.N, st);
      if (zs != MTF_OK) return zs;
    }
  }
  CUtensorMap map_a, map_b, map_c, map_m;
  mtf_status s;
  // operands: K-major = (K contiguous, M|N rows), box 64 x rows;  MN-major = (M|N contiguous, K rows), box 64 x 64
  // (a CTA of a sharing cluster loads 1/cn of its A rows and 1/cm of its B columns per box)
  const int b_rows = (t.cta_pair ? t.block_n / 2 : t.block_n) / cm;
  s = t.a_mn_major ? make_map(&map_a, A, 2, t.M, t.K, t.a_ld, 64, BK, t, t.outer_sA) : make_map(&map_a, A, 2, t.K, t.M, t.a_ld, 64, BM / cn, t, t.outer_sA);
  if (s != MTF_OK) return s;
  s = t.b_mn_major ? make_map(&map_b, B, 2, t.N, t.K, t.b_ld, 64, BK, t, t.outer_sB) : make_map(&map_b, B, 2, t.K, t.N, t.b_ld, 64, b_rows, t, t.outer_sB);
  if (s != MTF_OK) return s;
  ExtraMaps extra;
  for (int i = 0; i < 4; ++i) extra.m[i] = i % 2 == 0 ? map_a : map_b;
  for (int i = 1; i < n_terms; ++i) {
    const void* Ai = extra_operands[2 * (i - 1)];
    const void* Bi = extra_operands[2 * (i - 1) + 1];
    if (t.swapped) std::swap(Ai, Bi);
    if (!Ai || !Bi) return fail(MTF_ERR_INVALID_ARG, "multi-term contraction: NULL operand");
    s = t.a_mn_major ? make_map(&extra.m[2 * (i - 1)], Ai, 2, t.M, t.K, t.a_ld, 64, BK, t, t.outer_sA) : make_map(&extra.m[2 * (i - 1)], Ai, 2, t.K, t.M, t.a_ld, 64, BM / cn, t, t.outer_sA);
    if (s != MTF_OK) return s;
    s = t.b_mn_major ? make_map(&extra.m[2 * (i - 1) + 1], Bi, 2, t.N, t.K, t.b_ld, 64, BK, t, t.outer_sB) : make_map(&extra.m[2 * (i - 1) + 1], Bi, 2, t.K, t.N, t.b_ld, 64, b_rows, t, t.outer_sB);
    if (s != MTF_OK) return s;
  }
  // output: (N contiguous, M rows), boxes of 32 rows x 128 bytes for the staged stores
  const int c_bytes = plan.dtC == MTF_BF16 ? 2 : 4;
  if ((s = make_map(&map_c, C, c_bytes, t.N, t.M, t.ldc, 128 / c_bytes, 32, t, t.outer_sC)) != MTF_OK) return s;
  extra.c[0] = extra.c[1] = map_c;
  for (int g = 1; g < n_groups; ++g) {          // grouped launch: problem g's operands (caller's order) and output
    const void* Ag = group_operands[3 * (g - 1)];
    const void* Bg = group_operands[3 * (g - 1) + 1];
    void* Cg = const_cast<void*>(group_operands[3 * (g - 1) + 2]);
    if (t.swapped) std::swap(Ag, Bg);
    if (!Ag || !Bg || !Cg || (reinterpret_cast<uintptr_t>(Cg) & 15)) return fail(MTF_ERR_INVALID_ARG, "grouped launch: NULL or misaligned operand");
    s = t.a_mn_major ? make_map(&extra.m[2 * (g - 1)], Ag, 2, t.M, t.K, t.a_ld, 64, BK, t, t.outer_sA) : make_map(&extra.m[2 * (g - 1)], Ag, 2, t.K, t.M, t.a_ld, 64, BM / cn, t, t.outer_sA);
    if (s != MTF_OK) return s;
    s = t.b_mn_major ? make_map(&extra.m[2 * (g - 1) + 1], Bg, 2, t.N, t.K, t.b_ld, 64, BK, t, t.outer_sB) : make_map(&extra.m[2 * (g - 1) + 1], Bg, 2, t.K, t.N, t.b_ld, 64, b_rows, t, t.outer_sB);
    if (s != MTF_OK) return s;
    if ((s = make_map(&extra.c[g - 1], Cg, c_bytes, t.N, t.M, t.ldc, 128 / c_bytes, 32, t, t.outer_sC)) != MTF_OK) return s;
    a.C_group[g - 1] = Cg;
  }
  map_m = map_c;
  if (a.mask_tma && (s = make_map(&map_m, mask, 2, t.N, t.M, t.ldc, 64, 32, t, t.outer_sC)) != MTF_OK) return s;
  if (a.resid_tma && (s = make_map(&map_m, resid, c_bytes, t.N, t.M, t.ldc, 128 / c_bytes, 32, t, t.outer_sC)) != MTF_OK) return s;
  CUtensorMap map_w = map_c;      // (spare tensor-map slot of the kernel)

  // epilogue kind: the common combinations have kernels of their own, everything else (and every
  // launch that assembles tiles from fragments) takes the generic one
  int epi = EPI_GENERIC;
  if (row_softmax) epi = row_softmax >= 3 ? EPI_ROW_SOFTMAX_BWD : EPI_ROW_SOFTMAX;
  else if (row_lse) epi = EPI_ROW_LSE_BF16;
  else if (!resid && !bias && !relu && !mask && !rsum) epi = a.c_bf16 ? EPI_PLAIN_BF16 : EPI_PLAIN_F32;
  else if (scale == 1.f && !resid) {
    if (!bias && !relu && !mask && !rsum) epi = a.c_bf16 ? EPI_PLAIN_BF16 : EPI_PLAIN_F32;
    else if (a.ws_partials) epi = EPI_GENERIC;
    else if (bias && !a.bias_along_m && relu && !mask && !rsum && a.c_bf16) epi = EPI_BIAS_RELU_BF16;
    else if (a.mask_tma && rsum && !bias && !relu) epi = EPI_MASK_RSUM_BF16;
  }
  mtf_status ls;
  if (row_softmax >= 3) {
    if (wide) ls = launch_variant<true, 1, 1, EPI_ROW_SOFTMAX_BWD, true>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    else if (t.cta_pair) ls = launch_variant<true, 1, 1, EPI_ROW_SOFTMAX_BWD, false>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    else ls = launch_variant<false, 1, 1, EPI_ROW_SOFTMAX_BWD, false>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
  } else if (row_softmax) {
    if (wide) ls = launch_variant<true, 1, 1, EPI_ROW_SOFTMAX, true>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    else if (t.cta_pair) ls = launch_variant<true, 1, 1, EPI_ROW_SOFTMAX, false>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    else ls = launch_variant<false, 1, 1, EPI_ROW_SOFTMAX, false>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
  } else if (wide) {
    if (epi == EPI_PLAIN_BF16) ls = launch_variant<true, 1, 1, EPI_PLAIN_BF16, true>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    else if (epi == EPI_PLAIN_F32) ls = launch_variant<true, 1, 1, EPI_PLAIN_F32, true>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
    else ls = launch_variant<true, 1, 1, EPI_GENERIC, true>(map_a, map_b, map_c, map_m, map_w, extra, a, st);
  } else if (!t.cta_pair) ls = launch_kind<false, 1, 1, true>(epi, map_a, map_b, map_c, map_m, map_w, extra, a, st);
#if defined(MTF_CLUSTER_SHARE)
  else if (cm == 1 && cn == 2) ls = launch_kind<true, 1, 2, false>(epi, map_a, map_b, map_c, map_m, map_w, extra, a, st);
  else if (cm == 2 && cn == 1) ls = launch_kind<true, 2, 1, false>(epi, map_a, map_b, map_c, map_m, map_w, extra, a, st);
#endif
  else ls = launch_kind<true, 1, 1, true>(epi, map_a, map_b, map_c, map_m, map_w, extra, a, st);
  if (ls != MTF_OK) return ls;
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "gemm_tcgen05_kernel: %s", cudaGetErrorString(e));
  if (a.rsum_partial) return launch_colsum_finalize(a.rsum_partial, (int)rsum_groups, 1, (int)t.N, rsum, nullptr, stream);
  return MTF_OK;
}

// ---- built-in scratch for callers that cannot allocate device memory ---------------------------------
// Some callers run where no device allocation may happen: code replayed inside an already captured
// stream, plug-ins that are handed tensors but no allocator, real-time loops that forbid anything
// that may synchronise the device.  For them the workspace-mode contraction can run on scratch that
// is part of the library image: a fixed array every GPU that loads the library holds until exit.
constexpr size_t kBuiltinScratchBytes = 32u << 20;     // 32 MiB
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

size_t builtin_scratch_capacity() { return kBuiltinScratchBytes; }

int device_sm_count() { return sm_count(); }

// The array's name is only a host-side handle; the device address comes from the runtime, once per
// device, with that device current.
mtf_status builtin_scratch_ptr(void** out) {
  static std::mutex mu;
  static void* cached[kMaxDevices] = {nullptr};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(MTF_ERR_UNSUPPORTED, "device ordinal %d outside [0, %d)", dev, kMaxDevices);
  std::lock_guard<std::mutex> lock(mu);
  if (!cached[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_builtin_scratch);
    if (e != cudaSuccess || !p) return fail(MTF_ERR_CUDA, "cudaGetSymbolAddress(built-in scratch): %s", cudaGetErrorString(e));
    cached[dev] = p;
  }
  *out = cached[dev];
  return MTF_OK;
}

// Testing hook: limit of the bounded device-side waits in SM cycles (<= 0: the default of about two seconds) and,
// with skip_first_commit != 0, a signal that is deliberately never sent (see g_skip_first_commit).
mtf_status debug_wait_test(long long limit_cycles, int skip_first_commit) {
  const long long lim = limit_cycles > 0 ? limit_cycles : kTimeoutCycles;
  cudaError_t e = cudaMemcpyToSymbol(g_wait_limit, &lim, sizeof(lim));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_skip_first_commit, &skip_first_commit, sizeof(int));
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemcpyToSymbol: %s", cudaGetErrorString(e));
  return MTF_OK;
}

mtf_status read_device_status(int* code) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaDeviceSynchronize: %s", cudaGetErrorString(e));
  int v = 0;
  e = cudaMemcpyFromSymbol(&v, g_status, sizeof(int));
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemcpyFromSymbol: %s", cudaGetErrorString(e));
  if (v != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_status, &zero, sizeof(int));
    sched_clear_all();      // a launch that gave up may have left its tile counter behind
  }
  if (code) *code = v;
  if (v != 0) return fail(MTF_ERR_TIMEOUT, "a bounded device-side wait gave up (code 0x%x)", v);
  return MTF_OK;
}

}  // namespace mtf
