// Backward pass of the attention core of the Transformer layout (Section 9: batch and heads are the split
// dimensions, every (batch, head) pair is an independent problem) in ONE launch.  With the stored weights P and
// the incoming do:
//     dP[l, m]   = sum_v do[l, v] vv[m, v]
//     D[l]       = sum_m dP[l, m] P[l, m]                     (the softmax-backward row term, from the unrounded dP)
//     dS[l, m]   = P[l, m] (dP[l, m] - D[l])                  (gradient of the logits before the scale)
//     dvv[m, v]  = sum_l P[l, m] do[l, v]
//     dq[l, k]   = scale * sum_m dS[l, m] kk[m, k]
//     dkk[m, k]  = scale * sum_l dS[l, m] q[l, k]
// dP and dS never leave the chip: dP lives in tensor memory, dS is written as bf16 over the shared-memory tile
// of P it was made from (once the dvv MMAs have read that tile) and is the A operand of the two contractions
// that consume it.  The weights are read from HBM exactly once.
// d_k = d_v = 64, length = memory_length in {128, 256, 384, 512}; other shapes take the launch-per-einsum path.
// A causal P holds zeros right of the diagonal, so dS is zero there without being told; the blocks that lie
// wholly right of it are skipped.
//
// A persistent CTA (one per SM) walks (batch, head) pairs.  For a pair the work is cut into steps (j, i): key
// block j (128 keys, outer loop), query block i (128 queries), and the steps are walked twice.  Pass 0 forms the row
// terms: D[l] = sum_m dP[l, m] P[l, m] = sum_v do[l, v] O[l, v] with O = P vv, so the MMA thread alone accumulates the
// unrounded O_i = sum_j P_ij vv_j in fp32 in the tensor-memory columns that hold dq_i afterwards, and when the pass ends
// every warp multiplies its rows of O with its rows of do (read from global memory).  Pass 1 computes dP (four MMAs per
// step) and everything else.  The second read of a tile of P comes from L2 or HBM.
// Tensor memory (512 columns):
//   [0, 256)    pass 0: O of the (up to) four query blocks; pass 1: dq of the same blocks, accumulated over j
//   [256, 320)  dkk of key block j, [320, 384) dvv of key block j, accumulated over i
//   [384, 512)  dP of the current step (rows of at most 256: dq ends at column 128 and [128, 256) is a second dP buffer)
// Warp roles (320 threads):
//   warp 0     TMA producer: V_j (both passes) and K_j (pass 1) per key block; the 128 x 128 tile of P per step, q_i and do_i
//              per step of pass 1 (rings of three)
//   warp 1     MMA issuer:   pass 0: O_i += P_ij vv_j; pass 1: dP and dvv += P^T do of the NEXT step as soon as this step's dP
//                            has been read out of tensor memory, then this step's dkk += dS^T q, dq_i += dS kk_j
//   warps 2-9  two per tensor-memory lane quarter (each owns 64 of the step's 128 key columns): the row terms, dS from dP
//              and P, and the read-out of finished accumulators to HBM
// Every mbarrier wait is bounded; on expiry a code is recorded in the status word, a CTA-wide abort flag is
// raised, the remaining waits return at once and all roles leave through the teardown.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "mtf_internal.h"

namespace {

constexpr int kCompWarps = 8;
constexpr int kThreads = 64 + 32 * kCompWarps;
constexpr uint32_t kBox = 128 * 64 * 2;           // one 128-row x 64-column bf16 box (128-byte rows, 128B swizzle)
constexpr int kMaxL = 512;
constexpr long long kWaitCycles = 4000000000LL;
// shared memory (from a 1024-byte aligned base): K | V | q[3] | do[3] | P[3] (two boxes each; dS overwrites P in place) | barriers
constexpr int kRing = 3;
constexpr uint32_t kOffK = 0, kOffV = kBox, kOffQ = 2 * kBox, kOffDO = 5 * kBox, kOffP = 8 * kBox, kOffBars = 14 * kBox;
constexpr int kNumBars = 32;
constexpr size_t kSmemBytes = 1024 + kOffBars + kNumBars * 8 + 64;
// tensor-memory columns
constexpr uint32_t kColDK = 256, kColDV = 320, kColDP = 384;

enum { B_K_FULL = 0, B_K_EMPTY, B_V_FULL, B_V_EMPTY, B_DP_FULL /*2*/, B_DP_EMPTY = 6 /*2*/, B_DKV_FULL = 8, B_DKV_EMPTY, B_DQ_FULL, B_DQ_EMPTY, B_D_SYNC /*O of a pair complete*/,
       B_QDO_FULL = 13 /*3*/, B_QDO_EMPTY = 16 /*3*/, B_P_FULL = 19 /*3*/, B_P_EMPTY = 22 /*3*/, B_PV_DONE = 25 /*3*/, B_DS_FULL = 28 /*3*/ };

__device__ int g_attb_status = 0;

struct BwdArgs {
  int B, H, L;
  int causal;
  float scale;
  const __nv_bfloat16* dout;     // [B, L, H, 64]: read directly for the row terms
  __nv_bfloat16* ds_dump;        // [B, H, L, L] or NULL: where the gradient of the logits is written as well (testing)
  __nv_bfloat16* dq;             // [B, L, H, 64]
  __nv_bfloat16* dk;
  __nv_bfloat16* dv;
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
      atomicCAS(&g_attb_status, 0, code);
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
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
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
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, "
      "%26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]),
        "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]),
        "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st4(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Shared-memory matrix descriptor of a 128B-swizzled tile whose rows are 128 bytes (64 bf16):
//   K-major  (a row holds 64 k-elements of one m/n index; 8-row groups 1024 bytes apart)
//   MN-major (a row holds 64 m/n-elements of one k index; 8-row groups 1024 bytes apart; the next 64 m/n-elements
//             start `block_bytes` further on)
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, int mn_major, uint32_t block_bytes) {
  const uint64_t lbo = mn_major ? (uint64_t)(block_bytes >> 4) : 1u;
  const uint64_t sbo = 1024u >> 4;
  return (uint64_t)((addr & 0x3FFFF) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint32_t idesc_of(int a_mn, int b_mn, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h2);
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

// The steps of this CTA in order: pairs u = blockIdx.x, + gridDim.x, ...; per pair two passes (0: the row terms D, 1: the
// gradients); per pass key blocks j, per key block query blocks i (under the causal limit from j on).  Every role walks
// the same sequence.
struct StepIter {
  long long u, units, stride;
  int nb, causal;
  int pass, j, i;
  long long step_seq, s1_seq, kv_seq, k_seq, unit_seq;      // counts of steps / steps of pass 1 / key blocks (both passes) / key blocks of pass 1 / pairs before this one
  long long dpu0;                    // dP tiles before this step (one per step of pass 1)
  // Rows of at most 256 leave tensor-memory columns [128, 256) free (dq takes 64 per query block): dP then alternates
  // between two buffers, so the next step's dP is computed while the warps still read this one.
  __device__ int dp_buf() const { return nb <= 2 ? (int)(dpu0 & 1) : 0; }
  __device__ long long dp_use() const { return nb <= 2 ? (dpu0 >> 1) : dpu0; }      // earlier uses of this step's buffer
  __device__ uint32_t dp_col() const { return dp_buf() ? 128u : 384u; }
  bool valid;
  __device__ void init(long long first, long long stride_, long long units_, int nb_, int causal_) {
    u = first; stride = stride_; units = units_; nb = nb_; causal = causal_;
    pass = 0; j = 0; i = 0; step_seq = 0; s1_seq = 0; kv_seq = 0; k_seq = 0; unit_seq = 0; dpu0 = 0;
    valid = u < units;
  }
  // dP exists in pass 1 only, in one buffer
  __device__ bool last_of_pass0() const { return pass == 0 && j == nb - 1 && i == nb - 1; }
  __device__ bool first_i() const { return i == (causal ? j : 0); }
  __device__ bool last_i() const { return i == nb - 1; }
  __device__ bool first_of_unit() const { return pass == 0 && j == 0 && first_i(); }
  __device__ bool last_of_unit() const { return pass == 1 && j == nb - 1 && i == nb - 1; }
  __device__ void advance() {
    if (pass == 1) ++dpu0;
    ++step_seq;
    if (pass == 1) ++s1_seq;
    if (i + 1 < nb) { ++i; return; }
    ++kv_seq;
    if (pass == 1) ++k_seq;
    if (j + 1 < nb) { ++j; i = causal ? j : 0; return; }
    j = 0; i = 0;
    if (pass == 0) { pass = 1; return; }
    pass = 0;
    ++unit_seq;
    u += stride;
    valid = u < units;
  }
};

__global__ void __launch_bounds__(kThreads, 1)
attention_bwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const __grid_constant__ CUtensorMap map_do, const __grid_constant__ CUtensorMap map_p, const BwdArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = s_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int L = a.L, nb = L / 128;
  const uint32_t sK = base + kOffK, sV = base + kOffV, sQ = base + kOffQ, sDO = base + kOffDO, sP = base + kOffP;
  const uint32_t bar0 = base + kOffBars;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + kOffBars + kNumBars * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kNumBars; ++i) mb_init(bar(i), 1);
    mb_init(bar(B_DP_EMPTY), kCompWarps); mb_init(bar(B_DP_EMPTY + 1), kCompWarps);
    for (int i = 0; i < kRing; ++i) mb_init(bar(B_DS_FULL + i), kCompWarps);
    mb_init(bar(B_DKV_EMPTY), kCompWarps);
    mb_init(bar(B_DQ_EMPTY), kCompWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_do) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_p) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      StepIter it, pf;
      it.init(blockIdx.x, gridDim.x, a.units, nb, a.causal);
      // the tiles of P are asked into L2 kPrefetch steps before their load into shared memory is issued: the rings hold
      // two steps' worth of loads in flight, which alone does not cover the latency of HBM
      constexpr int kPrefetch = 6;
      pf = it;
      auto prefetch_p = [&](const StepIter& t) {
        const int pb = (int)(t.u / a.H), ph = (int)(t.u % a.H);
        tma_prefetch_4d(&map_p, t.j * 128, t.i * 128, ph, pb);
        tma_prefetch_4d(&map_p, t.j * 128 + 64, t.i * 128, ph, pb);
      };
      for (int n = 0; n < kPrefetch && pf.valid; ++n) { prefetch_p(pf); pf.advance(); }
      bool ok = true;
      while (ok && it.valid) {
        const int b = (int)(it.u / a.H), h = (int)(it.u % a.H);
        if (pf.valid) { prefetch_p(pf); pf.advance(); }
        const int slot = (int)(it.step_seq % kRing);
        const uint32_t par = (uint32_t)(it.step_seq / kRing) & 1u;
        const uint32_t kvpar = (uint32_t)it.kv_seq & 1u;
        if (it.first_i()) {      // a new key block: V first (the next step's dP wants it), K after this step's tiles
          if (!(ok = mb_wait(bar(B_V_EMPTY), kvpar ^ 1u, 0xA01, abort_flag))) break;
          mb_expect(bar(B_V_FULL), kBox);
          tma_load_4d(sV, &map_v, bar(B_V_FULL), 0, it.j * 128, h, b);
        }
        if (!(ok = mb_wait(bar(B_QDO_EMPTY + slot), par ^ 1u, 0xA02, abort_flag))) break;
        mb_expect(bar(B_QDO_FULL + slot), it.pass == 0 ? 0u : 2 * kBox);       // (pass 0 needs neither: the phase completes at once)
        if (it.pass == 1) {
          tma_load_4d(sQ + slot * kBox, &map_q, bar(B_QDO_FULL + slot), 0, it.i * 128, h, b);
          tma_load_4d(sDO + slot * kBox, &map_do, bar(B_QDO_FULL + slot), 0, it.i * 128, h, b);
        }
        if (!(ok = mb_wait(bar(B_P_EMPTY + slot), par ^ 1u, 0xA03, abort_flag))) break;
        mb_expect(bar(B_P_FULL + slot), 2 * kBox);
        tma_load_4d(sP + slot * 2 * kBox, &map_p, bar(B_P_FULL + slot), it.j * 128, it.i * 128, h, b);
        tma_load_4d(sP + slot * 2 * kBox + kBox, &map_p, bar(B_P_FULL + slot), it.j * 128 + 64, it.i * 128, h, b);
        if (it.pass == 1 && it.first_i()) {
          if (!(ok = mb_wait(bar(B_K_EMPTY), ((uint32_t)it.k_seq & 1u) ^ 1u, 0xA04, abort_flag))) break;
          mb_expect(bar(B_K_FULL), kBox);
          tma_load_4d(sK, &map_k, bar(B_K_FULL), 0, it.j * 128, h, b);
        }
        it.advance();
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer ---------------------------------
    if (lane == 0) {
      StepIter cur, nxt;
      cur.init(blockIdx.x, gridDim.x, a.units, nb, a.causal);
      nxt = cur;
      if (nxt.valid) nxt.advance();
      long long n_dp = 0;                      // dP tiles issued so far (one per step of pass 1)
      long long n_dv = 0;                      // dvv contributions issued so far (one per step of pass 1)
      bool ok = true;
      const uint32_t id_dp = idesc_of(0, 0, 128), id_kv = idesc_of(1, 1, 64), id_dq = idesc_of(0, 1, 64);
      // pass 0, one step: O_i += P_ij vv_j (M = queries, N = d_v, k = keys; A K-major over two 64-key boxes, B MN-major) into the
      // columns where dq_i will accumulate in pass 1.  Nothing of it concerns the warps until the pass ends.
      auto issue_o = [&](const StepIter& t) -> bool {
        const int slot = (int)(t.step_seq % kRing);
        const uint32_t par = (uint32_t)(t.step_seq / kRing) & 1u;
        if (t.first_of_unit() && !mb_wait(bar(B_DQ_EMPTY), ((uint32_t)t.unit_seq & 1u) ^ 1u, 0xB08, abort_flag)) return false;   // the previous pair's dq has been read out
        if (t.first_i() && !mb_wait(bar(B_V_FULL), (uint32_t)t.kv_seq & 1u, 0xB01, abort_flag)) return false;
        if (!mb_wait(bar(B_QDO_FULL + slot), par, 0xB02, abort_flag)) return false;      // (an empty phase in pass 0: keeps the ring's phases in step)
        if (!mb_wait(bar(B_P_FULL + slot), par, 0xB04, abort_flag)) return false;
        fence_after();
        const uint64_t da = smem_desc(sP + slot * 2 * kBox, 0, 0), db = smem_desc(sV, 1, kBox);
        const uint32_t acc = t.j != 0 ? 1u : 0u;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          umma(tmem + (uint32_t)t.i * 64u, da + (uint64_t)((ks >> 2) * (kBox >> 4) + (ks & 3) * 2), db + (uint64_t)(ks * (2048 >> 4)), id_dq, acc | (uint32_t)ks);
        umma_commit(bar(B_P_EMPTY + slot));
        umma_commit(bar(B_QDO_EMPTY + slot));
        if (t.last_i()) umma_commit(bar(B_V_EMPTY));
        if (t.last_of_pass0()) umma_commit(bar(B_D_SYNC));      // every O_i of the pair is complete
        return true;
      };
      // dP of a step of pass 1: wants do of the step, V of its key block and the dP columns read out by the warps
      auto issue_dp = [&](const StepIter& t) -> bool {
        const int slot = (int)(t.step_seq % kRing);
        const uint32_t par = (uint32_t)(t.step_seq / kRing) & 1u;
        if (t.first_i() && !mb_wait(bar(B_V_FULL), (uint32_t)t.kv_seq & 1u, 0xB01, abort_flag)) return false;
        if (!mb_wait(bar(B_QDO_FULL + slot), par, 0xB02, abort_flag)) return false;
        if (!mb_wait(bar(B_DP_EMPTY + t.dp_buf()), ((uint32_t)t.dp_use() & 1u) ^ 1u, 0xB03, abort_flag)) return false;      // the buffer's previous dP has been read out
        fence_after();
        const uint64_t da = smem_desc(sDO + slot * kBox, 0, 0), db = smem_desc(sV, 0, 0);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) umma(tmem + t.dp_col(), da + 2u * ks, db + 2u * ks, id_dp, ks != 0);
        umma_commit(bar(B_DP_FULL + t.dp_buf()));
        if (t.last_i()) umma_commit(bar(B_V_EMPTY));         // this key block's V is no longer read
        ++n_dp;
        return true;
      };
      // dvv_j += P^T do_i of a step of pass 1 (M = keys, N = d_v, k = queries; both operands MN-major).  It needs nothing
      // from the warps, and once it has run they may overwrite the tile of P with dS.
      auto issue_dv = [&](const StepIter& t) -> bool {
        const int slot = (int)(t.step_seq % kRing);
        const uint32_t par = (uint32_t)(t.step_seq / kRing) & 1u;
        if (!mb_wait(bar(B_P_FULL + slot), par, 0xB04, abort_flag)) return false;
        if (t.first_i() && !mb_wait(bar(B_DKV_EMPTY), ((uint32_t)t.k_seq & 1u) ^ 1u, 0xB06, abort_flag)) return false;   // the previous key block's dkk, dvv have been read out
        fence_after();
        const uint64_t da = smem_desc(sP + slot * 2 * kBox, 1, kBox), db = smem_desc(sDO + slot * kBox, 1, kBox);
        const uint32_t acc = t.first_i() ? 0u : 1u;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) umma(tmem + kColDV, da + (uint64_t)(ks * (2048 >> 4)), db + (uint64_t)(ks * (2048 >> 4)), id_kv, acc | (uint32_t)ks);
        umma_commit(bar(B_PV_DONE + (int)(t.s1_seq % kRing)));
        ++n_dv;
        return true;
      };
      while (ok && cur.valid) {
        if (cur.pass == 0) {
          if (!(ok = issue_o(cur))) break;
          cur = nxt;
          if (nxt.valid) nxt.advance();
          continue;
        }
        const int slot = (int)(cur.step_seq % kRing);
        if (n_dp == cur.s1_seq && !(ok = issue_dp(cur))) break;
        if (n_dv == cur.s1_seq && !(ok = issue_dv(cur))) break;
        // ahead of this step's remaining MMAs: the next step's dP (as soon as the warps have this step's dP in registers)
        // and, inside a key block, its dvv contribution, so that the warps work on the next step while these run
        if (nxt.valid && nxt.pass == 1) {
          if (!(ok = issue_dp(nxt))) break;
          if (!nxt.first_i() && !(ok = issue_dv(nxt))) break;
        }
        const int s1slot = (int)(cur.s1_seq % kRing);
        if (!(ok = mb_wait(bar(B_DS_FULL + s1slot), (uint32_t)(cur.s1_seq / kRing) & 1u, 0xB05, abort_flag))) break;      // dS stands where P stood
        if (cur.first_i() && !(ok = mb_wait(bar(B_K_FULL), (uint32_t)cur.k_seq & 1u, 0xB07, abort_flag))) break;
        fence_after();
        const uint32_t acc_kv = cur.first_i() ? 0u : 1u;
        const uint32_t dsS = sP + slot * 2 * kBox, qS = sQ + slot * kBox;
        {   // dkk_j += dS^T q_i
          const uint64_t da = smem_desc(dsS, 1, kBox), db = smem_desc(qS, 1, kBox);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) umma(tmem + kColDK, da + (uint64_t)(ks * (2048 >> 4)), db + (uint64_t)(ks * (2048 >> 4)), id_kv, acc_kv | (uint32_t)ks);
        }
        {   // dq_i += dS kk_j     (M = queries, N = d_k, k = keys; A K-major over two 64-key boxes, B MN-major)
          const uint64_t da = smem_desc(dsS, 0, 0), db = smem_desc(sK, 1, kBox);
          const uint32_t acc_q = cur.j != 0 ? 1u : 0u;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            umma(tmem + (uint32_t)cur.i * 64u, da + (uint64_t)((ks >> 2) * (kBox >> 4) + (ks & 3) * 2), db + (uint64_t)(ks * (2048 >> 4)), id_dq, acc_q | (uint32_t)ks);
        }
        umma_commit(bar(B_P_EMPTY + slot));
        umma_commit(bar(B_QDO_EMPTY + slot));
        if (cur.last_i()) { umma_commit(bar(B_DKV_FULL)); umma_commit(bar(B_K_EMPTY)); }
        if (cur.last_of_unit()) umma_commit(bar(B_DQ_FULL));
        cur = nxt;
        if (nxt.valid) nxt.advance();
      }
    }
  } else {
    // ------------------------------- dS and read-out warps ----------------------
    const int q = warp & 3;                        // tensor-memory lane quarter this warp may access
    const int half = (warp - 2) >> 2;              // which 64 of the step's 128 key columns
    const int row_l = q * 32 + lane;               // row inside a 128-row block
    const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16);
    const uint32_t sw = (uint32_t)(row_l & 7);
    auto wait_all = [&](int b, uint32_t parity, int code) -> bool {      // all lanes wait (lane 0 polls first)
      int w_ok = 1;
      if (lane == 0) w_ok = mb_wait(bar(b), parity, code, abort_flag) ? 1 : 0;
      w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
      if (!w_ok) return false;
      bool mine_ok = lane == 0 ? true : mb_wait(bar(b), parity, code, abort_flag);
      return __all_sync(0xffffffffu, mine_ok);
    };
    auto store_row = [&](__nv_bfloat16* dst, const uint32_t* r0, const uint32_t* r1, float s) {      // 64 fp32 -> one 128-byte row
      uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
      for (int g = 0; g < 4; ++g)
        d4[g] = make_uint4(pack2(__uint_as_float(r0[g * 8]) * s, __uint_as_float(r0[g * 8 + 1]) * s), pack2(__uint_as_float(r0[g * 8 + 2]) * s, __uint_as_float(r0[g * 8 + 3]) * s),
                           pack2(__uint_as_float(r0[g * 8 + 4]) * s, __uint_as_float(r0[g * 8 + 5]) * s), pack2(__uint_as_float(r0[g * 8 + 6]) * s, __uint_as_float(r0[g * 8 + 7]) * s));
#pragma unroll
      for (int g = 0; g < 4; ++g)
        d4[4 + g] = make_uint4(pack2(__uint_as_float(r1[g * 8]) * s, __uint_as_float(r1[g * 8 + 1]) * s), pack2(__uint_as_float(r1[g * 8 + 2]) * s, __uint_as_float(r1[g * 8 + 3]) * s),
                               pack2(__uint_as_float(r1[g * 8 + 4]) * s, __uint_as_float(r1[g * 8 + 5]) * s), pack2(__uint_as_float(r1[g * 8 + 6]) * s, __uint_as_float(r1[g * 8 + 7]) * s));
    };
    StepIter it;
    it.init(blockIdx.x, gridDim.x, a.units, nb, a.causal);
    float D0 = 0.f, D1 = 0.f, D2 = 0.f, D3 = 0.f;      // D of this thread's row in each of the pair's query blocks
    bool ok = true;
    while (ok && it.valid) {
      const int b = (int)(it.u / a.H), h = (int)(it.u % a.H);
      const int slot = (int)(it.step_seq % kRing);
      const uint32_t par = (uint32_t)(it.step_seq / kRing) & 1u;
      uint32_t r0[32], r1[32];
      if (it.pass == 0) {
        // pass 0 belongs to the MMA thread (O_i = sum_j P_ij vv_j in fp32, in the columns of dq_i).  When it ends, every warp
        // forms the row terms of its rows for all query blocks: D[l] = sum_v do[l, v] O[l, v], which equals sum_m dP[l, m] P[l, m]
        // with the unrounded dP.  (Both warps of a lane quarter do this for the same rows: cheaper than an exchange.)
        if (it.last_of_pass0()) {
          if (!(ok = wait_all(B_D_SYNC, (uint32_t)it.unit_seq & 1u, 0xC06))) break;
          fence_after();
          for (int i2 = 0; i2 < nb; ++i2) {
            tmem_ld32(taddr + (uint32_t)i2 * 64u, r0);
            tmem_ld32(taddr + (uint32_t)i2 * 64u + 32u, r1);
            const uint4* drow = reinterpret_cast<const uint4*>(a.dout + (((long long)b * L + i2 * 128 + row_l) * a.H + h) * 64);
            uint4 dv4[8];
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) dv4[pc] = __ldg(drow + pc);
            tmem_ld_wait();
            float d = 0.f;
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) {
              const uint32_t* rr = pc < 4 ? r0 + pc * 8 : r1 + (pc - 4) * 8;
              d = fmaf(bf_lo(dv4[pc].x), __uint_as_float(rr[0]), d); d = fmaf(bf_hi(dv4[pc].x), __uint_as_float(rr[1]), d);
              d = fmaf(bf_lo(dv4[pc].y), __uint_as_float(rr[2]), d); d = fmaf(bf_hi(dv4[pc].y), __uint_as_float(rr[3]), d);
              d = fmaf(bf_lo(dv4[pc].z), __uint_as_float(rr[4]), d); d = fmaf(bf_hi(dv4[pc].z), __uint_as_float(rr[5]), d);
              d = fmaf(bf_lo(dv4[pc].w), __uint_as_float(rr[6]), d); d = fmaf(bf_hi(dv4[pc].w), __uint_as_float(rr[7]), d);
            }
            if (i2 == 0) D0 = d; else if (i2 == 1) D1 = d; else if (i2 == 2) D2 = d; else D3 = d;
          }
          fence_before();
        }
        it.advance();
        continue;
      }
      if (!(ok = wait_all(B_DP_FULL + it.dp_buf(), (uint32_t)it.dp_use() & 1u, 0xC01))) break;
      fence_after();
      if (!(ok = wait_all(B_P_FULL + slot, par, 0xC02))) break;
      tmem_ld32(taddr + it.dp_col() + (uint32_t)half * 64u, r0);
      tmem_ld32(taddr + it.dp_col() + (uint32_t)half * 64u + 32u, r1);
      tmem_ld_wait();
      fence_before();
      __syncwarp();
      if (lane == 0) mb_arrive(bar(B_DP_EMPTY + it.dp_buf()));            // dP is in registers: the buffer's next dP may overwrite it
      const float Dr = it.i == 0 ? D0 : (it.i == 1 ? D1 : (it.i == 2 ? D2 : D3));
      const uint32_t prow = sP + (uint32_t)slot * 2u * kBox + (uint32_t)half * kBox + (uint32_t)row_l * 128u;
      uint4 out[8];
#pragma unroll
      for (int pc = 0; pc < 8; ++pc) {
        const uint4 pv = lds_v4(prow + ((((uint32_t)pc) ^ sw) << 4));
        const uint32_t* rr = pc < 4 ? r0 + pc * 8 : r1 + (pc - 4) * 8;
        out[pc] = make_uint4(pack2(bf_lo(pv.x) * (__uint_as_float(rr[0]) - Dr), bf_hi(pv.x) * (__uint_as_float(rr[1]) - Dr)),
                             pack2(bf_lo(pv.y) * (__uint_as_float(rr[2]) - Dr), bf_hi(pv.y) * (__uint_as_float(rr[3]) - Dr)),
                             pack2(bf_lo(pv.z) * (__uint_as_float(rr[4]) - Dr), bf_hi(pv.z) * (__uint_as_float(rr[5]) - Dr)),
                             pack2(bf_lo(pv.w) * (__uint_as_float(rr[6]) - Dr), bf_hi(pv.w) * (__uint_as_float(rr[7]) - Dr)));
      }
      const int s1slot = (int)(it.s1_seq % kRing);
      {   // dS goes where this tile of P stands: its last reader, the dvv MMAs of this step, must have run
        int w_ok = 1;
        if (lane == 0) w_ok = mb_wait(bar(B_PV_DONE + s1slot), (uint32_t)(it.s1_seq / kRing) & 1u, 0xC03, abort_flag) ? 1 : 0;
        w_ok = __shfl_sync(0xffffffffu, w_ok, 0);
        if (!w_ok) { ok = false; break; }
      }
      if (a.ds_dump) {      // (testing: the bf16 values the two contractions below consume)
        uint4* dd = reinterpret_cast<uint4*>(a.ds_dump + ((((long long)b * a.H + h) * L + it.i * 128 + row_l) * L + it.j * 128 + half * 64));
#pragma unroll
        for (int pc = 0; pc < 8; ++pc) dd[pc] = out[pc];
      }
      const uint32_t drow = prow;
#pragma unroll
      for (int pc = 0; pc < 8; ++pc) sts_v4(drow + ((((uint32_t)pc) ^ sw) << 4), out[pc].x, out[pc].y, out[pc].z, out[pc].w);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mb_arrive(bar(B_DS_FULL + s1slot));
      if (it.last_i()) {
        // key block j is complete: dkk (scaled) leaves through the warps of column half 0, dvv through those of half 1
        if (!(ok = wait_all(B_DKV_FULL, (uint32_t)it.k_seq & 1u, 0xC04))) break;
        fence_after();
        tmem_ld32(taddr + (half == 0 ? kColDK : kColDV), r0);
        tmem_ld32(taddr + (half == 0 ? kColDK : kColDV) + 32u, r1);
        tmem_ld_wait();
        const long long off = (((long long)b * L + it.j * 128 + row_l) * a.H + h) * 64;
        store_row((half == 0 ? a.dk : a.dv) + off, r0, r1, half == 0 ? a.scale : 1.f);
        fence_before();
        __syncwarp();
        if (lane == 0) mb_arrive(bar(B_DKV_EMPTY));
      }
      if (it.last_of_unit()) {
        if (!(ok = wait_all(B_DQ_FULL, (uint32_t)it.unit_seq & 1u, 0xC05))) break;
        fence_after();
        for (int i2 = half; i2 < nb; i2 += 2) {
          tmem_ld32(taddr + (uint32_t)i2 * 64u, r0);
          tmem_ld32(taddr + (uint32_t)i2 * 64u + 32u, r1);
          tmem_ld_wait();
          const long long off = (((long long)b * L + i2 * 128 + row_l) * a.H + h) * 64;
          store_row(a.dq + off, r0, r1, a.scale);
        }
        fence_before();
        __syncwarp();
        if (lane == 0) mb_arrive(bar(B_DQ_EMPTY));
      }
      it.advance();
    }
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

// bf16 tensor [d3][d2][d1][d0] (d0 contiguous) as a 4-d tensor map with 128B swizzle and boxes of 64 x 128; strides in elements
mtf_status map4(CUtensorMap* m, const void* base, const int64_t dims[4], const int64_t strides[3]) {
  EncodeTiledFn enc = encoder();
  if (!enc) return mtf::fail(MTF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  cuuint64_t d[4] = {(cuuint64_t)dims[0], (cuuint64_t)dims[1], (cuuint64_t)dims[2], (cuuint64_t)dims[3]};
  cuuint64_t s[3] = {(cuuint64_t)strides[0] * 2, (cuuint64_t)strides[1] * 2, (cuuint64_t)strides[2] * 2};
  cuuint32_t box[4] = {64, 128, 1, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), d, s, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return mtf::fail(MTF_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
  return MTF_OK;
}

}  // namespace

namespace mtf {

bool attention_bwd_fused_supported(int64_t L, int64_t d_k, int64_t d_v) { return d_k == 64 && d_v == 64 && L % 128 == 0 && L >= 128 && L <= kMaxL; }

// q, kk, vv, dout, dq, dkk, dvv [B, L, H, 64]; weights [B, H, L, L]; all bf16, dense, 16-byte aligned device pointers.
// dlogits_dump: NULL, or [B, H, L, L] bf16 that also receives the gradient of the logits (before the scale) as the contractions consume it
mtf_status launch_attention_bwd_fused(const void* q, const void* kk, const void* vv, const void* weights, const void* dout, void* dq, void* dkk, void* dvv,
                                      void* dlogits_dump, int64_t B, int64_t H, int64_t L, float scale, int causal, void* stream) {
  if (!attention_bwd_fused_supported(L, 64, 64)) return fail(MTF_ERR_UNSUPPORTED, "fused attention backward: length %lld", (long long)L);
  for (const void* p : {q, kk, vv, weights, dout, (const void*)dq, (const void*)dkk, (const void*)dvv})
    if (!p || (reinterpret_cast<uintptr_t>(p) & 15)) return fail(MTF_ERR_INVALID_ARG, "fused attention backward: NULL or misaligned tensor");
  if (B * H <= 0) return MTF_OK;
  CUtensorMap mq, mk, mv, md, mp;
  const int64_t qd[4] = {64, L, H, B}, qs[3] = {H * 64, 64, L * H * 64};
  const int64_t pd[4] = {L, L, H, B}, ps[3] = {L, L * L, H * L * L};
  mtf_status st;
  if ((st = map4(&mq, q, qd, qs)) != MTF_OK || (st = map4(&mk, kk, qd, qs)) != MTF_OK || (st = map4(&mv, vv, qd, qs)) != MTF_OK ||
      (st = map4(&md, dout, qd, qs)) != MTF_OK || (st = map4(&mp, weights, pd, ps)) != MTF_OK)
    return st;
  BwdArgs a;
  a.B = (int)B; a.H = (int)H; a.L = (int)L; a.causal = causal ? 1 : 0; a.scale = scale;
  a.dout = reinterpret_cast<const __nv_bfloat16*>(dout);
  a.ds_dump = reinterpret_cast<__nv_bfloat16*>(dlogits_dump);
  a.dq = reinterpret_cast<__nv_bfloat16*>(dq);
  a.dk = reinterpret_cast<__nv_bfloat16*>(dkk);
  a.dv = reinterpret_cast<__nv_bfloat16*>(dvv);
  a.units = B * H;
  if (dlogits_dump && causal) {      // the blocks the kernel skips under the hint hold zeros
    cudaError_t ze = cudaMemsetAsync(dlogits_dump, 0, (size_t)B * H * L * L * 2, (cudaStream_t)stream);
    if (ze != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(ze));
  }
  cudaError_t e = cudaFuncSetAttribute(attention_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  // Blocks 2k and 2k + 1 are launched as a cluster only so that they sit on the two SMs of one TPC: the blocks whose
  // share of the pairs is one round shorter are the last ones, and when they leave, whole TPCs become free for the CTA
  // pairs of an independent contraction launched behind this kernel.  The kernel itself uses nothing of the cluster.
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = 2; at[1].val.clusterDim.y = 1; at[1].val.clusterDim.z = 1;
  const long long grid = std::min<long long>(a.units, device_sm_count());
  cfg.gridDim = dim3((unsigned)grid, 1, 1); cfg.blockDim = dim3(kThreads, 1, 1); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = (cudaStream_t)stream;
  cfg.attrs = at; cfg.numAttrs = grid % 2 == 0 ? 2 : 1;
  e = cudaLaunchKernelEx(&cfg, attention_bwd_kernel, mq, mk, mv, md, mp, a);
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "attention_bwd_kernel: %s", cudaGetErrorString(e));
  count_launch();
  return MTF_OK;
}

mtf_status read_attention_bwd_status(int* code) {
  int v = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&v, g_attb_status, sizeof(int));
  if (e != cudaSuccess) return fail(MTF_ERR_CUDA, "cudaMemcpyFromSymbol: %s", cudaGetErrorString(e));
  if (v != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_attb_status, &zero, sizeof(int));
  }
  *code = v;
  return MTF_OK;
}

}  // namespace mtf
