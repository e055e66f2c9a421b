// OPTIONAL, single-GPU builds only: operand tiles shared between the CTA pairs of a cluster.
//
// This header holds the one TMA load form that writes a box into the shared memory of several CTAs
// of a cluster (counting its bytes on each destination pair's barrier), the two producer hooks of the
// contraction kernel that use it, and the host check that goes with them.  Only libmtf_b200_mc.so is
// built from it (the build force-includes it into the contraction kernel's translation unit, which
// defines MTF_CLUSTER_SHARE); libmtf_b200.so never contains the instruction and no other source file
// names it, so everything that may run on two or more GPUs ships and works without this file.
//
// Rules that hold for every use:
//   * the tensor maps handed to these loads cover memory of the GPU the kernel runs on, and nothing
//     else: cluster_share_operands_local() asks the runtime where both operands live and the launcher
//     falls back to unshared loads unless both are ordinary device allocations of the current device;
//   * only a process that drives exactly one GPU may load the library built from this file (the
//     Python binding asks for an explicit opt-in and refuses it when more than one device is visible
//     or a multi-rank launcher's variables are set).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

#define MTF_CLUSTER_SHARE 1

__device__ __forceinline__ void tma_load_5d_multicast(uint32_t dst, const CUtensorMap* map, uint32_t bar, uint16_t cta_mask,
                                                      int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
      " [%0], [%1, {%4, %5, %6, %7, %8}], [%2], %3;"
      ::"r"(dst), "l"(map), "r"(bar), "h"(cta_mask), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

// This CTA's 1/CN share of its 128 rows of A goes to the same-position CTA of every pair in its
// cluster row (pm, pn: the pair's row / column in the cluster; rows_share = 128 / CN).
__device__ __forceinline__ void cluster_share_load_a(uint32_t sa, const CUtensorMap* pa, uint32_t bar, int pm, int pn, int CN, int cta_rank,
                                                     int a_mn_major, int rows_share, int m0, int k0, int o2, int o1, int o0) {
  uint16_t mask = 0;
  for (int j = 0; j < CN; ++j) mask |= (uint16_t)(1u << (2 * (pm * CN + j) + cta_rank));
  if (a_mn_major) tma_load_5d_multicast(sa + 8192u * pn, pa, bar, mask, m0 + 64 * pn, k0, o2, o1, o0);
  else tma_load_5d_multicast(sa + (uint32_t)(pn * rows_share) * 128u, pa, bar, mask, k0, m0 + pn * rows_share, o2, o1, o0);
}

// This CTA's 1/CM share of its half of B's columns goes to the same-position CTA of every pair in
// its cluster column (cols_share = columns of B this CTA stages / CM).
__device__ __forceinline__ void cluster_share_load_b(uint32_t sb, const CUtensorMap* pb, uint32_t bar, int pm, int pn, int CM, int CN, int cta_rank,
                                                     int b_mn_major, int cols_share, int n0, int k0, int o2, int o1, int o0) {
  uint16_t mask = 0;
  for (int j = 0; j < CM; ++j) mask |= (uint16_t)(1u << (2 * (j * CN + pn) + cta_rank));
  if (b_mn_major) tma_load_5d_multicast(sb + 8192u * pm, pb, bar, mask, n0 + 64 * pm, k0, o2, o1, o0);
  else tma_load_5d_multicast(sb + (uint32_t)(pm * cols_share) * 128u, pb, bar, mask, k0, n0 + pm * cols_share, o2, o1, o0);
}

// Host: true only when both operands are plain device allocations of the current device (not host,
// managed, peer or imported memory).  Anything else keeps the launch on unshared loads.
static inline bool cluster_share_operands_local(const void* A, const void* B) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  for (const void* p : {A, B}) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    if (at.type != cudaMemoryTypeDevice || at.device != dev) return false;
  }
  return true;
}
