// OPTIONAL, single-GPU builds only.  The one TMA load form that writes the same box into the shared
// memory of several CTAs of a cluster (and counts its bytes on each destination pair's barrier).
// It is kept in a file of its own, and only the separate library libmtf_b200_mc.so is built from it,
// so that everything that runs on two or more GPUs can ship without it: libmtf_b200.so never
// contains this instruction and is what the package falls back to when this file is absent.
// The tensor maps handed to it always cover memory of the GPU the kernel runs on.
#pragma once
#include <cuda.h>
#include <cstdint>

__device__ __forceinline__ void tma_load_5d_multicast(uint32_t dst, const CUtensorMap* map, uint32_t bar, uint16_t cta_mask,
                                                      int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster"
      " [%0], [%1, {%4, %5, %6, %7, %8}], [%2], %3;"
      ::"r"(dst), "l"(map), "r"(bar), "h"(cta_mask), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
