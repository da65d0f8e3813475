// Pieces shared by the tensor-pipe projection kernel and the spectrum kernel:
// the +-1 basis matrix as mma.sync A fragments, ldmatrix / mma wrappers and the
// per-warp tile ring geometry.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace lbp {

struct MmaPlan {
  uint8_t nat_i[64];
  uint8_t nat_j[64];
};

template <int K>
struct MmaCfg {
  static constexpr int kTokens = K * K;
  static constexpr int kTileBytes = kTokens * 128;
  static constexpr int kKSteps = kTokens / 16;
  static constexpr int kWarps = (K == 16) ? 6 : 12;
  static constexpr int kStages = (K == 4) ? 4 : (K == 8 ? 2 : 1);
  static constexpr int kSmemBytes = kWarps * kStages * kTileBytes + kWarps * kStages * 8 + 1024;
};

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1,
                                                  uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr)
               : "memory");
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                               uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
      "{%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// bf16 bits of the basis entry B_{iq,jq}[tok] (+1, -1) or 0 for a padding row.
template <int K>
__device__ __forceinline__ uint32_t basis_bits(const MmaPlan& mp, int q, int r, int tok) {
  if (q >= r) return 0u;
  const int u = tok / K, v = tok % K;
  const int neg = (__popc(mp.nat_i[q] & u) + __popc(mp.nat_j[q] & v)) & 1;
  return neg ? 0xBF80u : 0x3F80u;
}

}  // namespace lbp
