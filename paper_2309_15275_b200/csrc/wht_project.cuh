// Shared between the two projection kernels (additions-only and tensor-pipe).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "lbp_internal.h"

namespace lbp {

// One launch projects up to two tensors that share the token grid (x and g_y of
// a layer): items [0, n_items0) belong to tensor 0, the rest to tensor 1.
struct ProjParams {
  int32_t nb, Hb, Wb, r;
  int32_t bpt, tile_rows;
  int32_t C[2], n_chunks[2];
  uint32_t n_items0, n_items;   // nb * n_chunks[0], nb * (n_chunks[0] + n_chunks[1])
  uint32_t* status;
  // factor applied to the +-1 sums of tensor 0 / 1: 1/k gives the orthonormal
  // coefficients of Eq. 6; the products kernel asks for other powers of two
  float scale[2];
  // 0: wait for the preceding kernel on the stream before the first access;
  // 1: the caller vouches that nothing this kernel touches is touched by that
  // kernel, and the wait moves to the end (it then only keeps completion ordered)
  int32_t defer_wait;
  // failure-injection hook of the test suite (lbp_test_stall_products, bit 1):
  // the TMA producers of the tcgen05 projection issue no load, so the other
  // roles run into their bounded waits
  int32_t test_stall;
};

template <int K, bool BF16>
struct ProjCfg {
  static constexpr int kTileBytesMax = K * K * 128;
  static constexpr int kWarps = (K == 16) ? 6 : 12;
  static constexpr int kStages = (K == 4) ? 4 : (K == 8 ? 2 : 1);
  static constexpr int kSmemBytes = kWarps * kStages * kTileBytesMax + kWarps * kStages * 8 + 128;
};

// Tensor-pipe projection (bf16 data): supported ranks per order.
bool project_mma_supported(int k, int r);
// Order 4 at low rank: items are strips of four blocks (4 x 16 token boxes).
bool project_mma_strips(int k, int r);
int launch_project_mma(const CUtensorMap* tmaps, __nv_bfloat16* out0, __nv_bfloat16* out1,
                       const ProjParams& p, const BasisPlan& bp, int sms, cudaStream_t stream);
// Orders 8 and 16, r <= 48 on the tcgen05 tensor cores (boxes of 64 tokens; in the
// parameters n_chunks counts items of four 64-channel chunks per block).
bool project_umma_supported(int k, int r);
int launch_project_umma(const CUtensorMap* tmaps, __nv_bfloat16* out0, __nv_bfloat16* out1,
                        const ProjParams& p, const BasisPlan& bp, int sms, cudaStream_t stream);
// Grid size and launch attributes of a projection launch under the per-thread
// launch shape (see ProjLaunch): `want` CTAs at most.
int projection_grid(uint32_t want, int sms, cudaLaunchAttribute* attr, unsigned* n_attr);

}  // namespace lbp
