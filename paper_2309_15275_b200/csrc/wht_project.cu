// Projection kernel (Eq. 6):  t_hat[blk, q, c] = (1/k) sum_{u,v} wal_iq[u] wal_jq[v] t[blk,u,v,c].
//
// HBM-bound streaming pass.  One warp owns a ring of shared-memory stages; lane
// 0 issues one 4-D TMA box per (block, channel chunk) -- k x k tokens by 128
// bytes of channels -- and the warp consumes it with conflict-free 32-bit
// shared loads (a lane owns one word of the channel axis).  The transform is
// additions only: pool to LB x LB, then a natural-order Hadamard butterfly.
#include <cuda_bf16.h>

#include "lbp_fused.cuh"
#include "lbp_internal.h"
#include "ptx_sm100.cuh"
#include "wht_device.cuh"
#include "wht_project.cuh"

namespace lbp {

template <typename T, bool BF16, int NCH>
__device__ __forceinline__ void store_coeff(T* __restrict__ out, long long row, int C, int c0,
                                            int pass, const float (&v)[NCH], float scale) {
  if constexpr (!BF16) {
    out[row * C + c0] = v[0] * scale;
  } else if constexpr (NCH == 2) {
    *reinterpret_cast<uint32_t*>(out + row * C + c0) = pack_bf16x2(v[0] * scale, v[1] * scale);
  } else {
    out[row * C + c0 + pass] = __float2bfloat16_rn(v[0] * scale);
  }
}

template <typename T, int K, int LB>
__global__ void __launch_bounds__(ProjCfg<K, sizeof(T) == 2>::kWarps * 32, 1)
    wht_project_kernel(const __grid_constant__ CUtensorMap tmap0,
                       const __grid_constant__ CUtensorMap tmap1, T* __restrict__ out0,
                       T* __restrict__ out1, const __grid_constant__ ProjParams p,
                       const __grid_constant__ DevicePlan plan) {
  constexpr bool BF16 = sizeof(T) == 2;
  using Cfg = ProjCfg<K, BF16>;
  constexpr int NW = Cfg::kWarps, S = Cfg::kStages;
  constexpr int CH_PER_WORD = BF16 ? 2 : 1;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + NW * S * Cfg::kTileBytesMax);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint64_t* my_bars = bars + warp * S;
  uint8_t* my_tiles = tiles + warp * S * Cfg::kTileBytesMax;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < S; ++s) ptx::mbar_init(&my_bars[s], 1);
    ptx::mbar_fence_init();
  }
  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap0);
    ptx::prefetch_tensormap(&tmap1);
  }
  __syncthreads();

  const uint32_t first = blockIdx.x * NW + warp;
  const uint32_t stride = gridDim.x * NW;
  const uint32_t n_my = first < p.n_items ? (p.n_items - first + stride - 1) / stride : 0;
  constexpr int ch_per_tile = 32 * CH_PER_WORD;   // a token is 128 B = 32 words wide in a tile
  constexpr int tw = 32;

  auto issue = [&](uint32_t idx, int s) {
    uint32_t item = first + idx * stride;
    const int which = item >= p.n_items0;
    if (which) item -= p.n_items0;
    const uint32_t nch = static_cast<uint32_t>(p.n_chunks[which]);
    const uint32_t blk = item / nch, chunk = item - blk * nch;
    const uint32_t bw = blk % p.Wb, t2 = blk / p.Wb, bh = t2 % p.Hb, b = t2 / p.Hb;
    ptx::mbar_expect_tx(&my_bars[s], static_cast<uint32_t>(Cfg::kTileBytesMax));
    ptx::tma_load_4d(my_tiles + s * Cfg::kTileBytesMax, which ? &tmap1 : &tmap0, &my_bars[s],
                     chunk * ch_per_tile, bw * K, bh * K, b);
  };

  if (lane == 0) {
    for (uint32_t i = 0; i < S && i < n_my; ++i) issue(i, i);
  }

  for (uint32_t idx = 0; idx < n_my; ++idx) {
    const int s = static_cast<int>(idx % S);
    const uint32_t parity = (idx / S) & 1u;
    const bool ok = ptx::mbar_wait(&my_bars[s], parity, p.status, (1u << 16) | 1u);
    if (!__all_sync(0xffffffffu, ok)) break;

    uint32_t item = first + idx * stride;
    const int which = item >= p.n_items0;
    if (which) item -= p.n_items0;
    const uint32_t nch = static_cast<uint32_t>(p.n_chunks[which]);
    const int blk = static_cast<int>(item / nch);
    const int chunk = static_cast<int>(item - blk * nch);
    const int C = p.C[which];
    T* __restrict__ out = which ? out1 : out0;
    const uint32_t* tile = reinterpret_cast<const uint32_t*>(my_tiles + s * Cfg::kTileBytesMax);
    const int c0 = chunk * ch_per_tile + lane * CH_PER_WORD;
    const bool active = c0 < C;   // channels past C are zero-filled by TMA and skipped
    const long long row0 =
        static_cast<long long>(blk / p.bpt) * p.tile_rows + static_cast<long long>(blk % p.bpt) * p.r;

    if (active) {
      if constexpr (LB < 16) {
        constexpr int RUN = K / LB;
        constexpr int NCH = (BF16 && LB <= 4) ? 2 : 1;
        constexpr int NPASS = (BF16 && NCH == 1) ? 2 : 1;
#pragma unroll 1
        for (int pass = 0; pass < NPASS; ++pass) {
          float acc[LB][LB][NCH];
#pragma unroll
          for (int a = 0; a < LB; ++a)
#pragma unroll
            for (int b = 0; b < LB; ++b)
#pragma unroll
              for (int c = 0; c < NCH; ++c) acc[a][b][c] = 0.f;
#pragma unroll
          for (int u = 0; u < K; ++u) {
#pragma unroll
            for (int v = 0; v < K; ++v) {
              float f[NCH];
              unpack_word<BF16, NCH>(tile[(u * K + v) * tw + lane], pass, f);
#pragma unroll
              for (int c = 0; c < NCH; ++c) acc[u / RUN][v / RUN][c] += f[c];
            }
            // keep the 256 loads of an order-16 block from being hoisted together
            if constexpr (K == 16) asm volatile("" ::: "memory");
          }
          hadamard_rows<LB, NCH>(acc);
          hadamard_cols<LB, NCH>(acc);
#pragma unroll
          for (int a = 0; a < LB; ++a) {
#pragma unroll
            for (int b = 0; b < LB; ++b) {
              const int q = plan.qmap[a * LB + b];
              if (q >= 0) store_coeff<T, BF16, NCH>(out, row0 + q, C, c0, pass, acc[a][b], p.scale[which]);
            }
          }
        }
      } else {
        // LB == 16 (K == 16): the 16 x 16 coefficient array does not fit in
        // registers.  Pass n_lo produces the natural-order columns
        // b = 4 * n_hi + n_lo: a sign-combination over the low two bits of v,
        // then a 4-point butterfly over the high two bits, then a 16-point
        // butterfly along u.
        constexpr int NPASS = BF16 ? 2 : 1;
#pragma unroll 1
        for (int pass = 0; pass < NPASS; ++pass) {
#pragma unroll 1
          for (int n_lo = 0; n_lo < 4; ++n_lo) {
            const float s1 = (n_lo & 1) ? -1.f : 1.f;   // sign of v_lo = 1
            const float s2 = (n_lo & 2) ? -1.f : 1.f;   // sign of v_lo = 2
            const float s3 = s1 * s2;                   // sign of v_lo = 3
            float R[4][16];                             // [n_hi][u]
#pragma unroll
            for (int u = 0; u < 16; ++u) {
              float y[4];
#pragma unroll
              for (int vh = 0; vh < 4; ++vh) {
                float f0[1], f1[1], f2[1], f3[1];
                unpack_word<BF16, 1>(tile[(u * 16 + vh * 4 + 0) * tw + lane], pass, f0);
                unpack_word<BF16, 1>(tile[(u * 16 + vh * 4 + 1) * tw + lane], pass, f1);
                unpack_word<BF16, 1>(tile[(u * 16 + vh * 4 + 2) * tw + lane], pass, f2);
                unpack_word<BF16, 1>(tile[(u * 16 + vh * 4 + 3) * tw + lane], pass, f3);
                y[vh] = (f0[0] + s1 * f1[0]) + (s2 * f2[0] + s3 * f3[0]);
              }
              hadamard_vec<4>(y);
#pragma unroll
              for (int nh = 0; nh < 4; ++nh) R[nh][u] = y[nh];
              asm volatile("" ::: "memory");
            }
#pragma unroll
            for (int nh = 0; nh < 4; ++nh) {
              hadamard_vec<16>(R[nh]);
#pragma unroll
              for (int a = 0; a < 16; ++a) {
                const int q = plan.qmap[a * 16 + nh * 4 + n_lo];
                if (q >= 0) {
                  const float v1[1] = {R[nh][a]};
                  store_coeff<T, BF16, 1>(out, row0 + q, C, c0, pass, v1, p.scale[which]);
                }
              }
            }
          }
        }
      }
      // rows of a padded row tile that no block owns are kept at zero
      if ((blk % p.bpt) == p.bpt - 1 || blk == p.nb - 1) {
        const long long tile_base = static_cast<long long>(blk / p.bpt) * p.tile_rows;
        for (long long row = row0 + p.r; row < tile_base + p.tile_rows; ++row) {
          if constexpr (BF16) {
            *reinterpret_cast<uint32_t*>(out + row * C + c0) = 0u;
          } else {
            out[row * C + c0] = 0.f;
          }
        }
      }
    }

    __syncwarp();
    if (lane == 0 && idx + S < n_my) {
      ptx::fence_proxy_async_smem();
      issue(idx + S, s);
    }
  }
}

template <typename T, int K, int LB>
static int launch_one(const CUtensorMap* tmaps, T* out0, T* out1, const ProjParams& p,
                      const DevicePlan& plan, int sms, cudaStream_t stream) {
  using Cfg = ProjCfg<K, sizeof(T) == 2>;
  auto kern = wht_project_kernel<T, K, LB>;
  static bool configured[64] = {};
  int dev = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    LBP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      Cfg::kSmemBytes));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const uint32_t want = (p.n_items + Cfg::kWarps - 1) / Cfg::kWarps;
  const int grid = static_cast<int>(want < static_cast<uint32_t>(sms) ? want : sms);
  kern<<<grid, Cfg::kWarps * 32, Cfg::kSmemBytes, stream>>>(tmaps[0], tmaps[1], out0, out1, p, plan);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

template <typename T, int K>
static int launch_k(int LB, const CUtensorMap* tmaps, T* out0, T* out1, const ProjParams& p,
                    const DevicePlan& plan, int sms, cudaStream_t stream) {
  switch (LB) {
    case 1: return launch_one<T, K, 1>(tmaps, out0, out1, p, plan, sms, stream);
    case 2: return launch_one<T, K, 2>(tmaps, out0, out1, p, plan, sms, stream);
    case 4: return launch_one<T, K, 4>(tmaps, out0, out1, p, plan, sms, stream);
    case 8:
      if constexpr (K >= 8) return launch_one<T, K, 8>(tmaps, out0, out1, p, plan, sms, stream);
      break;
    case 16:
      if constexpr (K >= 16) return launch_one<T, K, 16>(tmaps, out0, out1, p, plan, sms, stream);
      break;
  }
  return LBP_ERR_BASIS;
}

template <typename T>
static int launch_t(const CUtensorMap* tmaps, T* out0, T* out1, const ProjParams& p,
                    const BasisPlan& bp, const DevicePlan& plan, int sms, cudaStream_t stream) {
  switch (bp.k) {
    case 4: return launch_k<T, 4>(bp.LB, tmaps, out0, out1, p, plan, sms, stream);
    case 8: return launch_k<T, 8>(bp.LB, tmaps, out0, out1, p, plan, sms, stream);
    case 16: return launch_k<T, 16>(bp.LB, tmaps, out0, out1, p, plan, sms, stream);
  }
  return LBP_ERR_BLOCK;
}

int launch_project2(const void* t0, void* out0, int C0, const void* t1, void* out1, int C1,
                    int dtype, int B, int H, int W, const BasisPlan& bp, RowMap rows,
                    uint32_t* status, cudaStream_t stream, float scale0, float scale1,
                    const lbp_view* view0, const lbp_view* view1) {
  const int K = bp.k;
  const int es = dtype == LBP_BF16 ? 2 : 4;
  const int box_c = 128 / es;   // a box wider than C is legal: the excess is zero-filled

  CUtensorMap tmaps[2];
  if (int e = encode_block_tensor_map(&tmaps[0], t0, dtype, B, H, W, C0, K, box_c, false, view0)) return e;
  if (t1 != nullptr) {
    if (int e = encode_block_tensor_map(&tmaps[1], t1, dtype, B, H, W, C1, K, box_c, false, view1)) return e;
  } else {
    tmaps[1] = tmaps[0];
  }

  ProjParams p;
  p.Hb = blocks_along(H, K);
  p.Wb = blocks_along(W, K);
  p.nb = B * p.Hb * p.Wb;
  p.r = bp.r;
  p.bpt = rows.bpt;
  p.tile_rows = rows.tile_rows;
  p.C[0] = C0;
  p.C[1] = t1 ? C1 : C0;
  p.n_chunks[0] = (C0 + box_c - 1) / box_c;
  p.n_chunks[1] = t1 ? (C1 + box_c - 1) / box_c : 1;
  const long long n0 = static_cast<long long>(p.nb) * p.n_chunks[0];
  const long long n1 = t1 ? static_cast<long long>(p.nb) * p.n_chunks[1] : 0;
  if (n0 + n1 >= (1ll << 31)) return LBP_ERR_SHAPE;
  p.n_items0 = static_cast<uint32_t>(n0);
  p.n_items = static_cast<uint32_t>(n0 + n1);
  p.status = status;
  p.scale[0] = scale0 > 0.f ? scale0 : 1.0f / static_cast<float>(K);
  p.scale[1] = scale1 > 0.f ? scale1 : 1.0f / static_cast<float>(K);
  p.defer_wait = projection_defer_wait() ? 1 : 0;
  p.test_stall = test_stall_projection() ? 1 : 0;

  int dev = 0, sms = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));

  // The tcgen05 kernel works on four 64-channel chunks of a block at a time: with
  // channel counts that leave many of those places empty (48 and 192 channels:
  // half of them) the warp-level kernel is the faster one.
  const int chunks_all = p.n_chunks[0] + (t1 ? p.n_chunks[1] : 0);
  const int places_all = 4 * ((p.n_chunks[0] + 3) / 4 + (t1 ? (p.n_chunks[1] + 3) / 4 : 0));
  if (dtype == LBP_BF16 && tune_options().umma && project_umma_supported(K, bp.r) &&
      5 * chunks_all >= 4 * places_all) {
    // orders 8 and 16 at low rank: tcgen05 kernel, an item is a block x four 64-channel chunks
    CUtensorMap qm[2];
    // a box is 64 tokens: the block at order 8, four of its token rows at order 16
    const int box_h = 64 / K;
    if (int e = encode_box_tensor_map(&qm[0], t0, dtype, B, H, W, C0, box_c, K, box_h, true, view0)) return e;
    qm[1] = qm[0];
    if (t1 != nullptr)
      if (int e = encode_box_tensor_map(&qm[1], t1, dtype, B, H, W, C1, box_c, K, box_h, true, view1)) return e;
    ProjParams pq = p;
    pq.n_chunks[0] = (p.n_chunks[0] + 3) / 4;
    pq.n_chunks[1] = t1 ? (p.n_chunks[1] + 3) / 4 : 1;
    pq.n_items0 = static_cast<uint32_t>(static_cast<long long>(p.nb) * pq.n_chunks[0]);
    pq.n_items = pq.n_items0 + (t1 ? static_cast<uint32_t>(static_cast<long long>(p.nb) * pq.n_chunks[1]) : 0u);
    return launch_project_umma(qm, static_cast<__nv_bfloat16*>(out0), static_cast<__nv_bfloat16*>(out1),
                               pq, bp, sms, stream);
  }
  if (dtype == LBP_BF16 && project_mma_supported(K, bp.r)) {
    // bf16 data at moderate rank: the +-1 basis matrix is applied on the tensor pipe
    CUtensorMap sw[2];
    if (project_mma_strips(K, bp.r)) {
      // order 4 works on strips of four blocks along W (4 x 16 token boxes)
      if (int e = encode_box_tensor_map(&sw[0], t0, dtype, B, H, W, C0, box_c, 16, 4, true, view0)) return e;
      sw[1] = sw[0];
      if (t1 != nullptr)
        if (int e = encode_box_tensor_map(&sw[1], t1, dtype, B, H, W, C1, box_c, 16, 4, true, view1)) return e;
      ProjParams ps = p;
      const long long strips = static_cast<long long>(B) * p.Hb * ((p.Wb + 3) / 4);
      ps.n_items0 = static_cast<uint32_t>(strips * p.n_chunks[0]);
      ps.n_items = ps.n_items0 + (t1 ? static_cast<uint32_t>(strips * p.n_chunks[1]) : 0u);
      return launch_project_mma(sw, static_cast<__nv_bfloat16*>(out0),
                                static_cast<__nv_bfloat16*>(out1), ps, bp, sms, stream);
    }
    if (int e = encode_block_tensor_map(&sw[0], t0, dtype, B, H, W, C0, K, box_c, true, view0)) return e;
    sw[1] = sw[0];
    if (t1 != nullptr)
      if (int e = encode_block_tensor_map(&sw[1], t1, dtype, B, H, W, C1, K, box_c, true, view1)) return e;
    return launch_project_mma(sw, static_cast<__nv_bfloat16*>(out0),
                              static_cast<__nv_bfloat16*>(out1), p, bp, sms, stream);
  }

  DevicePlan plan;
  for (int n = 0; n < 256; ++n) plan.qmap[n] = bp.qmap[n];

  if (dtype == LBP_BF16)
    return launch_t<__nv_bfloat16>(tmaps, static_cast<__nv_bfloat16*>(out0),
                                   static_cast<__nv_bfloat16*>(out1), p, bp, plan, sms, stream);
  return launch_t<float>(tmaps, static_cast<float*>(out0), static_cast<float*>(out1), p, bp, plan,
                         sms, stream);
}

int launch_project(const void* t, void* t_hat, int dtype, int B, int H, int W, int C,
                   const BasisPlan& bp, RowMap rows, uint32_t* status, cudaStream_t stream,
                   float scale, const lbp_view* view) {
  return launch_project2(t, t_hat, C, nullptr, nullptr, 0, dtype, B, H, W, bp, rows, status, stream,
                         scale, scale, view, nullptr);
}

}  // namespace lbp
