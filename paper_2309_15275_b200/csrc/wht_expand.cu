// Expansion kernel (Eq. 7):  t[blk,u,v,c] = (1/k) sum_q wal_iq[u] wal_jq[v] t_hat[blk,q,c].
//
// A warp owns one (block, 32-word channel chunk).  Each lane gathers the r
// coefficients of its channel word into the LB x LB natural-order array, runs
// the Hadamard butterfly (its own inverse up to scale) and replicates every
// value over its (k/LB) x (k/LB) run of tokens.  Reads and writes are 128-byte
// coalesced per warp instruction.
#include <cuda_bf16.h>

#include "lbp_internal.h"
#include "wht_device.cuh"

namespace lbp {

struct ExpandParams {
  int32_t nb, Hb, Wb, H, W, C, r, n_chunks;
  int32_t bpt, tile_rows;
  long long n_items;
  float scale;
  long long s_image, s_row, s_tok;   // element strides of t (dense: H*W*C, W*C, C)
};

// Load the NCH channel values a lane owns from row `row` of the coefficient matrix.
template <typename TI, bool OUT_BF16, int NCH>
__device__ __forceinline__ void load_coeff(const TI* __restrict__ t_hat, long long row, int C,
                                           int c0, int pass, float (&f)[NCH]) {
  if constexpr (sizeof(TI) == 4) {
    if constexpr (NCH == 2) {
      const float2 v = *reinterpret_cast<const float2*>(t_hat + row * C + c0);
      f[0] = v.x;
      f[1] = v.y;
    } else {
      f[0] = t_hat[row * C + c0 + (OUT_BF16 ? pass : 0)];
    }
  } else {
    const uint32_t w = *reinterpret_cast<const uint32_t*>(t_hat + row * C + c0);
    unpack_word<true, NCH>(w, pass, f);
  }
}

template <typename TO, bool OUT_BF16, int NCH>
__device__ __forceinline__ void store_token(TO* __restrict__ t, long long off, int pass,
                                            const float (&v)[NCH], float scale) {
  if constexpr (!OUT_BF16) {
    t[off] = v[0] * scale;
  } else if constexpr (NCH == 2) {
    *reinterpret_cast<uint32_t*>(t + off) = pack_bf16x2(v[0] * scale, v[1] * scale);
  } else {
    t[off + pass] = __float2bfloat16_rn(v[0] * scale);
  }
}

template <typename TI, typename TO, int K, int LB>
__global__ void __launch_bounds__(256)
    wht_expand_kernel(const TI* __restrict__ t_hat, TO* __restrict__ t,
                      const __grid_constant__ ExpandParams p,
                      const __grid_constant__ DevicePlan plan) {
  constexpr bool OUT_BF16 = sizeof(TO) == 2;
  constexpr int CH_PER_WORD = OUT_BF16 ? 2 : 1;
  const int lane = threadIdx.x & 31;
  const long long warp0 = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const long long n_warps = (static_cast<long long>(gridDim.x) * blockDim.x) >> 5;

  for (long long item = warp0; item < p.n_items; item += n_warps) {
    const int chunk = static_cast<int>(item % p.n_chunks);
    const int blk = static_cast<int>(item / p.n_chunks);
    const int c0 = (chunk * 32 + lane) * CH_PER_WORD;
    if (c0 >= p.C) continue;
    const int bw = blk % p.Wb, bh = (blk / p.Wb) % p.Hb, b = blk / (p.Wb * p.Hb);
    const long long row0 =
        static_cast<long long>(blk / p.bpt) * p.tile_rows + static_cast<long long>(blk % p.bpt) * p.r;
    // offset of token (u, v) of this block: tok0 + u * s_row + v * s_tok
    const long long tok0 = static_cast<long long>(b) * p.s_image +
                           static_cast<long long>(bh * K) * p.s_row +
                           static_cast<long long>(bw * K) * p.s_tok + c0;
    // tokens of a last block that lie past the grid are not stored
    const int ulim = p.H - bh * K < K ? p.H - bh * K : K;
    const int vlim = p.W - bw * K < K ? p.W - bw * K : K;

    if constexpr (LB < 16) {
      constexpr int RUN = K / LB;
      constexpr int NCH = (OUT_BF16 && LB <= 4) ? 2 : 1;
      constexpr int NPASS = (OUT_BF16 && NCH == 1) ? 2 : 1;
#pragma unroll 1
      for (int pass = 0; pass < NPASS; ++pass) {
        float acc[LB][LB][NCH];
#pragma unroll
        for (int a = 0; a < LB; ++a) {
#pragma unroll
          for (int bb = 0; bb < LB; ++bb) {
            const int q = plan.qmap[a * LB + bb];
            if (q >= 0) {
              load_coeff<TI, OUT_BF16, NCH>(t_hat, row0 + q, p.C, c0, pass, acc[a][bb]);
            } else {
#pragma unroll
              for (int c = 0; c < NCH; ++c) acc[a][bb][c] = 0.f;
            }
          }
        }
        hadamard_rows<LB, NCH>(acc);
        hadamard_cols<LB, NCH>(acc);
        if (ulim == K && vlim == K) {
#pragma unroll
          for (int u = 0; u < K; ++u) {
#pragma unroll
            for (int v = 0; v < K; ++v) {
              store_token<TO, OUT_BF16, NCH>(t, tok0 + u * p.s_row + v * p.s_tok,
                                             pass, acc[u / RUN][v / RUN], p.scale);
            }
          }
        } else {   // a block that reaches past the grid: every token is checked
#pragma unroll
          for (int u = 0; u < K; ++u) {
#pragma unroll
            for (int v = 0; v < K; ++v) {
              if (u < ulim && v < vlim)
                store_token<TO, OUT_BF16, NCH>(t, tok0 + u * p.s_row + v * p.s_tok,
                                               pass, acc[u / RUN][v / RUN], p.scale);
            }
          }
        }
      }
    } else {
      // LB == 16: pass v_lo produces the output columns v = 4 * v_hi + v_lo.
      constexpr int NPASS = OUT_BF16 ? 2 : 1;
#pragma unroll 1
      for (int pass = 0; pass < NPASS; ++pass) {
#pragma unroll 1
        for (int v_lo = 0; v_lo < 4; ++v_lo) {
          const float s1 = (v_lo & 1) ? -1.f : 1.f;
          const float s2 = (v_lo & 2) ? -1.f : 1.f;
          const float s3 = s1 * s2;
          float R[4][16];  // [v_hi][a] then [v_hi][u]
#pragma unroll
          for (int a = 0; a < 16; ++a) {
            float z[4];
#pragma unroll
            for (int bh4 = 0; bh4 < 4; ++bh4) {
              float c4[4];
#pragma unroll
              for (int bl = 0; bl < 4; ++bl) {
                const int q = plan.qmap[a * 16 + bh4 * 4 + bl];
                float f[1] = {0.f};
                if (q >= 0) load_coeff<TI, OUT_BF16, 1>(t_hat, row0 + q, p.C, c0, pass, f);
                c4[bl] = f[0];
              }
              z[bh4] = (c4[0] + s1 * c4[1]) + (s2 * c4[2] + s3 * c4[3]);
            }
            hadamard_vec<4>(z);
#pragma unroll
            for (int vh = 0; vh < 4; ++vh) R[vh][a] = z[vh];
          }
#pragma unroll
          for (int vh = 0; vh < 4; ++vh) {
            hadamard_vec<16>(R[vh]);
#pragma unroll
            for (int u = 0; u < 16; ++u) {
              const float v1[1] = {R[vh][u]};
              if (u < ulim && vh * 4 + v_lo < vlim)
                store_token<TO, OUT_BF16, 1>(
                    t, tok0 + u * p.s_row + (vh * 4 + v_lo) * p.s_tok, pass, v1,
                    p.scale);
            }
          }
        }
      }
    }
  }
}

template <typename TI, typename TO, int K, int LB>
static int launch_one(const TI* t_hat, TO* t, const ExpandParams& p, const DevicePlan& plan,
                      int sms, cudaStream_t stream) {
  const long long warps_per_cta = 8;
  long long want = (p.n_items + warps_per_cta - 1) / warps_per_cta;
  const long long cap = static_cast<long long>(sms) * 8;
  const int grid = static_cast<int>(want < cap ? want : cap);
  wht_expand_kernel<TI, TO, K, LB><<<grid, 256, 0, stream>>>(t_hat, t, p, plan);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

template <typename TI, typename TO, int K>
static int launch_k(int LB, const TI* t_hat, TO* t, const ExpandParams& p, const DevicePlan& plan,
                    int sms, cudaStream_t stream) {
  switch (LB) {
    case 1: return launch_one<TI, TO, K, 1>(t_hat, t, p, plan, sms, stream);
    case 2: return launch_one<TI, TO, K, 2>(t_hat, t, p, plan, sms, stream);
    case 4: return launch_one<TI, TO, K, 4>(t_hat, t, p, plan, sms, stream);
    case 8:
      if constexpr (K >= 8) return launch_one<TI, TO, K, 8>(t_hat, t, p, plan, sms, stream);
      break;
    case 16:
      if constexpr (K >= 16) return launch_one<TI, TO, K, 16>(t_hat, t, p, plan, sms, stream);
      break;
  }
  return LBP_ERR_BASIS;
}

template <typename TI, typename TO>
static int launch_t(const TI* t_hat, TO* t, const ExpandParams& p, const BasisPlan& bp,
                    const DevicePlan& plan, int sms, cudaStream_t stream) {
  switch (bp.k) {
    case 4: return launch_k<TI, TO, 4>(bp.LB, t_hat, t, p, plan, sms, stream);
    case 8: return launch_k<TI, TO, 8>(bp.LB, t_hat, t, p, plan, sms, stream);
    case 16: return launch_k<TI, TO, 16>(bp.LB, t_hat, t, p, plan, sms, stream);
  }
  return LBP_ERR_BLOCK;
}

int launch_expand(const void* t_hat, bool in_f32, void* t, int dtype, int B, int H, int W, int C,
                  const BasisPlan& bp, RowMap rows, cudaStream_t stream, const lbp_view* view) {
  const int K = bp.k;
  ExpandParams p;
  const lbp_view sv = resolve_view(view, H, W, C);
  p.s_image = sv.image;
  p.s_row = sv.row;
  p.s_tok = sv.token;
  p.Hb = blocks_along(H, K);
  p.Wb = blocks_along(W, K);
  p.nb = B * p.Hb * p.Wb;
  p.H = H;
  p.W = W;
  p.C = C;
  p.r = bp.r;
  const int ch_per_chunk = 32 * (dtype == LBP_BF16 ? 2 : 1);
  p.n_chunks = (C + ch_per_chunk - 1) / ch_per_chunk;
  p.bpt = rows.bpt;
  p.tile_rows = rows.tile_rows;
  p.n_items = static_cast<long long>(p.nb) * p.n_chunks;
  p.scale = 1.0f / static_cast<float>(K);

  DevicePlan plan;
  for (int n = 0; n < 256; ++n) plan.qmap[n] = bp.qmap[n];

  int dev = 0, sms = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));

  if (dtype == LBP_BF16) {
    if (in_f32)
      return launch_t<float, __nv_bfloat16>(static_cast<const float*>(t_hat),
                                            static_cast<__nv_bfloat16*>(t), p, bp, plan, sms, stream);
    return launch_t<__nv_bfloat16, __nv_bfloat16>(static_cast<const __nv_bfloat16*>(t_hat),
                                                  static_cast<__nv_bfloat16*>(t), p, bp, plan, sms,
                                                  stream);
  }
  return launch_t<float, float>(static_cast<const float*>(t_hat), static_cast<float*>(t), p, bp,
                                plan, sms, stream);
}

}  // namespace lbp
