// Epilogue of one accumulator tile of the products kernels, shared by the
// one-CTA and the CTA-pair variants: a GW tile is written to g_W (or to an fp32
// K-slice plane); a GX tile is expanded with the transposed bases (Eq. 7) and
// written to g_x, so g_x_hat never leaves the chip.
//
// Four warps (one per TMEM lane quarter) form a group; group `eg` takes the
// 32-column chunks eg, eg + kEGroups, ... of the tile.  A chunk goes TMEM ->
// registers -> swizzled shared staging (row = low-rank row, 32 columns); then
// every thread owns NCH channels of one block, gathers that block's r
// coefficients, runs the LB x LB butterfly and stores the k x k tokens.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include <type_traits>

#include "lbp_fused.cuh"
#include "ptx_sm100.cuh"
#include "wht_device.cuh"

namespace lbp {
namespace fused {

constexpr int BM = 128;
constexpr int kEStride = 32;   // fp32 words per staged row; 16-byte chunk c of row i sits at chunk c ^ (i & 7)
constexpr int kEBytes = (BM + 1) * kEStride * 4;   // 128 staged rows + one row of zeros
constexpr int kEGroups = 2;                        // epilogue groups of 4 warps

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Barrier over `nthreads` threads that also ORs a predicate over them: every
// participant gets the same answer, so a decision taken on it (leave the tile
// loop after an expired wait) cannot split the threads that share the barrier.
__device__ __forceinline__ bool named_bar_or(int id, int nthreads, bool pred) {
  uint32_t any;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(any)
      : "r"(id), "r"(nthreads), "r"(static_cast<uint32_t>(pred))
      : "memory");
  return any != 0;
}

__device__ __forceinline__ int blocks_in_group(const FusedParams& p, int g) {
  const int left = p.nb - g * p.bpt;
  return left < p.bpt ? left : p.bpt;
}

// What the epilogue needs to know about the accumulator it drains.
struct DrainTile {
  int is_gw;
  int row_base;       // GW: first g_W row of these 128 accumulator rows
  int group;          // GX: 128-row group of low-rank rows
  int col_base;       // first output column (channel) of the tile
  int bn;             // accumulator columns in use
  int slice;          // GW: K slice (plane index when gw_splits > 1)
  uint32_t tmem_acc;  // TMEM address of column 0, lane 0 of the accumulator
};

// `release()` is called by lane 0 of every warp once the warp has read its last
// accumulator column (the tensor core may then overwrite the slot).
template <int K, int LB, int NEX, class Release>
__device__ __forceinline__ void drain_tile(const FusedParams& p, const FusedBasis& fb,
                                           const DrainTile& t, float* Eg, int bar_id, int eg,
                                           int etid, int quarter, int lane, Release release) {
  const uint32_t lane_bits = static_cast<uint32_t>(quarter * 32) << 16;
  bool released = false;

  if (t.is_gw) {
    // ---- GW tile: g_W[128 i + row, BNw j + col] ----
    // A chunk is staged like a GX chunk and written out with eight lanes along a
    // row, so that a store instruction covers whole 128-byte pieces of four rows.
    const int ew = etid >> 5;
    for (int c0 = eg * 32; c0 < t.bn; c0 += 32 * kEGroups) {
      uint32_t v[32];
      ptx::tmem_ld_32x32(t.tmem_acc + lane_bits + c0, v);
      ptx::tmem_ld_wait();
      if (c0 + 32 * kEGroups >= t.bn) {
        released = true;
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) release();
      }
      const int erow_i = quarter * 32 + lane;
      uint4* erow = reinterpret_cast<uint4*>(Eg + erow_i * kEStride);
#pragma unroll
      for (int q = 0; q < 8; ++q)
        erow[q ^ (erow_i & 7)] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      named_bar_sync(bar_id, 128);
      if (p.gw_splits > 1 || !p.gw_bf16) {
        // fp32 g_W, or a K slice: fp32 partial plane, summed by the reduce kernel that follows
        float* dst = p.gw_splits > 1
                         ? p.gw_planes + static_cast<long long>(t.slice) * p.Cout * p.Cin
                         : static_cast<float*>(p.g_W);
        const int o = lane & 7, rs = lane >> 3;
        const int col = t.col_base + c0 + o * 4;
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int row = it * 16 + ew * 4 + rs;
          const long long grow = static_cast<long long>(t.row_base) + row;
          if (grow < p.Cout && col < p.Cin)
            *reinterpret_cast<uint4*>(dst + grow * p.Cin + col) =
                *reinterpret_cast<const uint4*>(Eg + row * kEStride + ((o ^ (row & 7)) << 2));
        }
      } else {
        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.g_W);
        const int o = lane & 3, rs = lane >> 2;
        const int col = t.col_base + c0 + o * 8;
#pragma unroll
        for (int it = 0; it < 4; ++it) {
          const int row = it * 32 + ew * 8 + rs;
          const long long grow = static_cast<long long>(t.row_base) + row;
          if (grow < p.Cout && col < p.Cin) {
            const float4 f0 = *reinterpret_cast<const float4*>(
                Eg + row * kEStride + (((2 * o) ^ (row & 7)) << 2));
            const float4 f1 = *reinterpret_cast<const float4*>(
                Eg + row * kEStride + (((2 * o + 1) ^ (row & 7)) << 2));
            uint4 pk;
            pk.x = pack_bf16x2(f0.x, f0.y);
            pk.y = pack_bf16x2(f0.z, f0.w);
            pk.z = pack_bf16x2(f1.x, f1.y);
            pk.w = pack_bf16x2(f1.z, f1.w);
            *reinterpret_cast<uint4*>(dst + grow * p.Cin + col) = pk;
          }
        }
      }
      named_bar_sync(bar_id, 128);
    }
  } else {
    // ---- GX tile: expand g_x_hat (128 rows x BNx columns) into g_x ----
    const int m = t.group;
    const int bg = blocks_in_group(p, m);
    // channels per thread: an 8 x 8 coefficient array leaves registers for two
    constexpr int NCH = LB <= 4 ? 4 : 2;
    constexpr int RUN = K / LB;
    constexpr int CPT = 32 / NCH;       // threads across one 32-column chunk
    constexpr int BSLOTS = 128 / CPT;   // blocks expanded concurrently
    const int cc = etid % CPT, bs = etid / CPT;
    // element offsets of a token inside a block fit 32 bits (checked on the host)
    const int tok_stride = static_cast<int>(p.vgx.token), row_stride = static_cast<int>(p.vgx.row);
    // first token of block bl of this group (channel 0) and how many of its K x K
    // tokens lie on the grid
    auto block_origin = [&](int bl, __nv_bfloat16** o, int* ulim, int* vlim) {
      const int blk = m * p.bpt + bl;
      const int bw = blk % p.Wb, t2 = blk / p.Wb, bh = t2 % p.Hb, b = t2 / p.Hb;
      // the offset inside one image fits 32 bits (checked on the host)
      *o = p.g_x + (static_cast<long long>(b) * p.gx_image8 * 8 +
                   (bh * K * row_stride + bw * K * tok_stride));
      *ulim = p.H - bh * K < K ? p.H - bh * K : K;
      *vlim = p.W - bw * K < K ? p.W - bw * K : K;
    };
    // the first block a thread expands is the same for every chunk of the tile
    __nv_bfloat16* o_first = p.g_x;
    int ulim_first = K, vlim_first = K;
    if (bs < bg) {
      block_origin(bs, &o_first, &ulim_first, &vlim_first);
      o_first += t.col_base + cc * NCH;
    }
    for (int c0 = eg * 32; c0 < t.bn; c0 += 32 * kEGroups) {
      uint32_t v[32];
      ptx::tmem_ld_32x32(t.tmem_acc + lane_bits + c0, v);
      ptx::tmem_ld_wait();
      if (c0 + 32 * kEGroups >= t.bn) {
        released = true;
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) release();
      }
      const int erow_i = quarter * 32 + lane;
      uint4* erow = reinterpret_cast<uint4*>(Eg + erow_i * kEStride);
#pragma unroll
      for (int q = 0; q < 8; ++q)
        erow[q ^ (erow_i & 7)] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      named_bar_sync(bar_id, 128);
      const int ch = t.col_base + c0 + cc * NCH;
      if (ch < p.Cin) {
        for (int bl = bs; bl < bg; bl += BSLOTS) {
          float acc[LB][LB][NCH];
          const int row_b = bl * p.r;
#pragma unroll
          for (int a = 0; a < LB; ++a) {
#pragma unroll
            for (int b = 0; b < LB; ++b) {
              const int q = fb.qmap[a * LB + b];
              const int row_q = q >= 0 ? row_b + q : BM;
              if constexpr (NCH == 4) {
                const float4 f =
                    *reinterpret_cast<const float4*>(Eg + row_q * kEStride + ((cc ^ (row_q & 7)) << 2));
                acc[a][b][0] = f.x;
                acc[a][b][1] = f.y;
                acc[a][b][2] = f.z;
                acc[a][b][3] = f.w;
              } else if constexpr (NCH == 2) {
                const float2 f = *reinterpret_cast<const float2*>(
                    Eg + row_q * kEStride + (((cc >> 1) ^ (row_q & 7)) << 2) + (cc & 1) * 2);
                acc[a][b][0] = f.x;
                acc[a][b][1] = f.y;
              } else {
                acc[a][b][0] = Eg[row_q * kEStride + (((cc >> 2) ^ (row_q & 7)) << 2) + (cc & 3)];
              }
            }
          }
          hadamard_rows<LB, NCH>(acc);
          hadamard_cols<LB, NCH>(acc);
          __nv_bfloat16* o;
          int ulim, vlim;
          if (bl == bs) {
            o = o_first + (ch - t.col_base - cc * NCH);
            ulim = ulim_first;
            vlim = vlim_first;
          } else {
            block_origin(bl, &o, &ulim, &vlim);
            o += ch;
          }
          // Stores of one expanded block.  RAGGED: the block reaches past the grid
          // (a side that is no multiple of K) and every token is checked; all other
          // blocks take the unchecked form.  The 1/k of Eq. 7 is already in the
          // coefficients (g_y_hat carries 1/k^2), so a value is rounded as it is.
          auto emit = [&](auto ragged) {
            constexpr bool RAGGED = decltype(ragged)::value;
            if constexpr (NEX > 0) {
              // Bases outside the LB x LB core: B_{i,j}[u][v] = s_i(u) s_j(v) with
              // s = +-1, so each adds +-coefficient to every token.  The row sign is
              // folded into the coefficient once per token row, the column sign is
              // a +-1.0 factor of an FMA.
              static_assert(NCH == 4, "extras go with four channels per thread");
              float ce[NEX][NCH];
              uint32_t mu[NEX], mv[NEX];
#pragma unroll
              for (int x = 0; x < NEX; ++x) {
                const int q = fb.ex_q[x];
                const int row_q = q >= 0 ? row_b + q : BM;
                const float4 f =
                    *reinterpret_cast<const float4*>(Eg + row_q * kEStride + ((cc ^ (row_q & 7)) << 2));
                ce[x][0] = f.x;
                ce[x][1] = f.y;
                ce[x][2] = f.z;
                ce[x][3] = f.w;
                mu[x] = fb.ex_mu[x];
                mv[x] = fb.ex_mv[x];
              }
#pragma unroll
              for (int a = 0; a < LB; ++a) {
#pragma unroll 1
                for (int du = 0; du < RUN; ++du) {
                  const int u = a * RUN + du;
                  if (RAGGED && u >= ulim) break;
                  float ceu[NEX][NCH];
#pragma unroll
                  for (int x = 0; x < NEX; ++x) {
                    const float su = __uint_as_float(0x3f800000u | (((mu[x] >> u) & 1u) << 31));
#pragma unroll
                    for (int c = 0; c < NCH; ++c) ceu[x][c] = ce[x][c] * su;
                  }
                  __nv_bfloat16* orow = o + u * row_stride;
#pragma unroll
                  for (int v = 0; v < K; ++v) {
                    float val[NCH];
#pragma unroll
                    for (int c = 0; c < NCH; ++c) val[c] = acc[a][v / RUN][c];
#pragma unroll
                    for (int x = 0; x < NEX; ++x) {
                      const float sv = __uint_as_float(0x3f800000u | ((mv[x] << (31 - v)) & 0x80000000u));
#pragma unroll
                      for (int c = 0; c < NCH; ++c) val[c] = fmaf(sv, ceu[x][c], val[c]);
                    }
                    uint2 pk;
                    pk.x = pack_bf16x2(val[0], val[1]);
                    pk.y = pack_bf16x2(val[2], val[3]);
                    if (!RAGGED || v < vlim) *reinterpret_cast<uint2*>(orow + v * tok_stride) = pk;
                  }
                }
              }
            } else {
              // each of the LB x LB values covers a RUN x RUN patch of tokens: round
              // and pack once, store RUN * RUN times
#pragma unroll
              for (int a = 0; a < LB; ++a) {
#pragma unroll
                for (int b2 = 0; b2 < LB; ++b2) {
                  if constexpr (NCH == 4) {
                    uint2 pk;
                    pk.x = pack_bf16x2(acc[a][b2][0], acc[a][b2][1]);
                    pk.y = pack_bf16x2(acc[a][b2][2], acc[a][b2][3]);
#pragma unroll
                    for (int du = 0; du < RUN; ++du)
#pragma unroll
                      for (int dv = 0; dv < RUN; ++dv)
                        if (!RAGGED || (a * RUN + du < ulim && b2 * RUN + dv < vlim))
                          *reinterpret_cast<uint2*>(o + (a * RUN + du) * row_stride +
                                                    (b2 * RUN + dv) * tok_stride) = pk;
                  } else if constexpr (NCH == 1) {
                    const __nv_bfloat16 hv = __float2bfloat16_rn(acc[a][b2][0]);
#pragma unroll
                    for (int du = 0; du < RUN; ++du)
#pragma unroll
                      for (int dv = 0; dv < RUN; ++dv)
                        if (!RAGGED || (a * RUN + du < ulim && b2 * RUN + dv < vlim))
                          o[(a * RUN + du) * row_stride + (b2 * RUN + dv) * tok_stride] = hv;
                  } else {
                    const uint32_t pk = pack_bf16x2(acc[a][b2][0], acc[a][b2][1]);
#pragma unroll
                    for (int du = 0; du < RUN; ++du)
#pragma unroll
                      for (int dv = 0; dv < RUN; ++dv)
                        if (!RAGGED || (a * RUN + du < ulim && b2 * RUN + dv < vlim))
                          *reinterpret_cast<uint32_t*>(o + (a * RUN + du) * row_stride +
                                                       (b2 * RUN + dv) * tok_stride) = pk;
                  }
                }
              }
            }
          };
          if (ulim == K && vlim == K)
            emit(std::false_type{});
          else
            emit(std::true_type{});
        }
      }
      named_bar_sync(bar_id, 128);
    }
  }
  if (!released) {   // this group had no chunk of the tile
    ptx::tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) release();
  }
}

}  // namespace fused
}  // namespace lbp
