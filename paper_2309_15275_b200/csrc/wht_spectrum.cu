// Energy of the basis responses (Sec. 3.2, profiling step of the
// low-heuristic-error selection): sum of squares of a projected tensor per
// basis slot.  The tensor is stored (blocks * r, C) with slot q = row % r.
//
// One warp per row: the lanes square and add their share of the C channels in
// fp32, the warp total goes to a per-CTA fp64 table in shared memory, and each
// CTA adds its table to the result once.
//
// For bf16 data of order 4 and 8 a single pass does all of it: the kernel below
// streams the tensor once (the tile ring of the projection kernel), applies all
// k*k bases to a tile with warp MMAs and adds the squared responses to
// per-thread sums; nothing but the k*k energies is written.
#include <cuda_bf16.h>

#include "lbp_internal.h"
#include "ptx_sm100.cuh"
#include "wht_device.cuh"
#include "wht_mma.cuh"
#include "wht_project.cuh"

namespace lbp {

// ---- one pass: bf16 data, k = 4 or 8 ---------------------------------------
// Rows of the basis matrix are taken 32 at a time (two m16 tiles), so that the
// accumulators of one group (32 rows x 64 channels) fit the register file; the
// tile in shared memory is read once per group.
template <int K>
__global__ void __launch_bounds__(MmaCfg<K>::kWarps * 32, 1)
    wht_spectrum_mma_kernel(const __grid_constant__ CUtensorMap tmap,
                            const __grid_constant__ ProjParams p,
                            const __grid_constant__ MmaPlan mp, double* __restrict__ energy) {
  using Cfg = MmaCfg<K>;
  constexpr int NW = Cfg::kWarps, S = Cfg::kStages, KS = Cfg::kKSteps;
  constexpr int R = K * K;
  constexpr int MTT = R / 16;                 // m16 tiles over all k*k rows
  constexpr int GM = MTT < 2 ? MTT : 2;       // m16 tiles per group
  constexpr int NG = MTT / GM;                // groups

  extern __shared__ uint8_t smem_raw[];
  __shared__ double e_sm[R];
  uint8_t* tiles = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + NW * S * Cfg::kTileBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  uint64_t* my_bars = bars + warp * S;
  uint8_t* my_tiles = tiles + warp * S * Cfg::kTileBytes;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < S; ++s) ptx::mbar_init(&my_bars[s], 1);
    ptx::mbar_fence_init();
  }
  if (threadIdx.x == 0) ptx::prefetch_tensormap(&tmap);
  for (int i = threadIdx.x; i < R; i += NW * 32) e_sm[i] = 0.0;
  __syncthreads();

  const uint32_t first = blockIdx.x * NW + warp;
  const uint32_t stride = gridDim.x * NW;
  const uint32_t n_my = first < p.n_items ? (p.n_items - first + stride - 1) / stride : 0;
  const uint32_t nch = static_cast<uint32_t>(p.n_chunks[0]);
  const uint64_t stream_once = ptx::l2_policy_evict_first();   // the tensor is read exactly once

  auto issue = [&](uint32_t idx, int s) {
    const uint32_t item = first + idx * stride;
    const uint32_t blk = item / nch, chunk = item - blk * nch;
    const uint32_t bw = blk % p.Wb, t2 = blk / p.Wb, bh = t2 % p.Hb, b = t2 / p.Hb;
    ptx::mbar_expect_tx(&my_bars[s], static_cast<uint32_t>(Cfg::kTileBytes));
    ptx::tma_load_4d_hint(my_tiles + s * Cfg::kTileBytes, &tmap, &my_bars[s], chunk * 64, bw * K, bh * K, b,
                          stream_once);
  };
  if (lane == 0) {
    for (uint32_t i = 0; i < S && i < n_my; ++i) issue(i, i);
  }

  // A fragments (rows of the +-1 basis matrix), as in the projection kernel
  uint32_t afrag[NG][GM][KS][4];
#pragma unroll
  for (int ng = 0; ng < NG; ++ng)
#pragma unroll
    for (int mt = 0; mt < GM; ++mt)
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int q = (ng * GM + mt) * 16 + g + (j & 1) * 8;
          const int tok = ks * 16 + 2 * tq + (j >> 1) * 8;
          afrag[ng][mt][ks][j] = basis_bits<K>(mp, q, R, tok) | (basis_bits<K>(mp, q, R, tok + 1) << 16);
        }

  // per-thread sums of squared responses: rows g and g + 8 of every m16 tile
  float e[NG][GM][2];
#pragma unroll
  for (int ng = 0; ng < NG; ++ng)
#pragma unroll
    for (int mt = 0; mt < GM; ++mt) e[ng][mt][0] = e[ng][mt][1] = 0.f;

  const int ld_tok = ((lane >> 3) & 1) * 8 + (lane & 7);
  const int ld_chunk = lane >> 4;

  for (uint32_t idx = 0; idx < n_my; ++idx) {
    const int s = static_cast<int>(idx % S);
    const uint32_t parity = (idx / S) & 1u;
    const bool ok = ptx::mbar_wait(&my_bars[s], parity, p.status, (6u << 16) | 1u);
    if (!__all_sync(0xffffffffu, ok)) break;
    const uint32_t tile = ptx::smem_u32(my_tiles + s * Cfg::kTileBytes);

#pragma unroll
    for (int ng = 0; ng < NG; ++ng) {
      float d[GM][8][4];
#pragma unroll
      for (int mt = 0; mt < GM; ++mt)
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
          for (int j = 0; j < 4; ++j) d[mt][nt][j] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int tok = ks * 16 + ld_tok;
#pragma unroll
        for (int np = 0; np < 4; ++np) {
          const int c16 = np * 2 + ld_chunk;
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(tile + tok * 128 + ((c16 ^ (tok & 7)) << 4), b0, b1, b2, b3);
#pragma unroll
          for (int mt = 0; mt < GM; ++mt) {
            mma_bf16_16816(d[mt][2 * np], afrag[ng][mt][ks], b0, b1);
            mma_bf16_16816(d[mt][2 * np + 1], afrag[ng][mt][ks], b2, b3);
          }
        }
      }
      // channels past C were zero-filled by the TMA load and add nothing
#pragma unroll
      for (int mt = 0; mt < GM; ++mt)
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          e[ng][mt][0] = fmaf(d[mt][nt][0], d[mt][nt][0], e[ng][mt][0]);
          e[ng][mt][0] = fmaf(d[mt][nt][1], d[mt][nt][1], e[ng][mt][0]);
          e[ng][mt][1] = fmaf(d[mt][nt][2], d[mt][nt][2], e[ng][mt][1]);
          e[ng][mt][1] = fmaf(d[mt][nt][3], d[mt][nt][3], e[ng][mt][1]);
        }
    }

    __syncwarp();
    if (lane == 0 && idx + S < n_my) {
      ptx::fence_proxy_async_smem();
      issue(idx + S, s);
    }
  }

  // the four lanes of a quad hold different channels of the same rows
#pragma unroll
  for (int ng = 0; ng < NG; ++ng)
#pragma unroll
    for (int mt = 0; mt < GM; ++mt)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        float v = e[ng][mt][hh];
        v += __shfl_xor_sync(0xffffffffu, v, 1);
        v += __shfl_xor_sync(0xffffffffu, v, 2);
        if (tq == 0) atomicAdd(&e_sm[(ng * GM + mt) * 16 + g + hh * 8], static_cast<double>(v));
      }
  __syncthreads();
  // orthonormal coefficients: (1/k)^2 on the squares
  const double s2 = static_cast<double>(p.scale[0]) * static_cast<double>(p.scale[0]);
  for (int i = threadIdx.x; i < R; i += NW * 32) atomicAdd(&energy[i], e_sm[i] * s2);
}

// ---- one pass: bf16 data, k = 16 --------------------------------------------
// 256 responses per block are too many rows for the dense form above (4x the
// MMA work per byte of order 8).  The 2-D transform is separable: the transform
// along W (v) is a 16 x 16 Hadamard matrix applied by warp MMA to each of the 16
// token rows u of the block, one 8-channel n-tile at a time; the transform along H
// (u) is then a 16-point butterfly across the 16 accumulator sets, which a thread
// holds for the same (row, channel) positions.  Both in natural (Sylvester) order;
// `seq_of_nat` turns natural indices into sequency indices for the result.
struct Seq16 {
  uint8_t seq_of_nat[16];
};

__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];"
               : "=r"(r0), "=r"(r1)
               : "r"(addr)
               : "memory");
}

__global__ void __launch_bounds__(MmaCfg<16>::kWarps * 32, 1)
    wht_spectrum16_kernel(const __grid_constant__ CUtensorMap tmap,
                          const __grid_constant__ ProjParams p, const __grid_constant__ Seq16 sq,
                          double* __restrict__ energy) {
  using Cfg = MmaCfg<16>;
  constexpr int K = 16, NW = Cfg::kWarps, S = Cfg::kStages, R = K * K;

  extern __shared__ uint8_t smem_raw[];
  __shared__ double e_sm[R];
  uint8_t* tiles = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + NW * S * Cfg::kTileBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  uint64_t* my_bars = bars + warp * S;
  uint8_t* my_tiles = tiles + warp * S * Cfg::kTileBytes;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < S; ++s) ptx::mbar_init(&my_bars[s], 1);
    ptx::mbar_fence_init();
  }
  if (threadIdx.x == 0) ptx::prefetch_tensormap(&tmap);
  for (int i = threadIdx.x; i < R; i += NW * 32) e_sm[i] = 0.0;
  __syncthreads();

  const uint32_t first = blockIdx.x * NW + warp;
  const uint32_t stride = gridDim.x * NW;
  const uint32_t n_my = first < p.n_items ? (p.n_items - first + stride - 1) / stride : 0;
  const uint32_t nch = static_cast<uint32_t>(p.n_chunks[0]);
  const uint64_t stream_once = ptx::l2_policy_evict_first();

  auto issue = [&](uint32_t idx, int s) {
    const uint32_t item = first + idx * stride;
    const uint32_t blk = item / nch, chunk = item - blk * nch;
    const uint32_t bw = blk % p.Wb, t2 = blk / p.Wb, bh = t2 % p.Hb, b = t2 / p.Hb;
    ptx::mbar_expect_tx(&my_bars[s], static_cast<uint32_t>(Cfg::kTileBytes));
    ptx::tma_load_4d_hint(my_tiles + s * Cfg::kTileBytes, &tmap, &my_bars[s], chunk * 64, bw * K, bh * K, b,
                          stream_once);
  };
  if (lane == 0) {
    for (uint32_t i = 0; i < S && i < n_my; ++i) issue(i, i);
  }

  // A = natural-order Hadamard matrix H[b][v] = (-1)^popcount(b & v), m16 x k16
  uint32_t afrag[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int b = g + (j & 1) * 8;
    const int v = 2 * tq + (j >> 1) * 8;
    const uint32_t lo = (__popc(b & v) & 1) ? 0xBF80u : 0x3F80u;
    const uint32_t hi = (__popc(b & (v + 1)) & 1) ? 0xBF80u : 0x3F80u;
    afrag[j] = lo | (hi << 16);
  }

  // e[a][h]: natural row index a of the transform along H, column index g + 8 h
  float e[K][2];
#pragma unroll
  for (int a = 0; a < K; ++a) e[a][0] = e[a][1] = 0.f;

  // ldmatrix.x2.trans: lanes 0-15 give the rows; matrices 0 / 1 are v = 0..7 / 8..15
  const int ld_v = ((lane >> 3) & 1) * 8 + (lane & 7);

  for (uint32_t idx = 0; idx < n_my; ++idx) {
    const int s = static_cast<int>(idx % S);
    const uint32_t parity = (idx / S) & 1u;
    const bool ok = ptx::mbar_wait(&my_bars[s], parity, p.status, (6u << 16) | 2u);
    if (!__all_sync(0xffffffffu, ok)) break;
    const uint32_t tile = ptx::smem_u32(my_tiles + s * Cfg::kTileBytes);

#pragma unroll 1
    for (int nt = 0; nt < 8; ++nt) {
      float dd[4][K];   // [fragment position][u]
#pragma unroll
      for (int u = 0; u < K; ++u) {
        const int row = u * K + ld_v;
        uint32_t b0, b1;
        ldmatrix_x2_trans(tile + row * 128 + ((nt ^ (row & 7)) << 4), b0, b1);
        float d[4] = {0.f, 0.f, 0.f, 0.f};
        mma_bf16_16816(d, afrag, b0, b1);
#pragma unroll
        for (int j = 0; j < 4; ++j) dd[j][u] = d[j];
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        hadamard_vec<K>(dd[j]);
#pragma unroll
        for (int a = 0; a < K; ++a) e[a][j >> 1] = fmaf(dd[j][a], dd[j][a], e[a][j >> 1]);
      }
    }

    __syncwarp();
    if (lane == 0 && idx + S < n_my) {
      ptx::fence_proxy_async_smem();
      issue(idx + S, s);
    }
  }

#pragma unroll
  for (int a = 0; a < K; ++a)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float v = e[a][h];
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      if (tq == 0)
        atomicAdd(&e_sm[sq.seq_of_nat[a] * K + sq.seq_of_nat[g + 8 * h]], static_cast<double>(v));
    }
  __syncthreads();
  const double s2 = static_cast<double>(p.scale[0]) * static_cast<double>(p.scale[0]);
  for (int i = threadIdx.x; i < R; i += NW * 32) atomicAdd(&energy[i], e_sm[i] * s2);
}

bool spectrum_mma_supported(int k, int dtype) {
  return dtype == LBP_BF16 && (k == 4 || k == 8 || k == 16);
}

template <int K>
static int launch_spectrum_mma_k(const CUtensorMap& tmap, const ProjParams& p, const MmaPlan& mp,
                                 double* energy, int sms, cudaStream_t stream) {
  using Cfg = MmaCfg<K>;
  auto kern = wht_spectrum_mma_kernel<K>;
  LBP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
  const uint32_t want = (p.n_items + Cfg::kWarps - 1) / Cfg::kWarps;
  const int grid = static_cast<int>(want < static_cast<uint32_t>(sms) ? want : sms);
  kern<<<grid, Cfg::kWarps * 32, Cfg::kSmemBytes, stream>>>(tmap, p, mp, energy);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

// bp: the plan of all k*k pairs in raster order (i * k + j).
int launch_spectrum_mma(const void* t, int B, int H, int W, int C, const BasisPlan& bp, double* energy,
                        uint32_t* status, cudaStream_t stream) {
  const int K = bp.k;
  CUtensorMap tmap;
  if (int e = encode_block_tensor_map(&tmap, t, LBP_BF16, B, H, W, C, K, 64, true)) return e;
  ProjParams p{};
  p.Hb = blocks_along(H, K);
  p.Wb = blocks_along(W, K);
  p.nb = B * p.Hb * p.Wb;
  p.r = K * K;
  p.bpt = 1;
  p.tile_rows = p.r;
  p.C[0] = p.C[1] = C;
  p.n_chunks[0] = p.n_chunks[1] = (C + 63) / 64;
  const long long n0 = static_cast<long long>(p.nb) * p.n_chunks[0];
  if (n0 >= (1ll << 31)) return LBP_ERR_SHAPE;
  p.n_items0 = p.n_items = static_cast<uint32_t>(n0);
  p.status = status;
  p.scale[0] = p.scale[1] = 1.0f / static_cast<float>(K);
  MmaPlan mp;
  for (int q = 0; q < 64; ++q) {
    mp.nat_i[q] = q < bp.r ? bp.nat_i[q] : 0;
    mp.nat_j[q] = q < bp.r ? bp.nat_j[q] : 0;
  }
  LBP_CUDA_TRY(cudaMemsetAsync(energy, 0, static_cast<size_t>(K) * K * sizeof(double), stream));
  int dev = 0, sms = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (K == 16) {
    Seq16 sq;
    for (int sidx = 0; sidx < 16; ++sidx) sq.seq_of_nat[walsh_natural_index(16, sidx)] = static_cast<uint8_t>(sidx);
    using Cfg = MmaCfg<16>;
    LBP_CUDA_TRY(cudaFuncSetAttribute(wht_spectrum16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      Cfg::kSmemBytes));
    const uint32_t want = (p.n_items + Cfg::kWarps - 1) / Cfg::kWarps;
    const int grid = static_cast<int>(want < static_cast<uint32_t>(sms) ? want : sms);
    wht_spectrum16_kernel<<<grid, Cfg::kWarps * 32, Cfg::kSmemBytes, stream>>>(tmap, p, sq, energy);
    count_launch();
    LBP_CUDA_TRY(cudaGetLastError());
    return LBP_OK;
  }
  if (K == 4) return launch_spectrum_mma_k<4>(tmap, p, mp, energy, sms, stream);
  return launch_spectrum_mma_k<8>(tmap, p, mp, energy, sms, stream);
}

// ---- second pass of the two-pass form (fp32 data, order 16) -----------------

constexpr int kSqThreads = 256;

template <bool BF16>
__global__ void __launch_bounds__(kSqThreads)
    square_reduce_kernel(const void* __restrict__ t_hat, long long rows, int C, int r,
                         double* __restrict__ energy) {
  __shared__ double e_sm[256];
  for (int i = threadIdx.x; i < r; i += kSqThreads) e_sm[i] = 0.0;
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long first = static_cast<long long>(blockIdx.x) * (kSqThreads / 32) + warp;
  const long long stride = static_cast<long long>(gridDim.x) * (kSqThreads / 32);
  for (long long row = first; row < rows; row += stride) {
    float acc = 0.f;
    if constexpr (BF16) {
      const uint4* p = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(t_hat) + row * C);
      for (int v = lane; v < C / 8; v += 32) {
        const uint4 w = p[v];
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int n = 0; n < 4; ++n) {
          const float lo = bf16_lo(ws[n]), hi = bf16_hi(ws[n]);
          acc = fmaf(lo, lo, acc);
          acc = fmaf(hi, hi, acc);
        }
      }
    } else {
      const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(t_hat) + row * C);
      for (int v = lane; v < C / 4; v += 32) {
        const float4 w = p[v];
        acc = fmaf(w.x, w.x, acc);
        acc = fmaf(w.y, w.y, acc);
        acc = fmaf(w.z, w.z, acc);
        acc = fmaf(w.w, w.w, acc);
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) atomicAdd(&e_sm[static_cast<int>(row % r)], static_cast<double>(acc));
  }
  __syncthreads();
  for (int i = threadIdx.x; i < r; i += kSqThreads) atomicAdd(&energy[i], e_sm[i]);
}

// energy[q] = sum over rows with row % r == q and over the C channels of t_hat^2.
// C is a multiple of 8 (bf16) or 4 (fp32) and the rows are 16-byte aligned.
int launch_square_reduce(const void* t_hat, int dtype, long long rows, int C, int r, double* energy,
                         cudaStream_t stream) {
  if (r < 1 || r > 256) return LBP_ERR_BASIS;
  LBP_CUDA_TRY(cudaMemsetAsync(energy, 0, static_cast<size_t>(r) * sizeof(double), stream));
  int dev = 0, sms = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const long long want = (rows + kSqThreads / 32 - 1) / (kSqThreads / 32);
  const int grid = static_cast<int>(want < 4ll * sms ? want : 4ll * sms);
  if (dtype == LBP_BF16)
    square_reduce_kernel<true><<<grid, kSqThreads, 0, stream>>>(t_hat, rows, C, r, energy);
  else
    square_reduce_kernel<false><<<grid, kSqThreads, 0, stream>>>(t_hat, rows, C, r, energy);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

}  // namespace lbp
