// bf16 products of the low-rank space (Algorithm 1: g_W = g_y_hat^T x_hat and
// g_x_hat = g_y_hat W; Eq. 2 in the full-rank mode) on the tcgen05 tensor cores.
//
//   D[M, N] = sum_k A(m, k) * B(k, n),  fp32 accumulation in TMEM.
//   B is stored (K, N) row-major, i.e. N-contiguous ("MN-major" operand).
//   A is stored (M, K) row-major (K-major operand) or, when A_MN, (K, M)
//   row-major (MN-major operand).
// None of the operands is ever transposed in memory: the shared-memory matrix
// descriptors tell the tensor core which way each tile lies.
//
// One CTA computes one 128 x BN tile over one K slice.  Warp 0 feeds a 4-stage
// shared-memory ring with TMA (128-byte swizzle), warp 1 allocates TMEM and
// issues tcgen05.mma, warps 2-5 drain the accumulator.  Every wait is bounded.
#include <cuda_bf16.h>

#include "lbp_internal.h"
#include "ptx_sm100.cuh"

namespace lbp {

namespace {

constexpr int BM = 128;          // UMMA M
constexpr int BK = 64;           // k-elements per stage (128 B of a K-major row)
constexpr int kStages = 4;
constexpr int kABytes = BM * BK * 2;        // 16 KB
constexpr int kBBytesMax = 256 * BK * 2;    // 32 KB
constexpr int kStageBytes = kABytes + kBBytesMax;
constexpr int kChunkBytes = 64 * BK * 2;    // one 64-wide MN chunk of an MN-major tile: 8 KB
constexpr int kThreads = 192;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;

struct GemmParams {
  long long M, N, K;
  int32_t BN;            // 64, 128, 192 or 256
  int32_t kb_per_split;  // k-blocks per K slice
  int32_t num_kb;        // ceil(K / BK)
  int32_t splits;
  int32_t d_bf16;        // 1: D is bf16 (only when splits == 1)
  void* D;               // (M, N) row-major, or fp32 partials [split][M][N] when splits > 1
  uint32_t* status;
};

template <bool A_MN>
__global__ void __launch_bounds__(kThreads, 1)
    gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a,
                     const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* accum_bar = empty_bar + kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_bar + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long n0 = static_cast<long long>(blockIdx.x) * p.BN;
  const long long m0 = static_cast<long long>(blockIdx.y) * BM;
  const int split = blockIdx.z;
  const int kb_begin = split * p.kb_per_split;
  const int kb_end = min(kb_begin + p.kb_per_split, p.num_kb);
  const int n_kb = kb_end - kb_begin;
  const uint32_t tmem_cols = p.BN <= 64 ? 64u : (p.BN <= 128 ? 128u : 256u);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    ptx::mbar_init(accum_bar, 1);
    ptx::mbar_fence_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (ptx::elect_one()) {
      const uint32_t stage_tx = static_cast<uint32_t>(kABytes + p.BN * BK * 2);
      for (int i = 0; i < n_kb; ++i) {
        const int s = i % kStages;
        const uint32_t parity = static_cast<uint32_t>(((i / kStages) + 1) & 1);
        if (!ptx::mbar_wait(&empty_bar[s], parity, p.status, (2u << 16) | 1u)) break;
        uint8_t* sa = smem + s * kStageBytes;
        uint8_t* sb = sa + kABytes;
        const int k0 = (kb_begin + i) * BK;
        ptx::mbar_expect_tx(&full_bar[s], stage_tx);
        if constexpr (A_MN) {
          // A stored (K, M): two boxes of 64 m x 64 k
          ptx::tma_load_2d(sa, &tmap_a, &full_bar[s], static_cast<int32_t>(m0), k0);
          ptx::tma_load_2d(sa + kChunkBytes, &tmap_a, &full_bar[s], static_cast<int32_t>(m0 + 64),
                           k0);
        } else {
          // A stored (M, K): one box of 64 k x 128 m
          ptx::tma_load_2d(sa, &tmap_a, &full_bar[s], k0, static_cast<int32_t>(m0));
        }
        for (int c = 0; c < p.BN / 64; ++c)
          ptx::tma_load_2d(sb + c * kChunkBytes, &tmap_b, &full_bar[s],
                           static_cast<int32_t>(n0 + c * 64), k0);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (ptx::elect_one()) {
      const uint32_t idesc = ptx::idesc_bf16(BM, p.BN, A_MN, true);
      bool ok = true;
      for (int i = 0; i < n_kb && ok; ++i) {
        const int s = i % kStages;
        const uint32_t parity = static_cast<uint32_t>((i / kStages) & 1);
        ok = ptx::mbar_wait(&full_bar[s], parity, p.status, (2u << 16) | 2u);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t sa = ptx::smem_u32(smem + s * kStageBytes);
        const uint32_t sb = sa + kABytes;
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
          uint64_t da, db;
          if constexpr (A_MN)
            da = ptx::smem_desc_sw128(sa + kk * 2048, kChunkBytes, 1024);
          else
            da = ptx::smem_desc_sw128(sa + kk * 32, 16, 1024);
          db = ptx::smem_desc_sw128(sb + kk * 2048, kChunkBytes, 1024);
          ptx::mma_bf16_ss(tmem_base, da, db, idesc, (i > 0 || kk > 0) ? 1u : 0u);
        }
        ptx::mma_commit(&empty_bar[s]);   // frees the stage once the MMAs have read it
      }
      ptx::mma_commit(accum_bar);         // accumulator complete
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> global ----------------
    const int quarter = warp & 3;          // TMEM lane quarter this warp may read
    const long long row = m0 + quarter * 32 + lane;
    bool ok = true;
    if (n_kb > 0) ok = ptx::mbar_wait(accum_bar, 0, p.status, (2u << 16) | 3u);
    ok = __all_sync(0xffffffffu, ok);
    ptx::tc_fence_after_sync();
    if (ok) {
      for (int c0 = 0; c0 < p.BN; c0 += 32) {
        uint32_t v[32];
        if (n_kb > 0) {
          ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + c0, v);
          ptx::tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
        if (row < p.M) {
          if (p.d_bf16) {
            __nv_bfloat16* d = static_cast<__nv_bfloat16*>(p.D) + row * p.N;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              const long long col = n0 + c0 + j;
              if (col < p.N) {   // N is a multiple of 8
                uint4 o;
                __nv_bfloat162 t0 = __floats2bfloat162_rn(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                __nv_bfloat162 t1 = __floats2bfloat162_rn(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                __nv_bfloat162 t3 = __floats2bfloat162_rn(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                o.x = *reinterpret_cast<uint32_t*>(&t0);
                o.y = *reinterpret_cast<uint32_t*>(&t1);
                o.z = *reinterpret_cast<uint32_t*>(&t2);
                o.w = *reinterpret_cast<uint32_t*>(&t3);
                *reinterpret_cast<uint4*>(d + col) = o;
              }
            }
          } else {
            float* d = static_cast<float*>(p.D) +
                       (static_cast<long long>(split) * p.M + row) * p.N;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const long long col = n0 + c0 + j;
              if (col < p.N) {   // N is a multiple of 4
                *reinterpret_cast<uint4*>(d + col) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
              }
            }
          }
        }
      }
    }
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, tmem_cols);
  }
}

// Sum fp32 partial tiles [splits][M*N] and write D (fp32 or bf16).
__global__ void __launch_bounds__(256)
    splitk_reduce_kernel(const float* __restrict__ part, void* __restrict__ D, long long mn,
                         int splits, int d_bf16) {
  const long long i4 = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
  if (i4 >= mn) return;
  float4 acc = *reinterpret_cast<const float4*>(part + i4);
  for (int s = 1; s < splits; ++s) {
    const float4 v = *reinterpret_cast<const float4*>(part + static_cast<long long>(s) * mn + i4);
    acc.x += v.x;
    acc.y += v.y;
    acc.z += v.z;
    acc.w += v.w;
  }
  if (d_bf16) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t*>(&lo);
    o.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(D) + i4) = o;
  } else {
    *reinterpret_cast<float4*>(static_cast<float*>(D) + i4) = acc;
  }
}

struct Tiling {
  int BN;
  int splits;
  int kb_per_split;
  int num_kb;
};

// Rough cost model, in SM cycles, used only to rank tilings.
//   per k-block: the slower of the MMA (2 * BN cycles for 128 x BN x 64) and the
//   shared-memory fill of the stage (~100 B/cycle);
//   per CTA: set-up plus an epilogue proportional to the tile;
//   split-K adds a pass over the fp32 partial planes.
static long long max_splits_for(int num_kb, long long tiles, int sms) {
  long long s = sms / (tiles > 0 ? tiles : 1);
  const long long by_k = num_kb / 4 > 0 ? num_kb / 4 : 1;   // >= 4 k-blocks per slice
  if (s > by_k) s = by_k;
  return s < 1 ? 1 : s;
}

Tiling choose_tiling(long long M, long long N, long long K, int sms) {
  Tiling best{};
  double best_cost = -1.0;
  const int num_kb = static_cast<int>((K + BK - 1) / BK);
  const long long tiles_m = (M + BM - 1) / BM;
  const int n64 = static_cast<int>((N + 63) / 64) * 64;
  for (int bn = 256; bn >= 64; bn -= 64) {
    if (bn > n64) continue;   // wider than the matrix
    const long long tiles = tiles_m * ((N + bn - 1) / bn);
    const long long smax = max_splits_for(num_kb, tiles, sms);
    for (long long sp = 1; sp <= smax; ++sp) {
      const int per = static_cast<int>((num_kb + sp - 1) / sp);
      const int splits = (num_kb + per - 1) / per;
      if (splits != sp) continue;
      const long long ctas = tiles * splits;
      const long long waves = (ctas + sms - 1) / sms;
      const double mma = 2.0 * bn, fill = (kABytes + bn * 128.0) / 100.0;
      const double per_kb = mma > fill ? mma : fill;
      double cost = waves * (per * per_kb + 2500.0 + bn * 6.0);
      if (splits > 1)
        cost += 3000.0 + (splits + 1.0) * static_cast<double>(M) * N * 4.0 / 4300.0;
      if (best_cost < 0 || cost < best_cost) {
        best_cost = cost;
        best.BN = bn;
        best.splits = splits;
        best.kb_per_split = per;
        best.num_kb = num_kb;
      }
    }
  }
  if (best_cost < 0) {   // N narrower than 64: one 64-wide tile column
    best.BN = 64;
    best.num_kb = num_kb;
    best.splits = 1;
    best.kb_per_split = num_kb;
  }
  return best;
}

}  // namespace

int launch_gemm_fp32(const float* A, bool a_mn_major, const float* Bm, float* D, long long M,
                     long long N, long long K, cudaStream_t stream);

int launch_splitk_reduce(const float* planes, void* D, long long mn, int splits, bool d_bf16,
                         cudaStream_t stream) {
  const long long threads = (mn + 3) / 4;
  splitk_reduce_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, stream>>>(
      planes, D, mn, splits, d_bf16 ? 1 : 0);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

size_t gemm_splitk_ws_bytes(long long M, long long N, long long K, int in_dtype) {
  if (in_dtype != LBP_BF16) return 0;
  // Enough for the most split tiling the planner can pick on a device with up
  // to 256 SMs; launch_gemm never uses more slices than the scratch it is given.
  const int num_kb = static_cast<int>((K + BK - 1) / BK);
  const long long tiles_m = (M + BM - 1) / BM;
  long long most = 1;
  for (int bn = 64; bn <= 256; bn += 64) {
    const long long tiles = tiles_m * ((N + bn - 1) / bn);
    const long long sp = max_splits_for(num_kb, tiles, 256);
    if (sp > most) most = sp;
  }
  if (most <= 1) return 0;
  return static_cast<size_t>(most) * static_cast<size_t>(M) * static_cast<size_t>(N) * 4;
}

int launch_gemm(const void* A, bool a_mn_major, const void* Bm, void* D, int in_dtype, int d_dtype,
                long long M, long long N, long long K, float* splitk_ws, size_t splitk_ws_bytes,
                uint32_t* status, cudaStream_t stream) {
  if (in_dtype == LBP_F32) {
    if (d_dtype != LBP_F32) return LBP_ERR_DTYPE;
    return launch_gemm_fp32(static_cast<const float*>(A), a_mn_major, static_cast<const float*>(Bm),
                            static_cast<float*>(D), M, N, K, stream);
  }
  int dev = 0, sms = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  Tiling t = choose_tiling(M, N, K, sms);
  if (t.splits > 1) {
    const size_t need = static_cast<size_t>(t.splits) * M * N * 4;
    if (splitk_ws == nullptr || need > splitk_ws_bytes) {
      // not enough scratch for this split: fall back to fewer slices
      const int fit = splitk_ws ? static_cast<int>(splitk_ws_bytes / (static_cast<size_t>(M) * N * 4)) : 0;
      const int splits = fit >= 2 ? fit : 1;
      t.kb_per_split = (t.num_kb + splits - 1) / splits;
      t.splits = (t.num_kb + t.kb_per_split - 1) / t.kb_per_split;
    }
  }

  CUtensorMap tmap_a, tmap_b;
  if (a_mn_major) {
    if (int e = encode_matrix_tensor_map(&tmap_a, A, K, M, BK)) return e;
  } else {
    if (int e = encode_matrix_tensor_map(&tmap_a, A, M, K, BM)) return e;
  }
  if (int e = encode_matrix_tensor_map(&tmap_b, Bm, K, N, BK)) return e;

  GemmParams p;
  p.M = M;
  p.N = N;
  p.K = K;
  p.BN = t.BN;
  p.kb_per_split = t.kb_per_split;
  p.num_kb = t.num_kb;
  p.splits = t.splits;
  p.d_bf16 = (t.splits == 1 && d_dtype == LBP_BF16) ? 1 : 0;
  p.D = t.splits == 1 ? D : static_cast<void*>(splitk_ws);
  p.status = status;

  dim3 grid(static_cast<unsigned>((N + t.BN - 1) / t.BN), static_cast<unsigned>((M + BM - 1) / BM),
            static_cast<unsigned>(t.splits));
  static bool configured[2] = {false, false};
  if (a_mn_major) {
    if (!configured[1]) {
      LBP_CUDA_TRY(cudaFuncSetAttribute(gemm_bf16_kernel<true>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
      configured[1] = true;
    }
    gemm_bf16_kernel<true><<<grid, kThreads, kSmemBytes, stream>>>(tmap_a, tmap_b, p);
  } else {
    if (!configured[0]) {
      LBP_CUDA_TRY(cudaFuncSetAttribute(gemm_bf16_kernel<false>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
      configured[0] = true;
    }
    gemm_bf16_kernel<false><<<grid, kThreads, kSmemBytes, stream>>>(tmap_a, tmap_b, p);
  }
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());

  if (t.splits > 1) {
    const long long mn = M * N;
    const long long threads = (mn + 3) / 4;
    splitk_reduce_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, stream>>>(
        splitk_ws, D, mn, t.splits, d_dtype == LBP_BF16 ? 1 : 0);
    count_launch();
    LBP_CUDA_TRY(cudaGetLastError());
  }
  return LBP_OK;
}

}  // namespace lbp
