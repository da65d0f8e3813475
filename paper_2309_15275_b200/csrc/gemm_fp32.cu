// fp32 products of the low-rank space (Algorithm 1) on the FFMA pipe.
//
// fp32 data must meet a 1e-5 relative error, which a single-pass TF32 tensor
// product (10-bit mantissa) cannot; the fp32 shapes are small, so a plain
// shared-memory tiled FFMA kernel is used.
//   D[M, N] = sum_k A(m, k) * B(k, n),  B stored (K, N) row-major,
//   A stored (M, K) row-major or, when A_MN, (K, M) row-major.
#include "lbp_internal.h"

namespace lbp {

constexpr int kTM = 64, kTN = 64, kTK = 16;

template <bool A_MN>
__global__ void __launch_bounds__(256)
    gemm_fp32_kernel(const float* __restrict__ A, const float* __restrict__ Bm,
                     float* __restrict__ D, long long M, long long N, long long K) {
  __shared__ float As[kTK][kTM + 4];
  __shared__ float Bs[kTK][kTN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;  // 16 x 16 threads, 4 x 4 outputs each
  const long long m0 = static_cast<long long>(blockIdx.y) * kTM;
  const long long n0 = static_cast<long long>(blockIdx.x) * kTN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (long long k0 = 0; k0 < K; k0 += kTK) {
    // 64 x 16 elements of each operand, 4 per thread
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;
      {
        int kk, mm;
        if (A_MN) {
          kk = idx / kTM;
          mm = idx % kTM;
        } else {
          mm = idx / kTK;
          kk = idx % kTK;
        }
        const long long gm = m0 + mm, gk = k0 + kk;
        float v = 0.f;
        if (gm < M && gk < K) v = A_MN ? A[gk * M + gm] : A[gm * K + gk];
        As[kk][mm] = v;
      }
      {
        const int kk = idx / kTN, nn = idx % kTN;
        const long long gn = n0 + nn, gk = k0 + kk;
        Bs[kk][nn] = (gn < N && gk < K) ? Bm[gk * N + gn] : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kTK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const long long gn = n0 + tx * 4 + j;
      if (gn < N) D[gm * N + gn] = acc[i][j];
    }
  }
}

int launch_gemm_fp32(const float* A, bool a_mn_major, const float* Bm, float* D, long long M,
                     long long N, long long K, cudaStream_t stream) {
  dim3 grid(static_cast<unsigned>((N + kTN - 1) / kTN), static_cast<unsigned>((M + kTM - 1) / kTM));
  if (a_mn_major)
    gemm_fp32_kernel<true><<<grid, 256, 0, stream>>>(A, Bm, D, M, N, K);
  else
    gemm_fp32_kernel<false><<<grid, 256, 0, stream>>>(A, Bm, D, M, N, K);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

}  // namespace lbp
