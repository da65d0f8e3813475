// Energy of the basis responses (Sec. 3.2, profiling step of the
// low-heuristic-error selection): sum of squares of a projected tensor per
// basis slot.  The tensor is stored (blocks * r, C) with slot q = row % r.
//
// One warp per row: the lanes square and add their share of the C channels in
// fp32, the warp total goes to a per-CTA fp64 table in shared memory, and each
// CTA adds its table to the result once.
#include <cuda_bf16.h>

#include "lbp_internal.h"
#include "wht_device.cuh"

namespace lbp {

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
