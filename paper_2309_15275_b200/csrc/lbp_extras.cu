// Small kernels around Algorithm 1 that a ViT layer needs and the paper leaves
// out: accumulation into g_W, the bias gradient, and the row layout change for
// coefficients x_hat that were taken at forward time.
#include <cuda_bf16.h>

#include "lbp_internal.h"
#include "wht_device.cuh"

namespace lbp {

namespace {

// g_W <- beta * g_W + a (+ b):  a, b fp32 (Cout x Cin), g_W fp32 or bf16.
__global__ void __launch_bounds__(256)
    gw_combine_kernel(void* __restrict__ g_W, int gw_bf16, const float* __restrict__ a,
                      const float* __restrict__ b, float beta, long long n4) {
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 v = reinterpret_cast<const float4*>(a)[i];
  if (b != nullptr) {
    const float4 w = reinterpret_cast<const float4*>(b)[i];
    v.x += w.x;
    v.y += w.y;
    v.z += w.z;
    v.w += w.w;
  }
  if (gw_bf16) {
    uint2* dst = reinterpret_cast<uint2*>(g_W) + i;
    if (beta != 0.f) {
      const uint2 old = *dst;
      v.x = fmaf(beta, __uint_as_float(old.x << 16), v.x);
      v.y = fmaf(beta, __uint_as_float(old.x & 0xffff0000u), v.y);
      v.z = fmaf(beta, __uint_as_float(old.y << 16), v.z);
      v.w = fmaf(beta, __uint_as_float(old.y & 0xffff0000u), v.w);
    }
    *dst = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
  } else {
    float4* dst = reinterpret_cast<float4*>(g_W) + i;
    if (beta != 0.f) {
      const float4 old = *dst;
      v.x = fmaf(beta, old.x, v.x);
      v.y = fmaf(beta, old.y, v.y);
      v.z = fmaf(beta, old.z, v.z);
      v.w = fmaf(beta, old.w, v.w);
    }
    *dst = v;
  }
}

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Column sums of selected rows of a (rows, C) matrix, in fp64:
//   partial[slab][c] = sum over the slab's rows of m[row_of(i)][c]
// Row i of the selection is  (i / bpt) * tile_rows + (i % bpt) * r + q  (the DC
// coefficient of block i in a projected tensor) of a dense (rows, C) matrix, or,
// when r == 0, token i of a tensor laid out as `tm` says.
// grid = (ceil(C / 32), slabs); block = 32 x 8: lane = channel, 8 row phases.
template <typename T>
__global__ void __launch_bounds__(256)
    column_sum_kernel(const T* __restrict__ m, long long n_sel, int C, int bpt, int tile_rows, int r,
                      int q, TokenMap tm, double* __restrict__ partial) {
  __shared__ double sm[8][32];
  const int lane = threadIdx.x & 31, ph = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  const long long per = (n_sel + gridDim.y - 1) / gridDim.y;
  const long long i0 = static_cast<long long>(blockIdx.y) * per;
  const long long i1 = i0 + per < n_sel ? i0 + per : n_sel;
  double acc = 0.0;
  if (c < C) {
    for (long long i = i0 + ph; i < i1; i += 8) {
      const long long off =
          r == 0 ? tm.offset(i) : ((i / bpt) * tile_rows + (i % bpt) * r + q) * static_cast<long long>(C);
      acc += static_cast<double>(to_f32<T>(m[off + c]));
    }
  }
  sm[ph][lane] = acc;
  __syncthreads();
  if (ph == 0 && c < C) {
    double s = 0.0;
#pragma unroll
    for (int j = 0; j < 8; ++j) s += sm[j][lane];   // fixed order
    partial[static_cast<long long>(blockIdx.y) * C + c] = s;
  }
}

// g_bias[c] <- beta * g_bias[c] + scale_a * sum_slabs a[slab][c] + sum_slabs b[slab][c]
__global__ void __launch_bounds__(256)
    bias_finish_kernel(float* __restrict__ g_bias, int C, float beta, const double* __restrict__ a,
                       int slabs_a, double scale_a, const double* __restrict__ b, int slabs_b) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  double s = 0.0;
  for (int j = 0; j < slabs_a; ++j) s += a[static_cast<long long>(j) * C + c];
  s *= scale_a;
  for (int j = 0; j < slabs_b; ++j) s += b[static_cast<long long>(j) * C + c];
  if (beta != 0.f) s += static_cast<double>(beta) * static_cast<double>(g_bias[c]);
  g_bias[c] = static_cast<float>(s);
}

__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t w, float f) {
  return pack_bf16x2(bf16_lo(w) * f, bf16_hi(w) * f);
}

// Dense bf16 coefficient rows (block blk, slot q at row blk * r + q) -> rows
// padded to groups: (blk / bpt) * tile_rows + (blk % bpt) * r + q; rows no block
// owns are zero.  Values are multiplied by `factor`, a power of two (exact).
// One thread moves 16 bytes.
__global__ void __launch_bounds__(256)
    regroup_rows_kernel(const uint4* __restrict__ dense, uint4* __restrict__ grouped, int nb, int r,
                        int bpt, int tile_rows, int row_vec /* 16-byte pieces per row */,
                        long long n_vec /* groups * tile_rows * row_vec */, float factor) {
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n_vec) return;
  const long long row = i / row_vec;
  const int piece = static_cast<int>(i - row * row_vec);
  const long long g = row / tile_rows;
  const int j = static_cast<int>(row - g * tile_rows);
  const long long blk = g * bpt + j / r;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (j < bpt * r && blk < nb) {
    v = dense[(blk * r + j % r) * row_vec + piece];
    if (factor != 1.f) {
      v.x = scale_bf16x2(v.x, factor);
      v.y = scale_bf16x2(v.y, factor);
      v.z = scale_bf16x2(v.z, factor);
      v.w = scale_bf16x2(v.w, factor);
    }
  }
  grouped[i] = v;
}

// Moves n_tok tokens of C channels between a tensor laid out as `tm` says and a
// dense (n_tok, C) matrix; one thread moves 16 bytes.  Strides in 16-byte units.
__global__ void __launch_bounds__(256)
    copy_tokens_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, long long n_vec,
                       int row_vec, TokenMap tm16, int to_dense) {
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n_vec) return;
  const long long tok = i / row_vec;
  const int piece = static_cast<int>(i - tok * row_vec);
  const long long far = tm16.offset(tok) + piece;
  if (to_dense)
    dst[i] = src[far];
  else
    dst[far] = src[i];
}

}  // namespace

int launch_copy_tokens(const void* src, void* dst, bool to_dense, long long n_tok, int C, int dtype,
                       TokenMap tm, cudaStream_t stream) {
  if (n_tok <= 0) return LBP_OK;
  const int es = dtype == LBP_BF16 ? 2 : 4;
  const int per = 16 / es;   // elements per 16 bytes; every stride is a multiple of it
  const int row_vec = C / per;
  TokenMap tm16{tm.HW, tm.W, tm.s_image / per, tm.s_row / per, tm.s_tok / per};
  const long long n_vec = n_tok * row_vec;
  copy_tokens_kernel<<<static_cast<unsigned>((n_vec + 255) / 256), 256, 0, stream>>>(
      static_cast<const uint4*>(src), static_cast<uint4*>(dst), n_vec, row_vec, tm16, to_dense ? 1 : 0);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

int launch_gw_combine(void* g_W, bool gw_bf16, const float* a, const float* b, float beta,
                      long long mn, cudaStream_t stream) {
  const long long n4 = mn / 4;   // Cin * element size is a multiple of 16 bytes, so mn % 4 == 0
  gw_combine_kernel<<<static_cast<unsigned>((n4 + 255) / 256), 256, 0, stream>>>(
      g_W, gw_bf16 ? 1 : 0, a, b, beta, n4);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

int bias_slabs(long long n_sel) {
  if (n_sel <= 0) return 0;
  const long long s = (n_sel + 255) / 256;   // at least 256 rows per slab
  return static_cast<int>(s < 64 ? s : 64);
}

int launch_column_sum(const void* m, int dtype, long long n_sel, int C, RowMap rows, int r, int q,
                      double* partial, cudaStream_t stream, const TokenMap* tokens) {
  const TokenMap tm = tokens != nullptr ? *tokens : TokenMap{1, 1, C, C, C};
  const int slabs = bias_slabs(n_sel);
  if (slabs == 0) return LBP_OK;
  dim3 grid(static_cast<unsigned>((C + 31) / 32), static_cast<unsigned>(slabs));
  if (dtype == LBP_BF16)
    column_sum_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(m), n_sel, C, rows.bpt, rows.tile_rows, r, q, tm, partial);
  else
    column_sum_kernel<float><<<grid, 256, 0, stream>>>(static_cast<const float*>(m), n_sel, C,
                                                      rows.bpt, rows.tile_rows, r, q, tm, partial);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

int launch_bias_finish(float* g_bias, int C, float beta, const double* a, int slabs_a, double scale_a,
                       const double* b, int slabs_b, cudaStream_t stream) {
  bias_finish_kernel<<<(C + 255) / 256, 256, 0, stream>>>(g_bias, C, beta, a, slabs_a, scale_a, b,
                                                         slabs_b);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

int launch_regroup_rows(const void* dense, void* grouped, int nb, int r, RowMap rows, int C,
                        float factor, cudaStream_t stream) {
  const int row_vec = C * 2 / 16;
  const long long groups = (static_cast<long long>(nb) + rows.bpt - 1) / rows.bpt;
  const long long n_vec = groups * rows.tile_rows * row_vec;
  regroup_rows_kernel<<<static_cast<unsigned>((n_vec + 255) / 256), 256, 0, stream>>>(
      static_cast<const uint4*>(dense), static_cast<uint4*>(grouped), nb, r, rows.bpt,
      rows.tile_rows, row_vec, n_vec, factor);
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

}  // namespace lbp
