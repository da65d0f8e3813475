// Register-resident Walsh-Hadamard building blocks used by the projection
// (Eq. 6) and expansion (Eq. 7) kernels.
//
// A thread owns one 32-bit word of the channel axis: two bf16 channels or one
// fp32 channel.  A k x k block is first pooled to LB x LB partial sums (Walsh
// rows of sequency < LB are constant on runs of k/LB), then an LB x LB
// Hadamard butterfly in natural order produces all LB*LB low-order
// coefficients with additions and subtractions only.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace lbp {

// Kernel-side copy of the basis plan (passed by value in the launch).
struct DevicePlan {
  int16_t qmap[256];  // [a * LB + b] -> slot q, or -1
};

template <int LB, int NCH>
__device__ __forceinline__ void hadamard_rows(float (&S)[LB][LB][NCH]) {
#pragma unroll
  for (int len = 1; len < LB; len <<= 1) {
#pragma unroll
    for (int a = 0; a < LB; ++a) {
      if ((a & len) == 0) {
#pragma unroll
        for (int b = 0; b < LB; ++b) {
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            const float x = S[a][b][c], y = S[a + len][b][c];
            S[a][b][c] = x + y;
            S[a + len][b][c] = x - y;
          }
        }
      }
    }
  }
}

template <int LB, int NCH>
__device__ __forceinline__ void hadamard_cols(float (&S)[LB][LB][NCH]) {
#pragma unroll
  for (int len = 1; len < LB; len <<= 1) {
#pragma unroll
    for (int b = 0; b < LB; ++b) {
      if ((b & len) == 0) {
#pragma unroll
        for (int a = 0; a < LB; ++a) {
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            const float x = S[a][b][c], y = S[a][b + len][c];
            S[a][b][c] = x + y;
            S[a][b + len][c] = x - y;
          }
        }
      }
    }
  }
}

// Natural-order Hadamard butterfly of a length-N register vector.
template <int N>
__device__ __forceinline__ void hadamard_vec(float (&v)[N]) {
#pragma unroll
  for (int len = 1; len < N; len <<= 1) {
#pragma unroll
    for (int a = 0; a < N; ++a) {
      if ((a & len) == 0) {
        const float x = v[a], y = v[a + len];
        v[a] = x + y;
        v[a + len] = x - y;
      }
    }
  }
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&p);
}

// Unpack one 32-bit word into NCH channel values.
//   fp32 data: NCH = 1, the word is the value.
//   bf16 data: NCH = 2 -> both halves; NCH = 1 -> half `sel` (0 = low).
template <bool BF16, int NCH>
__device__ __forceinline__ void unpack_word(uint32_t w, int sel, float (&f)[NCH]) {
  if constexpr (!BF16) {
    f[0] = __uint_as_float(w);
  } else if constexpr (NCH == 2) {
    f[0] = bf16_lo(w);
    f[1] = bf16_hi(w);
  } else {
    f[0] = sel ? bf16_hi(w) : bf16_lo(w);
  }
}

}  // namespace lbp
