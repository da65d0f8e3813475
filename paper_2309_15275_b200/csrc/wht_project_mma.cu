// Projection kernel for bf16 data (Eq. 6 as the paper writes it: the block,
// as a k*k x C matrix, times the k*k x r matrix of +-1 bases).
//
// The pass is HBM-bound; what has to stay small is the instruction count per
// byte.  Applying the +-1 basis matrix with warp-level bf16 MMAs (exact
// products, fp32 accumulation) needs about a quarter of the instructions of the
// register butterfly, which keeps the load pipeline, not the issue slots, the
// limiter.  Data movement is the same as in the additions-only kernel: one warp
// owns a ring of shared-memory stages, lane 0 issues one 4-D TMA box per
// (block, 64-channel chunk), here with the 128-byte swizzle so that ldmatrix
// reads are conflict-free.
//
// Per tile:  D[q, c] = sum_tok A[q, tok] * X[tok, c]
//   A (r rows padded to 16*MT, k*k columns) lives in registers for the whole
//   kernel, X is the shared-memory tile (tokens x 64 channels), D is scaled by
//   1/k, rounded once to bf16 and stored.
#include <cuda_bf16.h>

#include "lbp_internal.h"
#include "ptx_sm100.cuh"
#include "wht_device.cuh"
#include "wht_mma.cuh"
#include "wht_project.cuh"

namespace lbp {

// Where a warp is in its list of items (item = one block x one 64-channel
// chunk of one of the two tensors; a warp takes every `stride`-th item).  The
// position is decoded with divisions once, then moved by precomputed steps with
// carries: a handful of additions per item where the divisions cost a third of
// the warp's instructions.
struct ItemSteps {
  uint32_t chunk, blk, bw, bh, b, grp, j;   // `stride` items, as steps of each coordinate
};
struct ItemCursor {
  uint32_t item;               // index over both tensors
  uint32_t which;              // 0 / 1: tensor
  uint32_t chunk, blk;         // 64-channel chunk, block
  uint32_t bw, bh, b;          // block coordinates on the grid
  uint32_t grp, j;             // row group and place inside it: blk = grp * bpt + j

  __device__ __forceinline__ void decode(const ProjParams& p, uint32_t it) {
    item = it;
    which = it >= p.n_items0 ? 1u : 0u;
    const uint32_t local = it - (which ? p.n_items0 : 0u);
    const uint32_t nch = static_cast<uint32_t>(p.n_chunks[which]);
    blk = local / nch;
    chunk = local - blk * nch;
    bw = blk % p.Wb;
    const uint32_t t2 = blk / p.Wb;
    bh = t2 % p.Hb;
    b = t2 / p.Hb;
    grp = blk / p.bpt;
    j = blk - grp * p.bpt;
  }
  static __device__ __forceinline__ ItemSteps steps(const ProjParams& p, uint32_t stride, int w) {
    ItemSteps s;
    const uint32_t nch = static_cast<uint32_t>(p.n_chunks[w]);
    s.blk = stride / nch;
    s.chunk = stride - s.blk * nch;
    s.bw = s.blk % p.Wb;
    const uint32_t t2 = s.blk / p.Wb;
    s.bh = t2 % p.Hb;
    s.b = t2 / p.Hb;
    s.grp = s.blk / p.bpt;
    s.j = s.blk - s.grp * p.bpt;
    return s;
  }
  // `stride` items further; st = the steps of the tensor the cursor is in
  __device__ __forceinline__ void advance(const ProjParams& p, uint32_t stride, const ItemSteps& st) {
    const uint32_t next = item + stride;
    if (which == 0u && next >= p.n_items0) {   // into the second tensor: once per warp
      decode(p, next);
      return;
    }
    item = next;
    const uint32_t nch = static_cast<uint32_t>(p.n_chunks[which]);
    chunk += st.chunk;
    const uint32_t carry = chunk >= nch ? 1u : 0u;
    chunk -= carry ? nch : 0u;
    blk += st.blk + carry;
    bw += st.bw + carry;
    if (bw >= static_cast<uint32_t>(p.Wb)) {
      bw -= p.Wb;
      bh += 1u;
    }
    bh += st.bh;
    if (bh >= static_cast<uint32_t>(p.Hb)) {
      bh -= p.Hb;
      b += 1u;
    }
    b += st.b;
    j += st.j + carry;
    if (j >= static_cast<uint32_t>(p.bpt)) {
      j -= p.bpt;
      grp += 1u;
    }
    grp += st.grp;
  }
};

template <int K, int MT>
__global__ void __launch_bounds__(MmaCfg<K>::kWarps * 32, 1)
    wht_project_mma_kernel(const __grid_constant__ CUtensorMap tmap0,
                           const __grid_constant__ CUtensorMap tmap1,
                           __nv_bfloat16* __restrict__ out0, __nv_bfloat16* __restrict__ out1,
                           const __grid_constant__ ProjParams p,
                           const __grid_constant__ MmaPlan mp) {
  using Cfg = MmaCfg<K>;
  constexpr int NW = Cfg::kWarps, S = Cfg::kStages, KS = Cfg::kKSteps;

  extern __shared__ uint8_t smem_raw[];
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
  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap0);
    ptx::prefetch_tensormap(&tmap1);
  }
  // a kernel launched behind this one with programmatic serialization may set
  // itself up as SMs free up; it still waits for this grid before reading
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __syncthreads();
  // this kernel itself may have been launched the same way behind an earlier
  // kernel on the stream (the products kernel of the previous call, which still
  // reads the buffers written below): nothing is read or written before that
  // kernel has completed (unless the caller vouches for disjoint buffers, see
  // ProjParams::defer_wait)
  if (!p.defer_wait) asm volatile("griddepcontrol.wait;" ::: "memory");

  const uint32_t first = blockIdx.x * NW + warp;
  const uint32_t stride = gridDim.x * NW;
  const uint32_t n_my = first < p.n_items ? (p.n_items - first + stride - 1) / stride : 0;
  // x and g_y are read exactly once: they should not push the coefficients just
  // written (read back from L2 by the products kernel) or W out of L2
  const uint64_t stream_once = ptx::l2_policy_evict_first();
  // the coefficients are read back from L2 by the kernel that follows
  const uint64_t keep = ptx::l2_policy_evict_last();

  const ItemSteps steps0 = ItemCursor::steps(p, stride, 0), steps1 = ItemCursor::steps(p, stride, 1);
  auto issue = [&](const ItemCursor& c, int s) {
    ptx::mbar_expect_tx(&my_bars[s], static_cast<uint32_t>(Cfg::kTileBytes));
    ptx::tma_load_4d_hint(my_tiles + s * Cfg::kTileBytes, c.which ? &tmap1 : &tmap0, &my_bars[s],
                          static_cast<int32_t>(c.chunk * 64), static_cast<int32_t>(c.bw * K),
                          static_cast<int32_t>(c.bh * K), static_cast<int32_t>(c.b), stream_once);
  };
  // cur: the item being transformed; ahead: the item S places further, the next to load
  ItemCursor cur, ahead;
  cur.decode(p, first);
  ahead = cur;
#pragma unroll
  for (uint32_t i = 0; i < static_cast<uint32_t>(S); ++i) {
    if (lane == 0 && i < n_my) issue(ahead, static_cast<int>(i));
    ahead.advance(p, stride, ahead.which ? steps1 : steps0);
  }

  // A fragments of m16n8k16, row-major: a0 (row g, k 2tq..+1), a1 (row g+8, same k),
  // a2 (row g, k+8), a3 (row g+8, k+8); the low half of a register is the lower k.
  // Order 16 with more than one row tile would need 64 registers of fragments per
  // tile.  There a k-step is one token row u of the block (16 tokens), so a
  // fragment is its u = 0 form (which depends on v only) with the sign of
  // wal_i(u) on top: four registers and two 16-bit sign masks per row tile.
  constexpr bool kSignsOnTheFly = K == 16 && MT >= 2;
  uint32_t afrag[kSignsOnTheFly ? 1 : MT][kSignsOnTheFly ? 1 : KS][4];
  uint32_t abase[kSignsOnTheFly ? MT : 1][4];
  uint32_t aflip[kSignsOnTheFly ? MT : 1][2];   // bit ks: wal_i(ks) = -1 for row g / g + 8
  if constexpr (!kSignsOnTheFly) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int q = mt * 16 + g + (j & 1) * 8;
          const int tok = ks * 16 + 2 * tq + (j >> 1) * 8;
          afrag[mt][ks][j] = basis_bits<K>(mp, q, p.r, tok) | (basis_bits<K>(mp, q, p.r, tok + 1) << 16);
        }
      }
    }
  } else {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int q = mt * 16 + g + (j & 1) * 8;
        const int v = 2 * tq + (j >> 1) * 8;   // token (u = 0, v)
        abase[mt][j] = basis_bits<K>(mp, q, p.r, v) | (basis_bits<K>(mp, q, p.r, v + 1) << 16);
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int q = mt * 16 + g + h * 8;
        uint32_t m = 0;
        if (q < p.r)
          for (int u = 0; u < 16; ++u) m |= static_cast<uint32_t>(__popc(mp.nat_i[q] & u) & 1) << u;
        aflip[mt][h] = m;
      }
    }
  }
  // fragment of row tile mt at k-step ks
  auto a_fragment = [&](int mt, int ks, uint32_t (&a)[4]) {
    if constexpr (!kSignsOnTheFly) {
#pragma unroll
      for (int j = 0; j < 4; ++j) a[j] = afrag[mt][ks][j];
    } else {
      const uint32_t s0 = ((aflip[mt][0] >> ks) & 1u) * 0x80008000u;
      const uint32_t s1 = ((aflip[mt][1] >> ks) & 1u) * 0x80008000u;
      a[0] = abase[mt][0] ^ s0;
      a[1] = abase[mt][1] ^ s1;
      a[2] = abase[mt][2] ^ s0;
      a[3] = abase[mt][3] ^ s1;
    }
  };

  // ldmatrix.x4.trans source rows: lane -> matrix (lane >> 3), row (lane & 7);
  // matrices 0/1 are tokens +0..7 / +8..15 of channels 0..7 of a 16-channel pair,
  // matrices 2/3 the same tokens of channels 8..15.
  const int ld_tok = ((lane >> 3) & 1) * 8 + (lane & 7);
  const int ld_chunk = lane >> 4;

  for (uint32_t idx = 0; idx < n_my; ++idx) {
    const int s = static_cast<int>(idx % S);
    const uint32_t parity = (idx / S) & 1u;
    const bool ok = ptx::mbar_wait(&my_bars[s], parity, p.status, (3u << 16) | 1u);
    if (!__all_sync(0xffffffffu, ok)) break;

    const int which = static_cast<int>(cur.which);
    const int blk = static_cast<int>(cur.blk);
    const int chunk = static_cast<int>(cur.chunk);
    const int C = p.C[which];
    const float sc = p.scale[which];
    __nv_bfloat16* __restrict__ out = which ? out1 : out0;
    const uint32_t tile = ptx::smem_u32(my_tiles + s * Cfg::kTileBytes);

    // D fragment: d[0..1] = (row g, channels 2tq..+1), d[2..3] = (row g+8, same channels)
    const long long row0 =
        static_cast<long long>(cur.grp) * p.tile_rows + static_cast<long long>(cur.j) * p.r;
    const int cbase = chunk * 64 + 2 * tq;
    // a chunk that lies inside C as a whole needs no check per group of 8 channels
    const bool whole = chunk * 64 + 64 <= C;
    // With three row tiles (ranks 33-48) the 64 channels are taken in two halves,
    // so that the accumulators of a half (3 x 4 x 4 values) fit the registers.
    constexpr int NH = MT >= 3 ? 2 : 1;
    constexpr int NPH = 4 / NH;     // ldmatrix.x4 channel pairs per half
    // order 16 with three row tiles: 192 tensor instructions per half; unrolled
    // as a whole the schedule runs out of registers
    constexpr int kUnrollKs = (kSignsOnTheFly && MT >= 3) ? 4 : KS;
#pragma unroll
    for (int nh = 0; nh < NH; ++nh) {
      if constexpr (kSignsOnTheFly) {
        // keep the compiler from forming all 16 fragments per row tile ahead of the
        // loop and holding them (the register cost this form exists to avoid)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          asm volatile("" : "+r"(aflip[mt][0]), "+r"(aflip[mt][1]));
        }
      }
      float d[MT][2 * NPH][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2 * NPH; ++nt)
#pragma unroll
          for (int j = 0; j < 4; ++j) d[mt][nt][j] = 0.f;

#pragma unroll(kUnrollKs)
      for (int ks = 0; ks < KS; ++ks) {
        const int tok = ks * 16 + ld_tok;
#pragma unroll
        for (int npl = 0; npl < NPH; ++npl) {
          const int c16 = (nh * NPH + npl) * 2 + ld_chunk;   // 16-byte chunk of the 128-byte token row
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(tile + tok * 128 + ((c16 ^ (tok & 7)) << 4), b0, b1, b2, b3);
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            uint32_t a[4];
            a_fragment(mt, ks, a);
            mma_bf16_16816(d[mt][2 * npl], a, b0, b1);
            mma_bf16_16816(d[mt][2 * npl + 1], a, b2, b3);
          }
        }
      }

#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const int q0 = mt * 16 + g, q1 = q0 + 8;
        __nv_bfloat16* o0 = out + (row0 + q0) * C + cbase + nh * (16 * NPH);
        __nv_bfloat16* o1 = o0 + 8 * static_cast<long long>(C);
        if (q0 < p.r) {
#pragma unroll
          for (int nt = 0; nt < 2 * NPH; ++nt)
            if (whole || cbase + nh * (16 * NPH) + nt * 8 < C)   // C is a multiple of 8: 8 channels are all in or all out
              ptx::st_global_hint_u32(o0 + nt * 8, pack_bf16x2(d[mt][nt][0] * sc, d[mt][nt][1] * sc), keep);
        }
        if (q1 < p.r) {
#pragma unroll
          for (int nt = 0; nt < 2 * NPH; ++nt)
            if (whole || cbase + nh * (16 * NPH) + nt * 8 < C)
              ptx::st_global_hint_u32(o1 + nt * 8, pack_bf16x2(d[mt][nt][2] * sc, d[mt][nt][3] * sc), keep);
        }
      }
    }
    // rows of a padded row tile that no block owns are kept at zero
    if (cur.j == static_cast<uint32_t>(p.bpt - 1) || blk == p.nb - 1) {
      const long long tile_base = static_cast<long long>(cur.grp) * p.tile_rows;
      const int c = chunk * 64 + lane * 2;
      if (c < C)
        for (long long row = row0 + p.r; row < tile_base + p.tile_rows; ++row)
          *reinterpret_cast<uint32_t*>(out + row * C + c) = 0u;
    }

    __syncwarp();
    if (lane == 0 && idx + S < n_my) {
      ptx::fence_proxy_async_smem();
      issue(ahead, s);
    }
    ahead.advance(p, stride, ahead.which ? steps1 : steps0);
    cur.advance(p, stride, cur.which ? steps1 : steps0);
  }
  // deferred: this grid must not complete before the kernel ahead of it has
  if (p.defer_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Order 4: a block is only 16 tokens (2 KB per 64 channels), too little per
// TMA request and per barrier wait.  One item is a strip of four blocks that are
// neighbours along W: a 4 x 16 token box, 8 KB, the tile size of order 8.  Row
// u * 16 + v of the tile holds token (u, v) of the strip; block j owns v = 4j..4j+3.
constexpr int kStripBlocks = 4;
constexpr int kStripWarps = 12, kStripStages = 2, kStripTileBytes = 64 * 128;
constexpr int kStripSmemBytes =
    kStripWarps * kStripStages * kStripTileBytes + kStripWarps * kStripStages * 8 + 1024;

__global__ void __launch_bounds__(kStripWarps * 32, 1)
    wht_project_mma_strip4_kernel(const __grid_constant__ CUtensorMap tmap0,
                                  const __grid_constant__ CUtensorMap tmap1,
                                  __nv_bfloat16* __restrict__ out0, __nv_bfloat16* __restrict__ out1,
                                  const __grid_constant__ ProjParams p,
                                  const __grid_constant__ MmaPlan mp) {
  constexpr int K = 4, NW = kStripWarps, S = kStripStages;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + NW * S * kStripTileBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  uint64_t* my_bars = bars + warp * S;
  uint8_t* my_tiles = tiles + warp * S * kStripTileBytes;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < S; ++s) ptx::mbar_init(&my_bars[s], 1);
    ptx::mbar_fence_init();
  }
  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap0);
    ptx::prefetch_tensormap(&tmap1);
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __syncthreads();
  if (!p.defer_wait) asm volatile("griddepcontrol.wait;" ::: "memory");   // see wht_project_mma_kernel

  // items count strips here: p.n_items0 / p.n_items = strips * chunks
  const uint32_t first = blockIdx.x * NW + warp;
  const uint32_t stride = gridDim.x * NW;
  const uint32_t n_my = first < p.n_items ? (p.n_items - first + stride - 1) / stride : 0;
  const uint32_t Wb4 = (static_cast<uint32_t>(p.Wb) + kStripBlocks - 1) / kStripBlocks;
  const uint64_t stream_once = ptx::l2_policy_evict_first();   // as in wht_project_mma_kernel
  const uint64_t keep = ptx::l2_policy_evict_last();

  auto issue = [&](uint32_t idx, int s) {
    uint32_t item = first + idx * stride;
    const int which = item >= p.n_items0;
    if (which) item -= p.n_items0;
    const uint32_t nch = static_cast<uint32_t>(p.n_chunks[which]);
    const uint32_t sg = item / nch, chunk = item - sg * nch;
    const uint32_t bw4 = sg % Wb4, t2 = sg / Wb4, bh = t2 % p.Hb, b = t2 / p.Hb;
    ptx::mbar_expect_tx(&my_bars[s], static_cast<uint32_t>(kStripTileBytes));
    // tokens past W (a last strip of fewer than four blocks) are zero-filled
    ptx::tma_load_4d_hint(my_tiles + s * kStripTileBytes, which ? &tmap1 : &tmap0, &my_bars[s],
                          chunk * 64, bw4 * (K * kStripBlocks), bh * K, b, stream_once);
  };
  if (lane == 0) {
    for (uint32_t i = 0; i < S && i < n_my; ++i) issue(i, i);
  }

  uint32_t afrag[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int q = g + (j & 1) * 8;
    const int tok = 2 * tq + (j >> 1) * 8;
    afrag[j] = basis_bits<K>(mp, q, p.r, tok) | (basis_bits<K>(mp, q, p.r, tok + 1) << 16);
  }

  // token t = 4 u + dv of block j sits in tile row 16 u + 4 j + dv
  const int ld_tok = ((lane >> 3) & 1) * 8 + (lane & 7);
  const int ld_row0 = (ld_tok >> 2) * 16 + (ld_tok & 3);
  const int ld_chunk = lane >> 4;

  for (uint32_t idx = 0; idx < n_my; ++idx) {
    const int s = static_cast<int>(idx % S);
    const uint32_t parity = (idx / S) & 1u;
    const bool ok = ptx::mbar_wait(&my_bars[s], parity, p.status, (3u << 16) | 2u);
    if (!__all_sync(0xffffffffu, ok)) break;

    uint32_t item = first + idx * stride;
    const int which = item >= p.n_items0;
    if (which) item -= p.n_items0;
    const uint32_t nch = static_cast<uint32_t>(p.n_chunks[which]);
    const uint32_t sg = item / nch;
    const int chunk = static_cast<int>(item - sg * nch);
    const uint32_t bw4 = sg % Wb4, t2 = sg / Wb4, bh = t2 % p.Hb, b = t2 / p.Hb;
    const int C = p.C[which];
    const float sc = p.scale[which];
    __nv_bfloat16* __restrict__ out = which ? out1 : out0;
    const uint32_t tile = ptx::smem_u32(my_tiles + s * kStripTileBytes);
    const int cbase = chunk * 64 + 2 * tq;

#pragma unroll
    for (int j = 0; j < kStripBlocks; ++j) {
      const int bw = static_cast<int>(bw4) * kStripBlocks + j;
      if (bw < p.Wb) {
        const int blk = static_cast<int>((b * p.Hb + bh) * p.Wb) + bw;
        float d[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) d[nt][jj] = 0.f;
        const int row = ld_row0 + 4 * j;
#pragma unroll
        for (int np = 0; np < 4; ++np) {
          const int c16 = np * 2 + ld_chunk;
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(tile + row * 128 + ((c16 ^ (row & 7)) << 4), b0, b1, b2, b3);
          mma_bf16_16816(d[2 * np], afrag, b0, b1);
          mma_bf16_16816(d[2 * np + 1], afrag, b2, b3);
        }
        const long long row0 = static_cast<long long>(blk / p.bpt) * p.tile_rows +
                               static_cast<long long>(blk % p.bpt) * p.r;
        const int q0 = g, q1 = g + 8;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const int c = cbase + nt * 8;
          if (c < C) {
            if (q0 < p.r)
              ptx::st_global_hint_u32(out + (row0 + q0) * C + c,
                                      pack_bf16x2(d[nt][0] * sc, d[nt][1] * sc), keep);
            if (q1 < p.r)
              ptx::st_global_hint_u32(out + (row0 + q1) * C + c,
                                      pack_bf16x2(d[nt][2] * sc, d[nt][3] * sc), keep);
          }
        }
        // rows of a padded row tile that no block owns are kept at zero
        if ((blk % p.bpt) == p.bpt - 1 || blk == p.nb - 1) {
          const long long tile_base = static_cast<long long>(blk / p.bpt) * p.tile_rows;
          const int c = chunk * 64 + lane * 2;
          if (c < C)
            for (long long r2 = row0 + p.r; r2 < tile_base + p.tile_rows; ++r2)
              *reinterpret_cast<uint32_t*>(out + r2 * C + c) = 0u;
        }
      }
    }

    __syncwarp();
    if (lane == 0 && idx + S < n_my) {
      ptx::fence_proxy_async_smem();
      issue(idx + S, s);
    }
  }
  // deferred: this grid must not complete before the kernel ahead of it has
  if (p.defer_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
}

int projection_grid(uint32_t want, int sms, cudaLaunchAttribute* attr, unsigned* n_attr) {
  const ProjLaunch shape = projection_launch();
  int cap = shape.max_ctas > 0 && shape.max_ctas < sms ? shape.max_ctas : sms;
  int grid = static_cast<int>(want < static_cast<uint32_t>(cap) ? want : cap);
  unsigned n = 0;
  if (shape.programmatic) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (shape.whole_tpcs && grid >= 2) {
    grid &= ~1;
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = 2;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  *n_attr = n;
  return grid;
}

static int launch_strip4(const CUtensorMap* tmaps, __nv_bfloat16* out0, __nv_bfloat16* out1,
                         const ProjParams& p, const MmaPlan& mp, int sms, cudaStream_t stream) {
  auto kern = wht_project_mma_strip4_kernel;
  LBP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kStripSmemBytes));
  const uint32_t want = (p.n_items + kStripWarps - 1) / kStripWarps;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.gridDim = dim3(projection_grid(want, sms, attr, &cfg.numAttrs));
  cfg.blockDim = dim3(kStripWarps * 32);
  cfg.dynamicSmemBytes = kStripSmemBytes;
  cfg.stream = stream;
  cfg.attrs = attr;
  LBP_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmaps[0], tmaps[1], out0, out1, p, mp));
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

bool project_mma_strips(int k, int r) { return k == 4 && r <= 8; }

bool project_mma_supported(int k, int r) {
  if (k == 4) return r <= 16;
  if (k == 8) return r <= 48;
  if (k == 16) return r <= 48;
  return false;
}

template <int K, int MT>
static int launch_mma_one(const CUtensorMap* tmaps, __nv_bfloat16* out0, __nv_bfloat16* out1,
                          const ProjParams& p, const MmaPlan& mp, int sms, cudaStream_t stream) {
  using Cfg = MmaCfg<K>;
  auto kern = wht_project_mma_kernel<K, MT>;
  static bool configured[64] = {};
  int dev = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    LBP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      Cfg::kSmemBytes));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const uint32_t want = (p.n_items + Cfg::kWarps - 1) / Cfg::kWarps;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.gridDim = dim3(projection_grid(want, sms, attr, &cfg.numAttrs));
  cfg.blockDim = dim3(Cfg::kWarps * 32);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = stream;
  cfg.attrs = attr;
  LBP_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmaps[0], tmaps[1], out0, out1, p, mp));
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

int launch_project_mma(const CUtensorMap* tmaps, __nv_bfloat16* out0, __nv_bfloat16* out1,
                       const ProjParams& p, const BasisPlan& bp, int sms, cudaStream_t stream) {
  MmaPlan mp;
  for (int q = 0; q < 64; ++q) {
    mp.nat_i[q] = q < bp.r ? bp.nat_i[q] : 0;
    mp.nat_j[q] = q < bp.r ? bp.nat_j[q] : 0;
  }
  const int mt = (bp.r + 15) / 16;
  switch (bp.k) {
    case 4:
      // few output rows: strips of four blocks (the caller encoded strip maps and
      // counted strips); at higher rank the stores of a strip outlast its loads
      if (project_mma_strips(bp.k, bp.r)) return launch_strip4(tmaps, out0, out1, p, mp, sms, stream);
      return launch_mma_one<4, 1>(tmaps, out0, out1, p, mp, sms, stream);
    case 8:
      if (mt == 1) return launch_mma_one<8, 1>(tmaps, out0, out1, p, mp, sms, stream);
      if (mt == 2) return launch_mma_one<8, 2>(tmaps, out0, out1, p, mp, sms, stream);
      return launch_mma_one<8, 3>(tmaps, out0, out1, p, mp, sms, stream);
    case 16:
      if (mt == 1) return launch_mma_one<16, 1>(tmaps, out0, out1, p, mp, sms, stream);
      if (mt == 2) return launch_mma_one<16, 2>(tmaps, out0, out1, p, mp, sms, stream);
      return launch_mma_one<16, 3>(tmaps, out0, out1, p, mp, sms, stream);
  }
  return LBP_ERR_BLOCK;
}

}  // namespace lbp
