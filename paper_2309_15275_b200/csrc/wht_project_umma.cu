// Projection of Eq. 6 for orders 8 and 16 on the tcgen05 tensor cores (bf16, r <= 48).
//
//   t_hat[blk, q, c] = scale * sum_tok B_q[tok] * t[blk, tok, c]
//
// is a product of the +-1 basis matrix (r x 64) with a block's 64 tokens x 64
// channels.  The warp-level mma.sync kernel spends a warp's time on ldmatrix,
// mma and 4-byte stores and moves 55-65 GB/s per SM; a TMA stream alone moves
// twice that.  Here no warp touches the tile: the TMA box lands in shared memory
// in the 128-byte-swizzled layout that is, as it lies, an MN-major B operand
// (k = token, n = channel); four boxes, the 64-channel chunks of an item, lie
// side by side (N = 256), and one elected thread issues four tcgen05.mma (N =
// 256, K = 16 each) per 32 KB of input.  A is the basis matrix, built once per CTA in shared memory,
// K-major; its 32 rows (r real ones, the rest zero) are repeated four times so
// that every lane quarter of TMEM holds all results and each of the four warps
// of an epilogue warpgroup can read the tile it stores from its own quarter.
// The accumulator (two slots of 256 columns) is read back with tcgen05.ld: lane
// q of a warp holds row q of one tile, 64 channels; the warp lays its r rows
// down in shared memory and one TMA store writes them as whole 128-byte lines
// (per-lane stores of 16 bytes to r different rows cost the SM more than the
// loads at r = 16).
//
// Order 16 (template K): a block's 256 tokens are taken as four parts of 64
// (four token rows each, a 4 x 16 box), every part a stage of its own with its
// own 64 columns of the basis matrix, and the four parts accumulate in the same
// accumulator slot: the tile, stage and epilogue shapes stay those of order 8.
//
// Roles: warps 0-3 TMA producers (one chunk each), warp 4 MMA issuer, warps 8-11
// and 12-15 two epilogue warpgroups (slot 0 / slot 1).  Ranks 33-48 (template
// HI): the basis rows repeat every 64 rows instead of every 32, lane quarters 0
// and 2 hold rows 0-31, quarters 1 and 3 rows 32-63; an epilogue warp then takes
// the row half of its quarter for two of the item's chunks, one after the other.  Every
// wait is bounded; a timeout raises the status word and all roles fall through
// to the exit.
#include <cuda_bf16.h>

#include "lbp_internal.h"
#include "ptx_sm100.cuh"
#include "wht_device.cuh"
#include "wht_mma.cuh"
#include "wht_project.cuh"

namespace lbp {
namespace umma {

constexpr int kTileBytes = 64 * 128;             // 64 tokens x 64 channels of bf16
constexpr int M = 128;                           // rows of the tensor-core tile
constexpr int kQuad = 4;                         // 64-channel chunks per item = per stage = per accumulator slot
constexpr int kStageBytes = kQuad * kTileBytes;  // 32 KB
constexpr int kProducers = 4;                    // warps 0-3: each fetches one chunk of an item
constexpr int kPanelBytes = 128 * 128;           // basis matrix for 64 tokens: 128 rows x 128 bytes
constexpr int kOutBytes = 32 * 128;              // an epilogue warp's rows on their way out
constexpr int kThreads = 16 * 32;
// Per order: parts of 64 tokens per block, stages of the ring, shared-memory map.
template <int K>
struct Cfg {
  static constexpr int kParts = K * K / 64;
  static constexpr int kStages = K == 8 ? 5 : 4;
  static constexpr int kOffA = kStages * kStageBytes;
  static constexpr int kOffOut = kOffA + kParts * kPanelBytes;
  static constexpr int kOffBar = kOffOut + 8 * kOutBytes;
  static constexpr int kSmemBytes = kOffBar + 256 + 1024;
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget of one CTA exceeded");
};
constexpr uint32_t kTmemCols = 512, kSlotCols = 256;

// One item (block x four 64-channel chunks of one of the two tensors; in
// ProjParams n_chunks counts such items per block), stepped through without
// divisions: the position is decoded once, then moved by
// precomputed steps with carries.
struct Steps {
  uint32_t chunk, blk, bw, bh, b, grp, j;
};
struct Cursor {
  uint32_t item, which, chunk, blk, bw, bh, b, grp, j;

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
  static __device__ __forceinline__ Steps steps(const ProjParams& p, uint32_t stride, int w) {
    Steps s;
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
  __device__ __forceinline__ void advance(const ProjParams& p, uint32_t stride, const Steps& st) {
    const uint32_t next = item + stride;
    if (which == 0u && next >= p.n_items0) {   // into the second tensor: once per cursor
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

// r rows x 64 channels from shared memory (128-byte swizzle) to the coefficient matrix
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* m, const void* smem_src, int32_t x,
                                                  int32_t y, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;" ::
          "l"(reinterpret_cast<uint64_t>(m)),
      "r"(ptx::smem_u32(smem_src)), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// the source of every committed store has been read / every store is complete
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

template <int K, bool HI>
__global__ void __launch_bounds__(kThreads, 1)
    wht_project_umma_kernel(const __grid_constant__ CUtensorMap tmap0,
                            const __grid_constant__ CUtensorMap tmap1,
                            const __grid_constant__ CUtensorMap tmout0,
                            const __grid_constant__ CUtensorMap tmout1,
                            const __grid_constant__ CUtensorMap tmout0h,   // HI: boxes of the rows from 32 on
                            const __grid_constant__ CUtensorMap tmout1h,
                            __nv_bfloat16* __restrict__ out0, __nv_bfloat16* __restrict__ out1,
                            const __grid_constant__ ProjParams p,
                            const __grid_constant__ MmaPlan mp) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  constexpr int kStages = Cfg<K>::kStages, kParts = Cfg<K>::kParts;
  uint8_t* sA = smem + Cfg<K>::kOffA;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg<K>::kOffBar);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* acc_full = empty_bar + kStages;   // [2]
  uint64_t* acc_empty = acc_full + 2;         // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full_bar[s], kProducers);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&acc_full[s], 1);
      ptx::mbar_init(&acc_empty[s], 4);   // the four warps of the slot's epilogue warpgroup
    }
    ptx::mbar_fence_init();
    *abort_flag = 0;
    ptx::prefetch_tensormap(&tmap0);
    ptx::prefetch_tensormap(&tmap1);
    ptx::prefetch_tensormap(&tmout0);
    ptx::prefetch_tensormap(&tmout1);
  }
  // The basis matrix as K-major A operands, one panel per part of 64 tokens: row
  // m holds basis m % 32 (m % 64 at ranks above 32; zero past r), 64 tokens = 128
  // bytes, 16-byte piece c of row m at piece c ^ (m & 7).
  for (int e = threadIdx.x; e < kParts * M * 8; e += kThreads) {
    const int part = e / (M * 8), m = (e >> 3) % M, c = e & 7;
    const int q = m & (HI ? 63 : 31);
    uint32_t w[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const int tok = part * 64 + c * 8 + 2 * h;
      w[h] = basis_bits<K>(mp, q, p.r, tok) | (basis_bits<K>(mp, q, p.r, tok + 1) << 16);
    }
    *reinterpret_cast<uint4*>(sA + part * kPanelBytes + m * 128 + ((c ^ (m & 7)) << 4)) =
        make_uint4(w[0], w[1], w[2], w[3]);
  }
  ptx::fence_proxy_async_smem();   // the tensor core reads A through the async proxy
  if (warp == 4) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  // a kernel launched behind this one with programmatic serialization may set
  // itself up as SMs free up; it still waits for this grid before reading
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // launched the same way behind an earlier kernel on the stream that may still
  // read the buffers written below: nothing is read or written before it has
  // completed, unless the caller vouches for disjoint buffers (then the wait
  // moves to the end and only keeps completion ordered)
  if (!p.defer_wait) asm volatile("griddepcontrol.wait;" ::: "memory");

  // items dealt to the CTAs round robin
  const uint32_t my_quads =
      blockIdx.x < p.n_items ? (p.n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
  const uint32_t quad_stride = gridDim.x;   // items between a CTA's consecutive ones

  if (warp < kProducers) {
    // =========================== TMA producers ===========================
    // One 8 KB box per chunk, each from a warp of its own: a thread issues TMA
    // requests too slowly to fetch an item alone, and a box of several chunks
    // completes later than its parts would (the stage's bytes are in flight
    // for longer).
    if (ptx::elect_one()) {
      // x and g_y are read exactly once: they should not push the coefficients
      // just written (read back from L2 by the next kernel) out of L2
      const uint64_t stream_once = ptx::l2_policy_evict_first();
      const Steps st0 = Cursor::steps(p, quad_stride, 0), st1 = Cursor::steps(p, quad_stride, 1);
      Cursor c;
      if (my_quads > 0) c.decode(p, blockIdx.x);
      bool ok = true;
      uint32_t it = 0;   // stages issued so far
      for (uint32_t n = 0; n < my_quads && !p.test_stall && ok; ++n) {
        const int chunk = static_cast<int>(c.chunk) * kQuad + warp;
        const bool have = chunk * 64 < p.C[c.which];
        for (int part = 0; part < kParts; ++part, ++it) {
          const int s = static_cast<int>(it % kStages);
          if (!ptx::mbar_wait(&empty_bar[s], ((it / kStages) + 1) & 1u, p.status, (6u << 16) | 1u)) {
            ok = false;
            break;
          }
          if (have) {
            // the whole box counts, also where it hangs over the tensor (zero fill);
            // order 16: part = four token rows of the block
            ptx::mbar_expect_tx(&full_bar[s], kTileBytes);
            ptx::tma_load_4d_hint(smem + s * kStageBytes + warp * kTileBytes, c.which ? &tmap1 : &tmap0,
                                  &full_bar[s], chunk * 64, static_cast<int32_t>(c.bw * K),
                                  static_cast<int32_t>(c.bh * K + part * (64 / K)),
                                  static_cast<int32_t>(c.b), stream_once);
          } else {
            ptx::mbar_arrive(&full_bar[s]);   // no such chunk: what lies in the stage is multiplied and dropped
          }
        }
        if (ok && n + 1 < my_quads) c.advance(p, quad_stride, c.which ? st1 : st0);
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == 4) {
    // =========================== tcgen05 issuer ===========================
    if (ptx::elect_one()) {
      const uint32_t idesc = ptx::idesc_bf16(M, kQuad * 64, false, true);
      const uint32_t a_addr = ptx::smem_u32(sA);
      bool ok = true;
      uint32_t it = 0;   // stages consumed so far
      for (uint32_t n = 0; n < my_quads && ok; ++n) {
        const int slot = static_cast<int>(n & 1u);
        if (!ptx::mbar_wait(&acc_empty[slot], ((n >> 1) + 1) & 1u, p.status, (6u << 16) | 2u)) {
          ok = false;
          break;
        }
        for (int part = 0; part < kParts; ++part, ++it) {
          const int s = static_cast<int>(it % kStages);
          if (!ptx::mbar_wait(&full_bar[s], (it / kStages) & 1u, p.status, (6u << 16) | 3u)) {
            ok = false;
            break;
          }
          ptx::tc_fence_after_sync();
          const uint32_t sb = ptx::smem_u32(smem + s * kStageBytes);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            // A: K-major, 16 tokens = 32 bytes further per step; B: MN-major, 16
            // tokens = 16 rows of 128 bytes further, the four chunks 8 KB apart
            const uint64_t da = ptx::smem_desc_sw128(a_addr + part * kPanelBytes + kk * 32, 16, 1024);
            const uint64_t db = ptx::smem_desc_sw128(sb + kk * 2048, kTileBytes, 1024);
            ptx::mma_bf16_ss(tmem_base + slot * kSlotCols, da, db, idesc, (part == 0 && kk == 0) ? 0u : 1u);
          }
          ptx::mma_commit(&empty_bar[s]);
        }
        if (!ok) break;
        ptx::mma_commit(&acc_full[slot]);
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp >= 8) {
    // =========================== epilogue ===========================
    // Warpgroup g drains slot g (the CTA's quads g, g + 2, ...); its warp w takes
    // item w of the quad and reads it from lane quarter w.
    const int g = (warp - 8) >> 2, w = warp & 3;
    const uint64_t keep = ptx::l2_policy_evict_last();   // read back from L2 by the next kernel
    const uint32_t stride2 = 2u * quad_stride;
    const Steps st0 = Cursor::steps(p, stride2, 0), st1 = Cursor::steps(p, stride2, 1);
    Cursor c;
    if (static_cast<uint32_t>(g) < my_quads) c.decode(p, blockIdx.x + g * gridDim.x);
    uint8_t* const my_out = smem + Cfg<K>::kOffOut + (warp - 8) * kOutBytes;
    // rows this warp reads from its lane quarter, and the chunks it takes
    const int half = HI ? (w & 1) : 0;
    const int nrows = HI ? (half ? p.r - 32 : 32) : p.r;
    constexpr int kTake = HI ? 2 : 1;
    for (uint32_t n = g; n < my_quads; n += 2) {
      const bool ok = ptx::mbar_wait(&acc_full[g], (n >> 1) & 1u, p.status, (6u << 16) | 4u);
      // one answer for the whole warp (the flag may be raised between two lanes' reads)
      if (__any_sync(0xffffffffu, !ok || *abort_flag != 0)) {
        if (lane == 0) *abort_flag = 1;
        break;
      }
      ptx::tc_fence_after_sync();
      const int which = static_cast<int>(c.which);
      const int C = p.C[which];
      const float sc = p.scale[which];
      __nv_bfloat16* __restrict__ out = which ? out1 : out0;
      const long long row0 =
          static_cast<long long>(c.grp) * p.tile_rows + static_cast<long long>(c.j) * p.r;
#pragma unroll
      for (int ci = 0; ci < kTake; ++ci) {
        const int cq = HI ? 2 * (w >> 1) + ci : w;   // chunk of the item
        uint32_t v[2][32];
        const uint32_t taddr =
            tmem_base + (static_cast<uint32_t>(32 * w) << 16) + g * kSlotCols + cq * 64;
        ptx::tmem_ld_32x32(taddr, v[0]);
        ptx::tmem_ld_32x32(taddr + 32, v[1]);
        ptx::tmem_ld_wait();
        if (ci == kTake - 1) {
          ptx::tc_fence_before_sync();
          if (lane == 0) ptx::mbar_arrive(&acc_empty[g]);   // the slot may be overwritten
        }
        const int cbase = (static_cast<int>(c.chunk) * kQuad + cq) * 64;
        if (cbase >= C) continue;
        // the previous store of this warp has read its rows
        if (lane == 0) bulk_wait_read();
        __syncwarp();
        if (lane < nrows) {
          uint8_t* orow = my_out + lane * 128;
#pragma unroll
          for (int piece = 0; piece < 8; ++piece) {
            const uint32_t* f = &v[piece >> 2][(piece & 3) * 8];
            uint4 pk;
            pk.x = pack_bf16x2(__uint_as_float(f[0]) * sc, __uint_as_float(f[1]) * sc);
            pk.y = pack_bf16x2(__uint_as_float(f[2]) * sc, __uint_as_float(f[3]) * sc);
            pk.z = pack_bf16x2(__uint_as_float(f[4]) * sc, __uint_as_float(f[5]) * sc);
            pk.w = pack_bf16x2(__uint_as_float(f[6]) * sc, __uint_as_float(f[7]) * sc);
            *reinterpret_cast<uint4*>(orow + ((piece ^ (lane & 7)) << 4)) = pk;
          }
          ptx::fence_proxy_async_smem();   // the TMA store reads through the async proxy
        }
        __syncwarp();
        if (lane == 0) {
          const CUtensorMap* m = half ? (which ? &tmout1h : &tmout0h) : (which ? &tmout1 : &tmout0);
          tma_store_2d_hint(m, my_out, cbase, static_cast<int32_t>(row0) + 32 * half, keep);
          bulk_commit();
        }
        // rows of a padded row group that no block owns are kept at zero
        if (half == 0 &&
            (c.j == static_cast<uint32_t>(p.bpt - 1) || c.blk == static_cast<uint32_t>(p.nb - 1))) {
          const long long end = static_cast<long long>(c.grp + 1) * p.tile_rows;
          const int piece = lane & 7;
          if (cbase + piece * 8 < C)   // C is a multiple of 8
            for (long long row = row0 + p.r + (lane >> 3); row < end; row += 4)
              *reinterpret_cast<uint4*>(out + row * C + cbase + piece * 8) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
      if (n + 2 < my_quads) c.advance(p, stride2, c.which ? st1 : st0);
    }
    if (lane == 0) bulk_wait_all();   // this warp's stores are complete before the CTA leaves
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
  // deferred: this grid must not complete before the kernel ahead of it has
  if (p.defer_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace umma

bool project_umma_supported(int k, int r) { return (k == 8 || k == 16) && r <= 48; }

int launch_project_umma(const CUtensorMap* tmaps, __nv_bfloat16* out0, __nv_bfloat16* out1,
                        const ProjParams& p, const BasisPlan& bp, int sms, cudaStream_t stream) {
  using namespace umma;
  MmaPlan mp;
  for (int q = 0; q < 64; ++q) {
    mp.nat_i[q] = q < bp.r ? bp.nat_i[q] : 0;
    mp.nat_j[q] = q < bp.r ? bp.nat_j[q] : 0;
  }
  const bool hi = bp.r > 32;
  const bool k16 = bp.k == 16;
  auto kern = k16 ? (hi ? wht_project_umma_kernel<16, true> : wht_project_umma_kernel<16, false>)
                  : (hi ? wht_project_umma_kernel<8, true> : wht_project_umma_kernel<8, false>);
  const int smem_bytes = k16 ? Cfg<16>::kSmemBytes : Cfg<8>::kSmemBytes;
  static bool configured[2][2][64] = {};
  int dev = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[k16][hi][dev]) {
    LBP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
    if (dev >= 0 && dev < 64) configured[k16][hi][dev] = true;
  }
  // coefficient matrices as 2-D maps: a box is the rows x 64 channels of one item
  // that one warp writes (all r rows; at ranks above 32 the first 32 and the rest)
  CUtensorMap tmout[2], tmouth[2];
  const long long rows = (static_cast<long long>(p.nb) + p.bpt - 1) / p.bpt * p.tile_rows;
  if (int e = encode_matrix_tensor_map(&tmout[0], out0, rows, p.C[0], hi ? 32 : bp.r)) return e;
  if (int e = encode_matrix_tensor_map(&tmouth[0], out0, rows, p.C[0], hi ? bp.r - 32 : bp.r)) return e;
  tmout[1] = tmout[0];
  tmouth[1] = tmouth[0];
  if (out1 != nullptr) {
    if (int e = encode_matrix_tensor_map(&tmout[1], out1, rows, p.C[1], hi ? 32 : bp.r)) return e;
    if (int e = encode_matrix_tensor_map(&tmouth[1], out1, rows, p.C[1], hi ? bp.r - 32 : bp.r)) return e;
  }
  const uint32_t want = p.n_items;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  // Alone on the chip the kernel is bound by HBM long before it runs out of SMs,
  // and on three quarters of them it is about 5 % faster than on all (fewer
  // requests in flight against one another); beside a products kernel the
  // caller's launch shape says how many it gets.
  const int sms_alone = projection_launch().max_ctas > 0 ? sms : (3 * sms + 3) / 4;
  cfg.gridDim = dim3(projection_grid(want, sms_alone, attr, &cfg.numAttrs));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cfg.attrs = attr;
  LBP_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmaps[0], tmaps[1], tmout[0], tmout[1], tmouth[0], tmouth[1], out0,
                                  out1, p, mp));
  count_launch();
  LBP_CUDA_TRY(cudaGetLastError());
  return LBP_OK;
}

}  // namespace lbp
