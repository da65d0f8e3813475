// CTA-pair variant of the persistent products + expansion kernel.
//
// Same work as lbp_products_kernel (both low-rank products of Algorithm 1 with
// Eq. 7 applied in the epilogue), but two CTAs on neighbouring SMs share one
// 256 x BN tile through tcgen05.mma.cta_group::2: each CTA loads its own 128
// rows of A and only half of the B columns, the tensor cores of both SMs read
// the two B halves from both shared memories.  Per SM that is a third less
// operand traffic than a 128 x 256 tile of its own, and operand delivery from
// L2 is what bounds these products.
//
// Pair-tile (CTA rank c = 0, 1):
//   GW (i, j):  rows 256 i + 128 c of g_W, columns BNw j .. ; B half: x_hat
//               columns BNw j + c BNw/2 ..
//   GX (g, n):  row group 2 g + c of g_y_hat; B half: W columns BNx n + c BNx/2 ..
//
// Roles per CTA as in the one-CTA kernel (TMA producer, MMA, eight epilogue
// warps); only the leader (rank 0) issues MMAs.  Barriers:
//   full[s]      leader's; its producer expects the bytes of both CTAs, and the
//                TMA loads of both CTAs complete on it (.cta_group::2 loads)
//   empty[s]     one per CTA; tcgen05.commit multicasts to both
//   acc_full[t]  one per CTA; commit multicasts to both
//   acc_empty[t] leader's; the epilogue warps of both CTAs arrive on it
// No cluster-multicast load is used.  Every wait is bounded.
#include <cuda_bf16.h>
#include <cstdio>
#include <cstdlib>

#include "lbp_fused.cuh"
#include "lbp_fused_epilogue.cuh"
#include "lbp_internal.h"
#include "ptx_sm100.cuh"
#include "wht_device.cuh"

namespace lbp {
namespace fused2 {

using fused::BM;
using fused::kEBytes;
constexpr int fused_max_extra = kFusedMaxExtra;
using fused::kEGroups;
using fused::kEStride;

constexpr int BK = 64;
constexpr int kStages = 6;
constexpr int kABytes = BM * BK * 2;             // 16 KB: this CTA's 128 rows of A
constexpr int kBBytes = 128 * BK * 2;            // 16 KB: this CTA's half of B (up to 128 columns)
constexpr int kStageBytes = kABytes + kBBytes;   // 32 KB
constexpr int kChunkBytes = 64 * BK * 2;
// warps 0-3: TMA producer, tensor-core issuer, two spare; then kEGroups epilogue
// groups of four warps, each a warpgroup of its own (register reallocation below)
constexpr int kThreads = (4 + 4 * kEGroups) * 32;
// Registers per thread once the roles have parted (setmaxnreg).  The launch
// gives each of the three warpgroups 128 x 168 registers; the first keeps
// kRegsFeed per thread, the two epilogue warpgroups grow to kRegsEpilogue.  The
// shares must add up to exactly what the block was launched with: a larger sum
// would leave the last warpgroup waiting for registers that never come.
constexpr int kRegsFeed = 104;
constexpr int kRegsEpilogue = 200;
static_assert(kEGroups == 2 && kRegsFeed + kEGroups * kRegsEpilogue == (1 + kEGroups) * 168,
              "register split must add up to what the block was launched with");
constexpr int kOffE = kStages * kStageBytes;
constexpr int kOffBar = kOffE + kEGroups * kEBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget of one CTA exceeded");
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSlotCols = 256;

// ---- PTX of the CTA-pair forms ------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::
                   : "memory");
}
// shared::cluster address of `local_smem_addr` in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion is signalled on a barrier that may live in the peer CTA
// `policy`: L2 eviction hint (the operands are read by several pairs, from L2)
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* m,
                                                 uint32_t bar_cluster_addr, int32_t x, int32_t y,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      ".L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(ptx::smem_u32(smem_dst)),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                   ptx::smem_u32(smem_dst)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void mma_bf16_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                                 uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at the same shared-memory offset in both CTAs of the pair
__device__ __forceinline__ void mma_commit_pair(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 "
      "[%0], %1;" ::"r"(ptx::smem_u32(bar)),
      "h"(mask)
      : "memory");
}

__device__ __forceinline__ void trace_mark(const FusedParams& p, int slot, bool first_only = false) {
#ifdef LBP_ROLE_TRACE
  if (p.trace != nullptr) {
    unsigned long long now;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
    unsigned long long* t = p.trace + blockIdx.x * kTraceSlots + slot;
    if (first_only) {
      if (*t == 0) *t = now;
    } else {
      atomicMax(t, now);
    }
  }
#else
  (void)p, (void)slot, (void)first_only;
#endif
}

// ------------------------------------------------------------------ kernel ----
template <int K, int LB, int NEX = 0>
__global__ void __launch_bounds__(kThreads, 1)
    lbp_products_pair_kernel(const __grid_constant__ CUtensorMap tm_gyhat_k,
                             const __grid_constant__ CUtensorMap tm_gyhat_mn,
                             const __grid_constant__ CUtensorMap tm_xhat,
                             const __grid_constant__ CUtensorMap tm_w,
                             const __grid_constant__ FusedParams p,
                             const __grid_constant__ FusedBasis fb,
                             const __grid_constant__ FusedSchedule sc) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  float* E = reinterpret_cast<float*>(smem + kOffE);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kOffBar);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* acc_full = empty_bar + kStages;   // [2]
  uint64_t* acc_empty = acc_full + 2;         // [2], the leader's are used
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&acc_full[s], 1);
      ptx::mbar_init(&acc_empty[s], 2 * 4 * kEGroups);   // epilogue warps of both CTAs
    }
    ptx::mbar_fence_init();
    *abort_flag = 0;
    ptx::prefetch_tensormap(&tm_gyhat_k);
    ptx::prefetch_tensormap(&tm_gyhat_mn);
    ptx::prefetch_tensormap(&tm_xhat);
    ptx::prefetch_tensormap(&tm_w);
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, kTmemCols);
    tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();   // the peer's barriers exist before anything is signalled on them
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int my_tiles = unit_tile_count(p, sc, pair, pairs);
  if (threadIdx.x == 0) trace_mark(p, 0);
  // the next kernel on the stream (the projection of the next call) may be
  // scheduled as SMs free up; it waits for this grid before touching memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // The roles part here, and with them the registers: the first warpgroup gives
  // up what it does not need, the epilogue warpgroups take it (the expansion
  // holds a whole coefficient array per thread).
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsFeed));
  if (warp == 0) {
    // =========================== TMA producer (both CTAs) ===========================
    if (ptx::elect_one()) {
      // launched with programmatic stream serialization: x_hat / g_y_hat of the
      // projection kernel may only be read after this wait
      asm volatile("griddepcontrol.wait;" ::: "memory");
      const uint64_t keep = ptx::l2_policy_evict_last();
      uint32_t it = 0;
      bool ok = true;
      for (int ti = 0; ti < my_tiles && ok && !p.test_stall; ++ti) {
        const WorkTile tl = unit_tile(p, sc, pair, pairs, ti);
        const int bn = tl.is_gw ? p.BNw : p.BNx;
        const int half = bn >> 1;
        const uint32_t tx_pair = 2u * static_cast<uint32_t>(kABytes + half * BK * 2);
        for (int kb = tl.kb0; kb < tl.kb0 + tl.n_kb; ++kb) {
          const int s = static_cast<int>(it % kStages);
          if (!ptx::mbar_wait(&empty_bar[s], ((it / kStages) + 1) & 1u, p.status, (5u << 16) | 1u)) {
            ok = false;
            break;
          }
          uint8_t* sa = smem + s * kStageBytes;
          uint8_t* sb = sa + kABytes;
          if (rank == 0) ptx::mbar_expect_tx(&full_bar[s], tx_pair);
          const uint32_t bar = map_to_rank(ptx::smem_u32(&full_bar[s]), 0);
          if (tl.is_gw) {
            const int m0 = tl.a * 256 + static_cast<int>(rank) * 128;
            tma_load_2d_pair(sa, &tm_gyhat_mn, bar, m0, kb * BK, keep);
            tma_load_2d_pair(sa + kChunkBytes, &tm_gyhat_mn, bar, m0 + 64, kb * BK, keep);
            const int n0 = tl.b * bn + static_cast<int>(rank) * half;
            for (int c = 0; c < half / 64; ++c)
              tma_load_2d_pair(sb + c * kChunkBytes, &tm_xhat, bar, n0 + c * 64, kb * BK, keep);
          } else {
            const int g = 2 * tl.a + static_cast<int>(rank);
            tma_load_2d_pair(sa, &tm_gyhat_k, bar, kb * BK, g * BM, keep);
            const int n0 = tl.b * bn + static_cast<int>(rank) * half;
            for (int c = 0; c < half / 64; ++c)
              tma_load_2d_pair(sb + c * kChunkBytes, &tm_w, bar, n0 + c * 64, kb * BK, keep);
          }
          ++it;
        }
      }
      if (!ok) *abort_flag = 1;
      trace_mark(p, 2);
    }
  } else if (warp == 1) {
    // =========================== tcgen05 issuer (leader only) ===========================
    if (rank == 0 && ptx::elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      const uint32_t idesc_w = ptx::idesc_bf16(256, p.BNw, true, true);
      const uint32_t idesc_x = ptx::idesc_bf16(256, p.BNx, false, true);
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        const WorkTile tl = unit_tile(p, sc, pair, pairs, ti);
        const int slot = ti & 1;
        const uint32_t d_tmem = tmem_base + slot * kSlotCols;
        const uint32_t idesc = tl.is_gw ? idesc_w : idesc_x;
        const uint32_t uses = static_cast<uint32_t>(ti >> 1);
        if (!ptx::mbar_wait(&acc_empty[slot], (uses + 1) & 1u, p.status, (5u << 16) | 4u)) {
          ok = false;
          break;
        }
        for (int kb = 0; kb < tl.n_kb; ++kb) {
          const int s = static_cast<int>(it % kStages);
          if (!ptx::mbar_wait(&full_bar[s], (it / kStages) & 1u, p.status, (5u << 16) | 3u)) {
            ok = false;
            break;
          }
          if (kb == 0 && ti < 15) trace_mark(p, 8 + 8 * ti);
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + s * kStageBytes);
          const uint32_t sb = sa + kABytes;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            const uint64_t da = tl.is_gw ? ptx::smem_desc_sw128(sa + kk * 2048, kChunkBytes, 1024)
                                         : ptx::smem_desc_sw128(sa + kk * 32, 16, 1024);
            const uint64_t db = ptx::smem_desc_sw128(sb + kk * 2048, kChunkBytes, 1024);
            mma_bf16_ss_pair(d_tmem, da, db, idesc, (kb == 0 && kk == 0) ? 0u : 1u);
          }
          mma_commit_pair(&empty_bar[s]);
          ++it;
        }
        if (!ok) break;
        mma_commit_pair(&acc_full[slot]);
        if (ti < 15) trace_mark(p, 8 + 8 * ti + 1);
      }
      if (!ok) *abort_flag = 1;
      trace_mark(p, 3);
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsEpilogue));
    // =========================== epilogue (both CTAs, own 128 rows) ===========================
    const int eg = (warp - 4) >> 2;
    const int ew = (warp - 4) & 3;
    const int quarter = warp & 3;
    const int etid = ew * 32 + lane;
    float* const Eg = E + eg * (kEBytes / 4);
    const int bar_id = 1 + eg;
    if (etid < kEStride) Eg[BM * kEStride + etid] = 0.f;   // the zero row of the staging buffer
    fused::named_bar_sync(bar_id, 128);
    for (int ti = 0; ti < my_tiles; ++ti) {
      const WorkTile tl = unit_tile(p, sc, pair, pairs, ti);
      const int slot = ti & 1;
      const uint32_t uses = static_cast<uint32_t>(ti >> 1);
      const bool ok = ptx::mbar_wait(&acc_full[slot], uses & 1u, p.status, (5u << 16) | 5u);
      // One answer for the whole group: a thread that saw its own wait expire, or
      // the flag another role raised, takes the other 127 threads with it (read
      // one by one after the barrier, the flag could split the group, and the
      // threads left inside the tile would wait on a barrier that never fills).
      if (fused::named_bar_or(bar_id, 128, !ok || *abort_flag != 0)) {
        if (etid == 0) *abort_flag = 1;
        break;
      }
      ptx::tc_fence_after_sync();
      if (etid == 0 && ti < 15) trace_mark(p, 8 + 8 * ti + 2 + 2 * eg);
      fused::DrainTile dt;
      dt.is_gw = tl.is_gw;
      dt.bn = tl.is_gw ? p.BNw : p.BNx;
      dt.row_base = tl.a * 256 + static_cast<int>(rank) * 128;
      dt.group = 2 * tl.a + static_cast<int>(rank);
      dt.col_base = tl.b * dt.bn;
      dt.slice = tl.slice;
      dt.tmem_acc = tmem_base + slot * kSlotCols;
      const uint32_t release_bar = map_to_rank(ptx::smem_u32(&acc_empty[slot]), 0);
      fused::drain_tile<K, LB, NEX>(p, fb, dt, Eg, bar_id, eg, etid, quarter, lane,
                               [release_bar]() { mbar_arrive_cluster(release_bar); });
      if (etid == 0 && ti < 15) {
        trace_mark(p, 8 + 8 * ti + 3 + 2 * eg);
#ifdef LBP_ROLE_TRACE
        if (eg == 0 && p.trace != nullptr)
          p.trace[blockIdx.x * kTraceSlots + 8 + 8 * ti + 6] =
              (static_cast<unsigned long long>(tl.is_gw) << 32) | static_cast<unsigned>(tl.n_kb);
#endif
      }
    }
    if (etid == 0) trace_mark(p, 4);
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();   // neither CTA leaves while the other may still touch its memory
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace fused2

// --------------------------------------------------------------- launcher ----
bool fused_pair_supported(const lbp_layer& L, int sms) {
  if (!tune_options().pair) return false;
  return L.Cin >= 128 && sms >= 2 && (sms % 2) == 0;
}

// `p` arrives with the geometry filled in (launch_fused); this chooses the
// pair-tile shapes, launches the projection and then the pair kernel.
int launch_fused_pair(const void* x, const void* x_hat_dense, const void* g_y, const void* W,
                      void* g_W, const lbp_layer& L,
                      const BasisPlan& bp, FusedParams p, const FusedBasis& fb,
                      const FusedLayout& lay, int sms, uint32_t* status, cudaStream_t stream,
                      FusedPhaseHook hook, void* hook_arg) {
  using namespace fused2;
  const FusedOverlap* ov = fused_overlap();
  const int pairs = ov != nullptr && ov->prod_units > 0 && ov->prod_units < sms / 2 ? ov->prod_units
                                                                                    : sms / 2;
  const int mt_w = (L.Cout + 255) / 256;    // 256 rows of g_W per pair-tile
  const int G2 = (p.G + 1) / 2;             // two row groups per GX pair-tile
  const int max_splits_by_ws =
      static_cast<int>(lay.planes_bytes / (static_cast<size_t>(L.Cout) * L.Cin * 4));

  PlanShape shape{};
  shape.Cin = L.Cin;
  shape.Cout = L.Cout;
  shape.G = p.G;
  shape.bpt = p.bpt;
  shape.k = L.k;
  shape.units = pairs;
  shape.pair = 1;
  shape.max_splits = max_splits_by_ws;
  shape.epi_kind = p.n_extra > 0 ? 1 : (p.lb_kernel == 8 ? 2 : 0);
  shape.num_kb_w = p.num_kb_w;
  shape.num_kb_x = p.num_kb_x;
  const TilePlan& plan = plan_products(shape);
  p.BNw = plan.BNw;
  p.BNx = plan.BNx;
  p.gw_splits = plan.splits;
  p.kb_per_split_w = plan.kbps;
#ifdef LBP_ROLE_TRACE
  p.trace = reinterpret_cast<unsigned long long*>(reinterpret_cast<uint8_t*>(p.x_hat) + lay.trace);
  LBP_CUDA_TRY(cudaMemsetAsync(p.trace, 0, kFusedTraceBytes, stream));
#endif
  p.mt_w = mt_w;
  p.n_tx = (L.Cin + p.BNx - 1) / p.BNx;
  p.nt_w = (L.Cin + p.BNw - 1) / p.BNw;
  p.n_gx_tiles = G2 * p.n_tx;
  p.n_gw_tiles = mt_w * p.nt_w * p.gw_splits;

  // Algorithm 1, steps 1-2: x_hat and g_y_hat, rows padded to 128-row groups
  if (int e = fused_project(x, x_hat_dense, g_y, L, bp, p, status, stream)) return e;
  if (hook != nullptr)
    if (int e = hook(hook_arg, stream)) return e;

  CUtensorMap tm_gyhat_k, tm_gyhat_mn, tm_xhat, tm_w;
  const long long rows = static_cast<long long>(p.G) * BM;
  if (int e = encode_matrix_tensor_map(&tm_gyhat_k, p.gy_hat, rows, L.Cout, BM)) return e;
  if (int e = encode_matrix_tensor_map(&tm_gyhat_mn, p.gy_hat, rows, L.Cout, BK)) return e;
  if (int e = encode_matrix_tensor_map(&tm_xhat, p.x_hat, rows, L.Cin, BK)) return e;
  if (int e = encode_matrix_tensor_map(&tm_w, W, L.Cout, L.Cin, BK)) return e;

  const int total_tiles = p.n_gw_tiles + p.n_gx_tiles;
  const int grid = 2 * (total_tiles < pairs ? total_tiles : pairs);

  auto launch = [&](auto kern) -> int {
    LBP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    // Beside a projection on another stream the kernel is launched in plain stream
    // order: launched early, its CTAs would sit on the SMs that projection is
    // meant to get while they wait for the kernel ahead.
    cfg.numAttrs = ov != nullptr ? 1 : 2;
    LBP_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tm_gyhat_k, tm_gyhat_mn, tm_xhat, tm_w, p, fb, plan.sched));
    count_launch();
    LBP_CUDA_TRY(cudaGetLastError());
    if (p.gw_splits > 1)
      return launch_splitk_reduce(p.gw_planes, g_W, static_cast<long long>(L.Cout) * L.Cin,
                                  p.gw_splits, p.gw_bf16 != 0, stream);
    return LBP_OK;
  };
  if (p.n_extra > 0) {
    if (L.k == 8) return launch(lbp_products_pair_kernel<8, 4, fused_max_extra>);
    if (L.k == 16) return launch(lbp_products_pair_kernel<16, 4, fused_max_extra>);
    return LBP_ERR_BASIS;
  }
  switch (L.k * 100 + p.lb_kernel) {
    case 401: return launch(lbp_products_pair_kernel<4, 1>);
    case 402: return launch(lbp_products_pair_kernel<4, 2>);
    case 404: return launch(lbp_products_pair_kernel<4, 4>);
    case 801: return launch(lbp_products_pair_kernel<8, 1>);
    case 802: return launch(lbp_products_pair_kernel<8, 2>);
    case 804: return launch(lbp_products_pair_kernel<8, 4>);
    case 808: return launch(lbp_products_pair_kernel<8, 8>);
    case 1601: return launch(lbp_products_pair_kernel<16, 1>);
    case 1602: return launch(lbp_products_pair_kernel<16, 2>);
    case 1604: return launch(lbp_products_pair_kernel<16, 4>);
    case 1608: return launch(lbp_products_pair_kernel<16, 8>);
  }
  return LBP_ERR_BASIS;
}

}  // namespace lbp
