// Persistent kernel for the low-rank products and the expansion of Algorithm 1
// (bf16 data, r <= 16), run after the projection kernel.
//
// One CTA per SM works through a static list of output tiles of the two
// products, fp32 accumulators in TMEM, operands fed by TMA:
//
//   GW tile (i, j):  g_W[128 i .., BNw j ..] = g_y_hat^T x_hat      K = all low-rank rows
//   GX tile (m, n):  g_x_hat[group m, BNx n ..] = g_y_hat[m] W      K = Cout
//
// A GX tile never leaves the chip as g_x_hat: the epilogue warps apply the
// transposed bases (Eq. 7) to the accumulator and write g_x directly, while
// the tensor core already works on the next tile (two accumulator slots in
// TMEM, used alternately).
//
// Warp roles: warp 0 TMA producer, warp 1 TMEM owner and tcgen05 issuer,
// warps 2-9 epilogue (two groups of four, alternating 32-column chunks of a
// tile).  All roles walk the same tile list.  Every wait is bounded and an
// expired wait is reported through the status block.
#include <cuda_bf16.h>
#include <cstdio>
#include <cstdlib>

#include "lbp_fused.cuh"
#include "lbp_fused_epilogue.cuh"
#include "lbp_internal.h"
#include "ptx_sm100.cuh"
#include "wht_device.cuh"

namespace lbp {
namespace fused {

constexpr int BK = 64;
constexpr int kStages = 4;
constexpr int kABytes = BM * BK * 2;             // 16 KB
constexpr int kBBytes = 256 * BK * 2;            // 32 KB (up to 256 columns)
constexpr int kStageBytes = kABytes + kBBytes;   // 48 KB
constexpr int kChunkBytes = 64 * BK * 2;         // 8 KB: one 64-wide chunk of an MN-major tile
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
constexpr uint32_t kSlotCols = 256;   // two accumulator slots; tile number t of a CTA uses slot t & 1

// Role timeline (diagnostic builds only): slot 0 kernel start, 2 producer done,
// 3 MMA issuer done, 4 epilogue done, 5 first tile drained.
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
    lbp_products_kernel(const __grid_constant__ CUtensorMap tm_gyhat_k,
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
  uint64_t* acc_full = empty_bar + kStages;   // [2]: accumulator slots
  uint64_t* acc_empty = acc_full + 2;         // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, grid = gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&acc_full[s], 1);
      ptx::mbar_init(&acc_empty[s], 4 * kEGroups);
    }
    ptx::mbar_fence_init();
    *abort_flag = 0;
    ptx::prefetch_tensormap(&tm_gyhat_k);
    ptx::prefetch_tensormap(&tm_gyhat_mn);
    ptx::prefetch_tensormap(&tm_xhat);
    ptx::prefetch_tensormap(&tm_w);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) trace_mark(p, 0);
  // the next kernel on the stream (the projection of the next call) may be
  // scheduled as SMs free up; it waits for this grid before touching memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int my_tiles = unit_tile_count(p, sc, cta, grid);

  // The roles part here, and with them the registers: the first warpgroup gives
  // up what it does not need, the epilogue warpgroups take it (the expansion
  // holds a whole coefficient array per thread).
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsFeed));
  if (warp == 0) {
    // =========================== TMA producer ===========================
    if (ptx::elect_one()) {
      // The kernel is launched with programmatic stream serialization: everything
      // above overlaps the tail of the projection kernel; its results (x_hat,
      // g_y_hat) may only be read after this wait.
      asm volatile("griddepcontrol.wait;" ::: "memory");
      // the operands are read by several CTAs, from L2
      const uint64_t keep = ptx::l2_policy_evict_last();
      uint32_t it = 0;
      bool ok = true;
      for (int ti = 0; ti < my_tiles && ok && !p.test_stall; ++ti) {
        const WorkTile tl = unit_tile(p, sc, cta, grid, ti);
        const int bn = tl.is_gw ? p.BNw : p.BNx;
        const uint32_t tx = static_cast<uint32_t>(kABytes + bn * BK * 2);
        for (int kb = tl.kb0; kb < tl.kb0 + tl.n_kb; ++kb) {
          const int s = static_cast<int>(it % kStages);
          if (!ptx::mbar_wait(&empty_bar[s], ((it / kStages) + 1) & 1u, p.status, (4u << 16) | 1u)) {
            ok = false;
            break;
          }
          uint8_t* sa = smem + s * kStageBytes;
          uint8_t* sb = sa + kABytes;
          ptx::mbar_expect_tx(&full_bar[s], tx);
          if (tl.is_gw) {
            // A = g_y_hat^T tile: stored (rows, Cout), MN-major, two 64-wide chunks
            ptx::tma_load_2d_hint(sa, &tm_gyhat_mn, &full_bar[s], tl.a * 128, kb * BK, keep);
            ptx::tma_load_2d_hint(sa + kChunkBytes, &tm_gyhat_mn, &full_bar[s], tl.a * 128 + 64, kb * BK, keep);
            for (int c = 0; c < bn / 64; ++c)
              ptx::tma_load_2d_hint(sb + c * kChunkBytes, &tm_xhat, &full_bar[s], tl.b * bn + c * 64,
                               kb * BK, keep);
          } else {
            // A = g_y_hat rows of group m, K-major
            ptx::tma_load_2d_hint(sa, &tm_gyhat_k, &full_bar[s], kb * BK, tl.a * BM, keep);
            for (int c = 0; c < bn / 64; ++c)
              ptx::tma_load_2d_hint(sb + c * kChunkBytes, &tm_w, &full_bar[s], tl.b * bn + c * 64, kb * BK, keep);
          }
          ++it;
        }
      }
      if (!ok) *abort_flag = 1;
      trace_mark(p, 2);
    }
  } else if (warp == 1) {
    // =========================== tcgen05 issuer ===========================
    if (ptx::elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      const uint32_t idesc_w = ptx::idesc_bf16(BM, p.BNw, true, true);
      const uint32_t idesc_x = ptx::idesc_bf16(BM, p.BNx, false, true);
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        const WorkTile tl = unit_tile(p, sc, cta, grid, ti);
        const int slot = ti & 1;
        const int n_kb = tl.n_kb;
        const uint32_t d_tmem = tmem_base + slot * kSlotCols;
        const uint32_t idesc = tl.is_gw ? idesc_w : idesc_x;
        const uint32_t uses = static_cast<uint32_t>(ti >> 1);   // earlier uses of this slot
        // the accumulator slot must have been drained by the epilogue
        if (!ptx::mbar_wait(&acc_empty[slot], (uses + 1) & 1u, p.status, (4u << 16) | 4u)) {
          ok = false;
          break;
        }
        for (int kb = 0; kb < n_kb; ++kb) {
          const int s = static_cast<int>(it % kStages);
          if (!ptx::mbar_wait(&full_bar[s], (it / kStages) & 1u, p.status, (4u << 16) | 3u)) {
            ok = false;
            break;
          }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + s * kStageBytes);
          const uint32_t sb = sa + kABytes;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            const uint64_t da = tl.is_gw ? ptx::smem_desc_sw128(sa + kk * 2048, kChunkBytes, 1024)
                                         : ptx::smem_desc_sw128(sa + kk * 32, 16, 1024);
            const uint64_t db = ptx::smem_desc_sw128(sb + kk * 2048, kChunkBytes, 1024);
            ptx::mma_bf16_ss(d_tmem, da, db, idesc, (kb == 0 && kk == 0) ? 0u : 1u);
          }
          ptx::mma_commit(&empty_bar[s]);
          ++it;
        }
        if (!ok) break;
        ptx::mma_commit(&acc_full[slot]);
      }
      if (!ok) *abort_flag = 1;
      trace_mark(p, 3);
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsEpilogue));
    // =========================== epilogue ===========================
    const int eg = (warp - 4) >> 2;          // epilogue group: chunks eg, eg + kEGroups, ...
    const int ew = (warp - 4) & 3;           // warp within the group
    const int quarter = warp & 3;            // TMEM lane quarter this warp may read
    const int etid = ew * 32 + lane;         // 0..127 within the group
    float* const Eg = E + eg * (kEBytes / 4);
    const int bar_id = 1 + eg;
    // row 128 stays zero: unselected coefficients are gathered from there, which
    // keeps the gather free of branches
    if (etid < kEStride) Eg[BM * kEStride + etid] = 0.f;
    named_bar_sync(bar_id, 128);
    for (int ti = 0; ti < my_tiles; ++ti) {
      const WorkTile tl = unit_tile(p, sc, cta, grid, ti);
      const int slot = ti & 1;
      const uint32_t uses = static_cast<uint32_t>(ti >> 1);
      const uint32_t acc_col = slot * kSlotCols;
      const bool ok = ptx::mbar_wait(&acc_full[slot], uses & 1u, p.status, (4u << 16) | 5u);
      // One answer for the whole group: a thread that saw its own wait expire, or
      // the flag another role raised, takes the other 127 threads with it (read
      // one by one after the barrier, the flag could split the group, and the
      // threads left inside the tile would wait on a barrier that never fills).
      if (named_bar_or(bar_id, 128, !ok || *abort_flag != 0)) {
        if (etid == 0) *abort_flag = 1;
        break;
      }
      ptx::tc_fence_after_sync();
      if (etid == 0 && eg == 0) trace_mark(p, 5, true);
      DrainTile dt;
      dt.is_gw = tl.is_gw;
      dt.row_base = tl.a * 128;
      dt.group = tl.a;
      dt.col_base = tl.b * (tl.is_gw ? p.BNw : p.BNx);
      dt.bn = tl.is_gw ? p.BNw : p.BNx;
      dt.slice = tl.slice;
      dt.tmem_acc = tmem_base + acc_col;
      uint64_t* release_bar = &acc_empty[slot];
      drain_tile<K, LB, NEX>(p, fb, dt, Eg, bar_id, eg, etid, quarter, lane,
                        [release_bar]() { ptx::mbar_arrive(release_bar); });
    }
    if (etid == 0) trace_mark(p, 4);   // latest of the groups
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace fused

// --------------------------------------------------------------- launcher ----
static thread_local const FusedOverlap* g_overlap = nullptr;
void set_fused_overlap(const FusedOverlap* ov) { g_overlap = ov; }
const FusedOverlap* fused_overlap() { return g_overlap; }

static thread_local bool g_test_stall = false;
void set_test_stall(bool on) { g_test_stall = on; }
bool test_stall() { return g_test_stall; }
static thread_local bool g_test_stall_projection = false;
void set_test_stall_projection(bool on) { g_test_stall_projection = on; }
bool test_stall_projection() { return g_test_stall_projection; }

bool fused_supported(const lbp_layer& L, const BasisPlan& bp) {
  // the epilogue addresses the tokens of an image with 32-bit element offsets
  const long long block_span = static_cast<long long>(L.H + L.k) * L.W * L.Cin;
  return L.dtype == LBP_BF16 && (L.k == 4 || L.k == 8 || L.k == 16) && bp.r <= fused_max_rank(L.k) && bp.LB <= 8 &&
         bp.LB <= L.k && block_span < (1ll << 31);
}

size_t fused_scratch_bytes(const lbp_layer& L, int r, FusedLayout* lay) {
  const long long nb = static_cast<long long>(L.B) * blocks_along(L.H, L.k) * blocks_along(L.W, L.k);
  // Blocks per 128-row group.  With very few groups (low rank on a small token
  // grid) the expansion of a whole group, (128 / r) * k * k tokens per tile, falls
  // on a handful of CTAs: groups are then filled only partly (rows left zero)
  // until there are about two dozen 256-row tiles per column strip.
  int bpt = 128 / r;
  {
    const long long n_tx = (L.Cin + 127) / 128;
    while (bpt > 1 && ((nb + bpt - 1) / bpt + 1) / 2 * n_tx < 24) bpt = (bpt + 1) / 2;
  }
  const long long G = (nb + bpt - 1) / bpt;
  FusedLayout l;
  size_t off = 0;
  l.x_hat = off;
  off += static_cast<size_t>(G) * 128 * L.Cin * 2;
  off = (off + 1023) / 1024 * 1024;
  l.gy_hat = off;
  off += static_cast<size_t>(G) * 128 * L.Cout * 2;
  off = (off + 1023) / 1024 * 1024;
  // fp32 planes for K slices of g_W: only layers with few GW tiles slice, and
  // slices * tiles stays below the SM count (bounded here for up to 256 SMs)
  l.planes = off;
  {
    const long long tiles_min = ((L.Cout + 127) / 128) * ((L.Cin + 255) / 256);
    long long s_cap = tiles_min >= 96 ? 1 : 192 / tiles_min;
    if (s_cap > 2 * G) s_cap = 2 * G;
    l.planes_bytes = s_cap > 1 ? static_cast<size_t>(s_cap) * L.Cout * L.Cin * 4 : 0;
    const size_t cap = 48u << 20;
    if (l.planes_bytes > cap) l.planes_bytes = cap;
  }
  off += l.planes_bytes;
  off = (off + 1023) / 1024 * 1024;
  l.trace = off;
  off += kFusedTraceBytes;
  l.total = (off + 1023) / 1024 * 1024;
  l.G = static_cast<int>(G);
  l.bpt = bpt;
  if (lay) *lay = l;
  return l.total;
}

// Expansion variant of a basis plan: 0 core butterfly, 1 4 x 4 core plus extra
// bases, 2 8 x 8 core.
static int epilogue_kind(const BasisPlan& bp) {
  int n_outside = 0;
  for (int q = 0; q < bp.r; ++q) n_outside += (bp.seq_i[q] >= 4 || bp.seq_j[q] >= 4) ? 1 : 0;
  if (bp.LB == 8 && n_outside <= kFusedMaxExtra) return 1;
  return bp.LB == 8 ? 2 : 0;
}

double fused_products_model_us(const lbp_layer& L, const BasisPlan& bp, int pairs) {
  FusedLayout lay;
  fused_scratch_bytes(L, bp.r, &lay);
  PlanShape shape{};
  shape.Cin = L.Cin;
  shape.Cout = L.Cout;
  shape.G = lay.G;
  shape.bpt = lay.bpt;
  shape.k = L.k;
  shape.units = pairs;
  shape.pair = 1;
  shape.max_splits = static_cast<int>(lay.planes_bytes / (static_cast<size_t>(L.Cout) * L.Cin * 4));
  shape.epi_kind = epilogue_kind(bp);
  shape.num_kb_w = lay.G * 2;
  shape.num_kb_x = (L.Cout + 63) / 64;
  // measured times sit about a third above the model (the stages of a unit share
  // its path to L2), plus the launch and the first operand tiles
  return 1.35 * plan_products(shape).model_us + 4.0;
}

double fused_projection_model_us(const lbp_layer& L, const BasisPlan& bp, int ctas) {
  const double T = static_cast<double>(L.B) * L.H * L.W;
  const double nb = static_cast<double>(L.B) * blocks_along(L.H, L.k) * blocks_along(L.W, L.k);
  const double bytes = 2.0 * (T + nb * bp.r) * (L.Cin + L.Cout);
  // one SM streams about 70 GB/s through its tile ring; the chip about 5.2 TB/s
  const double rate = ctas * 70e3 < 5.2e6 ? ctas * 70e3 : 5.2e6;   // bytes per microsecond
  return bytes / rate + 5.0;
}

int fused_project(const void* x, const void* x_hat_dense, const void* g_y, const lbp_layer& L,
                  const BasisPlan& bp, const FusedParams& p, uint32_t* status, cudaStream_t stream) {
  const RowMap grouped{p.bpt, fused::BM};
  const FusedOverlap* ov = fused_overlap();
  cudaStream_t ps = ov != nullptr ? ov->proj_stream : stream;
  if (ov != nullptr) set_projection_launch(ProjLaunch{ov->proj_ctas, ov->proj_ctas > 0, false});
  int e = LBP_OK;
  if (x_hat_dense == nullptr) {
    e = launch_project2(g_y, p.gy_hat, L.Cout, x, p.x_hat, L.Cin, LBP_BF16, L.B, L.H, L.W, bp, grouped,
                        status, ps, fused_scale_gy(L.k), fused_scale_x(L.k), &p.vgy, &p.vx);
  } else {
    // x_hat was taken at forward time (Eq. 3), as orthonormal coefficients: it
    // changes its row layout and its power-of-two scale
    e = launch_regroup_rows(x_hat_dense, p.x_hat, p.nb, bp.r, grouped, L.Cin,
                            fused_scale_x(L.k) * static_cast<float>(L.k), ps);
    if (e == LBP_OK)
      e = launch_project(g_y, p.gy_hat, LBP_BF16, L.B, L.H, L.W, L.Cout, bp, grouped, status, ps,
                         fused_scale_gy(L.k), &p.vgy);
  }
  if (ov != nullptr) {
    set_projection_launch(ProjLaunch{0, false, true});
    if (e != LBP_OK) return e;
    LBP_CUDA_TRY(cudaEventRecord(ov->proj_done, ps));
    LBP_CUDA_TRY(cudaStreamWaitEvent(stream, ov->proj_done, 0));
  }
  return e;
}

int launch_fused(const void* x, const void* x_hat_dense, const void* g_y, const void* W, void* g_x,
                 void* g_W, const lbp_layer& L, const BasisPlan& bp, uint8_t* scratch,
                 uint32_t* status, cudaStream_t stream, FusedPhaseHook hook, void* hook_arg,
                 const CallViews* views) {
  using namespace fused;
  FusedLayout lay;
  fused_scratch_bytes(L, bp.r, &lay);
  const int K = L.k;
  int dev = 0, sms = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  FusedParams p{};
  p.Hb = blocks_along(L.H, K);
  p.Wb = blocks_along(L.W, K);
  p.nb = L.B * p.Hb * p.Wb;
  p.H = L.H;
  p.W = L.W;
  p.r = bp.r;
  p.bpt = lay.bpt;
  p.G = lay.G;
  p.Cin = L.Cin;
  p.Cout = L.Cout;
  p.gw_bf16 = L.gw_dtype == LBP_BF16 ? 1 : 0;
  p.x_hat = reinterpret_cast<__nv_bfloat16*>(scratch + lay.x_hat);
  p.gy_hat = reinterpret_cast<__nv_bfloat16*>(scratch + lay.gy_hat);
  p.gw_planes = reinterpret_cast<float*>(scratch + lay.planes);
  p.g_x = static_cast<__nv_bfloat16*>(g_x);
  p.g_W = g_W;
  p.status = status;
  p.vx = resolve_view(views ? &views->x : nullptr, L.H, L.W, L.Cin);
  p.vgy = resolve_view(views ? &views->gy : nullptr, L.H, L.W, L.Cout);
  p.vgx = resolve_view(views ? &views->gx : nullptr, L.H, L.W, L.Cin);
  p.gx_image8 = static_cast<int32_t>(p.vgx.image / 8);
  p.test_stall = test_stall() ? 1 : 0;
  p.num_kb_x = (L.Cout + BK - 1) / BK;
  p.num_kb_w = p.G * (BM / BK);
  FusedBasis fb;
  for (int n = 0; n < 64; ++n) fb.qmap[n] = -1;
  for (int x = 0; x < kFusedMaxExtra; ++x) {
    fb.ex_q[x] = -1;
    fb.ex_mu[x] = fb.ex_mv[x] = 0;
  }
  p.lb_kernel = bp.LB;
  p.n_extra = 0;
  int n_outside = 0;   // bases with an index of 4 or more
  for (int q = 0; q < bp.r; ++q) n_outside += (bp.seq_i[q] >= 4 || bp.seq_j[q] >= 4) ? 1 : 0;
  if (bp.LB == 8 && n_outside <= kFusedMaxExtra) {
    // An 8 x 8 coefficient array that is empty but for a few entries outside its
    // 4 x 4 corner (PREFIX sets of rank 14-16): butterfly on the corner, the few
    // others added token by token.
    p.lb_kernel = 4;
    int x = 0;
    for (int q = 0; q < bp.r; ++q) {
      if (bp.seq_i[q] < 4 && bp.seq_j[q] < 4) {
        fb.qmap[walsh_natural_index(4, bp.seq_i[q]) * 4 + walsh_natural_index(4, bp.seq_j[q])] =
            static_cast<int16_t>(q);
      } else {
        fb.ex_q[x] = static_cast<int16_t>(q);
        for (int t = 0; t < K; ++t) {
          if (__builtin_popcount(static_cast<unsigned>(bp.nat_i[q] & t)) & 1) fb.ex_mu[x] |= static_cast<uint16_t>(1u << t);
          if (__builtin_popcount(static_cast<unsigned>(bp.nat_j[q] & t)) & 1) fb.ex_mv[x] |= static_cast<uint16_t>(1u << t);
        }
        ++x;
      }
    }
    p.n_extra = x;
  } else {
    for (int a = 0; a < bp.LB; ++a)
      for (int b = 0; b < bp.LB; ++b) fb.qmap[a * bp.LB + b] = bp.qmap[a * bp.LB + b];
  }
  if (fused_pair_supported(L, sms))
    return launch_fused_pair(x, x_hat_dense, g_y, W, g_W, L, bp, p, fb, lay, sms, status, stream, hook,
                             hook_arg);

  // column tiles (multiples of one 64-wide TMA chunk, up to 256), K slices of g_W
  // and the tile list of every CTA
  p.mt_w = (L.Cout + 127) / 128;
  const int max_splits_by_ws =
      static_cast<int>(lay.planes_bytes / (static_cast<size_t>(L.Cout) * L.Cin * 4));
  PlanShape shape{};
  shape.Cin = L.Cin;
  shape.Cout = L.Cout;
  shape.G = p.G;
  shape.bpt = p.bpt;
  shape.k = L.k;
  shape.units = sms;
  shape.pair = 0;
  shape.max_splits = max_splits_by_ws;
  shape.epi_kind = p.n_extra > 0 ? 1 : (p.lb_kernel == 8 ? 2 : 0);
  shape.num_kb_w = p.num_kb_w;
  shape.num_kb_x = p.num_kb_x;
  const TilePlan& plan = plan_products(shape);
  p.BNw = plan.BNw;
  p.BNx = plan.BNx;
  p.gw_splits = plan.splits;
  p.kb_per_split_w = plan.kbps;
  p.n_tx = (L.Cin + p.BNx - 1) / p.BNx;
  p.nt_w = (L.Cin + p.BNw - 1) / p.BNw;
  p.n_gx_tiles = p.G * p.n_tx;
  p.n_gw_tiles = p.mt_w * p.nt_w * p.gw_splits;
#ifdef LBP_ROLE_TRACE
  p.trace = reinterpret_cast<unsigned long long*>(scratch + lay.trace);
  LBP_CUDA_TRY(cudaMemsetAsync(p.trace, 0, kFusedTraceBytes, stream));
#endif

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
  const int grid = total_tiles < sms ? total_tiles : sms;

  auto launch = [&](auto kern) -> int {
    LBP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    LBP_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tm_gyhat_k, tm_gyhat_mn, tm_xhat, tm_w, p, fb, plan.sched));
    count_launch();
    LBP_CUDA_TRY(cudaGetLastError());
    if (p.gw_splits > 1)
      return launch_splitk_reduce(p.gw_planes, g_W, static_cast<long long>(L.Cout) * L.Cin,
                                  p.gw_splits, p.gw_bf16 != 0, stream);
    return LBP_OK;
  };
  if (p.n_extra > 0) {
    if (K == 8) return launch(lbp_products_kernel<8, 4, kFusedMaxExtra>);
    if (K == 16) return launch(lbp_products_kernel<16, 4, kFusedMaxExtra>);
    return LBP_ERR_BASIS;
  }
  switch (K * 100 + p.lb_kernel) {
    case 401: return launch(lbp_products_kernel<4, 1>);
    case 402: return launch(lbp_products_kernel<4, 2>);
    case 404: return launch(lbp_products_kernel<4, 4>);
    case 801: return launch(lbp_products_kernel<8, 1>);
    case 802: return launch(lbp_products_kernel<8, 2>);
    case 804: return launch(lbp_products_kernel<8, 4>);
    case 808: return launch(lbp_products_kernel<8, 8>);
    case 1601: return launch(lbp_products_kernel<16, 1>);
    case 1602: return launch(lbp_products_kernel<16, 2>);
    case 1604: return launch(lbp_products_kernel<16, 4>);
    case 1608: return launch(lbp_products_kernel<16, 8>);
  }
  return LBP_ERR_BASIS;
}

}  // namespace lbp
