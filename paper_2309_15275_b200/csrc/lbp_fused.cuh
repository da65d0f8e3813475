// Declarations of the persistent products + expansion kernel (bf16, r <= 16).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "lbp_internal.h"

namespace lbp {

// Highest rank the persistent products kernel takes: a 128-row group must hold
// several blocks, and the tensor-pipe projection must produce that many rows
// per block (orders 8 and 16: up to 48, which covers LP_L1-6, LP_L1-7 and LP_L1-8
// of the paper's tables; order 4: all 16).
inline int fused_max_rank(int k) { return k == 4 ? 16 : 48; }

// Scaling inside the products path.  Eq. 6-7 put 1/k on either side of the
// products; all of it is powers of two, so it can sit anywhere without changing
// a bit of the results.  Here g_y_hat carries 1/k^2 and x_hat none: g_W =
// g_y_hat^T x_hat comes out right, and g_x_hat = g_y_hat W already holds the 1/k
// of the reverse projection, which then only adds, subtracts and rounds.
inline float fused_scale_gy(int k) { return 1.0f / static_cast<float>(k * k); }
inline float fused_scale_x(int) { return 1.0f; }

struct FusedParams {
  // token grid and low-rank row layout: block blk of group g = blk / bpt owns rows
  // g * 128 + (blk % bpt) * r ... + r - 1 of x_hat / g_y_hat; the other rows of a
  // group are zero
  int32_t nb, Hb, Wb, H, W, r, bpt, G;
  int32_t Cin, Cout;
  // products
  int32_t BNx, n_tx, num_kb_x;            // GX: column tile, tiles per row group, k-blocks (Cout / 64)
  int32_t BNw, mt_w, nt_w, num_kb_w;      // GW: 128 x BNw tiles, k-blocks (G * 2)
  int32_t n_gx_tiles, n_gw_tiles;         // n_gw_tiles counts K slices: mt_w * nt_w * gw_splits
  int32_t gw_splits, kb_per_split_w;      // K slices of a GW tile (fp32 planes, reduced afterwards)
  float* gw_planes;                       // [gw_splits][Cout][Cin] when gw_splits > 1
  int32_t gw_bf16;
  int32_t lb_kernel, n_extra;             // epilogue core size and bases added token by token (host dispatch)
  __nv_bfloat16* x_hat;
  __nv_bfloat16* gy_hat;
  __nv_bfloat16* g_x;
  void* g_W;
  uint32_t* status;
  // element strides of x, g_y (read by the projection's tensor maps) and of g_x
  // (the expansion's stores); dense tensors: (H*W*C, W*C, C)
  lbp_view vx, vgy, vgx;
  int32_t gx_image8;   // vgx.image / 8 (a multiple of 8 elements: 16 bytes of bf16)
  // failure-injection hook of the test suite (lbp_test_stall_products): the TMA
  // producers issue no load, so every other role runs into its bounded wait
  int32_t test_stall;
#ifdef LBP_ROLE_TRACE
  unsigned long long* trace;              // role timeline, kTraceSlots slots per CTA (null = off)
#endif
};

// Which unit (a CTA, or a CTA pair) works on which tiles, in which order: planned
// on the host (lbp_fused_plan.cu) and handed to the kernel as a launch
// parameter.  Tile ids: [0, n_gw_tiles) are the GW tiles (id = tile * gw_splits +
// K slice), then the GX tiles (row group (pair), column tile).
constexpr int kSchedMaxItems = 1536;
constexpr int kSchedMaxUnits = 160;
struct FusedSchedule {
  int32_t listed;                        // 0: too many tiles for the table, the units deal them by formula
  uint16_t first[kSchedMaxUnits + 1];    // tiles of unit u: ids[first[u]] .. ids[first[u + 1] - 1]
  uint16_t ids[kSchedMaxItems];
};

// One tile of work as the kernels see it.
struct WorkTile {
  int is_gw;
  int a, b;        // GW: (row tile i, column tile j) ; GX: (row group (pair) m, column tile n)
  int kb0, n_kb;   // k-block range (a K slice for GW)
  int slice;
};

#ifdef __CUDACC__
__device__ __forceinline__ int unit_tile_count(const FusedParams& p, const FusedSchedule& sc, int unit,
                                               int units);
__device__ __forceinline__ WorkTile unit_tile(const FusedParams& p, const FusedSchedule& sc, int unit,
                                              int units, int nth);
#endif

constexpr int kFusedMaxExtra = 2;

struct FusedBasis {
  int16_t qmap[64];   // natural-order LB x LB position -> basis slot, -1 unused
  // Bases outside the LB x LB core (kernels instantiated with extras only): the
  // epilogue adds them token by token.  ex_q: slot, -1 = none; bit u of ex_mu /
  // bit v of ex_mv is set where the Walsh row along H / W is -1.
  int16_t ex_q[kFusedMaxExtra];
  uint16_t ex_mu[kFusedMaxExtra];
  uint16_t ex_mv[kFusedMaxExtra];
};

// Builds with -DLBP_ROLE_TRACE carry a per-CTA role timeline (diagnostics) in
// the last bytes of the scratch region; ordinary builds have neither the code
// nor the bytes.
#ifdef LBP_ROLE_TRACE
constexpr int kTraceSlots = 128;   // 8-byte slots per CTA: 8 for the roles, then 8 per tile
constexpr size_t kFusedTraceBytes = 256 * kTraceSlots * 8;
#else
constexpr size_t kFusedTraceBytes = 0;
#endif

struct FusedLayout {
  size_t x_hat, gy_hat, planes, planes_bytes, trace, total;
  int G, bpt;
};

// Side-stream mode of one call (set per thread by lbp_backward_batch): the
// projection goes to `proj_stream` on at most `proj_ctas` CTAs (0 = all SMs),
// `proj_done` is recorded behind it and the products kernel, on `prod_units`
// CTA pairs (0 = all), waits for it on the call's own stream.
struct FusedOverlap {
  cudaStream_t proj_stream;
  cudaEvent_t proj_done;
  int proj_ctas;
  int prod_units;
};
void set_fused_overlap(const FusedOverlap* ov);   // nullptr = off
const FusedOverlap* fused_overlap();

// Per-thread switch set by lbp_test_stall_products (test hook).
void set_test_stall(bool on);
bool test_stall();
void set_test_stall_projection(bool on);
bool test_stall_projection();

#ifdef __CUDACC__
// Without a table the tiles are dealt in a snake over the units (first pass
// forwards, second backwards, ...), in id order.
__device__ __forceinline__ int unit_tile_count(const FusedParams& p, const FusedSchedule& sc, int unit,
                                               int units) {
  if (sc.listed) return static_cast<int>(sc.first[unit + 1]) - static_cast<int>(sc.first[unit]);
  const int total = p.n_gw_tiles + p.n_gx_tiles;
  int n = 0;
  for (int round = 0; round * units < total; ++round) {
    const int pos = (round & 1) ? (units - 1 - unit) : unit;
    if (round * units + pos < total) ++n;
  }
  return n;
}
__device__ __forceinline__ WorkTile unit_tile(const FusedParams& p, const FusedSchedule& sc, int unit,
                                              int units, int nth) {
  int id = 0;
  if (sc.listed) {
    id = sc.ids[sc.first[unit] + nth];
  } else {
    const int total = p.n_gw_tiles + p.n_gx_tiles;
    int seen = 0;
    for (int round = 0; round * units < total; ++round) {
      const int pos = (round & 1) ? (units - 1 - unit) : unit;
      const int t = round * units + pos;
      if (t < total) {
        if (seen == nth) {
          id = t;
          break;
        }
        ++seen;
      }
    }
  }
  WorkTile tl;
  if (id < p.n_gw_tiles) {
    tl.is_gw = 1;
    const int t = id / p.gw_splits;
    tl.slice = id - t * p.gw_splits;
    tl.a = t / p.nt_w;
    tl.b = t - tl.a * p.nt_w;
    tl.kb0 = tl.slice * p.kb_per_split_w;
    const int end = tl.kb0 + p.kb_per_split_w;
    tl.n_kb = (end < p.num_kb_w ? end : p.num_kb_w) - tl.kb0;
  } else {
    id -= p.n_gw_tiles;
    tl.is_gw = 0;
    tl.slice = 0;
    tl.a = id / p.n_tx;
    tl.b = id - tl.a * p.n_tx;
    tl.kb0 = 0;
    tl.n_kb = p.num_kb_x;
  }
  return tl;
}
#endif

// ---- host-side tile plan (lbp_fused_plan.cu) ----
struct PlanShape {
  int Cin, Cout;
  int G;            // 128-row groups of low-rank rows
  int bpt, k;       // blocks per group, transform order (size of a group's expansion)
  int units;        // CTAs, or CTA pairs
  int pair;         // 1: a unit is a CTA pair working on 256-row tiles
  int max_splits;   // K slices of g_W the scratch has planes for
  int epi_kind;     // expansion variant: 0 core butterfly, 1 core + extra bases, 2 8 x 8 core
  int num_kb_w, num_kb_x;
};
struct TilePlan {
  int BNw, BNx, splits, kbps;
  double model_us;   // time of the products kernel under the planner's cost model
  FusedSchedule sched;
};
// Column tiles, K slices of g_W and the per-unit tile lists for this shape
// (remembered per calling thread for recent shapes).
const TilePlan& plan_products(const PlanShape& s);

// Called between the projection launch and the products launch (phase events).
using FusedPhaseHook = int (*)(void* arg, cudaStream_t stream);

bool fused_supported(const lbp_layer& L, const BasisPlan& bp);
size_t fused_scratch_bytes(const lbp_layer& L, int r, FusedLayout* lay);
// Strides of the three token tensors of a call (an entry that is all zero: dense).
struct CallViews {
  lbp_view x, gy, gx;
};
// Exactly one of x / x_hat_dense is given; x_hat_dense are coefficients p(x)
// taken earlier, stored densely (blocks * r, Cin).  views: null = all dense.
int launch_fused(const void* x, const void* x_hat_dense, const void* g_y, const void* W, void* g_x,
                 void* g_W, const lbp_layer& L, const BasisPlan& bp, uint8_t* scratch,
                 uint32_t* status, cudaStream_t stream, FusedPhaseHook hook, void* hook_arg,
                 const CallViews* views = nullptr);
// Algorithm 1, steps 1-2 for the products kernel: g_y_hat (and x_hat, from x or
// from dense coefficients) with rows padded to 128-row groups.
int fused_project(const void* x, const void* x_hat_dense, const void* g_y, const lbp_layer& L,
                  const BasisPlan& bp, const FusedParams& p, uint32_t* status, cudaStream_t stream);

// Modelled time (microseconds) of the products kernel of this layer on `pairs`
// CTA pairs, and of its projection kernel on `ctas` SMs (both from B200
// measurements); lbp_backward_batch balances the two when it runs the
// projection of one layer beside the products kernel of another.
double fused_products_model_us(const lbp_layer& L, const BasisPlan& bp, int pairs);
double fused_projection_model_us(const lbp_layer& L, const BasisPlan& bp, int ctas);

// CTA-pair variant (tcgen05 cta_group::2): used when Cin >= 128 and the SM count is even.
bool fused_pair_supported(const lbp_layer& L, int sms);
int launch_fused_pair(const void* x, const void* x_hat_dense, const void* g_y, const void* W,
                      void* g_W, const lbp_layer& L,
                      const BasisPlan& bp, FusedParams p, const FusedBasis& fb,
                      const FusedLayout& lay, int sms, uint32_t* status, cudaStream_t stream,
                      FusedPhaseHook hook, void* hook_arg);

}  // namespace lbp
