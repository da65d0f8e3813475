// Declarations of the persistent products + expansion kernel (bf16, r <= 16).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "lbp_internal.h"

namespace lbp {

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
  float scale;                            // 1/k
  __nv_bfloat16* x_hat;
  __nv_bfloat16* gy_hat;
  __nv_bfloat16* g_x;
  void* g_W;
  uint32_t* status;
  // failure-injection hook of the test suite (lbp_test_stall_products): the TMA
  // producers issue no load, so every other role runs into its bounded wait
  int32_t test_stall;
#ifdef LBP_ROLE_TRACE
  unsigned long long* trace;              // role timeline, 8 slots per CTA (null = off)
#endif
};

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
constexpr size_t kFusedTraceBytes = 256 * 8 * 8;
#else
constexpr size_t kFusedTraceBytes = 0;
#endif

struct FusedLayout {
  size_t x_hat, gy_hat, planes, planes_bytes, trace, total;
  int G, bpt;
};

// Per-thread switch set by lbp_test_stall_products (test hook).
void set_test_stall(bool on);
bool test_stall();

// Called between the projection launch and the products launch (phase events).
using FusedPhaseHook = int (*)(void* arg, cudaStream_t stream);

bool fused_supported(const lbp_layer& L, const BasisPlan& bp);
size_t fused_scratch_bytes(const lbp_layer& L, int r, FusedLayout* lay);
int launch_fused(const void* x, const void* g_y, const void* W, void* g_x, void* g_W,
                 const lbp_layer& L, const BasisPlan& bp, uint8_t* scratch, uint32_t* status,
                 cudaStream_t stream, FusedPhaseHook hook, void* hook_arg);

// CTA-pair variant (tcgen05 cta_group::2): used when Cin >= 128 and the SM count is even.
bool fused_pair_supported(const lbp_layer& L, int sms);
int launch_fused_pair(const void* x, const void* g_y, const void* W, void* g_W, const lbp_layer& L,
                      const BasisPlan& bp, FusedParams p, const FusedBasis& fb,
                      const FusedLayout& lay, int sms, uint32_t* status, cudaStream_t stream,
                      FusedPhaseHook hook, void* hook_arg);

}  // namespace lbp
