// Host-side tile plan of the persistent products kernels: column tile widths of
// the two products, K slices of g_W, and which unit (CTA or CTA pair) takes
// which tiles in which order.
//
// A unit is a two-stage pipeline: its tensor-core stage works through the
// unit's tiles one after the other, its epilogue warps drain them in the same
// order, and two accumulator slots let tile i + 1 be multiplied while tile i is
// drained (tile i + 2 has to wait for tile i's slot).  The stages cost very
// different amounts per tile kind:
//   GX tile (g_x_hat = g_y_hat W, expanded by Eq. 7 in the epilogue): short
//           product (K = Cout), long epilogue (writes k*k / r times its size);
//   GW tile (g_W = g_y_hat^T x_hat): long product (K = all low-rank rows), short
//           epilogue.
// So a unit takes its GX tiles first and its GW tiles (or K slices of them)
// after: the GW products run under the GX epilogues, and the last thing a unit
// does is a short epilogue.  Tiles are handed out greedily, each to the unit
// that would finish it first under the cost model below (measured on B200).
#include <cstdio>
#include <vector>

#include "lbp_fused.cuh"
#include "lbp_internal.h"

namespace lbp {

namespace {

// ---- cost model (microseconds) ----
// Operand delivery from L2 bounds the products: about 110 GB/s per SM.
constexpr double kFeedBytesPerUs = 110e3;
constexpr double kTileFixedUs = 0.3;
// The expansion writes g_x at about 34 GB/s per SM (core butterfly); the forms
// with extra bases or an 8 x 8 core are slower per byte.
constexpr double kExpandBytesPerUs[3] = {34e3, 21e3, 12e3};
constexpr double kGwStoreBytesPerUs = 30e3;
// K slices of g_W go through fp32 planes and one more kernel.
constexpr double kReduceFixedUs = 3.0;
constexpr double kReduceBytesPerUs = 4e6;

struct Costs {
  double mma_w, epi_w, mma_x, epi_x;
};

Costs tile_costs(const PlanShape& s, int bnw, int bnx, int kbps) {
  const double a_bytes = 128.0 * 64 * 2;                       // a CTA's 128 rows of A per k-block
  const double bw = (s.pair ? bnw / 2 : bnw) * 64.0 * 2;       // its share of B
  const double bx = (s.pair ? bnx / 2 : bnx) * 64.0 * 2;
  Costs c;
  c.mma_w = kTileFixedUs + kbps * (a_bytes + bw) / kFeedBytesPerUs;
  c.mma_x = kTileFixedUs + s.num_kb_x * (a_bytes + bx) / kFeedBytesPerUs;
  c.epi_w = kTileFixedUs + 128.0 * bnw * 4 / kGwStoreBytesPerUs;
  c.epi_x = 0.5 + static_cast<double>(s.bpt) * s.k * s.k * bnx * 2 / kExpandBytesPerUs[s.epi_kind];
  return c;
}

// State of one unit while tiles are handed out.
struct Unit {
  double mma_free = 0, epi_free = 0;
  double slot_free[2] = {0, 0};   // when the epilogue has read the accumulator slot
  int n = 0;
  double finish_if(double mma, double epi) const {
    const double start = mma_free > slot_free[n & 1] ? mma_free : slot_free[n & 1];
    const double mend = start + mma;
    return (mend > epi_free ? mend : epi_free) + epi;
  }
  void take(double mma, double epi) {
    const double start = mma_free > slot_free[n & 1] ? mma_free : slot_free[n & 1];
    mma_free = start + mma;
    const double estart = mma_free > epi_free ? mma_free : epi_free;
    epi_free = estart + epi;
    slot_free[n & 1] = epi_free;   // the slot is read until (nearly) the end of the epilogue
    ++n;
  }
};

// Hands out n_gx GX tiles, then n_gw GW tiles; returns the time the last unit
// finishes.  `owner` (optional) receives the unit of every tile, GX ids first.
double simulate(int units, int n_gx, int n_gw, const Costs& c, std::vector<int>* owner) {
  std::vector<Unit> u(units);
  if (owner) owner->assign(n_gx + n_gw, 0);
  auto place = [&](int idx, double mma, double epi) {
    int best = 0;
    double best_t = u[0].finish_if(mma, epi);
    for (int i = 1; i < units; ++i) {
      const double t = u[i].finish_if(mma, epi);
      if (t < best_t - 1e-9) {
        best_t = t;
        best = i;
      }
    }
    u[best].take(mma, epi);
    if (owner) (*owner)[idx] = best;
  };
  for (int i = 0; i < n_gx; ++i) place(i, c.mma_x, c.epi_x);
  for (int i = 0; i < n_gw; ++i) place(n_gx + i, c.mma_w, c.epi_w);
  double last = 0;
  for (const Unit& x : u) last = x.epi_free > last ? x.epi_free : last;
  return last;
}

bool same_shape(const PlanShape& a, const PlanShape& b) {
  return a.Cin == b.Cin && a.Cout == b.Cout && a.G == b.G && a.bpt == b.bpt && a.k == b.k &&
         a.units == b.units && a.pair == b.pair && a.max_splits == b.max_splits &&
         a.epi_kind == b.epi_kind && a.num_kb_w == b.num_kb_w && a.num_kb_x == b.num_kb_x;
}

struct Cached {
  PlanShape shape;
  TilePlan plan;
};

}  // namespace

const TilePlan& plan_products(const PlanShape& s) {
  static thread_local std::vector<Cached> cache;
  static thread_local size_t next = 0;
  for (const Cached& c : cache)
    if (same_shape(c.shape, s)) return c.plan;

  const int row_tile = s.pair ? 256 : 128;
  const int mt_w = (s.Cout + row_tile - 1) / row_tile;
  const int gx_rows = s.pair ? (s.G + 1) / 2 : s.G;
  const int bn_step = s.pair ? 128 : 64;
  const int cin_pad = (s.Cin + bn_step - 1) / bn_step * bn_step;
  static const int kSplitChoices[] = {1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64, 96, 128, 192};

  TilePlan best{};
  double best_t = -1.0;
  const TuneOptions& tune = tune_options();
  for (int bnw = bn_step; bnw <= 256; bnw += bn_step) {
    for (int bnx = bn_step; bnx <= 256; bnx += bn_step) {
      if (bnw > cin_pad || bnx > cin_pad) continue;
      for (int want : kSplitChoices) {
        if (want > 1 && (want > s.max_splits || want > s.num_kb_w / 4)) continue;
        if (tune.has_tiles &&
            (bnw != tune.tiles_bnw || bnx != tune.tiles_bnx || want != tune.tiles_splits))
          continue;
        const int kbps = (s.num_kb_w + want - 1) / want;
        const int splits = (s.num_kb_w + kbps - 1) / kbps;
        const int nt_w = (s.Cin + bnw - 1) / bnw, n_tx = (s.Cin + bnx - 1) / bnx;
        const int n_gw = mt_w * nt_w * splits, n_gx = gx_rows * n_tx;
        const Costs c = tile_costs(s, bnw, bnx, kbps);
        const int units = n_gw + n_gx < s.units ? n_gw + n_gx : s.units;
        double t = simulate(units, n_gx, n_gw, c, nullptr);
        if (splits > 1)
          t += kReduceFixedUs + (splits + 1.0) * s.Cout * static_cast<double>(s.Cin) * 4 / kReduceBytesPerUs;
        if (best_t < 0 || t < best_t - 1e-9) {
          best_t = t;
          best.BNw = bnw;
          best.BNx = bnx;
          best.splits = splits;
          best.kbps = kbps;
        }
      }
    }
  }
  best.model_us = best_t;
  if (best_t < 0) {   // an override that fits nothing: the widest tiles, no slices
    best.BNw = best.BNx = cin_pad < 256 ? cin_pad : 256;
    best.splits = 1;
    best.kbps = s.num_kb_w;
  }

  // per-unit tile lists of the chosen plan
  const int nt_w = (s.Cin + best.BNw - 1) / best.BNw, n_tx = (s.Cin + best.BNx - 1) / best.BNx;
  const int n_gw = mt_w * nt_w * best.splits, n_gx = gx_rows * n_tx;
  const int units = n_gw + n_gx < s.units ? n_gw + n_gx : s.units;
  FusedSchedule& sc = best.sched;
  sc.listed = 0;
  if (n_gw + n_gx <= kSchedMaxItems && units <= kSchedMaxUnits) {
    std::vector<int> owner;
    simulate(units, n_gx, n_gw, tile_costs(s, best.BNw, best.BNx, best.kbps), &owner);
    std::vector<std::vector<uint16_t>> lists(units);
    // tile ids as the kernels number them: the GW tiles come first
    for (int i = 0; i < n_gx; ++i) lists[owner[i]].push_back(static_cast<uint16_t>(n_gw + i));
    for (int i = 0; i < n_gw; ++i) lists[owner[n_gx + i]].push_back(static_cast<uint16_t>(i));
    int at = 0;
    for (int uidx = 0; uidx < units; ++uidx) {
      sc.first[uidx] = static_cast<uint16_t>(at);
      for (uint16_t id : lists[uidx]) sc.ids[at++] = id;
    }
    for (int uidx = units; uidx <= kSchedMaxUnits; ++uidx) sc.first[uidx] = static_cast<uint16_t>(at);
    sc.listed = 1;
  }
  if (tune.verbose)
    fprintf(stderr, "lbp products plan (%s): G=%d BNw=%d BNx=%d gw_splits=%d kb/split=%d tiles=%d+%d "
                    "units=%d listed=%d model=%.1f us\n",
            s.pair ? "CTA pairs" : "CTAs", s.G, best.BNw, best.BNx, best.splits, best.kbps, n_gx, n_gw,
            units, sc.listed, best_t);

  if (cache.capacity() < 128) cache.reserve(128);
  if (cache.size() < 128) {
    cache.push_back(Cached{s, best});
    return cache.back().plan;
  }
  cache[next] = Cached{s, best};
  const TilePlan& out = cache[next].plan;
  next = (next + 1) % cache.size();
  return out;
}

}  // namespace lbp
