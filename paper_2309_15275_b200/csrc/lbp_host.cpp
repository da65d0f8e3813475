// Host-only part of liblbp: basis tables (Sec. 3.2, Eq. 8-9), the +-1 basis
// matrix of Eq. 6, the cost model of Table 1, status strings, and the basis
// plan the transform kernels consume.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <cmath>
#include <vector>

#include "lbp_internal.h"

namespace lbp {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int>(e); }
void note_cuda_failure(cudaError_t e, const char* file, int line) {
  const char* v = std::getenv("LBP_VERBOSE_ERRORS");
  if (v != nullptr && v[0] == '1')
    std::fprintf(stderr, "lbp: CUDA error %d at %s:%d\n", static_cast<int>(e), file, line);
}

thread_local bool g_defer_wait = false;
void set_projection_defer_wait(bool on) { g_defer_wait = on; }
bool projection_defer_wait() { return g_defer_wait; }
thread_local ProjLaunch g_proj_launch = {0, false, true};
void set_projection_launch(ProjLaunch shape) { g_proj_launch = shape; }
ProjLaunch projection_launch() { return g_proj_launch; }

thread_local long long g_launches = 0;
void count_launch(int n) { g_launches += n; }

int check_order(int k) { return (k == 4 || k == 8 || k == 16) ? LBP_OK : LBP_ERR_BLOCK; }

static int log2_int(int n) {
  int b = 0;
  while ((1 << b) < n) ++b;
  return b;
}

// The Walsh row with s sign changes is the Sylvester-Hadamard row whose index
// is the bit reversal of the Gray code of s.
int walsh_natural_index(int n, int s) {
  const int bits = log2_int(n);
  const int gray = s ^ (s >> 1);
  int rev = 0;
  for (int b = 0; b < bits; ++b)
    if (gray & (1 << b)) rev |= 1 << (bits - 1 - b);
  return rev;
}

int walsh_sign(int k, int s, int u) {
  const int row = walsh_natural_index(k, s);
  return (__builtin_popcount(static_cast<unsigned>(row & u)) & 1) ? -1 : 1;
}

static int validate_set(int k, const lbp_basis* set, int r) {
  if (int e = check_order(k)) return e;
  if (set == nullptr) return LBP_ERR_NULL;
  if (r < 1 || r > k * k) return LBP_ERR_BASIS;
  bool seen[kMaxRank];
  std::memset(seen, 0, sizeof(seen));
  for (int q = 0; q < r; ++q) {
    const int i = set[q].i, j = set[q].j;
    if (i < 0 || i >= k || j < 0 || j >= k) return LBP_ERR_BASIS;
    if (seen[i * k + j]) return LBP_ERR_BASIS;
    seen[i * k + j] = true;
  }
  return LBP_OK;
}

int make_basis_plan(int k, const lbp_basis* set, int r, BasisPlan* plan) {
  if (int e = validate_set(k, set, r)) return e;
  int top = 0;
  for (int q = 0; q < r; ++q) top = std::max(top, std::max(set[q].i, set[q].j));
  int LB = 1;
  while (LB <= top) LB <<= 1;
  plan->k = k;
  plan->r = r;
  plan->LB = LB;
  for (int n = 0; n < kMaxRank; ++n) plan->qmap[n] = -1;
  for (int q = 0; q < r; ++q) {
    // pooled to LB values, the order-k Walsh row of sequency s < LB is the
    // order-LB Walsh row of the same sequency
    const int a = walsh_natural_index(LB, set[q].i);
    const int b = walsh_natural_index(LB, set[q].j);
    plan->qmap[a * LB + b] = static_cast<int16_t>(q);
    plan->nat_i[q] = static_cast<uint8_t>(walsh_natural_index(k, set[q].i));
    plan->nat_j[q] = static_cast<uint8_t>(walsh_natural_index(k, set[q].j));
    plan->seq_i[q] = static_cast<uint8_t>(set[q].i);
    plan->seq_j[q] = static_cast<uint8_t>(set[q].j);
  }
  return LBP_OK;
}

struct PairKey {
  int i, j;
};

static bool prefix_less(const PairKey& a, const PairKey& b) {
  const int sa = a.i + a.j, sb = b.i + b.j;
  if (sa != sb) return sa < sb;
  const int ma = std::max(a.i, a.j), mb = std::max(b.i, b.j);
  if (ma != mb) return ma < mb;
  return a.i < b.i;
}

}  // namespace lbp

using namespace lbp;

namespace lbp {
static TuneOptions g_tune;
static bool g_tune_loaded = false;
void reload_tune_options() {
  TuneOptions t{};
  const char* e = std::getenv("LBP_FUSED");
  t.fused = !(e != nullptr && e[0] == '0');
  e = std::getenv("LBP_PAIR");
  t.pair = !(e != nullptr && e[0] == '0');
  e = std::getenv("LBP_PROJECT_UMMA");
  t.umma = !(e != nullptr && e[0] == '0');
  e = std::getenv("LBP_FUSED_VERBOSE");
  t.verbose = e != nullptr && e[0] == '1';
  e = std::getenv("LBP_FUSED_TILES");
  t.has_tiles = e != nullptr &&
                std::sscanf(e, "%d,%d,%d", &t.tiles_bnw, &t.tiles_bnx, &t.tiles_splits) == 3;
  e = std::getenv("LBP_BATCH_PROJ_SMS");
  t.batch_proj_sms = e != nullptr ? std::atoi(e) : -1;
  g_tune = t;
  g_tune_loaded = true;
}
const TuneOptions& tune_options() {
  if (!g_tune_loaded) reload_tune_options();
  return g_tune;
}
}  // namespace lbp

extern "C" {

int lbp_select_bases(int k, int rule, int param, lbp_basis* out, int cap, int* r_out) {
  if (int e = check_order(k)) return e;
  if (r_out == nullptr) return LBP_ERR_NULL;
  std::vector<PairKey> all;
  for (int i = 0; i < k; ++i)
    for (int j = 0; j < k; ++j) all.push_back({i, j});
  std::sort(all.begin(), all.end(), prefix_less);
  std::vector<PairKey> sel;
  switch (rule) {
    case LBP_SEL_L1:
      if (param < 1 || param > 2 * k - 1) return LBP_ERR_BASIS;
      for (const auto& p : all)
        if (p.i + p.j <= param - 1) sel.push_back(p);
      break;
    case LBP_SEL_LINF:
      if (param < 1 || param > k) return LBP_ERR_BASIS;
      for (const auto& p : all)
        if (std::max(p.i, p.j) <= param - 1) sel.push_back(p);
      break;
    case LBP_SEL_PREFIX:
      if (param < 1 || param > k * k) return LBP_ERR_BASIS;
      sel.assign(all.begin(), all.begin() + param);
      break;
    default:
      return LBP_ERR_BASIS;
  }
  *r_out = static_cast<int>(sel.size());
  if (out == nullptr) return LBP_ERR_NULL;
  if (cap < static_cast<int>(sel.size())) return LBP_ERR_CAPACITY;
  for (size_t q = 0; q < sel.size(); ++q) {
    out[q].i = sel[q].i;
    out[q].j = sel[q].j;
  }
  return LBP_OK;
}

int lbp_select_lhe(const double* energy, int k, int r, lbp_basis* out) {
  if (int e = check_order(k)) return e;
  if (energy == nullptr || out == nullptr) return LBP_ERR_NULL;
  if (r < 1 || r > k * k) return LBP_ERR_BASIS;
  for (int n = 0; n < k * k; ++n)
    if (!(energy[n] >= 0.0) || !std::isfinite(energy[n])) return LBP_ERR_BASIS;
  std::vector<PairKey> all;
  for (int i = 0; i < k; ++i)
    for (int j = 0; j < k; ++j) all.push_back({i, j});
  // strongest first; equal energies in the PREFIX order
  std::sort(all.begin(), all.end(), [&](const PairKey& a, const PairKey& b) {
    const double ea = energy[a.i * k + a.j], eb = energy[b.i * k + b.j];
    if (ea != eb) return ea > eb;
    return prefix_less(a, b);
  });
  for (int q = 0; q < r; ++q) {
    out[q].i = all[q].i;
    out[q].j = all[q].j;
  }
  return LBP_OK;
}

int lbp_basis_matrix(int k, const lbp_basis* set, int r, int8_t* P_out) {
  if (P_out == nullptr) return LBP_ERR_NULL;
  BasisPlan plan;
  if (int e = make_basis_plan(k, set, r, &plan)) return e;
  for (int u = 0; u < k; ++u)
    for (int v = 0; v < k; ++v)
      for (int q = 0; q < r; ++q)
        P_out[(u * k + v) * r + q] =
            static_cast<int8_t>(walsh_sign(k, set[q].i, u) * walsh_sign(k, set[q].j, v));
  return LBP_OK;
}

double lbp_flops(int Cin, int Cout, long long L, int r, int which) {
  const double cx = Cin, cy = Cout, l = static_cast<double>(L), rr = r;
  const double proj = (cx + cy) * l * rr, mm = 4.0 * cx * cy * rr, rev = cx * l * rr;
  switch (which) {
    case 0: return 4.0 * cx * cy * l;
    case 1: return proj;
    case 2: return mm;
    case 3: return rev;
    case 4: return proj + mm + rev;
    default: return -1.0;
  }
}

const char* lbp_status_string(int status) {
  switch (status) {
    case LBP_OK: return "ok";
    case LBP_ERR_NULL: return "null pointer";
    case LBP_ERR_SHAPE: return "bad shape (dimension <= 0 or grid not divisible by k)";
    case LBP_ERR_BLOCK: return "block size k must be 4, 8 or 16";
    case LBP_ERR_BASIS: return "bad basis list (rank, index range or duplicate)";
    case LBP_ERR_DTYPE: return "unsupported dtype";
    case LBP_ERR_ALIGN: return "pointer or channel extent not 16-byte aligned";
    case LBP_ERR_WORKSPACE: return "workspace missing or too small";
    case LBP_ERR_ARCH: return "device is not sm_100";
    case LBP_ERR_CUDA: return "CUDA call failed";
    case LBP_ERR_TIMEOUT: return "bounded device wait expired";
    case LBP_ERR_CAPACITY: return "output array too small";
    case LBP_ERR_OVERLAP: return "buffers of different problems of a batch overlap";
    default: return "unknown status";
  }
}

int lbp_last_cuda_error(void) { return g_last_cuda_error; }

long long lbp_launch_count(void) { return lbp::g_launches; }

size_t lbp_status_bytes(void) { return kStatusBytes; }

}  // extern "C"
