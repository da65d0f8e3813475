// C-ABI entry points that touch the device: argument validation, workspace
// layout, TMA descriptor encoding and the launch sequence of Algorithm 1.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "lbp_fused.cuh"
#include "lbp_internal.h"
#include "lbp_test_hooks.h"

namespace lbp {

// ---------------------------------------------------------------- helpers ----
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static int elem_size(int dtype) { return dtype == LBP_BF16 ? 2 : 4; }
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_device_arch() {
  int dev = 0, major = 0;
  // Every device entry point passes through here before it launches anything.
  // A non-sticky error left behind on this thread by other code in the process
  // (cudaGetLastError() not yet called on it) would otherwise be reported by
  // the launch checks below as this library's own.
  (void)cudaGetLastError();
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  // Tensor maps are encoded through the driver API, which needs the device's
  // primary context current on the calling thread.  A thread that has made no
  // runtime call yet (a framework's worker thread) has none: selecting the
  // device it already has binds it, and changes nothing else.
  LBP_CUDA_TRY(cudaSetDevice(dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  return major == 10 ? LBP_OK : LBP_ERR_ARCH;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is resolved at run time so that the library loads
// (for its host-only functions) on machines without a CUDA driver.
static int get_encode_fn(EncodeTiledFn* out) {
  static EncodeTiledFn cached = nullptr;
  if (cached == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    LBP_CUDA_TRY(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000,
                                                  cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) {
      set_last_cuda_error(cudaErrorNotSupported);
      return LBP_ERR_CUDA;
    }
    cached = reinterpret_cast<EncodeTiledFn>(fn);
  }
  *out = cached;
  return LBP_OK;
}

int encode_block_tensor_map(CUtensorMap* map, const void* base, int dtype, int B, int H, int W,
                            int C, int k, int box_c, bool swizzle128, const lbp_view* view) {
  return encode_box_tensor_map(map, base, dtype, B, H, W, C, box_c, k, k, swizzle128, view);
}

int encode_box_tensor_map(CUtensorMap* map, const void* base, int dtype, int B, int H, int W, int C,
                          int box_c, int box_w, int box_h, bool swizzle128, const lbp_view* view) {
  EncodeTiledFn enc;
  if (int e = get_encode_fn(&enc)) return e;
  const cuuint64_t es = static_cast<cuuint64_t>(elem_size(dtype));
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W),
                              static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(B)};
  const lbp_view v = resolve_view(view, H, W, C);
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(v.token) * es,
                                 static_cast<cuuint64_t>(v.row) * es,
                                 static_cast<cuuint64_t>(v.image) * es};
  const cuuint32_t box[4] = {static_cast<cuuint32_t>(box_c), static_cast<cuuint32_t>(box_w),
                             static_cast<cuuint32_t>(box_h), 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r =
      enc(map, dtype == LBP_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
          4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
          // a box row is 128 bytes; fetching 256 measured 4-5 % slower on the projection
          CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    // CUresult and cudaError_t share their numbering
    set_last_cuda_error(static_cast<cudaError_t>(r));
    note_cuda_failure(static_cast<cudaError_t>(r), __FILE__, __LINE__);
    return LBP_ERR_CUDA;
  }
  return LBP_OK;
}

int encode_matrix_tensor_map(CUtensorMap* map, const void* base, long long rows, long long cols,
                             int box_rows) {
  EncodeTiledFn enc;
  if (int e = get_encode_fn(&enc)) return e;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
  const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    // CUresult and cudaError_t share their numbering
    set_last_cuda_error(static_cast<cudaError_t>(r));
    note_cuda_failure(static_cast<cudaError_t>(r), __FILE__, __LINE__);
    return LBP_ERR_CUDA;
  }
  return LBP_OK;
}

static int check_grid(int B, int H, int W, int C, int k, int dtype) {
  if (int e = check_order(k)) return e;
  if (dtype != LBP_F32 && dtype != LBP_BF16) return LBP_ERR_DTYPE;
  if (B <= 0 || H <= 0 || W <= 0 || C <= 0) return LBP_ERR_SHAPE;
  if ((static_cast<long long>(C) * elem_size(dtype)) % 16 != 0) return LBP_ERR_ALIGN;
  return LBP_OK;
}

static int check_layer(const lbp_layer* L) {
  if (L == nullptr) return LBP_ERR_NULL;
  if (int e = check_grid(L->B, L->H, L->W, L->Cin, L->k, L->dtype)) return e;
  if (int e = check_grid(L->B, L->H, L->W, L->Cout, L->k, L->dtype)) return e;
  if (L->gw_dtype != LBP_F32 && L->gw_dtype != LBP_BF16) return LBP_ERR_DTYPE;
  if (L->dtype == LBP_F32 && L->gw_dtype != LBP_F32) return LBP_ERR_DTYPE;
  return LBP_OK;
}

// Workspace layout of lbp_backward at rank r < k*k.
struct Layout {
  size_t x_hat, gy_hat, gx_hat, splitk, splitk_bytes, fused, total;
  long long rows;   // M_hat = blocks * r
};

// Scratch of lbp_backward_ex beyond `Layout::total`: two fp32 (Cout, Cin)
// matrices (this call's g_W before it is added to the caller's, the term of the
// tokens outside the grid) and the fp64 column-sum partials of the bias gradient.
struct ExtrasLayout {
  size_t gw0, gw1, bias_a, bias_b, total;
  // dense copies of tensors given as views, where a kernel wants dense operands
  // (0: not needed): the token tensors in the full-rank mode, the extra tokens
  size_t pack_x, pack_gy, pack_gx, ex_x, ex_gy, ex_gx;
};
constexpr int kBiasSlabsMax = 64;

static bool pitched(int64_t pitch, int C) { return pitch != 0 && pitch != C; }

static ExtrasLayout plan_extras(const lbp_layer& L, size_t base_total, int r, const lbp_extras* ex) {
  ExtrasLayout e{};
  size_t off = align_up(base_total, 1024);
  const size_t gw = static_cast<size_t>(L.Cout) * L.Cin * 4;
  e.gw0 = off;
  off = align_up(off + gw, 1024);
  e.gw1 = off;
  off = align_up(off + gw, 1024);
  const size_t part = static_cast<size_t>(kBiasSlabsMax) * L.Cout * 8;
  e.bias_a = off;
  off = align_up(off + part, 1024);
  e.bias_b = off;
  off = align_up(off + part, 1024);
  if (ex != nullptr) {
    const size_t es = static_cast<size_t>(elem_size(L.dtype));
    auto take = [&](size_t* where, size_t bytes) {
      *where = off;
      off = align_up(off + bytes, 1024);
    };
    if (r == L.k * L.k) {
      const size_t T = static_cast<size_t>(L.B) * L.H * L.W;
      if (!is_dense(&ex->x_view)) take(&e.pack_x, T * L.Cin * es);
      if (!is_dense(&ex->gy_view)) take(&e.pack_gy, T * L.Cout * es);
      if (!is_dense(&ex->gx_view)) take(&e.pack_gx, T * L.Cin * es);
    }
    if (ex->n_extra > 0) {
      const size_t n = static_cast<size_t>(ex->n_extra);
      if (pitched(ex->x_extra_pitch, L.Cin)) take(&e.ex_x, n * L.Cin * es);
      if (pitched(ex->gy_extra_pitch, L.Cout)) take(&e.ex_gy, n * L.Cout * es);
      if (pitched(ex->gx_extra_pitch, L.Cin)) take(&e.ex_gx, n * L.Cin * es);
    }
  }
  e.total = off;
  return e;
}

// The persistent products kernel can be switched off (LBP_FUSED=0) to run the
// separate product and expansion kernels instead.
static bool fused_enabled() { return tune_options().fused; }

static Layout plan_layout(const lbp_layer& L, int r) {
  Layout w{};
  const long long T = static_cast<long long>(L.B) * L.H * L.W;
  // blocks of the grid extended with zero tokens to multiples of k
  const long long nb = static_cast<long long>(L.B) * blocks_along(L.H, L.k) * blocks_along(L.W, L.k);
  const int es = elem_size(L.dtype);
  size_t off = kStatusBytes;
  if (r < L.k * L.k) {
    w.rows = nb * r;
    w.x_hat = off = align_up(off, 1024);
    off += static_cast<size_t>(w.rows) * L.Cin * es;
    w.gy_hat = off = align_up(off, 1024);
    off += static_cast<size_t>(w.rows) * L.Cout * es;
    w.gx_hat = off = align_up(off, 1024);
    off += static_cast<size_t>(w.rows) * L.Cin * 4;
    const size_t a = gemm_splitk_ws_bytes(L.Cout, L.Cin, w.rows, L.dtype);
    const size_t b = gemm_splitk_ws_bytes(w.rows, L.Cin, L.Cout, L.dtype);
    w.splitk_bytes = a > b ? a : b;
  } else {
    w.rows = T;
    const size_t a = gemm_splitk_ws_bytes(L.Cout, L.Cin, T, L.dtype);
    const size_t b = gemm_splitk_ws_bytes(T, L.Cin, L.Cout, L.dtype);
    w.splitk_bytes = a > b ? a : b;
  }
  w.splitk = off = align_up(off, 1024);
  off += w.splitk_bytes;
  // scratch of the persistent products kernel (bf16, r <= 16): x_hat and
  // g_y_hat with rows padded to 128-row groups
  w.fused = off = align_up(off, 1024);
  if (r < L.k * L.k && L.dtype == LBP_BF16 && r <= fused_max_rank(L.k))
    off += fused_scratch_bytes(L, r, nullptr);
  w.total = align_up(off, 256);
  return w;
}

// Phase-event hook (see lbp_set_phase_events).
static thread_local void** g_phase_events = nullptr;
static thread_local int g_phase_n = 0;
constexpr int kPhaseCount = 6;

static int mark_phase(int i, cudaStream_t stream) {
  if (g_phase_events != nullptr && i < g_phase_n && g_phase_events[i] != nullptr)
    LBP_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(g_phase_events[i]), stream));
  return LBP_OK;
}

static int run_fullrank(const void* x, const void* g_y, const void* W, void* g_x, void* g_W,
                        const lbp_layer& L, uint8_t* ws, cudaStream_t stream) {
  const Layout lay = plan_layout(L, L.k * L.k);
  const long long T = lay.rows;
  uint32_t* status = reinterpret_cast<uint32_t*>(ws);
  float* sk = reinterpret_cast<float*>(ws + lay.splitk);
  if (int e = mark_phase(0, stream)) return e;
  // Eq. 2: g_W = g_y^T x
  if (int e = launch_gemm(g_y, /*a_mn_major=*/true, x, g_W, L.dtype, L.gw_dtype, L.Cout, L.Cin, T,
                          sk, lay.splitk_bytes, status, stream))
    return e;
  if (int e = mark_phase(3, stream)) return e;
  // Eq. 2: g_x = g_y W
  if (int e = launch_gemm(g_y, /*a_mn_major=*/false, W, g_x, L.dtype, L.dtype, T, L.Cin, L.Cout,
                          sk, lay.splitk_bytes, status, stream))
    return e;
  return mark_phase(4, stream);
}

}  // namespace lbp

using namespace lbp;

extern "C" {

size_t lbp_workspace_bytes(const lbp_layer* layer, int r) {
  if (check_layer(layer) != LBP_OK) return 0;
  if (r < 1 || r > layer->k * layer->k) return 0;
  return plan_layout(*layer, r).total;
}

int lbp_project(const void* t, void* t_hat, int B, int H, int W, int C, int k,
                const lbp_basis* set, int r, int dtype, void* ws, size_t ws_bytes, void* stream) {
  if (t == nullptr || t_hat == nullptr) return LBP_ERR_NULL;
  if (int e = check_grid(B, H, W, C, k, dtype)) return e;
  BasisPlan plan;
  if (int e = make_basis_plan(k, set, r, &plan)) return e;
  if (!aligned16(t) || !aligned16(t_hat) || !aligned16(ws)) return LBP_ERR_ALIGN;
  if (ws == nullptr || ws_bytes < kStatusBytes) return LBP_ERR_WORKSPACE;
  if (int e = check_device_arch()) return e;
  return launch_project(t, t_hat, dtype, B, H, W, C, plan, RowMap{1, r},
                        static_cast<uint32_t*>(ws), static_cast<cudaStream_t>(stream));
}

size_t lbp_spectrum_workspace_bytes(int B, int H, int W, int C, int k, int dtype) {
  if (check_grid(B, H, W, C, k, dtype) != LBP_OK) return 0;
  const size_t es = dtype == LBP_BF16 ? 2 : 4;
  // all k*k coefficients per block of the zero-extended grid
  const size_t coef = static_cast<size_t>(B) * blocks_along(H, k) * blocks_along(W, k) * k * k * C * es;
  return kStatusBytes + (coef + 255) / 256 * 256;
}

int lbp_spectrum(const void* t, double* energy, int B, int H, int W, int C, int k, int dtype,
                 void* ws, size_t ws_bytes, void* stream) {
  if (t == nullptr || energy == nullptr) return LBP_ERR_NULL;
  if (int e = check_grid(B, H, W, C, k, dtype)) return e;
  const int r = k * k;
  lbp_basis all[256];
  for (int i = 0; i < k; ++i)
    for (int j = 0; j < k; ++j) all[i * k + j] = lbp_basis{i, j};
  BasisPlan plan;
  if (int e = make_basis_plan(k, all, r, &plan)) return e;
  if (!aligned16(t) || !aligned16(ws) || (reinterpret_cast<uintptr_t>(energy) & 7u) != 0)
    return LBP_ERR_ALIGN;
  if (ws == nullptr || ws_bytes < lbp_spectrum_workspace_bytes(B, H, W, C, k, dtype))
    return LBP_ERR_WORKSPACE;
  if (int e = check_device_arch()) return e;
  uint8_t* wsb = static_cast<uint8_t*>(ws);
  void* coef = wsb + kStatusBytes;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (spectrum_mma_supported(k, dtype))   // one pass, nothing materialised
    return launch_spectrum_mma(t, B, H, W, C, plan, energy, static_cast<uint32_t*>(ws), st);
  if (int e = launch_project(t, coef, dtype, B, H, W, C, plan, RowMap{1, r},
                             static_cast<uint32_t*>(ws), st))
    return e;
  const long long rows = static_cast<long long>(B) * blocks_along(H, k) * blocks_along(W, k) * k * k;
  return launch_square_reduce(coef, dtype, rows, C, r, energy, st);
}

int lbp_expand(const void* t_hat, void* t, int B, int H, int W, int C, int k,
               const lbp_basis* set, int r, int dtype, void* ws, size_t ws_bytes, void* stream) {
  if (t == nullptr || t_hat == nullptr) return LBP_ERR_NULL;
  if (int e = check_grid(B, H, W, C, k, dtype)) return e;
  BasisPlan plan;
  if (int e = make_basis_plan(k, set, r, &plan)) return e;
  if (!aligned16(t) || !aligned16(t_hat) || !aligned16(ws)) return LBP_ERR_ALIGN;
  if (ws == nullptr || ws_bytes < kStatusBytes) return LBP_ERR_WORKSPACE;
  if (int e = check_device_arch()) return e;
  return launch_expand(t_hat, /*in_f32=*/dtype == LBP_F32, t, dtype, B, H, W, C, plan,
                       RowMap{1, r}, static_cast<cudaStream_t>(stream));
}

// Host-side checks of one lbp_backward problem; nothing is enqueued.
static int validate_backward(const void* x, const void* g_y, const void* W, const void* g_x,
                             const void* g_W, const lbp_layer* layer, const lbp_basis* set, int r,
                             const void* ws, size_t ws_bytes, BasisPlan* plan, Layout* lay) {
  if (x == nullptr || g_y == nullptr || W == nullptr || g_x == nullptr || g_W == nullptr)
    return LBP_ERR_NULL;
  if (int e = check_layer(layer)) return e;
  if (int e = make_basis_plan(layer->k, set, r, plan)) return e;
  if (!aligned16(x) || !aligned16(g_y) || !aligned16(W) || !aligned16(g_x) || !aligned16(g_W) ||
      !aligned16(ws))
    return LBP_ERR_ALIGN;
  *lay = plan_layout(*layer, r);
  if (ws == nullptr || ws_bytes < lay->total) return LBP_ERR_WORKSPACE;
  return LBP_OK;
}

}  // extern "C"

namespace lbp {

// Stream and events of the library's own for lbp_backward_batch, one set per
// device, created at the first batch call on that device and kept.
struct SideStream {
  cudaStream_t stream;
  cudaEvent_t fork;
  cudaEvent_t done[64];
};
static int side_stream(SideStream** out) {
  static SideStream per_device[64];
  static bool ready[64] = {};
  static std::mutex mu;
  int dev = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return LBP_ERR_ARCH;
  std::lock_guard<std::mutex> lock(mu);
  if (!ready[dev]) {
    SideStream& s = per_device[dev];
    LBP_CUDA_TRY(cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking));
    LBP_CUDA_TRY(cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming));
    for (int i = 0; i < 64; ++i)
      LBP_CUDA_TRY(cudaEventCreateWithFlags(&s.done[i], cudaEventDisableTiming));
    ready[dev] = true;
  }
  *out = &per_device[dev];
  return LBP_OK;
}

// How lbp_backward_batch runs its problems: in which order, whether the
// projections go to the side stream, and how many SMs the projection at each
// position gets beside the products kernel before it.
struct BatchPlan {
  bool side;
  int sms;
  int order[64];
  int proj_sms[64];   // by position; 0 = all SMs
};

static int plan_batch(int n, const lbp_layer* layers, const lbp_basis* set, int r, BatchPlan* out) {
  BatchPlan& bp = *out;
  bp.side = false;
  bp.sms = 0;
  for (int i = 0; i < n; ++i) {
    bp.order[i] = i;
    bp.proj_sms[i] = 0;
  }
  const int want = tune_options().batch_proj_sms;
  if (n < 2 || !fused_enabled() || want == 0 || r > 48) return LBP_OK;
  if (int e = check_device_arch()) return e;
  int dev = 0, sms = 0;
  LBP_CUDA_TRY(cudaGetDevice(&dev));
  LBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (sms < 96) return LBP_OK;
  bp.sms = sms;

  // recent answers (the search below evaluates the cost models many times)
  struct Key {
    int n, r, sms, want;
    lbp_layer layers[8];
    lbp_basis set[16];
    BatchPlan plan;
  };
  static thread_local Key cache[8];
  static thread_local int cache_n = 0, cache_next = 0;
  const bool keyed = n <= 8;
  auto same = [&](const Key& k) {
    if (k.n != n || k.r != r || k.sms != sms || k.want != want) return false;
    for (int i = 0; i < n; ++i)
      if (std::memcmp(&k.layers[i], &layers[i], sizeof(lbp_layer)) != 0) return false;
    for (int q = 0; q < r; ++q)
      if (k.set[q].i != set[q].i || k.set[q].j != set[q].j) return false;
    return true;
  };
  if (keyed)
    for (int c = 0; c < cache_n; ++c)
      if (same(cache[c])) {
        bp = cache[c].plan;
        return LBP_OK;
      }

  BasisPlan plans[64];
  for (int i = 0; i < n; ++i) {
    if (make_basis_plan(layers[i].k, set, r, &plans[i]) != LBP_OK || r >= layers[i].k * layers[i].k ||
        !fused_supported(layers[i], plans[i]) || !fused_pair_supported(layers[i], sms))
      return LBP_OK;   // a problem that takes another path: one stream, given order
  }
  bp.side = true;

  // cost of running problem a's products kernel beside problem b's projection,
  // and the SM split that gives it
  auto pair_cost = [&](int a, int b, int* ps_out) {
    double best = -1.0;
    int lo = 40, hi = sms - 40;
    if (want > 0) lo = hi = want & ~1;
    for (int ps = lo; ps <= hi; ps += 4) {
      const double tp = fused_projection_model_us(layers[b], plans[b], ps);
      const double tq = fused_products_model_us(layers[a], plans[a], (sms - ps) / 2);
      const double t = tp > tq ? tp : tq;
      if (best < 0 || t < best) {
        best = t;
        *ps_out = ps;
      }
    }
    return best;
  };
  if (n <= 6) {
    // every order: first projection alone + pairs + last products kernel alone
    static thread_local double pc[6][6];
    static thread_local int pps[6][6];
    double first[6], last[6];
    for (int a = 0; a < n; ++a) {
      first[a] = fused_projection_model_us(layers[a], plans[a], sms);
      last[a] = fused_products_model_us(layers[a], plans[a], sms / 2);
      for (int b = 0; b < n; ++b)
        if (a != b) pc[a][b] = pair_cost(a, b, &pps[a][b]);
    }
    int perm[6], best_perm[6];
    for (int i = 0; i < n; ++i) perm[i] = best_perm[i] = i;
    double best = -1.0;
    do {
      double t = first[perm[0]] + last[perm[n - 1]];
      for (int i = 0; i + 1 < n; ++i) t += pc[perm[i]][perm[i + 1]];
      if (best < 0 || t < best - 1e-9) {
        best = t;
        for (int i = 0; i < n; ++i) best_perm[i] = perm[i];
      }
    } while (std::next_permutation(perm, perm + n));
    if (tune_options().verbose) {
      for (int a = 0; a < n; ++a) {
        fprintf(stderr, "lbp batch model: problem %d projection alone %.1f, products alone %.1f; beside:", a,
                first[a], last[a]);
        for (int b = 0; b < n; ++b)
          if (a != b) fprintf(stderr, " [%d] %.1f @%d", b, pc[a][b], pps[a][b]);
        fprintf(stderr, "\n");
      }
    }
    if (const char* e = std::getenv("LBP_BATCH_ORDER")) {   // tuning override: "1,3,2,0"
      int o[6] = {0, 1, 2, 3, 4, 5};
      bool seen[6] = {};
      bool ok = std::sscanf(e, "%d,%d,%d,%d,%d,%d", &o[0], &o[1], &o[2], &o[3], &o[4], &o[5]) >= n;
      for (int i = 0; i < n && ok; ++i) {
        ok = o[i] >= 0 && o[i] < n && !seen[o[i]];
        if (ok) seen[o[i]] = true;
      }
      if (ok)
        for (int i = 0; i < n; ++i) best_perm[i] = o[i];
    }
    for (int i = 0; i < n; ++i) bp.order[i] = best_perm[i];
    for (int i = 1; i < n; ++i) bp.proj_sms[i] = pps[best_perm[i - 1]][best_perm[i]];
  } else {
    for (int i = 1; i < n; ++i) pair_cost(i - 1, i, &bp.proj_sms[i]);
  }
  if (tune_options().verbose) {
    fprintf(stderr, "lbp batch: order");
    for (int i = 0; i < n; ++i) fprintf(stderr, " %d", bp.order[i]);
    fprintf(stderr, "; SMs of each projection beside the products kernel before it:");
    for (int i = 1; i < n; ++i) fprintf(stderr, " %d", bp.proj_sms[i]);
    fprintf(stderr, "\n");
  }
  if (keyed) {
    Key& k = cache[cache_next];
    k.n = n;
    k.r = r;
    k.sms = sms;
    k.want = want;
    for (int i = 0; i < n; ++i) k.layers[i] = layers[i];
    for (int q = 0; q < r; ++q) k.set[q] = set[q];
    k.plan = bp;
    cache_next = (cache_next + 1) % 8;
    if (cache_n < 8) ++cache_n;
  }
  return LBP_OK;
}

int validate_backward_call(const void* x, const void* g_y, const void* W, const void* g_x,
                           const void* g_W, const lbp_layer* layer, const lbp_basis* set, int r,
                           const void* ws, size_t ws_bytes) {
  BasisPlan plan;
  Layout lay;
  return validate_backward(x, g_y, W, g_x, g_W, layer, set, r, ws, ws_bytes, &plan, &lay);
}
}  // namespace lbp

extern "C" {

int lbp_test_tile_plan(int Cin, int Cout, int G, int bpt, int k, int units, int pair,
                       int max_splits, int epi_kind, int32_t* out6, uint16_t* first, uint16_t* ids) {
  if (out6 == nullptr || first == nullptr || ids == nullptr) return LBP_ERR_NULL;
  if (Cin < 1 || Cout < 1 || G < 1 || bpt < 1 || units < 1 || units > kSchedMaxUnits ||
      epi_kind < 0 || epi_kind > 2)
    return LBP_ERR_SHAPE;
  PlanShape s{};
  s.Cin = Cin;
  s.Cout = Cout;
  s.G = G;
  s.bpt = bpt;
  s.k = k;
  s.units = units;
  s.pair = pair ? 1 : 0;
  s.max_splits = max_splits;
  s.epi_kind = epi_kind;
  s.num_kb_w = G * 2;
  s.num_kb_x = (Cout + 63) / 64;
  const TilePlan& t = plan_products(s);
  out6[0] = t.BNw;
  out6[1] = t.BNx;
  out6[2] = t.splits;
  out6[3] = t.kbps;
  out6[4] = t.sched.listed;
  out6[5] = t.sched.listed ? t.sched.first[kSchedMaxUnits] : 0;
  for (int i = 0; i <= kSchedMaxUnits; ++i) first[i] = t.sched.first[i];
  for (int i = 0; i < kSchedMaxItems; ++i) ids[i] = t.sched.ids[i];
  return LBP_OK;
}

size_t lbp_test_struct_size(int which) {
  switch (which) {
    case 0: return sizeof(lbp_layer);
    case 1: return sizeof(lbp_extras);
    case 2: return sizeof(lbp_view);
    case 3: return sizeof(lbp_basis);
  }
  return 0;
}

int lbp_test_reload_env(void) {
  reload_tune_options();
  return LBP_OK;
}

int lbp_test_stall_products(int on) {
  set_test_stall((on & 1) != 0);
  set_test_stall_projection((on & 2) != 0);
  return LBP_OK;
}

int lbp_backward_batch(int n, const void* const* x, const void* const* g_y, const void* const* W,
                       void* const* g_x, void* const* g_W, const lbp_layer* layers,
                       const lbp_basis* set, int r, void* const* ws, const size_t* ws_bytes,
                       void* const* done_events, void* stream) {
  if (n < 1 || n > 64) return LBP_ERR_SHAPE;
  if (x == nullptr || g_y == nullptr || W == nullptr || g_x == nullptr || g_W == nullptr ||
      layers == nullptr || ws == nullptr || ws_bytes == nullptr)
    return LBP_ERR_NULL;
  struct Range {
    uintptr_t lo, hi;
  };
  auto range = [](const void* p, size_t bytes) {
    const uintptr_t lo = reinterpret_cast<uintptr_t>(p);
    return Range{lo, lo + bytes};
  };
  auto overlap = [](const Range& a, const Range& b) { return a.lo < b.hi && b.lo < a.hi; };
  Range in[64][3], out[64][3];
  for (int i = 0; i < n; ++i) {
    BasisPlan plan;
    Layout lay;
    if (int e = validate_backward(x[i], g_y[i], W[i], g_x[i], g_W[i], &layers[i], set, r, ws[i],
                                  ws_bytes[i], &plan, &lay))
      return e;
    const lbp_layer& L = layers[i];
    const size_t T = static_cast<size_t>(L.B) * L.H * L.W, es = elem_size(L.dtype);
    in[i][0] = range(x[i], T * L.Cin * es);
    in[i][1] = range(g_y[i], T * L.Cout * es);
    in[i][2] = range(W[i], static_cast<size_t>(L.Cout) * L.Cin * es);
    out[i][0] = range(g_x[i], T * L.Cin * es);
    out[i][1] = range(g_W[i], static_cast<size_t>(L.Cout) * L.Cin * elem_size(L.gw_dtype));
    out[i][2] = range(ws[i], lay.total);
  }
  // what one problem writes, no other problem may read or write
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j) {
      if (i == j) continue;
      for (int a = 0; a < 3; ++a)
        for (int b = 0; b < 3; ++b)
          if (overlap(out[i][a], in[j][b]) || (i < j && overlap(out[i][a], out[j][b])))
            return LBP_ERR_OVERLAP;
    }
  // Side-stream mode.  The projection streams x and g_y from HBM, the products
  // kernel lives on operands that sit in L2: run beside each other on disjoint
  // SMs they use different parts of the machine.  The projections of all problems
  // go to a stream of the library's own, one after the other; the projection of
  // the next problem gets some of the SMs while the products kernel of a problem
  // runs on the others (on the caller's stream, behind an event of its
  // projection).  The problems are independent, so they are taken in the order
  // that hides most: what stays exposed is the first projection and the last
  // products kernel.
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  BatchPlan bplan;
  if (int e = plan_batch(n, layers, set, r, &bplan)) return e;
  const bool side = bplan.side;
  SideStream* ss = nullptr;
  if (side) {
    if (int e = side_stream(&ss)) return e;
    // everything enqueued so far on the caller's stream comes before the first projection
    LBP_CUDA_TRY(cudaEventRecord(ss->fork, st));
    LBP_CUDA_TRY(cudaStreamWaitEvent(ss->stream, ss->fork, 0));
  }
  int status = LBP_OK;
  for (int pos = 0; pos < n && status == LBP_OK; ++pos) {
    const int i = bplan.order[pos];
    FusedOverlap ov{};
    if (side) {
      ov.proj_stream = ss->stream;
      ov.proj_done = ss->done[pos];
      ov.proj_ctas = bplan.proj_sms[pos];   // 0 (all SMs) for the first one: nothing runs beside it
      // nor beside the last products kernel
      ov.prod_units = pos == n - 1 ? 0 : (bplan.sms - bplan.proj_sms[pos + 1]) / 2;
      set_fused_overlap(&ov);
    } else {
      // One stream: from the second problem on, the projection kernel need not wait
      // for the kernel ahead of it (the previous problem's products kernel): it
      // starts on the SMs that kernel has already left.
      set_projection_defer_wait(pos > 0);
    }
    status = lbp_backward(x[i], g_y[i], W[i], g_x[i], g_W[i], &layers[i], set, r, ws[i],
                          ws_bytes[i], stream);
    set_fused_overlap(nullptr);
    if (status == LBP_OK && done_events != nullptr && done_events[i] != nullptr) {
      const cudaError_t ce = cudaEventRecord(static_cast<cudaEvent_t>(done_events[i]),
                                             static_cast<cudaStream_t>(stream));
      if (ce != cudaSuccess) {
        set_last_cuda_error(ce);
        status = LBP_ERR_CUDA;
      }
    }
  }
  set_projection_defer_wait(false);
  return status;
}

}  // extern "C"

namespace lbp {

// Where g_y_hat of a call lies (for the bias gradient): null when the call ran
// the full-rank mode and materialised nothing.
struct CoefLoc {
  const void* ptr;
  RowMap rows;
  double dc_to_sum;   // token sum of a block = dc_to_sum * its (0,0) coefficient as stored
};

// Algorithm 1 after validation.  Exactly one of x / x_hat is given: x_hat are the
// dense coefficients p(x), (blocks * r, Cin), taken earlier (Eq. 3).
// views: strides of x, g_y, g_x when they are not dense (low-rank paths only).
static int run_core(const void* x, const void* x_hat_in, const void* g_y, const void* W, void* g_x,
                    void* g_W, const lbp_layer& L, const BasisPlan& plan, const Layout& lay,
                    uint8_t* wsb, cudaStream_t st, CoefLoc* gy_loc,
                    const CallViews* views = nullptr) {
  const int r = plan.r;
  gy_loc->ptr = nullptr;
  if (r == L.k * L.k && x_hat_in == nullptr) return run_fullrank(x, g_y, W, g_x, g_W, L, wsb, st);

  uint32_t* status = reinterpret_cast<uint32_t*>(wsb);
  // the expansion of the products kernel addresses the tokens of an image with
  // 32-bit offsets (dense tensors: checked by fused_supported)
  const bool span_ok = views == nullptr || is_dense(&views->gx) ||
                       (views->gx.row * L.H + views->gx.token * L.W < (1ll << 31) &&
                        views->gx.image / 8 < (1ll << 31));
  if (fused_enabled() && fused_supported(L, plan) && span_ok) {
    FusedLayout fl;
    fused_scratch_bytes(L, r, &fl);
    gy_loc->ptr = wsb + lay.fused + fl.gy_hat;
    gy_loc->rows = RowMap{fl.bpt, 128};
    gy_loc->dc_to_sum = 1.0 / static_cast<double>(fused_scale_gy(L.k));
    // projection kernel, then one persistent kernel for both products with the
    // expansion fused into the g_x_hat epilogue
    if (int e = mark_phase(0, st)) return e;
    auto after_projection = [](void*, cudaStream_t s) -> int {
      if (int e = mark_phase(1, s)) return e;
      return mark_phase(2, s);
    };
    if (int e = launch_fused(x, x_hat_in, g_y, W, g_x, g_W, L, plan, wsb + lay.fused, status, st,
                             after_projection, nullptr, views))
      return e;
    for (int ph = 3; ph <= 5; ++ph)
      if (int e = mark_phase(ph, st)) return e;
    return LBP_OK;
  }
  const void* x_hat = x_hat_in != nullptr ? x_hat_in : wsb + lay.x_hat;
  void* gy_hat = wsb + lay.gy_hat;
  float* gx_hat = reinterpret_cast<float*>(wsb + lay.gx_hat);
  float* sk = reinterpret_cast<float*>(wsb + lay.splitk);
  const RowMap dense{1, r};
  gy_loc->ptr = gy_hat;
  gy_loc->rows = dense;
  gy_loc->dc_to_sum = static_cast<double>(L.k);   // orthonormal: coefficient = block sum / k

  if (int e = mark_phase(0, st)) return e;
  if (x_hat_in != nullptr) {
    // x_hat was taken at forward time: only g_y is projected
    if (int e = launch_project(g_y, gy_hat, L.dtype, L.B, L.H, L.W, L.Cout, plan, dense, status, st,
                               0.f, views ? &views->gy : nullptr))
      return e;
  } else {
    // Algorithm 1, steps 1-2: x_hat = p(x), g_y_hat = p(g_y), one launch for both
    if (int e = launch_project2(g_y, gy_hat, L.Cout, x, wsb + lay.x_hat, L.Cin, L.dtype, L.B, L.H,
                                L.W, plan, dense, status, st, 0.f, 0.f, views ? &views->gy : nullptr,
                                views ? &views->x : nullptr))
      return e;
  }
  if (int e = mark_phase(1, st)) return e;
  if (int e = mark_phase(2, st)) return e;
  // step 3: g_W = g_y_hat^T x_hat
  if (int e = launch_gemm(gy_hat, /*a_mn_major=*/true, x_hat, g_W, L.dtype, L.gw_dtype, L.Cout,
                          L.Cin, lay.rows, sk, lay.splitk_bytes, status, st))
    return e;
  if (int e = mark_phase(3, st)) return e;
  // step 4: g_x_hat = g_y_hat W   (kept in fp32)
  if (int e = launch_gemm(gy_hat, /*a_mn_major=*/false, W, gx_hat, L.dtype, LBP_F32, lay.rows,
                          L.Cin, L.Cout, sk, lay.splitk_bytes, status, st))
    return e;
  if (int e = mark_phase(4, st)) return e;
  // step 5: g_x = p^-1(g_x_hat)
  if (int e = launch_expand(gx_hat, /*in_f32=*/true, g_x, L.dtype, L.B, L.H, L.W, L.Cin, plan,
                            dense, st, views ? &views->gx : nullptr))
    return e;
  return mark_phase(5, st);
}

// A view is all zero (dense) or three positive strides, the token stride at
// least C, each a multiple of 16 bytes and within what a tensor map can hold.
static int check_view(const lbp_view& v, int C, int es) {
  if (v.image == 0 && v.row == 0 && v.token == 0) return LBP_OK;
  if (v.image <= 0 || v.row <= 0 || v.token < C) return LBP_ERR_SHAPE;
  const int64_t lim = (int64_t{1} << 40) / es;
  if (v.image >= lim || v.row >= lim || v.token >= lim) return LBP_ERR_SHAPE;
  if ((v.image * es) % 16 != 0 || (v.row * es) % 16 != 0 || (v.token * es) % 16 != 0)
    return LBP_ERR_ALIGN;
  return LBP_OK;
}

static int check_pitch(int64_t pitch, int C, int es) {
  if (pitch == 0) return LBP_OK;
  if (pitch < C) return LBP_ERR_SHAPE;
  return (pitch * es) % 16 != 0 ? LBP_ERR_ALIGN : LBP_OK;
}

static int check_extras(const lbp_extras* ex, const lbp_layer* L) {
  if (ex == nullptr) return LBP_OK;
  if (!(ex->beta == ex->beta)) return LBP_ERR_SHAPE;   // NaN
  if (ex->n_extra < 0) return LBP_ERR_SHAPE;
  const int es = elem_size(L->dtype);
  if (ex->n_extra > 0) {
    if (ex->x_extra == nullptr || ex->gy_extra == nullptr || ex->gx_extra == nullptr)
      return LBP_ERR_NULL;
    if (!aligned16(ex->x_extra) || !aligned16(ex->gy_extra) || !aligned16(ex->gx_extra))
      return LBP_ERR_ALIGN;
    if (int e = check_pitch(ex->x_extra_pitch, L->Cin, es)) return e;
    if (int e = check_pitch(ex->gy_extra_pitch, L->Cout, es)) return e;
    if (int e = check_pitch(ex->gx_extra_pitch, L->Cin, es)) return e;
  }
  if (ex->g_bias != nullptr && !aligned16(ex->g_bias)) return LBP_ERR_ALIGN;
  if (int e = check_view(ex->x_view, L->Cin, es)) return e;
  if (int e = check_view(ex->gy_view, L->Cout, es)) return e;
  if (int e = check_view(ex->gx_view, L->Cin, es)) return e;
  return LBP_OK;
}

// lbp_backward_ex after validation.
static int run_backward_ex(const void* x, const void* x_hat, const void* g_y, const void* W,
                           void* g_x, void* g_W, const lbp_layer& L, const BasisPlan& plan,
                           const Layout& lay, const lbp_extras* ex, uint8_t* wsb, cudaStream_t st) {
  CoefLoc gy_loc{};
  if (ex == nullptr) return run_core(x, x_hat, g_y, W, g_x, g_W, L, plan, lay, wsb, st, &gy_loc);

  CallViews cv{ex->x_view, ex->gy_view, ex->gx_view};
  const bool strided = !is_dense(&cv.x) || !is_dense(&cv.gy) || !is_dense(&cv.gx);
  const bool accumulate = ex->beta != 0.f || ex->n_extra > 0;
  if (!accumulate && ex->g_bias == nullptr && !strided)
    return run_core(x, x_hat, g_y, W, g_x, g_W, L, plan, lay, wsb, st, &gy_loc);

  const ExtrasLayout el = plan_extras(L, lay.total, plan.r, ex);
  uint32_t* status = reinterpret_cast<uint32_t*>(wsb);
  float* gw0 = reinterpret_cast<float*>(wsb + el.gw0);
  float* gw1 = reinterpret_cast<float*>(wsb + el.gw1);
  float* sk = reinterpret_cast<float*>(wsb + lay.splitk);
  const long long T = static_cast<long long>(L.B) * L.H * L.W;
  lbp_layer Lg = L;
  if (accumulate) Lg.gw_dtype = LBP_F32;   // this call's term in fp32, added below
  void* gw_core = accumulate ? static_cast<void*>(gw0) : g_W;

  // g_y as the bias gradient reads it when no coefficients serve
  const void* gy_tokens = g_y;
  TokenMap gy_map = token_map(resolve_view(&cv.gy, L.H, L.W, L.Cout), L.H, L.W);
  if (plan.r == L.k * L.k && x_hat == nullptr && strided) {
    // Eq. 2 runs on dense matrices: views go through dense copies
    const void* xd = x;
    const void* gyd = g_y;
    void* gxd = g_x;
    if (el.pack_x != 0) {
      if (int e = launch_copy_tokens(x, wsb + el.pack_x, true, T, L.Cin, L.dtype,
                                     token_map(cv.x, L.H, L.W), st))
        return e;
      xd = wsb + el.pack_x;
    }
    if (el.pack_gy != 0) {
      if (int e = launch_copy_tokens(g_y, wsb + el.pack_gy, true, T, L.Cout, L.dtype,
                                     token_map(cv.gy, L.H, L.W), st))
        return e;
      gyd = wsb + el.pack_gy;
      gy_tokens = gyd;
      gy_map = TokenMap{1, 1, L.Cout, L.Cout, L.Cout};
    }
    if (el.pack_gx != 0) gxd = wsb + el.pack_gx;
    if (int e = run_core(xd, nullptr, gyd, W, gxd, gw_core, Lg, plan, lay, wsb, st, &gy_loc)) return e;
    if (el.pack_gx != 0)
      if (int e = launch_copy_tokens(gxd, g_x, false, T, L.Cin, L.dtype, token_map(cv.gx, L.H, L.W), st))
        return e;
  } else {
    if (int e = run_core(x, x_hat, g_y, W, g_x, gw_core, Lg, plan, lay, wsb, st, &gy_loc,
                         strided ? &cv : nullptr))
      return e;
  }
  const TokenMap gye_map{1, 1, pitched(ex->gy_extra_pitch, L.Cout) ? ex->gy_extra_pitch : L.Cout, 0, 0};
  if (ex->n_extra > 0) {
    // tokens outside the grid (a class token): Eq. 2 exactly, on dense rows
    const void* xe = ex->x_extra;
    const void* gye = ex->gy_extra;
    void* gxe = ex->gx_extra;
    if (el.ex_x != 0) {
      if (int e = launch_copy_tokens(xe, wsb + el.ex_x, true, ex->n_extra, L.Cin, L.dtype,
                                     TokenMap{1, 1, ex->x_extra_pitch, 0, 0}, st))
        return e;
      xe = wsb + el.ex_x;
    }
    if (el.ex_gy != 0) {
      if (int e = launch_copy_tokens(gye, wsb + el.ex_gy, true, ex->n_extra, L.Cout, L.dtype, gye_map, st))
        return e;
      gye = wsb + el.ex_gy;
    }
    if (el.ex_gx != 0) gxe = wsb + el.ex_gx;
    if (int e = launch_gemm(gye, /*a_mn_major=*/true, xe, gw1, L.dtype, LBP_F32, L.Cout, L.Cin,
                            ex->n_extra, sk, lay.splitk_bytes, status, st))
      return e;
    if (int e = launch_gemm(gye, /*a_mn_major=*/false, W, gxe, L.dtype, L.dtype, ex->n_extra, L.Cin,
                            L.Cout, sk, lay.splitk_bytes, status, st))
      return e;
    if (el.ex_gx != 0)
      if (int e = launch_copy_tokens(gxe, ex->gx_extra, false, ex->n_extra, L.Cin, L.dtype,
                                     TokenMap{1, 1, ex->gx_extra_pitch, 0, 0}, st))
        return e;
  }
  if (accumulate)
    if (int e = launch_gw_combine(g_W, L.gw_dtype == LBP_BF16, gw0, ex->n_extra > 0 ? gw1 : nullptr,
                                  ex->beta, static_cast<long long>(L.Cout) * L.Cin, st))
      return e;
  if (ex->g_bias != nullptr) {
    // Sum of g_y over all tokens.  With the DC basis (0,0) selected that is k times
    // the sum of the DC coefficients of g_y_hat, which the call has just produced;
    // otherwise g_y is read once more.
    double* pa = reinterpret_cast<double*>(wsb + el.bias_a);
    double* pb = reinterpret_cast<double*>(wsb + el.bias_b);
    int q_dc = -1;
    for (int q = 0; q < plan.r; ++q)
      if (plan.seq_i[q] == 0 && plan.seq_j[q] == 0) q_dc = q;
    long long n_a;
    double scale_a;
    if (gy_loc.ptr != nullptr && q_dc >= 0) {
      n_a = static_cast<long long>(L.B) * blocks_along(L.H, L.k) * blocks_along(L.W, L.k);
      scale_a = gy_loc.dc_to_sum;
      if (int e = launch_column_sum(gy_loc.ptr, L.dtype, n_a, L.Cout, gy_loc.rows, plan.r, q_dc, pa, st))
        return e;
    } else {
      n_a = T;
      scale_a = 1.0;
      if (int e = launch_column_sum(gy_tokens, L.dtype, n_a, L.Cout, RowMap{1, 1}, 0, 0, pa, st, &gy_map))
        return e;
    }
    if (ex->n_extra > 0)
      if (int e = launch_column_sum(ex->gy_extra, L.dtype, ex->n_extra, L.Cout, RowMap{1, 1}, 0, 0, pb,
                                    st, &gye_map))
        return e;
    if (int e = launch_bias_finish(static_cast<float*>(ex->g_bias), L.Cout, ex->beta, pa,
                                   bias_slabs(n_a), scale_a, pb, bias_slabs(ex->n_extra), st))
      return e;
  }
  return LBP_OK;
}

}  // namespace lbp

extern "C" {

int lbp_backward(const void* x, const void* g_y, const void* W, void* g_x, void* g_W,
                 const lbp_layer* layer, const lbp_basis* set, int r, void* ws, size_t ws_bytes,
                 void* stream) {
  BasisPlan plan;
  Layout lay;
  if (int e = validate_backward(x, g_y, W, g_x, g_W, layer, set, r, ws, ws_bytes, &plan, &lay))
    return e;
  if (int e = check_device_arch()) return e;
  CoefLoc loc{};
  return run_core(x, nullptr, g_y, W, g_x, g_W, *layer, plan, lay, static_cast<uint8_t*>(ws),
                  static_cast<cudaStream_t>(stream), &loc);
}

size_t lbp_workspace_bytes_ex(const lbp_layer* layer, int r, const lbp_extras* ex) {
  const size_t base = lbp_workspace_bytes(layer, r);
  if (base == 0 || check_extras(ex, layer) != LBP_OK) return 0;
  if (ex == nullptr) return base;
  const bool strided = !is_dense(&ex->x_view) || !is_dense(&ex->gy_view) || !is_dense(&ex->gx_view);
  if (ex->beta == 0.f && ex->n_extra == 0 && ex->g_bias == nullptr && !strided) return base;
  return plan_extras(*layer, base, r, ex).total;
}

int lbp_backward_ex(const void* x, const void* x_hat, const void* g_y, const void* W, void* g_x,
                    void* g_W, const lbp_layer* layer, const lbp_basis* set, int r,
                    const lbp_extras* ex, void* ws, size_t ws_bytes, void* stream) {
  if ((x == nullptr) == (x_hat == nullptr)) return LBP_ERR_NULL;   // exactly one of the two
  const void* xin = x != nullptr ? x : x_hat;
  BasisPlan plan;
  Layout lay;
  if (int e = validate_backward(xin, g_y, W, g_x, g_W, layer, set, r, ws, ws_bytes, &plan, &lay))
    return e;
  if (int e = check_extras(ex, layer)) return e;
  if (ws_bytes < lbp_workspace_bytes_ex(layer, r, ex)) return LBP_ERR_WORKSPACE;
  if (int e = check_device_arch()) return e;
  return run_backward_ex(x, x_hat, g_y, W, g_x, g_W, *layer, plan, lay, ex,
                         static_cast<uint8_t*>(ws), static_cast<cudaStream_t>(stream));
}

int lbp_backward_projected(const void* x_hat, const void* g_y, const void* W, void* g_x, void* g_W,
                           const lbp_layer* layer, const lbp_basis* set, int r, void* ws,
                           size_t ws_bytes, void* stream) {
  return lbp_backward_ex(nullptr, x_hat, g_y, W, g_x, g_W, layer, set, r, nullptr, ws, ws_bytes,
                         stream);
}

int lbp_backward_fullrank(const void* x, const void* g_y, const void* W, void* g_x, void* g_W,
                          const lbp_layer* layer, void* ws, size_t ws_bytes, void* stream) {
  if (x == nullptr || g_y == nullptr || W == nullptr || g_x == nullptr || g_W == nullptr)
    return LBP_ERR_NULL;
  if (int e = check_layer(layer)) return e;
  if (!aligned16(x) || !aligned16(g_y) || !aligned16(W) || !aligned16(g_x) || !aligned16(g_W) ||
      !aligned16(ws))
    return LBP_ERR_ALIGN;
  const Layout lay = plan_layout(*layer, layer->k * layer->k);
  if (ws == nullptr || ws_bytes < lay.total) return LBP_ERR_WORKSPACE;
  if (int e = check_device_arch()) return e;
  return run_fullrank(x, g_y, W, g_x, g_W, *layer, static_cast<uint8_t*>(ws),
                      static_cast<cudaStream_t>(stream));
}

int lbp_set_phase_events(void** events, int n) {
  if (events != nullptr && n < 1) return LBP_ERR_SHAPE;
  g_phase_events = events;
  g_phase_n = events ? n : 0;
  return LBP_OK;
}

int lbp_phase_count(void) { return kPhaseCount; }

const char* lbp_phase_name(int phase) {
  switch (phase) {
    case 0: return "start";
    case 1: return "project_x_gy";
    case 2: return "unused";
    case 3: return "gw_product";
    case 4: return "gxhat_product";
    case 5: return "expand";
    default: return "";
  }
}

int lbp_poll_status(void* ws, void* stream) {
  if (ws == nullptr) return LBP_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  LBP_CUDA_TRY(cudaStreamSynchronize(st));
  uint32_t words[4] = {0, 0, 0, 0};
  LBP_CUDA_TRY(cudaMemcpy(words, ws, sizeof(words), cudaMemcpyDeviceToHost));
  if (words[2] != kStatusMagic) return LBP_OK;
  LBP_CUDA_TRY(cudaMemset(ws, 0, sizeof(words)));
  return words[0] == 0 ? LBP_OK : static_cast<int>(words[0]);
}

}  // extern "C"
