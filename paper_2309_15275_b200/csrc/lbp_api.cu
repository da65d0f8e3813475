// C-ABI entry points that touch the device: argument validation, workspace
// layout, TMA descriptor encoding and the launch sequence of Algorithm 1.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>

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
                            int C, int k, int box_c, bool swizzle128) {
  return encode_box_tensor_map(map, base, dtype, B, H, W, C, box_c, k, k, swizzle128);
}

int encode_box_tensor_map(CUtensorMap* map, const void* base, int dtype, int B, int H, int W, int C,
                          int box_c, int box_w, int box_h, bool swizzle128) {
  EncodeTiledFn enc;
  if (int e = get_encode_fn(&enc)) return e;
  const cuuint64_t es = static_cast<cuuint64_t>(elem_size(dtype));
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W),
                              static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(B)};
  const cuuint64_t strides[3] = {dims[0] * es, dims[0] * dims[1] * es,
                                 dims[0] * dims[1] * dims[2] * es};
  const cuuint32_t box[4] = {static_cast<cuuint32_t>(box_c), static_cast<cuuint32_t>(box_w),
                             static_cast<cuuint32_t>(box_h), 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r =
      enc(map, dtype == LBP_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
          4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
          CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
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
  if (H % k != 0 || W % k != 0) return LBP_ERR_SHAPE;
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

// The persistent products kernel can be switched off (LBP_FUSED=0) to run the
// separate product and expansion kernels instead.
static bool fused_enabled() { return tune_options().fused; }

static Layout plan_layout(const lbp_layer& L, int r) {
  Layout w{};
  const long long T = static_cast<long long>(L.B) * L.H * L.W;
  const long long nb = T / (L.k * L.k);
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
  if (r < L.k * L.k && L.dtype == LBP_BF16 && r <= 16)
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
  const size_t coef = static_cast<size_t>(B) * H * W * C * es;   // all k*k coefficients per block
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
  const long long rows = static_cast<long long>(B) * H * W;   // blocks * k * k
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
int validate_backward_call(const void* x, const void* g_y, const void* W, const void* g_x,
                           const void* g_W, const lbp_layer* layer, const lbp_basis* set, int r,
                           const void* ws, size_t ws_bytes) {
  BasisPlan plan;
  Layout lay;
  return validate_backward(x, g_y, W, g_x, g_W, layer, set, r, ws, ws_bytes, &plan, &lay);
}
}  // namespace lbp

extern "C" {

int lbp_test_reload_env(void) {
  reload_tune_options();
  return LBP_OK;
}

int lbp_test_stall_products(int on) {
  set_test_stall(on != 0);
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
  int status = LBP_OK;
  for (int i = 0; i < n && status == LBP_OK; ++i) {
    // From the second problem on, the projection kernel need not wait for the
    // kernel ahead of it (the previous problem's products kernel): it starts on
    // the SMs that kernel has already left.
    set_projection_defer_wait(i > 0);
    status = lbp_backward(x[i], g_y[i], W[i], g_x[i], g_W[i], &layers[i], set, r, ws[i],
                          ws_bytes[i], stream);
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

int lbp_backward(const void* x, const void* g_y, const void* W, void* g_x, void* g_W,
                 const lbp_layer* layer, const lbp_basis* set, int r, void* ws, size_t ws_bytes,
                 void* stream) {
  BasisPlan plan;
  Layout lay;
  if (int e = validate_backward(x, g_y, W, g_x, g_W, layer, set, r, ws, ws_bytes, &plan, &lay))
    return e;
  const lbp_layer& L = *layer;
  if (int e = check_device_arch()) return e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* wsb = static_cast<uint8_t*>(ws);
  if (r == L.k * L.k) return run_fullrank(x, g_y, W, g_x, g_W, L, wsb, st);

  uint32_t* status = reinterpret_cast<uint32_t*>(wsb);
  if (fused_enabled() && fused_supported(L, plan)) {
    // projection kernel, then one persistent kernel for both products with the
    // expansion fused into the g_x_hat epilogue
    if (int e = mark_phase(0, st)) return e;
    auto after_projection = [](void*, cudaStream_t s) -> int {
      if (int e = mark_phase(1, s)) return e;
      return mark_phase(2, s);
    };
    if (int e = launch_fused(x, g_y, W, g_x, g_W, L, plan, wsb + lay.fused, status, st,
                             after_projection, nullptr))
      return e;
    for (int ph = 3; ph <= 5; ++ph)
      if (int e = mark_phase(ph, st)) return e;
    return LBP_OK;
  }
  void* x_hat = wsb + lay.x_hat;
  void* gy_hat = wsb + lay.gy_hat;
  float* gx_hat = reinterpret_cast<float*>(wsb + lay.gx_hat);
  float* sk = reinterpret_cast<float*>(wsb + lay.splitk);
  const RowMap dense{1, r};

  if (int e = mark_phase(0, st)) return e;
  // Algorithm 1, steps 1-2: x_hat = p(x), g_y_hat = p(g_y), one launch for both
  if (int e = launch_project2(g_y, gy_hat, L.Cout, x, x_hat, L.Cin, L.dtype, L.B, L.H, L.W, plan,
                              dense, status, st))
    return e;
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
                            dense, st))
    return e;
  return mark_phase(5, st);
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
