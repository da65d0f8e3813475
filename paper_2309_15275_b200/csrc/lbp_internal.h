// Internal declarations shared by the translation units of liblbp:
// host-side plan structures, launch prototypes and error plumbing.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "lbp.h"

namespace lbp {

constexpr int kMaxOrder = 16;                    // largest WHT order k
constexpr int kMaxRank = kMaxOrder * kMaxOrder;  // r <= k*k

// Device status block at the start of every workspace (256 B reserved).
//   word 0: an lbp_status (LBP_ERR_TIMEOUT) written by a kernel whose wait expired
//   word 1: where that wait gave up (kernel id << 16 | site)
//   word 2: kStatusMagic, written together with word 0; the block counts as
//           "no error" unless the magic is present, so the caller's scratch
//           needs no initialisation.
constexpr size_t kStatusBytes = 256;
constexpr uint32_t kStatusMagic = 0x4C425045u;

// A validated basis list, prepared for the transform kernels.
//
// The kernels pool each k x k block down to LB x LB (LB = smallest power of two
// above the largest selected index; Walsh rows of sequency < LB are constant on
// runs of k/LB), run an LB x LB Hadamard butterfly in natural (Sylvester) order
// and pick the selected coefficients.  `qmap` maps a natural-order position
// (a, b) of that LB x LB array to the slot q of the basis list, -1 = unused.
struct BasisPlan {
  int32_t k;
  int32_t r;
  int32_t LB;
  int16_t qmap[kMaxRank];  // [a * LB + b]
  // order-k natural (Sylvester) row indices of the selected Walsh rows:
  // wal_{i_q}[u] = (-1)^popcount(nat_i[q] & u), likewise for j along W
  uint8_t nat_i[kMaxRank];
  uint8_t nat_j[kMaxRank];
  // the selected pairs themselves (sequency indices), slot by slot
  uint8_t seq_i[kMaxRank];
  uint8_t seq_j[kMaxRank];
};

// Validates (k, set, r) and fills `plan`.  Returns an lbp_status.
int make_basis_plan(int k, const lbp_basis* set, int r, BasisPlan* plan);

// Natural (Sylvester) row index of the length-n Walsh row with s sign changes.
int walsh_natural_index(int n, int s);
// wal_s[u] for order k: +1 or -1.
int walsh_sign(int k, int s, int u);

int check_order(int k);
// Blocks along a grid side of n tokens: sides that are not multiples of k are
// extended with zero tokens at their high end.
inline int blocks_along(int n, int k) { return (n + k - 1) / k; }

void set_last_cuda_error(cudaError_t e);
void count_launch(int n = 1);   // bumps the per-thread kernel-launch counter
void note_cuda_failure(cudaError_t e, const char* file, int line);   // LBP_VERBOSE_ERRORS=1: one line on stderr
#define LBP_CUDA_TRY(expr)                                 \
  do {                                                     \
    cudaError_t e__ = (expr);                              \
    if (e__ != cudaSuccess) {                              \
      ::lbp::set_last_cuda_error(e__);                     \
      ::lbp::note_cuda_failure(e__, __FILE__, __LINE__);   \
      return LBP_ERR_CUDA;                                 \
    }                                                      \
  } while (0)

// ---- tensor maps (TMA descriptors), encoded on the host ------------------
// 4-D channels-last tensor (B, H, W, C): box = one k x k block x box_c
// channels; no swizzle, or the 128-byte swizzle (box_c * element size must be 128).
// `view`: strides of a tensor that is not dense (null, or all zero: dense).
int encode_block_tensor_map(CUtensorMap* map, const void* base, int dtype, int B, int H, int W,
                            int C, int k, int box_c, bool swizzle128,
                            const lbp_view* view = nullptr);
// Same tensor with an explicit box of box_h x box_w tokens.
int encode_box_tensor_map(CUtensorMap* map, const void* base, int dtype, int B, int H, int W, int C,
                          int box_c, int box_w, int box_h, bool swizzle128,
                          const lbp_view* view = nullptr);
// The strides a view stands for (dense when null or all zero).
inline lbp_view resolve_view(const lbp_view* v, int H, int W, int C) {
  if (v != nullptr && v->token != 0) return *v;
  return lbp_view{static_cast<int64_t>(H) * W * C, static_cast<int64_t>(W) * C, C};
}
inline bool is_dense(const lbp_view* v) { return v == nullptr || v->token == 0; }
// 2-D row-major bf16 matrix (rows, cols): box = box_rows x 64 columns (128 B),
// 128-byte swizzle.
int encode_matrix_tensor_map(CUtensorMap* map, const void* base, long long rows, long long cols,
                             int box_rows);

// ---- kernel launchers (each returns an lbp_status) ------------------------
// Row q of block blk of a projected tensor lives at
//   (blk / bpt) * tile_rows + (blk % bpt) * r + q ;   dense: bpt = 1, tile_rows = r.
struct RowMap {
  int32_t bpt;
  int32_t tile_rows;
};

// `scale` multiplies the +-1 sums; 0 selects 1/k, the orthonormal coefficients of Eq. 6.
int launch_project(const void* t, void* t_hat, int dtype, int B, int H, int W, int C,
                   const BasisPlan& plan, RowMap rows, uint32_t* status, cudaStream_t stream,
                   float scale = 0.f, const lbp_view* view = nullptr);

// Per-thread switch read by the projection launchers (see ProjParams::defer_wait).
void set_projection_defer_wait(bool on);
bool projection_defer_wait();

// Per-thread launch shape of the tensor-pipe projection kernels (set around a
// launch by the side-stream mode of lbp_backward_batch):
//   max_ctas      0 = one CTA per SM, else at most this many CTAs
//   whole_tpcs    launch the CTAs as clusters of two, so that they fill both SMs
//                 of a TPC and leave the other TPCs whole for the CTA pairs of a
//                 products kernel that runs beside them
//   programmatic  launch with programmatic stream serialization
struct ProjLaunch {
  int max_ctas;
  bool whole_tpcs;
  bool programmatic;
};
void set_projection_launch(ProjLaunch shape);
ProjLaunch projection_launch();

// Projects two tensors that share the token grid (x and g_y) in one launch.
int launch_project2(const void* t0, void* out0, int C0, const void* t1, void* out1, int C1,
                    int dtype, int B, int H, int W, const BasisPlan& plan, RowMap rows,
                    uint32_t* status, cudaStream_t stream, float scale0 = 0.f, float scale1 = 0.f,
                    const lbp_view* view0 = nullptr, const lbp_view* view1 = nullptr);

// One-pass spectrum (bf16 data, k = 4 or 8): energy[i*k + j] of all k*k responses.
// plan: all k*k pairs in raster order.
bool spectrum_mma_supported(int k, int dtype);
int launch_spectrum_mma(const void* t, int B, int H, int W, int C, const BasisPlan& plan,
                        double* energy, uint32_t* status, cudaStream_t stream);

// energy[q] (device, r doubles, overwritten) = sum of squares of the rows
// q, q + r, ... of t_hat (rows x C of `dtype`).
int launch_square_reduce(const void* t_hat, int dtype, long long rows, int C, int r, double* energy,
                         cudaStream_t stream);

// t_hat is fp32 when `in_f32`, else of `dtype`; t is of `dtype`.
int launch_expand(const void* t_hat, bool in_f32, void* t, int dtype, int B, int H, int W, int C,
                  const BasisPlan& plan, RowMap rows, cudaStream_t stream,
                  const lbp_view* view = nullptr);

// D[M, N] = sum_k A(m, k) * B(k, n), fp32 accumulation.
//   a_mn_major == false: A is stored (M, K) row-major;  true: A is stored (K, M) row-major.
//   B is stored (K, N) row-major.  D is (M, N) row-major of d_dtype.
// bf16 operands run on tcgen05 tensor cores; fp32 operands on FFMA.
// `splitk_ws` holds fp32 partial tiles when the kernel splits K.
int launch_gemm(const void* A, bool a_mn_major, const void* Bm, void* D, int in_dtype, int d_dtype,
                long long M, long long N, long long K, float* splitk_ws, size_t splitk_ws_bytes,
                uint32_t* status, cudaStream_t stream);
size_t gemm_splitk_ws_bytes(long long M, long long N, long long K, int in_dtype);
// D[i] = sum over `splits` fp32 planes of mn elements each (mn a multiple of 4), in plane order.
int launch_splitk_reduce(const float* planes, void* D, long long mn, int splits, bool d_bf16,
                         cudaStream_t stream);

int check_device_arch();

// ---- kernels around Algorithm 1 (lbp_extras.cu) ----
// g_W <- beta * g_W + a (+ b); a, b fp32 of mn elements, g_W fp32 or bf16.
int launch_gw_combine(void* g_W, bool gw_bf16, const float* a, const float* b, float beta,
                      long long mn, cudaStream_t stream);
// Where token i of a tensor of HW-token images (rows of W tokens) starts, in
// the units of the strides: (i / HW) * s_image + ((i % HW) / W) * s_row + (i % W) * s_tok.
// Rows with a pitch: HW = W = 1, s_image = pitch.
struct TokenMap {
  int32_t HW, W;
  long long s_image, s_row, s_tok;
  __host__ __device__ long long offset(long long i) const {
    const long long b = i / HW;
    const int t = static_cast<int>(i - b * HW);
    return b * s_image + (t / W) * s_row + (t % W) * s_tok;
  }
};
inline TokenMap token_map(const lbp_view& v, int H, int W) {
  return TokenMap{H * W, W, v.image, v.row, v.token};
}
// Column sums in fp64 of n_sel selected rows of a matrix of `dtype`, as
// bias_slabs(n_sel) partial rows of C doubles.  r == 0: tokens 0..n_sel-1 under
// `tokens` (null: a dense (n_sel, C) matrix); r > 0: the row of slot q of block i
// of a dense coefficient matrix under the row map `rows`.
int bias_slabs(long long n_sel);
int launch_column_sum(const void* m, int dtype, long long n_sel, int C, RowMap rows, int r, int q,
                      double* partial, cudaStream_t stream, const TokenMap* tokens = nullptr);
// Gathers (to_dense) or scatters n_tok tokens of C channels between a tensor
// laid out as `tm` says (element strides, multiples of 16 bytes) and a dense
// (n_tok, C) matrix.
int launch_copy_tokens(const void* src, void* dst, bool to_dense, long long n_tok, int C, int dtype,
                       TokenMap tm, cudaStream_t stream);
// g_bias[c] <- beta * g_bias[c] + scale_a * (sum of the slabs of a) + (sum of the slabs of b)
int launch_bias_finish(float* g_bias, int C, float beta, const double* a, int slabs_a, double scale_a,
                       const double* b, int slabs_b, cudaStream_t stream);
// Dense coefficient rows (blocks * r, C) -> rows padded to groups under `rows`
// (rows no block owns are zero), every bf16 value multiplied by `factor` (a power of two).
int launch_regroup_rows(const void* dense, void* grouped, int nb, int r, RowMap rows, int C,
                        float factor, cudaStream_t stream);

// Tuning switches, read from the environment once (first use):
//   LBP_FUSED=0          separate product and expansion kernels instead of the
//                        persistent products kernel
//   LBP_PAIR=0           one-CTA products kernel also on wide layers
//   LBP_PROJECT_UMMA=0   projection of orders 8 and 16 on warp-level mma.sync instead of tcgen05
//   LBP_FUSED_TILES=a,b,c  column tiles of the two products and K slices of g_W
//   LBP_FUSED_VERBOSE=1  print the chosen tile plan
//   LBP_BATCH_PROJ_SMS=n lbp_backward_batch: SMs given to the projection of the next
//                        layer while the products kernel of a layer runs (0 = one
//                        kernel at a time; unset = chosen per pair of layers)
//   LBP_BATCH_ORDER=a,b,.. lbp_backward_batch (up to 6 problems): the order in which
//                        the problems are taken (read at every call)
struct TuneOptions {
  bool fused, pair, umma, verbose, has_tiles;
  int tiles_bnw, tiles_bnx, tiles_splits;
  int batch_proj_sms;   // -1 = library default
};
const TuneOptions& tune_options();
void reload_tune_options();   // test hook: read the environment again

// Every host-side check of one lbp_backward call (pointers, layer, basis list,
// alignment, workspace size); nothing is enqueued.  Returns an lbp_status.
int validate_backward_call(const void* x, const void* g_y, const void* W, const void* g_x,
                           const void* g_W, const lbp_layer* layer, const lbp_basis* set, int r,
                           const void* ws, size_t ws_bytes);

}  // namespace lbp
