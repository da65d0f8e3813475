/*
 * lbp.h -- C ABI of the LBP-WHT linear-layer backward library for NVIDIA B200
 * (sm_100a).
 *
 * The library computes the backward pass of a linear layer y = x w^T the
 * LBP-WHT way (Low-rank BackPropagation via Walsh-Hadamard Transformation,
 * arXiv 2309.15275): x and g_y are projected onto r two-dimensional
 * Walsh-Hadamard bases per k x k block of the token grid (Eq. 3, Eq. 6), the
 * two gradient products run in that low-rank space (Eq. 4, Algorithm 1), and
 * the low-rank input gradient is expanded back with the transposed bases
 * (Eq. 5, Eq. 7).
 *
 * Conventions, valid for every entry point unless it says otherwise
 *  - Tensor pointers (x, g_y, W, g_x, g_W, t, t_hat, ws) are DEVICE pointers
 *    owned by the caller; they must be 16-byte aligned and C * element size
 *    must be a multiple of 16 bytes.  The library never allocates or frees
 *    device memory and keeps no per-call state.
 *  - Basis lists, layer descriptors and every other pointer are HOST pointers,
 *    read during the call and not retained.
 *  - Layouts are dense, channels-last raster:
 *        x   (B, H, W, Cin)     g_y (B, H, W, Cout)     g_x (B, H, W, Cin)
 *        W, g_W (Cout, Cin) row-major (w in R^{Cy x Cx} of Eq. 1)
 *        t_hat (B, ceil(H/k), ceil(W/k), r, C): coefficient q of a block follows
 *        the order of the basis list.
 *    Tokens are grouped into non-overlapping, origin-aligned k x k blocks of
 *    the (H, W) grid.  The paper does not say what happens to a grid whose
 *    sides are not multiples of the transform order (its own 7 x 7 maps of
 *    Sec. 3.3 and Table 5); here such a grid is extended with zero tokens at
 *    its high end (bottom rows, right columns) to the next multiples of k: a
 *    side of n tokens has ceil(n / k) blocks, the zero tokens are never read
 *    from or written to memory, and g_x is produced for the real tokens only.
 *  - Bases are orthonormal: the +-1 Walsh bases of Eq. 6-7 are scaled by 1/k
 *    in the projection and by 1/k in the reverse projection, so that all k*k
 *    bases reproduce exact backpropagation (Sec. 3, completeness).
 *  - A basis (i, j) is the outer product of the Walsh rows with i sign changes
 *    along H and j sign changes along W, 0 <= i, j < k (sequency order: a
 *    smaller index is a lower frequency, Sec. 3.2).
 *  - `stream` is a cudaStream_t passed as void*.  Device work is enqueued on
 *    it and the call returns without synchronising.  Argument errors are
 *    detected before anything is enqueued: on a non-zero return no output has
 *    been touched.  Waits inside kernels are bounded; an expired wait is
 *    reported through the status word in `ws` (lbp_poll_status).
 *  - Every function returns an lbp_status (0 = LBP_OK) unless it returns a
 *    size, a number or a string.
 */
#ifndef LBP_H_
#define LBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LBP_OK = 0,
  LBP_ERR_NULL = 1,       /* a required pointer is NULL                         */
  LBP_ERR_SHAPE = 2,      /* a dimension or count out of range                  */
  LBP_ERR_BLOCK = 3,      /* k not in {4, 8, 16}                                */
  LBP_ERR_BASIS = 4,      /* r < 1, r > k*k, index outside [0,k), duplicate pair */
  LBP_ERR_DTYPE = 5,      /* unknown dtype, or a combination not supported      */
  LBP_ERR_ALIGN = 6,      /* pointer or C * element size not 16-byte aligned    */
  LBP_ERR_WORKSPACE = 7,  /* ws is NULL or smaller than lbp_workspace_bytes()   */
  LBP_ERR_ARCH = 8,       /* current device is not compute capability 10.x      */
  LBP_ERR_CUDA = 9,       /* a CUDA call failed; see lbp_last_cuda_error()      */
  LBP_ERR_TIMEOUT = 10,   /* a bounded device-side wait expired                 */
  LBP_ERR_CAPACITY = 11,  /* output array too small (lbp_select_bases)          */
  LBP_ERR_OVERLAP = 12    /* buffers of different problems of a batch overlap   */
} lbp_status;

typedef enum { LBP_F32 = 0, LBP_BF16 = 1 } lbp_dtype;

/* Basis-selection rules of Sec. 3.2.  LP_L1 and LP_Linf are Eq. 8 and Eq. 9
 * with 0-based indices (i + j <= m-1, max(i,j) <= m-1; ranks m(m+1)/2 and m*m,
 * the ranks the paper's tables print).  PREFIX-r keeps the first r pairs of the
 * total order key(i,j) = (i+j, max(i,j), i), which lists every LP_L1 set as a
 * prefix and defines ranks that are neither triangular nor square. */
typedef enum { LBP_SEL_L1 = 0, LBP_SEL_LINF = 1, LBP_SEL_PREFIX = 2 } lbp_rule;

typedef struct { int32_t i, j; } lbp_basis;   /* 0-based sequency indices    */

typedef struct {
  int32_t B, H, W;        /* batch and token grid                               */
  int32_t Cin, Cout;      /* C_x and C_y of Eq. 1                               */
  int32_t k;              /* WHT order = block edge, 4, 8 or 16                 */
  int32_t dtype;          /* lbp_dtype of x, g_y, W, g_x                        */
  int32_t gw_dtype;       /* lbp_dtype of g_W (LBP_F32 allowed with bf16 data)  */
} lbp_layer;

/* ---- host-only helpers (no device needed) ------------------------------- */

/* Sec. 3.2, Eq. 8-9.  Writes the ordered basis list chosen by `rule` with
 * parameter `param` (m for LP_L1 / LP_Linf, r for PREFIX) for order k into
 * out[0..*r_out).  All rules list their pairs in the PREFIX total order.
 * out: host array of `cap` entries.  LBP_ERR_CAPACITY if cap is too small
 * (*r_out still receives the needed count), LBP_ERR_BLOCK / LBP_ERR_BASIS for
 * a bad k / param. */
int lbp_select_bases(int k, int rule, int param, lbp_basis* out, int cap, int* r_out);

/* Eq. 6: the k*k x r matrix (B_{i1,j1} ... B_{ir,jr}) of +-1 entries, row
 * u*k+v (raster position inside a block), column q.  P_out: host array of
 * k*k*r int8, row-major.  Validates the list like every other call. */
int lbp_basis_matrix(int k, const lbp_basis* set, int r, int8_t* P_out);

/* Sec. 3.2, low-heuristic-error (LHE) selection: the r bases with the largest
 * profiled energy, strongest first.  energy: host array of k*k doubles as
 * written by lbp_spectrum (index i*k + j).  The paper does not order equal
 * energies; the pair that comes first in the PREFIX order wins a tie, so the
 * list is unique.  out: host array of at least r entries.  LBP_ERR_BASIS for
 * r outside 1..k*k or an energy that is negative or not finite. */
int lbp_select_lhe(const double* energy, int k, int r, lbp_basis* out);

/* Table 1 closed forms, in FLOPs.  which: 0 vanilla BP 4 Cx Cy L, 1 projection
 * (Cx+Cy) L r, 2 low-rank products 4 Cx Cy r, 3 reverse projection Cx L r,
 * 4 = 1+2+3.  Returns a negative number for a bad `which`. */
double lbp_flops(int Cin, int Cout, long long L, int r, int which);

const char* lbp_status_string(int status);

/* cudaError_t (as int) of the most recent failed CUDA call made by this
 * library on the calling thread; 0 if none. */
int lbp_last_cuda_error(void);

/* ---- device entry points ------------------------------------------------- */

/* Bytes of scratch the calls below need for this layer at rank r (Algorithm 1
 * materialises x_hat and g_y_hat; the status word lives there too).  Returns 0
 * for an invalid layer.  lbp_project / lbp_expand need lbp_status_bytes(). */
size_t lbp_workspace_bytes(const lbp_layer* layer, int r);
size_t lbp_status_bytes(void);

/* Eq. 6 per block:  t_hat[b,bh,bw,q,c] = (1/k) sum_{u,v} wal_iq[u] wal_jq[v]
 *                                         t[b, bh*k+u, bw*k+v, c].
 * t (B,H,W,C) -> t_hat (B,ceil(H/k),ceil(W/k),r,C), both of `dtype`; fp32 accumulation,
 * one rounding to the output type.  ws: >= lbp_status_bytes(). */
int lbp_project(const void* t, void* t_hat, int B, int H, int W, int C, int k,
                const lbp_basis* set, int r, int dtype,
                void* ws, size_t ws_bytes, void* stream);

/* Sec. 3.2 (LHE profiling): energy of every basis response of t,
 *   energy[i*k + j] = sum over blocks and channels of t_hat[.., (i,j), ..]^2
 * with t_hat the coefficients of Eq. 6 for all k*k bases, so that the k*k
 * energies add up to ||t||^2.  t (B,H,W,C) of `dtype`; energy: DEVICE array of
 * k*k doubles, overwritten.  bf16 data: one pass over t, fp32
 * responses squared and summed in fp32 per thread, fp64 across threads, and
 * the workspace holds only the status block.  Otherwise the coefficients are
 * materialised in `dtype` (fp32 accumulation, one rounding) in the workspace
 * and their squares summed in fp32 per row, in fp64 across rows.
 * ws: >= lbp_spectrum_workspace_bytes(...); 0 from that call = invalid shape. */
size_t lbp_spectrum_workspace_bytes(int B, int H, int W, int C, int k, int dtype);
int lbp_spectrum(const void* t, double* energy, int B, int H, int W, int C, int k, int dtype,
                 void* ws, size_t ws_bytes, void* stream);

/* Eq. 7 per block:  t[b,bh*k+u,bw*k+v,c] = (1/k) sum_q wal_iq[u] wal_jq[v]
 *                                          t_hat[b,bh,bw,q,c].
 * t_hat (B,ceil(H/k),ceil(W/k),r,C) -> t (B,H,W,C), both of `dtype`. */
int lbp_expand(const void* t_hat, void* t, int B, int H, int W, int C, int k,
               const lbp_basis* set, int r, int dtype,
               void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1:  x_hat = p(x), g_y_hat = p(g_y), g_W = g_y_hat^T x_hat (summed
 * over batch, blocks and bases), g_x_hat = g_y_hat W, g_x = p^-1(g_x_hat).
 * g_x and g_W are overwritten.  With bf16 data x_hat and g_y_hat are rounded to
 * bf16, products accumulate in fp32, g_x_hat stays fp32 until g_x is rounded
 * once.  r == k*k (any order of the complete set) runs the full-rank mode.
 * ws: >= lbp_workspace_bytes(layer, r). */
int lbp_backward(const void* x, const void* g_y, const void* W,
                 void* g_x, void* g_W, const lbp_layer* layer,
                 const lbp_basis* set, int r,
                 void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1 for n (1..64) independent problems in one call, e.g. the linear
 * layers of a block whose inputs are all at hand: problem i is
 * lbp_backward(x[i], g_y[i], W[i], g_x[i], g_W[i], &layers[i], set, r, ws[i],
 * ws_bytes[i]); g_x is bit-identical to that call's, g_W equal up to the fp32
 * summation order of its K slices (the tile plan follows the SMs a problem
 * gets); results are deterministic.  x .. ws, ws_bytes: host arrays
 * of n entries.  What one problem writes (g_x, g_W, ws) no other problem may
 * read or write (LBP_ERR_OVERLAP); inputs may be shared.  Knowing that, the
 * library overlaps the problems:
 *  - bf16 problems of low rank (<= 16 at k = 4, <= 48 at k = 8 and 16) on wide layers: the projections run on a
 *    stream of the library's own (one non-blocking stream and a set of events
 *    per device, created at the first such call on that device and kept: make
 *    that call outside any stream capture; later calls may be captured into a
 *    CUDA graph, the library's stream joins the capture and leaves it before
 *    the call returns), the projection of one problem on
 *    part of the SMs beside the products kernel of another on the rest; the
 *    problems are taken in the order that leaves least of it exposed, not
 *    necessarily the given one.  Everything is ordered behind what `stream` held
 *    at the call, and `stream` ends up behind all of it.
 *  - otherwise the projection kernel of problem i + 1 starts on the SMs that the
 *    products kernel of problem i has already left instead of waiting for its
 *    last tile.
 * done_events: NULL, or a host array of n cudaEvent_t handles (as void*,
 * an entry may be NULL): event i is recorded on `stream` behind the last kernel
 * of problem i, so that the caller can start what consumes g_W[i] / g_x[i] on
 * another stream (the data-parallel all-reduce of g_W, the one exchange step
 * of the path) while the problems that follow still run.  All arguments are
 * checked before anything is enqueued. */
int lbp_backward_batch(int n, const void* const* x, const void* const* g_y, const void* const* W,
                       void* const* g_x, void* const* g_W, const lbp_layer* layers,
                       const lbp_basis* set, int r, void* const* ws, const size_t* ws_bytes,
                       void* const* done_events, void* stream);

/* Element strides of a (B,H,W,C) tensor with contiguous channels; all zero
 * means dense (H*W*C, W*C, C). */
typedef struct {
  int64_t image, row, token;
} lbp_view;

/* What a linear layer of a real ViT needs around Algorithm 1 and the paper
 * leaves out (Eq. 1 has no bias; Sec. 3 knows only the tokens of the grid).
 * All pointers are device pointers; the struct itself is read on the host. */
typedef struct {
  /* g_W <- beta * g_W + (g_W of this call); 0 overwrites.  beta = 1 adds a
   * micro-batch to an accumulated gradient.  g_bias follows the same rule. */
  float beta;
  /* NULL, or fp32[Cout]: gradient of a bias added to y, the sum of g_y over all
   * tokens (grid and extra).  With the basis (0,0) in the list this is k times
   * the sum of the DC coefficients of g_y_hat (exact in exact arithmetic: that
   * basis is the block sum scaled by 1/k); otherwise g_y is read once more. */
  void* g_bias;
  /* Tokens that are not part of the grid (a class token per image): the method
   * says nothing about them, so they take Eq. 2 exactly: g_x_extra = g_y_extra W
   * and g_y_extra^T x_extra is added to g_W.  n_extra = 0: none.
   * x_extra (n_extra, Cin), gy_extra (n_extra, Cout), gx_extra (n_extra, Cin),
   * of the layer's dtype. */
  int32_t n_extra;
  const void* x_extra;
  const void* gy_extra;
  void* gx_extra;
  /* Tensors that are views of larger ones (the tokens of a (B, 1 + H*W, C)
   * sequence behind its class token; a channel slice of a wider tensor).  A
   * view gives, in elements, the distance between consecutive images, rows and
   * tokens of a (B,H,W,C) tensor whose C channels stay contiguous.  All three
   * zero: dense.  Otherwise all three are positive, token >= C, and each times
   * the element size is a multiple of 16 bytes.  The low-rank path reads and
   * writes such tensors in place (the projection's TMA boxes and the
   * expansion's stores take the strides); the full-rank mode (r = k*k) goes
   * through dense copies in the workspace.  x_view is ignored when x_hat is
   * given.  Elements of g_x between the tokens are not written. */
  lbp_view x_view, gy_view, gx_view;
  /* Distance in elements between consecutive extra tokens (0: dense rows);
   * same rules as a view's strides.  With one class token per image in a
   * (B, 1 + H*W, C) sequence this is (1 + H*W) * C. */
  int64_t x_extra_pitch, gy_extra_pitch, gx_extra_pitch;
} lbp_extras;

/* Scratch for lbp_backward_ex (>= lbp_workspace_bytes; 0 = invalid arguments). */
size_t lbp_workspace_bytes_ex(const lbp_layer* layer, int r, const lbp_extras* ex);

/* Algorithm 1 with the parts above.  Exactly one of x and x_hat is given:
 *  - x (B,H,W,Cin): as lbp_backward;
 *  - x_hat (B,ceil(H/k),ceil(W/k),r,Cin) = p(x), the output of lbp_project with the
 *    same k and basis list (Eq. 3), taken at forward time so that only r / k^2
 *    of the activation is kept until the backward pass; Algorithm 1 then starts
 *    at its second step (g_y_hat = p(g_y)).  The result equals lbp_backward on
 *    x up to the rounding of x_hat to `dtype` that both take.
 * ex may be NULL (then this is lbp_backward / lbp_backward_projected).
 * ws: >= lbp_workspace_bytes_ex(layer, r, ex). */
int lbp_backward_ex(const void* x, const void* x_hat, const void* g_y, const void* W,
                    void* g_x, void* g_W, const lbp_layer* layer,
                    const lbp_basis* set, int r, const lbp_extras* ex,
                    void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1 from its second step on (Eq. 3 applied to x beforehand):
 * lbp_backward_ex with x = NULL and no extras.  ws: >= lbp_workspace_bytes. */
int lbp_backward_projected(const void* x_hat, const void* g_y, const void* W,
                           void* g_x, void* g_W, const lbp_layer* layer,
                           const lbp_basis* set, int r,
                           void* ws, size_t ws_bytes, void* stream);

/* Eq. 2, exact backpropagation: g_W = g_y^T x over all tokens, g_x = g_y W.
 * This is what all k*k bases give (P P^T = I), computed without transforms.
 * ws: >= lbp_workspace_bytes(layer, k*k). */
int lbp_backward_fullrank(const void* x, const void* g_y, const void* W,
                          void* g_x, void* g_W, const lbp_layer* layer,
                          void* ws, size_t ws_bytes, void* stream);

/* No counterpart in the paper: a packaging variant of lbp_backward for callers
 * that cannot allocate device memory.  Examples are a server that handed all
 * device memory to its own pool at start-up and forbids cudaMalloc afterwards,
 * a plug-in whose host framework passes it nothing but input and output
 * buffers, and code on a path where an allocation would synchronise the device
 * or is not permitted.  The scratch that lbp_backward takes from the caller
 * comes here from an array of LBP_STATIC_SCRATCH_BYTES that is part of the
 * library image: every GPU on which the library is loaded holds that much
 * memory until the process exits.
 *  - Same arguments, layouts and results as lbp_backward, minus ws / ws_bytes.
 *    The call allocates and frees nothing.
 *  - Layers with lbp_workspace_bytes(layer, r) > LBP_STATIC_SCRATCH_BYTES are
 *    rejected with LBP_ERR_WORKSPACE before anything is enqueued.
 *  - The first call on a device looks up the array's device address (no
 *    allocation, but a runtime query): make that first call outside any stream
 *    capture.  The device that is current at the call owns the scratch used.
 *  - All calls on a device share the one array.  Its status block is cleared
 *    on `stream` at the start of every call; everything else in it is
 *    overwritten before it is read.  Two calls whose device work overlaps in
 *    time (different streams, or different host threads) race on the array:
 *    order them on one stream or with events.
 *  - The status block is not reachable through lbp_poll_status; a caller that
 *    needs the device status uses lbp_backward with its own workspace. */
#define LBP_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
int lbp_backward_static(const void* x, const void* g_y, const void* W,
                        void* g_x, void* g_W, const lbp_layer* layer,
                        const lbp_basis* set, int r, void* stream);

/* Synchronises `stream`, reads the device status word at the start of ws and
 * clears it.  Returns LBP_OK, LBP_ERR_TIMEOUT (a bounded wait in a kernel
 * expired; outputs of that call are undefined, the context stays usable) or
 * LBP_ERR_CUDA. */
int lbp_poll_status(void* ws, void* stream);

/* ---- measurement hooks (no effect on results) ---------------------------- */

/* Number of kernels this library has launched from the calling thread since it
 * was loaded (a running count; take differences). */
long long lbp_launch_count(void);

/* Phase timing.  `events` is a HOST array of n cudaEvent_t handles (as void*),
 * or NULL to switch the hook off; the setting is per calling thread and the
 * array must stay valid while it is set.  While set, lbp_backward records
 * events[0] on `stream` before its first kernel and events[i] after phase i
 * (i < n), so that the elapsed time between events[i-1] and events[i] is the
 * device time of phase i of Algorithm 1:
 *   1 project x and g_y (one launch)   2 (unused, recorded with 1)
 *   3 g_W product   4 g_x_hat product   5 expand
 * Where one kernel covers several phases (bf16 on the persistent path: both products
 * and the expansion) its time shows up in the first of them and the others are
 * recorded right behind it; the full-rank mode records 0, 3 and 4 only.  lbp_phase_count() is the
 * number of events a call may record, lbp_phase_name(i) a short label. */
int lbp_set_phase_events(void** events, int n);
int lbp_phase_count(void);
const char* lbp_phase_name(int phase);

#ifdef __cplusplus
}
#endif
#endif /* LBP_H_ */
