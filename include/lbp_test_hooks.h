/*
 * lbp_test_hooks.h -- entry points of liblbp that exist for the test suite
 * only.  They are not part of the library's interface (include/lbp.h) and an
 * application has no use for them.
 */
#ifndef LBP_TEST_HOOKS_H_
#define LBP_TEST_HOOKS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Failure injection for the bounded waits of the persistent products kernel
 * (bf16 low-rank path of lbp_backward).  While switched on (per calling
 * thread), the TMA producer of every products launch issues no load at all.
 * Nothing is then in flight, the tensor-core issuer and the epilogue warps run
 * into their wait limits (about a second), the kernel reports LBP_ERR_TIMEOUT
 * in the status block of the call's workspace, releases its tensor memory and
 * returns; the outputs of that call are undefined and the context stays
 * usable.  The paper has no counterpart; this is how the exit path behind
 * lbp_poll_status is exercised without faulting or hanging a device.
 * `on`: bit 0 stalls the products kernels as described; bit 1 does the same to
 * the TMA producers of the tcgen05 projection kernel (orders 8 and 16, bf16, r <= 48:
 * lbp_project and the first kernel of lbp_backward); 0 switches both off.
 * Returns LBP_OK. */
int lbp_test_stall_products(int on);

/* Host-side tile plan of the persistent products kernel for a layer of Cin x
 * Cout channels whose low-rank rows fill G groups of 128 rows (bpt blocks per
 * group, order k), on `units` CTAs (pair = 0) or CTA pairs (pair = 1).
 * out6 = {BNw, BNx, K slices of g_W, k-blocks per slice, listed, tiles listed};
 * first: 161 entries, ids: 1536 entries: unit u works, in this order, on the
 * tiles ids[first[u]] .. ids[first[u+1]-1]; ids below (row tiles of g_W) *
 * (column tiles) * slices are GW tiles, the others GX tiles.  No device needed. */
int lbp_test_tile_plan(int Cin, int Cout, int G, int bpt, int k, int units, int pair,
                       int max_splits, int epi_kind, int32_t* out6, uint16_t* first, uint16_t* ids);

/* The library reads its tuning switches (LBP_FUSED, LBP_PAIR, LBP_FUSED_TILES,
 * LBP_FUSED_VERBOSE) from the environment once, at first use.  This reads them
 * again, so that one test process can run the same layer through the paths
 * the switches select.  Returns LBP_OK. */
int lbp_test_reload_env(void);

/* sizeof of the structs of include/lbp.h as the library was compiled (which: 0
 * lbp_layer, 1 lbp_extras, 2 lbp_view, 3 lbp_basis; anything else: 0), so that a
 * binding in another language can check its own declarations against them. */
size_t lbp_test_struct_size(int which);

#ifdef __cplusplus
}
#endif
#endif /* LBP_TEST_HOOKS_H_ */
