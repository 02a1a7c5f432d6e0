/*
 * harts_conv -- tree-aware depthwise causal convolution on compact tokens for sm_100a (B200): C ABI.
 *
 * The operation (paper Section 4.2, "KDA state reuse and causal convolution"): the short causal convolution
 * that precedes the linear-attention core runs ONCE per compact token, and its history is the token's true
 * ancestors in the rollout tree -- never the rows that happen to precede it in the packed layout; positions
 * before the start of a trajectory contribute zero.  With taps indexed like a library conv1d (the last tap
 * multiplies the current token), per channel c:
 *
 *     y_t[c] = sum_{i=0}^{w-1} W[c, w-1-i] * x_{anc_i(t)}[c],    anc_0(t) = t, anc_{i+1}(t) = predecessor of anc_i(t)
 *
 * Backward of L = sum_t <dy_t, y_t>:  dx_a = sum over descendants t of a within w-1 steps, on every branch,
 * of W[:, w-1-i] * dy_t;  dW[c, w-1-i] = sum_t dy_t[c] * x_{anc_i(t)}[c].  The paper builds a temporary input
 * view with w-1 prepended ancestor rows per sequence; here the kernels follow an index table instead, so no view
 * is materialised and every row of x and dy is read from HBM once.
 *
 * Conventions are those of harts_la.h (int32 status, caller-owned device memory, caller's stream, no CPU
 * fallback).  x, y, dy, dx: row-major [n_rows, D] in physical compact rows, HARTS_BF16 or HARTS_FP32, D a
 * multiple of 8, 16-byte aligned.  W, dW: fp32 [D, w], 2 <= w <= 4.
 */
#ifndef HARTS_CONV_H_
#define HARTS_CONV_H_

#include <stddef.h>
#include <stdint.h>

#include "harts_la.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Index tables of a forest, in physical rows.  Host in, host out.
 *   tree_node_ptr, node_parent, node_fork_off, node_len: as for harts_la_plan()
 *   row_of_token [C] or NULL (identity): canonical token index -> physical row
 *   prev_row  [C] out: physical row of the token's predecessor on its trajectory, -1 at the start of a root
 *   next_row  [C] out: the row's only successor, -1 if it has none (a trajectory end), -2 if it has several (a fork)
 *   child_ptr [C+1], child_row [C - n_trees] out: CSR of successors (the tokens whose predecessor is the row),
 *             children of one row in canonical order
 * Errors: HARTS_EINVAL for a malformed forest or a row map that is not a permutation.
 */
int32_t harts_conv_index(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                         const int32_t* node_fork_off, const int32_t* node_len, const int32_t* row_of_token,
                         int32_t* prev_row, int32_t* next_row, int32_t* child_ptr, int32_t* child_row);

/* Forward.  All pointers device.  prev_row [n_rows] from harts_conv_index. */
int32_t harts_conv_fwd(const void* x, const float* W, const int32_t* prev_row, void* y, int32_t n_rows, int32_t D,
                       int32_t w, int32_t dtype, void* stream);

/* Bytes of the fp32 scratch the backward needs for the per-CTA partial sums of dW. */
int32_t harts_conv_scratch_bytes(int32_t D, int32_t w, size_t* bytes);

/*
 * Backward.  All pointers device.  dx [n_rows, D] (dtype of x) and dW [D, w] fp32 are overwritten; partial sums
 * of dW are combined in a fixed order (deterministic).  scratch: harts_conv_scratch_bytes(), 16-byte aligned,
 * needs no clearing.  next_row, child_ptr, child_row from harts_conv_index.
 */
int32_t harts_conv_bwd(const void* x, const float* W, const void* dy, const int32_t* next_row,
                       const int32_t* child_ptr, const int32_t* child_row, void* dx, float* dW, void* scratch,
                       int32_t n_rows, int32_t D, int32_t w, int32_t dtype, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HARTS_CONV_H_ */
