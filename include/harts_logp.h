/*
 * harts_logp -- compact-to-semantic log-probability for sm_100a (B200): C ABI.
 *
 * The operation (paper Section 3.5 "Preserving RL and MoE semantics without expansion", paragraphs
 * "Compact-to-semantic log-probability computation" and "Gradient accumulation for reused compact
 * logits", Eqs. 17 and 19): the language-model head produces one logit row z_c in R^V per COMPACT token.
 * Every non-terminal semantic position s (a token occurrence of one trajectory, in original batch order)
 * reuses the row m(s) and has its own target y_s, the next token of its trajectory.  Forward:
 *
 *     lse_c    = log sum_v exp z[c, v]                 once per compact row        (O(C V))
 *     lambda_s = z[m(s), y_s] - lse_{m(s)}             once per semantic position  (O(S))
 *
 * Backward, with g_s = dL/dlambda_s (exactly 0 where the action mask drops s):
 *
 *     dz[c, v] = sum_{s: m(s)=c} g_s * ([v == y_s] - exp(z[c, v] - lse_c))
 *
 * No S x V array is ever formed.  Contributions of positions sharing a row are summed in fp32 in the
 * order of the caller's CSR (deterministic), then rounded once to the logit dtype.
 *
 * Conventions are those of harts_la.h: int32 status returns (HARTS_OK / HARTS_E*), no allocation of
 * device memory by the library, kernels enqueued on the caller's stream (cudaStream_t as void*) without
 * synchronising, no CPU fallback.  z and dz are row-major [n_rows, ld] with ld >= V elements between rows
 * (HARTS_FP32 or HARTS_BF16); any V and any row alignment are accepted, rows whose start is 16-byte
 * aligned take the vector path.  Index arrays are int32.
 */
#ifndef HARTS_LOGP_H_
#define HARTS_LOGP_H_

#include <stddef.h>
#include <stdint.h>

#include "harts_la.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Semantic positions of a forest (the set P of Eq. 17) in original batch order: trajectory by trajectory
 * (trees in input order, inside a tree by leaf node index; a node's end is a trajectory end unless a child
 * forks exactly there), positions inside a trajectory in token order, the last token of each trajectory left out.
 *   tree_node_ptr, node_parent, node_fork_off, node_len: host, as for harts_la_plan()
 *   row_of_token [C] host or NULL: canonical token index -> row of z (a plan's row_of_token); NULL = identity
 *   token_id     [C] host: vocabulary id of every compact token, canonical order
 *   cap: capacity of m and y (entries).  m, y may be NULL to query the sizes only.
 *   m [cap] host out: row of z that position s reuses;  y [cap] host out: its target id
 *   traj_pos_ptr [n_traj+1] host out or NULL: first position of each trajectory (sized by a first query call)
 *   *n_pos, *n_traj host out: |P| and the number of trajectories (always written)
 * Errors: HARTS_EINVAL for a malformed forest or cap < |P| with non-NULL m/y (nothing is written to m/y).
 */
int32_t harts_logp_positions(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                             const int32_t* node_fork_off, const int32_t* node_len, const int32_t* row_of_token,
                             const int32_t* token_id, int64_t cap, int32_t* m, int32_t* y, int64_t* traj_pos_ptr,
                             int64_t* n_pos, int64_t* n_traj);

/*
 * Multiplicity of every compact token (Section 3.5, Eq. 20: q_c = |{s : m(s) = c}|, terminal positions included):
 * the number of root-to-leaf trajectories that contain the token.  A loss or auxiliary statistic that the
 * trajectory-wise run would average over semantic positions is reproduced on compact rows by weighting row c with q_c.
 *   forest arrays, row_of_token: host, as for harts_logp_positions()
 *   n_rows: rows of the compact tensors (>= number of compact tokens);  mult [n_rows] host out (rows that hold no
 *   token get 0)
 * Errors: HARTS_EINVAL for a malformed forest, n_rows too small or a row_of_token entry outside [0, n_rows).
 */
int32_t harts_logp_multiplicity(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                                const int32_t* node_fork_off, const int32_t* node_len, const int32_t* row_of_token,
                                int64_t n_rows, int32_t* mult);

/*
 * Positions grouped by the row they reuse (the index set of the sum in Eq. 19), stable in position order.
 *   m [n_pos] host;  row_pos_ptr [n_rows+1] host out;  row_pos [n_pos] host out (position ids)
 * Errors: HARTS_EINVAL if some m[s] is outside [0, n_rows).
 */
int32_t harts_logp_csr(int32_t n_rows, int64_t n_pos, const int32_t* m, int32_t* row_pos_ptr, int32_t* row_pos);

/*
 * Forward (Eq. 17).  All pointers device.
 *   z [n_rows, ldz];  m, y [n_pos];  lse [n_rows] fp32 out;  lambda [n_pos] fp32 out
 *   dev_status: int32[2] device or NULL.  A position with m outside [0,n_rows) or y outside [0,V) is skipped
 *   (lambda = 0), and dev_status[0] = HARTS_EINVAL, dev_status[1] = the position; read it with harts_la_check().
 * One pass over z (n_rows * V elements read), n_pos gathers.
 */
int32_t harts_logp_fwd(const void* z, int32_t dtype, int32_t n_rows, int32_t V, int64_t ldz, int64_t n_pos,
                       const int32_t* m, const int32_t* y, float* lse, float* lambda, int32_t* dev_status,
                       void* stream);

/*
 * Backward (Eq. 19).  All pointers device.
 *   z, lse as in the forward;  y, g [n_pos] (g fp32);  row_pos_ptr [n_rows+1], row_pos [n_pos] from harts_logp_csr
 *   dz [n_rows, lddz] out, dtype of z; every element of the V columns is written (rows that no position with
 *   g != 0 reuses are zero-filled without reading z).  dz may not alias z.
 *   v_begin, V_total: for a vocabulary shard, z holds columns [v_begin, v_begin+V) of V_total; targets outside
 *   the shard add nothing here.  Pass 0 and V for the unsharded case.
 */
int32_t harts_logp_bwd(const void* z, int32_t dtype, int32_t n_rows, int32_t V, int64_t ldz, int64_t n_pos,
                       const int32_t* y, const int32_t* row_pos_ptr, const int32_t* row_pos, const float* lse,
                       const float* g, void* dz, int64_t lddz, int32_t v_begin, int32_t V_total,
                       int32_t* dev_status, void* stream);

/*
 * Vocabulary-parallel forward (same paragraph: ranks exchange only per-row maximum and sum-exp scalars and
 * one target-logit scalar per position, never logit rows).  One call per shard:
 *   z holds columns [v_begin, v_begin+V) of the vocabulary.
 *   row_max [n_rows], row_sum [n_rows] fp32 out: max_v z and sum_v exp(z - max) over the shard's columns
 *   target  [n_pos] fp32 out: z[m(s), y_s - v_begin] if the target lies in this shard, else 0
 */
int32_t harts_logp_fwd_shard(const void* z, int32_t dtype, int32_t n_rows, int32_t V, int64_t ldz, int32_t v_begin,
                             int64_t n_pos, const int32_t* m, const int32_t* y, float* row_max, float* row_sum,
                             float* target, int32_t* dev_status, void* stream);

/*
 * Combine the shard scalars (after an all-gather of them, or on one GPU that ran all shards):
 *   row_max, row_sum [n_shards, n_rows], target [n_shards, n_pos] device, shard-major
 *   lse [n_rows], lambda [n_pos] out:  lse = M + log sum_k row_sum_k exp(row_max_k - M), M = max_k row_max_k;
 *   lambda_s = sum_k target_k[s] - lse[m(s)]
 */
int32_t harts_logp_combine(int32_t n_shards, int32_t n_rows, int64_t n_pos, const int32_t* m, const float* row_max,
                           const float* row_sum, const float* target, float* lse, float* lambda, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HARTS_LOGP_H_ */
