/*
 * harts_attn -- full (softmax) attention on compact tokens of rollout trees for sm_100a (B200): C ABI.
 *
 * The operation (paper Section 3.4 "Full attention on compact tokens"; Section 4.2 "MLA execution with asymmetric
 * packed Q/KV views", Eqs. 21-22): every compact token has ONE query and attends to the keys/values of its true
 * ancestors in the tree and of itself.  For a branch with h ancestor tokens and l own tokens this is the packed
 * view of Eq. 21 (l queries, h + l keys) with the bottom-right causal alignment of Eq. 22 (query i sees key j iff
 * j <= h + i).  Per query head (GQA: kv head = query head / (Hq / Hkv)):
 *
 *     o_t = sum_{s in path(t)} softmax_s(scale * q_t . k_s) v_s
 *
 * The paper gathers each branch's ancestor K/V into a temporary packed view and calls a packed-attention backend;
 * the gather's backward scatter-adds into the shared ancestors.  Here no view is materialised: the kernels walk an
 * index of the tree ("pieces": runs of rows that are contiguous both in memory and on the trajectory, with no
 * fork inside) and read ancestor K/V tiles straight from the compact rows; in the backward one CTA owns a K/V
 * tile and visits every query tile that sees it (own branch and all descendants), so dk/dv of a shared ancestor
 * are accumulated on chip and written once -- no scatter-add, no atomics, deterministic.
 *
 * Conventions are those of harts_la.h.  q, o, dO, dq: [n_rows, Hq, 128]; k, v, dk, dv: [n_rows, Hkv, 128];
 * HARTS_BF16 only, head dimension 128, physical compact rows (the plan's order), 16-byte aligned.
 * lse: fp32 [n_rows, Hq], natural-log units of the scaled scores.
 */
#ifndef HARTS_ATTN_H_
#define HARTS_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#include "harts_la.h"

#ifdef __cplusplus
extern "C" {
#endif

#define HARTS_ATTN_HEADER_WORDS 24

/*
 * Index of a forest for the attention kernels, one int32 blob.  Host in, host out.
 *   tree_node_ptr, node_parent, node_fork_off, node_len: as for harts_la_plan()
 *   row_of_token [C] or NULL (identity): canonical token index -> physical row
 *   cap_words: capacity of blob in int32 words; blob may be NULL to query the size only
 *   *n_words out: size of the index in words (always written)
 * Blob layout: HARTS_ATTN_HEADER_WORDS header words
 *     [0] n_rows  [1] n_pieces  [2] n_anc_runs  [3] n_desc  [4] n_q_items  [5] n_kv_items  [6] total words
 *     [8..] word offsets of the arrays, in this order:
 *   piece_row0 [P], piece_len [P], piece_parent [P]      pieces in physical-row order; parent = -1 for a root
 *   anc_ptr [P+1], anc_row0 [], anc_len []               ancestor rows of a piece, root first, adjacent pieces merged
 *   desc_ptr [P+1], desc_piece []                        all descendant pieces of a piece, in piece order
 *   q_item [2 * n_q_items]   (piece, tile of 128 query rows), most work first
 *   kv_item [2 * n_kv_items] (piece, tile of 128 key rows), most work first
 * The same blob is copied to the device unchanged (plain memcpy) for the kernel calls.
 * Errors: HARTS_EINVAL (malformed forest, bad row map, cap_words too small with non-NULL blob).
 */
int32_t harts_attn_index(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                         const int32_t* node_fork_off, const int32_t* node_len, const int32_t* row_of_token,
                         int64_t cap_words, int32_t* blob, int64_t* n_words);

/*
 * Forward.  host_index / dev_index: the blob on the host and its copy on the device.  Other pointers device.
 * Writes o and lse for every row.  dev_status: int32 device status word (bounded waits), read with harts_la_check().
 */
int32_t harts_attn_fwd(const int32_t* host_index, const int32_t* dev_index, const void* q, const void* k,
                       const void* v, void* o, float* lse, int32_t Hq, int32_t Hkv, int32_t d, float scale,
                       int32_t dtype, int32_t* dev_status, void* stream);

/*
 * Backward of L = sum_t <dO_t, o_t>.  o and lse are the forward's.  delta: fp32 [n_rows, Hq] scratch (rowsum(dO*o)),
 * overwritten.  Writes dq, dk, dv for every row.
 */
int32_t harts_attn_bwd(const int32_t* host_index, const int32_t* dev_index, const void* q, const void* k,
                       const void* v, const void* o, const float* lse, const void* dO, void* dq, void* dk_, void* dv_,
                       float* delta, int32_t Hq, int32_t Hkv, int32_t d, float scale, int32_t dtype,
                       int32_t* dev_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HARTS_ATTN_H_ */
