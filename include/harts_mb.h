/*
 * harts_mb -- prefix-aware microbatch planning and schedule construction: C ABI (host only).
 *
 * The operation (paper Section 3.2, Eqs. 4-10): the root-to-leaf trajectories of a batch of rollout trees are
 * grouped into K microbatches (K a multiple of the data-parallel degree D), each within a capacity of T compact
 * tokens, where the work of a microbatch is the number of unique token nodes of the trie that merges its
 * trajectories (Eq. 5); every microbatch gets a replica and a slot.  Candidate plans are ranked lexicographically by
 *     J = ( total compact work,  sum over slots of the heaviest microbatch,  heaviest replica )          (Eq. 4)
 * Candidates: the natural partition (recursive cuts at the lowest adjacent-LCP valley), for N <= 512 trajectories the
 * exact dynamic program over contiguous partitions (Eq. 9) for every K of Eq. 8, for N > 512 merge/split evolution
 * of the natural partition towards at most 32 sampled K, the best of eight trie-aware greedy placements (Eq. 10),
 * and local refinement (boundary moves, sparse repair) of the anchors the section names.  Guarantees of every
 * returned plan: exact coverage, non-empty microbatches within capacity, K mod D = 0, K / D microbatches per replica.
 *
 * Trajectories are numbered in "lexicographic" order, which for a forest given as trees is a depth-first order:
 * trees in input order; inside a node, fork points by ascending offset, the children of one fork point in input
 * order, the node's own continuation last.  A node's end is a trajectory end unless a child forks exactly there.
 * Everything is host memory; int32 status codes as in harts_la.h.
 */
#ifndef HARTS_MB_H_
#define HARTS_MB_H_

#include <stddef.h>
#include <stdint.h>

#include "harts_la.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct harts_mb_plan harts_mb_plan_t; /* opaque, host memory, library-owned */

/* which generator produced the selected plan */
#define HARTS_MB_NATURAL 0
#define HARTS_MB_EXACT 1      /* contiguous dynamic program, Eq. 9 */
#define HARTS_MB_EVOLVED 2    /* merge/split evolution of the natural partition */
#define HARTS_MB_GREEDY 3     /* trie-aware greedy placement, Eq. 10 */

typedef struct harts_mb_view {
    int32_t n_traj;            /* N */
    int32_t n_mb;              /* K */
    int32_t D;
    int32_t source;            /* HARTS_MB_* of the selected plan */
    int32_t refined;           /* 1 if local refinement changed the selected plan */
    int32_t natural_mb;        /* K_0 */
    int32_t n_candidates;      /* valid candidates compared under Eq. 4 */
    int32_t reserved;
    int64_t T;
    int64_t J[3];              /* Eq. 4 of the selected plan */
    int64_t total_work_all;    /* G = C(X): all trajectories in one trie */
    int64_t natural_work;      /* total work of the natural partition */
    const int32_t* traj_leaf;  /* [N] global node index of the node the trajectory ends in */
    const int32_t* traj_len;   /* [N] tokens */
    const int32_t* traj_lcp;   /* [N] LCP with the previous trajectory in this order (0 for the first) */
    const int32_t* traj_mb;    /* [N] microbatch of the trajectory */
    const int64_t* mb_work;    /* [K] compact tokens */
    const int32_t* mb_replica; /* [K] 0..D-1 */
    const int32_t* mb_slot;    /* [K] 0..K/D-1 */
} harts_mb_view_t;

/*
 * Plans the microbatches of a forest.  Forest arrays as for harts_la_plan().  D >= 1, T >= 1.
 * Errors: HARTS_EINVAL (malformed forest, a trajectory longer than T, fewer trajectories than D), HARTS_ENOMEM.
 */
int32_t harts_mb_plan(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                      const int32_t* node_fork_off, const int32_t* node_len, int32_t D, int64_t T,
                      harts_mb_plan_t** out);
void harts_mb_plan_free(harts_mb_plan_t* plan);
int32_t harts_mb_plan_view(const harts_mb_plan_t* plan, harts_mb_view_t* out);

/*
 * The compact forest of one microbatch, ready for harts_la_plan(): the union of its trajectories' paths, every node
 * cut to the extent some trajectory of the microbatch uses.
 *   cap_trees, cap_nodes: capacities of the output arrays (tree_node_ptr needs cap_trees + 1 entries)
 *   node_src [cap_nodes] or NULL: global index of the source node of every output node
 * Call with NULL arrays to get *n_trees and *n_nodes only.  Errors: HARTS_EINVAL (bad index, capacity too small).
 */
int32_t harts_mb_extract(const harts_mb_plan_t* plan, int32_t mb, int32_t cap_trees, int32_t cap_nodes,
                         int32_t* tree_node_ptr, int32_t* node_parent, int32_t* node_fork_off, int32_t* node_len,
                         int32_t* node_src, int32_t* n_trees, int32_t* n_nodes);

/*
 * The placement pass of the trie-aware greedy (Section 3.2 "Scale-independent trie-aware greedy", Eq. 10) on the
 * trajectories of `plan`, step by step, as a record that can be checked against the definition of the compact-work
 * increase: step i placed trajectory step_traj[i] (index in the plan's lexicographic order) into microbatch
 * step_mb[i] (numbered in creation order; step_created[i] = 1 when it was opened for this trajectory) and claimed
 * the work increase step_delta[i].
 *   order  0 ascending lexicographic, 1 descending, 2 descending length, 3 descending unique-suffix score
 *   policy 0 best-fit (largest work after insertion), 1 max-shared (largest |x| - delta); ties: earliest microbatch
 *   cap    capacity of the four HOST output arrays; pass NULL arrays to get *n_steps (= number of trajectories) only
 * The capacity T is the plan's.  Errors: HARTS_EINVAL.
 */
int32_t harts_mb_greedy_trace(const harts_mb_plan_t* plan, int32_t order, int32_t policy, int32_t cap,
                              int32_t* step_traj, int32_t* step_mb, int32_t* step_created, int64_t* step_delta,
                              int32_t* n_steps);

#ifdef __cplusplus
}
#endif
#endif /* HARTS_MB_H_ */
