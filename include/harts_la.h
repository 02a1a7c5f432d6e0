/*
 * harts_la -- tree-packed chunkwise linear attention for sm_100a (B200): C ABI.
 *
 * The operation (paper Section 3.3 "Minimum-Call Planning", Section 3.4 "Differentiable
 * boundary states" / "Round-wise execution", Eq. 16): a forest of rollout trees is turned into
 * compact token rows (each shared-prefix token stored once), grouped into the minimum number of
 * sequential packed calls ("rounds", Algorithm 1).  Every sequence of a round starts from a zero
 * state or from a chunk-boundary state that an earlier round exported ("slot"), replays the
 * fewer-than-one-chunk ancestor interval between that boundary and its fork (Eq. 2), and then
 * runs its own rows.  Gradients flow back through the state hand-off and through the replayed
 * rows.  The recurrence is Eq. 1 specialised to a scalar gate:
 *
 *     S_t = exp(g_t) S_{t-1} + k_t^T v_t,     o_t = q_t S_t        (per head, S in R^{dk x dv})
 *
 * Conventions
 *   - Every function returns an int32 status: HARTS_OK or a negative HARTS_E* code.  Nothing
 *     throws, aborts or prints.  harts_la_strerror() gives text.
 *   - The library allocates NO device memory.  Tensors, slots, workspaces and the uploaded index
 *     tables are caller-owned device buffers; their sizes come from the query calls.
 *   - "host" / "device" in a comment says where the pointer must point.
 *   - Kernels are enqueued on the caller's stream (a cudaStream_t passed as void*) and the calls
 *     return without synchronising.  Device-detected errors (a bounded wait that ran out) are
 *     written to a caller-owned device status word and read back by harts_la_check().  After a time-out the
 *     outputs of that call are undefined; zero the status word before reusing it.
 *   - There is no CPU fallback: an unsupported (dtype, dk, dv, chunk) gives HARTS_EUNSUPPORTED.
 *   - Tensor layout: row-major [rows, H, d] with physical compact rows outermost (plan order,
 *     see row_of_token), heads next, the feature dimension contiguous.  Base pointers must be
 *     16-byte aligned.  g and dg are fp32 [rows, H]; g is the log-decay (<= 0) itself.
 */
#ifndef HARTS_LA_H_
#define HARTS_LA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HARTS_OK 0
#define HARTS_EINVAL (-1)        /* bad argument: null/misaligned pointer, malformed tree, bad size */
#define HARTS_ENOMEM (-2)        /* host allocation failed */
#define HARTS_EUNSUPPORTED (-3)  /* no kernel for this (dtype, dk, dv, chunk) */
#define HARTS_ETIMEOUT (-4)      /* a bounded device-side wait ran out (from harts_la_check) */
#define HARTS_EINTERNAL (-5)
#define HARTS_ECUDA (-6)         /* a CUDA runtime/driver call failed */
#define HARTS_ESCRATCH (-7)      /* the problem needs more scratch than the library's fixed scratch array holds */

#define HARTS_FP32 0
#define HARTS_BF16 1

/* flags */
#define HARTS_FLAG_FMA_KERNELS 1u /* use the fp32 CUDA-core (non tensor-core) kernels also for bf16 inputs */
/* Debug check for hand-built tables (harts_la_fwd_seqs / harts_la_bwd_seqs): before the kernels of the call a small
 * validation kernel checks every index they would follow (CSR pointers monotone and in range, rows < n_rows, slots <
 * n_slots, replay shorter than a chunk, chunk counts consistent, consumer and replay-gradient tables in range).  On a
 * bad entry the status word becomes HARTS_EINVAL (dev_status[1] = which table, 1-based in the order of
 * harts_la_tables_t; dev_status[2] = position), the kernels of this and of later calls with the flag return without
 * reading or writing anything, and harts_la_check() reports HARTS_EINVAL.  Needs dev_status (at least 4 int32). */
#define HARTS_FLAG_CHECK_TABLES 2u
/* harts_la_fwd / harts_la_bwd with round 0 run ALL rounds in one launch per pass when the problem has few (sequence,
 * head) work items per persistent CTA (bf16, dk = dv = 128, at most 32 rounds): the CTAs draw the items from a ticket
 * counter in round order, and a sequence waits for the flag of the boundary state it starts from (backward: for the
 * initial-state gradients of the sequences that started at a boundary) instead of for the end of the previous round's
 * kernel, so the rounds overlap as far as the tree allows.  Same arithmetic, same bits.  With this flag every round
 * gets its own launch, as with explicit round numbers. */
#define HARTS_FLAG_ROUND_LAUNCHES 16u

typedef struct harts_la_plan harts_la_plan_t; /* opaque, host memory, library-owned */

/*
 * Host view of a plan.  All pointers are const HOST arrays owned by the plan.
 * Sequences are numbered globally in execution order: round-major, inside a round by the
 * canonical index of their first own token (canonical = tree, node, offset order of the input).
 * Physical rows follow the same order, the own rows of a sequence are contiguous, no padding rows.
 */
typedef struct harts_la_plan_view {
    int32_t chunk;            /* B of Section 2.2 */
    int32_t n_rounds;         /* minimum number of sequential packed calls (T_pre(root), max over trees) */
    int32_t n_rows;           /* C: compact token rows */
    int32_t n_replay;         /* R of Eq. 15 */
    int32_t n_seq;
    int32_t n_slots;          /* requested chunk-boundary states */
    int32_t n_chunks;         /* sum over sequences of ceil((replay + own) / chunk) */
    int32_t n_rg_rows;        /* compact rows that are replayed by at least one sequence */
    const int32_t* row_of_token;   /* [n_rows]   canonical token index -> physical row */
    const int32_t* round_seq_ptr;  /* [n_rounds+1] sequences of round r are [ptr[r], ptr[r+1]) */
    const int32_t* seq_tree;       /* [n_seq] */
    const int32_t* seq_own_begin;  /* [n_seq+1] first physical row of the own rows (cu_seqlens; last = n_rows) */
    const int32_t* seq_own_len;    /* [n_seq] */
    const int32_t* seq_start_pos;  /* [n_seq] absolute position of the start anchor (multiple of chunk) */
    const int32_t* seq_init_slot;  /* [n_seq] slot holding the initial state, -1 = zero state */
    const int32_t* seq_replay_ptr; /* [n_seq+1] CSR into replay_row */
    const int32_t* replay_row;     /* [n_replay] physical rows replayed before the own rows, path order */
    const int32_t* seq_req_ptr;    /* [n_seq+1] slots [ptr[i], ptr[i+1]) are produced by sequence i */
    const int32_t* slot_chunk;     /* [n_slots] chunk index (>= 1) whose start state goes to the slot */
    const int32_t* seq_chunk_ptr;  /* [n_seq+1] CSR of chunk counts (addresses the chunk-state workspace) */
    const int32_t* slot_cons_ptr;  /* [n_slots+1] CSR: sequences whose initial state is that slot */
    const int32_t* slot_cons_seq;
    const int32_t* rg_row;         /* [n_rg_rows] replayed physical rows, ascending */
    const int32_t* rg_ptr;         /* [n_rg_rows+1] CSR into rg_entry */
    const int32_t* rg_entry;       /* [n_replay] indices into replay_row whose gradients land on rg_row */
    const int32_t* seq_order;      /* [n_seq] per round, its sequences sorted by decreasing chunk count: the order in
                                      which the kernels pick up work (longest first); a scheduling hint only */
} harts_la_plan_view_t;

/*
 * Device-side index tables for one problem (all DEVICE pointers, int32, same meaning as in the
 * view).  harts_la_plan_tables() fills it from an uploaded plan; a caller that wants to drive the
 * per-call contract of Eq. 16 without the planner fills it by hand.
 */
typedef struct harts_la_tables {
    int32_t chunk, n_rows, n_replay, n_seq, n_slots, n_chunks, n_rg_rows;
    const int32_t* seq_own_begin;
    const int32_t* seq_init_slot;
    const int32_t* seq_replay_ptr;
    const int32_t* replay_row;
    const int32_t* seq_req_ptr;
    const int32_t* slot_chunk;
    const int32_t* seq_chunk_ptr;
    const int32_t* slot_cons_ptr;
    const int32_t* slot_cons_seq;
    const int32_t* rg_row;
    const int32_t* rg_ptr;
    const int32_t* rg_entry;
    const int32_t* seq_order;      /* may be NULL: sequences are then processed in index order.  When set, a call's
                                      range [seq_lo, seq_hi) must be one over which seq_order is a permutation of
                                      itself (the planner's table is one per whole round): the tensor-core kernels
                                      take sequence seq_order[seq_lo + i] as their i-th work item, so a sub-range of
                                      a round needs seq_order = NULL */
} harts_la_tables_t;

const char* harts_la_strerror(int32_t code);

/*
 * Minimum-call planning (Section 3.3, Algorithm 1, Eqs. 11-15) plus the compact physical
 * ordering of Section 4.2.  O(nodes + tokens) time.
 *   tree_node_ptr [n_trees+1] host: CSR into the node arrays
 *   node_parent   [n_nodes]   host: tree-local parent index (< own index), -1 for a root (node 0 of a tree)
 *   node_fork_off [n_nodes]   host: offset inside the parent at which the node forks, 1..len(parent); 0 for roots
 *   node_len      [n_nodes]   host: tokens in the node, >= 1
 *   chunk: B.  *out is created by the library; free it with harts_la_plan_free().
 * Errors: HARTS_EINVAL for a malformed forest (nothing is created), HARTS_ENOMEM.
 */
int32_t harts_la_plan(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                      const int32_t* node_fork_off, const int32_t* node_len, int32_t chunk,
                      harts_la_plan_t** out);
void harts_la_plan_free(harts_la_plan_t* plan);
int32_t harts_la_plan_view(const harts_la_plan_t* plan, harts_la_plan_view_t* out);

/* Size of the flat index blob, upload of it (one cudaMemcpyAsync on `stream`; dev_blob is a
 * caller-owned DEVICE buffer of that size, 16-byte aligned), and the table of device pointers
 * into an uploaded blob (pure pointer arithmetic, no CUDA call). */
int32_t harts_la_plan_device_bytes(const harts_la_plan_t* plan, size_t* bytes);
int32_t harts_la_plan_upload(const harts_la_plan_t* plan, void* dev_blob, void* stream);
int32_t harts_la_plan_tables(const harts_la_plan_t* plan, const void* dev_blob, harts_la_tables_t* out);

/*
 * Workspace sizes (Section 3.4 "Full-layer activation recomputation": the forward keeps only
 * chunk-boundary states, the backward recomputes everything inside a chunk from them).
 *   chunk_state_bytes: [n_chunks, H, dk, dv] start-of-chunk states in the run dtype, written by the
 *                      forward, read by the backward, followed by (n_slots + n_seq) * H int32 flags that the
 *                      one-launch forms of round 0 use (the library clears them itself).
 *   scratch_bytes:     backward scratch: per-sequence initial-state gradients [n_seq, H, dk, dv] fp32
 *                      and replay-row gradients [n_replay, H, dk + dv + 1] fp32.
 */
int32_t harts_la_workspace_bytes(const harts_la_tables_t* tables, int32_t H, int32_t dk, int32_t dv,
                                 int32_t dtype, uint32_t flags, size_t* chunk_state_bytes,
                                 size_t* scratch_bytes);

/*
 * One packed call of Eq. 16 over sequences [seq_lo, seq_hi) (one round).  All tensors DEVICE.
 *   q,k [n_rows,H,dk], v [n_rows,H,dv] in `dtype`; g [n_rows,H] fp32.  Never modified.
 *   o   [n_rows,H,dv]: the own rows of the issued sequences are written exactly once; replay rows
 *       produce no output (Section 3.4 "Round-wise execution").
 *   slots [n_slots,H,dk,dv] fp32: read as initial states (seq_init_slot), written for the requested
 *       boundaries of the issued sequences (no second state scan).  A slot read by this call must have
 *       been written by an earlier call on the same stream.
 *   chunk_states: workspace above (may be NULL: then no backward is possible).
 * Errors: HARTS_EINVAL (null/misaligned pointers, bad range), HARTS_EUNSUPPORTED, HARTS_ECUDA.
 */
int32_t harts_la_fwd_seqs(const harts_la_tables_t* tables, int32_t seq_lo, int32_t seq_hi, const void* q,
                          const void* k, const void* v, const float* g, void* o, float* slots,
                          void* chunk_states, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                          uint32_t flags, int32_t* dev_status, void* stream);

/*
 * Backward of the same call.  Calls must be issued in the reverse order of the forward calls, on
 * one stream: a sequence reads the initial-state gradients of the consumers of its slots
 * (Section 3.4: several consumers of one boundary are summed) from `scratch`, where those
 * consumers' calls left them.
 *   dO [n_rows,H,dv]; dq,dk_ [n_rows,H,dk], dv_ [n_rows,H,dv] in `dtype`; dg [n_rows,H] fp32: own rows
 *   of the issued sequences are overwritten.  Gradients of replayed rows go to `scratch` and are
 *   folded into their ancestor rows by harts_la_bwd_finish().
 */
int32_t harts_la_bwd_seqs(const harts_la_tables_t* tables, int32_t seq_lo, int32_t seq_hi, const void* q,
                          const void* k, const void* v, const float* g, const void* dO, void* dq, void* dk_,
                          void* dv_, float* dg, const void* chunk_states, void* scratch, int32_t H,
                          int32_t dk, int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status,
                          void* stream);

/* Adds the replay-row gradients (Section 4.2: the gather's backward sums every consumer into the
 * unique producer row) into dk_, dv_, dg.  Call once, after the backward of the first round. */
int32_t harts_la_bwd_finish(const harts_la_tables_t* tables, void* dk_, void* dv_, float* dg,
                            const void* scratch, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                            void* stream);

/*
 * Plan-driven wrappers: round r in 1..n_rounds issues that round's packed call; round 0 issues all
 * rounds in order (forward: 1..K; backward: K..1 followed by harts_la_bwd_finish).  With explicit
 * rounds the backward of round 1 also runs harts_la_bwd_finish.  dev_blob is the uploaded blob.
 */
int32_t harts_la_fwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q,
                     const void* k, const void* v, const float* g, void* o, float* slots, void* chunk_states,
                     int32_t H, int32_t dk, int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status,
                     void* stream);
int32_t harts_la_bwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q,
                     const void* k, const void* v, const float* g, const void* dO, void* dq, void* dk_,
                     void* dv_, float* dg, const void* chunk_states, void* scratch, int32_t H, int32_t dk,
                     int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream);

/*
 * One whole step on HOST buffers (the end-to-end form of Eq. 16's round loop): copies q, k, v, g, dO (physical row
 * order, layouts as above) from host memory into the caller's device tensors, runs every forward round and every
 * backward round with the replay-gradient fold, and copies o, dq, dk, dv, dg back -- all enqueued on `stream`, in
 * that order, without synchronising (the host results are complete once the stream has drained; use pinned host
 * memory for the copies to be asynchronous).  host_*: HOST pointers; dev_*, slots, chunk_states, scratch: caller-owned
 * DEVICE buffers of the sizes harts_la_fwd / harts_la_bwd expect (the library allocates nothing).
 * Errors: HARTS_EINVAL (a missing buffer), HARTS_ECUDA (a copy could not be enqueued), those of harts_la_fwd / _bwd.
 */
int32_t harts_la_step_host(const harts_la_plan_t* plan, const void* dev_blob, const void* host_q, const void* host_k,
                           const void* host_v, const float* host_g, const void* host_dO, void* host_o, void* host_dq,
                           void* host_dk, void* host_dv, float* host_dg, void* dev_q, void* dev_k, void* dev_v,
                           float* dev_g, void* dev_dO, void* dev_o, void* dev_dq, void* dev_dk, void* dev_dv,
                           float* dev_dg, float* slots, void* chunk_states, void* scratch, int32_t H, int32_t dk,
                           int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream);

/*
 * The same path for the recurrence with a PER-CHANNEL decay, the first term of Eq. 1 (Section 2.2, the Diag(gamma)
 * decay on the key dimension of the state; Section 4.1 names a backend of this family as the one evaluated):
 *
 *     S_t = Diag(exp(g_t)) S_{t-1} + k_t^T v_t,     o_t = q_t S_t,       g_t in R^{dk}, g_t <= 0
 *
 * (the scalar gate above is its special case with all channels equal; the delta-rule part of Eq. 1, U - W S, is not
 * defined by the paper and is not provided).  Plan, uploaded tables, slots, replay rows, chunk states and the
 * hand-off of initial-state gradients are exactly those of harts_la_fwd / harts_la_bwd; only
 *   gk  [n_rows, H, dk] fp32 DEVICE: the per-channel log-decay (never modified), and
 *   dgk [n_rows, H, dk] fp32 DEVICE: its gradient (own rows overwritten; replayed rows folded in by the round-1 call)
 * replace g and dg, and the backward scratch is larger (harts_la_gk_workspace_bytes: the replay-row gradient of g is
 * a vector; its chunk-state figure includes the flags of the one-launch forms).  Rounds as for harts_la_fwd /
 * harts_la_bwd (0 = all; on the tensor-core path in one launch per pass under the same conditions).  Served: fp32 with dk = dv = 64, bf16 with
 * dk = dv = 64 or 128, chunk 64.  bf16 with dk = dv = 128 runs its dense products on the tensor cores (bf16
 * operands, fp32 accumulation; decayed operands, scores and chunk states rounded to bf16); everything else, and that
 * shape too under HARTS_FLAG_FMA_KERNELS, runs in fp32 on the CUDA cores.  Every decay factor is exp of a
 * difference of running sums that is <= 0 for g <= 0: exp(b_t[i] - b_j[i]) with j <= t directly, or, on the
 * tensor-core path for t and j in different 16-row blocks of a chunk, exp(b_t[i] - a[i]) exp(a[i] - b_j[i]) with a the
 * running sum at the first row of t's block (and for t, j in the same block too, while no channel of the chunk decays by
 * more than 2^100 over a block, which bounds exp(a[i] - b_j[i])) -- so no gate value g <= 0 can overflow.  Errors as for harts_la_fwd /
 * harts_la_bwd.
 */
int32_t harts_la_gk_workspace_bytes(const harts_la_tables_t* tables, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                                    size_t* chunk_state_bytes, size_t* scratch_bytes);
int32_t harts_la_gk_fwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q, const void* k,
                        const void* v, const float* gk, void* o, float* slots, void* chunk_states, int32_t H, int32_t dk,
                        int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream);
int32_t harts_la_gk_bwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q, const void* k,
                        const void* v, const float* gk, const void* dO, void* dq, void* dk_, void* dv_, float* dgk,
                        const void* chunk_states, void* scratch, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                        uint32_t flags, int32_t* dev_status, void* stream);

/*
 * (No counterpart in the paper: an addition for a kind of caller, not part of the method.)
 * Backward of ALL rounds followed by the replay-gradient fold, like harts_la_bwd(plan, blob, 0, ...), but with the
 * scratch area inside the library instead of in a caller-owned buffer.  It is meant for callers that have no way to
 * get device memory at the point where they run the backward: code that runs inside a step whose device memory was
 * handed out in full beforehand (a framework's arena, a fixed-size serving budget), where one more allocation would
 * either fail or stall the device, and plug-in style callers that are given tensors but no allocator.  This call
 * allocates nothing -- no cudaMalloc, cudaFree or allocating library routine -- and the caller still passes every
 * input and output tensor and the chunk-state workspace the forward filled.
 *   - The scratch is a fixed device array of HARTS_STATIC_SCRATCH_BYTES that every GPU which loads the library
 *     holds until the process ends.  A problem whose scratch need (harts_la_workspace_bytes) is larger is rejected
 *     with HARTS_ESCRATCH before anything is launched.
 *   - The first call on a device looks up the array's device address (one runtime query, result kept per device);
 *     make that first call with the device current and before any stream capture begins.  With CUDA's lazy module
 *     loading that query is also the moment the driver sets the array up on the device, so make the first call while
 *     the device still has HARTS_STATIC_SCRATCH_BYTES to spare: HARTS_ECUDA from a first call can mean exactly that
 *     the device had no room left for it.  Later calls touch no allocator at all.
 *   - All calls on a device share the one array, and it keeps whatever the last call left in it.  The backward
 *     writes every scratch entry before it reads it, so nothing needs clearing; but two calls that overlap on the
 *     GPU (different streams, or another host thread) race on the array and corrupt each other's gradients.
 * Arguments, layouts and the other error codes are those of harts_la_bwd.
 */
#define HARTS_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
int32_t harts_la_bwd_static(const harts_la_plan_t* plan, const void* dev_blob, const void* q, const void* k,
                            const void* v, const float* g, const void* dO, void* dq, void* dk_, void* dv_, float* dg,
                            const void* chunk_states, int32_t H, int32_t dk, int32_t dv, int32_t dtype, uint32_t flags,
                            int32_t* dev_status, void* stream);

/*
 * Trajectory-wise view of a forest (host; the conventional execution the paper compares with in Section 5): every
 * root-to-leaf trajectory as a sequence of its own, with the semantic map m of Eq. 3 -- for every position of every
 * trajectory the canonical index (tree, node, offset order of the input) of the compact token it shares.  A
 * trajectory ends in every node that no child continues from its last token; trajectories are listed by tree, then
 * by the index of that node.  Running harts_la_plan on single-node trees of the returned lengths, with inputs
 * gathered through src_token, is the trajectory-wise run of the same kernels.
 *   traj_len  [cap_traj]   host, out: tokens of every trajectory
 *   src_token [cap_tokens] host, out: canonical compact token of every expanded position, trajectories back to back
 * Pass both arrays NULL to get *n_traj and *n_tokens only.  Errors: HARTS_EINVAL (malformed forest, capacity).
 */
int32_t harts_la_expand(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                        const int32_t* node_fork_off, const int32_t* node_len, int64_t cap_traj, int64_t cap_tokens,
                        int32_t* traj_len, int64_t* src_token, int64_t* n_traj, int64_t* n_tokens);

/* Synchronises `stream`, reads the device status word and returns HARTS_OK, HARTS_ETIMEOUT,
 * HARTS_EINVAL (an out-of-range index met by a harts_logp_* kernel, see harts_logp.h) or HARTS_ECUDA.  dev_status must be zeroed by the caller before the first launch. */
int32_t harts_la_check(const int32_t* dev_status, void* stream);

/*
 * Self-test of the failure path of the device-side waits (every wait on an mbarrier in the kernels of this library is
 * bounded: about half a second of wall time, after which the CTA records HARTS_ETIMEOUT in the status word, stops
 * waiting anywhere else, leaves its loops, lets its copies and MMAs in flight finish, frees its tensor memory and
 * returns).  This call launches one small CTA that waits, with a limit of one millisecond, on a barrier nothing arrives
 * at.  Afterwards harts_la_check(dev_status) gives HARTS_ETIMEOUT and the context stays usable.
 *   dev_status  DEVICE int32 status word (zeroed by the caller)
 *   dev_report  DEVICE int32[8] or NULL: {first wait succeeded (0 expected), second wait succeeded (0), microseconds
 *               in the first wait (about 1000), microseconds in the second (about 0: the latch was set), CTA saw the
 *               latch (1), then for the flag wait of the one-launch forms (a flag nobody sets; first with a limit of
 *               one millisecond, then with the status word already set): bits {1: first succeeded, 2: second
 *               succeeded, 4: first latched, 8: second latched} (12 expected), microseconds in the first (about 1000),
 *               microseconds in the second (about 0: a set status word ends a flag wait)}
 */
int32_t harts_la_selftest_timeout(int32_t* dev_status, int32_t* dev_report, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HARTS_LA_H_ */
