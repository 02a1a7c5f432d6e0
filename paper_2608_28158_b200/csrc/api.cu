// C ABI: argument checks, kernel selection and launches.  No device memory is allocated here.
#include "kernels.h"
#include "plan.h"

namespace {

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

int32_t check_common(const harts_la_tables_t* tb, int32_t seq_lo, int32_t seq_hi, int32_t H, int32_t dk, int32_t dv,
                     int32_t dtype) {
    if (!tb) return HARTS_EINVAL;
    if (seq_lo < 0 || seq_hi < seq_lo || seq_hi > tb->n_seq) return HARTS_EINVAL;
    if (H < 1 || dk < 1 || dv < 1) return HARTS_EINVAL;
    if (dtype != HARTS_FP32 && dtype != HARTS_BF16) return HARTS_EUNSUPPORTED;
    if (tb->chunk != 64) return HARTS_EUNSUPPORTED;
    if (!harts::fma_supported(dtype, dk, dv)) return HARTS_EUNSUPPORTED;
    if (!tb->seq_own_begin || !tb->seq_init_slot || !tb->seq_replay_ptr || !tb->replay_row || !tb->seq_req_ptr ||
        !tb->slot_chunk || !tb->seq_chunk_ptr || !tb->slot_cons_ptr || !tb->slot_cons_seq || !tb->rg_row ||
        !tb->rg_ptr || !tb->rg_entry)
        return HARTS_EINVAL;
    return HARTS_OK;
}

// The tensor-core kernels serve bf16 with d_k = d_v = 128 unless the caller asks for the FMA kernels.
inline bool use_tc(int32_t dtype, int32_t dk, int32_t dv, uint32_t flags) {
    return !(flags & HARTS_FLAG_FMA_KERNELS) && harts::tc_supported(dtype, dk, dv);
}

}  // namespace

extern "C" {

const char* harts_la_strerror(int32_t code) {
    switch (code) {
        case HARTS_OK: return "ok";
        case HARTS_EINVAL: return "invalid argument";
        case HARTS_ENOMEM: return "out of host memory";
        case HARTS_EUNSUPPORTED: return "unsupported dtype / head dimension / chunk size";
        case HARTS_ETIMEOUT: return "a bounded device-side wait ran out";
        case HARTS_EINTERNAL: return "internal error";
        case HARTS_ECUDA: return "CUDA call failed";
        case HARTS_ESCRATCH: return "scratch need exceeds the library's fixed scratch array";
        default: return "unknown status";
    }
}

int32_t harts_la_plan_upload(const harts_la_plan_t* plan, void* dev_blob, void* stream) {
    const harts::Plan* p = harts_la_plan_internal(plan);
    if (!p || !dev_blob || misaligned(dev_blob)) return HARTS_EINVAL;
    cudaError_t e = cudaMemcpyAsync(dev_blob, p->blob.data(), p->blob.size() * sizeof(int32_t), cudaMemcpyHostToDevice,
                                    static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

int32_t harts_la_workspace_bytes(const harts_la_tables_t* tb, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                                 uint32_t /*flags*/, size_t* chunk_state_bytes, size_t* scratch_bytes) {
    if (!tb || H < 1 || dk < 1 || dv < 1) return HARTS_EINVAL;
    if (dtype != HARTS_FP32 && dtype != HARTS_BF16) return HARTS_EUNSUPPORTED;
    size_t elem = dtype == HARTS_FP32 ? 4 : 2;
    if (chunk_state_bytes)      // the states, then the flags of the one-launch forms
        *chunk_state_bytes = harts::chunk_state_payload(*tb, H, dk, dv, elem) + harts::fused_flag_bytes(*tb, H);
    if (scratch_bytes) *scratch_bytes = harts::scratch_layout(*tb, H, dk, dv).total;
    return HARTS_OK;
}

int32_t harts_la_fwd_seqs(const harts_la_tables_t* tb, int32_t seq_lo, int32_t seq_hi, const void* q, const void* k,
                          const void* v, const float* g, void* o, float* slots, void* chunk_states, int32_t H,
                          int32_t dk, int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream) {
    int32_t rc = check_common(tb, seq_lo, seq_hi, H, dk, dv, dtype);
    if (rc != HARTS_OK) return rc;
    if (!q || !k || !v || !g || !o || (tb->n_slots > 0 && !slots)) return HARTS_EINVAL;
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(g) || misaligned(o) || misaligned(slots) ||
        misaligned(chunk_states))
        return HARTS_EINVAL;
    harts::FwdArgs a{*tb, seq_lo, seq_hi, q, k, v, g, o, slots, chunk_states, H, dk, dv, dtype, flags, dev_status,
                     static_cast<cudaStream_t>(stream)};
    if (flags & HARTS_FLAG_CHECK_TABLES)
        if ((rc = harts::check_tables(*tb, seq_lo, seq_hi, dev_status, a.stream)) != HARTS_OK) return rc;
    if (use_tc(dtype, dk, dv, flags)) return harts::tc_fwd(a);
    return harts::fma_fwd(a);
}

int32_t harts_la_bwd_seqs(const harts_la_tables_t* tb, int32_t seq_lo, int32_t seq_hi, const void* q, const void* k,
                          const void* v, const float* g, const void* dO, void* dq, void* dk_, void* dv_, float* dg,
                          const void* chunk_states, void* scratch, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                          uint32_t flags, int32_t* dev_status, void* stream) {
    int32_t rc = check_common(tb, seq_lo, seq_hi, H, dk, dv, dtype);
    if (rc != HARTS_OK) return rc;
    if (!q || !k || !v || !g || !dO || !dq || !dk_ || !dv_ || !dg || !chunk_states || !scratch) return HARTS_EINVAL;
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(g) || misaligned(dO) || misaligned(dq) ||
        misaligned(dk_) || misaligned(dv_) || misaligned(dg) || misaligned(chunk_states) || misaligned(scratch))
        return HARTS_EINVAL;
    harts::BwdArgs a{*tb, seq_lo, seq_hi, q, k, v, g, dO, dq, dk_, dv_, dg, chunk_states, scratch, H, dk, dv, dtype,
                     flags, dev_status, static_cast<cudaStream_t>(stream)};
    if (flags & HARTS_FLAG_CHECK_TABLES)
        if ((rc = harts::check_tables(*tb, seq_lo, seq_hi, dev_status, a.stream)) != HARTS_OK) return rc;
    if (use_tc(dtype, dk, dv, flags)) return harts::tc_bwd(a);
    return harts::fma_bwd(a);
}

int32_t harts_la_bwd_finish(const harts_la_tables_t* tb, void* dk_, void* dv_, float* dg, const void* scratch,
                            int32_t H, int32_t dk, int32_t dv, int32_t dtype, void* stream) {
    int32_t rc = check_common(tb, 0, 0, H, dk, dv, dtype);
    if (rc != HARTS_OK) return rc;
    if (!dk_ || !dv_ || !dg || !scratch) return HARTS_EINVAL;
    return harts::replay_reduce(*tb, dk_, dv_, dg, scratch, H, dk, dv, dtype, static_cast<cudaStream_t>(stream));
}

int32_t harts_la_fwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q, const void* k,
                     const void* v, const float* g, void* o, float* slots, void* chunk_states, int32_t H, int32_t dk,
                     int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream) {
    const harts::Plan* p = harts_la_plan_internal(plan);
    if (!p || round < 0 || round > p->n_rounds) return HARTS_EINVAL;
    harts_la_tables_t tb;
    int32_t rc = harts_la_plan_tables(plan, dev_blob, &tb);
    if (rc != HARTS_OK) return rc;
    int32_t r0 = round == 0 ? 1 : round, r1 = round == 0 ? p->n_rounds : round;
    if (round == 0 && p->n_rounds > 1 && p->n_rounds <= harts::MAX_FUSED_ROUNDS && chunk_states &&
        !(flags & HARTS_FLAG_ROUND_LAUNCHES) &&
        use_tc(dtype, dk, dv, flags)) {
        // every round in one launch: a sequence waits for the flag of the state it starts from instead of for the
        // end of the previous round's kernel
        rc = check_common(&tb, 0, tb.n_seq, H, dk, dv, dtype);
        if (rc != HARTS_OK) return rc;
        if (!q || !k || !v || !g || !o || (tb.n_slots > 0 && !slots)) return HARTS_EINVAL;
        if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(g) || misaligned(o) || misaligned(slots) ||
            misaligned(chunk_states))
            return HARTS_EINVAL;
        harts::FwdArgs a{tb, 0, tb.n_seq, q, k, v, g, o, slots, chunk_states, H, dk, dv, dtype, flags, dev_status,
                         static_cast<cudaStream_t>(stream)};
        if (flags & HARTS_FLAG_CHECK_TABLES) {
            if (!dev_status) return HARTS_EINVAL;
            if ((rc = harts::check_tables(tb, 0, tb.n_seq, dev_status, a.stream)) != HARTS_OK) return rc;
        }
        int* fl = reinterpret_cast<int*>(static_cast<char*>(chunk_states) + harts::chunk_state_payload(tb, H, dk, dv, 2));
        rc = harts::tc_fwd_fused(a, fl, fl + harts::fused_flag_count(tb, H));
        if (rc != HARTS_EUNSUPPORTED) return rc;         // else: not all CTAs can be resident, launch round by round
    }
    for (int32_t r = r0; r <= r1; r++) {
        rc = harts_la_fwd_seqs(&tb, p->round_seq_ptr[r - 1], p->round_seq_ptr[r], q, k, v, g, o, slots, chunk_states,
                               H, dk, dv, dtype, flags, dev_status, stream);
        if (rc != HARTS_OK) return rc;
    }
    return HARTS_OK;
}

int32_t harts_la_bwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q, const void* k,
                     const void* v, const float* g, const void* dO, void* dq, void* dk_, void* dv_, float* dg,
                     const void* chunk_states, void* scratch, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                     uint32_t flags, int32_t* dev_status, void* stream) {
    const harts::Plan* p = harts_la_plan_internal(plan);
    if (!p || round < 0 || round > p->n_rounds) return HARTS_EINVAL;
    harts_la_tables_t tb;
    int32_t rc = harts_la_plan_tables(plan, dev_blob, &tb);
    if (rc != HARTS_OK) return rc;
    int32_t r1 = round == 0 ? p->n_rounds : round, r0 = round == 0 ? 1 : round;
    bool done = false;
    if (round == 0 && p->n_rounds > 1 && p->n_rounds <= harts::MAX_FUSED_ROUNDS && !(flags & HARTS_FLAG_ROUND_LAUNCHES) &&
        use_tc(dtype, dk, dv, flags)) {
        rc = check_common(&tb, 0, tb.n_seq, H, dk, dv, dtype);
        if (rc != HARTS_OK) return rc;
        if (!q || !k || !v || !g || !dO || !dq || !dk_ || !dv_ || !dg || !chunk_states || !scratch) return HARTS_EINVAL;
        if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(g) || misaligned(dO) || misaligned(dq) ||
            misaligned(dk_) || misaligned(dv_) || misaligned(dg) || misaligned(chunk_states) || misaligned(scratch))
            return HARTS_EINVAL;
        harts::BwdArgs a{tb, 0, tb.n_seq, q, k, v, g, dO, dq, dk_, dv_, dg, chunk_states, scratch, H, dk, dv, dtype, flags,
                         dev_status, static_cast<cudaStream_t>(stream)};
        if (flags & HARTS_FLAG_CHECK_TABLES) {
            if (!dev_status) return HARTS_EINVAL;
            if ((rc = harts::check_tables(tb, 0, tb.n_seq, dev_status, a.stream)) != HARTS_OK) return rc;
        }
        // the flags sit behind the chunk states; the backward's come after the forward's (n_slots * H), the two
        // ticket counters after both
        int* fl = reinterpret_cast<int*>(const_cast<char*>(static_cast<const char*>(chunk_states)) +
                                         harts::chunk_state_payload(tb, H, dk, dv, 2));
        harts::RoundOrder ro;
        ro.n = p->n_rounds;
        for (int32_t r = 0; r <= p->n_rounds; r++) ro.ptr[r] = p->round_seq_ptr[r];
        rc = harts::tc_bwd_fused(a, fl + (size_t)tb.n_slots * H, fl + harts::fused_flag_count(tb, H) + 1, ro);
        if (rc == HARTS_OK) done = true;
        else if (rc != HARTS_EUNSUPPORTED) return rc;
    }
    for (int32_t r = r1; r >= r0 && !done; r--) {
        rc = harts_la_bwd_seqs(&tb, p->round_seq_ptr[r - 1], p->round_seq_ptr[r], q, k, v, g, dO, dq, dk_, dv_, dg,
                               chunk_states, scratch, H, dk, dv, dtype, flags, dev_status, stream);
        if (rc != HARTS_OK) return rc;
    }
    if (r0 == 1) return harts_la_bwd_finish(&tb, dk_, dv_, dg, scratch, H, dk, dv, dtype, stream);
    return HARTS_OK;
}

int32_t harts_la_step_host(const harts_la_plan_t* plan, const void* dev_blob, const void* host_q, const void* host_k,
                           const void* host_v, const float* host_g, const void* host_dO, void* host_o, void* host_dq,
                           void* host_dk, void* host_dv, float* host_dg, void* dev_q, void* dev_k, void* dev_v,
                           float* dev_g, void* dev_dO, void* dev_o, void* dev_dq, void* dev_dk, void* dev_dv,
                           float* dev_dg, float* slots, void* chunk_states, void* scratch, int32_t H, int32_t dk,
                           int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream) {
    const harts::Plan* p = harts_la_plan_internal(plan);
    if (!p || H < 1 || dk < 1 || dv < 1) return HARTS_EINVAL;
    if (dtype != HARTS_FP32 && dtype != HARTS_BF16) return HARTS_EUNSUPPORTED;
    if (!host_q || !host_k || !host_v || !host_g || !host_dO || !host_o || !host_dq || !host_dk || !host_dv || !host_dg)
        return HARTS_EINVAL;
    const size_t elem = dtype == HARTS_FP32 ? 4 : 2, rows = (size_t)p->n_rows * H;
    const size_t nk = rows * dk * elem, nv = rows * dv * elem, ng = rows * sizeof(float);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const struct { void* dst; const void* src; size_t n; } in[5] = {
        {dev_q, host_q, nk}, {dev_k, host_k, nk}, {dev_v, host_v, nv}, {dev_g, host_g, ng}, {dev_dO, host_dO, nv}};
    for (const auto& c : in) {
        if (!c.dst) return HARTS_EINVAL;
        if (cudaMemcpyAsync(c.dst, c.src, c.n, cudaMemcpyHostToDevice, s) != cudaSuccess) return HARTS_ECUDA;
    }
    int32_t rc = harts_la_fwd(plan, dev_blob, 0, dev_q, dev_k, dev_v, dev_g, dev_o, slots, chunk_states, H, dk, dv, dtype,
                              flags, dev_status, stream);
    if (rc != HARTS_OK) return rc;
    rc = harts_la_bwd(plan, dev_blob, 0, dev_q, dev_k, dev_v, dev_g, dev_dO, dev_dq, dev_dk, dev_dv, dev_dg, chunk_states,
                      scratch, H, dk, dv, dtype, flags, dev_status, stream);
    if (rc != HARTS_OK) return rc;
    const struct { void* dst; const void* src; size_t n; } out[5] = {
        {host_o, dev_o, nv}, {host_dq, dev_dq, nk}, {host_dk, dev_dk, nk}, {host_dv, dev_dv, nv}, {host_dg, dev_dg, ng}};
    for (const auto& c : out)
        if (cudaMemcpyAsync(c.dst, c.src, c.n, cudaMemcpyDeviceToHost, s) != cudaSuccess) return HARTS_ECUDA;
    return HARTS_OK;
}

// ---- per-channel decay (the Diag(gamma) term of Eq. 1) -------------------------------------------------------------------
int32_t harts_la_gk_workspace_bytes(const harts_la_tables_t* tb, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                                    size_t* chunk_state_bytes, size_t* scratch_bytes) {
    if (!tb || H < 1 || dk < 1 || dv < 1) return HARTS_EINVAL;
    if (dtype != HARTS_FP32 && dtype != HARTS_BF16) return HARTS_EUNSUPPORTED;
    const size_t elem = dtype == HARTS_FP32 ? 4 : 2;
    if (chunk_state_bytes)      // the states, then the flags of the one-launch forms
        *chunk_state_bytes = harts::chunk_state_payload(*tb, H, dk, dv, elem) + harts::fused_flag_bytes(*tb, H);
    if (scratch_bytes) *scratch_bytes = harts::gk_scratch_layout(*tb, H, dk, dv).total;
    return HARTS_OK;
}

int32_t harts_la_gk_fwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q, const void* k,
                        const void* v, const float* gk, void* o, float* slots, void* chunk_states, int32_t H, int32_t dk,
                        int32_t dv, int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream) {
    const harts::Plan* p = harts_la_plan_internal(plan);
    if (!p || round < 0 || round > p->n_rounds) return HARTS_EINVAL;
    harts_la_tables_t tb;
    int32_t rc = harts_la_plan_tables(plan, dev_blob, &tb);
    if (rc != HARTS_OK) return rc;
    if (H < 1 || tb.chunk != 64 || !harts::gk_supported(dtype, dk, dv)) return H < 1 ? HARTS_EINVAL : HARTS_EUNSUPPORTED;
    if (!q || !k || !v || !gk || !o || (tb.n_slots > 0 && !slots)) return HARTS_EINVAL;
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(gk) || misaligned(o) || misaligned(slots) ||
        misaligned(chunk_states))
        return HARTS_EINVAL;
    if ((flags & HARTS_FLAG_CHECK_TABLES) && !dev_status) return HARTS_EINVAL;
    const int32_t r0 = round == 0 ? 1 : round, r1 = round == 0 ? p->n_rounds : round;
    const bool one_launch = round == 0 && p->n_rounds > 1 && p->n_rounds <= harts::MAX_FUSED_ROUNDS && chunk_states &&
                            !(flags & (HARTS_FLAG_ROUND_LAUNCHES | HARTS_FLAG_FMA_KERNELS)) &&
                            harts::gk_mma_supported(dtype, dk, dv);
    if (one_launch) {           // flags and tickets sit behind the chunk states, as for the scalar-gate calls
        harts::FwdArgs a{tb, 0, tb.n_seq, q, k, v, gk, o, slots, chunk_states, H, dk, dv, dtype, flags, dev_status,
                         static_cast<cudaStream_t>(stream)};
        if (flags & HARTS_FLAG_CHECK_TABLES)
            if ((rc = harts::check_tables(tb, 0, tb.n_seq, dev_status, a.stream)) != HARTS_OK) return rc;
        int* fl = reinterpret_cast<int*>(static_cast<char*>(chunk_states) + harts::chunk_state_payload(tb, H, dk, dv, 2));
        rc = harts::gk_mma_fwd_all(a, fl, fl + harts::fused_flag_count(tb, H));
        if (rc != HARTS_EUNSUPPORTED) return rc;
    }
    for (int32_t r = r0; r <= r1; r++) {
        harts::FwdArgs a{tb, p->round_seq_ptr[r - 1], p->round_seq_ptr[r], q, k, v, gk, o, slots, chunk_states, H, dk, dv,
                         dtype, flags, dev_status, static_cast<cudaStream_t>(stream)};
        if (flags & HARTS_FLAG_CHECK_TABLES)
            if ((rc = harts::check_tables(tb, a.seq_lo, a.seq_hi, dev_status, a.stream)) != HARTS_OK) return rc;
        if ((rc = harts::gk_fwd(a)) != HARTS_OK) return rc;
    }
    return HARTS_OK;
}

int32_t harts_la_gk_bwd(const harts_la_plan_t* plan, const void* dev_blob, int32_t round, const void* q, const void* k,
                        const void* v, const float* gk, const void* dO, void* dq, void* dk_, void* dv_, float* dgk,
                        const void* chunk_states, void* scratch, int32_t H, int32_t dk, int32_t dv, int32_t dtype,
                        uint32_t flags, int32_t* dev_status, void* stream) {
    const harts::Plan* p = harts_la_plan_internal(plan);
    if (!p || round < 0 || round > p->n_rounds) return HARTS_EINVAL;
    harts_la_tables_t tb;
    int32_t rc = harts_la_plan_tables(plan, dev_blob, &tb);
    if (rc != HARTS_OK) return rc;
    if (H < 1 || tb.chunk != 64 || !harts::gk_supported(dtype, dk, dv)) return H < 1 ? HARTS_EINVAL : HARTS_EUNSUPPORTED;
    if (!q || !k || !v || !gk || !dO || !dq || !dk_ || !dv_ || !dgk || !chunk_states || !scratch) return HARTS_EINVAL;
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(gk) || misaligned(dO) || misaligned(dq) ||
        misaligned(dk_) || misaligned(dv_) || misaligned(dgk) || misaligned(chunk_states) || misaligned(scratch))
        return HARTS_EINVAL;
    if ((flags & HARTS_FLAG_CHECK_TABLES) && !dev_status) return HARTS_EINVAL;
    const int32_t r1 = round == 0 ? p->n_rounds : round, r0 = round == 0 ? 1 : round;
    bool done = false;
    if (round == 0 && p->n_rounds > 1 && p->n_rounds <= harts::MAX_FUSED_ROUNDS &&
        !(flags & (HARTS_FLAG_ROUND_LAUNCHES | HARTS_FLAG_FMA_KERNELS)) && harts::gk_mma_supported(dtype, dk, dv)) {
        harts::BwdArgs a{tb, 0, tb.n_seq, q, k, v, gk, dO, dq, dk_, dv_, dgk, chunk_states, scratch, H, dk, dv, dtype, flags,
                         dev_status, static_cast<cudaStream_t>(stream)};
        if (flags & HARTS_FLAG_CHECK_TABLES)
            if ((rc = harts::check_tables(tb, 0, tb.n_seq, dev_status, a.stream)) != HARTS_OK) return rc;
        int* fl = reinterpret_cast<int*>(const_cast<char*>(static_cast<const char*>(chunk_states)) +
                                         harts::chunk_state_payload(tb, H, dk, dv, 2));
        harts::RoundOrder ro;
        ro.n = p->n_rounds;
        for (int32_t r = 0; r <= p->n_rounds; r++) ro.ptr[r] = p->round_seq_ptr[r];
        rc = harts::gk_mma_bwd_all(a, fl + (size_t)tb.n_slots * H, fl + harts::fused_flag_count(tb, H) + 1, ro);
        if (rc == HARTS_OK) done = true;
        else if (rc != HARTS_EUNSUPPORTED) return rc;
    }
    for (int32_t r = r1; r >= r0 && !done; r--) {
        harts::BwdArgs a{tb, p->round_seq_ptr[r - 1], p->round_seq_ptr[r], q, k, v, gk, dO, dq, dk_, dv_, dgk,
                         chunk_states, scratch, H, dk, dv, dtype, flags, dev_status, static_cast<cudaStream_t>(stream)};
        if (flags & HARTS_FLAG_CHECK_TABLES)
            if ((rc = harts::check_tables(tb, a.seq_lo, a.seq_hi, dev_status, a.stream)) != HARTS_OK) return rc;
        if ((rc = harts::gk_bwd(a)) != HARTS_OK) return rc;
    }
    if (r0 == 1)
        return harts::gk_replay_reduce(tb, dk_, dv_, dgk, scratch, H, dk, dv, dtype, static_cast<cudaStream_t>(stream));
    return HARTS_OK;
}

int32_t harts_la_check(const int32_t* dev_status, void* stream) {
    if (!dev_status) return HARTS_EINVAL;
    int32_t host = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&host, dev_status, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess) return HARTS_ECUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return HARTS_ECUDA;
    if (host == 0) return HARTS_OK;
    return host == HARTS_EINVAL ? HARTS_EINVAL : HARTS_ETIMEOUT;   // EINVAL: an index check of harts_logp_*
}

}  // extern "C"
