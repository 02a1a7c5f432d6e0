// Device-side validation of hand-built index tables (HARTS_FLAG_CHECK_TABLES): every index that the kernels of a
// packed call would follow is checked against its range before they run.  A bad entry puts HARTS_EINVAL into the
// status word (and the offending table and position behind it); the kernels of the call then return without touching
// anything.  Nothing here faults: an entry is only read after the pointers that lead to it were found in range.
#include "kernels.h"

namespace harts {
namespace {

enum Table {
    T_OWN_BEGIN = 1, T_INIT_SLOT, T_REPLAY_PTR, T_REPLAY_ROW, T_REQ_PTR, T_SLOT_CHUNK, T_CHUNK_PTR, T_CONS_PTR,
    T_CONS_SEQ, T_RG_ROW, T_RG_PTR, T_RG_ENTRY, T_SEQ_ORDER
};

__device__ void fail(int32_t* status, int table, int index) {
    if (atomicCAS(status, 0, HARTS_EINVAL) == 0) {
        status[1] = table;
        status[2] = index;
    }
}

// Non-decreasing CSR pointers ptr[lo..hi] inside [0, limit]; returns false on the first violation.
__device__ bool csr_ok(const int32_t* ptr, int lo, int hi, int limit, int32_t* status, int table) {
    int prev = ptr[lo];
    if (prev < 0 || prev > limit) {
        fail(status, table, lo);
        return false;
    }
    for (int i = lo + 1; i <= hi; i++) {
        const int cur = ptr[i];
        if (cur < prev || cur > limit) {
            fail(status, table, i);
            return false;
        }
        prev = cur;
    }
    return true;
}

// One thread checks the pointer arrays (they are short: one entry per sequence or slot); then all threads check the
// entries those pointers address.
__global__ void check_tables_kernel(const harts_la_tables_t tb, int seq_lo, int seq_hi, int32_t* status) {
    __shared__ int ok;
    if (threadIdx.x == 0) {
        bool good = *reinterpret_cast<volatile int32_t*>(status) == 0;
        good = good && csr_ok(tb.seq_own_begin, seq_lo, seq_hi, tb.n_rows, status, T_OWN_BEGIN);
        good = good && csr_ok(tb.seq_replay_ptr, seq_lo, seq_hi, tb.n_replay, status, T_REPLAY_PTR);
        good = good && csr_ok(tb.seq_req_ptr, seq_lo, seq_hi, tb.n_slots, status, T_REQ_PTR);
        good = good && csr_ok(tb.seq_chunk_ptr, seq_lo, seq_hi, tb.n_chunks, status, T_CHUNK_PTR);
        good = good && (tb.n_slots == 0 || csr_ok(tb.slot_cons_ptr, 0, tb.n_slots, tb.n_seq, status, T_CONS_PTR));
        good = good && (tb.n_rg_rows == 0 || csr_ok(tb.rg_ptr, 0, tb.n_rg_rows, tb.n_replay, status, T_RG_PTR));
        ok = good ? 1 : 0;
    }
    __syncthreads();
    if (!ok) return;
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int s = seq_lo + tid; s < seq_hi; s += nt) {
        const int n_rep = tb.seq_replay_ptr[s + 1] - tb.seq_replay_ptr[s];
        const int own = tb.seq_own_begin[s + 1] - tb.seq_own_begin[s];
        const int chunks = (n_rep + own + tb.chunk - 1) / tb.chunk;
        if (n_rep >= tb.chunk) fail(status, T_REPLAY_PTR, s);                       // a replay is shorter than a chunk
        if (tb.seq_chunk_ptr[s + 1] - tb.seq_chunk_ptr[s] != chunks) fail(status, T_CHUNK_PTR, s);
        const int init = tb.seq_init_slot[s];
        if (init < -1 || init >= tb.n_slots) fail(status, T_INIT_SLOT, s);
        int prev_chunk = 0;
        for (int r = tb.seq_req_ptr[s]; r < tb.seq_req_ptr[s + 1]; r++) {           // ascending chunk indices inside the sequence
            const int c = tb.slot_chunk[r];
            if (c <= prev_chunk || c >= chunks) fail(status, T_SLOT_CHUNK, r);
            prev_chunk = c;
        }
        if (tb.seq_order) {
            const int o = tb.seq_order[s];
            if (o < seq_lo || o >= seq_hi) fail(status, T_SEQ_ORDER, s);
        }
    }
    for (int e = tb.seq_replay_ptr[seq_lo] + tid; e < tb.seq_replay_ptr[seq_hi]; e += nt)
        if (tb.replay_row[e] < 0 || tb.replay_row[e] >= tb.n_rows) fail(status, T_REPLAY_ROW, e);
    if (tb.n_slots)
        for (int e = tid; e < tb.slot_cons_ptr[tb.n_slots]; e += nt)
            if (tb.slot_cons_seq[e] < 0 || tb.slot_cons_seq[e] >= tb.n_seq) fail(status, T_CONS_SEQ, e);
    for (int e = tid; e < tb.n_rg_rows; e += nt)
        if (tb.rg_row[e] < 0 || tb.rg_row[e] >= tb.n_rows) fail(status, T_RG_ROW, e);
    if (tb.n_rg_rows)
        for (int e = tid; e < tb.rg_ptr[tb.n_rg_rows]; e += nt)
            if (tb.rg_entry[e] < 0 || tb.rg_entry[e] >= tb.n_replay) fail(status, T_RG_ENTRY, e);
}

}  // namespace

int32_t check_tables(const harts_la_tables_t& tb, int32_t seq_lo, int32_t seq_hi, int32_t* dev_status, cudaStream_t stream) {
    if (!dev_status) return HARTS_EINVAL;
    check_tables_kernel<<<1, 1024, 0, stream>>>(tb, seq_lo, seq_hi, dev_status);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
