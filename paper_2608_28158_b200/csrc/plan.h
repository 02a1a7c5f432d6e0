// Host-side plan object shared by the planner (plan.cc) and the launch code (api.cu).
#pragma once
#include <cstdint>
#include <vector>

#include "../../include/harts_la.h"

namespace harts {

constexpr int N_DEVICE_TABLES = 13;

struct Plan {
    int32_t chunk = 0, n_rounds = 0, n_rows = 0, n_replay = 0, n_seq = 0, n_slots = 0, n_chunks = 0,
            n_rg_rows = 0;
    std::vector<int32_t> row_of_token, round_seq_ptr, seq_tree, seq_own_begin, seq_own_len, seq_start_pos,
        seq_init_slot, seq_replay_ptr, replay_row, seq_req_ptr, slot_chunk, seq_chunk_ptr, slot_cons_ptr,
        slot_cons_seq, rg_row, rg_ptr, rg_entry, seq_order;
    std::vector<int32_t> blob;                 // device tables back to back, 16-byte aligned starts
    size_t table_offset[N_DEVICE_TABLES] = {}; // in int32 words
    void pack();
    void tables(const void* dev_blob, harts_la_tables_t* out) const;
};

int32_t build_plan(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                   const int32_t* node_fork_off, const int32_t* node_len, int32_t chunk, Plan& out);

}  // namespace harts

extern "C" const harts::Plan* harts_la_plan_internal(const harts_la_plan_t* plan);
