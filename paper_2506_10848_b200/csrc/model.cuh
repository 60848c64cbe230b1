// Model and session objects behind the opaque handles of the C ABI.
#pragma once
#include "sfs_common.cuh"
#include <vector>

struct sfs_model {
    sfs_config cfg;
    // borrowed device pointers (copied pointer tables)
    const void *tok_emb, *final_norm, *lm_head;
    std::vector<const void *> attn_norm, wq, wk, wv, wo, mlp_norm, w_gate, w_up, w_down;
    float2 *rope_table = nullptr;        // [max positions, head_dim/2] (cos, sin), owned
    int32_t rope_positions = 0;
};

struct sfs_session {
    sfs_model *model = nullptr;          // may be NULL: a selection-only session
    int32_t max_batch = 0, max_seq = 0, vocab = 0;
    // selection scratch
    unsigned long long *pos_sq = nullptr;    // [max_batch*max_seq]
    int32_t *pos_arg = nullptr;              // [max_batch*max_seq]
    int32_t *seq_rows = nullptr;             // [max_batch*max_seq]
    int32_t *seq_row_count = nullptr;        // [max_batch]
    int32_t *ticket = nullptr;               // [1]
    std::vector<void *> owned;               // everything to cudaFree at destroy
};
