// Model and session objects behind the opaque handles of the C ABI.
#pragma once
#include "sfs_common.cuh"
#include "gemm.cuh"
#include "attention.cuh"
#include <vector>
#include <map>

struct sfs_model {
    sfs_config cfg;
    // borrowed device pointers (copied pointer tables)
    const void *tok_emb, *final_norm, *lm_head;
    std::vector<const void *> attn_norm, wq, wk, wv, wo, mlp_norm, w_gate, w_up, w_down;
};

struct LayerPlans { sfs::GemmPlan qkv, o, gate_up, down; };
// cached mode: per layer, independent of how many rows are recomputed
struct CacheLayerPlans { sfs::GemmPlan vproj, o_store, down_store; sfs::AttnPlan attn; };
// cached mode: projections over the compact buffer of recomputed rows, per layer, for one row count
struct GatherLayerPlans { sfs::GemmPlan qkv, o, gate_up, down; };

struct sfs_session {
    sfs_model *model = nullptr;          // NULL: a selection-only session
    int32_t max_batch = 0, max_seq = 0, vocab = 0;
    // selection scratch
    unsigned long long *pos_sq = nullptr;    // [max_batch*max_seq]
    int32_t *pos_arg = nullptr;              // [max_batch*max_seq]
    unsigned long long *pos_lo = nullptr, *pos_hi = nullptr;   // [max_batch*max_seq] enclosures of the two-pass row statistics
    float *slice_partials = nullptr; int32_t *row_tickets = nullptr;   // scratch of its first pass
    int32_t *pos_row = nullptr, *refine_list = nullptr, *refine_count = nullptr;   // rows its second pass recomputes
    float *pos_max = nullptr;                                                       // exact row maximum per position
    int32_t *seq_rows = nullptr;             // [max_batch*max_seq]
    int32_t *seq_row_count = nullptr;        // [max_batch]
    int32_t *ticket = nullptr;               // [1]
    // forward workspace (model sessions only); T = max_batch*max_seq
    float *x = nullptr;                      // [T, d] fp32 residual stream
    float *partial = nullptr;                // [kMaxSplits, T, d] split-K partial products of the residual projections
    __nv_bfloat16 *h = nullptr;              // [T, d] normalised activations
    __nv_bfloat16 *qk = nullptr;             // [T, 2d] q | k
    __nv_bfloat16 *vt = nullptr;             // [d, T] V transposed
    __nv_bfloat16 *attn = nullptr;           // [T, d]
    __nv_bfloat16 *hid = nullptr;            // [T, d_ff]
    __nv_bfloat16 *hfin = nullptr;           // [T, d] gathered + normalised rows for the LM head
    __nv_bfloat16 *logits = nullptr;         // [T, vocab]
    float2 *rope_table = nullptr;            // [max_seq, head_dim/2]
    // generation state
    int32_t *tokens = nullptr;               // [T]
    uint8_t *mask = nullptr;                 // [T]
    sfs_state *state = nullptr;              // [max_batch]
    int32_t *rows[2] = {nullptr, nullptr};   // [T] row lists of the current / next step
    int32_t *ctrl = nullptr;                 // [0..1] row counts (double buffer), [2] active sequences
    int32_t *host_active = nullptr;          // pinned, device-mapped mirror of ctrl[2]
    int32_t *host_active_dev = nullptr;      // its device address
    // plans for the shapes of the current call
    int32_t plan_B = 0, plan_S = 0;
    std::vector<LayerPlans> layer_plans;
    sfs::AttnPlan attn_plan;
    sfs::GemmPlan lm_plan;
    float4 *lm_stats = nullptr; size_t lm_stats_cap = 0;     // row-statistics records the LM head's epilogue leaves (fused first pass)
    // what the next RMSNorm must fold into x: n slabs `pending_stride` floats apart (split-K partials or a cached increment)
    const float *pending_ptr = nullptr; int pending_n = 0; long long pending_stride = 0;
    // feature cache (dLLM-Cache-style), allocated by sfs_cache_enable
    bool cache_on = false;
    sfs_cache_params cache_params{};
    int cache_t = 0, cache_B = 0, cache_S = 0, cache_P = 0;   // step counter and the shape the cached features belong to
    std::vector<__nv_bfloat16 *> Kc, Vtc;    // per layer: rotated keys [T, d], values transposed [d, T]
    std::vector<float *> Ac, Fc;             // per layer: residual increments of the attention and MLP branches [T, d]
    __nv_bfloat16 *hg = nullptr;             // [T, d] gathered normalised rows
    __nv_bfloat16 *vnew_t = nullptr;         // [d, T] fresh values of every row, transposed
    float *sim_partial = nullptr;            // [kSimSlices, T, 3]
    int32_t *sel_rows = nullptr;             // [T] rows recomputed in the current layer
    int32_t *dump_sets = nullptr; float *dump_sims = nullptr;   // caller's buffers for the sets / similarities of generate steps
    std::vector<CacheLayerPlans> cache_plans;
    std::map<int, std::vector<GatherLayerPlans>> gather_plans;
    // generation bookkeeping (host)
    int32_t gen_B = 0, gen_P = 0, gen_L = 0, gen_cur = 0, gen_steps = 0, gen_max_steps = 0;
    sfs_params gen_params;
    bool generating = false;
    std::vector<void *> owned;               // device allocations to free at destroy
    // optional per-kernel-class timing (CUDA events around every launch) and launch counting
    bool profile = false;
    long long launches = 0;
    struct Timed { int cls; cudaEvent_t e0, e1; };
    std::vector<Timed> timed;
};
