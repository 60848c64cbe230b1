// Internal interface of the tcgen05 attention kernel.
#pragma once
#include "sfs_common.cuh"
#include <cuda.h>
#include <string.h>
#include <math.h>

namespace sfs {

struct AttnArgs {
    int B, S, n_heads, d_model;
    int kq;                            // query rows per sequence (S, or fewer when the queries are a compact subset)
    int k_col0;                        // first key column in the key tensor
    float scale_log2;                  // log2(e) / sqrt(head_dim)
    __nv_bfloat16 *out; long long ld_out;
    int32_t *err;
    const int32_t *d_active;           // optional: the kernel does nothing when *d_active == 0
};

struct AttnPlan {
    CUtensorMap tmQ, tmK, tmVt;
    AttnArgs args;
    int head_dim;
};

// qkv: [B*S, >= 2*d] bf16 rows (q at columns [0, d), k at [d, 2d), RoPE applied), ld_qkv elements between rows;
// vt:  [d, B*S] bf16 (V transposed: feature-major), ld_vt elements between feature rows;
// out: [B*S, d] bf16.
int32_t attn_plan_create(AttnPlan *p, const void *qkv, int64_t ld_qkv, const void *vt, int64_t ld_vt,
                         void *out, int64_t ld_out, int32_t B, int32_t S, int32_t n_heads, int32_t head_dim);
// Queries and keys in separate tensors: q [B*kq_max rows, d] (sequence b's queries are rows b*kq .. b*kq+kq-1 at launch),
// k [B*S, k_cols] with the keys at columns [k_col0, k_col0 + d); out has the layout of q.
int32_t attn_plan_create_split(AttnPlan *p, const void *q, int64_t ld_q, const void *k, int64_t ld_k, int32_t k_cols, int32_t k_col0,
                               const void *vt, int64_t ld_vt, void *out, int64_t ld_out, int32_t B, int32_t S, int32_t n_heads, int32_t head_dim);
int32_t attn_launch_queries(const AttnPlan &p, int32_t kq, const int32_t *d_active, int32_t *err, cudaStream_t stream);
int32_t attn_launch(const AttnPlan &p, const int32_t *d_active, int32_t *err, cudaStream_t stream);

}  // namespace sfs
