// Internal launchers of the memory-bound forward kernels.
#pragma once
#include "sfs_common.cuh"

namespace sfs {
int32_t launch_embed(const int32_t *tokens, const void *emb, float *x, int T, int d, int vocab, cudaStream_t s);
// h[r,:] = bf16(RMSNorm(y[rows ? rows[r] : r, :]) * gain) with y = x + the n_partial slabs of `partial` (partial_stride
// floats apart, added in slab order; may be NULL).  Without a row list y is written back to x.  The row count may
// come from the device (n_rows).
int32_t launch_rmsnorm(float *x, const float *partial, int n_partial, long long partial_stride, const void *gain, void *h,
                       const int32_t *rows, const int32_t *n_rows, int max_rows, int d, float eps, cudaStream_t s);
int32_t launch_rope_table(float2 *table, int positions, int head_dim, float theta, cudaStream_t s);
// rotates q and k (the first 2*n_heads*head_dim columns of each row) in place; position = token index mod S, the token
// index of row t being rows[t] when a row list is given (compact rows) and t otherwise
int32_t launch_rope(void *qk, int64_t ld, int T, int S, int n_heads, int head_dim, const float2 *table, const int32_t *rows, cudaStream_t s);
}  // namespace sfs
