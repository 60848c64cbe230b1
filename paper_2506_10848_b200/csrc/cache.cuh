// Internal launchers of the feature-cache kernels (dLLM-Cache-style reuse of per-layer K, V and branch outputs).
#pragma once
#include "sfs_common.cuh"

namespace sfs {

constexpr int kSimSlices = 32;         // the feature dimension is cut into this many slices for the similarity sums

// partial[slice][t][0..2] = sum over the slice's features of (v_new * v_old, v_new^2, v_old^2) for the tokens
// t_first <= t < t_first + t_count (t_first even); both operands are feature-major bf16 [d, T] with ld elements between
// feature rows; partial is [kSimSlices, T, 3] whatever the token range.
int32_t launch_sim_partial(const void *vnew_t, const void *vold_t, long long ld, int d, int t_first, int t_count, int T, float *partial,
                           cudaStream_t s);

struct CacheSelectArgs {
    const float *partial;              // [kSimSlices, T, 3]
    const sfs_state *state;            // [B] or NULL (NULL: every step is treated as a slow step)
    int B, S, P, L, T;
    int refresh_p, refresh_r;          // whole-segment refresh flags of this step
    int n_adapt;                       // rows the adaptive rule recomputes per sequence (when !refresh_r)
    int n_sel;                         // rows listed per sequence = (refresh_p ? P : 0) + (refresh_r ? L : n_adapt)
    int32_t *sel_rows;                 // [B, n_sel] flat token indices
    float *sims_dump;                  // optional [B, L]
    int32_t *sets_dump;                // optional [B, n_sel]
};
// Chooses, per sequence, the n_adapt candidate response positions whose new value is least similar to the cached one
// (cosine similarity, ties to the lower position), ascending, padded by repeating the last one; candidates are all
// response positions in a slow step and the span [s_cycle, hi) in a fast step.
int32_t launch_cache_select(const CacheSelectArgs &a, cudaStream_t s);

int32_t launch_gather_rows_bf16(const void *src, const int32_t *rows, int n_rows, int d, void *dst, cudaStream_t s);
// dst[rows[j], :] = sum over k < n_slabs of src[k * slab_stride + j * d + :]   (fp32 rows of d elements; slabs = the partial
// products of a split-K projection, added in slab order)
int32_t launch_scatter_rows_f32(const float *src, int n_slabs, long long slab_stride, const int32_t *rows, int n_rows, int d, float *dst,
                                cudaStream_t s);
// K rows: dst[rows[j], 0:d] = src[j, col0 : col0 + d] (bf16, src ld = ld_src);  V columns: dst_t[f, rows[j]] = src_t[f, j]
int32_t launch_scatter_kv(const void *qk_src, long long ld_src, int col0, const void *vt_src, long long ld_vt_src,
                          const int32_t *rows, int n_rows, int d, void *k_dst, void *vt_dst, long long ld_vt_dst, cudaStream_t s);

// rope (as launch_rope, on the compact rows) + rotated k rows into the K cache + new value columns into V^T, one launch
int32_t launch_rope_scatter_kv(void *qk, long long ld, int n_rows, int S, int n_heads, int head_dim, const float2 *table, const int32_t *rows,
                               void *k_dst, const void *vt_src, long long ld_vt_src, void *vt_dst, long long ld_vt_dst, cudaStream_t s);
// inc[rows[j], :] = sum of the slabs of compact row j (slab order); h[j, :] = bf16(RMSNorm(x[rows[j], :] + inc[rows[j], :]) * gain)
int32_t launch_fold_norm_rows(const float *slabs, int n_slabs, long long slab_stride, const int32_t *rows, int n_rows, const float *x, float *inc,
                              const void *gain, void *h, int d, float eps, cudaStream_t s);

}  // namespace sfs
