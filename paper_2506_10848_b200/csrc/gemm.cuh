// Internal interface of the tcgen05 GEMM (C = A * B^T, bf16 in, fp32 accumulate).
#pragma once
#include "sfs_common.cuh"
#include <cuda.h>
#include <string.h>

namespace sfs {

enum GemmMode {
    GEMM_STORE = 0,          // C = scale * acc   (bf16 or fp32); optionally the trailing columns go transposed to `vt`
    GEMM_RESIDUAL_F32 = 1,   // C (fp32) += acc
    GEMM_SWIGLU = 2,         // C (bf16) = silu(acc_gate) * acc_up, gate and up rows loaded side by side into one tile
};

struct GemmArgs {
    int M, N, K;
    const int32_t *d_m;      // optional device-side row count (<= M)
    int mode, out_f32;
    float scale;
    void *C; long long ldc;
    __nv_bfloat16 *vt; long long ldvt; int vt_col0;
    int tiles_per_map;       // column tiles per B matrix (concatenated outputs)
    int n_per_map;           // rows of each B matrix
    int bn, stages;          // tile width (multiple of 16, <= 256) and depth of the shared-memory ring
    int mb;                  // 256-row blocks per tile (1 or 2)
    int one_cta;             // 1: tiles of 128 rows computed by single CTAs (few rows: the weights stream through every SM)
    int tile_rows;           // output rows per tile: mb * 256, or 128
    int n_col_tiles;         // column tiles over all B matrices
    int splits, kb_per_split;        // split-K: the k-blocks are cut into `splits` ranges, range s writes slab s of C
    long long split_stride;          // elements between slabs
    int acc_bufs;            // accumulator buffers in tensor memory (2 when they fit: epilogue overlaps the next tile)
    // Optional (GEMM_STORE, bf16 output, no split): row statistics of the stored values, taken in the epilogue.  Per output
    // row, column tile and epilogue-warp parity one record (maximum, reference, sum of 2^((x - reference) log2 e), first
    // position of the maximum as int bits) at stats[row * stats_ld + 2 * column_tile + parity]: the first pass of the
    // selection step's row statistics, fused into the LM head (the logits are not read back for it).
    float4 *stats; int stats_ld;
    int32_t *err;            // device status word, set to SFS_ERR_TIMEOUT if a bounded wait gives up
    const int32_t *d_active; // optional: the kernel does nothing when *d_active == 0
};

struct GemmPlan {
    CUtensorMap tmA, tmB[3];
    GemmArgs args;
    int bn, n_maps, n_per_map;
    const void *A, *Bs[3]; long long lda, ldb;       // kept so that the plan can be rebuilt at another tile shape
};

// Optional overrides of the tile shape the planner would pick (0 = keep the planner's choice); for measurements.
struct GemmTune { int mb, bn, stages, splits; };

// Bs: n_maps weight matrices [n_per_map, K] (ldb elements between rows) whose outputs are concatenated along
// the columns of C (QKV), or gate / up for GEMM_SWIGLU (then C has n_per_map columns).
int32_t gemm_plan_create(GemmPlan *p, const void *A, int64_t lda, int32_t M, int32_t K,
                         const void *const *Bs, int32_t n_maps, int32_t n_per_map, int64_t ldb,
                         int32_t mode, void *C, int64_t ldc, int32_t out_f32, float scale,
                         __nv_bfloat16 *vt, int64_t ldvt, int32_t vt_col0, const GemmTune *tune);
// Split-K for the residual projections (mode GEMM_RESIDUAL_F32): when `ws` is given and the planner finds that cutting
// K fills the machine better, the plan writes `args.splits` fp32 partial products to the slabs ws + s * M * ldc (plain
// stores, C itself is not touched) and the consumer of the residual stream adds them in slab order (launch_rmsnorm does),
// so the sum does not depend on which CTA finishes first.  ws must hold max_splits * M * ldc floats.
int32_t gemm_plan_enable_split(GemmPlan *p, float *ws, int32_t max_splits, const GemmTune *tune);
int32_t gemm_launch(const GemmPlan &p, const int32_t *d_m, const int32_t *d_active, int32_t *err, cudaStream_t stream);

}  // namespace sfs
