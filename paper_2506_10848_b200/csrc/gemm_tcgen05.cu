// Dense projections of the mask predictor (QKV / O / gate-up / down / LM head): C = A * B^T with bf16
// operands and fp32 accumulation in tensor memory.
//
// A pair of CTAs (a cluster of two, on the two SMs of a TPC) computes a (MB x 256) x BN output tile with
// tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of every 256-row block of A and its own half of
// the BN weight rows, so a weight tile enters the pair once and the bytes an SM pulls through its L2 port per
// FLOP drop (the operand stream from L2, not the tensor core, bounds these shapes).  The pair walks a static
// list of tiles (persistent kernel).  In each CTA warp 0 streams 128-byte-swizzled operand tiles into a ring of
// shared-memory stages with TMA (completion is counted on the leader CTA's barrier), the leader's warp 1 issues
// the MMAs and releases stages in both CTAs with a multicast tcgen05.commit, and warps 2-9 read the accumulator
// back with tcgen05.ld and run the fused epilogue (scale / fp32 residual add / SwiGLU / transposed V store).
// When two accumulators fit tensor memory the epilogue of a tile overlaps the next tile's main loop.  The row
// count may live on the device, so the LM head can follow the shrinking set of masked rows without a host
// round trip.
#include "sfs_common.cuh"
#include "tc05.cuh"
#include "gemm.cuh"

namespace sfs {

// ---- host: tensor maps -------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

int32_t make_tmap_bf16(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows)
{
    EncodeTiledFn enc = get_encode();
    SFS_REQUIRE(enc != nullptr, SFS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    SFS_REQUIRE(aligned_to(base, 16) && (ld % 8) == 0 && rows >= 1 && cols >= 1 && box_rows >= 1 && box_rows <= 256,
                SFS_ERR_INVALID_ARG, "tensor map: base must be 16-byte aligned, ld a multiple of 8 (ld=%llu rows=%llu cols=%llu)",
                (unsigned long long)ld, (unsigned long long)rows, (unsigned long long)cols);
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    SFS_REQUIRE(r == CUDA_SUCCESS, SFS_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
    return SFS_OK;
}

namespace {

constexpr int BM = 128, BK = 64;         // rows per CTA of one 256-row MMA block; K elements per stage
constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr int A_BYTES = BM * BK * 2;
constexpr int kMaxStages = 8;
constexpr int kSmemBudget = 227 * 1024 - 64;      // the opt-in maximum minus the kernel's static shared memory
// barriers: full[kMaxStages], empty[kMaxStages], acc_full[2], acc_empty[2]; then the TMEM base slot
constexpr int kBarBytes = (2 * kMaxStages + 4) * 8 + 16;
constexpr int kTmemCols = 512;
constexpr int kEpiStageBytes = kEpiWarps * 32 * 128;   // one 32-row x 128-byte output unit per epilogue warp

// x * sigmoid(x) with the special-function unit's exponential and reciprocal (a few ulp: the result is rounded to bf16)
__device__ __forceinline__ float silu_f(float x) { return __fdividef(x, 1.0f + __expf(-x)); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

// which output columns / weight rows a tile covers
struct TileCoord {
    int split;       // which range of k-blocks (split-K), 0 when K is not split
    int m0;          // first output row of the pair's tile
    int map_idx;     // which B matrix (concatenated outputs), 0 for SwiGLU
    int n_local;     // first row of that B matrix (SwiGLU: first gate row = first up row)
    int ncol0;       // first output column
    int ncols;       // valid output columns of the tile (<= BN, SwiGLU: <= BN/2)
};

__device__ __forceinline__ TileCoord tile_coord(const GemmArgs &g, int tile, int m_groups)
{
    TileCoord t;
    const int rest = tile / m_groups;
    t.m0 = (tile - rest * m_groups) * g.tile_rows;         // row groups fastest: pairs that share a weight tile run together
    const int n_tile = rest / g.splits;
    t.split = rest - n_tile * g.splits;
    if (g.mode == GEMM_SWIGLU) {
        const int half = g.bn >> 1;
        t.map_idx = 0; t.n_local = n_tile * half; t.ncol0 = t.n_local; t.ncols = min(half, g.N - t.ncol0);
    } else {
        t.map_idx = n_tile / g.tiles_per_map;
        t.n_local = (n_tile - t.map_idx * g.tiles_per_map) * g.bn;
        t.ncol0 = t.map_idx * g.n_per_map + t.n_local;
        t.ncols = min(g.bn, g.n_per_map - t.n_local);
    }
    return t;
}

// ---- epilogue --------------------------------------------------------------------------------------------
// tcgen05.ld hands every lane one accumulator ROW, so storing from those registers makes each store instruction
// touch 32 different lines.  Instead a warp parks a 32-row x 128-byte unit of output in shared memory (16-byte
// chunks XOR-swizzled by row, so both directions are conflict-free) and writes it out as 4 rows x 128 contiguous
// bytes per instruction.  A unit is 32 fp32 or 64 bf16 output columns.
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void red_add_v4_f32(float *p, uint4 v) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 ::"l"(p), "f"(__uint_as_float(v.x)), "f"(__uint_as_float(v.y)), "f"(__uint_as_float(v.z)), "f"(__uint_as_float(v.w)) : "memory");
}
// lane = row: park 4 consecutive 16-byte chunks (chunk0 .. chunk0+3) of this lane's row
__device__ __forceinline__ void park16(uint32_t stage, int lane, int chunk0, const uint32_t *w) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
        st_shared_v4(stage + lane * 128 + (((chunk0 + c) ^ (lane & 7)) << 4), w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
}

// Writes the parked unit out.  Row r of the unit is output row grow0 + r; its 128 bytes start at output column col0.
// ELEM = bytes per output element (2 or 4); columns at or beyond `lim` and rows at or beyond M are skipped.
// Every output element belongs to exactly one tile, so the residual add (one vector red per chunk) is deterministic.
template <int ELEM, bool RESIDUAL>
__device__ __forceinline__ void flush_unit(const GemmArgs &g, long long slab, uint32_t stage, int lane, int grow0, int M, int col0, int lim)
{
    constexpr int PER = 16 / ELEM;                       // elements per 16-byte chunk
    const int c = lane & 7, col = col0 + c * PER;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + (lane >> 3), grow = grow0 + r;
        if (grow >= M || col >= lim) continue;
        const uint4 v = ld_shared_v4(stage + r * 128 + ((c ^ (r & 7)) << 4));
        uint8_t *dst = reinterpret_cast<uint8_t *>(g.C) + (slab + (long long)grow * g.ldc + col) * ELEM;
        if (col + PER <= lim) {
            if (RESIDUAL) red_add_v4_f32(reinterpret_cast<float *>(dst), v);
            else *reinterpret_cast<uint4 *>(dst) = v;
        } else {                                         // ragged last chunk of the matrix: element by element
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            for (int e = 0; e < PER && col + e < lim; ++e) {
                if (RESIDUAL) atomicAdd(reinterpret_cast<float *>(dst) + e, __uint_as_float(w[e]));
                else if (ELEM == 4) reinterpret_cast<uint32_t *>(dst)[e] = w[e];
                else reinterpret_cast<uint16_t *>(dst)[e] = (uint16_t)(w[e >> 1] >> ((e & 1) * 16));
            }
        }
    }
}

// One warp's share of a tile's epilogue: TMEM lane quarter q (32 rows) of every 256-row block, the units of parity `par`.
// A unit may reach past the tile's valid columns: those accumulator columns exist (inside the 256-column buffer) and
// are never stored.  The tensor-memory loads of the next piece are issued as soon as the current piece has been
// converted, so their latency hides behind the parking and the stores of the current one.
template <bool STATS>
__device__ __forceinline__ void epilogue_tile(const GemmArgs &g, const TileCoord &t, uint32_t tmem_acc, uint32_t bn_pad, uint32_t stage,
                                              int q, int par, int lane, int rank, int M)
{
    const int HALF = g.bn >> 1;
    const int lim = min(t.ncol0 + t.ncols, g.N);         // first output column this tile must not touch
    const uint32_t tq = tmem_acc + ((uint32_t)(q * 32) << 16);
    const int grow_q = t.m0 + rank * BM + q * 32;        // first row of block 0 handled by this warp
    if (g.mode == GEMM_SWIGLU || (g.mode == GEMM_STORE && !g.out_f32 && !(g.vt != nullptr && t.ncol0 >= g.vt_col0))) {
        // ---- bf16 output (plain or SwiGLU): units of 64 output columns, handled as two pieces of 32
        const bool swiglu = (g.mode == GEMM_SWIGLU);
        // the units of all 256-row blocks, numbered block by block, alternate between the two warps of a lane quarter
        const int upb = (t.ncols + 63) / 64;                              // units per 256-row block
        const int n_pieces = 2 * ((g.mb * upb - par + 1) / 2);
        auto piece_addr = [&](int pc) {                                   // tensor-memory column of piece pc
            const int u = par + 2 * (pc >> 1), b = u / upb, c = 64 * (u - b * upb);
            return tq + (uint32_t)(b * bn_pad + c + 32 * (pc & 1));
        };
        uint32_t x0[32], x1[32];
        if (n_pieces > 0) {
            tc::tmem_ld32(piece_addr(0), x0);
            if (swiglu) tc::tmem_ld32(piece_addr(0) + HALF, x1);
        }
        // fused row statistics (LM head): this lane's row of the current 256-row block
        const bool stats_on = STATS && (g.stats != nullptr) && !swiglu;
        float st_mx = -INFINITY, st_ref = 0.f, st_nref = 0.f, st_sum = 0.f;
        int st_arg = 0x7FFFFFFF, st_b = -1;
        const int n_tile = (t.ncol0 / g.bn);                             // one weight matrix: column tile index
        auto stats_flush = [&]() {
            if (st_b < 0) return;
            const int grow = grow_q + st_b * 2 * BM + lane;
            if (grow < M) g.stats[(long long)grow * g.stats_ld + 2 * n_tile + par] = make_float4(st_mx, st_ref, st_sum, __int_as_float(st_arg));
        };
        for (int pc = 0; pc < n_pieces; ++pc) {
            uint32_t o[16];
            tc::tmem_ld_wait32(x0);
            if (swiglu) tc::tmem_ld_wait32(x1);
            if (swiglu) {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    o[j] = pack_bf16(silu_f(__uint_as_float(x0[2 * j])) * __uint_as_float(x1[2 * j]),
                                     silu_f(__uint_as_float(x0[2 * j + 1])) * __uint_as_float(x1[2 * j + 1]));
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) o[j] = pack_bf16(__uint_as_float(x0[2 * j]) * g.scale, __uint_as_float(x0[2 * j + 1]) * g.scale);
            }
            if (pc + 1 < n_pieces) {
                tc::tmem_ld32(piece_addr(pc + 1), x0);
                if (swiglu) tc::tmem_ld32(piece_addr(pc + 1) + HALF, x1);
            }
            if (stats_on) {
                // statistics of the ROUNDED values, as a reader of the stored logits would see them
                const int u = par + 2 * (pc >> 1), b = u / upb, col0 = t.ncol0 + 64 * (u - b * upb) + 32 * (pc & 1);
                if (b != st_b) { stats_flush(); st_b = b; st_mx = -INFINITY; st_sum = 0.f; st_arg = 0x7FFFFFFF; st_ref = 0.f; st_nref = 0.f; }
                const int nvalid = min(32, lim - col0);                  // columns of this piece inside the matrix (warp-uniform)
                float pm = -INFINITY;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float lo = __uint_as_float(o[j] << 16), hi = __uint_as_float(o[j] & 0xFFFF0000u);
                    if (2 * j < nvalid) pm = fmaxf(pm, lo);
                    if (2 * j + 1 < nvalid) pm = fmaxf(pm, hi);
                }
                if (st_mx == -INFINITY && st_sum == 0.f) {               // first piece of this row: it gives the reference
                    st_ref = (fabsf(pm) <= 3.0e38f) ? pm : 0.f;
                    st_nref = -st_ref * 1.4426950408889634f;
                }
                if (pm > st_mx) {                                        // strict: the first position of the maximum
                    st_mx = pm;
#pragma unroll
                    for (int j = 15; j >= 0; --j) {
                        const float lo = __uint_as_float(o[j] << 16), hi = __uint_as_float(o[j] & 0xFFFF0000u);
                        if (2 * j + 1 < nvalid && hi == pm) st_arg = col0 + 2 * j + 1;
                        if (2 * j < nvalid && lo == pm) st_arg = col0 + 2 * j;
                    }
                }
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float lo = __uint_as_float(o[j] << 16), hi = __uint_as_float(o[j] & 0xFFFF0000u);
                    const float e0 = tc::ex2_approx(__fmaf_rn(lo, 1.4426950408889634f, st_nref));
                    const float e1 = tc::ex2_approx(__fmaf_rn(hi, 1.4426950408889634f, st_nref));
                    s0 += (2 * j < nvalid) ? e0 : 0.f;
                    s1 += (2 * j + 1 < nvalid) ? e1 : 0.f;
                }
                st_sum += s0 + s1;
            }
            park16(stage, lane, 4 * (pc & 1), o);
            if (pc & 1) {
                const int u = par + 2 * (pc >> 1), b = u / upb, c = 64 * (u - b * upb);
                __syncwarp();
                flush_unit<2, false>(g, 0, stage, lane, grow_q + b * 2 * BM, M, t.ncol0 + c, lim);
                __syncwarp();
            }
        }
        if (stats_on) stats_flush();
    } else if (g.vt != nullptr && t.ncol0 >= g.vt_col0) {
        // ---- V columns of the QKV projection go out transposed: the 32 lanes hold 32 consecutive tokens of a feature
        const int upb = (t.ncols + 31) / 32;
        const int n_pieces = (g.mb * upb - par + 1) / 2;
        auto piece_col = [&](int pc, int *b) { const int u = par + 2 * pc; *b = u / upb; return 32 * (u - *b * upb); };
        uint32_t v[32];
        int b0;
        if (n_pieces > 0) { const int c = piece_col(0, &b0); tc::tmem_ld32(tq + (uint32_t)(b0 * bn_pad + c), v); }
        for (int pc = 0; pc < n_pieces; ++pc) {
            int b;
            const int c = piece_col(pc, &b);
            uint16_t h[32];
            tc::tmem_ld_wait32(v);
#pragma unroll
            for (int j = 0; j < 32; ++j) { __nv_bfloat16 r = __float2bfloat16_rn(__uint_as_float(v[j]) * g.scale); h[j] = *reinterpret_cast<uint16_t *>(&r); }
            if (pc + 1 < n_pieces) { int bn2; const int c2 = piece_col(pc + 1, &bn2); tc::tmem_ld32(tq + (uint32_t)(bn2 * bn_pad + c2), v); }
            const int grow = grow_q + b * 2 * BM + lane;
            if (grow < M) {
                uint16_t *dst = reinterpret_cast<uint16_t *>(g.vt) + (long long)(t.ncol0 + c - g.vt_col0) * g.ldvt + grow;
                const int nv = lim - (t.ncol0 + c);                        // valid features of this piece
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (j < nv) dst[(long long)j * g.ldvt] = h[j];
            }
        }
    } else {
        // ---- fp32 output (residual add, split-K slab, or fp32 logits): units of 32 columns
        const int upb = (t.ncols + 31) / 32;
        const int n_pieces = (g.mb * upb - par + 1) / 2;
        auto piece_col = [&](int pc, int *b) { const int u = par + 2 * pc; *b = u / upb; return 32 * (u - *b * upb); };
        const bool scale = (g.mode != GEMM_RESIDUAL_F32 && g.scale != 1.0f);
        uint32_t v[32];
        int b0;
        if (n_pieces > 0) { const int c = piece_col(0, &b0); tc::tmem_ld32(tq + (uint32_t)(b0 * bn_pad + c), v); }
        for (int pc = 0; pc < n_pieces; ++pc) {
            int b;
            const int c = piece_col(pc, &b);
            uint32_t o[32];
            tc::tmem_ld_wait32(v);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = scale ? __float_as_uint(__uint_as_float(v[j]) * g.scale) : v[j];
            if (pc + 1 < n_pieces) { int bn2; const int c2 = piece_col(pc + 1, &bn2); tc::tmem_ld32(tq + (uint32_t)(bn2 * bn_pad + c2), v); }
            park16(stage, lane, 0, o);
            park16(stage, lane, 4, o + 16);
            __syncwarp();
            if (g.mode == GEMM_RESIDUAL_F32 && g.splits == 1) flush_unit<4, true>(g, 0, stage, lane, grow_q + b * 2 * BM, M, t.ncol0 + c, lim);
            else flush_unit<4, false>(g, (long long)t.split * g.split_stride, stage, lane, grow_q + b * 2 * BM, M, t.ncol0 + c, lim);
            __syncwarp();
        }
    }
}

template <bool STATS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
            const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, GemmArgs g)
{
    // This kernel may have been scheduled while the one before it in the stream still runs (programmatic dependent launch):
    // everything up to pdl_wait() touches only this CTA's shared and tensor memory.
    pdl_trigger();
    const int MB = g.mb;
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    // uniform over the pair, before any barrier or allocation: pairs beyond the tiles of even the largest row count
    if (pair >= ((g.M + MB * 2 * BM - 1) / (MB * 2 * BM)) * g.n_col_tiles * g.splits) return;

    const int BN = g.bn, STAGES = g.stages, HALF = BN >> 1;
    const int STAGE_BYTES = MB * A_BYTES + HALF * BK * 2;   // per CTA: MB blocks of 128 A rows, half of the weight rows
    const uint32_t rank = tc::cluster_ctarank();            // 0 = leader (issues the MMAs), 1 = peer

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kMaxStages + 4);
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (g.K + BK - 1) / BK;
    const uint32_t smem_base = tc::smem_u32(smem);
    const uint32_t bar_full = tc::smem_u32(bars), bar_empty = bar_full + 8 * kMaxStages;
    const uint32_t bar_acc_full = bar_full + 16 * kMaxStages, bar_acc_empty = bar_acc_full + 16;
    // the leader's copies of the barriers both CTAs signal
    const uint32_t lead_full = tc::mapa(bar_full, 0), lead_acc_empty = tc::mapa(bar_acc_empty, 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(bar_full + 8 * s, 1); tc::mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(bar_acc_full + 8 * b, 1); tc::mbar_init(bar_acc_empty + 8 * b, 2 * kEpiWarps); }
        s_abort = 0;
        tc::mbar_init_fence();
    }
    __syncwarp();
    if (warp == 1) { tc::tmem_alloc_2cta(tc::smem_u32(tmem_slot), kTmemCols); tc::tmem_relinquish_2cta(); }
    tc::tc_fence_before();
    tc::cluster_sync();                                     // barriers of both CTAs are initialised, TMEM is allocated
    tc::tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);
    const uint32_t bn_pad = (uint32_t)((BN + 31) & ~31);
    const uint32_t n_bufs = (uint32_t)g.acc_bufs, buf_stride = 256;     // two buffers only when MB * bn_pad <= 256
    const bool swiglu = (g.mode == GEMM_SWIGLU);

    pdl_wait();                                             // the kernel before this one has completed: global memory from here on
    // nothing left to decode, or fewer rows than planned: the loops below find no tile (same values in both CTAs of the pair)
    const bool live = !(g.d_active && *g.d_active == 0);
    const int M = g.d_m ? min(*g.d_m, g.M) : g.M;
    const int m_groups = (M + MB * 2 * BM - 1) / (MB * 2 * BM);
    const int num_tiles = live ? m_groups * g.n_col_tiles * g.splits : 0;

    // The producer and MMA loops are run by all 32 lanes of their warp with warp-uniform operands; one elected lane
    // issues each asynchronous instruction.  (Issued from a single-lane branch, every tcgen05.mma cost the thread
    // about 90 cycles and an already-complete mbarrier wait about 200: the loop, not the tensor core, set the pace.)
    // The readiness of the next stage is polled (without blocking) before the current stage's instructions are
    // issued, so the latency of that poll overlaps the issue.
    if (warp == 0) {
        // ---------------- TMA producer (both CTAs; completion bytes are counted on the leader's barrier)
        if (lane == 0) { tc::tma_prefetch_desc(&tmA); tc::tma_prefetch_desc(&tmB0); }
        uint32_t it = 0;
        bool ok = true;
        bool ready = tc::mbar_test(bar_empty, 1u);
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
            const TileCoord t = tile_coord(g, tile, m_groups);
            // leader: first half of the weight rows (SwiGLU: the gate rows); peer: second half (the up rows)
            const CUtensorMap *mb = swiglu ? (rank == 0 ? &tmB0 : &tmB1)
                                           : (t.map_idx == 0 ? &tmB0 : (t.map_idx == 1 ? &tmB1 : &tmB2));
            const int brow = swiglu ? t.n_local : t.n_local + (int)rank * HALF;
            const int arow = t.m0 + (int)rank * BM;
            const int kb0 = t.split * g.kb_per_split, kb1 = min(num_kb, kb0 + g.kb_per_split);
            for (int kb = kb0; kb < kb1; ++kb, ++it) {
                const uint32_t s = it % (uint32_t)STAGES, ph = (it / (uint32_t)STAGES) & 1u;
                if (!ready) ready = tc::mbar_wait(bar_empty + 8 * s, ph ^ 1u, &s_abort);
                ok = __all_sync(0xffffffffu, ready);
                if (!ok) break;
                const uint32_t nx = it + 1u, ns = nx % (uint32_t)STAGES, nph = (nx / (uint32_t)STAGES) & 1u;
                ready = tc::mbar_test(bar_empty + 8 * ns, nph ^ 1u);
                const uint32_t sa = smem_base + s * STAGE_BYTES;
                if (rank == 0) tc::mbar_expect_tx_elect(bar_full + 8 * s, 2u * (uint32_t)STAGE_BYTES);
                tc::tma_load_2d_2cta_elect(sa, &tmA, kb * BK, arow, lead_full + 8 * s);
                if (MB == 2) tc::tma_load_2d_2cta_elect(sa + A_BYTES, &tmA, kb * BK, arow + 2 * BM, lead_full + 8 * s);
                tc::tma_load_2d_2cta_elect(sa + MB * A_BYTES, mb, kb * BK, brow, lead_full + 8 * s);
            }
        }
        if (s_abort && rank == 0 && lane == 0) {
            // give copies already in flight (both CTAs') a bounded chance to land before the pair retires
            const uint32_t first = it > (uint32_t)STAGES ? it - (uint32_t)STAGES : 0u;
            for (uint32_t j = first; j < it; ++j) {
                const uint32_t bar = bar_full + 8 * (j % (uint32_t)STAGES), ph = (j / (uint32_t)STAGES) & 1u;
                for (int i = 0; i < (1 << 16) && !tc::mbar_try(bar, ph); ++i) {}
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---------------- MMA issuer (leader CTA only)
            const uint32_t idesc = tc::idesc_bf16_f32(2 * BM, BN);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            bool ready = tc::mbar_test(bar_full, 0u);
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++lt) {
                const uint32_t buf = lt % n_bufs, use = lt / n_bufs;
                // both CTAs' epilogues have drained this accumulator buffer
                ok = __all_sync(0xffffffffu, tc::mbar_wait(bar_acc_empty + 8 * buf, (use & 1u) ^ 1u, &s_abort));
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * buf_stride;
                const int kb0 = tile_coord(g, tile, m_groups).split * g.kb_per_split, kb1 = min(num_kb, kb0 + g.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const uint32_t s = it % (uint32_t)STAGES, ph = (it / (uint32_t)STAGES) & 1u;
                    if (!ready) ready = tc::mbar_wait(bar_full + 8 * s, ph, &s_abort);
                    ok = __all_sync(0xffffffffu, ready);
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t nx = it + 1u, ns = nx % (uint32_t)STAGES, nph = (nx / (uint32_t)STAGES) & 1u;
                    ready = tc::mbar_test(bar_full + 8 * ns, nph);
                    const uint32_t sa = smem_base + s * STAGE_BYTES;
                    const uint64_t da = tc::smem_desc_sw128(sa), db = tc::smem_desc_sw128(sa + MB * A_BYTES);
                    const uint32_t acc = kb != kb0 ? 1u : 0u;
                    tc::mma_bf16_2cta_elect(d_tmem, da, db, idesc, acc);
#pragma unroll
                    for (int kk = 1; kk < BK / 16; ++kk) tc::mma_bf16_2cta_elect(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, 1u);
                    if (MB == 2) {
                        const uint64_t da1 = tc::smem_desc_sw128(sa + A_BYTES);
                        tc::mma_bf16_2cta_elect(d_tmem + bn_pad, da1, db, idesc, acc);
#pragma unroll
                        for (int kk = 1; kk < BK / 16; ++kk) tc::mma_bf16_2cta_elect(d_tmem + bn_pad, da1 + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, 1u);
                    }
                    tc::mma_commit_2cta_elect(bar_empty + 8 * s);     // frees the stage in both CTAs once these MMAs have read it
                }
                tc::mma_commit_2cta_elect(bar_acc_full + 8 * buf);    // accumulator complete (or abandoned), both CTAs
            }
        }
    } else {
        // ---------------- epilogue: 8 warps; warp w reads TMEM lanes 32*(w%4).., the column units of parity (w-2)/4
        const int q = warp & 3, par = (warp - 2) >> 2;
        const uint32_t stage = smem_base + STAGES * STAGE_BYTES + kBarBytes + (uint32_t)(warp - 2) * (32 * 128);
        uint32_t lt = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++lt) {
            const TileCoord t = tile_coord(g, tile, m_groups);
            const uint32_t buf = lt % n_bufs, use = lt / n_bufs;
            ok = tc::mbar_wait(bar_acc_full + 8 * buf, use & 1u, &s_abort) && !s_abort;
            if (!ok) break;
            tc::tc_fence_after();
            epilogue_tile<STATS>(g, t, tmem_base + buf * buf_stride, bn_pad, stage, q, par, lane, (int)rank, M);
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive_cluster(lead_acc_empty + 8 * buf);
        }
    }

    // ---------------- teardown: no CTA of the pair leaves while the other may still signal its barriers
    __syncwarp();                                           // the diverged roles rejoin their warps
    tc::tc_fence_before();
    tc::cluster_sync();
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc_2cta(tmem_base, kTmemCols); }
    if (threadIdx.x == 0 && s_abort && g.err) atomicExch(g.err, SFS_ERR_TIMEOUT);
}

// ---- few rows (M <= 128): one CTA per tile ------------------------------------------------------------------
// With at most 128 rows half of a pair's 256-row MMA would multiply padding, and what bounds the projection is streaming the
// weights: every SM should pull its own slab of weight rows at full rate.  A CTA computes a 128 x BN tile with
// tcgen05.mma.cta_group::1 (M = 128, N = BN), loading the 128 activation rows and BN weight rows of every k-block itself (the
// weight rows as two boxes of BN / 2, SwiGLU: gate rows then up rows, so the accumulator layout and the epilogue are those
// of the pair kernel); BN is chosen so that the tiles fill the SMs in whole waves.  Same warp roles, ring and bounded waits.
template <bool STATS>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel_1cta(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                 const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, GemmArgs g)
{
    pdl_trigger();
    if ((int)blockIdx.x >= ((g.M + BM - 1) / BM) * g.n_col_tiles * g.splits) return;     // beyond the tiles of even the largest row count

    const int BN = g.bn, STAGES = g.stages, HALF = BN >> 1;
    const int STAGE_BYTES = A_BYTES + BN * BK * 2;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kMaxStages + 4);
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (g.K + BK - 1) / BK;
    const uint32_t smem_base = tc::smem_u32(smem);
    const uint32_t bar_full = tc::smem_u32(bars), bar_empty = bar_full + 8 * kMaxStages;
    const uint32_t bar_acc_full = bar_full + 16 * kMaxStages, bar_acc_empty = bar_acc_full + 16;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(bar_full + 8 * s, 1); tc::mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(bar_acc_full + 8 * b, 1); tc::mbar_init(bar_acc_empty + 8 * b, kEpiWarps); }
        s_abort = 0;
        tc::mbar_init_fence();
    }
    __syncwarp();
    if (warp == 1) { tc::tmem_alloc(tc::smem_u32(tmem_slot), kTmemCols); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);
    const uint32_t bn_pad = (uint32_t)((BN + 31) & ~31);
    const uint32_t n_bufs = (uint32_t)g.acc_bufs, buf_stride = 256;
    const bool swiglu = (g.mode == GEMM_SWIGLU);
    const int num_ctas = (int)gridDim.x;

    pdl_wait();                                             // the kernel before this one has completed: global memory from here on
    const bool live = !(g.d_active && *g.d_active == 0);    // nothing left to decode: the loops below find no tile
    const int M = g.d_m ? min(*g.d_m, g.M) : g.M;
    const int m_groups = (M + BM - 1) / BM;
    const int num_tiles = live ? m_groups * g.n_col_tiles * g.splits : 0;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) { tc::tma_prefetch_desc(&tmA); tc::tma_prefetch_desc(&tmB0); }
        uint32_t it = 0;
        bool ok = true;
        bool ready = tc::mbar_test(bar_empty, 1u);
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += num_ctas) {
            const TileCoord t = tile_coord(g, tile, m_groups);
            const CUtensorMap *m0 = swiglu ? &tmB0 : (t.map_idx == 0 ? &tmB0 : (t.map_idx == 1 ? &tmB1 : &tmB2));
            const CUtensorMap *m1 = swiglu ? &tmB1 : m0;
            const int brow1 = swiglu ? t.n_local : t.n_local + HALF;
            const int kb0 = t.split * g.kb_per_split, kb1 = min(num_kb, kb0 + g.kb_per_split);
            for (int kb = kb0; kb < kb1; ++kb, ++it) {
                const uint32_t s = it % (uint32_t)STAGES, ph = (it / (uint32_t)STAGES) & 1u;
                if (!ready) ready = tc::mbar_wait(bar_empty + 8 * s, ph ^ 1u, &s_abort);
                ok = __all_sync(0xffffffffu, ready);
                if (!ok) break;
                const uint32_t nx = it + 1u, ns = nx % (uint32_t)STAGES, nph = (nx / (uint32_t)STAGES) & 1u;
                ready = tc::mbar_test(bar_empty + 8 * ns, nph ^ 1u);
                const uint32_t sa = smem_base + s * STAGE_BYTES;
                tc::mbar_expect_tx_elect(bar_full + 8 * s, (uint32_t)STAGE_BYTES);
                tc::tma_load_2d_elect(sa, &tmA, kb * BK, t.m0, bar_full + 8 * s);
                tc::tma_load_2d_elect(sa + A_BYTES, m0, kb * BK, t.n_local, bar_full + 8 * s);
                tc::tma_load_2d_elect(sa + A_BYTES + HALF * BK * 2, m1, kb * BK, brow1, bar_full + 8 * s);
            }
        }
        if (s_abort && lane == 0) {
            // give copies already in flight a bounded chance to land before the CTA retires
            const uint32_t first = it > (uint32_t)STAGES ? it - (uint32_t)STAGES : 0u;
            for (uint32_t j = first; j < it; ++j) {
                const uint32_t bar = bar_full + 8 * (j % (uint32_t)STAGES), ph = (j / (uint32_t)STAGES) & 1u;
                for (int i = 0; i < (1 << 16) && !tc::mbar_try(bar, ph); ++i) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        const uint32_t idesc = tc::idesc_bf16_f32(BM, BN);
        uint32_t it = 0, lt = 0;
        bool ok = true;
        bool ready = tc::mbar_test(bar_full, 0u);
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += num_ctas, ++lt) {
            const uint32_t buf = lt % n_bufs, use = lt / n_bufs;
            ok = __all_sync(0xffffffffu, tc::mbar_wait(bar_acc_empty + 8 * buf, (use & 1u) ^ 1u, &s_abort));
            if (!ok) break;
            tc::tc_fence_after();
            const uint32_t d_tmem = tmem_base + buf * buf_stride;
            const int kb0 = tile_coord(g, tile, m_groups).split * g.kb_per_split, kb1 = min(num_kb, kb0 + g.kb_per_split);
            for (int kb = kb0; kb < kb1; ++kb, ++it) {
                const uint32_t s = it % (uint32_t)STAGES, ph = (it / (uint32_t)STAGES) & 1u;
                if (!ready) ready = tc::mbar_wait(bar_full + 8 * s, ph, &s_abort);
                ok = __all_sync(0xffffffffu, ready);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t nx = it + 1u, ns = nx % (uint32_t)STAGES, nph = (nx / (uint32_t)STAGES) & 1u;
                ready = tc::mbar_test(bar_full + 8 * ns, nph);
                const uint32_t sa = smem_base + s * STAGE_BYTES;
                const uint64_t da = tc::smem_desc_sw128(sa), db = tc::smem_desc_sw128(sa + A_BYTES);
                tc::mma_bf16_elect(d_tmem, da, db, idesc, kb != kb0 ? 1u : 0u);
#pragma unroll
                for (int kk = 1; kk < BK / 16; ++kk) tc::mma_bf16_elect(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, 1u);
                tc::mma_commit_elect(bar_empty + 8 * s);          // frees the stage once these MMAs have read it
            }
            tc::mma_commit_elect(bar_acc_full + 8 * buf);         // accumulator complete (or abandoned)
        }
    } else {
        // ---------------- epilogue: 8 warps; warp w reads TMEM lanes 32*(w%4).., the column units of parity (w-2)/4
        const int q = warp & 3, par = (warp - 2) >> 2;
        const uint32_t stage = smem_base + STAGES * STAGE_BYTES + kBarBytes + (uint32_t)(warp - 2) * (32 * 128);
        uint32_t lt = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += num_ctas, ++lt) {
            const TileCoord t = tile_coord(g, tile, m_groups);
            const uint32_t buf = lt % n_bufs, use = lt / n_bufs;
            ok = tc::mbar_wait(bar_acc_full + 8 * buf, use & 1u, &s_abort) && !s_abort;
            if (!ok) break;
            tc::tc_fence_after();
            epilogue_tile<STATS>(g, t, tmem_base + buf * buf_stride, bn_pad, stage, q, par, lane, 0, M);
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bar_acc_empty + 8 * buf);
        }
    }

    __syncwarp();
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc(tmem_base, kTmemCols); }
    if (threadIdx.x == 0 && s_abort && g.err) atomicExch(g.err, SFS_ERR_TIMEOUT);
}

int num_sms()
{
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

// column tiles of a problem at tile width bn
int col_tiles(int mode, int n_maps, int n_per_map, int bn)
{
    if (mode == GEMM_SWIGLU) return (n_per_map + bn / 2 - 1) / (bn / 2);
    return n_maps * ((n_per_map + bn - 1) / bn);
}

int stages_for(int mb, int bn)
{
    const int stage_bytes = mb * A_BYTES + (bn / 2) * BK * 2;
    const int s = (kSmemBudget - 1024 - kBarBytes - kEpiStageBytes) / stage_bytes;
    return s > kMaxStages ? kMaxStages : s;
}

// Modelled clocks of one candidate: waves x (k-blocks x clocks per k-block + exposed epilogue), per pair of SMs.
// Per k-block and CTA the tensor core needs MB*bn*2 clocks (8192 FLOP/clk/SM); the operand stream is
// (MB*128 + bn/2) rows x 128 B at the ~40 B/clk an SM sustains from L2 when every SM streams; below ~750 clocks the
// k-block time stops shrinking with the tile (load latency over the bytes a CTA can keep in flight).  All measured.
// The epilogue hides behind the next tile when two accumulators fit tensor memory, except for a pair's last tile.
// Splitting K pays for few rows only: the slabs grow with M, the idle pairs they avoid do not.
long long model_clocks(int M, int K, int mode, int n_maps, int n_per_map, int pairs, int mb, int bn, int splits)
{
    const long long num_kb = (K + BK - 1) / BK, kbps = (num_kb + splits - 1) / splits;
    const int m_groups = (M + mb * 2 * BM - 1) / (mb * 2 * BM);
    const long long tiles = (long long)m_groups * col_tiles(mode, n_maps, n_per_map, bn) * ((num_kb + kbps - 1) / kbps);
    const long long waves = (tiles + pairs - 1) / pairs;
    const long long mma = (long long)mb * bn * 2, load = (long long)(mb * BM + bn / 2) * 128 / 40;
    long long kb_clk = mma > load ? mma : load;
    if (kb_clk < 750) kb_clk = 750;
    const long long epi = (long long)mb * bn * 16 + 3000;
    const bool hidden = mb * ((bn + 31) & ~31) <= 256;
    // a split K also costs the fp32 slab that the next RMSNorm reads back: M x N x 4 bytes, measured at ~1.2e-3 clocks per element
    const long long n_out = (mode == GEMM_SWIGLU) ? n_per_map : (long long)n_maps * n_per_map;
    const long long slab = 1500 + (long long)((double)M * (double)n_out * 1.2e-3);
    return waves * kbps * kb_clk + (hidden ? 1 : waves) * epi + (splits > 1 ? slab * splits : 0);
}

// Tile shape (MB blocks of 256 rows, width bn) and number of K ranges with the smallest modelled time.  Wide, tall tiles
// win when there are many tiles; narrower or shorter ones, or a split K, when a big tile would leave most pairs idle.
void pick_tile(int M, int K, int mode, int n_maps, int n_per_map, int pairs, int max_splits, int *mb_out, int *bn_out, int *splits_out)
{
    const int step = (mode == GEMM_SWIGLU) ? 32 : 16;
    long long best_cost = -1;
    for (int mb = (M > 2 * BM ? 2 : 1); mb >= 1; --mb)
        for (int bn = 256; bn >= 32; bn -= step)
            for (int sp = 1; sp <= max_splits; ++sp) {
                const long long cost = model_clocks(M, K, mode, n_maps, n_per_map, pairs, mb, bn, sp);
                if (best_cost < 0 || cost < best_cost) { best_cost = cost; *mb_out = mb; *bn_out = bn; *splits_out = sp; }
            }
}

// Few rows: tiles of 128 x bn on single CTAs.  Per k-block a CTA streams (128 + bn) rows x 128 B at the ~40 B/clk an SM gets
// from L2 when all SMs stream, against 2 * bn clocks of tensor-core work; 600 clocks is where the k-block time stops shrinking.
long long model_clocks_1cta(int M, int K, int mode, int n_maps, int n_per_map, int sms, int bn, int splits)
{
    const long long num_kb = (K + BK - 1) / BK, kbps = (num_kb + splits - 1) / splits;
    const long long tiles = (long long)col_tiles(mode, n_maps, n_per_map, bn) * ((num_kb + kbps - 1) / kbps);
    const long long waves = (tiles + sms - 1) / sms;
    const long long mma = 2LL * bn, load = (long long)(BM + bn) * 128 / 40;
    long long kb_clk = mma > load ? mma : load;
    if (kb_clk < 600) kb_clk = 600;
    const long long epi = (long long)bn * 16 + 3000;
    const long long n_out = (mode == GEMM_SWIGLU) ? n_per_map : (long long)n_maps * n_per_map;
    const long long slab = 1500 + (long long)((double)M * (double)n_out * 1.2e-3);
    return waves * kbps * kb_clk + epi + (splits > 1 ? slab * splits : 0);
}

void pick_tile_1cta(int M, int K, int mode, int n_maps, int n_per_map, int sms, int max_splits, int *bn_out, int *splits_out)
{
    const int step = (mode == GEMM_SWIGLU) ? 32 : 16;
    long long best_cost = -1;
    for (int bn = 256; bn >= 32; bn -= step)
        for (int sp = 1; sp <= max_splits; ++sp) {
            const long long cost = model_clocks_1cta(M, K, mode, n_maps, n_per_map, sms, bn, sp);
            if (best_cost < 0 || cost < best_cost) { best_cost = cost; *bn_out = bn; *splits_out = sp; }
        }
}

int stages_for_1cta(int bn)
{
    const int stage_bytes = A_BYTES + bn * BK * 2;
    const int s = (kSmemBudget - 1024 - kBarBytes - kEpiStageBytes) / stage_bytes;
    return s > kMaxStages ? kMaxStages : s;
}

}  // namespace

int32_t gemm_plan_create(GemmPlan *p, const void *A, int64_t lda, int32_t M, int32_t K,
                         const void *const *Bs, int32_t n_maps, int32_t n_per_map, int64_t ldb,
                         int32_t mode, void *C, int64_t ldc, int32_t out_f32, float scale,
                         __nv_bfloat16 *vt, int64_t ldvt, int32_t vt_col0, const GemmTune *tune)
{
    SFS_REQUIRE(M >= 1 && K >= 1 && n_per_map >= 1 && n_maps >= 1 && n_maps <= 3, SFS_ERR_INVALID_ARG, "gemm: bad sizes");
    SFS_REQUIRE((K % 8) == 0 && (lda % 8) == 0 && (ldb % 8) == 0, SFS_ERR_INVALID_ARG, "gemm: K, lda, ldb must be multiples of 8");
    SFS_REQUIRE(mode != GEMM_SWIGLU || n_maps == 2, SFS_ERR_INVALID_ARG, "gemm: SwiGLU takes two B matrices");
    memset(p, 0, sizeof(*p));
    const int N = (mode == GEMM_SWIGLU) ? n_per_map : n_per_map * n_maps;
    SFS_REQUIRE(aligned_to(C, 16) && (ldc % 8) == 0, SFS_ERR_INVALID_ARG, "gemm: C must be 16-byte aligned, ldc a multiple of 8");
    int mb = 1, bn = 256;
    int sp_unused = 1;
    // at most 128 rows: single-CTA tiles (a pair's 256-row MMA would be half padding); tune->mb = 1 or 2 forces the pair kernel
    const bool one_cta = (M <= BM) && !(tune && (tune->mb == 1 || tune->mb == 2));
    if (one_cta) pick_tile_1cta(M, K, mode, n_maps, n_per_map, num_sms(), 1, &bn, &sp_unused);
    else pick_tile(M, K, mode, n_maps, n_per_map, num_sms() / 2, 1, &mb, &bn, &sp_unused);
    if (tune) {                                              // measurement overrides; invalid values are ignored
        if (tune->mb == 1 || tune->mb == 2) mb = tune->mb;
        if (tune->bn >= 32 && tune->bn <= 256 && (tune->bn % ((mode == GEMM_SWIGLU) ? 32 : 16)) == 0) bn = tune->bn;
    }
    p->bn = bn; p->n_maps = n_maps; p->n_per_map = n_per_map;
    int32_t rc = make_tmap_bf16(&p->tmA, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM);
    if (rc != SFS_OK) return rc;
    for (int i = 0; i < 3; ++i) {
        const void *b = Bs[i < n_maps ? i : 0];
        rc = make_tmap_bf16(&p->tmB[i], b, (uint64_t)n_per_map, (uint64_t)K, (uint64_t)ldb, (uint32_t)(bn / 2));
        if (rc != SFS_OK) return rc;
    }
    GemmArgs &g = p->args;
    g.M = M; g.N = N; g.K = K; g.mode = mode; g.out_f32 = out_f32; g.scale = scale;
    g.C = C; g.ldc = ldc; g.vt = vt; g.ldvt = ldvt; g.vt_col0 = vt_col0;
    g.bn = bn; g.mb = one_cta ? 1 : mb; g.n_per_map = n_per_map;
    g.one_cta = one_cta ? 1 : 0; g.tile_rows = one_cta ? BM : mb * 2 * BM;
    g.tiles_per_map = (mode == GEMM_SWIGLU) ? 0x3FFFFFFF : (n_per_map + bn - 1) / bn;
    g.n_col_tiles = col_tiles(mode, n_maps, n_per_map, bn);
    g.stages = one_cta ? stages_for_1cta(bn) : stages_for(mb, bn);
    if (tune && tune->stages >= 1 && tune->stages <= g.stages) g.stages = tune->stages;
    g.acc_bufs = (g.mb * ((bn + 31) & ~31) <= 256) ? 2 : 1;
    g.splits = 1; g.kb_per_split = (K + BK - 1) / BK; g.split_stride = 0;
    p->A = A; p->lda = lda; p->ldb = ldb;
    for (int i = 0; i < 3; ++i) p->Bs[i] = Bs[i < n_maps ? i : 0];
    return SFS_OK;
}

int32_t gemm_plan_enable_split(GemmPlan *p, float *ws, int32_t max_splits, const GemmTune *tune)
{
    GemmArgs &g = p->args;
    const bool f32_out = g.mode == GEMM_RESIDUAL_F32 || (g.mode == GEMM_STORE && g.out_f32 && g.vt == nullptr);
    if (!f32_out || ws == nullptr || max_splits < 2) return SFS_OK;
    int mb = g.mb, bn = g.bn, sp = 1;
    const bool one_cta = g.one_cta != 0;
    if (one_cta) pick_tile_1cta(g.M, g.K, g.mode, p->n_maps, p->n_per_map, num_sms(), max_splits, &bn, &sp);
    else pick_tile(g.M, g.K, g.mode, p->n_maps, p->n_per_map, num_sms() / 2, max_splits, &mb, &bn, &sp);
    if (tune) {
        if (tune->mb == 1 || tune->mb == 2) mb = tune->mb;
        if (tune->bn >= 32 && tune->bn <= 256 && (tune->bn % 16) == 0) bn = tune->bn;
        if (tune->splits >= 1 && tune->splits <= max_splits) sp = tune->splits;
    }
    if (sp <= 1 && !tune) return SFS_OK;
    // rebuild the plan at the new tile shape, then cut K
    GemmPlan q;
    GemmTune t2 = {one_cta ? 0 : mb, bn, tune ? tune->stages : 0, 0};
    int32_t rc = gemm_plan_create(&q, p->A, p->lda, g.M, g.K, p->Bs, p->n_maps, p->n_per_map, p->ldb, g.mode, g.C, g.ldc, g.out_f32,
                                  g.scale, g.vt, g.ldvt, g.vt_col0, &t2);
    if (rc != SFS_OK) return rc;
    *p = q;
    GemmArgs &h = p->args;
    const int num_kb = (h.K + BK - 1) / BK;
    if (sp > num_kb) sp = num_kb;
    if (sp > 1) {
        h.kb_per_split = (num_kb + sp - 1) / sp;
        h.splits = (num_kb + h.kb_per_split - 1) / h.kb_per_split;
        h.split_stride = (long long)h.M * h.ldc;
        h.C = ws;
    }
    return SFS_OK;
}

int32_t gemm_launch(const GemmPlan &p, const int32_t *d_m, const int32_t *d_active, int32_t *err, cudaStream_t stream)
{
    // always ask for more than half of an SM's shared memory: one CTA per SM, so the allocation of all 512
    // tensor-memory columns can never wait for a co-resident CTA
    static bool configured[kMaxDevices] = {};
    bool &done = configured[current_device_slot()];
    if (!done) {
        SFS_CUDA(cudaFuncSetAttribute(gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
        SFS_CUDA(cudaFuncSetAttribute(gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
        done = true;
    }
    GemmArgs g = p.args;
    g.d_m = d_m; g.err = err; g.d_active = d_active;
    if (g.one_cta) {
        static bool configured1[kMaxDevices] = {};
        bool &done1 = configured1[current_device_slot()];
        if (!done1) {
            SFS_CUDA(cudaFuncSetAttribute(gemm_kernel_1cta<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
            SFS_CUDA(cudaFuncSetAttribute(gemm_kernel_1cta<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
            done1 = true;
        }
        size_t smem1 = (size_t)g.stages * (A_BYTES + g.bn * BK * 2) + kBarBytes + kEpiStageBytes + 1024;
        if (smem1 < 120 * 1024) smem1 = 120 * 1024;            // one CTA per SM: all 512 tensor-memory columns are its own
        const long long tiles1 = (long long)((g.M + BM - 1) / BM) * g.n_col_tiles * g.splits;
        const int sms = num_sms();
        const unsigned grid1 = (unsigned)(tiles1 < sms ? tiles1 : sms);
        if (g.stats) SFS_CUDA(launch_pdl(gemm_kernel_1cta<true>, dim3(grid1), dim3(kGemmThreads), smem1, stream, p.tmA, p.tmB[0], p.tmB[1], p.tmB[2], g));
        else SFS_CUDA(launch_pdl(gemm_kernel_1cta<false>, dim3(grid1), dim3(kGemmThreads), smem1, stream, p.tmA, p.tmB[0], p.tmB[1], p.tmB[2], g));
        return SFS_OK;
    }
    size_t smem = (size_t)g.stages * (g.mb * A_BYTES + (g.bn / 2) * BK * 2) + kBarBytes + kEpiStageBytes + 1024;
    if (smem < 120 * 1024) smem = 120 * 1024;
    const long long tiles = (long long)((g.M + g.mb * 2 * BM - 1) / (g.mb * 2 * BM)) * g.n_col_tiles * g.splits;
    const int pairs = num_sms() / 2;
    dim3 grid((unsigned)(2 * (tiles < pairs ? tiles : pairs)), 1, 1);
    if (g.stats) SFS_CUDA(launch_pdl(gemm_kernel<true>, grid, dim3(kGemmThreads), smem, stream, p.tmA, p.tmB[0], p.tmB[1], p.tmB[2], g));
    else SFS_CUDA(launch_pdl(gemm_kernel<false>, grid, dim3(kGemmThreads), smem, stream, p.tmA, p.tmB[0], p.tmB[1], p.tmB[2], g));
    return SFS_OK;
}

}  // namespace sfs
