// Dense projections of the mask predictor (QKV / O / gate-up / down / LM head): C = A * B^T with bf16
// operands and fp32 accumulation in tensor memory.
//
// One CTA computes a 128 x BN output tile.  Warp 0 streams 128-byte-swizzled operand tiles into a ring of
// shared-memory stages with TMA, warp 1 issues tcgen05.mma (one elected thread) and releases stages with
// tcgen05.commit, warps 2-5 read the accumulator back with tcgen05.ld and run the fused epilogue
// (scale / fp32 residual add / SwiGLU / transposed V store).  The row count may live on the device, so the
// LM head can follow the shrinking set of masked rows without a host round trip.
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

constexpr int BM = 128, BK = 64;
constexpr int kGemmThreads = 192;
constexpr int A_BYTES = BM * BK * 2;

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

template <int BN, int STAGES>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
            const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, GemmArgs g)
{
    constexpr int B_BYTES = BN * BK * 2;
    constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr int HALF = BN / 2;

    if (g.d_active && *g.d_active == 0) return;             // nothing left to decode: uniform early exit
    const int M = g.d_m ? min(*g.d_m, g.M) : g.M;
    const int m_tile = blockIdx.x, n_tile = blockIdx.y;
    const int m0 = m_tile * BM;
    if (m0 >= M) return;                                    // uniform: before any barrier or allocation

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 1);
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (g.K + BK - 1) / BK;
    const uint32_t smem_base = tc::smem_u32(smem);
    const uint32_t bar_full = tc::smem_u32(bars), bar_empty = bar_full + 8 * STAGES, bar_tmem = bar_full + 16 * STAGES;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(bar_full + 8 * s, 1); tc::mbar_init(bar_empty + 8 * s, 1); }
        tc::mbar_init(bar_tmem, 1);
        s_abort = 0;
        tc::mbar_init_fence();
    }
    if (warp == 1) { tc::tmem_alloc(tc::smem_u32(tmem_slot), BN); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);

    // which B rows feed this tile
    const bool swiglu = (g.mode == GEMM_SWIGLU);
    const int map_idx = swiglu ? 0 : (n_tile / g.tiles_per_map);
    const int n_local = swiglu ? n_tile * HALF : (n_tile % g.tiles_per_map) * BN;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer
            tc::tma_prefetch_desc(&tmA);
            const CUtensorMap *mb0 = swiglu ? &tmB0 : (map_idx == 0 ? &tmB0 : (map_idx == 1 ? &tmB1 : &tmB2));
            const CUtensorMap *mb1 = swiglu ? &tmB1 : mb0;
            const int row1 = swiglu ? n_local : n_local + HALF;
            int issued = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
                if (!tc::mbar_wait(bar_empty + 8 * s, ph ^ 1u, &s_abort)) break;
                const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
                tc::mbar_expect_tx(bar_full + 8 * s, STAGE_BYTES);
                tc::tma_load_2d(sa, &tmA, kb * BK, m0, bar_full + 8 * s);
                tc::tma_load_2d(sb, mb0, kb * BK, n_local, bar_full + 8 * s);
                tc::tma_load_2d(sb + HALF * BK * 2, mb1, kb * BK, row1, bar_full + 8 * s);
                issued = kb + 1;
            }
            if (s_abort) {
                // give copies already in flight a bounded chance to land before the CTA retires
                for (int kb = max(0, issued - STAGES); kb < issued; ++kb) {
                    const uint32_t bar = bar_full + 8 * (kb % STAGES), ph = (uint32_t)(kb / STAGES) & 1u;
                    for (int i = 0; i < (1 << 16) && !tc::mbar_try(bar, ph); ++i) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer
            constexpr uint32_t idesc = tc::idesc_bf16_f32(BM, BN);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
                ok = tc::mbar_wait(bar_full + 8 * s, ph, &s_abort);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_BYTES;
                const uint64_t da = tc::smem_desc_sw128(sa), db = tc::smem_desc_sw128(sb);
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk)
                    tc::mma_bf16(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (kb | kk) != 0 ? 1u : 0u);
                tc::mma_commit(bar_empty + 8 * s);           // frees the stage once these MMAs have read it
            }
            tc::mma_commit(bar_tmem);                        // accumulator complete (or abandoned)
        }
    } else {
        // ---------------- epilogue: 4 warps, one TMEM lane quarter each
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int grow = m0 + row;
        const bool row_ok = grow < M;
        const bool ok = tc::mbar_wait(bar_tmem, 0, &s_abort) && !s_abort;
        tc::tc_fence_after();
        const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16);
        if (ok) {
            if (swiglu) {
                __nv_bfloat16 *C = reinterpret_cast<__nv_bfloat16 *>(g.C);
                for (int c = 0; c < HALF / 32; ++c) {
                    uint32_t gt[32], up[32];
                    tc::tmem_ld32(tbase + c * 32, gt);
                    tc::tmem_ld32(tbase + HALF + c * 32, up);
                    tc::tmem_ld_wait();
                    const int col0 = n_local + c * 32;
                    if (row_ok) {
                        __nv_bfloat16 *dst = C + (long long)grow * g.ldc + col0;
                        if (col0 + 32 <= g.N) {
                            uint32_t o[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float a = silu_f(__uint_as_float(gt[2 * j])) * __uint_as_float(up[2 * j]);
                                const float b = silu_f(__uint_as_float(gt[2 * j + 1])) * __uint_as_float(up[2 * j + 1]);
                                o[j] = pack_bf16(a, b);
                            }
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                reinterpret_cast<uint4 *>(dst)[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                        } else {
                            _Pragma("unroll")
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < g.N) dst[j] = __float2bfloat16_rn(silu_f(__uint_as_float(gt[j])) * __uint_as_float(up[j]));
                        }
                    }
                }
            } else {
                const int ncol0 = n_tile * BN;
                const bool to_vt = (g.vt != nullptr) && (ncol0 >= g.vt_col0);
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t v[32];
                    tc::tmem_ld32(tbase + c * 32, v);
                    tc::tmem_ld_wait();
                    const int col0 = ncol0 + c * 32;
                    if (!row_ok || col0 >= g.N) continue;
                    const bool full = col0 + 32 <= g.N;
                    if (g.mode == GEMM_RESIDUAL_F32) {
                        float *dst = reinterpret_cast<float *>(g.C) + (long long)grow * g.ldc + col0;
                        if (full) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                float4 x = reinterpret_cast<float4 *>(dst)[j];
                                x.x += __uint_as_float(v[4 * j]);     x.y += __uint_as_float(v[4 * j + 1]);
                                x.z += __uint_as_float(v[4 * j + 2]); x.w += __uint_as_float(v[4 * j + 3]);
                                reinterpret_cast<float4 *>(dst)[j] = x;
                            }
                        } else {
                            _Pragma("unroll")
                            for (int j = 0; j < 32; ++j) if (col0 + j < g.N) dst[j] += __uint_as_float(v[j]);
                        }
                    } else if (to_vt) {
                        // transposed store: 32 lanes hold 32 consecutive tokens of one feature column
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col0 + j < g.N)
                                g.vt[(long long)(col0 + j - g.vt_col0) * g.ldvt + grow] = __float2bfloat16_rn(__uint_as_float(v[j]) * g.scale);
                    } else if (g.out_f32) {
                        float *dst = reinterpret_cast<float *>(g.C) + (long long)grow * g.ldc + col0;
                        if (full) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                reinterpret_cast<float4 *>(dst)[j] = make_float4(__uint_as_float(v[4 * j]) * g.scale, __uint_as_float(v[4 * j + 1]) * g.scale,
                                                                                 __uint_as_float(v[4 * j + 2]) * g.scale, __uint_as_float(v[4 * j + 3]) * g.scale);
                        } else {
                            _Pragma("unroll")
                            for (int j = 0; j < 32; ++j) if (col0 + j < g.N) dst[j] = __uint_as_float(v[j]) * g.scale;
                        }
                    } else {
                        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(g.C) + (long long)grow * g.ldc + col0;
                        if (full) {
                            uint32_t o[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) o[j] = pack_bf16(__uint_as_float(v[2 * j]) * g.scale, __uint_as_float(v[2 * j + 1]) * g.scale);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                reinterpret_cast<uint4 *>(dst)[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                        } else {
                            _Pragma("unroll")
                            for (int j = 0; j < 32; ++j) if (col0 + j < g.N) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]) * g.scale);
                        }
                    }
                }
            }
        }
    }

    // ---------------- teardown
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc(tmem_base, BN); }
    if (threadIdx.x == 0 && s_abort && g.err) atomicExch(g.err, SFS_ERR_TIMEOUT);
}

template <int BN, int STAGES>
int32_t launch_cfg(const GemmPlan &p, const int32_t *d_m, const int32_t *d_active, int32_t *err, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)STAGES * (A_BYTES + BN * BK * 2) + (2 * STAGES + 1) * 8 + 16 + 1024;
    static bool configured = false;
    if (!configured) {
        SFS_CUDA(cudaFuncSetAttribute(gemm_kernel<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured = true;
    }
    GemmArgs g = p.args;
    g.d_m = d_m; g.err = err; g.d_active = d_active;
    const int cols_per_tile = (g.mode == GEMM_SWIGLU) ? BN / 2 : BN;
    int n_tiles;
    if (g.mode == GEMM_SWIGLU || p.n_maps == 1) { n_tiles = (g.N + cols_per_tile - 1) / cols_per_tile; g.tiles_per_map = 0x3FFFFFFF; }
    else { g.tiles_per_map = p.n_per_map / BN; n_tiles = g.tiles_per_map * p.n_maps; }
    dim3 grid((unsigned)((g.M + BM - 1) / BM), (unsigned)n_tiles, 1);
    gemm_kernel<BN, STAGES><<<grid, kGemmThreads, smem, stream>>>(p.tmA, p.tmB[0], p.tmB[1], p.tmB[2], g);
    SFS_LAUNCH_CHECK();
    return SFS_OK;
}

}  // namespace

int32_t gemm_plan_create(GemmPlan *p, const void *A, int64_t lda, int32_t M, int32_t K,
                         const void *const *Bs, int32_t n_maps, int32_t n_per_map, int64_t ldb,
                         int32_t mode, void *C, int64_t ldc, int32_t out_f32, float scale,
                         __nv_bfloat16 *vt, int64_t ldvt, int32_t vt_col0, int32_t force_bn)
{
    SFS_REQUIRE(M >= 1 && K >= 1 && n_per_map >= 1 && n_maps >= 1 && n_maps <= 3, SFS_ERR_INVALID_ARG, "gemm: bad sizes");
    SFS_REQUIRE((K % 8) == 0 && (lda % 8) == 0 && (ldb % 8) == 0, SFS_ERR_INVALID_ARG, "gemm: K, lda, ldb must be multiples of 8");
    SFS_REQUIRE(mode != GEMM_SWIGLU || n_maps == 2, SFS_ERR_INVALID_ARG, "gemm: SwiGLU takes two B matrices");
    memset(p, 0, sizeof(*p));
    const int N = (mode == GEMM_SWIGLU) ? n_per_map : n_per_map * n_maps;
    SFS_REQUIRE(aligned_to(C, 16) && (ldc % 8) == 0, SFS_ERR_INVALID_ARG, "gemm: C must be 16-byte aligned, ldc a multiple of 8");
    // tile width: wide tiles when they still fill the machine, else narrow ones
    const int m_tiles = (M + BM - 1) / BM;
    const int cols256 = (mode == GEMM_SWIGLU) ? 128 : 256;
    int bn = ((long long)m_tiles * ((N + cols256 - 1) / cols256) >= 148) ? 256 : 128;
    if (n_maps > 1 && mode != GEMM_SWIGLU && (n_per_map % 256) != 0) bn = 128;
    if (force_bn == 128 || force_bn == 256) bn = force_bn;
    SFS_REQUIRE(n_maps == 1 || mode == GEMM_SWIGLU || (n_per_map % bn) == 0, SFS_ERR_UNSUPPORTED,
                "gemm: concatenated outputs need a width that is a multiple of %d (got %d)", bn, n_per_map);
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
    return SFS_OK;
}

int32_t gemm_launch(const GemmPlan &p, const int32_t *d_m, const int32_t *d_active, int32_t *err, cudaStream_t stream)
{
    if (p.bn == 256) return launch_cfg<256, 4>(p, d_m, d_active, err, stream);
    return launch_cfg<128, 6>(p, d_m, d_active, err, stream);
}

}  // namespace sfs
