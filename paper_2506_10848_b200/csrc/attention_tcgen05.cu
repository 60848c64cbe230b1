// Bidirectional (unmasked) multi-head attention of the mask predictor: out = softmax(q k^T / sqrt(dh)) v
// over all S positions of the same sequence.
//
// One CTA owns 128 query rows of one (sequence, head).  Warp 0 streams K tiles [128 keys x dh] and V^T tiles
// [dh x 128 keys] through two two-stage TMA rings.  Warp 1 issues tcgen05.mma: S_j = Q K_j^T into one of two score
// buffers in tensor memory, and O += P_j V_j into an accumulator that stays in tensor memory for the whole row of tiles;
// S_{j+1} is issued before P_j V_j, so the tensor core computes the next scores while the softmax runs.  Warps 2-9 (two
// threads per query row: each takes half of a tile's keys and half of the output columns) read S back with tcgen05.ld,
// run the online softmax in fp32 and write P as bf16 into shared memory in the 128-byte-swizzled K-major layout the
// next MMA consumes.  The exponentials use a reference maximum that is moved (with a rescale of O and of the denominator)
// only when the true running maximum has outgrown it by 2^8: the result is the same softmax, most tiles skip the pass
// over O.  V is consumed transposed (features x tokens); the QKV projection's epilogue writes it that way.
#include "sfs_common.cuh"
#include "tc05.cuh"
#include "attention.cuh"

namespace sfs {
namespace {

constexpr int kAttnThreads = 64 + 256;   // TMA warp, MMA warp, 8 softmax warps
constexpr int QT = 128;                 // query rows per CTA
constexpr int KT = 128;                 // keys per tile
constexpr int KV_STAGES = 2;
constexpr int kAttnBars = 4 * KV_STAGES + 6;   // K full/empty, V full/empty, Q, S (two), P, O, exchange

template <int DH>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmVt, AttnArgs a)
{
    constexpr int KB = DH / 64;                          // 64-element K-blocks along the head dimension
    constexpr int Q_BYTES = QT * DH * 2;
    constexpr int K_BYTES = KT * DH * 2;
    constexpr int V_BYTES = DH * KT * 2;
    constexpr int P_BYTES = QT * KT * 2;
    constexpr uint32_t TMEM_COLS = 512;                  // S (two buffers of 128 columns) and O (DH columns)

    pdl_trigger();                                       // (may run beside the end of the kernel before it: see pdl_wait below)
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem, *sK = smem + Q_BYTES, *sV = sK + KV_STAGES * K_BYTES, *sP = sV + KV_STAGES * V_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sP + P_BYTES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + kAttnBars);
    __shared__ int s_abort;
    __shared__ float s_xch[2][2][QT];                      // [tile parity][key half][row]: maxima (denominators at the end)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q0 = blockIdx.x * QT, h = blockIdx.y, b = blockIdx.z;
    const int S = a.S;
    const int tok0 = b * S;                                // first key / value token of this sequence
    const int qrow0 = b * a.kq + q0;                       // first query row of this CTA (queries may be a compact subset)
    const int nkv = (S + KT - 1) / KT;

    const uint32_t bar_kfull = tc::smem_u32(bars), bar_kempty = bar_kfull + 8 * KV_STAGES;
    const uint32_t bar_vfull = bar_kempty + 8 * KV_STAGES, bar_vempty = bar_vfull + 8 * KV_STAGES;
    const uint32_t bar_q = bar_vempty + 8 * KV_STAGES, bar_s = bar_q + 8 /* two */, bar_p = bar_q + 24, bar_o = bar_q + 32, bar_x = bar_q + 40;

    if (threadIdx.x == 0) {
        for (int s = 0; s < KV_STAGES; ++s) {
            tc::mbar_init(bar_kfull + 8 * s, 1); tc::mbar_init(bar_kempty + 8 * s, 1);
            tc::mbar_init(bar_vfull + 8 * s, 1); tc::mbar_init(bar_vempty + 8 * s, 1);
        }
        tc::mbar_init(bar_q, 1); tc::mbar_init(bar_s, 1); tc::mbar_init(bar_s + 8, 1);
        tc::mbar_init(bar_p, 256); tc::mbar_init(bar_o, 1); tc::mbar_init(bar_x, 256);
        s_abort = 0;
        tc::mbar_init_fence();
    }
    if (warp == 1) { tc::tmem_alloc(tc::smem_u32(tmem_slot), TMEM_COLS); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);
    const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 2 * KT;

    pdl_wait();                                          // the kernel before this one has completed: global memory from here on
    const bool live = !(a.d_active && *a.d_active == 0); // nothing left to decode: straight to the teardown (uniform)
    if (live) {
    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer: Q once, then K tiles and V^T tiles through their own rings (a K stage is free
            // again as soon as its S = Q K^T has been computed, a V stage after its P V)
            tc::mbar_expect_tx(bar_q, Q_BYTES);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
                tc::tma_load_2d(tc::smem_u32(sQ) + kb * (QT * 128), &tmQ, h * DH + kb * 64, qrow0, bar_q);
            int issued_k = 0, issued_v = 0;
            for (int j = 0; j < nkv; ++j) {
                const int s = j % KV_STAGES;
                const uint32_t ph = (uint32_t)(j / KV_STAGES) & 1u;
                if (!tc::mbar_wait(bar_kempty + 8 * s, ph ^ 1u, &s_abort)) break;
                const uint32_t sk = tc::smem_u32(sK) + s * K_BYTES;
                tc::mbar_expect_tx(bar_kfull + 8 * s, K_BYTES);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tc::tma_load_2d(sk + kb * (KT * 128), &tmK, a.k_col0 + h * DH + kb * 64, tok0 + j * KT, bar_kfull + 8 * s);
                issued_k = j + 1;
                if (!tc::mbar_wait(bar_vempty + 8 * s, ph ^ 1u, &s_abort)) break;
                const uint32_t sv = tc::smem_u32(sV) + s * V_BYTES;
                tc::mbar_expect_tx(bar_vfull + 8 * s, V_BYTES);
#pragma unroll
                for (int kb = 0; kb < KT / 64; ++kb)
                    tc::tma_load_2d(sv + kb * (DH * 128), &tmVt, tok0 + j * KT + kb * 64, h * DH, bar_vfull + 8 * s);
                issued_v = j + 1;
            }
            if (s_abort) {
                // give copies already in flight a bounded chance to land before the CTA retires
                for (int j = max(0, issued_k - KV_STAGES); j < issued_k; ++j) {
                    const uint32_t bar = bar_kfull + 8 * (j % KV_STAGES), ph = (uint32_t)(j / KV_STAGES) & 1u;
                    for (int i = 0; i < (1 << 16) && !tc::mbar_try(bar, ph); ++i) {}
                }
                for (int j = max(0, issued_v - KV_STAGES); j < issued_v; ++j) {
                    const uint32_t bar = bar_vfull + 8 * (j % KV_STAGES), ph = (uint32_t)(j / KV_STAGES) & 1u;
                    for (int i = 0; i < (1 << 16) && !tc::mbar_try(bar, ph); ++i) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer: the whole warp runs the loop with warp-uniform operands, one elected lane issues.
        // S_{j+1} = Q K_{j+1}^T is issued (into the other S buffer) before O += P_j V_j, so the tensor core computes the next
        // scores while the softmax warps work on the current ones.
        constexpr uint32_t idesc_s = tc::idesc_bf16_f32(QT, KT);
        constexpr uint32_t idesc_o = tc::idesc_bf16_f32(QT, DH);
        auto issue_S = [&](int j) {
            const int s = j % KV_STAGES;
            const uint32_t sk = tc::smem_u32(sK) + s * K_BYTES, d = tmem_S + (uint32_t)(j & 1) * KT;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                const uint64_t dq = tc::smem_desc_sw128(tc::smem_u32(sQ) + kb * (QT * 128));
                const uint64_t dk = tc::smem_desc_sw128(sk + kb * (KT * 128));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    tc::mma_bf16_elect(d, dq + (uint64_t)(kk * 2), dk + (uint64_t)(kk * 2), idesc_s, (kb | kk) != 0 ? 1u : 0u);
            }
            tc::mma_commit_elect(bar_s + 8 * (j & 1));
            tc::mma_commit_elect(bar_kempty + 8 * s);
        };
        bool ok = __all_sync(0xffffffffu, tc::mbar_wait(bar_q, 0, &s_abort));
        ok = ok && __all_sync(0xffffffffu, tc::mbar_wait(bar_kfull, 0, &s_abort));
        if (ok) { tc::tc_fence_after(); issue_S(0); }
        for (int j = 0; j < nkv && ok; ++j) {
            const int s = j % KV_STAGES;
            if (j + 1 < nkv) {
                // the S buffer of tile j+1 was last read for tile j-1, before the softmax warps arrived on bar_p (waited below)
                ok = __all_sync(0xffffffffu, tc::mbar_wait(bar_kfull + 8 * ((j + 1) % KV_STAGES), (uint32_t)((j + 1) / KV_STAGES) & 1u, &s_abort));
                if (!ok) break;
                tc::tc_fence_after();
                issue_S(j + 1);
            }
            ok = __all_sync(0xffffffffu, tc::mbar_wait(bar_vfull + 8 * s, (uint32_t)(j / KV_STAGES) & 1u, &s_abort));
            ok = ok && __all_sync(0xffffffffu, tc::mbar_wait(bar_p, (uint32_t)j & 1u, &s_abort));   // P_j written, O rescaled
            if (!ok) break;
            tc::tc_fence_after();
            const uint32_t sv = tc::smem_u32(sV) + s * V_BYTES;
#pragma unroll
            for (int kb = 0; kb < KT / 64; ++kb) {
                const uint64_t dp = tc::smem_desc_sw128(tc::smem_u32(sP) + kb * (QT * 128));
                const uint64_t dv = tc::smem_desc_sw128(sv + kb * (DH * 128));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    tc::mma_bf16_elect(tmem_O, dp + (uint64_t)(kk * 2), dv + (uint64_t)(kk * 2), idesc_o, (j | kb | kk) != 0 ? 1u : 0u);
            }
            tc::mma_commit_elect(bar_o);
            tc::mma_commit_elect(bar_vempty + 8 * s);
        }
    } else {
        // ---------------- online softmax: two threads per query row.  O accumulates in tensor memory over the tiles; the
        // exponentials are taken against a reference maximum that follows the true running maximum lazily: it is moved (and
        // O and the denominator rescaled) only when the true one has risen by more than 2^8, so most tiles need no pass over O.
        constexpr int HK = KT / 2;                         // keys of a tile per thread
        constexpr int HD = DH / 2;                         // output columns per thread
        constexpr float kLazy = 8.0f;                      // in log2 units: probabilities stay below 2^8
        const int qd = warp & 3, half = (warp - 2) >> 2;
        const int row = qd * 32 + lane;
        const uint32_t lane_off = (uint32_t)(qd * 32) << 16;
        const float c = a.scale_log2;                      // log2(e) / sqrt(dh)
        float m = -INFINITY, l = 0.f;                      // m: reference maximum; l: this thread's keys only
        bool ok = true;
        for (int j = 0; j < nkv && ok; ++j) {
            ok = tc::mbar_wait(bar_s + 8 * (j & 1), (uint32_t)(j >> 1) & 1u, &s_abort);
            if (!ok) break;
            tc::tc_fence_after();
            const int valid = min(KT, S - j * KT) - half * HK;     // keys of this thread's half that belong to the sequence
            uint32_t v[HK];
#pragma unroll
            for (int cc = 0; cc < HK / 32; ++cc) tc::tmem_ld32(tmem_S + (uint32_t)(j & 1) * KT + lane_off + half * HK + cc * 32, v + cc * 32);
            tc::tmem_ld_wait();
            const bool full = valid >= HK;                 // uniform over the warp: no per-key test on whole tiles
            float mx = -INFINITY;
            if (full) {
                float mx1 = -INFINITY;
#pragma unroll
                for (int i = 0; i < HK; i += 2) { mx = fmaxf(mx, __uint_as_float(v[i])); mx1 = fmaxf(mx1, __uint_as_float(v[i + 1])); }
                mx = fmaxf(mx, mx1);
            } else {
#pragma unroll
                for (int i = 0; i < HK; ++i)
                    if (i < valid) mx = fmaxf(mx, __uint_as_float(v[i]));
            }
            s_xch[j & 1][half][row] = mx;                  // exchange the two halves' maxima (bounded wait, like every other)
            tc::mbar_arrive(bar_x);
            ok = tc::mbar_wait(bar_x, (uint32_t)j & 1u, &s_abort);
            if (!ok) break;
            const float m_row = fmaxf(mx, s_xch[j & 1][half ^ 1][row]);   // both threads of a row see the same value
            if (j == 0) {
                m = m_row;
            } else {
                // P_{j-1} V_{j-1} has finished: O may be rescaled, and the P buffer rewritten
                ok = tc::mbar_wait(bar_o, (uint32_t)(j - 1) & 1u, &s_abort);
                if (!ok) break;
                const bool move = (m_row - m) * c > kLazy;
                if (__any_sync(0xffffffffu, move)) {
                    tc::tc_fence_after();
                    const float alpha = move ? tc::ex2_approx((m - m_row) * c) : 1.0f;
#pragma unroll
                    for (int cc = 0; cc < HD / 32; ++cc) {
                        uint32_t o[32];
                        tc::tmem_ld32(tmem_O + lane_off + half * HD + cc * 32, o);
                        tc::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tc::tmem_st32(tmem_O + lane_off + half * HD + cc * 32, o);
                    }
                    tc::tmem_st_wait();
                    if (move) { l *= alpha; m = m_row; }
                }
            }
            const float mc = m * c;
            float lsum = 0.f, lsum1 = 0.f;
#pragma unroll
            for (int cc = 0; cc < HK / 32; ++cc) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float p0 = tc::ex2_approx(fmaf(__uint_as_float(v[cc * 32 + 2 * i]), c, -mc));
                    float p1 = tc::ex2_approx(fmaf(__uint_as_float(v[cc * 32 + 2 * i + 1]), c, -mc));
                    if (!full) {
                        if (cc * 32 + 2 * i >= valid) p0 = 0.f;
                        if (cc * 32 + 2 * i + 1 >= valid) p1 = 0.f;
                    }
                    if (i & 1) lsum1 += p0 + p1; else lsum += p0 + p1;
                    __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
                    pk[i] = *reinterpret_cast<uint32_t *>(&hh);
                }
                // keys kc*32 .. kc*32+31 of this row (kc counts 32-key groups of the tile): K-block kc/2, 16-byte chunks
                // (kc%2)*4 .. +3, swizzled by row
                const int kc = half * (HK / 32) + cc;
                uint8_t *prow = sP + (kc >> 1) * (QT * 128) + row * 128;
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int chunk = ((kc & 1) * 4 + q4) ^ (row & 7);
                    *reinterpret_cast<uint4 *>(prow + chunk * 16) = make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
                }
            }
            l += lsum + lsum1;
            tc::fence_proxy_async_smem();                  // P visible to the tensor core's shared-memory reads
            tc::tc_fence_before();                         // S_j has been read, O has been rescaled
            tc::mbar_arrive(bar_p);
        }
        // the last P V, then the two halves of a row add their partial denominators
        ok = ok && tc::mbar_wait(bar_o, (uint32_t)(nkv - 1) & 1u, &s_abort);
        s_xch[nkv & 1][half][row] = l;
        tc::mbar_arrive(bar_x);
        ok = ok && tc::mbar_wait(bar_x, (uint32_t)nkv & 1u, &s_abort);
        if (ok && !s_abort) {
            tc::tc_fence_after();
            const float inv = 1.0f / (l + s_xch[nkv & 1][half ^ 1][row]);
            const bool live = q0 + row < a.kq;
            __nv_bfloat16 *dst = a.out + (long long)(qrow0 + row) * a.ld_out + h * DH + half * HD;
#pragma unroll
            for (int cc = 0; cc < HD / 32; ++cc) {
                uint32_t o[32];
                tc::tmem_ld32(tmem_O + lane_off + half * HD + cc * 32, o);      // warp-collective: every lane takes part
                tc::tmem_ld_wait();
                if (live) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t w[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 2 * t]) * inv, __uint_as_float(o[8 * i + 2 * t + 1]) * inv);
                            w[t] = *reinterpret_cast<uint32_t *>(&hh);
                        }
                        reinterpret_cast<uint4 *>(dst)[cc * 4 + i] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
    }
    }   // live

    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc(tmem_base, TMEM_COLS); }
    if (threadIdx.x == 0 && s_abort && a.err) atomicExch(a.err, SFS_ERR_TIMEOUT);
}

template <int DH>
int32_t launch_dh(const AttnPlan &p, int kq, const int32_t *d_active, int32_t *err, cudaStream_t stream)
{
    constexpr size_t smem = (size_t)QT * DH * 2 + KV_STAGES * (size_t)(KT * DH * 2 + DH * KT * 2) + QT * KT * 2
                          + kAttnBars * 8 + 16 + 1024;
    static bool configured[kMaxDevices] = {};
    bool &done = configured[current_device_slot()];
    if (!done) {
        SFS_CUDA(cudaFuncSetAttribute(attention_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        done = true;
    }
    AttnArgs a = p.args;
    a.err = err; a.d_active = d_active;
    if (kq > 0) a.kq = kq;
    dim3 grid((unsigned)((a.kq + QT - 1) / QT), (unsigned)a.n_heads, (unsigned)a.B);
    SFS_CUDA(launch_pdl(attention_kernel<DH>, grid, dim3(kAttnThreads), smem, stream, p.tmQ, p.tmK, p.tmVt, a));
    return SFS_OK;
}

}  // namespace

int32_t attn_plan_create_split(AttnPlan *p, const void *q, int64_t ld_q, const void *k, int64_t ld_k, int32_t k_cols, int32_t k_col0,
                               const void *vt, int64_t ld_vt, void *out, int64_t ld_out, int32_t B, int32_t S, int32_t n_heads, int32_t head_dim)
{
    SFS_REQUIRE(head_dim == 64 || head_dim == 128, SFS_ERR_UNSUPPORTED, "attention: head_dim %d (64 or 128 supported)", head_dim);
    SFS_REQUIRE((S % 8) == 0, SFS_ERR_UNSUPPORTED, "attention: sequence length %d must be a multiple of 8", S);
    SFS_REQUIRE(aligned_to(out, 16) && (ld_out % 8) == 0, SFS_ERR_INVALID_ARG, "attention: output must be 16-byte aligned");
    memset(p, 0, sizeof(*p));
    const int d = n_heads * head_dim;
    int32_t rc = make_tmap_bf16(&p->tmQ, q, (uint64_t)B * S, (uint64_t)d, (uint64_t)ld_q, 128);
    if (rc != SFS_OK) return rc;
    rc = make_tmap_bf16(&p->tmK, k, (uint64_t)B * S, (uint64_t)k_cols, (uint64_t)ld_k, 128);
    if (rc != SFS_OK) return rc;
    rc = make_tmap_bf16(&p->tmVt, vt, (uint64_t)d, (uint64_t)B * S, (uint64_t)ld_vt, (uint32_t)head_dim);
    if (rc != SFS_OK) return rc;
    AttnArgs &a = p->args;
    a.B = B; a.S = S; a.n_heads = n_heads; a.d_model = d; a.kq = S; a.k_col0 = k_col0;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)head_dim);
    a.out = reinterpret_cast<__nv_bfloat16 *>(out); a.ld_out = ld_out;
    p->head_dim = head_dim;
    return SFS_OK;
}

int32_t attn_plan_create(AttnPlan *p, const void *qkv, int64_t ld_qkv, const void *vt, int64_t ld_vt,
                         void *out, int64_t ld_out, int32_t B, int32_t S, int32_t n_heads, int32_t head_dim)
{
    const int d = n_heads * head_dim;
    return attn_plan_create_split(p, qkv, ld_qkv, qkv, ld_qkv, 2 * d, d, vt, ld_vt, out, ld_out, B, S, n_heads, head_dim);
}

int32_t attn_launch(const AttnPlan &p, const int32_t *d_active, int32_t *err, cudaStream_t stream)
{
    return attn_launch_queries(p, 0, d_active, err, stream);
}

int32_t attn_launch_queries(const AttnPlan &p, int32_t kq, const int32_t *d_active, int32_t *err, cudaStream_t stream)
{
    if (p.head_dim == 128) return launch_dh<128>(p, kq, d_active, err, stream);
    return launch_dh<64>(p, kq, d_active, err, stream);
}

}  // namespace sfs
