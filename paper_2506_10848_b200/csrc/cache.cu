// Feature cache of the mask predictor (the adaptive caching the paper's sampler integrates, Section 2.2 and the
// (K_p, K_r) settings of Table 4): value-similarity sums, the least-similar row choice, and the gathers / scatters
// that move the recomputed rows between the compact buffers the GEMMs work on and the per-layer caches.
#include "sfs_common.cuh"
#include "cache.cuh"

namespace sfs {
namespace {

// grid (ceil(tokens / 64), kSimSlices), 256 threads: lane = two neighbouring tokens, warp = every 8th feature of the slice
__global__ void __launch_bounds__(256)
sim_partial_kernel(const __nv_bfloat16 *__restrict__ a, const __nv_bfloat16 *__restrict__ b, long long ld, int d, int t_first, int t_end, int T,
                   float *__restrict__ partial)
{
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t0 = t_first + blockIdx.x * 64 + 2 * lane;             // t_first is even: 4-byte loads of two tokens stay aligned
    const int per = (d + kSimSlices - 1) / kSimSlices;
    const int f0 = blockIdx.y * per, f1 = min(d, f0 + per);
    float acc[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (t0 < t_end) {
        auto term = [&](uint32_t wa, uint32_t wb) {
            const float a0 = bf16_bits_to_f32(wa & 0xFFFFu), a1 = bf16_bits_to_f32(wa >> 16);
            const float b0 = bf16_bits_to_f32(wb & 0xFFFFu), b1 = bf16_bits_to_f32(wb >> 16);
            acc[0] = fmaf(a0, b0, acc[0]); acc[1] = fmaf(a0, a0, acc[1]); acc[2] = fmaf(b0, b0, acc[2]);
            acc[3] = fmaf(a1, b1, acc[3]); acc[4] = fmaf(a1, a1, acc[4]); acc[5] = fmaf(b1, b1, acc[5]);
        };
        int f = f0 + warp;
        for (; f + 24 < f1; f += 32) {                               // four features per round: eight loads in flight
            uint32_t wa[4], wb[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                wa[u] = *reinterpret_cast<const uint32_t *>(a + (long long)(f + 8 * u) * ld + t0);
                wb[u] = *reinterpret_cast<const uint32_t *>(b + (long long)(f + 8 * u) * ld + t0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) term(wa[u], wb[u]);           // same feature order as the plain loop
        }
        for (; f < f1; f += 8)
            term(*reinterpret_cast<const uint32_t *>(a + (long long)f * ld + t0), *reinterpret_cast<const uint32_t *>(b + (long long)f * ld + t0));
    }
    __shared__ float s[8][32][6];
#pragma unroll
    for (int i = 0; i < 6; ++i) s[warp][lane][i] = acc[i];
    __syncthreads();
    if (warp == 0 && t0 < t_end) {
        float r[6];
#pragma unroll
        for (int i = 0; i < 6; ++i) { r[i] = s[0][lane][i]; for (int w = 1; w < 8; ++w) r[i] += s[w][lane][i]; }   // fixed order
        float *o = partial + ((long long)blockIdx.y * T + t0) * 3;
        o[0] = r[0]; o[1] = r[1]; o[2] = r[2];
        if (t0 + 1 < t_end) { o[3] = r[3]; o[4] = r[4]; o[5] = r[5]; }
    }
}

__device__ __forceinline__ uint32_t float_order_key(float f) {       // monotone map float -> uint32
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// one CTA per sequence; dynamic shared memory: u64 keys[L], u8 chosen[L]
__global__ void __launch_bounds__(1024) cache_select_kernel(CacheSelectArgs a)
{
    pdl_wait();
    pdl_trigger();
    extern __shared__ __align__(16) unsigned long long s_key[];
    const int b = blockIdx.x, tid = threadIdx.x, L = a.L, P = a.P, S = a.S;
    int32_t *out = a.sel_rows + (long long)b * a.n_sel;
    int base = 0;
    if (a.refresh_p) {
        for (int i = tid; i < P; i += blockDim.x) out[i] = b * S + i;
        base = P;
    }
    if (a.refresh_r) {
        for (int i = tid; i < L; i += blockDim.x) out[base + i] = b * S + P + i;
    } else if (a.n_adapt > 0) {
        int lo = 0, hi = L;
        if (a.state != nullptr && a.state[b].phase == SFS_PHASE_FAST && !a.state[b].done) { lo = a.state[b].s_cycle; hi = a.state[b].hi; }
        lo = max(0, min(lo, L)); hi = max(lo, min(hi, L));
        for (int i = tid; i < L; i += blockDim.x) {
            float dot = 0.f, na = 0.f, nb = 0.f;
            const long long t = (long long)b * S + P + i;
            const float *__restrict__ part = a.partial;
            float pd[kSimSlices], pa[kSimSlices], pb[kSimSlices];
#pragma unroll
            for (int sl = 0; sl < kSimSlices; ++sl) {                // all loads first: one latency, not kSimSlices of them
                const float *p = part + ((long long)sl * a.T + t) * 3;
                pd[sl] = __ldg(p); pa[sl] = __ldg(p + 1); pb[sl] = __ldg(p + 2);
            }
#pragma unroll
            for (int sl = 0; sl < kSimSlices; ++sl) { dot += pd[sl]; na += pa[sl]; nb += pb[sl]; }   // fixed order
            const float den = __fmul_rn(__fsqrt_rn(na), __fsqrt_rn(nb));
            const float sim = den > 0.f ? __fdiv_rn(dot, den) : 0.f;
            if (a.sims_dump) a.sims_dump[(long long)b * L + i] = sim;
            s_key[i] = (i >= lo && i < hi) ? (((unsigned long long)float_order_key(sim) << 32) | (unsigned)i) : ~0ull;
        }
        const int Lp = (L + 1) & ~1;                               // keys are scanned two at a time: an odd L gets a sentinel
        if (tid == 0 && Lp != L) s_key[L] = ~0ull;
        __syncthreads();
        const int n_cand = hi - lo;
        const int k = min(a.n_adapt, n_cand);
        __shared__ int s_last, s_wcnt[32];
        if (tid == 0) s_last = -1;
        // rank by counting: candidate i is chosen when fewer than k candidate keys are smaller.  `parts` adjacent lanes share
        // a candidate, each counting over its own range of the keys (16-byte loads, two keys each).
        uint8_t *s_sel = reinterpret_cast<uint8_t *>(s_key + Lp);
        int parts = 1;
        while (parts < 32 && (long long)L * parts * 2 <= (long long)blockDim.x) parts *= 2;
        const int span = ((Lp / 2 + parts - 1) / parts) * 2;      // keys per part (even)
        const ulonglong2 *k2 = reinterpret_cast<const ulonglong2 *>(s_key);
        const int items = ((L * parts + 31) / 32) * 32;           // whole warps take part in the shuffles
        for (int it = tid; it < items; it += blockDim.x) {
            const int i = it / parts, part = it - i * parts;
            const unsigned long long ki = i < L ? s_key[i] : ~0ull;
            int rank = 0;
            if (ki != ~0ull) {
                const int j0 = part * span, j1 = min(Lp, j0 + span);
                for (int j = j0; j < j1; j += 2) { const ulonglong2 kk = k2[j >> 1]; rank += (kk.x < ki ? 1 : 0) + (kk.y < ki ? 1 : 0); }
            }
            for (int o = 1; o < parts; o <<= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
            if (part == 0 && i < L) s_sel[i] = (ki != ~0ull && rank < k) ? 1 : 0;
        }
        __syncthreads();
        // its slot in the ascending list is the number of chosen positions before it (ballots and per-warp counts)
        const int lane = tid & 31, warp = tid >> 5, n_warps = (int)blockDim.x >> 5;
        int run = 0;
        for (int i0 = 0; i0 < L; i0 += blockDim.x) {
            const int i = i0 + tid;
            const bool chosen = i < L && s_sel[i] != 0;
            const unsigned bal = __ballot_sync(0xffffffffu, chosen);
            if (lane == 0) s_wcnt[warp] = __popc(bal);
            __syncthreads();
            int before = run, total = 0;
            for (int w = 0; w < n_warps; ++w) { const int cnt = s_wcnt[w]; total += cnt; if (w < warp) before += cnt; }
            if (chosen) {
                const int slot = before + __popc(bal & ((1u << lane) - 1u));
                out[base + slot] = b * S + P + i;
                if (slot == k - 1) s_last = b * S + P + i;
            }
            run += total;
            __syncthreads();
        }
        const int pad = (k > 0) ? s_last : b * S + P;                  // nothing to choose from: recompute the first response row
        for (int j = k + tid; j < a.n_adapt; j += blockDim.x) out[base + j] = pad;
    }
    if (a.sets_dump) {
        __syncthreads();
        for (int j = tid; j < a.n_sel; j += blockDim.x) a.sets_dump[(long long)b * a.n_sel + j] = out[j];
    }
}

__global__ void gather_rows_bf16_kernel(const uint4 *__restrict__ src, const int32_t *__restrict__ rows, int chunks, uint4 *__restrict__ dst)
{
    pdl_wait();
    pdl_trigger();
    const int j = blockIdx.x;
    const uint4 *s = src + (long long)rows[j] * chunks;
    uint4 *o = dst + (long long)j * chunks;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) o[c] = s[c];
}

__global__ void scatter_rows_f32_kernel(const float4 *__restrict__ src, int n_slabs, long long slab_chunks, const int32_t *__restrict__ rows,
                                        int chunks, float4 *__restrict__ dst)
{
    pdl_wait();
    pdl_trigger();
    const int j = blockIdx.x;
    const float4 *s = src + (long long)j * chunks;
    float4 *o = dst + (long long)rows[j] * chunks;
    for (int c = blockIdx.y * blockDim.x + threadIdx.x; c < chunks; c += gridDim.y * blockDim.x) {
        float4 v = s[c];
        for (int k = 1; k < n_slabs; ++k) {                  // split-K partial products, added in slab order
            const float4 p = s[(long long)k * slab_chunks + c];
            v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
        }
        o[c] = v;
    }
}

// K rows: block j copies compact row j to its token row
__global__ void scatter_k_kernel(const __nv_bfloat16 *__restrict__ qk, long long ld_src, int col0, const int32_t *__restrict__ rows,
                                 int d, __nv_bfloat16 *__restrict__ k_dst)
{
    const int j = blockIdx.x;
    const uint4 *s = reinterpret_cast<const uint4 *>(qk + (long long)j * ld_src + col0);
    uint4 *o = reinterpret_cast<uint4 *>(k_dst + (long long)rows[j] * d);
    for (int c = threadIdx.x; c < d / 8; c += blockDim.x) o[c] = s[c];
}

// V^T columns: a block owns 8 features; compact rows run fastest over the threads, so the reads are contiguous
__global__ void scatter_vt_kernel(const __nv_bfloat16 *__restrict__ vt_src, long long ld_vt_src, const int32_t *__restrict__ rows, int n_rows,
                                  int d, __nv_bfloat16 *__restrict__ vt_dst, long long ld_vt_dst)
{
    const int f0 = blockIdx.x * 8;
    for (int idx = threadIdx.x; idx < 8 * n_rows; idx += blockDim.x) {
        const int f = f0 + idx / n_rows, j = idx - (idx / n_rows) * n_rows;
        if (f < d) vt_dst[(long long)f * ld_vt_dst + rows[j]] = vt_src[(long long)f * ld_vt_src + j];
    }
}

// One launch for what follows the QKV projection of the recomputed rows: the rotary embedding of q and k (in place, on the
// compact rows; the arithmetic of rope_kernel), the rotated k also written to the token's row of the K cache, and the new
// value columns scattered into V^T.  Blocks [0, rope_blocks) rotate, the rest scatter values (8 features per block).
__global__ void __launch_bounds__(256)
rope_scatter_kv_kernel(__nv_bfloat16 *__restrict__ qk, long long ld, int n_rows, int S, int n_heads, int dh, const float2 *__restrict__ table,
                       const int32_t *__restrict__ rows, __nv_bfloat16 *__restrict__ k_dst, const __nv_bfloat16 *__restrict__ vt_src,
                       long long ld_vt_src, __nv_bfloat16 *__restrict__ vt_dst, long long ld_vt_dst, int rope_blocks)
{
    pdl_wait();
    pdl_trigger();
    const int d = n_heads * dh;
    if ((int)blockIdx.x >= rope_blocks) {
        const int f0 = ((int)blockIdx.x - rope_blocks) * 8;
        for (int idx = threadIdx.x; idx < 8 * n_rows; idx += blockDim.x) {
            const int f = f0 + idx / n_rows, j = idx - (idx / n_rows) * n_rows;
            if (f < d) vt_dst[(long long)f * ld_vt_dst + rows[j]] = vt_src[(long long)f * ld_vt_src + j];
        }
        return;
    }
    const int half = dh / 2, groups = half / 8;
    const unsigned idx = blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned total = (unsigned)n_rows * 2u * (unsigned)n_heads * (unsigned)groups;
    if (idx >= total) return;
    const unsigned per_token = (unsigned)groups * 2u * (unsigned)n_heads;
    const int t = (int)(idx / per_token);
    const unsigned rem = idx - (unsigned)t * per_token;
    const int hh = (int)(rem / (unsigned)groups);              // q heads then k heads: contiguous columns
    const int g = (int)(rem - (unsigned)hh * (unsigned)groups);
    const int tok = rows[t], pos = tok % S;
    __nv_bfloat16 *base = qk + (long long)t * ld + (long long)hh * dh + g * 8;
    uint4 lo = *reinterpret_cast<uint4 *>(base), hi = *reinterpret_cast<uint4 *>(base + half);
    const float2 *tb = table + (long long)pos * half + g * 8;
    uint32_t *lw = reinterpret_cast<uint32_t *>(&lo), *hw = reinterpret_cast<uint32_t *>(&hi);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        float x1[2] = {bf16_bits_to_f32(lw[w] & 0xFFFFu), bf16_bits_to_f32(lw[w] >> 16)};
        float x2[2] = {bf16_bits_to_f32(hw[w] & 0xFFFFu), bf16_bits_to_f32(hw[w] >> 16)};
        float o1[2], o2[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float2 cs = tb[2 * w + e];
            o1[e] = x1[e] * cs.x - x2[e] * cs.y;
            o2[e] = x2[e] * cs.x + x1[e] * cs.y;
        }
        __nv_bfloat162 a = __floats2bfloat162_rn(o1[0], o1[1]), b2 = __floats2bfloat162_rn(o2[0], o2[1]);
        lw[w] = *reinterpret_cast<uint32_t *>(&a);
        hw[w] = *reinterpret_cast<uint32_t *>(&b2);
    }
    *reinterpret_cast<uint4 *>(base) = lo;
    *reinterpret_cast<uint4 *>(base + half) = hi;
    if (hh >= n_heads) {                                       // a key head: also the token's row of the K cache
        __nv_bfloat16 *kd = k_dst + (long long)tok * d + (long long)(hh - n_heads) * dh + g * 8;
        *reinterpret_cast<uint4 *>(kd) = lo;
        *reinterpret_cast<uint4 *>(kd + half) = hi;
    }
}

// One launch for what follows the output projection of the recomputed rows: the split-K slabs of compact row j are added in
// slab order into the attention increment of its token (inc[rows[j]] = sum of slabs), and the MLP branch's input
// h[j] = bf16(RMSNorm(x[rows[j]] + inc[rows[j]]) * gain) is written to the compact buffer.
__global__ void __launch_bounds__(1024)
fold_norm_rows_kernel(const float *__restrict__ slabs, int n_slabs, long long slab_stride, const int32_t *__restrict__ rows,
                      const float *__restrict__ x, float *__restrict__ inc, const __nv_bfloat16 *__restrict__ gain,
                      __nv_bfloat16 *__restrict__ h, int d, float eps)
{
    pdl_wait();
    pdl_trigger();
    const int j = blockIdx.x, chunks = d / 4;
    const long long src = rows[j];
    const float4 *sp = reinterpret_cast<const float4 *>(slabs + (long long)j * d);
    const float4 *xr = reinterpret_cast<const float4 *>(x + src * d);
    float4 *ir = reinterpret_cast<float4 *>(inc + src * d);
    __shared__ float s_part[32];
    extern __shared__ float4 s_y[];                            // the row, kept between the two passes
    float ss = 0.f;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        float4 v = sp[c];
        for (int k = 1; k < n_slabs; ++k) {
            const float4 p = sp[(long long)k * (slab_stride / 4) + c];
            v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
        }
        ir[c] = v;
        const float4 xv = xr[c];
        const float4 y = make_float4(xv.x + v.x, xv.y + v.y, xv.z + v.z, xv.w + v.w);
        s_y[c] = y;
        ss += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < ((int)blockDim.x >> 5); ++w) tot += s_part[w];
    const float inv = rsqrtf(tot / (float)d + eps);
    const uint2 *gp = reinterpret_cast<const uint2 *>(gain);
    uint2 *hp = reinterpret_cast<uint2 *>(h + (long long)j * d);
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        const float4 v = s_y[c];
        const uint2 g = gp[c];
        __nv_bfloat162 o0 = __floats2bfloat162_rn(v.x * inv * bf16_bits_to_f32(g.x & 0xFFFFu), v.y * inv * bf16_bits_to_f32(g.x >> 16));
        __nv_bfloat162 o1 = __floats2bfloat162_rn(v.z * inv * bf16_bits_to_f32(g.y & 0xFFFFu), v.w * inv * bf16_bits_to_f32(g.y >> 16));
        hp[c] = make_uint2(*reinterpret_cast<uint32_t *>(&o0), *reinterpret_cast<uint32_t *>(&o1));
    }
}

}  // namespace

int32_t launch_rope_scatter_kv(void *qk, long long ld, int n_rows, int S, int n_heads, int head_dim, const float2 *table, const int32_t *rows,
                               void *k_dst, const void *vt_src, long long ld_vt_src, void *vt_dst, long long ld_vt_dst, cudaStream_t s)
{
    if (n_rows <= 0) return SFS_OK;
    const long long total = (long long)n_rows * 2 * n_heads * (head_dim / 16);
    SFS_REQUIRE(total < (1LL << 31), SFS_ERR_INVALID_ARG, "rope: %lld items do not fit a 32-bit index", total);
    const int rope_blocks = (int)((total + 255) / 256), d = n_heads * head_dim;
    SFS_CUDA(launch_pdl(rope_scatter_kv_kernel, dim3((unsigned)(rope_blocks + (d + 7) / 8)), dim3((unsigned)(256)), (size_t)(0), s, reinterpret_cast<__nv_bfloat16 *>(qk), ld, n_rows, S, n_heads, head_dim, table, rows,
                                                                      reinterpret_cast<__nv_bfloat16 *>(k_dst), reinterpret_cast<const __nv_bfloat16 *>(vt_src),
                                                                      ld_vt_src, reinterpret_cast<__nv_bfloat16 *>(vt_dst), ld_vt_dst, rope_blocks));
    return SFS_OK;
}

int32_t launch_fold_norm_rows(const float *slabs, int n_slabs, long long slab_stride, const int32_t *rows, int n_rows, const float *x, float *inc,
                              const void *gain, void *h, int d, float eps, cudaStream_t s)
{
    if (n_rows <= 0) return SFS_OK;
    SFS_REQUIRE((size_t)d * 4 <= 96 * 1024, SFS_ERR_UNSUPPORTED, "d_model %d too wide for the fused fold + norm", d);
    const size_t smem = (size_t)d * 4;
    if (smem > 48 * 1024) SFS_CUDA(cudaFuncSetAttribute(fold_norm_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    SFS_CUDA(launch_pdl(fold_norm_rows_kernel, dim3((unsigned)(n_rows)), dim3((unsigned)(d >= 4096 ? 1024 : (d >= 2048 ? 512 : 256))), (size_t)(smem), s, slabs, n_slabs < 1 ? 1 : n_slabs, slab_stride, rows, x, inc, reinterpret_cast<const __nv_bfloat16 *>(gain),
                                                    reinterpret_cast<__nv_bfloat16 *>(h), d, eps));
    return SFS_OK;
}

int32_t launch_sim_partial(const void *vnew_t, const void *vold_t, long long ld, int d, int t_first, int t_count, int T, float *partial,
                           cudaStream_t s)
{
    if (t_count <= 0) return SFS_OK;
    SFS_REQUIRE((t_first % 2) == 0 && (ld % 2) == 0, SFS_ERR_INVALID_ARG, "similarity: first token and row stride must be even");
    dim3 grid((unsigned)((t_count + 63) / 64), kSimSlices, 1);
    SFS_CUDA(launch_pdl(sim_partial_kernel, grid, dim3((unsigned)(256)), (size_t)(0), s, reinterpret_cast<const __nv_bfloat16 *>(vnew_t), reinterpret_cast<const __nv_bfloat16 *>(vold_t),
                                            ld, d, t_first, t_first + t_count, T, partial));
    return SFS_OK;
}

int32_t launch_cache_select(const CacheSelectArgs &a, cudaStream_t s)
{
    // 1024 threads: the ranking is O(L^2 / threads); shared memory: the keys (an even number of them), then one byte per position
    SFS_CUDA(launch_pdl(cache_select_kernel, dim3((unsigned)(a.B)), dim3((unsigned)(1024)), (size_t)((size_t)(a.L + 1) * 9 + 16), s, a));
    return SFS_OK;
}

int32_t launch_gather_rows_bf16(const void *src, const int32_t *rows, int n_rows, int d, void *dst, cudaStream_t s)
{
    if (n_rows <= 0) return SFS_OK;
    SFS_CUDA(launch_pdl(gather_rows_bf16_kernel, dim3((unsigned)(n_rows)), dim3((unsigned)(128)), (size_t)(0), s, reinterpret_cast<const uint4 *>(src), rows, d / 8, reinterpret_cast<uint4 *>(dst)));
    return SFS_OK;
}

int32_t launch_scatter_rows_f32(const float *src, int n_slabs, long long slab_stride, const int32_t *rows, int n_rows, int d, float *dst,
                                cudaStream_t s)
{
    if (n_rows <= 0) return SFS_OK;
    SFS_CUDA(launch_pdl(scatter_rows_f32_kernel, dim3((unsigned)n_rows, 4, 1), dim3((unsigned)(256)), (size_t)(0), s, reinterpret_cast<const float4 *>(src), n_slabs < 1 ? 1 : n_slabs, slab_stride / 4, rows, d / 4,
                                                   reinterpret_cast<float4 *>(dst)));
    return SFS_OK;
}

int32_t launch_scatter_kv(const void *qk_src, long long ld_src, int col0, const void *vt_src, long long ld_vt_src,
                          const int32_t *rows, int n_rows, int d, void *k_dst, void *vt_dst, long long ld_vt_dst, cudaStream_t s)
{
    if (n_rows <= 0) return SFS_OK;
    scatter_k_kernel<<<n_rows, 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16 *>(qk_src), ld_src, col0, rows, d,
                                            reinterpret_cast<__nv_bfloat16 *>(k_dst));
    SFS_LAUNCH_CHECK();
    scatter_vt_kernel<<<(d + 7) / 8, 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16 *>(vt_src), ld_vt_src, rows, n_rows, d,
                                                  reinterpret_cast<__nv_bfloat16 *>(vt_dst), ld_vt_dst);
    SFS_LAUNCH_CHECK();
    return SFS_OK;
}

}  // namespace sfs
