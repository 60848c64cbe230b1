// Memory-bound glue of the mask predictor's forward pass: embedding gather, RMSNorm (with optional row
// gather), rotary position embedding, and the RoPE table.  All of them move 16 bytes per thread per access.
#include "sfs_common.cuh"
#include "elementwise.cuh"

namespace sfs {
namespace {

// x[t, :] = E[tok[t], :]  (bf16 -> fp32 residual stream)
__global__ void embed_kernel(const int32_t *__restrict__ tokens, const __nv_bfloat16 *__restrict__ emb,
                             float *__restrict__ x, int T, int d, int vocab)
{
    pdl_wait();
    pdl_trigger();
    const int t = blockIdx.x;
    if (t >= T) return;
    int id = tokens[t];
    id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);         // out-of-range ids are clamped, never dereferenced
    const uint4 *src = reinterpret_cast<const uint4 *>(emb + (long long)id * d);
    float4 *dst = reinterpret_cast<float4 *>(x + (long long)t * d);
    for (int c = threadIdx.x; c < d / 8; c += blockDim.x) {
        const uint4 v = src[c];
        dst[2 * c]     = make_float4(bf16_bits_to_f32(v.x & 0xFFFFu), bf16_bits_to_f32(v.x >> 16),
                                     bf16_bits_to_f32(v.y & 0xFFFFu), bf16_bits_to_f32(v.y >> 16));
        dst[2 * c + 1] = make_float4(bf16_bits_to_f32(v.z & 0xFFFFu), bf16_bits_to_f32(v.z >> 16),
                                     bf16_bits_to_f32(v.w & 0xFFFFu), bf16_bits_to_f32(v.w >> 16));
    }
}

// h[r, :] = bf16( y * rsqrt(mean(y^2) + eps) * g ),  y = x[src(r), :] + sum_s partial[s][src(r), :],  src(r) = rows ? rows[r] : r.
// The partial products of a split-K projection are added in slab order (the sum does not depend on which CTA of the
// projection finished first); without a row list y is written back to x, so the residual stream is complete again.
// A thread keeps its part of the row in registers between the two passes (rows of up to kNormThreads * 16 elements).
constexpr int kNormThreads = 256;
constexpr int kNormRegChunks = 4;                          // float4 chunks a thread keeps
__global__ void __launch_bounds__(kNormThreads)
rmsnorm_kernel(float *__restrict__ x, const float *__restrict__ partial, int n_partial, long long partial_stride,
               const __nv_bfloat16 *__restrict__ gain, __nv_bfloat16 *__restrict__ h,
               const int32_t *__restrict__ rows, const int32_t *__restrict__ n_rows_ptr, int max_rows, int d, float eps)
{
    pdl_wait();
    pdl_trigger();
    const int n_rows = n_rows_ptr ? min(*n_rows_ptr, max_rows) : max_rows;
    __shared__ float s_part[kNormThreads / 32];
    const int chunks = d / 4;
    for (int r = blockIdx.x; r < n_rows; r += gridDim.x) {
        const long long src = rows ? rows[r] : r;
        float4 *xr = reinterpret_cast<float4 *>(x + src * d);
        const float4 *pr = reinterpret_cast<const float4 *>(partial + src * d);
        const long long pstride4 = partial_stride / 4;
        auto load = [&](int c) {                              // x + the partial products, slab by slab
            float4 v = xr[c];
            for (int s = 0; s < n_partial; ++s) {
                const float4 p = pr[(long long)s * pstride4 + c];
                v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
            }
            return v;
        };
        // the first kNormRegChunks chunks of a thread stay in registers (statically indexed); longer rows re-read the rest
        float4 keep[kNormRegChunks];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < kNormRegChunks; ++k) {
            const int c = threadIdx.x + k * kNormThreads;
            keep[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c < chunks) keep[k] = load(c);
        }
#pragma unroll
        for (int k = 0; k < kNormRegChunks; ++k) {
            const int c = threadIdx.x + k * kNormThreads;
            const float4 v = keep[k];
            if (c < chunks && n_partial > 0 && rows == nullptr) xr[c] = v;
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        for (int c = threadIdx.x + kNormRegChunks * kNormThreads; c < chunks; c += kNormThreads) {
            const float4 v = load(c);
            if (n_partial > 0 && rows == nullptr) xr[c] = v;
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ss = warp_sum(ss);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kNormThreads / 32; ++w) tot += s_part[w];
        const float inv = rsqrtf(tot / (float)d + eps);
        const uint2 *gp = reinterpret_cast<const uint2 *>(gain);
        uint2 *hp = reinterpret_cast<uint2 *>(h + (long long)r * d);
        auto emit = [&](int c, const float4 &v) {
            const uint2 g = gp[c];
            __nv_bfloat162 o0 = __floats2bfloat162_rn(v.x * inv * bf16_bits_to_f32(g.x & 0xFFFFu), v.y * inv * bf16_bits_to_f32(g.x >> 16));
            __nv_bfloat162 o1 = __floats2bfloat162_rn(v.z * inv * bf16_bits_to_f32(g.y & 0xFFFFu), v.w * inv * bf16_bits_to_f32(g.y >> 16));
            hp[c] = make_uint2(*reinterpret_cast<uint32_t *>(&o0), *reinterpret_cast<uint32_t *>(&o1));
        };
#pragma unroll
        for (int k = 0; k < kNormRegChunks; ++k) {
            const int c = threadIdx.x + k * kNormThreads;
            if (c < chunks) emit(c, keep[k]);
        }
        for (int c = threadIdx.x + kNormRegChunks * kNormThreads; c < chunks; c += kNormThreads) {
            // long rows: rebuild the value the first pass saw (x already holds it when it was written back)
            const float4 v = (rows == nullptr && n_partial > 0) ? xr[c] : load(c);
            emit(c, v);
        }
        __syncthreads();
    }
}

// table[pos, j] = (cos, sin)(pos * theta^(-2j/dh)), evaluated in double
__global__ void rope_table_kernel(float2 *table, int positions, int half, double theta)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= positions * half) return;
    const int pos = idx / half, j = idx % half;
    const double ang = (double)pos * pow(theta, -2.0 * (double)j / (double)(2 * half));
    table[idx] = make_float2((float)cos(ang), (float)sin(ang));
}

// in place on q and k: pairs (j, j + dh/2) of every head rotate by the angle of the token's position
__global__ void rope_kernel(__nv_bfloat16 *__restrict__ qk, long long ld, int T, int S, int n_heads, int dh,
                            const float2 *__restrict__ table, const int32_t *__restrict__ rows)
{
    // one thread handles 8 consecutive j of one (token, q-or-k, head)
    pdl_wait();
    pdl_trigger();
    const int half = dh / 2, groups = half / 8;
    const unsigned idx = blockIdx.x * blockDim.x + threadIdx.x;   // the launcher checks that the item count fits 31 bits
    const unsigned total = (unsigned)T * 2u * (unsigned)n_heads * (unsigned)groups;
    if (idx >= total) return;
    const unsigned per_token = (unsigned)groups * 2u * (unsigned)n_heads;
    const int t = (int)(idx / per_token);
    const unsigned rem = idx - (unsigned)t * per_token;
    const int hh = (int)(rem / (unsigned)groups);              // q heads then k heads: contiguous columns
    const int g = (int)(rem - (unsigned)hh * (unsigned)groups);
    const int pos = (rows ? rows[t] : t) % S;              // compact rows carry the token index they came from
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
}

}  // namespace

int32_t launch_embed(const int32_t *tokens, const void *emb, float *x, int T, int d, int vocab, cudaStream_t s)
{
    SFS_CUDA(launch_pdl(embed_kernel, dim3((unsigned)(T)), dim3((unsigned)(128)), (size_t)(0), s, tokens, reinterpret_cast<const __nv_bfloat16 *>(emb), x, T, d, vocab));
    return SFS_OK;
}

int32_t launch_rmsnorm(float *x, const float *partial, int n_partial, long long partial_stride, const void *gain, void *h,
                       const int32_t *rows, const int32_t *n_rows, int max_rows, int d, float eps, cudaStream_t s)
{
    if (max_rows <= 0) return SFS_OK;
    const int grid = max_rows < 148 * 16 ? max_rows : 148 * 16;
    if (partial == nullptr) n_partial = 0;
    SFS_CUDA(launch_pdl(rmsnorm_kernel, dim3(grid), dim3(kNormThreads), 0, s, x, partial ? partial : x, n_partial, partial_stride,
                        reinterpret_cast<const __nv_bfloat16 *>(gain), reinterpret_cast<__nv_bfloat16 *>(h), rows, n_rows, max_rows, d, eps));
    return SFS_OK;
}

int32_t launch_rope_table(float2 *table, int positions, int head_dim, float theta, cudaStream_t s)
{
    const int n = positions * (head_dim / 2);
    rope_table_kernel<<<(n + 255) / 256, 256, 0, s>>>(table, positions, head_dim / 2, (double)theta);
    SFS_LAUNCH_CHECK();
    return SFS_OK;
}

int32_t launch_rope(void *qk, int64_t ld, int T, int S, int n_heads, int head_dim, const float2 *table, const int32_t *rows, cudaStream_t s)
{
    const long long total = (long long)T * 2 * n_heads * (head_dim / 16);
    SFS_REQUIRE(total < (1LL << 31), SFS_ERR_INVALID_ARG, "rope: %lld items do not fit a 32-bit index", total);
    SFS_CUDA(launch_pdl(rope_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, s, reinterpret_cast<__nv_bfloat16 *>(qk), (long long)ld, T, S,
                        n_heads, head_dim, table, rows));
    return SFS_OK;
}

}  // namespace sfs
