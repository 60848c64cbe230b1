// Row statistics of the sampling epilogue (paper Section 3.1): per logits row the greedy token
// r_hat = argmax_v x_v and the canonical fixed-point softmax denominator S_q (c = 2^28 / S_q).
//
// Fast paths (bf16 logits): a thread-block cluster owns one row and HBM is read exactly once.  Pass 1 finds the exact row
// maximum, the CTAs push their slice maxima to each other through distributed shared memory (one cluster barrier), pass 2
// evaluates the fixed-point exponentials with packed f32x2 arithmetic and sums them as integers; sums and first-maximum
// candidates reach rank 0 by remote shared-memory atomics.  Integer sums make the result independent of how the row is
// split over threads, warps and CTAs.  Rows of 128 KB and more are staged: each of 8 CTAs brings its contiguous slice into
// shared memory with one bulk asynchronous copy (no registers tied up in flight, seven CTAs per SM); shorter rows stay in
// registers (every thread keeps its 16-byte chunks between the passes).
//
// Generic path (bf16 or fp32, any vocabulary size or stride): one CTA per row, two sweeps over global memory.
#include "sfs_common.cuh"

#include <cooperative_groups.h>
namespace cg = cooperative_groups;

namespace sfs {
namespace {

constexpr float kLog2e = 0x1.715476p+0f;
constexpr float kLn2   = 0x1.62e430p-1f;
constexpr float kMagic = 12582912.0f;           // 1.5 * 2^23
constexpr float kC1 = 0x1.fffa48p-1f;
constexpr float kC2 = 0x1.fff8fcp-2f;
constexpr float kC3 = 0x1.57f67cp-3f;
constexpr float kC4 = 0x1.57de66p-5f;
constexpr uint32_t kShiftBase = 0x4B400003u;    // bits(kMagic) + 3

__device__ __forceinline__ uint32_t shr_clamp(uint32_t x, uint32_t s) {
    uint32_t r;
    asm("shr.u32 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(s));   // PTX semantics: shift >= 32 gives 0
    return r;
}

// one term e_v = trunc(2^28 * exp(x - m)), scalar form (generic kernel)
__device__ __forceinline__ uint32_t canon_term(float x, float m) {
    const float d = __fsub_rn(x, m);
    const float r = __fmaf_rn(d, kLog2e, kMagic);
    const float n = __fsub_rn(r, kMagic);
    const float f = __fmaf_rn(n, -kLn2, d);
    float q = __fmaf_rn(f, kC4, kC3);
    q = __fmaf_rn(f, q, kC2);
    q = __fmaf_rn(f, q, kC1);
    const float P = __fmaf_rn(f, q, 3.0f);
    return shr_clamp(__float_as_uint(P) << 9, kShiftBase - __float_as_uint(r));
}

// ---- packed f32x2 arithmetic (two lanes per instruction) ----------------------------------------------
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, uint32_t &lo, uint32_t &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r;
}

struct Consts2 { f32x2 negm, l2e, magic, negmagic, negln2, c1, c2, c3, c4, three; };

// two terms from one 32-bit word holding two bf16 logits; returns e_lo + e_hi (each < 1.42 * 2^28)
__device__ __forceinline__ uint32_t canon_pair(uint32_t w, const Consts2 &k) {
    const f32x2 x = pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    const f32x2 d = add2(x, k.negm);
    const f32x2 r = fma2(d, k.l2e, k.magic);
    const f32x2 n = add2(r, k.negmagic);
    const f32x2 f = fma2(n, k.negln2, d);
    f32x2 q = fma2(f, k.c4, k.c3);
    q = fma2(f, q, k.c2);
    q = fma2(f, q, k.c1);
    const f32x2 P = fma2(f, q, k.three);
    uint32_t r0, r1, p0, p1;
    unpack2(r, r0, r1);
    unpack2(P, p0, p1);
    return shr_clamp(p0 << 9, kShiftBase - r0) + shr_clamp(p1 << 9, kShiftBase - r1);
}

// orders this thread's shared-memory traffic inside the cluster (cheaper than a device-wide fence)
__device__ __forceinline__ void cluster_fence() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) { return *reinterpret_cast<__nv_bfloat162 *>(&w); }
__device__ __forceinline__ float bf162_max(uint32_t w) {
    return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

struct RowOut {
    const int32_t *rows;            // flat token index per logits row, or null
    int32_t *argmax; unsigned long long *sq; float *conf;       // dense by logits row (optional)
    unsigned long long *pos_sq; int32_t *pos_arg;               // scattered by flat token index (optional)
    int32_t n_positions;                                        // size of the scattered arrays
    int32_t *err;                                               // device status word (optional)
};

__device__ __forceinline__ void write_row(const RowOut &o, int row, int arg, unsigned long long S) {
    if (o.argmax) o.argmax[row] = arg;
    if (o.sq) o.sq[row] = S;
    if (o.conf) o.conf[row] = (float)((double)(1u << SFS_CONF_QBITS) / (double)S);
    if (o.rows && o.pos_sq) {
        const int p = o.rows[row];
        if ((unsigned)p < (unsigned)o.n_positions) {
            o.pos_sq[p] = S;
            o.pos_arg[p] = arg;
        } else if (o.err) {
            atomicExch(o.err, SFS_ERR_INVALID_ARG);               // a row index outside the token grid: skipped, reported
        }
    }
}

constexpr int kThreads = 256;
constexpr uint32_t kNegInf2 = 0xFF80FF80u;

// One cluster (1, 2, 4 or 8 CTAs) per logits row; NV 16-byte chunks per thread.
template <int NV>
__global__ void __launch_bounds__(kThreads, 4)
rowstats_cluster_bf16(const uint4 *__restrict__ logits, long long ld_chunks, int nchunks, int vocab,
                      const int32_t *__restrict__ n_rows_ptr, int max_rows, RowOut out, int32_t *err)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int C    = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int row  = blockIdx.x / C;
    const int n_rows = n_rows_ptr ? min(*n_rows_ptr, max_rows) : max_rows;
    if (row >= n_rows) return;                              // uniform over the cluster

    __shared__ float s_wmax[kThreads / 32];
    __shared__ unsigned long long s_wsum[kThreads / 32];
    __shared__ float s_max_of[8];                           // slice maxima of all CTAs of the cluster, pushed by their owners
    __shared__ unsigned long long s_row_sum;                // rank 0 only: the peers add their sums here ...
    __shared__ int s_row_arg, s_arrived;                    // ... and their first-maximum candidates, then count themselves in
    __shared__ int s_cta_arg;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4 *rp = logits + (long long)row * ld_chunks;

    // ---- the only pass over HBM: this thread's chunks of the row, kept in registers
    uint4 v[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const int chunk = (j * C + rank) * kThreads + tid;
        v[j] = (chunk < nchunks) ? ld_stream(rp + chunk) : make_uint4(kNegInf2, kNegInf2, kNegInf2, kNegInf2);
    }
    if (tid == 0) { s_cta_arg = 0x7FFFFFFF; s_row_sum = 0; s_row_arg = 0x7FFFFFFF; s_arrived = 0; }

    // ---- pass 1: exact maximum
    __nv_bfloat162 mx = as_bf162(kNegInf2);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        mx = __hmax2(mx, __hmax2(__hmax2(as_bf162(v[j].x), as_bf162(v[j].y)), __hmax2(as_bf162(v[j].z), as_bf162(v[j].w))));
    }
    const float lmax = bf162_max(*reinterpret_cast<uint32_t *>(&mx));
    float m = warp_max(lmax);
    if (lane == 0) s_wmax[warp] = m;
    __syncthreads();
    if (C > 1) {
        // every CTA pushes its slice maximum into every CTA's table; after the one cluster barrier nobody reads a peer's
        // shared memory any more (only rank 0's is written to, and rank 0 stays until everybody has reported)
        if (tid < C) {
            float t = s_wmax[0];
#pragma unroll
            for (int w = 1; w < kThreads / 32; ++w) t = fmaxf(t, s_wmax[w]);
            *cluster.map_shared_rank(&s_max_of[rank], tid) = t;
        }
        cluster.sync();
        m = s_max_of[0];
        for (int r = 1; r < C; ++r) m = fmaxf(m, s_max_of[r]);
    } else {
        m = s_wmax[0];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) m = fmaxf(m, s_wmax[w]);
    }

    // ---- first position of the maximum (only threads that hold it look)
    if (lmax == m) {
        int best = 0x7FFFFFFF;
#pragma unroll
        for (int j = NV - 1; j >= 0; --j) {
            const int chunk = (j * C + rank) * kThreads + tid;
            const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
            for (int e = 7; e >= 0; --e) {
                const float x = (e & 1) ? __uint_as_float(w[e >> 1] & 0xFFFF0000u) : __uint_as_float(w[e >> 1] << 16);
                const int idx = chunk * 8 + e;
                if (x == m && idx < vocab) best = idx;
            }
        }
        if (best != 0x7FFFFFFF) atomicMin(&s_cta_arg, best);
    }

    // ---- pass 2: fixed-point exponentials, integer sum
    Consts2 k;
    k.negm = pack2(-m, -m);           k.l2e = pack2(kLog2e, kLog2e);
    k.magic = pack2(kMagic, kMagic);  k.negmagic = pack2(-kMagic, -kMagic);
    k.negln2 = pack2(-kLn2, -kLn2);
    k.c1 = pack2(kC1, kC1); k.c2 = pack2(kC2, kC2); k.c3 = pack2(kC3, kC3); k.c4 = pack2(kC4, kC4);
    k.three = pack2(3.0f, 3.0f);
    unsigned long long acc = 0;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const uint32_t a = canon_pair(v[j].x, k) + canon_pair(v[j].y, k) + canon_pair(v[j].z, k) + canon_pair(v[j].w, k);
        acc += a;                                           // 8 terms < 8 * 1.42 * 2^28 < 2^32
    }
    acc = warp_sum_u64(acc);
    if (lane == 0) s_wsum[warp] = acc;
    __syncthreads();
    if (tid == 0) {
        unsigned long long t = 0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) t += s_wsum[w];
        const int arg = s_cta_arg;
        if (C > 1) {
            // report to rank 0 (integer adds and a minimum: any arrival order gives the same result), then leave
            unsigned long long *rs = cluster.map_shared_rank(&s_row_sum, 0);
            int *ra = cluster.map_shared_rank(&s_row_arg, 0), *rn = cluster.map_shared_rank(&s_arrived, 0);
            atomicAdd(rs, t);
            atomicMin(ra, arg);
            cluster_fence();
            atomicAdd(rn, 1);
            if (rank == 0) {
                int spins = 0;
                while (*reinterpret_cast<volatile int *>(&s_arrived) < C && ++spins < (1 << 24)) {}
                if (spins >= (1 << 24) && err) atomicExch(err, SFS_ERR_TIMEOUT);   // a peer never reported
                cluster_fence();
                const int a2 = *reinterpret_cast<volatile int *>(&s_row_arg);
                write_row(out, row, a2 == 0x7FFFFFFF ? 0 : a2, *reinterpret_cast<volatile unsigned long long *>(&s_row_sum));
            }
        } else {
            write_row(out, row, arg == 0x7FFFFFFF ? 0 : arg, t);
        }
    }
}

// ---- long rows: slices staged in shared memory ------------------------------------------------------------------
// Same arithmetic, other staging: a cluster of 8 CTAs of 128 threads owns a row, and each CTA brings its contiguous slice
// into shared memory with ONE bulk asynchronous copy, so no registers are tied up while the bytes are in flight and seven
// CTAs (seven 32 KB slices) fit an SM instead of four.  The two passes then read shared memory.
constexpr int kStagedThreads = 128;
constexpr int kStagedCluster = 8;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(kStagedThreads)
rowstats_staged_bf16(const uint4 *__restrict__ logits, long long ld_chunks, int nchunks, int per_cta, int vocab,
                     const int32_t *__restrict__ n_rows_ptr, int max_rows, RowOut out, int32_t *err)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int C    = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int row  = blockIdx.x / C;
    const int n_rows = n_rows_ptr ? min(*n_rows_ptr, max_rows) : max_rows;
    if (row >= n_rows) return;                              // uniform over the cluster

    extern __shared__ __align__(16) uint4 s_slice[];
    __shared__ __align__(8) unsigned long long s_bar;
    __shared__ float s_wmax[kStagedThreads / 32];
    __shared__ unsigned long long s_wsum[kStagedThreads / 32];
    __shared__ float s_max_of[kStagedCluster];
    __shared__ unsigned long long s_row_sum;
    __shared__ int s_row_arg, s_arrived, s_cta_arg;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c0 = rank * per_cta;                          // first 16-byte chunk of this CTA's slice
    const int n = max(0, min(per_cta, nchunks - c0));
    const uint32_t bar = smem_addr(&s_bar);
    if (tid == 0) {
        s_cta_arg = 0x7FFFFFFF; s_row_sum = 0; s_row_arg = 0x7FFFFFFF; s_arrived = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (n > 0) {
            const uint32_t bytes = (uint32_t)n * 16u;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(s_slice)), "l"(logits + (long long)row * ld_chunks + c0), "r"(bytes), "r"(bar) : "memory");
        } else {
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
        }
    }
    __syncthreads();
    {   // bounded wait for the slice; on expiry the status word is set and the row's result is meaningless
        uint32_t ok = 0;
        for (int i = 0; i < (1 << 20) && !ok; ++i)
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(bar) : "memory");
        if (!ok && err) atomicExch(err, SFS_ERR_TIMEOUT);
    }

    // ---- pass 1: exact maximum
    __nv_bfloat162 mx = as_bf162(kNegInf2);
    for (int c = tid; c < n; c += kStagedThreads) {
        const uint4 v = s_slice[c];
        mx = __hmax2(mx, __hmax2(__hmax2(as_bf162(v.x), as_bf162(v.y)), __hmax2(as_bf162(v.z), as_bf162(v.w))));
    }
    const float lmax = bf162_max(*reinterpret_cast<uint32_t *>(&mx));
    float m = warp_max(lmax);
    if (lane == 0) s_wmax[warp] = m;
    __syncthreads();
    if (tid < C) {
        float t = s_wmax[0];
#pragma unroll
        for (int w = 1; w < kStagedThreads / 32; ++w) t = fmaxf(t, s_wmax[w]);
        *cluster.map_shared_rank(&s_max_of[rank], tid) = t;
    }
    cluster.sync();                                         // the only cluster barrier: all slice maxima are here
    m = s_max_of[0];
    for (int r = 1; r < C; ++r) m = fmaxf(m, s_max_of[r]);

    // ---- first position of the maximum (only threads that hold it look), then pass 2
    if (lmax == m) {
        int best = 0x7FFFFFFF;
        for (int c = tid; c < n && best == 0x7FFFFFFF; c += kStagedThreads) {
            const uint4 v = s_slice[c];
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 7; e >= 0; --e) {
                const float x = (e & 1) ? __uint_as_float(w[e >> 1] & 0xFFFF0000u) : __uint_as_float(w[e >> 1] << 16);
                const int idx = (c0 + c) * 8 + e;
                if (x == m && idx < vocab) best = idx;
            }
        }
        if (best != 0x7FFFFFFF) atomicMin(&s_cta_arg, best);
    }
    Consts2 k;
    k.negm = pack2(-m, -m);           k.l2e = pack2(kLog2e, kLog2e);
    k.magic = pack2(kMagic, kMagic);  k.negmagic = pack2(-kMagic, -kMagic);
    k.negln2 = pack2(-kLn2, -kLn2);
    k.c1 = pack2(kC1, kC1); k.c2 = pack2(kC2, kC2); k.c3 = pack2(kC3, kC3); k.c4 = pack2(kC4, kC4);
    k.three = pack2(3.0f, 3.0f);
    unsigned long long acc = 0;
#pragma unroll 4
    for (int c = tid; c < n; c += kStagedThreads) {
        const uint4 v = s_slice[c];
        const uint32_t a = canon_pair(v.x, k) + canon_pair(v.y, k) + canon_pair(v.z, k) + canon_pair(v.w, k);
        acc += a;                                           // 8 terms < 8 * 1.42 * 2^28 < 2^32
    }
    acc = warp_sum_u64(acc);
    if (lane == 0) s_wsum[warp] = acc;
    __syncthreads();
    if (tid == 0) {
        unsigned long long t = 0;
#pragma unroll
        for (int w = 0; w < kStagedThreads / 32; ++w) t += s_wsum[w];
        const int arg = s_cta_arg;
        unsigned long long *rs = cluster.map_shared_rank(&s_row_sum, 0);
        int *ra = cluster.map_shared_rank(&s_row_arg, 0), *rn = cluster.map_shared_rank(&s_arrived, 0);
        atomicAdd(rs, t);
        atomicMin(ra, arg);
        cluster_fence();
        atomicAdd(rn, 1);
        if (rank == 0) {
            int spins = 0;
            while (*reinterpret_cast<volatile int *>(&s_arrived) < C && ++spins < (1 << 24)) {}
            if (spins >= (1 << 24) && err) atomicExch(err, SFS_ERR_TIMEOUT);   // a peer never reported
            cluster_fence();
            const int a2 = *reinterpret_cast<volatile int *>(&s_row_arg);
            write_row(out, row, a2 == 0x7FFFFFFF ? 0 : a2, *reinterpret_cast<volatile unsigned long long *>(&s_row_sum));
        }
    }
}

int32_t launch_staged(const uint4 *logits, long long ld_chunks, int nchunks, int vocab, const int32_t *d_n_rows,
                      int max_rows, const RowOut &out, cudaStream_t stream)
{
    const int per_cta = (nchunks + kStagedCluster - 1) / kStagedCluster;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(max_rows * kStagedCluster), 1, 1);
    cfg.blockDim = dim3(kStagedThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)per_cta * 16;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)kStagedCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    SFS_CUDA(cudaLaunchKernelEx(&cfg, rowstats_staged_bf16, logits, ld_chunks, nchunks, per_cta, vocab, d_n_rows, max_rows, out, out.err));
    return SFS_OK;
}

// ---- generic path ------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float load_as_f32(const T *p, long long i);
template <> __device__ __forceinline__ float load_as_f32<float>(const float *p, long long i) { return p[i]; }
template <> __device__ __forceinline__ float load_as_f32<__nv_bfloat16>(const __nv_bfloat16 *p, long long i) {
    return bf16_bits_to_f32(reinterpret_cast<const unsigned short *>(p)[i]);
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
rowstats_generic(const T *__restrict__ logits, long long ld, int vocab,
                 const int32_t *__restrict__ n_rows_ptr, int max_rows, RowOut out)
{
    const int n_rows = n_rows_ptr ? min(*n_rows_ptr, max_rows) : max_rows;
    __shared__ float s_wmax[kThreads / 32];
    __shared__ unsigned long long s_wsum[kThreads / 32];
    __shared__ float s_max;
    __shared__ int s_arg;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int row = blockIdx.x; row < n_rows; row += gridDim.x) {
        const T *rp = logits + (long long)row * ld;
        float lm = -INFINITY;
        for (int v = tid; v < vocab; v += kThreads) lm = fmaxf(lm, load_as_f32(rp, v));
        lm = warp_max(lm);
        if (lane == 0) s_wmax[warp] = lm;
        if (tid == 0) s_arg = 0x7FFFFFFF;
        __syncthreads();
        if (tid == 0) {
            float t = s_wmax[0];
            for (int w = 1; w < kThreads / 32; ++w) t = fmaxf(t, s_wmax[w]);
            s_max = t;
        }
        __syncthreads();
        const float m = s_max;
        unsigned long long acc = 0;
        int best = 0x7FFFFFFF;
        for (int v = tid; v < vocab; v += kThreads) {
            const float x = load_as_f32(rp, v);
            acc += canon_term(x, m);
            if (x == m && v < best) best = v;
        }
        if (best != 0x7FFFFFFF) atomicMin(&s_arg, best);
        acc = warp_sum_u64(acc);
        if (lane == 0) s_wsum[warp] = acc;
        __syncthreads();
        if (tid == 0) {
            unsigned long long S = 0;
            for (int w = 0; w < kThreads / 32; ++w) S += s_wsum[w];
            write_row(out, row, s_arg == 0x7FFFFFFF ? 0 : s_arg, S);
        }
        __syncthreads();
    }
}

template <int NV>
int32_t launch_cluster(const uint4 *logits, long long ld_chunks, int nchunks, int vocab, const int32_t *d_n_rows,
                       int max_rows, int C, const RowOut &out, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(max_rows * C), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    SFS_CUDA(cudaLaunchKernelEx(&cfg, rowstats_cluster_bf16<NV>, logits, ld_chunks, nchunks, vocab, d_n_rows, max_rows, out, out.err));
    return SFS_OK;
}

}  // namespace

int32_t launch_row_stats(const void *d_logits, int32_t logits_dtype, int32_t vocab, int64_t ld,
                         const int32_t *d_n_rows, int32_t max_rows, const int32_t *d_rows,
                         int32_t *d_argmax, unsigned long long *d_sq, float *d_conf,
                         unsigned long long *d_pos_sq, int32_t *d_pos_arg, int32_t n_positions, int32_t *d_err,
                         cudaStream_t stream)
{
    if (max_rows <= 0) return SFS_OK;
    RowOut out{d_rows, d_argmax, d_sq, d_conf, d_pos_sq, d_pos_arg, n_positions, d_err};
    const bool fast = logits_dtype == SFS_LOGITS_BF16 && (vocab % 8) == 0 && (ld % 8) == 0 && aligned_to(d_logits, 16);
    if (fast) {
        const int nchunks = vocab / 8;
        // long rows (128 KB and more, slices of at most 40 KB): staged through shared memory
        if (nchunks >= 8192 && (nchunks + kStagedCluster - 1) / kStagedCluster <= 2560)
            return launch_staged(reinterpret_cast<const uint4 *>(d_logits), ld / 8, nchunks, vocab, d_n_rows, max_rows, out, stream);
        // smallest (cluster size, chunks per thread) that covers the row; at most 8 CTAs x 256 threads x 8 chunks
        const int per_cta1 = kThreads;                      // chunks covered by one CTA with NV = 1
        int C = 1, NV = 1;
        auto covers = [&](int c, int nv) { return (long long)c * nv * per_cta1 >= nchunks; };
        if (covers(1, 1)) { C = 1; NV = 1; }
        else if (covers(1, 2)) { C = 1; NV = 2; }
        else if (covers(1, 4)) { C = 1; NV = 4; }
        else if (covers(2, 4)) { C = 2; NV = 4; }
        else if (covers(4, 4)) { C = 4; NV = 4; }
        else if (covers(8, 4)) { C = 8; NV = 4; }
        else if (covers(8, 8)) { C = 8; NV = 8; }
        else C = 0;
        if (C) {
            const uint4 *lp = reinterpret_cast<const uint4 *>(d_logits);
            switch (NV) {
                case 1: return launch_cluster<1>(lp, ld / 8, nchunks, vocab, d_n_rows, max_rows, C, out, stream);
                case 2: return launch_cluster<2>(lp, ld / 8, nchunks, vocab, d_n_rows, max_rows, C, out, stream);
                case 4: return launch_cluster<4>(lp, ld / 8, nchunks, vocab, d_n_rows, max_rows, C, out, stream);
                default: return launch_cluster<8>(lp, ld / 8, nchunks, vocab, d_n_rows, max_rows, C, out, stream);
            }
        }
    }
    const int grid = max_rows < 4096 ? max_rows : 4096;
    if (logits_dtype == SFS_LOGITS_BF16) {
        rowstats_generic<__nv_bfloat16><<<grid, kThreads, 0, stream>>>(
            reinterpret_cast<const __nv_bfloat16 *>(d_logits), ld, vocab, d_n_rows, max_rows, out);
    } else {
        rowstats_generic<float><<<grid, kThreads, 0, stream>>>(
            reinterpret_cast<const float *>(d_logits), ld, vocab, d_n_rows, max_rows, out);
    }
    SFS_LAUNCH_CHECK();
    return SFS_OK;
}

}  // namespace sfs
