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
#include <math_constants.h>
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
    // every CTA of the cluster announces that it runs (its shared memory exists) before anybody writes into a peer
    if (C > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

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
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");      // all peers run
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

// Pass 2 of the two-pass form, first half: one CTA per sequence looks at what the step's rule will ask of its candidate rows
// and sorts them into "the enclosure [lo, hi] of pass 1 answers it" (the lower bound is handed to the selection kernel) and
// "must be recomputed canonically" (the logits row goes on a list that the staged kernel then works through).
//   * a threshold is open when lo and hi fall on different sides of it;
//   * the ranking (k most confident candidates, smallest S_q first) is open for every candidate whose lo does not exceed
//     U = the k-th smallest hi among the candidates: the k rows with the smallest hi all have S_q <= U, so a row with
//     lo > U is not among the k most confident, and its lower bound (still > U) orders it behind them.  Only k = 1 is
//     evaluated this way (U = the smallest hi); for k > 1 every candidate is recomputed.
constexpr int kDecideThreads = 256;
__global__ void __launch_bounds__(kDecideThreads) refine_decide_kernel(RefineArgs rf)
{
    pdl_wait();
    pdl_trigger();
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, L = rf.L;
    const sfs_state &st = rf.state[b];
    if (st.done || st.status != SFS_OK) return;
    const StepAsk ask = step_ask(rf.params, st, L);
    const long long base = (long long)b * rf.S + rf.P;
    const uint8_t *msk = rf.mask + base;
    const unsigned long long *plo = rf.pos_lo + base, *phi = rf.pos_hi + base;
    __shared__ int s_cnt[kDecideThreads / 32];
    __shared__ unsigned long long s_min[kDecideThreads / 32];
    int cnt = 0;
    unsigned long long umin = ~0ull;
    for (int j = ask.lo + tid; j < ask.hi; j += kDecideThreads) {
        if (!msk[j]) continue;
        cnt++;
        if (plo[j] != 0) umin = min(umin, phi[j]);
    }
    cnt = warp_sum_i32(cnt);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) umin = min(umin, __shfl_xor_sync(0xffffffffu, umin, o));
    if (lane == 0) { s_cnt[warp] = cnt; s_min[warp] = umin; }
    __syncthreads();
    int n_cand = 0;
    unsigned long long U = ~0ull;
    for (int w = 0; w < kDecideThreads / 32; ++w) { n_cand += s_cnt[w]; U = min(U, s_min[w]); }
    int k_top = 0;
    if (ask.rank_needed) {
        if (rf.params.sampler == SFS_SAMPLER_LOW_CONFIDENCE) {
            const BlockStep blk = block_step(rf.params, L, st.steps_done);
            const long long Lb = ask.hi - ask.lo, Nb = blk.steps_per_block;
            k_top = (int)max(0ll, (Lb * (Nb - blk.k_b + 1)) / Nb - (Lb - n_cand));
        } else {
            k_top = (st.phase == SFS_PHASE_SLOW) ? rf.params.k_slow : rf.params.k_fast;
        }
        if (k_top >= n_cand) k_top = 0;                     // everything is chosen: no ranking
    }
    for (int j = ask.lo + tid; j < ask.hi; j += kDecideThreads) {
        if (!msk[j]) continue;
        const unsigned long long lo = plo[j], hi = phi[j];
        if (lo == 0) continue;                              // no row supplied for this candidate
        bool need = false;
        if (ask.tau > 0.f) need = conf_exceeds(lo, ask.tau) && !conf_exceeds(hi, ask.tau);
        if (k_top > 1) need = true;
        else if (k_top == 1) need = need || lo <= U;
        if (need) rf.refine_list[atomicAdd(rf.refine_count, 1)] = rf.pos_row[base + j];
        else rf.pos_sq[base + j] = lo;
    }
}

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
    // every CTA of the cluster announces that it runs (its shared memory exists) before anybody writes into a peer
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
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
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");      // all peers run
    if (tid < C) {
        float t = s_wmax[0];
#pragma unroll
        for (int w = 1; w < kStagedThreads / 32; ++w) t = fmaxf(t, s_wmax[w]);
        *cluster.map_shared_rank(&s_max_of[rank], tid) = t;
    }
    cluster.sync();                                         // all slice maxima are here
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

// ---- pass 1 of the two-pass form: exact maximum / argmax, approximate denominator with a proven enclosure -----------------
// No staging and no cluster here: a row is cut into kSlices slices, one CTA per (row, slice) streams its slice straight from
// HBM into registers (kInFlight 16-byte loads per thread in flight) and evaluates it as it arrives.  Measured on 256 rows of
// 126464 logits, back to back, cold: a bare read of the 64.75 MB takes 12.5 us, this kernel 18.4 us, the staged cluster form
// of the same arithmetic 27 us (its staging and cluster barrier, not its arithmetic, set the pace).  Packed f32x2 arithmetic,
// a deeper or software-pipelined load queue and fewer registers each moved the time by less than 1 us: the special-function
// unit (two ex2 per 32-bit word: 7 us of its time) overlaps the loads only in part, and every CTA ends with the same short
// serial tail (block reduction, ticket).  The canonical kernel needs the row maximum before its first term and keeps the
// staged form.  The exponentials are taken against a reference c = the maximum of the WARP's first batch of chunks (no
// CTA-wide barrier before the stream starts); a warp's sum is moved to the slice maximum when the CTA reduces, and the CTA
// that completes a row (a ticket per row) moves the slice sums to the row maximum and adds them in slice order:
//     S~ = sum over slices, warps of ex2((c - m) log2 e) * sum_v ex2.approx(fma(x_v, log2 e, -c log2 e))       (fp32)
// The canonical S_q = sum_v trunc(2^28 exp~(x_v - m)) lies in
//     [ 2^28 S~ (1 - kEps) - V - 1 ,  2^28 S~ (1 + kEps) + 1 ]  intersected with [2^28, inf):
// the canonical exponential is within 1e-5 relative of exp (degree-4 fit 3.3e-6, its fp32 steps < 1e-6) and truncation loses
// less than 1 per term (V terms); on this side an exponent (x - c) log2 e of magnitude up to 100 is rounded to 2^-24
// relative (< 6e-6 absolute, i.e. < 4.2e-6 relative in the term), the same again for each of the two moves, ex2.approx is
// within 2^-22 three times, and the fp32 sums (at most 32 sequential adds per thread, then pairwise levels) within 3e-6.
// Worst case 2.8e-5; kEps = 6e-5.  A reference more than 100 (in log2 units) below the maximum it is moved to, and a sum
// that is not a finite number >= 1, yield an enclosure that contains everything, which sends the row to the canonical pass.
constexpr double kEps = 6e-5;
constexpr int kSlices = 8;
constexpr int kBoundsThreads = 128;

__device__ __forceinline__ float ex2_fast(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

struct BoundsOut {
    const int32_t *rows;                                    // flat token index per logits row, or null (dense outputs only)
    unsigned long long *lo, *hi; int32_t *argmax;           // dense by logits row (optional)
    unsigned long long *pos_lo, *pos_hi; int32_t *pos_arg;  // scattered by flat token index (optional)
    int32_t *pos_row;                                       // with them: the logits row a position's statistics came from
    float *pos_max;                                         //            and the exact row maximum
    int32_t *list_count;                                    // optional: counter of the recompute list, cleared by this launch
    int32_t n_positions; int32_t *err;
    float4 *partial;                                        // scratch [max_rows * kSlices]: (slice max, reference, sum, argmax bits)
    int32_t *tickets;                                       // scratch [max_rows], zero between launches
};

// the enclosure of the canonical S_q from the approximate sum `tot` (relative to the row maximum m), and the scattered outputs
__device__ __forceinline__ void write_enclosure(const BoundsOut &out, int row, float tot, int arg, float m, bool open, int vocab)
{
    if (arg == 0x7FFFFFFF) arg = 0;
    const double Sd = (double)tot * (double)(1u << SFS_CONF_QBITS);
    const double dlo = Sd * (1.0 - kEps) - (double)vocab - 1.0, dhi = Sd * (1.0 + kEps) + 1.0;
    const unsigned long long floor_q = 1ull << SFS_CONF_QBITS;     // the maximum alone contributes 2^28
    unsigned long long lo = dlo > (double)floor_q ? (unsigned long long)dlo : floor_q;
    unsigned long long hi = (unsigned long long)dhi + 1ull;
    if (open || !(tot >= 0.999f) || !(tot <= 3.0e38f)) { lo = 1ull; hi = ~0ull >> 1; }
    if (out.lo) out.lo[row] = lo;
    if (out.hi) out.hi[row] = hi;
    if (out.argmax) out.argmax[row] = arg;
    if (out.rows && out.pos_lo) {
        const int p = out.rows[row];
        if ((unsigned)p < (unsigned)out.n_positions) {
            out.pos_lo[p] = lo; out.pos_hi[p] = hi; out.pos_arg[p] = arg; out.pos_row[p] = row; out.pos_max[p] = m;
        } else if (out.err) {
            atomicExch(out.err, SFS_ERR_INVALID_ARG);
        }
    }
}

// Pass 1 when the LM head has already taken the statistics in its epilogue: per row, n_parts records (maximum, reference,
// sum of 2^((x - reference) log2 e), first position of the maximum) are combined exactly like the slices of the streaming
// kernel — one warp per row, the lanes' shares added in a fixed order — into the row's argmax and enclosure.  The logits are
// not read.
__global__ void __launch_bounds__(128)
combine_partials_kernel(const float4 *__restrict__ stats, int stats_ld, int n_parts, const int32_t *__restrict__ n_rows_ptr, int max_rows,
                        int vocab, BoundsOut out)
{
    pdl_wait();
    pdl_trigger();
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int n_rows = n_rows_ptr ? min(*n_rows_ptr, max_rows) : max_rows;
    if (blockIdx.x == 0 && threadIdx.x == 0 && out.list_count) *out.list_count = 0;
    if (row >= n_rows) return;
    const float4 *ps = stats + (long long)row * stats_ld;
    float m = -INFINITY;
    for (int q = lane; q < n_parts; q += 32) m = fmaxf(m, __ldg(&ps[q]).x);
    m = warp_max(m);
    const float nm = __fmul_rn(-m, kLog2e);
    int arg = 0x7FFFFFFF;
    float tot = 0.f;
    int open = 0;
    for (int q = lane; q < n_parts; q += 32) {
        const float4 r = __ldg(&ps[q]);
        if (r.x == m) arg = min(arg, __float_as_int(r.w));
        if (r.z != 0.f) {
            const float shift = __fmaf_rn(r.y, kLog2e, nm);
            if (!(shift >= -100.f) || !(shift <= 100.f)) open = 1;
            tot += r.z * ex2_fast(shift);
        }
    }
    tot = warp_sum(tot);
    arg = warp_min_i32(arg);
    open = warp_max_i32(open);
    if (lane == 0) write_enclosure(out, row, tot, arg, m, open != 0, vocab);
}

__device__ __forceinline__ uint32_t chunk_max2(const uint4 &v) {
    __nv_bfloat162 m = __hmax2(__hmax2(as_bf162(v.x), as_bf162(v.y)), __hmax2(as_bf162(v.z), as_bf162(v.w)));
    return *reinterpret_cast<uint32_t *>(&m);
}

template <int kInFlight, bool PACKED, bool PIPE>
__global__ void __launch_bounds__(kBoundsThreads)
rowstats_bounds_bf16(const uint4 *__restrict__ logits, long long ld_chunks, int nchunks, int vocab,
                     const int32_t *__restrict__ n_rows_ptr, int max_rows, int slices, BoundsOut out)
{
    const int row = blockIdx.x / slices, sl = blockIdx.x - row * slices;
    const int n_rows = n_rows_ptr ? min(*n_rows_ptr, max_rows) : max_rows;
    if (blockIdx.x == 0 && threadIdx.x == 0 && out.list_count) *out.list_count = 0;
    if (row >= n_rows) return;
    const int per = (nchunks + slices - 1) / slices;
    const int c0 = sl * per, c1 = min(nchunks, c0 + per);
    const uint4 *rp = logits + (long long)row * ld_chunks;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = kBoundsThreads / 32;
    __shared__ float s_wmax[NW], s_wsum[NW], s_wref[NW];
    __shared__ int s_arg;
    const uint4 neg = make_uint4(kNegInf2, kNegInf2, kNegInf2, kNegInf2);

    // ---- first batch: also gives the reference, per warp (no CTA-wide barrier before the stream starts)
    uint4 v[kInFlight], nx[kInFlight];
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) { const int c = c0 + tid + u * kBoundsThreads; v[u] = c < c1 ? ld_stream(rp + c) : neg; }
    int c = c0 + tid + kInFlight * kBoundsThreads;
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) { const int cc = c + u * kBoundsThreads; nx[u] = cc < c1 ? ld_stream(rp + cc) : neg; }
    if (tid == 0) s_arg = 0x7FFFFFFF;
    float fm = -INFINITY;
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) fm = fmaxf(fm, bf162_max(chunk_max2(v[u])));
    float cref = warp_max(fm);
    if (!(fabsf(cref) <= 3.0e38f)) cref = 0.f;
    const float nc = __fmul_rn(-cref, kLog2e);
    const f32x2 l2e2 = pack2(kLog2e, kLog2e), nc2 = pack2(nc, nc);

    float mx = -INFINITY, a0 = 0.f, a1 = 0.f;
    int best_c = -1;
    auto eat = [&](const uint4 &q, int cq) {
        const float cm = bf162_max(chunk_max2(q));
        if (cm > mx) { mx = cm; best_c = cq; }              // strict: the first chunk of this thread that holds its maximum
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        float e[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (PACKED) {
                const f32x2 t = fma2(pack2(__uint_as_float(w[k] << 16), __uint_as_float(w[k] & 0xFFFF0000u)), l2e2, nc2);
                uint32_t t0, t1;
                unpack2(t, t0, t1);
                e[2 * k] = ex2_fast(__uint_as_float(t0)); e[2 * k + 1] = ex2_fast(__uint_as_float(t1));
            } else {
                e[2 * k] = ex2_fast(__fmaf_rn(__uint_as_float(w[k] << 16), kLog2e, nc));
                e[2 * k + 1] = ex2_fast(__fmaf_rn(__uint_as_float(w[k] & 0xFFFF0000u), kLog2e, nc));
            }
        }
        a0 += (e[0] + e[1]) + (e[2] + e[3]); a1 += (e[4] + e[5]) + (e[6] + e[7]);
    };
    if (PIPE) {
        // software pipeline: the next batch is in flight while the current one is evaluated (chunks past the slice are -inf:
        // they add nothing and never win the maximum)
        for (int cur = c0 + tid; cur < c1; cur += kInFlight * kBoundsThreads) {
            uint4 w2[kInFlight];
            const int c2 = cur + 2 * kInFlight * kBoundsThreads;
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) { const int cc = c2 + u * kBoundsThreads; w2[u] = cc < c1 ? ld_stream(rp + cc) : neg; }
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) if (cur + u * kBoundsThreads < c1) eat(v[u], cur + u * kBoundsThreads);
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) { v[u] = nx[u]; nx[u] = w2[u]; }
        }
    } else {
        int cur = c0 + tid;
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) if (cur + u * kBoundsThreads < c1) eat(v[u], cur + u * kBoundsThreads);
        cur += kInFlight * kBoundsThreads;
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) if (cur + u * kBoundsThreads < c1) eat(nx[u], cur + u * kBoundsThreads);
        cur += kInFlight * kBoundsThreads;
        for (; cur < c1; cur += kInFlight * kBoundsThreads) {
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) { const int cc = cur + u * kBoundsThreads; v[u] = cc < c1 ? ld_stream(rp + cc) : neg; }
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) if (cur + u * kBoundsThreads < c1) eat(v[u], cur + u * kBoundsThreads);
        }
    }

    // ---- slice maximum, its first position, slice sum
    const float wm = warp_max(mx), ws = warp_sum(a0 + a1);
    if (lane == 0) { s_wmax[warp] = wm; s_wsum[warp] = ws; s_wref[warp] = cref; }
    __syncthreads();
    const float m_slice = fmaxf(fmaxf(s_wmax[0], s_wmax[1]), fmaxf(s_wmax[2], s_wmax[3]));
    if (mx == m_slice && best_c >= 0) {
        const uint4 q = rp[best_c];                         // this thread's first chunk that holds the slice maximum
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        int best = 0x7FFFFFFF;
#pragma unroll
        for (int e = 7; e >= 0; --e) {
            const float x = (e & 1) ? __uint_as_float(w[e >> 1] & 0xFFFF0000u) : __uint_as_float(w[e >> 1] << 16);
            const int idx = best_c * 8 + e;
            if (x == m_slice && idx < vocab) best = idx;
        }
        if (best != 0x7FFFFFFF) atomicMin(&s_arg, best);
    }
    __syncthreads();
    if (tid != 0) return;
    // the warps' sums, moved from each warp's reference to the slice maximum (the table holds sums relative to it)
    float sum = 0.f;
    bool far = false;
    const float nms = __fmul_rn(-m_slice, kLog2e);
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        if (s_wsum[w] == 0.f) continue;                     // nothing finite in this warp's share
        const float shift = __fmaf_rn(s_wref[w], kLog2e, nms);
        if (!(shift >= -100.f)) far = true;
        sum += s_wsum[w] * ex2_fast(shift);
    }
    if (far) sum = CUDART_INF_F;                            // leaves the row to the canonical pass
    out.partial[(long long)row * kSlices + sl] = make_float4(m_slice, m_slice, c1 > c0 ? sum : 0.f, __int_as_float(s_arg));
    __threadfence();
    if (atomicAdd(&out.tickets[row], 1) != slices - 1) return;

    // ---- the CTA that completes the row combines its slices, in slice order
    __threadfence();
    out.tickets[row] = 0;
    float4 ps[kSlices];
#pragma unroll
    for (int q = 0; q < kSlices; ++q)
        ps[q] = q < slices ? __ldcg(&out.partial[(long long)row * kSlices + q]) : make_float4(-INFINITY, 0.f, 0.f, __int_as_float(0x7FFFFFFF));
    float m = ps[0].x;
#pragma unroll
    for (int q = 1; q < kSlices; ++q) m = fmaxf(m, ps[q].x);
    int arg = 0x7FFFFFFF;
    float tot = 0.f;
    bool open = false;
    const float nm = __fmul_rn(-m, kLog2e);
#pragma unroll
    for (int q = 0; q < kSlices; ++q) {
        if (ps[q].x == m && arg == 0x7FFFFFFF) arg = __float_as_int(ps[q].w);     // slices are in position order
        if (ps[q].z != 0.f) {
            const float shift = __fmaf_rn(ps[q].y, kLog2e, nm);                      // (c - m) log2 e <= 0
            if (!(shift >= -100.f)) open = true;                                     // the reference was too far below the maximum
            tot += ps[q].z * ex2_fast(shift);
        }
    }
    write_enclosure(out, row, tot, arg, m, open, vocab);
}

// Pass 2 of the two-pass form, second half: the canonical S_q of the listed rows.  Pass 1 has left the exact row maximum, so one
// sweep is enough; a listed row is cut into kListParts parts, a CTA takes (row, part) items in turn, reads its part (from L2:
// pass 1 has just streamed the logits) and adds its integer partial sum to pos_sq with one atomic — integer addition commutes, so
// the result does not depend on the order of arrival.  pos_sq of a listed row is zero on entry (the selection kernel clears what
// it has consumed, and the deciding kernel writes only the rows it does not list).
constexpr int kListParts = 8;
constexpr int kListThreads = 256;
__global__ void __launch_bounds__(kListThreads)
rowstats_list_bf16(const uint4 *__restrict__ logits, long long ld_chunks, int nchunks, const int32_t *__restrict__ rows,
                   const int32_t *__restrict__ list, const int32_t *__restrict__ list_count, const float *__restrict__ pos_max,
                   unsigned long long *__restrict__ pos_sq, int n_positions)
{
    pdl_wait();
    pdl_trigger();
    const int n_items = *list_count * kListParts;
    const int per = (nchunks + kListParts - 1) / kListParts;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ unsigned long long s_w[kListThreads / 32];
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int row = list[item / kListParts], part = item % kListParts;
        const int p = rows[row];
        if ((unsigned)p >= (unsigned)n_positions) continue;           // uniform over the CTA
        const float m = pos_max[p];
        Consts2 k;
        k.negm = pack2(-m, -m);           k.l2e = pack2(kLog2e, kLog2e);
        k.magic = pack2(kMagic, kMagic);  k.negmagic = pack2(-kMagic, -kMagic);
        k.negln2 = pack2(-kLn2, -kLn2);
        k.c1 = pack2(kC1, kC1); k.c2 = pack2(kC2, kC2); k.c3 = pack2(kC3, kC3); k.c4 = pack2(kC4, kC4);
        k.three = pack2(3.0f, 3.0f);
        const uint4 *rp = logits + (long long)row * ld_chunks;
        const int c0 = part * per, c1 = min(nchunks, c0 + per);
        unsigned long long acc = 0;
        int c = c0 + tid;
        for (; c + 3 * kListThreads < c1; c += 4 * kListThreads) {    // four loads in flight
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = rp[c + u * kListThreads];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                acc += (unsigned long long)(canon_pair(v[u].x, k) + canon_pair(v[u].y, k)) + (unsigned long long)(canon_pair(v[u].z, k) + canon_pair(v[u].w, k));
        }
        for (; c < c1; c += kListThreads) {
            const uint4 v = rp[c];
            acc += (unsigned long long)(canon_pair(v.x, k) + canon_pair(v.y, k)) + (unsigned long long)(canon_pair(v.z, k) + canon_pair(v.w, k));
        }
        acc = warp_sum_u64(acc);
        if (lane == 0) s_w[warp] = acc;
        __syncthreads();
        if (tid == 0) {
            unsigned long long t = 0;
#pragma unroll
            for (int w = 0; w < kListThreads / 32; ++w) t += s_w[w];
            atomicAdd(&pos_sq[p], t);
        }
        __syncthreads();
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

int num_sms_rowstats();
int32_t launch_bounds(const uint4 *logits, long long ld_chunks, int nchunks, int vocab, const int32_t *d_n_rows, int max_rows,
                      const BoundsOut &out, cudaStream_t stream)
{
    // slices per row (at most kSlices): the count whose CTAs fill whole waves best at 9 resident CTAs per SM, longer slices
    // winning ties (fewer reductions); a last wave that is nearly empty costs as much as a full one
    const int per_wave = 9 * num_sms_rowstats();
    int slices = kSlices;
    double best = -1.0;
    for (int sl = kSlices; sl >= 3; --sl) {
        const long long ctas = (long long)max_rows * sl, waves = (ctas + per_wave - 1) / per_wave;
        const double fill = (double)ctas / (double)(waves * per_wave);
        if (fill > best + 0.02) { best = fill; slices = sl; }
    }
    rowstats_bounds_bf16<4, false, false><<<(unsigned)(max_rows * slices), kBoundsThreads, 0, stream>>>(logits, ld_chunks, nchunks, vocab, d_n_rows,
                                                                                                          max_rows, slices, out);
    SFS_LAUNCH_CHECK();
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

namespace { int num_sms_rowstats()
{
    static int n[kMaxDevices] = {};
    int &v = n[current_device_slot()];
    if (v == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    }
    return v;
} }

static bool staged_shape(int32_t logits_dtype, int32_t vocab, int64_t ld, const void *d_logits)
{
    const bool fast = logits_dtype == SFS_LOGITS_BF16 && (vocab % 8) == 0 && (ld % 8) == 0 && aligned_to(d_logits, 16);
    const int nchunks = vocab / 8;
    return fast && nchunks >= 8192 && (nchunks + kStagedCluster - 1) / kStagedCluster <= 2560;
}

bool row_stats_two_pass_applies(const void *d_logits, int32_t logits_dtype, int32_t vocab, int64_t ld)
{
    return staged_shape(logits_dtype, vocab, ld, d_logits);
}

int32_t launch_row_stats_bounds(const void *d_logits, int32_t vocab, int64_t ld, const int32_t *d_n_rows, int32_t max_rows,
                                unsigned long long *d_lo, unsigned long long *d_hi, int32_t *d_argmax, int32_t *d_err, cudaStream_t stream)
{
    if (max_rows <= 0) return SFS_OK;
    SFS_REQUIRE(staged_shape(SFS_LOGITS_BF16, vocab, ld, d_logits), SFS_ERR_UNSUPPORTED,
                "row-statistics enclosures: bf16 rows of 65536 to 163840 entries, 16-byte aligned, only");
    // scratch of this entry point: one table per device, grown on demand and kept (the selection path brings its session's)
    static float4 *s_partial[kMaxDevices] = {};
    static int32_t *s_tickets[kMaxDevices] = {};
    static int s_rows[kMaxDevices] = {};
    const int dev = current_device_slot();
    if (s_rows[dev] < max_rows) {
        SFS_CUDA(cudaDeviceSynchronize());
        if (s_partial[dev]) { cudaFree(s_partial[dev]); cudaFree(s_tickets[dev]); s_partial[dev] = nullptr; s_tickets[dev] = nullptr; s_rows[dev] = 0; }
        SFS_CUDA(cudaMalloc(&s_partial[dev], (size_t)max_rows * kSlices * sizeof(float4)));
        SFS_CUDA(cudaMalloc(&s_tickets[dev], (size_t)max_rows * sizeof(int32_t)));
        SFS_CUDA(cudaMemset(s_tickets[dev], 0, (size_t)max_rows * sizeof(int32_t)));
        s_rows[dev] = max_rows;
    }
    BoundsOut out{nullptr, d_lo, d_hi, d_argmax, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, d_err, s_partial[dev], s_tickets[dev]};
    return launch_bounds(reinterpret_cast<const uint4 *>(d_logits), ld / 8, vocab / 8, vocab, d_n_rows, max_rows, out, stream);
}

int32_t launch_row_stats_two_pass(const void *d_logits, int32_t vocab, int64_t ld, const int32_t *d_n_rows, int32_t max_rows,
                                  const int32_t *d_rows, const RefineArgs &rf, int32_t *d_err, cudaStream_t stream)
{
    if (max_rows <= 0) return SFS_OK;
    const uint4 *lp = reinterpret_cast<const uint4 *>(d_logits);
    BoundsOut bo{d_rows, nullptr, nullptr, nullptr, rf.pos_lo, rf.pos_hi, rf.pos_arg, rf.pos_row, rf.pos_max, rf.refine_count, rf.B * rf.S, d_err,
                 reinterpret_cast<float4 *>(rf.slice_partials), rf.row_tickets};
    int32_t rc = launch_bounds(lp, ld / 8, vocab / 8, vocab, d_n_rows, max_rows, bo, stream);
    if (rc != SFS_OK) return rc;
    SFS_CUDA(launch_pdl(refine_decide_kernel, dim3((unsigned)(rf.B)), dim3((unsigned)(kDecideThreads)), (size_t)(0), stream, rf));
    const int items = max_rows * kListParts, cap = 2 * num_sms_rowstats();
    SFS_CUDA(launch_pdl(rowstats_list_bf16, dim3((unsigned)(items < cap ? items : cap)), dim3((unsigned)(kListThreads)), (size_t)(0), stream, lp, ld / 8, vocab / 8, d_rows, rf.refine_list, rf.refine_count,
                                                                              rf.pos_max, rf.pos_sq, rf.B * rf.S));
    return SFS_OK;
}

int32_t launch_row_stats_from_partials(const void *stats, int32_t stats_ld, int32_t n_parts, const void *d_logits, int32_t vocab, int64_t ld,
                                       const int32_t *d_n_rows, int32_t max_rows, const int32_t *d_rows, const RefineArgs &rf, int32_t *d_err,
                                       cudaStream_t stream)
{
    if (max_rows <= 0) return SFS_OK;
    BoundsOut bo{d_rows, nullptr, nullptr, nullptr, rf.pos_lo, rf.pos_hi, rf.pos_arg, rf.pos_row, rf.pos_max, rf.refine_count, rf.B * rf.S, d_err,
                 nullptr, nullptr};
    SFS_CUDA(launch_pdl(combine_partials_kernel, dim3((unsigned)((max_rows + 3) / 4)), dim3((unsigned)(128)), (size_t)(0), stream, reinterpret_cast<const float4 *>(stats), stats_ld, n_parts, d_n_rows, max_rows, vocab, bo));
    SFS_CUDA(launch_pdl(refine_decide_kernel, dim3((unsigned)(rf.B)), dim3((unsigned)(kDecideThreads)), (size_t)(0), stream, rf));
    const uint4 *lp = reinterpret_cast<const uint4 *>(d_logits);
    const int items = max_rows * kListParts, cap = 2 * num_sms_rowstats();
    SFS_CUDA(launch_pdl(rowstats_list_bf16, dim3((unsigned)(items < cap ? items : cap)), dim3((unsigned)(kListThreads)), (size_t)(0), stream, lp, ld / 8, vocab / 8, d_rows, rf.refine_list, rf.refine_count,
                                                                              rf.pos_max, rf.pos_sq, rf.B * rf.S));
    return SFS_OK;
}

}  // namespace sfs
