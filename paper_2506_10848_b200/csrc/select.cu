// The transition rule S of one denoising step, on the device: the SlowFast rule (paper Section 3.3, Algorithm 1) or one of
// the LLaDA strategies of Section 3.1 (low-confidence / random remasking, optionally block by block).
// One CTA per sequence: it reads the row statistics the epilogue scattered by token position, applies the
// exploratory (slow) or accelerated (fast) rule, unmasks the chosen positions in place, advances the
// per-sequence state (k, s_cycle, e_cycle, H_W, phase) and lists the rows the next step needs.  The last CTA
// to finish concatenates the per-sequence row lists (sequence-major, positions ascending) so that the
// next forward pass gets one deterministic row list without a host round trip.
#include "sfs_common.cuh"

namespace sfs {
namespace {

constexpr int kSelThreads = 256;
constexpr unsigned long long kNoKey = ~0ull;
constexpr int kPosBits = 17;                 // key = S_q << 17 | position  (S_q < 2^47, position < 2^17)

__device__ __forceinline__ bool exceeds(unsigned long long sq, float tau) {
    // c > tau  <=>  S_q * tau < 2^28, one IEEE double multiply
    return __dmul_rn((double)sq, (double)tau) < (double)(1u << SFS_CONF_QBITS);
}

struct BlockRed {
    int n_cand, n_high, max_above, min_cand, n_masked, missing;
};

__device__ BlockRed block_reduce(BlockRed v, int *s_tmp /* [6 * 8] */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v.n_cand = warp_sum_i32(v.n_cand);   v.n_high = warp_sum_i32(v.n_high);
    v.max_above = warp_max_i32(v.max_above); v.min_cand = warp_min_i32(v.min_cand);
    v.n_masked = warp_sum_i32(v.n_masked);   v.missing = warp_sum_i32(v.missing);
    __syncthreads();
    if (lane == 0) {
        s_tmp[warp * 6 + 0] = v.n_cand; s_tmp[warp * 6 + 1] = v.n_high; s_tmp[warp * 6 + 2] = v.max_above;
        s_tmp[warp * 6 + 3] = v.min_cand; s_tmp[warp * 6 + 4] = v.n_masked; s_tmp[warp * 6 + 5] = v.missing;
    }
    __syncthreads();
    BlockRed r{0, 0, -1, 0x7FFFFFFF, 0, 0};
    for (int w = 0; w < kSelThreads / 32; ++w) {
        r.n_cand += s_tmp[w * 6 + 0]; r.n_high += s_tmp[w * 6 + 1];
        r.max_above = max(r.max_above, s_tmp[w * 6 + 2]); r.min_cand = min(r.min_cand, s_tmp[w * 6 + 3]);
        r.n_masked += s_tmp[w * 6 + 4]; r.missing += s_tmp[w * 6 + 5];
    }
    __syncthreads();
    return r;
}

__device__ int block_sum(int v, int *s_tmp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum_i32(v);
    __syncthreads();
    if (lane == 0) s_tmp[warp] = v;
    __syncthreads();
    int r = 0;
    for (int w = 0; w < kSelThreads / 32; ++w) r += s_tmp[w];
    __syncthreads();
    return r;
}

enum { MODE_ALL = 0, MODE_TOPK = 1, MODE_HIGH = 2, MODE_RANDOM = 3 };

// Philox-4x32-10 (Salmon et al., SC'11): ten rounds of multiply / xor on a 128-bit counter under a 64-bit key; the first
// output word is returned.  Random remasking draws one word per (position, step, sequence).
__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
        const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
        c0 = h1 ^ c1 ^ k0; c1 = l1; c2 = h0 ^ c3 ^ k1; c3 = l0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}

// dynamic shared memory: keys u64[L] | flags u8[L] (selected) | flags u8[L] (above tau_high)
__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectArgs a)
{
    pdl_wait();
    pdl_trigger();
    extern __shared__ unsigned long long s_keys[];
    const int L = a.L, S = a.S, P = a.P, b = blockIdx.x, tid = threadIdx.x;
    uint8_t *s_sel  = reinterpret_cast<uint8_t *>(s_keys + L);
    uint8_t *s_high = s_sel + L;
    __shared__ int s_tmp[6 * (kSelThreads / 32)];
    __shared__ sfs_state st;
    __shared__ int s_last;

    if (tid < (int)(sizeof(sfs_state) / 4)) reinterpret_cast<int *>(&st)[tid] = reinterpret_cast<const int *>(a.state + b)[tid];
    __syncthreads();

    int32_t *tok = a.tokens + (long long)b * S + P;
    uint8_t *msk = a.mask + (long long)b * S + P;
    unsigned long long *psq = a.pos_sq + (long long)b * S + P;
    int32_t *parg = a.pos_arg + (long long)b * S + P;
    const sfs_params &p = a.params;

    const bool active = !st.done && st.status == SFS_OK;
    const bool vanilla = p.sampler != SFS_SAMPLER_SLOWFAST;
    int n_sel = 0, e_cand = -1, stable = 0;
    int rec_phase = st.phase, rec_s = st.s_cycle;
    int rec_hi = (st.phase == SFS_PHASE_SLOW) ? L : st.hi;
    const BlockStep blk = block_step(p, L, st.steps_done);
    if (vanilla) { rec_phase = blk.j; rec_s = blk.lo; rec_hi = blk.hi; e_cand = blk.k_b; }

    if (active) {
        const bool forced = !vanilla && (st.k_remaining == 1);
        const int lo = vanilla ? blk.lo : (forced ? 0 : st.s_cycle);
        const int hi = vanilla ? blk.hi : (forced ? L : ((st.phase == SFS_PHASE_SLOW) ? L : st.hi));

        // ---- candidates of this step and their statistics
        BlockRed r{0, 0, -1, 0x7FFFFFFF, 0, 0};
        for (int i = tid; i < L; i += kSelThreads) {
            const bool m = msk[i] != 0;
            const bool cand = m && i >= lo && i < hi;
            unsigned long long key = kNoKey;
            uint8_t high = 0;
            if (cand) {
                const unsigned long long sq = psq[i];
                if (sq == 0) r.missing++;
                key = (sq << kPosBits) | (unsigned long long)i;
                r.n_cand++;
                r.min_cand = min(r.min_cand, i);
                if (exceeds(sq, p.tau_min_conf)) r.max_above = max(r.max_above, i);
                if (exceeds(sq, p.tau_high_conf)) { high = 1; r.n_high++; }
            }
            r.n_masked += m ? 1 : 0;
            s_keys[i] = key; s_high[i] = high; s_sel[i] = 0;
        }
        r = block_reduce(r, s_tmp);

        if (r.missing > 0 || (r.n_cand == 0 && !vanilla)) {
            // a needed row was not supplied (or the state is inconsistent): report, change nothing
            if (tid == 0) st.status = SFS_ERR_MISSING_ROW;
        } else {
            int mode, k_top = 0;
            if (p.sampler == SFS_SAMPLER_LOW_CONFIDENCE) {
                // Section 3.1: after this step floor(L_b (1 - (k_b - 1) / N_b)) positions of the block are unmasked
                const long long Lb = hi - lo, Nb = blk.steps_per_block;
                const long long target = (Lb * (Nb - blk.k_b + 1)) / Nb;
                mode = MODE_TOPK; k_top = (int)max(0ll, target - (Lb - r.n_cand));
            } else if (p.sampler == SFS_SAMPLER_RANDOM) mode = MODE_RANDOM;
            else if (forced) mode = MODE_ALL;
            else if (st.phase == SFS_PHASE_SLOW) { mode = MODE_TOPK; k_top = p.k_slow; }
            else if (r.n_high >= p.min_high_count) mode = MODE_HIGH;
            else { mode = MODE_TOPK; k_top = p.k_fast; }

            // ---- choose
            int my_sel = 0;
            for (int i = tid; i < L; i += kSelThreads) {
                const unsigned long long key = s_keys[i];
                if (key == kNoKey) continue;
                bool sel;
                if (mode == MODE_ALL) sel = true;
                else if (mode == MODE_HIGH) sel = s_high[i] != 0;
                else if (mode == MODE_RANDOM)
                    sel = (unsigned long long)philox_first_word((uint32_t)i, (uint32_t)st.steps_done, (uint32_t)b, 0u, p.seed_lo, p.seed_hi)
                          * (unsigned long long)blk.k_b < (1ull << 32);
                else {
                    int rank = 0;                           // candidates that are more confident (ties: smaller position)
                    for (int j = 0; j < L; ++j) rank += (s_keys[j] < key) ? 1 : 0;
                    sel = rank < k_top;
                }
                if (sel) { s_sel[i] = 1; my_sel++; tok[i] = parg[i]; msk[i] = 0; }
            }
            n_sel = block_sum(my_sel, s_tmp);

            // ---- scheduler state (Algorithm 1), one thread
            if (tid == 0) {
                st.n_masked = r.n_masked - n_sel;
                st.steps_done++;
                if (vanilla) {
                    st.k_remaining--;
                } else if (forced) {
                    st.k_remaining = 0;
                } else if (st.phase == SFS_PHASE_SLOW) {
                    e_cand = (r.max_above >= 0) ? r.max_above : r.min_cand;
                    if (st.hist_len < p.w_hist) st.hist[st.hist_len++] = e_cand;
                    else { for (int h = 1; h < p.w_hist; ++h) st.hist[h - 1] = st.hist[h]; st.hist[p.w_hist - 1] = e_cand; }
                    st.k_remaining--; st.step_count++; st.n_slow++;
                    long long sum = 0, sum2 = 0;
                    for (int h = 0; h < st.hist_len; ++h) { sum += st.hist[h]; sum2 += (long long)st.hist[h] * st.hist[h]; }
                    const long long n = st.hist_len;
                    const long long num = n * sum2 - sum * sum;           // n^2 * population variance, exact
                    if (st.hist_len >= p.w_hist && (double)num < (double)p.sigma2_stable * (double)(n * n)) {
                        stable = 1;
                        st.phase = SFS_PHASE_FAST; st.hi = (int)(sum / n) + 1;   // floor(mean(H_W)) + 1
                    } else if (st.step_count >= p.k_max) {
                        st.phase = SFS_PHASE_FAST; st.hi = e_cand + 1;
                    }
                } else {
                    st.k_remaining--; st.n_fast++;
                    if (mode == MODE_TOPK) st.n_fallback++;
                }
            }
            __syncthreads();

            // ---- is the span clean?  (decides whether the next cycle starts)
            if (!vanilla && !forced && st.phase == SFS_PHASE_FAST) {
                int cnt = 0;
                for (int i = st.s_cycle + tid; i < st.hi && i < L; i += kSelThreads) cnt += msk[i] ? 1 : 0;
                cnt = block_sum(cnt, s_tmp);
                if (tid == 0 && cnt == 0 && st.n_masked > 0) {
                    st.s_cycle = st.hi; st.phase = SFS_PHASE_SLOW; st.hist_len = 0; st.step_count = 0; st.n_cycles++;
                }
            }
            if (tid == 0 && (st.n_masked == 0 || st.k_remaining == 0)) {
                st.done = 1;
                if (st.n_masked > 0) st.status = SFS_ERR_STEP_LIMIT;
            }
        }
        __syncthreads();
        // the statistics of this step are consumed: a later step must bring its own
        for (int i = tid; i < L; i += kSelThreads) psq[i] = 0;
        if (a.pos_lo) for (int i = tid; i < L; i += kSelThreads) a.pos_lo[(long long)b * S + P + i] = 0;
    } else {
        // a finished (or stopped) sequence consumes the statistics supplied for it as well: nothing stale is left for a
        // later generation that reuses the scratch
        for (int i = tid; i < L; i += kSelThreads) { s_sel[i] = 0; psq[i] = 0; if (a.pos_lo) a.pos_lo[(long long)b * S + P + i] = 0; }
    }
    __syncthreads();

    // ---- ordered outputs (warp 0: ballot scan): selected positions, and the rows of the next step
    if (tid < 32) {
        const bool next_active = !st.done && st.status == SFS_OK;
        const bool nforced = !vanilla && st.k_remaining == 1;
        const BlockStep nblk = block_step(p, L, st.steps_done);
        const int nlo = vanilla ? nblk.lo : (nforced ? 0 : st.s_cycle);
        const int nhi = vanilla ? nblk.hi : (nforced ? L : ((st.phase == SFS_PHASE_SLOW) ? L : st.hi));
        int n_out = 0, n_next = 0;
        for (int base = 0; base < L; base += 32) {
            const int i = base + tid;
            const bool sel = i < L && s_sel[i];
            const bool need = next_active && i < L && msk[i] && i >= nlo && i < nhi;
            const unsigned bs = __ballot_sync(0xffffffffu, sel), bn = __ballot_sync(0xffffffffu, need);
            const unsigned lt = (1u << tid) - 1u;
            if (sel && a.sel_pos) {
                const int o = n_out + __popc(bs & lt);
                a.sel_pos[(long long)b * L + o] = i;
                a.sel_tok[(long long)b * L + o] = tok[i];
            }
            if (need) a.seq_rows[(long long)b * L + n_next + __popc(bn & lt)] = b * S + P + i;
            n_out += __popc(bs); n_next += __popc(bn);
        }
        if (tid == 0) {
            if (a.sel_count) a.sel_count[b] = n_out;
            a.seq_row_count[b] = n_next;
            if (a.trace) {
                int32_t *t = a.trace + (long long)b * SFS_TRACE_INTS;
                t[0] = rec_phase; t[1] = rec_s; t[2] = rec_hi; t[3] = e_cand; t[4] = stable; t[5] = n_sel;
                t[6] = st.n_masked; t[7] = st.k_remaining;
            }
        }
    }
    __syncthreads();
    if (tid < (int)(sizeof(sfs_state) / 4)) reinterpret_cast<int *>(a.state + b)[tid] = reinterpret_cast<const int *>(&st)[tid];

    // ---- last CTA: concatenate the row lists, count the active sequences
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(a.ticket, 1) == (int)gridDim.x - 1) ? 1 : 0;
    __syncthreads();
    if (s_last) {
        __threadfence();
        if (tid == 0) {
            int total = 0, act = 0;
            for (int q = 0; q < a.B; ++q) {
                total += __ldcg(&a.seq_row_count[q]);
                act += (__ldcg(&a.state[q].done) == 0 && __ldcg(&a.state[q].status) == SFS_OK) ? 1 : 0;
            }
            if (a.next_n_rows) *a.next_n_rows = total;
            if (a.n_active) *a.n_active = act;
            *a.ticket = 0;
        }
        if (a.next_rows) {
            int off = 0;
            for (int q = 0; q < a.B; ++q) {
                const int c = __ldcg(&a.seq_row_count[q]);
                for (int i = tid; i < c; i += kSelThreads) a.next_rows[off + i] = __ldcg(&a.seq_rows[(long long)q * L + i]);
                off += c;
            }
        }
    }
}

__global__ void state_init_kernel(sfs_state *state, int B, int L, sfs_params p)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    sfs_state s;
    memset(&s, 0, sizeof(s));
    s.phase = SFS_PHASE_SLOW;
    s.k_remaining = p.max_steps > 0 ? p.max_steps : L;
    s.n_masked = L;
    s.done = (L == 0) ? 1 : 0;
    state[b] = s;
}

}  // namespace

int32_t launch_select(const SelectArgs &a, cudaStream_t stream)
{
    const size_t smem = (size_t)a.L * (sizeof(unsigned long long) + 2);
    SFS_REQUIRE(smem <= 200 * 1024, SFS_ERR_UNSUPPORTED, "gen_len %d too long for the selection kernel", a.L);
    if (smem > 48 * 1024) {
        SFS_CUDA(cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    SFS_CUDA(launch_pdl(select_kernel, dim3((unsigned)(a.B)), dim3((unsigned)(kSelThreads)), (size_t)(smem), stream, a));
    return SFS_OK;
}

int32_t launch_state_init(sfs_state *d_state, int32_t B, int32_t L, const sfs_params &p, int32_t *, cudaStream_t stream)
{
    state_init_kernel<<<(B + 63) / 64, 64, 0, stream>>>(d_state, B, L, p);
    SFS_LAUNCH_CHECK();
    return SFS_OK;
}

}  // namespace sfs
