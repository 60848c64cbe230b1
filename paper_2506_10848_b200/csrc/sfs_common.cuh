// Shared host/device helpers of libsfs (error reporting, small device utilities).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>
#include <stdarg.h>

#include "../../include/sfs.h"

static_assert(sizeof(sfs_state) == 128, "sfs_state is 32 int32");

namespace sfs {

// ---- host-side error reporting ---------------------------------------------------------------------
void set_error(const char *fmt, ...);          // stores a message for sfs_last_error() (thread-local)

#define SFS_REQUIRE(cond, code, ...)                                   \
    do {                                                               \
        if (!(cond)) { ::sfs::set_error(__VA_ARGS__); return (code); } \
    } while (0)

#define SFS_CUDA(call)                                                                           \
    do {                                                                                         \
        cudaError_t e__ = (call);                                                                \
        if (e__ != cudaSuccess) {                                                                \
            ::sfs::set_error("%s failed: %s (%s:%d)", #call, cudaGetErrorString(e__), __FILE__, __LINE__); \
            return (e__ == cudaErrorMemoryAllocation) ? SFS_ERR_OOM : SFS_ERR_CUDA;              \
        }                                                                                        \
    } while (0)

#define SFS_LAUNCH_CHECK()  SFS_CUDA(cudaGetLastError())

static inline bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Per-device bookkeeping (kernel attributes, the sticky status word) is indexed by the ordinal of the current device.
constexpr int kMaxDevices = 64;
static inline int current_device_slot()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    return dev;
}
// The current device's sticky status word (set by kernels whose bounded waits give up, or that skip an invalid row);
// allocated on first use, null if that allocation fails.  The _if_any form never allocates.
int32_t *device_status_word();
int32_t *device_status_word_if_any();

// ---- programmatic dependent launch -----------------------------------------------------------------------
// A kernel launched with launch_pdl may start (be scheduled, run its prologue) while the kernel before it in the stream is
// still running; it calls pdl_wait() before its first access to global memory, which returns once that kernel has completed
// and its writes are visible.  pdl_trigger() tells the runtime that the kernels after this one may be scheduled.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// ---- device helpers ---------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h16) { return __uint_as_float(h16 << 16); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum_i32(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_min_i32(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ int warp_max_i32(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// block structure of the LLaDA strategies: which positions the step with index t works on, and the block's countdown
struct BlockStep { int j, lo, hi, k_b, steps_per_block; };
__device__ __forceinline__ BlockStep block_step(const sfs_params &p, int L, int t)
{
    const int N = p.max_steps > 0 ? p.max_steps : L;
    const int bl = (p.block_len > 0 && p.block_len < L) ? p.block_len : max(L, 1);
    const int nb = (L + bl - 1) / bl;
    BlockStep s;
    s.steps_per_block = max(N / max(nb, 1), 1);
    s.j = t / s.steps_per_block;
    s.k_b = s.steps_per_block - (t - s.j * s.steps_per_block);
    s.lo = min(L, s.j * bl);
    s.hi = min(L, s.lo + bl);
    return s;
}

// what one denoising step asks of the row statistics of sequence state `st`: the candidate window [lo, hi) of response
// positions, the confidence threshold whose outcome is read (0 = none) and how many most-confident candidates are ranked
// (k_top; n_cand = number of masked positions in the window, needed by the low-confidence rule only)
struct StepAsk { int lo, hi; float tau; bool rank_needed; };
__device__ __forceinline__ StepAsk step_ask(const sfs_params &p, const sfs_state &st, int L)
{
    StepAsk a;
    a.tau = 0.f; a.rank_needed = false;
    if (p.sampler != SFS_SAMPLER_SLOWFAST) {
        const BlockStep b = block_step(p, L, st.steps_done);
        a.lo = b.lo; a.hi = b.hi;
        a.rank_needed = (p.sampler == SFS_SAMPLER_LOW_CONFIDENCE);
    } else if (st.k_remaining == 1) {
        a.lo = 0; a.hi = L;                                 // last permitted step: everything is unmasked, nothing is compared
    } else if (st.phase == SFS_PHASE_SLOW) {
        a.lo = st.s_cycle; a.hi = L; a.tau = p.tau_min_conf; a.rank_needed = true;
    } else {
        a.lo = st.s_cycle; a.hi = st.hi; a.tau = p.tau_high_conf; a.rank_needed = true;
    }
    return a;
}

// c > tau  <=>  S_q * tau < 2^28, one IEEE double multiply
__device__ __forceinline__ bool conf_exceeds(unsigned long long sq, float tau) {
    return __dmul_rn((double)sq, (double)tau) < (double)(1u << SFS_CONF_QBITS);
}
#endif

// ---- internal launchers (defined in the .cu files) --------------------------------------------------
// Row statistics (Section 3.1: greedy token and confidence).  Results are written densely by logits row
// (d_argmax/d_sq/d_conf, each optional) and, when d_rows is given, scattered to d_pos_sq/d_pos_arg at the
// flat token index of each row; an index outside [0, n_positions) is skipped and reported as SFS_ERR_INVALID_ARG
// in *d_err (a device status word, optional), as is a bounded wait that gives up (SFS_ERR_TIMEOUT).
int32_t launch_row_stats(const void *d_logits, int32_t logits_dtype, int32_t vocab, int64_t ld,
                         const int32_t *d_n_rows, int32_t max_rows, const int32_t *d_rows,
                         int32_t *d_argmax, unsigned long long *d_sq, float *d_conf,
                         unsigned long long *d_pos_sq, int32_t *d_pos_arg, int32_t n_positions, int32_t *d_err,
                         cudaStream_t stream);

// Row statistics for the selection step in two passes over long bf16 rows (the filter + exact form):
//   pass 1 streams every row from HBM once and finds the exact maximum and argmax plus an APPROXIMATE denominator (special-
//     function exponentials, fp32 sum) with a proven enclosure [lo, lo + w] of the canonical S_q;
//   pass 2 looks, per sequence, at what the step's rule will ask of its rows (which threshold, which top-k), lists the rows
//     whose enclosure leaves an answer open and recomputes the canonical S_q of those; every other candidate row gets its
//     lower bound.
// The selection kernel then runs unchanged on pos_sq, and its decisions equal those taken on all-canonical values.
struct RefineArgs {
    const int32_t *tokens_unused; const uint8_t *mask; int32_t B, S, P, L;
    const sfs_state *state; sfs_params params;
    unsigned long long *pos_lo, *pos_hi;                    // [B*S] enclosures written by pass 1 (lo == 0: no row supplied)
    unsigned long long *pos_sq; int32_t *pos_arg;           // [B*S] what the selection kernel reads
    float *slice_partials; int32_t *row_tickets;            // scratch of pass 1: [max rows * 8 * 4] floats, [max rows] (zeroed)
    int32_t *pos_row; float *pos_max;                       // [B*S] logits row and exact row maximum of each position (pass 1)
    int32_t *refine_list, *refine_count;                    // [max rows], [1]: logits rows pass 2 recomputes
};
constexpr int kRowStatsSlices = 8;
// true when the two-pass form applies to this logits layout (long bf16 rows, 16-byte aligned)
bool row_stats_two_pass_applies(const void *d_logits, int32_t logits_dtype, int32_t vocab, int64_t ld);
int32_t launch_row_stats_two_pass(const void *d_logits, int32_t vocab, int64_t ld, const int32_t *d_n_rows, int32_t max_rows,
                                  const int32_t *d_rows, const RefineArgs &rf, int32_t *d_err, cudaStream_t stream);
// the same with pass 1 already taken by the LM head's epilogue: `stats` holds n_parts records per row (stats_ld apart)
int32_t launch_row_stats_from_partials(const void *stats, int32_t stats_ld, int32_t n_parts, const void *d_logits, int32_t vocab, int64_t ld,
                                       const int32_t *d_n_rows, int32_t max_rows, const int32_t *d_rows, const RefineArgs &rf, int32_t *d_err,
                                       cudaStream_t stream);
// pass 1 alone, dense outputs by logits row (for tests): d_lo / d_hi enclose the canonical S_q
int32_t launch_row_stats_bounds(const void *d_logits, int32_t vocab, int64_t ld, const int32_t *d_n_rows, int32_t max_rows,
                                unsigned long long *d_lo, unsigned long long *d_hi, int32_t *d_argmax, int32_t *d_err, cudaStream_t stream);

struct SelectArgs {
    int32_t *tokens; uint8_t *mask; int32_t B, S, P, L;
    sfs_state *state; sfs_params params;
    unsigned long long *pos_sq; int32_t *pos_arg;          // [B*S] scratch written by the row-stats kernel
    unsigned long long *pos_lo;                             // optional [B*S]: enclosures of the two-pass form, cleared with pos_sq
    int32_t *sel_count, *sel_pos, *sel_tok;                 // [B], [B,L], [B,L]   (optional)
    int32_t *seq_rows, *seq_row_count;                      // [B,L], [B] scratch: next step's rows per sequence
    int32_t *next_rows, *next_n_rows;                       // optional flat list (sequence-major) + count
    int32_t *n_active;                                      // optional: sequences not done after this step
    int32_t *ticket;                                        // scratch counter (zero between launches)
    int32_t *trace;                                         // optional [B, SFS_TRACE_INTS]
};
int32_t launch_select(const SelectArgs &a, cudaStream_t stream);
int32_t launch_state_init(sfs_state *d_state, int32_t B, int32_t L, const sfs_params &p, int32_t *seq_rows_unused,
                          cudaStream_t stream);

}  // namespace sfs
