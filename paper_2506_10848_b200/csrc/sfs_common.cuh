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

struct SelectArgs {
    int32_t *tokens; uint8_t *mask; int32_t B, S, P, L;
    sfs_state *state; sfs_params params;
    unsigned long long *pos_sq; int32_t *pos_arg;          // [B*S] scratch written by the row-stats kernel
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
