// sfs_select_static: the selection step for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off the table: inside a region that is being captured
// or replayed as a CUDA graph, inside a serving loop that forbids allocator calls for latency reasons, or in
// a process whose memory pool is owned (and fully claimed) by another runtime.  Those callers cannot create
// an sfs_session, because a session allocates its scratch.  This entry point does the same work as
// sfs_select with the scratch (per-position row statistics, per-sequence row lists, the completion ticket)
// placed in one file-scope __device__ array of fixed size that is part of the library image.
//
// Consequences the caller must know:
//   * every GPU that loads the library holds the array (SFS_STATIC_SCRATCH_BYTES) until the process exits;
//   * B * S must not exceed SFS_STATIC_MAX_POSITIONS and B must not exceed SFS_STATIC_MAX_BATCH;
//   * all calls share the one array: two calls whose kernels can overlap on the GPU (different streams,
//     different host threads) race with each other - serialise them;
//   * the first call on each device looks up the array's device address (cudaGetSymbolAddress); make that
//     first call before starting any stream capture.
#include "sfs_common.cuh"

namespace {

struct StaticScratch {
    unsigned long long pos_sq[SFS_STATIC_MAX_POSITIONS];
    int32_t pos_arg[SFS_STATIC_MAX_POSITIONS];
    int32_t seq_rows[SFS_STATIC_MAX_POSITIONS];
    int32_t seq_row_count[SFS_STATIC_MAX_BATCH];
    int32_t ticket[4];
    int32_t status[4];            // [0]: device status of the call in flight (a bounded wait that gave up, a row index outside the grid)
};

// In host code this name is only a handle for the runtime, not a device address: it is never passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

StaticScratch *g_scratch_ptr[sfs::kMaxDevices] = {};

// folds the call's device status into every sequence's state.status (first error wins), so that a caller that may not
// allocate still sees a device-side failure where it already looks
__global__ void fold_status_kernel(const int32_t *status, sfs_state *state, int B)
{
    const int32_t s = *status;
    if (s == SFS_OK) return;
    for (int b = threadIdx.x; b < B; b += blockDim.x)
        if (state[b].status == SFS_OK) state[b].status = s;
}

// device address of the array on the current device, looked up once per device
int32_t scratch_for_current_device(StaticScratch **out)
{
    int dev = -1;
    SFS_CUDA(cudaGetDevice(&dev));
    SFS_REQUIRE(dev >= 0 && dev < sfs::kMaxDevices, SFS_ERR_UNSUPPORTED, "device ordinal %d not supported", dev);
    if (g_scratch_ptr[dev] == nullptr) {
        void *p = nullptr;
        SFS_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        SFS_REQUIRE(p != nullptr, SFS_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_scratch_ptr[dev] = reinterpret_cast<StaticScratch *>(p);
    }
    *out = g_scratch_ptr[dev];
    return SFS_OK;
}

}  // namespace

extern "C" int32_t sfs_select_static(int32_t vocab, const void *d_logits, int32_t logits_dtype, int64_t ld,
                                     const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                                     int32_t *d_tokens, uint8_t *d_mask, int32_t B, int32_t S, int32_t P,
                                     sfs_state *d_state, const sfs_params *params,
                                     int32_t *d_sel_count, int32_t *d_sel_pos, int32_t *d_sel_tok,
                                     int32_t *d_next_rows, int32_t *d_next_n_rows, int32_t *d_trace, void *stream)
{
    using namespace sfs;
    SFS_REQUIRE(d_logits && d_rows && d_tokens && d_mask && d_state && params, SFS_ERR_INVALID_ARG, "select_static: NULL pointer");
    SFS_REQUIRE((d_sel_pos == nullptr) == (d_sel_tok == nullptr), SFS_ERR_INVALID_ARG, "d_sel_pos and d_sel_tok go together");
    SFS_REQUIRE(vocab >= 1 && vocab < (1 << 19) && ld >= vocab, SFS_ERR_INVALID_ARG, "select_static: vocab %d / ld %lld", vocab, (long long)ld);
    SFS_REQUIRE(logits_dtype == SFS_LOGITS_BF16 || logits_dtype == SFS_LOGITS_F32, SFS_ERR_INVALID_ARG, "logits_dtype %d", logits_dtype);
    SFS_REQUIRE(B >= 1 && S >= 1 && P >= 0 && P <= S, SFS_ERR_INVALID_ARG, "select_static: B=%d S=%d P=%d", B, S, P);
    SFS_REQUIRE(B <= SFS_STATIC_MAX_BATCH && (long long)B * S <= SFS_STATIC_MAX_POSITIONS, SFS_ERR_UNSUPPORTED,
                "select_static: B=%d, B*S=%lld exceed the built-in scratch (at most %d sequences, %d token positions); "
                "use sfs_select with a session", B, (long long)B * S, SFS_STATIC_MAX_BATCH, SFS_STATIC_MAX_POSITIONS);
    SFS_REQUIRE(max_rows >= 0 && max_rows <= B * S, SFS_ERR_INVALID_ARG, "max_rows %d outside [0, B*S]", max_rows);
    SFS_REQUIRE(params->w_hist >= 1 && params->w_hist <= SFS_MAX_W_HIST && params->k_max >= 1 && params->k_slow >= 1 &&
                params->k_fast >= 1 && params->max_steps >= 0 && params->min_high_count >= 1, SFS_ERR_INVALID_ARG,
                "select_static: hyper-parameters out of range");
    SFS_REQUIRE(params->sampler >= SFS_SAMPLER_SLOWFAST && params->sampler <= SFS_SAMPLER_RANDOM && params->block_len >= 0,
                SFS_ERR_INVALID_ARG, "select_static: sampler %d / block_len %d", params->sampler, params->block_len);
    if (params->sampler != SFS_SAMPLER_SLOWFAST && S > P) {
        const int L = S - P, N = params->max_steps > 0 ? params->max_steps : L;
        const int bl = (params->block_len > 0 && params->block_len < L) ? params->block_len : L;
        SFS_REQUIRE(N % ((L + bl - 1) / bl) == 0, SFS_ERR_INVALID_ARG, "select_static: max_steps %d is not a multiple of the number of blocks", N);
    }
    StaticScratch *sc = nullptr;
    int32_t rc = scratch_for_current_device(&sc);
    if (rc != SFS_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps what the previous call left: everything that must start at zero is cleared here
    SFS_CUDA(cudaMemsetAsync(sc->pos_sq, 0, sizeof(unsigned long long) * (size_t)B * S, st));
    SFS_CUDA(cudaMemsetAsync(sc->ticket, 0, sizeof(sc->ticket) + sizeof(sc->status), st));
    rc = launch_row_stats(d_logits, logits_dtype, vocab, ld, d_n_rows, max_rows, d_rows, nullptr, nullptr, nullptr,
                          sc->pos_sq, sc->pos_arg, B * S, sc->status, st);
    if (rc != SFS_OK) return rc;
    SelectArgs a{};
    a.tokens = d_tokens; a.mask = d_mask; a.B = B; a.S = S; a.P = P; a.L = S - P;
    a.state = d_state; a.params = *params;
    a.pos_sq = sc->pos_sq; a.pos_arg = sc->pos_arg;
    a.sel_count = d_sel_count; a.sel_pos = d_sel_pos; a.sel_tok = d_sel_tok;
    a.seq_rows = sc->seq_rows; a.seq_row_count = sc->seq_row_count;
    a.next_rows = d_next_rows; a.next_n_rows = d_next_n_rows; a.n_active = nullptr;
    a.ticket = sc->ticket; a.trace = d_trace;
    if ((rc = launch_select(a, st)) != SFS_OK) return rc;
    fold_status_kernel<<<1, 64, 0, st>>>(sc->status, d_state, B);
    SFS_LAUNCH_CHECK();
    return SFS_OK;
}
