// C-ABI entry points of libsfs (declared in include/sfs.h): argument validation, workspace ownership and
// the order in which the kernels of one denoising step are enqueued.
#include "sfs_common.cuh"
#include "model.cuh"
#include "gemm.cuh"

#include <new>
#include <string.h>

namespace sfs {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

static int32_t check_params(const sfs_params *p)
{
    SFS_REQUIRE(p != nullptr, SFS_ERR_INVALID_ARG, "params is NULL");
    SFS_REQUIRE(p->w_hist >= 1 && p->w_hist <= SFS_MAX_W_HIST, SFS_ERR_INVALID_ARG, "w_hist %d outside [1, %d]", p->w_hist, SFS_MAX_W_HIST);
    SFS_REQUIRE(p->k_max >= 1, SFS_ERR_INVALID_ARG, "k_max %d must be >= 1", p->k_max);
    SFS_REQUIRE(p->k_slow >= 1 && p->k_fast >= 1, SFS_ERR_INVALID_ARG, "k_slow / k_fast must be >= 1");
    SFS_REQUIRE(p->max_steps >= 0 && p->min_high_count >= 1, SFS_ERR_INVALID_ARG, "max_steps must be >= 0 and min_high_count >= 1");
    SFS_REQUIRE(p->sigma2_stable == p->sigma2_stable && p->tau_min_conf == p->tau_min_conf && p->tau_high_conf == p->tau_high_conf,
                SFS_ERR_INVALID_ARG, "NaN threshold");
    return SFS_OK;
}

// one sticky device status word per process (set by kernels whose bounded waits give up)
int32_t *device_status_word()
{
    static int32_t *w = nullptr;
    if (!w) {
        if (cudaMalloc(&w, 256) != cudaSuccess) { w = nullptr; return nullptr; }
        cudaMemset(w, 0, 256);
    }
    return w;
}

}  // namespace sfs

using namespace sfs;

extern "C" {

const char *sfs_last_error(void) { return g_err; }
int32_t sfs_version(void) { return 100; }

const char *sfs_status_string(int32_t s)
{
    switch (s) {
        case SFS_OK: return "ok";
        case SFS_ERR_INVALID_ARG: return "invalid argument";
        case SFS_ERR_UNSUPPORTED: return "unsupported shape";
        case SFS_ERR_CUDA: return "CUDA error";
        case SFS_ERR_OOM: return "out of device memory";
        case SFS_ERR_STEP_LIMIT: return "step budget exhausted with masked positions left";
        case SFS_ERR_TIMEOUT: return "bounded device wait gave up";
        case SFS_ERR_MISSING_ROW: return "row statistics missing for a needed position";
        default: return "unknown status";
    }
}

int32_t sfs_row_stats(const void *d_logits, int32_t logits_dtype, int32_t vocab, int64_t ld,
                      const int32_t *d_n_rows, int32_t max_rows,
                      int32_t *d_argmax, uint64_t *d_sq, float *d_conf, void *stream)
{
    SFS_REQUIRE(d_logits != nullptr, SFS_ERR_INVALID_ARG, "d_logits is NULL");
    SFS_REQUIRE(logits_dtype == SFS_LOGITS_BF16 || logits_dtype == SFS_LOGITS_F32, SFS_ERR_INVALID_ARG, "logits_dtype %d", logits_dtype);
    SFS_REQUIRE(vocab >= 1 && vocab < (1 << 19), SFS_ERR_INVALID_ARG, "vocab %d outside [1, 2^19)", vocab);
    SFS_REQUIRE(ld >= vocab, SFS_ERR_INVALID_ARG, "ld %lld < vocab %d", (long long)ld, vocab);
    SFS_REQUIRE(max_rows >= 0, SFS_ERR_INVALID_ARG, "max_rows %d", max_rows);
    SFS_REQUIRE(aligned_to(d_logits, logits_dtype == SFS_LOGITS_BF16 ? 2 : 4), SFS_ERR_INVALID_ARG, "d_logits misaligned");
    return launch_row_stats(d_logits, logits_dtype, vocab, ld, d_n_rows, max_rows, nullptr, d_argmax,
                            reinterpret_cast<unsigned long long *>(d_sq), d_conf, nullptr, nullptr, (cudaStream_t)stream);
}

int32_t sfs_state_init(sfs_state *d_state, int32_t B, int32_t gen_len, const sfs_params *params, void *stream)
{
    SFS_REQUIRE(d_state != nullptr && B >= 1 && gen_len >= 0, SFS_ERR_INVALID_ARG, "state_init: bad arguments");
    int32_t rc = check_params(params);
    if (rc != SFS_OK) return rc;
    return launch_state_init(d_state, B, gen_len, *params, nullptr, (cudaStream_t)stream);
}

int32_t sfs_select(sfs_session *s, const void *d_logits, int32_t logits_dtype, int64_t ld,
                   const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                   int32_t *d_tokens, uint8_t *d_mask, int32_t B, int32_t S, int32_t P,
                   sfs_state *d_state, const sfs_params *params,
                   int32_t *d_sel_count, int32_t *d_sel_pos, int32_t *d_sel_tok,
                   int32_t *d_next_rows, int32_t *d_next_n_rows, int32_t *d_trace, void *stream)
{
    SFS_REQUIRE(s != nullptr, SFS_ERR_INVALID_ARG, "session is NULL");
    SFS_REQUIRE(d_logits && d_rows && d_tokens && d_mask && d_state, SFS_ERR_INVALID_ARG, "select: NULL device pointer");
    SFS_REQUIRE((d_sel_pos == nullptr) == (d_sel_tok == nullptr), SFS_ERR_INVALID_ARG, "d_sel_pos and d_sel_tok go together");
    SFS_REQUIRE(B >= 1 && B <= s->max_batch && S >= 1 && S <= s->max_seq && P >= 0 && P <= S, SFS_ERR_INVALID_ARG,
                "select: B=%d S=%d P=%d outside the session's limits (%d, %d)", B, S, P, s->max_batch, s->max_seq);
    SFS_REQUIRE(max_rows >= 0 && max_rows <= B * S, SFS_ERR_INVALID_ARG, "max_rows %d outside [0, B*S]", max_rows);
    SFS_REQUIRE(logits_dtype == SFS_LOGITS_BF16 || logits_dtype == SFS_LOGITS_F32, SFS_ERR_INVALID_ARG, "logits_dtype %d", logits_dtype);
    const int32_t vocab = s->vocab;
    SFS_REQUIRE(ld >= vocab, SFS_ERR_INVALID_ARG, "ld %lld < vocab %d", (long long)ld, vocab);
    int32_t rc = check_params(params);
    if (rc != SFS_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    rc = launch_row_stats(d_logits, logits_dtype, vocab, ld, d_n_rows, max_rows, d_rows, nullptr, nullptr, nullptr,
                          s->pos_sq, s->pos_arg, st);
    if (rc != SFS_OK) return rc;
    SelectArgs a{};
    a.tokens = d_tokens; a.mask = d_mask; a.B = B; a.S = S; a.P = P; a.L = S - P;
    a.state = d_state; a.params = *params;
    a.pos_sq = s->pos_sq; a.pos_arg = s->pos_arg;
    a.sel_count = d_sel_count; a.sel_pos = d_sel_pos; a.sel_tok = d_sel_tok;
    a.seq_rows = s->seq_rows; a.seq_row_count = s->seq_row_count;
    a.next_rows = d_next_rows; a.next_n_rows = d_next_n_rows; a.n_active = nullptr;
    a.ticket = s->ticket; a.trace = d_trace;
    return launch_select(a, st);
}

}  // extern "C"

// ---- sessions -------------------------------------------------------------------------------------------
namespace sfs {
template <typename T>
static int32_t dev_alloc(sfs_session *s, T **out, size_t count, bool zero)
{
    void *p = nullptr;
    SFS_CUDA(cudaMalloc(&p, count * sizeof(T) > 0 ? count * sizeof(T) : 16));
    s->owned.push_back(p);
    if (zero) SFS_CUDA(cudaMemset(p, 0, count * sizeof(T)));
    *out = reinterpret_cast<T *>(p);
    return SFS_OK;
}
}  // namespace sfs

extern "C" {

static int32_t session_alloc_select(sfs_session *s)
{
    const size_t n = (size_t)s->max_batch * s->max_seq;
    int32_t rc;
    if ((rc = dev_alloc(s, &s->pos_sq, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->pos_arg, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->seq_rows, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->seq_row_count, (size_t)s->max_batch, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->ticket, 4, true)) != SFS_OK) return rc;
    return SFS_OK;
}

int32_t sfs_session_destroy(sfs_session *s)
{
    if (!s) return SFS_OK;
    cudaDeviceSynchronize();
    for (void *p : s->owned) cudaFree(p);
    delete s;
    return SFS_OK;
}

int32_t sfs_select_session_create(int32_t vocab, int32_t max_batch, int32_t max_seq, sfs_session **out)
{
    SFS_REQUIRE(out != nullptr, SFS_ERR_INVALID_ARG, "out is NULL");
    SFS_REQUIRE(vocab >= 1 && vocab < (1 << 19), SFS_ERR_INVALID_ARG, "vocab %d outside [1, 2^19)", vocab);
    SFS_REQUIRE(max_batch >= 1 && max_seq >= 1 && max_seq < (1 << 17) && (long long)max_batch * max_seq < (1ll << 30),
                SFS_ERR_INVALID_ARG, "max_batch %d / max_seq %d out of range", max_batch, max_seq);
    sfs_session *s = new (std::nothrow) sfs_session();
    SFS_REQUIRE(s != nullptr, SFS_ERR_OOM, "host allocation failed");
    s->max_batch = max_batch; s->max_seq = max_seq; s->vocab = vocab;
    int32_t rc = session_alloc_select(s);
    if (rc != SFS_OK) { sfs_session_destroy(s); return rc; }
    SFS_CUDA(cudaDeviceSynchronize());
    *out = s;
    return SFS_OK;
}

}  // extern "C"

extern "C" {

int32_t sfs_linear(const void *d_A, int64_t lda, const void *d_B, int64_t ldb, void *d_C, int64_t ldc,
                   int32_t M, int32_t N, int32_t K, int32_t out_dtype, float scale, void *stream)
{
    SFS_REQUIRE(d_A && d_B && d_C, SFS_ERR_INVALID_ARG, "linear: NULL pointer");
    SFS_REQUIRE(M >= 1 && N >= 1 && K >= 1, SFS_ERR_INVALID_ARG, "linear: M, N, K must be positive");
    SFS_REQUIRE(out_dtype == 0 || out_dtype == 1, SFS_ERR_INVALID_ARG, "linear: out_dtype %d", out_dtype);
    int32_t *err = device_status_word();
    SFS_REQUIRE(err != nullptr, SFS_ERR_OOM, "cannot allocate the device status word");
    GemmPlan plan;
    const void *bs[1] = {d_B};
    int32_t rc = gemm_plan_create(&plan, d_A, lda, M, K, bs, 1, N, ldb, GEMM_STORE, d_C, ldc, out_dtype, scale, nullptr, 0, 0, 0);
    if (rc != SFS_OK) return rc;
    return gemm_launch(plan, nullptr, err, (cudaStream_t)stream);
}

int32_t sfs_check_device_status(void *stream)
{
    int32_t *err = device_status_word();
    SFS_REQUIRE(err != nullptr, SFS_ERR_OOM, "cannot allocate the device status word");
    SFS_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    int32_t h = 0;
    SFS_CUDA(cudaMemcpy(&h, err, 4, cudaMemcpyDeviceToHost));
    if (h != 0) {
        cudaMemset(err, 0, 4);
        set_error("a kernel reported device status %d (%s)", h, sfs_status_string(h));
    }
    return h;
}

}  // extern "C"
