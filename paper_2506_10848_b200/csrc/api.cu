// C-ABI entry points of libsfs (declared in include/sfs.h): argument validation, workspace ownership and
// the order in which the kernels of one denoising step are enqueued.
#include "sfs_common.cuh"
#include "model.cuh"
#include "gemm.cuh"
#include "attention.cuh"
#include "elementwise.cuh"
#include "cache.cuh"
#include <math.h>

#include <new>
#include <string.h>

namespace sfs {

static thread_local char g_err[512] = "";
static constexpr int kMaxSplits = 6;           // slabs of the split-K workspace of the residual projections

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

// gen_len < 0: the response length is not known to the caller of this check
static int32_t check_params(const sfs_params *p, int32_t gen_len = -1)
{
    SFS_REQUIRE(p != nullptr, SFS_ERR_INVALID_ARG, "params is NULL");
    SFS_REQUIRE(p->sampler >= SFS_SAMPLER_SLOWFAST && p->sampler <= SFS_SAMPLER_RANDOM, SFS_ERR_INVALID_ARG, "sampler %d", p->sampler);
    SFS_REQUIRE(p->block_len >= 0, SFS_ERR_INVALID_ARG, "block_len %d must be >= 0", p->block_len);
    if (p->sampler != SFS_SAMPLER_SLOWFAST && gen_len > 0) {
        const int N = p->max_steps > 0 ? p->max_steps : gen_len;
        const int bl = (p->block_len > 0 && p->block_len < gen_len) ? p->block_len : gen_len;
        const int nb = (gen_len + bl - 1) / bl;
        SFS_REQUIRE(N % nb == 0, SFS_ERR_INVALID_ARG, "max_steps %d must be a multiple of the %d blocks of %d positions", N, nb, bl);
    }
    SFS_REQUIRE(p->w_hist >= 1 && p->w_hist <= SFS_MAX_W_HIST, SFS_ERR_INVALID_ARG, "w_hist %d outside [1, %d]", p->w_hist, SFS_MAX_W_HIST);
    SFS_REQUIRE(p->k_max >= 1, SFS_ERR_INVALID_ARG, "k_max %d must be >= 1", p->k_max);
    SFS_REQUIRE(p->k_slow >= 1 && p->k_fast >= 1, SFS_ERR_INVALID_ARG, "k_slow / k_fast must be >= 1");
    SFS_REQUIRE(p->max_steps >= 0 && p->min_high_count >= 1, SFS_ERR_INVALID_ARG, "max_steps must be >= 0 and min_high_count >= 1");
    SFS_REQUIRE(p->sigma2_stable == p->sigma2_stable && p->tau_min_conf == p->tau_min_conf && p->tau_high_conf == p->tau_high_conf,
                SFS_ERR_INVALID_ARG, "NaN threshold");
    return SFS_OK;
}

// one sticky status word per device
static int32_t *g_status_word[kMaxDevices] = {};
int32_t *device_status_word()
{
    int32_t *&w = g_status_word[current_device_slot()];
    if (!w) {
        if (cudaMalloc(&w, 256) != cudaSuccess) { w = nullptr; return nullptr; }
        cudaMemset(w, 0, 256);
    }
    return w;
}
int32_t *device_status_word_if_any() { return g_status_word[current_device_slot()]; }

template <typename T>
static int32_t dev_alloc(sfs_session *s, T **out, size_t count, bool zero)
{
    void *p = nullptr;
    const size_t bytes = count * sizeof(T) > 0 ? count * sizeof(T) : 16;
    SFS_CUDA(cudaMalloc(&p, bytes));
    s->owned.push_back(p);
    if (zero) SFS_CUDA(cudaMemset(p, 0, bytes));
    *out = reinterpret_cast<T *>(p);
    return SFS_OK;
}

// Row statistics of one selection step into the session's scratch: the two-pass (filter + exact) form for long bf16 rows,
// the all-canonical kernels otherwise.  Either way the selection kernel finds, for every supplied row the rule reads, a
// value in pos_sq that gives the decisions of the canonical S_q.
static int32_t step_row_stats(sfs_session *s, const void *d_logits, int32_t logits_dtype, int32_t vocab, int64_t ld,
                              const int32_t *d_n_rows, int32_t max_rows, const int32_t *d_rows, const uint8_t *d_mask,
                              int32_t B, int32_t S, int32_t P, const sfs_state *d_state, const sfs_params &params, bool *two_pass,
                              cudaStream_t st, const float4 *lm_stats = nullptr, int32_t lm_stats_ld = 0)
{
    int32_t *err = device_status_word();
    *two_pass = row_stats_two_pass_applies(d_logits, logits_dtype, vocab, ld);
    if (!*two_pass)
        return launch_row_stats(d_logits, logits_dtype, vocab, ld, d_n_rows, max_rows, d_rows, nullptr, nullptr, nullptr,
                                s->pos_sq, s->pos_arg, B * S, err, st);
    RefineArgs rf{};
    rf.mask = d_mask; rf.B = B; rf.S = S; rf.P = P; rf.L = S - P; rf.state = d_state; rf.params = params;
    rf.pos_lo = s->pos_lo; rf.pos_hi = s->pos_hi; rf.pos_sq = s->pos_sq; rf.pos_arg = s->pos_arg;
    rf.slice_partials = s->slice_partials; rf.row_tickets = s->row_tickets;
    rf.pos_row = s->pos_row; rf.pos_max = s->pos_max; rf.refine_list = s->refine_list; rf.refine_count = s->refine_count;
    if (lm_stats != nullptr)       // the LM head's epilogue has taken the first pass: the logits are read only for the listed rows
        return launch_row_stats_from_partials(lm_stats, lm_stats_ld, lm_stats_ld, d_logits, vocab, ld, d_n_rows, max_rows, d_rows, rf, err, st);
    return launch_row_stats_two_pass(d_logits, vocab, ld, d_n_rows, max_rows, d_rows, rf, err, st);
}

static int32_t session_alloc_select(sfs_session *s)
{
    const size_t n = (size_t)s->max_batch * s->max_seq;
    int32_t rc;
    if ((rc = dev_alloc(s, &s->pos_sq, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->pos_arg, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->pos_lo, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->pos_hi, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->slice_partials, n * kRowStatsSlices * 4, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->row_tickets, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->pos_row, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->pos_max, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->refine_list, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->refine_count, 4, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->seq_rows, n, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->seq_row_count, (size_t)s->max_batch, true)) != SFS_OK) return rc;
    if ((rc = dev_alloc(s, &s->ticket, 4, true)) != SFS_OK) return rc;
    return SFS_OK;
}

// (re)build the GEMM / attention plans of a model session for B sequences of S tokens
static int32_t session_plan(sfs_session *s, int32_t B, int32_t S)
{
    if (s->plan_B == B && s->plan_S == S) return SFS_OK;
    const sfs_model *m = s->model;
    const sfs_config &c = m->cfg;
    const int T = B * S, d = c.d_model, ff = c.d_ff;
    SFS_REQUIRE((S % 8) == 0, SFS_ERR_UNSUPPORTED, "sequence length %d must be a multiple of 8", S);
    s->layer_plans.resize(c.n_layers);
    int32_t rc;
    for (int l = 0; l < c.n_layers; ++l) {
        LayerPlans &lp = s->layer_plans[l];
        const void *qkv[3] = {m->wq[l], m->wk[l], m->wv[l]};
        // q | k go row-major into qk [T, 2d]; the v columns (>= 2d) go transposed into vt [d, T]
        rc = gemm_plan_create(&lp.qkv, s->h, d, T, d, qkv, 3, d, d, GEMM_STORE, s->qk, 2 * d, 0, 1.0f, s->vt, T, 2 * d, nullptr);
        if (rc != SFS_OK) return rc;
        const void *wo[1] = {m->wo[l]};
        rc = gemm_plan_create(&lp.o, s->attn, d, T, d, wo, 1, d, d, GEMM_RESIDUAL_F32, s->x, d, 1, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        if ((rc = gemm_plan_enable_split(&lp.o, s->partial, kMaxSplits, nullptr)) != SFS_OK) return rc;
        const void *gu[2] = {m->w_gate[l], m->w_up[l]};
        rc = gemm_plan_create(&lp.gate_up, s->h, d, T, d, gu, 2, ff, d, GEMM_SWIGLU, s->hid, ff, 0, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        const void *wd[1] = {m->w_down[l]};
        rc = gemm_plan_create(&lp.down, s->hid, ff, T, ff, wd, 1, d, ff, GEMM_RESIDUAL_F32, s->x, d, 1, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        if ((rc = gemm_plan_enable_split(&lp.down, s->partial, kMaxSplits, nullptr)) != SFS_OK) return rc;
    }
    rc = attn_plan_create(&s->attn_plan, s->qk, 2 * d, s->vt, T, s->attn, d, B, S, c.n_heads, c.head_dim);
    if (rc != SFS_OK) return rc;
    s->plan_B = B; s->plan_S = S;
    return SFS_OK;
}

// Runs one launch; when profiling is on, brackets it with CUDA events tagged with the kernel class.
template <typename F>
static int32_t timed_launch(sfs_session *s, int cls, cudaStream_t st, F &&f)
{
    s->launches++;
    if (!s->profile) return f();
    sfs_session::Timed t; t.cls = cls;
    SFS_CUDA(cudaEventCreate(&t.e0)); SFS_CUDA(cudaEventCreate(&t.e1));
    SFS_CUDA(cudaEventRecord(t.e0, st));
    int32_t rc = f();
    SFS_CUDA(cudaEventRecord(t.e1, st));
    s->timed.push_back(t);
    return rc;
}

// the transformer body: tokens -> residual stream x [T, d]
static int32_t run_body(sfs_session *s, const int32_t *d_tokens, int32_t B, int32_t S, const int32_t *d_active, cudaStream_t st)
{
    const sfs_model *m = s->model;
    const sfs_config &c = m->cfg;
    const int T = B * S, d = c.d_model;
    int32_t *err = device_status_word();
    SFS_REQUIRE(err != nullptr, SFS_ERR_OOM, "cannot allocate the device status word");
    int32_t rc;
    if ((rc = timed_launch(s, SFS_K_EMBED, st, [&] { return launch_embed(d_tokens, m->tok_emb, s->x, T, d, c.vocab, st); })) != SFS_OK) return rc;
    // A split-K projection leaves its partial products in s->partial; the next RMSNorm folds them into x.
    const long long pstride = (long long)T * d;
    int pending = 0;
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerPlans &lp = s->layer_plans[l];
        if ((rc = timed_launch(s, SFS_K_RMSNORM, st, [&] { return launch_rmsnorm(s->x, s->partial, pending, pstride, m->attn_norm[l], s->h, nullptr, nullptr, T, d, c.rms_eps, st); })) != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_GEMM_QKV, st, [&] { return gemm_launch(lp.qkv, nullptr, d_active, err, st); })) != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_ROPE, st, [&] { return launch_rope(s->qk, 2 * d, T, S, c.n_heads, c.head_dim, s->rope_table, nullptr, st); })) != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_ATTENTION, st, [&] { return attn_launch(s->attn_plan, d_active, err, st); })) != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_GEMM_O, st, [&] { return gemm_launch(lp.o, nullptr, d_active, err, st); })) != SFS_OK) return rc;
        pending = lp.o.args.splits > 1 ? lp.o.args.splits : 0;
        if ((rc = timed_launch(s, SFS_K_RMSNORM, st, [&] { return launch_rmsnorm(s->x, s->partial, pending, pstride, m->mlp_norm[l], s->h, nullptr, nullptr, T, d, c.rms_eps, st); })) != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_GEMM_GATE_UP, st, [&] { return gemm_launch(lp.gate_up, nullptr, d_active, err, st); })) != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_GEMM_DOWN, st, [&] { return gemm_launch(lp.down, nullptr, d_active, err, st); })) != SFS_OK) return rc;
        pending = lp.down.args.splits > 1 ? lp.down.args.splits : 0;
    }
    s->pending_ptr = s->partial; s->pending_n = pending; s->pending_stride = pstride;      // for the final RMSNorm of the caller
    return SFS_OK;
}

// ---- cached steps --------------------------------------------------------------------------------------
// per-layer plans of the cached mode that do not depend on the number of recomputed rows
static int32_t cache_plan(sfs_session *s, int32_t B, int32_t S, int32_t P)
{
    const sfs_model *m = s->model;
    const sfs_config &c = m->cfg;
    const int T = B * S, d = c.d_model, ff = c.d_ff;
    if ((int)s->cache_plans.size() == c.n_layers && s->cache_B == B && s->cache_S == S && s->cache_P == P) return SFS_OK;
    s->cache_plans.assign(c.n_layers, CacheLayerPlans());
    s->gather_plans.clear();
    int32_t rc;
    for (int l = 0; l < c.n_layers; ++l) {
        CacheLayerPlans &cp = s->cache_plans[l];
        const void *wv[1] = {m->wv[l]};
        // fresh values of the candidate rows, written transposed (every output column goes through the transposed store): the
        // response rows of a single sequence are one contiguous range; with several sequences every row is projected
        const int v_first = (B == 1) ? P : 0, v_rows = (B == 1) ? S - P : T;
        rc = gemm_plan_create(&cp.vproj, s->h + (size_t)v_first * d, d, v_rows, d, wv, 1, d, d, GEMM_STORE, s->attn, d, 0, 1.0f, s->vnew_t + v_first, T, 0,
                              nullptr);
        if (rc != SFS_OK) return rc;
        const void *wo[1] = {m->wo[l]};
        rc = gemm_plan_create(&cp.o_store, s->attn, d, T, d, wo, 1, d, d, GEMM_STORE, s->Ac[l], d, 1, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        const void *wd[1] = {m->w_down[l]};
        rc = gemm_plan_create(&cp.down_store, s->hid, ff, T, ff, wd, 1, d, ff, GEMM_STORE, s->Fc[l], d, 1, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        rc = attn_plan_create_split(&cp.attn, s->qk, 2 * d, s->Kc[l], d, d, 0, s->Vtc[l], T, s->attn, d, B, S, c.n_heads, c.head_dim);
        if (rc != SFS_OK) return rc;
    }
    return SFS_OK;
}

// projections over the compact buffers of NR recomputed rows
static int32_t gather_plan(sfs_session *s, int32_t NR, int32_t T, std::vector<GatherLayerPlans> **out)
{
    auto it = s->gather_plans.find(NR);
    if (it != s->gather_plans.end()) { *out = &it->second; return SFS_OK; }
    const sfs_model *m = s->model;
    const sfs_config &c = m->cfg;
    const int d = c.d_model, ff = c.d_ff;
    std::vector<GatherLayerPlans> v(c.n_layers);
    int32_t rc;
    for (int l = 0; l < c.n_layers; ++l) {
        GatherLayerPlans &gp = v[l];
        const void *qkv[3] = {m->wq[l], m->wk[l], m->wv[l]};
        rc = gemm_plan_create(&gp.qkv, s->hg, d, NR, d, qkv, 3, d, d, GEMM_STORE, s->qk, 2 * d, 0, 1.0f, s->vt, T, 2 * d, nullptr);
        if (rc != SFS_OK) return rc;
        const void *wo[1] = {m->wo[l]};
        rc = gemm_plan_create(&gp.o, s->attn, d, NR, d, wo, 1, d, d, GEMM_STORE, s->partial, d, 1, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        if ((rc = gemm_plan_enable_split(&gp.o, s->partial, kMaxSplits, nullptr)) != SFS_OK) return rc;   // few rows: K is split
        const void *gu[2] = {m->w_gate[l], m->w_up[l]};
        rc = gemm_plan_create(&gp.gate_up, s->hg, d, NR, d, gu, 2, ff, d, GEMM_SWIGLU, s->hid, ff, 0, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        const void *wd[1] = {m->w_down[l]};
        rc = gemm_plan_create(&gp.down, s->hid, ff, NR, ff, wd, 1, d, ff, GEMM_STORE, s->partial, d, 1, 1.0f, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        if ((rc = gemm_plan_enable_split(&gp.down, s->partial, kMaxSplits, nullptr)) != SFS_OK) return rc;
    }
    auto ins = s->gather_plans.emplace(NR, std::move(v));
    *out = &ins.first->second;
    return SFS_OK;
}

// One cached step of the transformer body (the rule is stated with sfs_cache_params in sfs.h): tokens -> x [T, d],
// leaving the last layer's MLP increment pending for the caller's final RMSNorm.
static int32_t run_body_cached(sfs_session *s, const int32_t *d_tokens, int32_t B, int32_t S, int32_t P, const sfs_state *d_state,
                               const int32_t *d_active, int32_t *d_sets, float *d_sims, int32_t *n_sel_out, cudaStream_t st)
{
    const sfs_model *m = s->model;
    const sfs_config &c = m->cfg;
    const int T = B * S, L = S - P, d = c.d_model;
    SFS_REQUIRE(s->cache_on, SFS_ERR_INVALID_ARG, "cached step: call sfs_cache_enable first");
    SFS_REQUIRE(P >= 0 && L >= 1, SFS_ERR_INVALID_ARG, "cached step: P=%d S=%d", P, S);
    if (s->cache_t != 0)
        SFS_REQUIRE(s->cache_B == B && s->cache_S == S && s->cache_P == P, SFS_ERR_INVALID_ARG,
                    "cached step: the cached features belong to B=%d S=%d P=%d; call sfs_cache_reset before changing the shape",
                    s->cache_B, s->cache_S, s->cache_P);
    int32_t *err = device_status_word();
    SFS_REQUIRE(err != nullptr, SFS_ERR_OOM, "cannot allocate the device status word");
    int32_t rc;
    if ((rc = session_plan(s, B, S)) != SFS_OK) return rc;
    if ((rc = cache_plan(s, B, S, P)) != SFS_OK) return rc;
    s->cache_B = B; s->cache_S = S; s->cache_P = P;
    const sfs_cache_params &cp = s->cache_params;
    const bool rp = (s->cache_t % cp.k_prompt) == 0, rr = (s->cache_t % cp.k_response) == 0;
    int n_adapt = (int)ceil(cp.rho * (double)L);
    n_adapt = n_adapt < 0 ? 0 : (n_adapt > L ? L : n_adapt);
    const int n_sel = (rp ? P : 0) + (rr ? L : n_adapt);
    if (n_sel_out) *n_sel_out = (rp && rr) ? S : n_sel;
    const int NR = B * n_sel;

    if ((rc = timed_launch(s, SFS_K_EMBED, st, [&] { return launch_embed(d_tokens, m->tok_emb, s->x, T, d, c.vocab, st); })) != SFS_OK) return rc;
    const float *pend = nullptr;
    // Rows whose residual stream this step keeps up to date: all of them, except that a single sequence whose prompt is not
    // refreshed needs only its response rows (nothing reads the prompt rows of x or h then).
    const int r_first = (B == 1 && !rp) ? P : 0, r_count = (B == 1 && !rp) ? L : T;
    // tokens whose fresh values are compared with the cached ones: the response of a single sequence (from an even index), else all
    const int sim_first = (B == 1) ? (P & ~1) : 0, sim_count = (B == 1) ? S - sim_first : T;
    auto norm_all = [&](const void *gain) {
        return timed_launch(s, SFS_K_RMSNORM, st, [&] {
            return launch_rmsnorm(s->x + (size_t)r_first * d, pend ? pend + (size_t)r_first * d : nullptr, pend ? 1 : 0, 0, gain,
                                  s->h + (size_t)r_first * d, nullptr, nullptr, r_count, d, c.rms_eps, st);
        });
    };
    if (rp && rr) {
        // everything is recomputed: the uncached layer pipeline, with the increments stored instead of added and K / V copied out
        for (int l = 0; l < c.n_layers; ++l) {
            const LayerPlans &lp = s->layer_plans[l];
            const CacheLayerPlans &cl = s->cache_plans[l];
            if ((rc = norm_all(m->attn_norm[l])) != SFS_OK) return rc;
            if ((rc = timed_launch(s, SFS_K_GEMM_QKV, st, [&] { return gemm_launch(lp.qkv, nullptr, d_active, err, st); })) != SFS_OK) return rc;
            if ((rc = timed_launch(s, SFS_K_ROPE, st, [&] { return launch_rope(s->qk, 2 * d, T, S, c.n_heads, c.head_dim, s->rope_table, nullptr, st); })) != SFS_OK) return rc;
            SFS_CUDA(cudaMemcpy2DAsync(s->Kc[l], (size_t)d * 2, s->qk + d, (size_t)2 * d * 2, (size_t)d * 2, (size_t)T, cudaMemcpyDeviceToDevice, st));
            SFS_CUDA(cudaMemcpyAsync(s->Vtc[l], s->vt, (size_t)d * T * 2, cudaMemcpyDeviceToDevice, st));
            if ((rc = timed_launch(s, SFS_K_ATTENTION, st, [&] { return attn_launch(s->attn_plan, d_active, err, st); })) != SFS_OK) return rc;
            if ((rc = timed_launch(s, SFS_K_GEMM_O, st, [&] { return gemm_launch(cl.o_store, nullptr, d_active, err, st); })) != SFS_OK) return rc;
            pend = s->Ac[l];
            if ((rc = norm_all(m->mlp_norm[l])) != SFS_OK) return rc;
            if ((rc = timed_launch(s, SFS_K_GEMM_GATE_UP, st, [&] { return gemm_launch(lp.gate_up, nullptr, d_active, err, st); })) != SFS_OK) return rc;
            if ((rc = timed_launch(s, SFS_K_GEMM_DOWN, st, [&] { return gemm_launch(cl.down_store, nullptr, d_active, err, st); })) != SFS_OK) return rc;
            pend = s->Fc[l];
            if (d_sets) {   // the dump lists every token
                CacheSelectArgs a{}; a.B = B; a.S = S; a.P = P; a.L = L; a.T = T; a.refresh_p = 1; a.refresh_r = 1; a.n_sel = S;
                a.sel_rows = d_sets + (size_t)l * B * S;
                if ((rc = launch_cache_select(a, st)) != SFS_OK) return rc;
            }
        }
    } else {
        std::vector<GatherLayerPlans> *gps = nullptr;
        if (NR > 0 && (rc = gather_plan(s, NR, T, &gps)) != SFS_OK) return rc;
        // Here the attention increment of a layer stays pending through its MLP branch: the MLP norm reads x + A_l for the
        // recomputed rows only (straight into the compact buffer), and the next layer's first norm folds A_l and F_l together.
        const long long inc_stride = (long long)s->max_batch * s->max_seq * d;     // A_l -> F_l
        int n_pend = 0;
        for (int l = 0; l < c.n_layers; ++l) {
            const CacheLayerPlans &cl = s->cache_plans[l];
            rc = timed_launch(s, SFS_K_RMSNORM, st, [&] {
                return launch_rmsnorm(s->x + (size_t)r_first * d, pend ? pend + (size_t)r_first * d : nullptr, n_pend, inc_stride, m->attn_norm[l],
                                      s->h + (size_t)r_first * d, nullptr, nullptr, r_count, d, c.rms_eps, st);
            });
            if (rc != SFS_OK) return rc;
            if (NR > 0) {
                const GatherLayerPlans &gp = (*gps)[l];
                if (!rr && n_adapt > 0) {
                    if ((rc = timed_launch(s, SFS_K_GEMM_QKV, st, [&] { return gemm_launch(cl.vproj, nullptr, d_active, err, st); })) != SFS_OK) return rc;
                    if ((rc = timed_launch(s, SFS_K_CACHE, st, [&] { return launch_sim_partial(s->vnew_t, s->Vtc[l], T, d, sim_first, sim_count, T, s->sim_partial, st); })) != SFS_OK) return rc;
                }
                CacheSelectArgs a{};
                a.partial = s->sim_partial; a.state = d_state; a.B = B; a.S = S; a.P = P; a.L = L; a.T = T;
                a.refresh_p = rp; a.refresh_r = rr; a.n_adapt = rr ? 0 : n_adapt; a.n_sel = n_sel; a.sel_rows = s->sel_rows;
                a.sims_dump = (d_sims && !rr) ? d_sims + (size_t)l * B * L : nullptr;
                a.sets_dump = d_sets ? d_sets + (size_t)l * NR : nullptr;
                if ((rc = timed_launch(s, SFS_K_CACHE, st, [&] { return launch_cache_select(a, st); })) != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_CACHE, st, [&] { return launch_gather_rows_bf16(s->h, s->sel_rows, NR, d, s->hg, st); })) != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_GEMM_QKV, st, [&] { return gemm_launch(gp.qkv, nullptr, d_active, err, st); })) != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_ROPE, st, [&] { return launch_rope_scatter_kv(s->qk, 2 * d, NR, S, c.n_heads, c.head_dim, s->rope_table, s->sel_rows, s->Kc[l], s->vt, T, s->Vtc[l], T, st); })) != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_ATTENTION, st, [&] { return attn_launch_queries(cl.attn, n_sel, d_active, err, st); })) != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_GEMM_O, st, [&] { return gemm_launch(gp.o, nullptr, d_active, err, st); })) != SFS_OK) return rc;
            }
            pend = s->Ac[l]; n_pend = 2;
            if (NR > 0) {
                const GatherLayerPlans &gp = (*gps)[l];
                // the O projection's slabs become the attention increments of the recomputed tokens, and the MLP's input rows
                rc = timed_launch(s, SFS_K_RMSNORM, st, [&] {
                    return launch_fold_norm_rows(s->partial, gp.o.args.splits, gp.o.args.split_stride, s->sel_rows, NR, s->x, s->Ac[l],
                                                 m->mlp_norm[l], s->hg, d, c.rms_eps, st);
                });
                if (rc != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_GEMM_GATE_UP, st, [&] { return gemm_launch(gp.gate_up, nullptr, d_active, err, st); })) != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_GEMM_DOWN, st, [&] { return gemm_launch(gp.down, nullptr, d_active, err, st); })) != SFS_OK) return rc;
                if ((rc = timed_launch(s, SFS_K_CACHE, st, [&] { return launch_scatter_rows_f32(s->partial, gp.down.args.splits, gp.down.args.split_stride, s->sel_rows, NR, d, s->Fc[l], st); })) != SFS_OK) return rc;
            }
        }
        s->pending_ptr = pend; s->pending_n = pend ? n_pend : 0; s->pending_stride = inc_stride;
        s->cache_t++;
        return SFS_OK;
    }
    s->pending_ptr = pend; s->pending_n = pend ? 1 : 0; s->pending_stride = 0;
    s->cache_t++;
    return SFS_OK;
}

__global__ void generate_init_kernel(const int32_t *prompt, int32_t *tokens, uint8_t *mask, int32_t *rows, int32_t *ctrl,
                                     int32_t *host_active, unsigned long long *pos_sq, int B, int P, int L, int mask_id)
{
    const int S = P + L;
    const long long n = (long long)B * S;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int b = (int)(i / S), pos = (int)(i % S);
        tokens[i] = pos < P ? prompt[(long long)b * P + pos] : mask_id;
        mask[i] = pos < P ? 0 : 1;
        pos_sq[i] = 0;
        if (pos >= P) rows[(long long)b * L + (pos - P)] = (int)i;         // first step: every response row, sequence-major
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctrl[0] = B * L; ctrl[1] = 0; ctrl[2] = (L > 0) ? B : 0;
        *host_active = (L > 0) ? B : 0;
    }
}

// host_active[0]: sequences still decoding; host_active[1]: denoising steps the device has finished in this generation
__global__ void mirror_active_kernel(const int32_t *ctrl_active, int32_t *host_active, int32_t steps_done)
{
    pdl_wait();
    pdl_trigger();
    host_active[1] = steps_done;
    __threadfence_system();
    host_active[0] = *ctrl_active;
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

// ---- model ----------------------------------------------------------------------------------------------
int32_t sfs_model_create(const sfs_config *cfg, const sfs_weights *w, sfs_model **out)
{
    SFS_REQUIRE(cfg && w && out, SFS_ERR_INVALID_ARG, "model_create: NULL argument");
    SFS_REQUIRE(cfg->n_layers >= 1 && cfg->d_model >= 8 && cfg->n_heads >= 1 && cfg->d_ff >= 8 && cfg->vocab >= 8,
                SFS_ERR_INVALID_ARG, "model_create: sizes must be positive");
    SFS_REQUIRE(cfg->head_dim == 64 || cfg->head_dim == 128, SFS_ERR_UNSUPPORTED, "head_dim %d (64 or 128 supported)", cfg->head_dim);
    SFS_REQUIRE(cfg->n_heads * cfg->head_dim == cfg->d_model, SFS_ERR_INVALID_ARG, "n_heads * head_dim != d_model");
    SFS_REQUIRE((cfg->d_model % 128) == 0, SFS_ERR_UNSUPPORTED, "d_model %d must be a multiple of 128", cfg->d_model);
    SFS_REQUIRE((cfg->d_ff % 8) == 0 && (cfg->vocab % 8) == 0, SFS_ERR_UNSUPPORTED, "d_ff and vocab must be multiples of 8");
    SFS_REQUIRE(cfg->vocab < (1 << 19), SFS_ERR_UNSUPPORTED, "vocab %d must be below 2^19", cfg->vocab);
    SFS_REQUIRE(cfg->mask_id >= 0 && cfg->mask_id < cfg->vocab, SFS_ERR_INVALID_ARG, "mask_id outside the vocabulary");
    SFS_REQUIRE(w->tok_emb && w->final_norm && w->lm_head && w->attn_norm && w->wq && w->wk && w->wv && w->wo &&
                w->mlp_norm && w->w_gate && w->w_up && w->w_down, SFS_ERR_INVALID_ARG, "model_create: NULL weight table");
    sfs_model *m = new (std::nothrow) sfs_model();
    SFS_REQUIRE(m != nullptr, SFS_ERR_OOM, "host allocation failed");
    m->cfg = *cfg;
    m->tok_emb = w->tok_emb; m->final_norm = w->final_norm; m->lm_head = w->lm_head;
    bool ok = aligned_to(w->tok_emb, 16) && aligned_to(w->final_norm, 16) && aligned_to(w->lm_head, 16);
    for (int l = 0; l < cfg->n_layers; ++l) {
        const void *ps[9] = {w->attn_norm[l], w->wq[l], w->wk[l], w->wv[l], w->wo[l], w->mlp_norm[l], w->w_gate[l], w->w_up[l], w->w_down[l]};
        for (const void *p : ps) ok = ok && p != nullptr && aligned_to(p, 16);
        m->attn_norm.push_back(ps[0]); m->wq.push_back(ps[1]); m->wk.push_back(ps[2]); m->wv.push_back(ps[3]);
        m->wo.push_back(ps[4]); m->mlp_norm.push_back(ps[5]); m->w_gate.push_back(ps[6]); m->w_up.push_back(ps[7]);
        m->w_down.push_back(ps[8]);
    }
    if (!ok) { delete m; set_error("model_create: every weight pointer must be non-NULL and 16-byte aligned"); return SFS_ERR_INVALID_ARG; }
    // whatever wrote the weights (on any stream) has finished before a forward pass on another stream reads them
    if (cudaDeviceSynchronize() != cudaSuccess) { delete m; set_error("model_create: device synchronisation failed"); return SFS_ERR_CUDA; }
    *out = m;
    return SFS_OK;
}

int32_t sfs_model_destroy(sfs_model *m)
{
    delete m;
    return SFS_OK;
}

// ---- sessions -------------------------------------------------------------------------------------------
int32_t sfs_session_destroy(sfs_session *s)
{
    if (!s) return SFS_OK;
    cudaDeviceSynchronize();
    for (void *p : s->owned) cudaFree(p);
    if (s->host_active) cudaFreeHost(s->host_active);
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
    if (device_status_word() == nullptr) { sfs_session_destroy(s); set_error("cannot allocate the device status word"); return SFS_ERR_OOM; }
    SFS_CUDA(cudaDeviceSynchronize());
    *out = s;
    return SFS_OK;
}

int32_t sfs_session_create(sfs_model *m, int32_t max_batch, int32_t max_seq, sfs_session **out)
{
    SFS_REQUIRE(m && out, SFS_ERR_INVALID_ARG, "session_create: NULL argument");
    SFS_REQUIRE(max_batch >= 1 && max_seq >= 8 && max_seq < (1 << 17) && (long long)max_batch * max_seq < (1ll << 24),
                SFS_ERR_INVALID_ARG, "max_batch %d / max_seq %d out of range", max_batch, max_seq);
    sfs_session *s = new (std::nothrow) sfs_session();
    SFS_REQUIRE(s != nullptr, SFS_ERR_OOM, "host allocation failed");
    s->model = m; s->max_batch = max_batch; s->max_seq = max_seq; s->vocab = m->cfg.vocab;
    const sfs_config &c = m->cfg;
    const size_t T = (size_t)max_batch * max_seq, d = c.d_model;
    int32_t rc = session_alloc_select(s);
    auto fail = [&](int32_t code) { sfs_session_destroy(s); return code; };
    if (rc != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->x, T * d, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->h, T * d, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->partial, (size_t)kMaxSplits * T * d, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->qk, T * 2 * d, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->vt, T * d, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->attn, T * d, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->hid, T * (size_t)c.d_ff, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->hfin, T * d, true)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->logits, T * (size_t)c.vocab, false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->rope_table, (size_t)max_seq * (c.head_dim / 2), false)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->tokens, T, true)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->mask, T, true)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->state, (size_t)max_batch, true)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->rows[0], T, true)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->rows[1], T, true)) != SFS_OK) return fail(rc);
    if ((rc = dev_alloc(s, &s->ctrl, 16, true)) != SFS_OK) return fail(rc);
    if (cudaHostAlloc(reinterpret_cast<void **>(&s->host_active), 64, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer(reinterpret_cast<void **>(&s->host_active_dev), s->host_active, 0) != cudaSuccess) {
        set_error("pinned host allocation failed");
        return fail(SFS_ERR_OOM);
    }
    *s->host_active = 0;
    if ((rc = launch_rope_table(s->rope_table, max_seq, c.head_dim, c.rope_theta, 0)) != SFS_OK) return fail(rc);
    if (device_status_word() == nullptr) { set_error("cannot allocate the device status word"); return fail(SFS_ERR_OOM); }
    if (cudaDeviceSynchronize() != cudaSuccess) { set_error("device synchronisation failed after session set-up"); return fail(SFS_ERR_CUDA); }
    *out = s;
    return SFS_OK;
}

// ---- single steps ---------------------------------------------------------------------------------------
int32_t sfs_forward(sfs_session *s, const int32_t *d_tokens, int32_t B, int32_t S,
                    const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                    void *d_logits, int32_t logits_dtype, void *stream)
{
    SFS_REQUIRE(s && s->model, SFS_ERR_INVALID_ARG, "forward: needs a session created from a model");
    SFS_REQUIRE(d_tokens && d_logits, SFS_ERR_INVALID_ARG, "forward: NULL device pointer");
    SFS_REQUIRE(B >= 1 && B <= s->max_batch && S >= 8 && S <= s->max_seq, SFS_ERR_INVALID_ARG,
                "forward: B=%d S=%d outside the session's limits (%d, %d)", B, S, s->max_batch, s->max_seq);
    SFS_REQUIRE(max_rows >= 1 && max_rows <= B * S, SFS_ERR_INVALID_ARG, "forward: max_rows %d outside [1, B*S]", max_rows);
    SFS_REQUIRE(logits_dtype == SFS_LOGITS_BF16 || logits_dtype == SFS_LOGITS_F32, SFS_ERR_INVALID_ARG, "logits_dtype %d", logits_dtype);
    SFS_REQUIRE(d_rows != nullptr || (max_rows == B * S && d_n_rows == nullptr), SFS_ERR_INVALID_ARG,
                "forward: without a row list all B*S rows are produced");
    cudaStream_t st = (cudaStream_t)stream;
    const sfs_config &c = s->model->cfg;
    int32_t rc = session_plan(s, B, S);
    if (rc != SFS_OK) return rc;
    if ((rc = run_body(s, d_tokens, B, S, nullptr, st)) != SFS_OK) return rc;
    if ((rc = timed_launch(s, SFS_K_RMSNORM, st, [&] { return launch_rmsnorm(s->x, s->pending_ptr, s->pending_n, s->pending_stride, s->model->final_norm, s->hfin, d_rows, d_n_rows, max_rows, c.d_model, c.rms_eps, st); })) != SFS_OK) return rc;
    GemmPlan lm;
    const void *lmw[1] = {s->model->lm_head};
    rc = gemm_plan_create(&lm, s->hfin, c.d_model, max_rows, c.d_model, lmw, 1, c.vocab, c.d_model, GEMM_STORE, d_logits, c.vocab,
                          logits_dtype == SFS_LOGITS_F32 ? 1 : 0, c.logit_scale, nullptr, 0, 0, nullptr);
    if (rc != SFS_OK) return rc;
    return timed_launch(s, SFS_K_GEMM_LM_HEAD, st, [&] { return gemm_launch(lm, d_n_rows, nullptr, device_status_word(), st); });
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
                            reinterpret_cast<unsigned long long *>(d_sq), d_conf, nullptr, nullptr, 0, device_status_word_if_any(),
                            (cudaStream_t)stream);
}

int32_t sfs_row_stats_bounds(const void *d_logits, int32_t vocab, int64_t ld, const int32_t *d_n_rows, int32_t max_rows,
                             uint64_t *d_lo, uint64_t *d_hi, int32_t *d_argmax, void *stream)
{
    SFS_REQUIRE(d_logits != nullptr && d_lo != nullptr && d_hi != nullptr, SFS_ERR_INVALID_ARG, "row_stats_bounds: NULL pointer");
    SFS_REQUIRE(vocab >= 1 && vocab < (1 << 19) && ld >= vocab && max_rows >= 0, SFS_ERR_INVALID_ARG, "row_stats_bounds: bad sizes");
    return launch_row_stats_bounds(d_logits, vocab, ld, d_n_rows, max_rows, reinterpret_cast<unsigned long long *>(d_lo),
                                   reinterpret_cast<unsigned long long *>(d_hi), d_argmax, device_status_word_if_any(), (cudaStream_t)stream);
}

int32_t sfs_state_init(sfs_state *d_state, int32_t B, int32_t gen_len, const sfs_params *params, void *stream)
{
    SFS_REQUIRE(d_state != nullptr && B >= 1 && gen_len >= 0, SFS_ERR_INVALID_ARG, "state_init: bad arguments");
    int32_t rc = check_params(params, gen_len);
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
    int32_t rc = check_params(params, S - P);
    if (rc != SFS_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    bool two_pass = false;
    rc = step_row_stats(s, d_logits, logits_dtype, vocab, ld, d_n_rows, max_rows, d_rows, d_mask, B, S, P, d_state, *params, &two_pass, st);
    if (rc != SFS_OK) return rc;
    SelectArgs a{};
    a.pos_lo = two_pass ? s->pos_lo : nullptr;
    a.tokens = d_tokens; a.mask = d_mask; a.B = B; a.S = S; a.P = P; a.L = S - P;
    a.state = d_state; a.params = *params;
    a.pos_sq = s->pos_sq; a.pos_arg = s->pos_arg;
    a.sel_count = d_sel_count; a.sel_pos = d_sel_pos; a.sel_tok = d_sel_tok;
    a.seq_rows = s->seq_rows; a.seq_row_count = s->seq_row_count;
    a.next_rows = d_next_rows; a.next_n_rows = d_next_n_rows; a.n_active = nullptr;
    a.ticket = s->ticket; a.trace = d_trace;
    return launch_select(a, st);
}

// ---- feature cache ----------------------------------------------------------------------------------------
int32_t sfs_cache_enable(sfs_session *s, const sfs_cache_params *p)
{
    SFS_REQUIRE(s && s->model, SFS_ERR_INVALID_ARG, "cache_enable: needs a session created from a model");
    if (p == nullptr) { s->cache_on = false; return SFS_OK; }
    SFS_REQUIRE(p->k_prompt >= 1 && p->k_response >= 1 && p->rho >= 0.0 && p->rho <= 1.0, SFS_ERR_INVALID_ARG,
                "cache_enable: k_prompt %d, k_response %d must be >= 1 and rho %g within [0, 1]", p->k_prompt, p->k_response, p->rho);
    const sfs_config &c = s->model->cfg;
    const size_t T = (size_t)s->max_batch * s->max_seq, d = c.d_model;
    if (s->Kc.empty()) {
        int32_t rc;
        s->Kc.resize(c.n_layers); s->Vtc.resize(c.n_layers); s->Ac.resize(c.n_layers); s->Fc.resize(c.n_layers);
        for (int l = 0; l < c.n_layers; ++l) {
            if ((rc = dev_alloc(s, &s->Kc[l], T * d, true)) != SFS_OK) return rc;
            if ((rc = dev_alloc(s, &s->Vtc[l], T * d, true)) != SFS_OK) return rc;
            // the two increments of a layer lie T * d floats apart, so one norm can fold both as two slabs
            if ((rc = dev_alloc(s, &s->Ac[l], 2 * T * d, true)) != SFS_OK) return rc;
            s->Fc[l] = s->Ac[l] + T * d;
        }
        if ((rc = dev_alloc(s, &s->hg, T * d, true)) != SFS_OK) return rc;
        if ((rc = dev_alloc(s, &s->vnew_t, T * d, true)) != SFS_OK) return rc;
        if ((rc = dev_alloc(s, &s->sim_partial, (size_t)kSimSlices * T * 3, true)) != SFS_OK) return rc;
        if ((rc = dev_alloc(s, &s->sel_rows, T, true)) != SFS_OK) return rc;
        SFS_CUDA(cudaDeviceSynchronize());
    }
    s->cache_params = *p;
    s->cache_on = true;
    s->cache_t = 0;
    return SFS_OK;
}

int32_t sfs_cache_reset(sfs_session *s)
{
    SFS_REQUIRE(s != nullptr, SFS_ERR_INVALID_ARG, "cache_reset: session is NULL");
    s->cache_t = 0;
    return SFS_OK;
}

int32_t sfs_cache_dump(sfs_session *s, int32_t *d_sets, float *d_sims)
{
    SFS_REQUIRE(s && s->model, SFS_ERR_INVALID_ARG, "cache_dump: needs a session created from a model");
    s->dump_sets = d_sets; s->dump_sims = d_sims;
    return SFS_OK;
}

int32_t sfs_forward_cached(sfs_session *s, const int32_t *d_tokens, int32_t B, int32_t S, int32_t P,
                           const sfs_state *d_state, const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                           void *d_logits, int32_t logits_dtype, int32_t *d_sets, float *d_sims, int32_t *n_sel, void *stream)
{
    SFS_REQUIRE(s && s->model, SFS_ERR_INVALID_ARG, "forward_cached: needs a session created from a model");
    SFS_REQUIRE(d_tokens && d_logits, SFS_ERR_INVALID_ARG, "forward_cached: NULL device pointer");
    SFS_REQUIRE(B >= 1 && B <= s->max_batch && S >= 8 && S <= s->max_seq && P >= 0 && P < S, SFS_ERR_INVALID_ARG,
                "forward_cached: B=%d S=%d P=%d outside the session's limits (%d, %d)", B, S, P, s->max_batch, s->max_seq);
    SFS_REQUIRE(max_rows >= 1 && max_rows <= B * S, SFS_ERR_INVALID_ARG, "forward_cached: max_rows %d outside [1, B*S]", max_rows);
    SFS_REQUIRE(logits_dtype == SFS_LOGITS_BF16 || logits_dtype == SFS_LOGITS_F32, SFS_ERR_INVALID_ARG, "logits_dtype %d", logits_dtype);
    SFS_REQUIRE(d_rows != nullptr || (max_rows == B * S && d_n_rows == nullptr), SFS_ERR_INVALID_ARG,
                "forward_cached: without a row list all B*S rows are produced");
    cudaStream_t st = (cudaStream_t)stream;
    const sfs_config &c = s->model->cfg;
    int32_t rc = run_body_cached(s, d_tokens, B, S, P, d_state, nullptr, d_sets, d_sims, n_sel, st);
    if (rc != SFS_OK) return rc;
    if ((rc = timed_launch(s, SFS_K_RMSNORM, st, [&] { return launch_rmsnorm(s->x, s->pending_ptr, s->pending_n, s->pending_stride, s->model->final_norm, s->hfin, d_rows, d_n_rows, max_rows, c.d_model, c.rms_eps, st); })) != SFS_OK) return rc;
    GemmPlan lm;
    const void *lmw[1] = {s->model->lm_head};
    rc = gemm_plan_create(&lm, s->hfin, c.d_model, max_rows, c.d_model, lmw, 1, c.vocab, c.d_model, GEMM_STORE, d_logits, c.vocab,
                          logits_dtype == SFS_LOGITS_F32 ? 1 : 0, c.logit_scale, nullptr, 0, 0, nullptr);
    if (rc != SFS_OK) return rc;
    return timed_launch(s, SFS_K_GEMM_LM_HEAD, st, [&] { return gemm_launch(lm, d_n_rows, nullptr, device_status_word(), st); });
}

// ---- the whole loop -------------------------------------------------------------------------------------
int32_t sfs_generate_begin(sfs_session *s, const int32_t *d_prompt, int32_t B, int32_t P, int32_t gen_len,
                           const sfs_params *params, void *stream)
{
    SFS_REQUIRE(s && s->model, SFS_ERR_INVALID_ARG, "generate: needs a session created from a model");
    SFS_REQUIRE(B >= 1 && B <= s->max_batch && P >= 0 && gen_len >= 1 && P + gen_len <= s->max_seq, SFS_ERR_INVALID_ARG,
                "generate: B=%d P=%d gen_len=%d outside the session's limits (%d, %d)", B, P, gen_len, s->max_batch, s->max_seq);
    SFS_REQUIRE(P == 0 || d_prompt != nullptr, SFS_ERR_INVALID_ARG, "generate: d_prompt is NULL");
    int32_t rc = check_params(params, gen_len);
    if (rc != SFS_OK) return rc;
    const int S = P + gen_len;
    if ((rc = session_plan(s, B, S)) != SFS_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    {   // the LM head sees at most B * gen_len rows: plan it for that many, not for all B * S tokens
        const sfs_config &c = s->model->cfg;
        const void *lm[1] = {s->model->lm_head};
        rc = gemm_plan_create(&s->lm_plan, s->hfin, c.d_model, B * gen_len, c.d_model, lm, 1, c.vocab, c.d_model, GEMM_STORE,
                              s->logits, c.vocab, 0, c.logit_scale, nullptr, 0, 0, nullptr);
        if (rc != SFS_OK) return rc;
        // Long bf16 rows: the LM head takes the first pass of the row statistics in its epilogue (one record per row,
        // column tile and epilogue-warp parity), so the selection step never streams the logits back from memory.
        // (tiles of at least 128 columns: then both epilogue-warp parities own columns of every 256-row block)
        if (row_stats_two_pass_applies(s->logits, SFS_LOGITS_BF16, c.vocab, c.vocab) && s->lm_plan.args.splits == 1 && s->lm_plan.args.bn >= 128) {
            const int parts = 2 * s->lm_plan.args.n_col_tiles;
            const size_t need = (size_t)B * gen_len * parts;
            if (s->lm_stats_cap < need) {
                SFS_CUDA(cudaStreamSynchronize(st));
                if (s->lm_stats) {
                    for (auto it = s->owned.begin(); it != s->owned.end(); ++it) if (*it == (void *)s->lm_stats) { s->owned.erase(it); break; }
                    cudaFree(s->lm_stats); s->lm_stats = nullptr; s->lm_stats_cap = 0;
                }
                if ((rc = dev_alloc(s, &s->lm_stats, need, true)) != SFS_OK) return rc;
                s->lm_stats_cap = need;
            }
            s->lm_plan.args.stats = s->lm_stats; s->lm_plan.args.stats_ld = parts;
        }
    }
    generate_init_kernel<<<64, 256, 0, st>>>(d_prompt, s->tokens, s->mask, s->rows[0], s->ctrl, s->host_active_dev, s->pos_sq,
                                             B, P, gen_len, s->model->cfg.mask_id);
    SFS_LAUNCH_CHECK();
    if ((rc = launch_state_init(s->state, B, gen_len, *params, nullptr, st)) != SFS_OK) return rc;
    s->gen_B = B; s->gen_P = P; s->gen_L = gen_len; s->gen_cur = 0; s->gen_steps = 0;
    s->gen_max_steps = params->max_steps > 0 ? params->max_steps : gen_len;
    s->gen_params = *params;
    s->cache_t = 0;                                          // a new generation starts with a full refresh
    s->generating = true;
    s->host_active[0] = B; s->host_active[1] = 0;
    return SFS_OK;
}

int32_t sfs_generate_steps(sfs_session *s, int32_t n_steps, int32_t *d_trace, int32_t max_trace_steps,
                           void *d_logits_dump, int32_t *d_rows_dump, int32_t *d_n_rows_dump, void *stream)
{
    SFS_REQUIRE(s && s->model && s->generating, SFS_ERR_INVALID_ARG, "generate_steps: call sfs_generate_begin first");
    SFS_REQUIRE(n_steps >= 0, SFS_ERR_INVALID_ARG, "generate_steps: n_steps %d", n_steps);
    SFS_REQUIRE(d_logits_dump == nullptr || n_steps == 1, SFS_ERR_INVALID_ARG, "generate_steps: a logits dump takes exactly one step");
    cudaStream_t st = (cudaStream_t)stream;
    const sfs_config &c = s->model->cfg;
    const int B = s->gen_B, P = s->gen_P, L = s->gen_L, S = P + L;
    int32_t *err = device_status_word();
    int32_t rc;
    for (int i = 0; i < n_steps; ++i) {
        if (s->gen_steps >= s->gen_max_steps) break;                 // every sequence is done by construction
        const int cur = s->gen_cur, nxt = cur ^ 1;
        const int32_t *d_active = s->ctrl + 2;
        const int32_t *rows = s->rows[cur], *n_rows = s->ctrl + cur;
        if (s->cache_on) rc = run_body_cached(s, s->tokens, B, S, P, s->state, d_active, s->dump_sets, s->dump_sims, nullptr, st);
        else rc = run_body(s, s->tokens, B, S, d_active, st);
        if (rc != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_RMSNORM, st, [&] { return launch_rmsnorm(s->x, s->pending_ptr, s->pending_n, s->pending_stride, s->model->final_norm, s->hfin, rows, n_rows, B * L, c.d_model, c.rms_eps, st); })) != SFS_OK) return rc;
        if ((rc = timed_launch(s, SFS_K_GEMM_LM_HEAD, st, [&] { return gemm_launch(s->lm_plan, n_rows, d_active, err, st); })) != SFS_OK) return rc;
        if (d_logits_dump) {
            SFS_CUDA(cudaMemcpyAsync(d_logits_dump, s->logits, (size_t)B * L * c.vocab * 2, cudaMemcpyDeviceToDevice, st));
            if (d_rows_dump) SFS_CUDA(cudaMemcpyAsync(d_rows_dump, rows, (size_t)B * L * 4, cudaMemcpyDeviceToDevice, st));
            if (d_n_rows_dump) SFS_CUDA(cudaMemcpyAsync(d_n_rows_dump, n_rows, 4, cudaMemcpyDeviceToDevice, st));
        }
        bool two_pass = false;
        if ((rc = timed_launch(s, SFS_K_ROW_STATS, st, [&] {
                 return step_row_stats(s, s->logits, SFS_LOGITS_BF16, c.vocab, c.vocab, n_rows, B * L, rows, s->mask, B, S, P, s->state,
                                       s->gen_params, &two_pass, st, s->lm_plan.args.stats, s->lm_plan.args.stats_ld); })) != SFS_OK) return rc;
        SelectArgs a{};
        a.pos_lo = two_pass ? s->pos_lo : nullptr;
        a.tokens = s->tokens; a.mask = s->mask; a.B = B; a.S = S; a.P = P; a.L = L;
        a.state = s->state; a.params = s->gen_params;
        a.pos_sq = s->pos_sq; a.pos_arg = s->pos_arg;
        a.seq_rows = s->seq_rows; a.seq_row_count = s->seq_row_count;
        a.next_rows = s->rows[nxt]; a.next_n_rows = s->ctrl + nxt; a.n_active = s->ctrl + 2;
        a.ticket = s->ticket;
        a.trace = (d_trace && s->gen_steps < max_trace_steps) ? d_trace + (size_t)s->gen_steps * B * SFS_TRACE_INTS : nullptr;
        if ((rc = timed_launch(s, SFS_K_SELECT, st, [&] { return launch_select(a, st); })) != SFS_OK) return rc;
        SFS_CUDA(launch_pdl(mirror_active_kernel, dim3((unsigned)(1)), dim3((unsigned)(1)), (size_t)(0), st, s->ctrl + 2, s->host_active_dev, s->gen_steps + 1));
        s->launches++;
        s->gen_cur = nxt;
        s->gen_steps++;
    }
    return SFS_OK;
}

int32_t sfs_generate_end(sfs_session *s, int32_t *d_out_tokens, sfs_state *d_state_out, int32_t *n_active,
                         int32_t *steps_enqueued, void *stream)
{
    SFS_REQUIRE(s && s->model && s->generating, SFS_ERR_INVALID_ARG, "generate_end: call sfs_generate_begin first");
    cudaStream_t st = (cudaStream_t)stream;
    const int B = s->gen_B, S = s->gen_P + s->gen_L;
    if (d_out_tokens) SFS_CUDA(cudaMemcpyAsync(d_out_tokens, s->tokens, (size_t)B * S * 4, cudaMemcpyDeviceToDevice, st));
    if (d_state_out) SFS_CUDA(cudaMemcpyAsync(d_state_out, s->state, (size_t)B * sizeof(sfs_state), cudaMemcpyDeviceToDevice, st));
    std::vector<sfs_state> hs((size_t)B);
    SFS_CUDA(cudaMemcpyAsync(hs.data(), s->state, (size_t)B * sizeof(sfs_state), cudaMemcpyDeviceToHost, st));
    int32_t dev = sfs_check_device_status(stream);                 // synchronises
    if (steps_enqueued) *steps_enqueued = s->gen_steps;
    int act = 0, bad = SFS_OK;
    for (const sfs_state &h : hs) {
        if (!h.done && h.status == SFS_OK) act++;
        if (h.status != SFS_OK && bad == SFS_OK) bad = h.status;
    }
    if (n_active) *n_active = act;
    if (dev != SFS_OK) return dev;
    if (bad != SFS_OK) { set_error("a sequence stopped with device status %d (%s)", bad, sfs_status_string(bad)); return bad; }
    return SFS_OK;
}

int32_t sfs_generate(sfs_session *s, const int32_t *d_prompt, int32_t B, int32_t P, int32_t gen_len,
                     const sfs_params *params, int32_t *d_out_tokens, sfs_state *d_state_out,
                     int32_t *d_trace, int32_t max_trace_steps, void *stream)
{
    // the pinned mirror must not receive values of an earlier generation whose kernels are still in flight
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) { set_error("generate: the stream is in an error state"); return SFS_ERR_CUDA; }
    int32_t rc = sfs_generate_begin(s, d_prompt, B, P, gen_len, params, stream);
    if (rc != SFS_OK) return rc;
    // Steps are enqueued at most kAhead ahead of the device (enough to keep it busy: a step's launches are enqueued in a
    // fraction of the time the step runs); the pinned mirror of the active-sequence count stops the enqueueing when the
    // last sequence finishes, so at most kAhead surplus steps are ever enqueued, and their kernels exit at once.
    constexpr int kAhead = 2;
    volatile int32_t *mirror = reinterpret_cast<volatile int32_t *>(s->host_active);
    while (s->gen_steps < s->gen_max_steps) {
        long long spins = 0;
        while (mirror[0] != 0 && s->gen_steps - mirror[1] >= kAhead) {
            if (++spins > (1ll << 34) || ((spins & 0xFFFFF) == 0 && cudaStreamQuery((cudaStream_t)stream) == cudaSuccess)) break;   // the stream drained or stalled
        }
        if (mirror[0] == 0) break;
        if ((rc = sfs_generate_steps(s, 1, d_trace, max_trace_steps, nullptr, nullptr, nullptr, stream)) != SFS_OK) return rc;
    }
    int32_t act = 0;
    rc = sfs_generate_end(s, d_out_tokens, d_state_out, &act, nullptr, stream);
    if (rc != SFS_OK) return rc;
    if (act != 0) { set_error("%d sequence(s) unfinished after %d steps", act, s->gen_steps); return SFS_ERR_STEP_LIMIT; }
    return SFS_OK;
}

// ---- instrumentation ------------------------------------------------------------------------------------
int32_t sfs_profile(sfs_session *s, int32_t enable, float *ms_per_class, int64_t *launches_per_class, int64_t *total_launches)
{
    SFS_REQUIRE(s != nullptr, SFS_ERR_INVALID_ARG, "profile: session is NULL");
    if (ms_per_class || launches_per_class) {
        SFS_CUDA(cudaDeviceSynchronize());
        for (int i = 0; i < SFS_K_CLASSES; ++i) { if (ms_per_class) ms_per_class[i] = 0.f; if (launches_per_class) launches_per_class[i] = 0; }
        for (auto &t : s->timed) {
            float ms = 0.f;
            SFS_CUDA(cudaEventElapsedTime(&ms, t.e0, t.e1));
            if (ms_per_class) ms_per_class[t.cls] += ms;
            if (launches_per_class) launches_per_class[t.cls] += 1;
        }
    }
    if (total_launches) *total_launches = s->launches;
    for (auto &t : s->timed) { cudaEventDestroy(t.e0); cudaEventDestroy(t.e1); }
    s->timed.clear();
    s->profile = enable != 0;
    return SFS_OK;
}

// ---- building blocks ------------------------------------------------------------------------------------
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
    int32_t rc = gemm_plan_create(&plan, d_A, lda, M, K, bs, 1, N, ldb, GEMM_STORE, d_C, ldc, out_dtype, scale, nullptr, 0, 0, nullptr);
    if (rc != SFS_OK) return rc;
    return gemm_launch(plan, nullptr, nullptr, err, (cudaStream_t)stream);
}

int32_t sfs_attention(const void *d_qk, const void *d_vt, void *d_out, int32_t B, int32_t S,
                      int32_t n_heads, int32_t head_dim, void *stream)
{
    SFS_REQUIRE(d_qk && d_vt && d_out, SFS_ERR_INVALID_ARG, "attention: NULL pointer");
    SFS_REQUIRE(B >= 1 && S >= 8 && n_heads >= 1, SFS_ERR_INVALID_ARG, "attention: bad sizes");
    int32_t *err = device_status_word();
    SFS_REQUIRE(err != nullptr, SFS_ERR_OOM, "cannot allocate the device status word");
    const int d = n_heads * head_dim;
    AttnPlan plan;
    int32_t rc = attn_plan_create(&plan, d_qk, 2 * d, d_vt, (int64_t)B * S, d_out, d, B, S, n_heads, head_dim);
    if (rc != SFS_OK) return rc;
    return attn_launch(plan, nullptr, err, (cudaStream_t)stream);
}

}  // extern "C"
