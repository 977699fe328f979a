// The C ABI of libmetasd: context life cycle, argument validation, state blobs, and the dispatch
// of one verify round to the streaming or the fused kernels.  Declarations: include/metasd.h.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "metasd_internal.h"

using namespace metasd;

struct metasd_ctx {
    metasd_config cfg;
    BanditState st;
    RowStats *stats;     // scratch of the streaming path: [max_batch, max_draft + 1]
    uint32_t *status;    // device status word
    const void **table_clean;   // the checked copy of the caller's drafter table (16 entries)
    const int32_t *draft_len;   // the caller's per-sequence draft lengths (device), or nullptr
    uint64_t launches;
    // staging for metasd_verify_host
    void *stage_target, *stage_draft;
    int32_t *stage_tokens, *stage_acc, *stage_tok;
    float *stage_reward;
    bool fused_ready;
    FusedPlan plan;
    int keep_permille;   // share of every row that the streaming kernel asks L2 to keep between its sweeps
    int k1_stages;       // depth of the row-statistics kernel's cp.async pipeline (0 or 1: plain loads)
    // split streaming path
    int grp_size, grp_ctas;
    GroupRecord *grp_rec;
    double *grp_min;
    uint32_t *grp_count;
};

namespace {

struct BlobHeader {
    uint32_t magic, version;
    int32_t max_batch, n_drafters, window, bandit;
};
constexpr uint32_t BLOB_MAGIC = 0x4D534453u;  // "MSDS"

size_t logit_size(int dtype) { return dtype == METASD_BF16 ? 2 : 4; }

int cuda_fail(cudaError_t e) { return e == cudaErrorMemoryAllocation ? METASD_ERR_NO_MEMORY : METASD_ERR_CUDA; }

#define CK(call)                                   \
    do {                                           \
        cudaError_t e_ = (call);                   \
        if (e_ != cudaSuccess) return cuda_fail(e_); \
    } while (0)

int validate_config(const metasd_config *c)
{
    if (!c) return METASD_ERR_INVALID_ARGUMENT;
    if (c->max_batch < 1 || c->max_batch > 65535) return METASD_ERR_INVALID_ARGUMENT;
    if (c->n_drafters < 1 || c->n_drafters > 16) return METASD_ERR_INVALID_ARGUMENT;
    if (c->max_draft < 1 || c->max_draft > 16) return METASD_ERR_INVALID_ARGUMENT;
    if (c->vocab < 1) return METASD_ERR_INVALID_ARGUMENT;
    if (c->logit_dtype != METASD_BF16 && c->logit_dtype != METASD_FP32) return METASD_ERR_UNSUPPORTED;
    if (c->bandit < METASD_UCB || c->bandit > METASD_PETC) return METASD_ERR_UNSUPPORTED;
    if (c->reward != METASD_REWARD_BD && c->reward != METASD_REWARD_BE) return METASD_ERR_UNSUPPORTED;
    if (c->path < METASD_PATH_AUTO || c->path > METASD_PATH_FUSED) return METASD_ERR_UNSUPPORTED;
    if (c->window < 1 || c->window > (1 << 20)) return METASD_ERR_INVALID_ARGUMENT;
    if (c->device < 0) return METASD_ERR_INVALID_ARGUMENT;
    if (!(c->beta >= 0.0) || !isfinite(c->beta)) return METASD_ERR_INVALID_ARGUMENT;
    if (!(c->gamma > 0.0) || !(c->gamma <= 1.0)) return METASD_ERR_INVALID_ARGUMENT;
    if (!(c->reward_temperature > 0.0) || !isfinite(c->reward_temperature)) return METASD_ERR_INVALID_ARGUMENT;
    if ((uint64_t)c->vocab * (uint64_t)(c->max_draft + 1) >= (1ull << 31)) return METASD_ERR_UNSUPPORTED;
    return METASD_OK;
}

void free_all(metasd_ctx *c)
{
    cudaFree(c->st.t); cudaFree(c->st.arm); cudaFree(c->st.stat_a); cudaFree(c->st.stat_b);
    cudaFree(c->st.win_arm); cudaFree(c->st.win_reward); cudaFree(c->stats); cudaFree(c->status);
    cudaFree(c->stage_target); cudaFree(c->stage_draft); cudaFree(c->stage_tokens);
    cudaFree(c->stage_acc); cudaFree(c->stage_tok); cudaFree(c->stage_reward);
    cudaFree(c->grp_rec); cudaFree(c->grp_min); cudaFree(c->grp_count);
}

}  // namespace

extern "C" {

void metasd_default_config(metasd_config *cfg)
{
    if (!cfg) return;
    memset(cfg, 0, sizeof *cfg);
    cfg->max_batch = 1;
    cfg->n_drafters = 1;
    cfg->max_draft = 5;
    cfg->vocab = 32000;
    cfg->logit_dtype = METASD_BF16;
    cfg->bandit = METASD_UCB;
    cfg->reward = METASD_REWARD_BD;
    cfg->window = 50;
    cfg->device = 0;
    cfg->path = METASD_PATH_AUTO;
    cfg->sequence_base = 0;
    cfg->host_staging = 0;
    cfg->beta = 0.01;
    cfg->gamma = 0.975;
    cfg->reward_temperature = 1.0;
}

int metasd_init(metasd_ctx **out, const metasd_config *cfg)
{
    if (!out) return METASD_ERR_INVALID_ARGUMENT;
    *out = nullptr;
    int rc = validate_config(cfg);
    if (rc != METASD_OK) return rc;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device >= n_dev) return METASD_ERR_CUDA;
    CK(cudaSetDevice(cfg->device));
    if (cfg->path == METASD_PATH_FUSED && !fused_supported(cfg->logit_dtype, cfg->vocab, cfg->max_draft))
        return METASD_ERR_UNSUPPORTED;

    metasd_ctx *c = new (std::nothrow) metasd_ctx();
    if (!c) return METASD_ERR_NO_MEMORY;
    memset(c, 0, sizeof *c);
    c->cfg = *cfg;
    {   // the best measured values on B200 for 128k-152k vocabularies (METASD_KEEP_PERMILLE overrides, for tuning)
        const char *kp = getenv("METASD_KEEP_PERMILLE");
        const int v = kp && *kp ? atoi(kp) : (cfg->logit_dtype == METASD_BF16 ? 750 : 900);
        c->keep_permille = v < 0 ? 0 : (v > 1000 ? 1000 : v);
    }
    {
        // 4: rows staged through shared memory; 0 (METASD_K1_STAGES=0, for comparison): plain loads
        const char *ks = getenv("METASD_K1_STAGES");
        c->k1_stages = ks && *ks ? atoi(ks) : 4;
    }
    const size_t B = cfg->max_batch, K = cfg->n_drafters, tau = cfg->window, kp1 = cfg->max_draft + 1;
    cudaError_t e = cudaSuccess;
    auto alloc = [&](void **p, size_t bytes) {
        if (e == cudaSuccess) e = cudaMalloc(p, bytes);
    };
    alloc((void **)&c->st.t, B * sizeof(int32_t));
    alloc((void **)&c->st.arm, B * sizeof(int32_t));
    alloc((void **)&c->st.stat_a, B * K * sizeof(double));
    alloc((void **)&c->st.stat_b, B * K * sizeof(double));
    alloc((void **)&c->st.win_arm, B * tau * sizeof(int32_t));
    alloc((void **)&c->st.win_reward, B * tau * sizeof(double));
    alloc((void **)&c->stats, B * kp1 * sizeof(RowStats));
    alloc((void **)&c->status, sizeof(uint32_t));
    alloc((void **)&c->table_clean, 16 * sizeof(void *));
    if (cfg->host_staging) {
        const size_t row = (size_t)cfg->vocab * logit_size(cfg->logit_dtype);
        alloc(&c->stage_target, B * kp1 * row);
        alloc(&c->stage_draft, B * (kp1 - 1) * row);
        alloc((void **)&c->stage_tokens, B * (kp1 - 1) * sizeof(int32_t));
        alloc((void **)&c->stage_acc, B * sizeof(int32_t));
        alloc((void **)&c->stage_tok, B * sizeof(int32_t));
        alloc((void **)&c->stage_reward, B * sizeof(float));
    }
    if (e == cudaSuccess) {
        e = split_prepare(cfg->device, cfg->logit_dtype, cfg->vocab, &c->grp_ctas, &c->grp_size);
        if (e == cudaSuccess && c->grp_size > 1) {
            alloc((void **)&c->grp_rec, B * kp1 * c->grp_size * sizeof(GroupRecord));
            alloc((void **)&c->grp_min, B * kp1 * c->grp_size * sizeof(double));
            alloc((void **)&c->grp_count, B * kp1 * sizeof(uint32_t));
        }
    }
    if (e == cudaSuccess) e = cudaMemset(c->status, 0, sizeof(uint32_t));
    if (e == cudaSuccess) e = launch_reset(c->st, cfg->max_batch, cfg->n_drafters, cfg->window, cfg->bandit, cfg->gamma,
                                            cfg->sequence_base, nullptr, cfg->max_batch, 0);
    if (e == cudaSuccess && cfg->path == METASD_PATH_FUSED &&
        fused_supported(cfg->logit_dtype, cfg->vocab, cfg->max_draft)) {
        e = fused_prepare(cfg->device, cfg->logit_dtype, cfg->vocab, cfg->max_batch, &c->plan);
        c->fused_ready = (e == cudaSuccess);
        if (cfg->path == METASD_PATH_AUTO && e != cudaSuccess) { (void)cudaGetLastError(); e = cudaSuccess; }
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        free_all(c);
        delete c;
        return cuda_fail(e);
    }
    *out = c;
    return METASD_OK;
}

void metasd_destroy(metasd_ctx *ctx)
{
    if (!ctx) return;
    cudaSetDevice(ctx->cfg.device);
    free_all(ctx);
    delete ctx;
}

int metasd_reset(metasd_ctx *ctx, const int32_t *seq_ids, int32_t n, void *stream)
{
    if (!ctx || n < 0) return METASD_ERR_INVALID_ARGUMENT;
    if (!seq_ids) n = ctx->cfg.max_batch;
    CK(launch_reset(ctx->st, ctx->cfg.max_batch, ctx->cfg.n_drafters, ctx->cfg.window, ctx->cfg.bandit, ctx->cfg.gamma,
                    ctx->cfg.sequence_base, seq_ids, n, (cudaStream_t)stream));
    ctx->launches += n > 0;
    return METASD_OK;
}

int metasd_select(metasd_ctx *ctx, int32_t batch, int32_t *arm_out, void *stream)
{
    if (!ctx || !arm_out || batch < 1 || batch > ctx->cfg.max_batch) return METASD_ERR_INVALID_ARGUMENT;
    CK(launch_select(ctx->st, batch, arm_out, (cudaStream_t)stream));
    ctx->launches += 1;
    return METASD_OK;
}

int metasd_resolved_path(const metasd_ctx *ctx, int32_t k)
{
    if (!ctx) return METASD_ERR_INVALID_ARGUMENT;
    // AUTO takes the streaming kernels: on B200 they are the faster path at every measured shape (the fused
    // cluster kernel reads each logit once but is bound by its exchange and instruction overheads).
    if (ctx->cfg.path != METASD_PATH_FUSED) return METASD_PATH_STREAMING;
    if (ctx->fused_ready && fused_supported(ctx->cfg.logit_dtype, ctx->cfg.vocab, k)) return METASD_PATH_FUSED;
    return METASD_PATH_STREAMING;
}

int metasd_verify(metasd_ctx *ctx, int32_t batch, int32_t k, const void *target_logits, const void *draft_logits,
                  const void *const *drafter_ptrs, const int32_t *draft_tokens, int64_t token_arm_stride,
                  float temperature, uint64_t seed, int32_t *accepted_len, int32_t *next_token, float *reward,
                  metasd_diag *diag, void *stream)
{
    if (!ctx) return METASD_ERR_INVALID_ARGUMENT;
    const metasd_config &cfg = ctx->cfg;
    if (batch < 1 || batch > cfg.max_batch || k < 1 || k > cfg.max_draft) return METASD_ERR_INVALID_ARGUMENT;
    if (!target_logits || !draft_tokens || !accepted_len || !next_token || !reward) return METASD_ERR_INVALID_ARGUMENT;
    if ((draft_logits == nullptr) == (drafter_ptrs == nullptr)) return METASD_ERR_INVALID_ARGUMENT;
    if (!(temperature >= 0.f) || !isfinite(temperature) || token_arm_stride < 0) return METASD_ERR_INVALID_ARGUMENT;

    VerifyParams p;
    memset(&p, 0, sizeof p);
    p.batch = batch; p.k = k; p.V = cfg.vocab;
    p.K = cfg.n_drafters; p.bandit = cfg.bandit; p.reward_kind = cfg.reward; p.tau = cfg.window;
    p.sequence_base = cfg.sequence_base;
    p.target = target_logits; p.draft = draft_logits; p.drafter_ptrs = drafter_ptrs;
    p.tokens = draft_tokens; p.token_arm_stride = token_arm_stride;
    p.draft_len = ctx->draft_len;
    p.greedy = temperature == 0.f;
    const double T = p.greedy ? cfg.reward_temperature : (double)temperature;
    p.c = (float)(1.4426950408889634 / T);
    p.seed = seed; p.beta = cfg.beta; p.gamma = cfg.gamma;
    p.accepted_len = accepted_len; p.next_token = next_token; p.reward = reward; p.diag = diag;
    p.st = ctx->st; p.stats = ctx->stats; p.status = ctx->status;
    p.keep_permille = ctx->keep_permille;
    {
        const long long nvec = (long long)cfg.vocab * (long long)logit_size(cfg.logit_dtype) / 16;
        p.keep_from_vec = (int32_t)(nvec - nvec * ctx->keep_permille / 1000);
    }
    p.k1_stages = ctx->k1_stages;
    p.grp_size = ctx->grp_size; p.grp_ctas = ctx->grp_ctas;
    p.grp_rec = ctx->grp_rec; p.grp_min = ctx->grp_min; p.grp_count = ctx->grp_count;
    const size_t row_bytes = (size_t)cfg.vocab * logit_size(cfg.logit_dtype);
    // with a pointer table the per-drafter bases are not visible here: the caller's contract is that
    // they are aligned like the target
    p.vector_ok = row_bytes % 16 == 0 && ((uintptr_t)target_logits % 16) == 0 &&
                  (draft_logits ? ((uintptr_t)draft_logits % 16) == 0 : 1);

    cudaError_t e;
    if (drafter_ptrs && metasd_resolved_path(ctx, k) != METASD_PATH_FUSED) {   // the fused kernel checks for itself
        const uint32_t mask = p.vector_ok ? 15u : (uint32_t)(logit_size(cfg.logit_dtype) - 1);
        e = launch_sanitize_table(drafter_ptrs, cfg.n_drafters, target_logits, mask, ctx->table_clean, ctx->status,
                                  (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e);
        ctx->launches += 1;
        p.drafter_ptrs = ctx->table_clean;
    }
    if (ctx->draft_len && cfg.path == METASD_PATH_FUSED) return METASD_ERR_UNSUPPORTED;
    if (metasd_resolved_path(ctx, k) == METASD_PATH_FUSED && p.vector_ok)
        e = launch_fused(p, cfg.logit_dtype, ctx->plan, (cudaStream_t)stream, &ctx->launches);
    else if (cfg.path == METASD_PATH_FUSED)
        return METASD_ERR_UNSUPPORTED;
    else
        e = launch_streaming(p, cfg.logit_dtype, (cudaStream_t)stream, &ctx->launches);
    return e == cudaSuccess ? METASD_OK : cuda_fail(e);
}

int metasd_set_draft_lengths(metasd_ctx *ctx, const int32_t *draft_len)
{
    if (!ctx) return METASD_ERR_INVALID_ARGUMENT;
    ctx->draft_len = draft_len;
    return METASD_OK;
}

int metasd_verify_host(metasd_ctx *ctx, int32_t batch, int32_t k, const void *host_target_logits,
                       const void *host_draft_logits, const int32_t *host_draft_tokens, float temperature,
                       uint64_t seed, int32_t *host_accepted_len, int32_t *host_next_token, float *host_reward,
                       int32_t *host_arm_next, void *stream)
{
    if (!ctx || !ctx->stage_target) return METASD_ERR_INVALID_ARGUMENT;
    const metasd_config &cfg = ctx->cfg;
    if (batch < 1 || batch > cfg.max_batch || k < 1 || k > cfg.max_draft) return METASD_ERR_INVALID_ARGUMENT;
    if (!host_target_logits || !host_draft_logits || !host_draft_tokens || !host_accepted_len || !host_next_token ||
        !host_reward)
        return METASD_ERR_INVALID_ARGUMENT;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t row = (size_t)cfg.vocab * logit_size(cfg.logit_dtype);
    CK(cudaMemcpyAsync(ctx->stage_target, host_target_logits, (size_t)batch * (k + 1) * row, cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(ctx->stage_draft, host_draft_logits, (size_t)batch * k * row, cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(ctx->stage_tokens, host_draft_tokens, (size_t)batch * k * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    int rc = metasd_verify(ctx, batch, k, ctx->stage_target, ctx->stage_draft, nullptr, ctx->stage_tokens, 0, temperature,
                           seed, ctx->stage_acc, ctx->stage_tok, ctx->stage_reward, nullptr, stream);
    if (rc != METASD_OK) return rc;
    CK(cudaMemcpyAsync(host_accepted_len, ctx->stage_acc, (size_t)batch * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(host_next_token, ctx->stage_tok, (size_t)batch * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(host_reward, ctx->stage_reward, (size_t)batch * sizeof(float), cudaMemcpyDeviceToHost, s));
    if (host_arm_next)
        CK(cudaMemcpyAsync(host_arm_next, ctx->st.arm, (size_t)batch * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    return METASD_OK;
}

size_t metasd_state_bytes(const metasd_ctx *ctx)
{
    if (!ctx) return 0;
    const size_t B = ctx->cfg.max_batch, K = ctx->cfg.n_drafters, tau = ctx->cfg.window;
    return sizeof(BlobHeader) + 2 * B * sizeof(int32_t) + 2 * B * K * sizeof(double) + B * tau * sizeof(int32_t) +
           B * tau * sizeof(double);
}

int metasd_state_export(metasd_ctx *ctx, void *host_buf, size_t bytes, void *stream)
{
    if (!ctx || !host_buf || bytes < metasd_state_bytes(ctx)) return METASD_ERR_INVALID_ARGUMENT;
    const size_t B = ctx->cfg.max_batch, K = ctx->cfg.n_drafters, tau = ctx->cfg.window;
    cudaStream_t s = (cudaStream_t)stream;
    BlobHeader h = {BLOB_MAGIC, 1u, ctx->cfg.max_batch, ctx->cfg.n_drafters, ctx->cfg.window, ctx->cfg.bandit};
    char *w = (char *)host_buf;
    memcpy(w, &h, sizeof h);
    w += sizeof h;
    auto pull = [&](const void *src, size_t n) -> cudaError_t {
        cudaError_t e = cudaMemcpyAsync(w, src, n, cudaMemcpyDeviceToHost, s);
        w += n;
        return e;
    };
    CK(pull(ctx->st.t, B * sizeof(int32_t)));
    CK(pull(ctx->st.arm, B * sizeof(int32_t)));
    CK(pull(ctx->st.stat_a, B * K * sizeof(double)));
    CK(pull(ctx->st.stat_b, B * K * sizeof(double)));
    CK(pull(ctx->st.win_arm, B * tau * sizeof(int32_t)));
    CK(pull(ctx->st.win_reward, B * tau * sizeof(double)));
    CK(cudaStreamSynchronize(s));
    return METASD_OK;
}

int metasd_state_import(metasd_ctx *ctx, const void *host_buf, size_t bytes, void *stream)
{
    if (!ctx || !host_buf || bytes < metasd_state_bytes(ctx)) return METASD_ERR_INVALID_ARGUMENT;
    BlobHeader h;
    memcpy(&h, host_buf, sizeof h);
    if (h.magic != BLOB_MAGIC || h.version != 1u || h.max_batch != ctx->cfg.max_batch ||
        h.n_drafters != ctx->cfg.n_drafters || h.window != ctx->cfg.window || h.bandit != ctx->cfg.bandit)
        return METASD_ERR_BAD_STATE_BLOB;
    const size_t B = ctx->cfg.max_batch, K = ctx->cfg.n_drafters, tau = ctx->cfg.window;
    cudaStream_t s = (cudaStream_t)stream;
    const char *r = (const char *)host_buf + sizeof h;
    auto push = [&](void *dst, size_t n) -> cudaError_t {
        cudaError_t e = cudaMemcpyAsync(dst, r, n, cudaMemcpyHostToDevice, s);
        r += n;
        return e;
    };
    CK(push(ctx->st.t, B * sizeof(int32_t)));
    CK(push(ctx->st.arm, B * sizeof(int32_t)));
    CK(push(ctx->st.stat_a, B * K * sizeof(double)));
    CK(push(ctx->st.stat_b, B * K * sizeof(double)));
    CK(push(ctx->st.win_arm, B * tau * sizeof(int32_t)));
    CK(push(ctx->st.win_reward, B * tau * sizeof(double)));
    CK(cudaStreamSynchronize(s));
    return METASD_OK;
}

int metasd_last_status(metasd_ctx *ctx, uint32_t *host_flags, void *stream)
{
    if (!ctx || !host_flags) return METASD_ERR_INVALID_ARGUMENT;
    cudaStream_t s = (cudaStream_t)stream;
    CK(cudaMemcpyAsync(host_flags, ctx->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    CK(cudaMemsetAsync(ctx->status, 0, sizeof(uint32_t), s));
    CK(cudaStreamSynchronize(s));
    return METASD_OK;
}

uint64_t metasd_kernel_launches(const metasd_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *metasd_strerror(int code)
{
    switch (code) {
    case METASD_OK: return "ok";
    case METASD_ERR_INVALID_ARGUMENT: return "invalid argument";
    case METASD_ERR_UNSUPPORTED: return "unsupported configuration";
    case METASD_ERR_CUDA: return "CUDA error (no device, or a runtime call failed)";
    case METASD_ERR_NO_MEMORY: return "out of memory";
    case METASD_ERR_BAD_STATE_BLOB: return "state blob does not match this context";
    default: return "unknown error";
    }
}

}  // extern "C"
