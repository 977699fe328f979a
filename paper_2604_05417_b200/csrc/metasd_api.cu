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
    const int32_t *draft_len;   // the caller's per-sequence draft lengths (device), or nullptr
    uint64_t launches;
    // staging for metasd_verify_host
    void *stage_target, *stage_draft;
    int32_t *stage_tokens, *stage_acc, *stage_tok;
    float *stage_reward;
    bool fused_ready;
    FusedPlan plan;
    RowGeometry geo;     // shape of the row-statistics launch
    int keep_permille;   // share of every row that the row-statistics kernel asks L2 to keep between its sweeps
};

namespace {

struct BlobHeader {
    uint32_t magic, version;
    int32_t max_batch, n_drafters, window, bandit;
};
constexpr uint32_t BLOB_MAGIC = 0x4D534453u;  // "MSDS"

size_t logit_size(int dtype) { return dtype == METASD_BF16 ? 2 : 4; }

size_t blob_bytes(const metasd_config &c)
{
    const size_t B = c.max_batch, K = c.n_drafters, tau = c.window;
    return sizeof(BlobHeader) + 2 * B * sizeof(int32_t) + 2 * B * K * sizeof(double) + B * tau * sizeof(int32_t) +
           B * tau * sizeof(double);
}

// Makes the context's device current for the lifetime of the object and restores the caller's on the way out.
struct DeviceScope {
    int previous = -1;
    cudaError_t error = cudaSuccess;
    explicit DeviceScope(int device)
    {
        error = cudaGetDevice(&previous);
        if (error == cudaSuccess && previous != device) error = cudaSetDevice(device);
        else if (error == cudaSuccess) previous = -1;   // nothing to restore
    }
    ~DeviceScope()
    {
        if (previous >= 0) cudaSetDevice(previous);
    }
};
#define ON_DEVICE_OF(ctx)                                   \
    DeviceScope scope_((ctx)->cfg.device);                  \
    if (scope_.error != cudaSuccess) return cuda_fail(scope_.error)

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
    if (c->row_kernel < METASD_ROWS_AUTO || c->row_kernel > METASD_ROWS_BULK) return METASD_ERR_UNSUPPORTED;
    if (c->row_threads < 0 || c->row_stages < 0 || c->keep_permille > 1000) return METASD_ERR_INVALID_ARGUMENT;
    if (c->fused_cluster < 0 || c->fused_cluster > 16 || c->fused_threads < 0 || c->fused_threads % 32 != 0)
        return METASD_ERR_INVALID_ARGUMENT;
    if (c->wait_poll_limit < 0 || c->row_cluster < 0 || c->row_cluster > 8) return METASD_ERR_INVALID_ARGUMENT;
    if ((uint64_t)c->vocab * (uint64_t)(c->max_draft + 1) >= (1ull << 31)) return METASD_ERR_UNSUPPORTED;
    return METASD_OK;
}

void free_all(metasd_ctx *c)
{
    cudaFree(c->st.t); cudaFree(c->st.arm); cudaFree(c->st.stat_a); cudaFree(c->st.stat_b);
    cudaFree(c->st.win_arm); cudaFree(c->st.win_reward); cudaFree(c->stats); cudaFree(c->status);
    cudaFree(c->stage_target); cudaFree(c->stage_draft); cudaFree(c->stage_tokens);
    cudaFree(c->stage_acc); cudaFree(c->stage_tok); cudaFree(c->stage_reward);
}

}  // namespace

// Everything of a blob's payload that a kernel later uses as an index or divides by: round counters, arms, the arms
// in the SW-UCB windows, and finite, non-negative statistics.  Plain host code: no CUDA call.
int metasd::validate_state_payload(const metasd_config &cfg, const void *payload)
{
    const size_t B = cfg.max_batch, K = cfg.n_drafters, tau = cfg.window;
    const char *r = (const char *)payload;
    auto take = [&](void *dst, size_t n) { memcpy(dst, r, n); r += n; };
    for (size_t i = 0; i < B; ++i) {
        int32_t t;
        take(&t, sizeof t);
        if (t < 0 || t >= 0x7FFFFFF0) return METASD_ERR_BAD_STATE_BLOB;
    }
    for (size_t i = 0; i < B; ++i) {
        int32_t arm;
        take(&arm, sizeof arm);
        if (arm < 0 || arm >= (int32_t)K) return METASD_ERR_BAD_STATE_BLOB;
    }
    for (size_t i = 0; i < 2 * B * K; ++i) {   // stat_a (means, sums, weights), stat_b (counts, memberships)
        double x;
        take(&x, sizeof x);
        if (!isfinite(x) || (i >= B * K && x < 0.0)) return METASD_ERR_BAD_STATE_BLOB;
        if (cfg.bandit == METASD_EXP3 && i < B * K && x < 0.0) return METASD_ERR_BAD_STATE_BLOB;
    }
    for (size_t i = 0; i < B * tau; ++i) {
        int32_t arm;
        take(&arm, sizeof arm);
        if (arm < 0 || arm >= (int32_t)K) return METASD_ERR_BAD_STATE_BLOB;
    }
    for (size_t i = 0; i < B * tau; ++i) {
        double x;
        take(&x, sizeof x);
        if (!isfinite(x)) return METASD_ERR_BAD_STATE_BLOB;
    }
    return METASD_OK;
}

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
    if (cfg->path == METASD_PATH_FUSED && !fused_supported(cfg->logit_dtype, cfg->vocab, cfg->max_draft))
        return METASD_ERR_UNSUPPORTED;

    metasd_ctx *c = new (std::nothrow) metasd_ctx();
    if (!c) return METASD_ERR_NO_MEMORY;
    memset(c, 0, sizeof *c);
    c->cfg = *cfg;
    DeviceScope scope(cfg->device);
    if (scope.error != cudaSuccess) { delete c; return cuda_fail(scope.error); }
    // the share of a row that L2 is asked to keep: the best measured values on B200 for 128k-152k vocabularies
    c->keep_permille = cfg->keep_permille == 0 ? (cfg->logit_dtype == METASD_BF16 ? 750 : 900)
                                               : (cfg->keep_permille < 0 ? 0 : cfg->keep_permille);
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
    if (cfg->host_staging) {
        const size_t row = (size_t)cfg->vocab * logit_size(cfg->logit_dtype);
        alloc(&c->stage_target, B * kp1 * row);
        alloc(&c->stage_draft, B * (kp1 - 1) * row);
        alloc((void **)&c->stage_tokens, B * (kp1 - 1) * sizeof(int32_t));
        alloc((void **)&c->stage_acc, B * sizeof(int32_t));
        alloc((void **)&c->stage_tok, B * sizeof(int32_t));
        alloc((void **)&c->stage_reward, B * sizeof(float));
    }
    bool unsupported = false;
    if (e == cudaSuccess) {
        e = streaming_prepare(cfg->device, cfg->logit_dtype, *cfg, &c->geo);
        if (e == cudaErrorNotSupported) { unsupported = true; (void)cudaGetLastError(); }
    }
    if (e == cudaSuccess) e = cudaMemset(c->status, 0, sizeof(uint32_t));
    if (e == cudaSuccess) e = launch_reset(c->st, cfg->max_batch, cfg->n_drafters, cfg->window, cfg->bandit, cfg->gamma,
                                            cfg->sequence_base, nullptr, cfg->max_batch, 0);
    if (e == cudaSuccess && cfg->path == METASD_PATH_FUSED) {
        e = fused_prepare(cfg->device, cfg->logit_dtype, cfg->vocab, cfg->max_batch, cfg->fused_cluster, cfg->fused_threads,
                          &c->plan);
        c->fused_ready = (e == cudaSuccess);
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        free_all(c);
        delete c;
        return unsupported ? METASD_ERR_UNSUPPORTED : cuda_fail(e);
    }
    *out = c;
    return METASD_OK;
}

void metasd_destroy(metasd_ctx *ctx)
{
    if (!ctx) return;
    {
        DeviceScope scope(ctx->cfg.device);
        free_all(ctx);
    }
    delete ctx;
}

int metasd_reset(metasd_ctx *ctx, const int32_t *seq_ids, int32_t n, void *stream)
{
    if (!ctx || n < 0) return METASD_ERR_INVALID_ARGUMENT;
    ON_DEVICE_OF(ctx);
    if (!seq_ids) n = ctx->cfg.max_batch;
    CK(launch_reset(ctx->st, ctx->cfg.max_batch, ctx->cfg.n_drafters, ctx->cfg.window, ctx->cfg.bandit, ctx->cfg.gamma,
                    ctx->cfg.sequence_base, seq_ids, n, (cudaStream_t)stream));
    ctx->launches += n > 0;
    return METASD_OK;
}

int metasd_select(metasd_ctx *ctx, int32_t batch, int32_t *arm_out, void *stream)
{
    if (!ctx || !arm_out || batch < 1 || batch > ctx->cfg.max_batch) return METASD_ERR_INVALID_ARGUMENT;
    ON_DEVICE_OF(ctx);
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

int metasd_resolved_row_kernel(const metasd_ctx *ctx) { return ctx ? ctx->geo.kernel : METASD_ERR_INVALID_ARGUMENT; }

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
    const int path = metasd_resolved_path(ctx, k);
    if (ctx->draft_len && cfg.path == METASD_PATH_FUSED) return METASD_ERR_UNSUPPORTED;
    ON_DEVICE_OF(ctx);

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
    {
        const long long nvec = (long long)cfg.vocab * (long long)logit_size(cfg.logit_dtype) / 16;
        p.keep_from_vec = (int32_t)(nvec - nvec * ctx->keep_permille / 1000);
    }
    p.poll_limit = cfg.wait_poll_limit > 0 ? (uint32_t)cfg.wait_poll_limit : (1u << 18);
    const size_t row_bytes = (size_t)cfg.vocab * logit_size(cfg.logit_dtype);
    // with a pointer table the per-drafter bases are not visible here: the kernels check every entry they use
    // against table_mask and never dereference one that fails
    p.vector_ok = row_bytes % 16 == 0 && ((uintptr_t)target_logits % 16) == 0 &&
                  (draft_logits ? ((uintptr_t)draft_logits % 16) == 0 : 1);
    p.table_mask = p.vector_ok ? 15u : (uint32_t)(logit_size(cfg.logit_dtype) - 1);

    cudaError_t e;
    if (path == METASD_PATH_FUSED && p.vector_ok)
        e = launch_fused(p, cfg.logit_dtype, ctx->plan, (cudaStream_t)stream, &ctx->launches);
    else if (cfg.path == METASD_PATH_FUSED)
        return METASD_ERR_UNSUPPORTED;
    else
        e = launch_streaming(p, cfg.logit_dtype, ctx->geo, (cudaStream_t)stream, &ctx->launches);
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
    ON_DEVICE_OF(ctx);
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

size_t metasd_state_bytes(const metasd_ctx *ctx) { return ctx ? blob_bytes(ctx->cfg) : 0; }

int metasd_state_export(metasd_ctx *ctx, void *host_buf, size_t bytes, void *stream)
{
    if (!ctx || !host_buf || bytes < metasd_state_bytes(ctx)) return METASD_ERR_INVALID_ARGUMENT;
    ON_DEVICE_OF(ctx);
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

int metasd_state_validate(const metasd_config *cfg, const void *host_buf, size_t bytes)
{
    int rc = validate_config(cfg);
    if (rc != METASD_OK) return rc;
    if (!host_buf || bytes < blob_bytes(*cfg)) return METASD_ERR_INVALID_ARGUMENT;
    BlobHeader h;
    memcpy(&h, host_buf, sizeof h);
    if (h.magic != BLOB_MAGIC || h.version != 1u || h.max_batch != cfg->max_batch || h.n_drafters != cfg->n_drafters ||
        h.window != cfg->window || h.bandit != cfg->bandit)
        return METASD_ERR_BAD_STATE_BLOB;
    return validate_state_payload(*cfg, (const char *)host_buf + sizeof h);
}

int metasd_state_import(metasd_ctx *ctx, const void *host_buf, size_t bytes, void *stream)
{
    if (!ctx || !host_buf || bytes < metasd_state_bytes(ctx)) return METASD_ERR_INVALID_ARGUMENT;
    // the kernels index with what the blob holds (arms, window entries, round counters): nothing reaches the device
    // before every value has been checked on the host
    int rc = metasd_state_validate(&ctx->cfg, host_buf, bytes);
    if (rc != METASD_OK) return rc;
    ON_DEVICE_OF(ctx);
    const size_t B = ctx->cfg.max_batch, K = ctx->cfg.n_drafters, tau = ctx->cfg.window;
    cudaStream_t s = (cudaStream_t)stream;
    const char *r = (const char *)host_buf + sizeof(BlobHeader);
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
    ON_DEVICE_OF(ctx);
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
    case METASD_ERR_BAD_STATE_BLOB: return "state blob does not match this context or holds values outside their range";
    default: return "unknown error";
    }
}

}  // extern "C"
