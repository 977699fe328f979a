/*
 * metasd.h -- C ABI of the MetaSD draft-verify hot path on NVIDIA B200 (sm_100a).
 *
 * One MetaSD round (Algorithm 1 of the paper: the bandit picks a drafter, one speculative-decoding
 * step runs with it, the alignment reward of that step updates the bandit) for a batch of
 * B independent sequences, each with its own bandit instance over K drafters:
 *
 *   metasd_select  : the drafter each sequence plays this round           (Algorithm 2, selection rule)
 *   metasd_verify  : speculative-sampling verification of k drafted tokens (Algorithm 4, verification loop),
 *                    the alignment reward (Definition 2, Eq. 4; or block efficiency, Sec. 2.3),
 *                    the bandit update (Algorithm 2, statistics update; Discounted UCB and Sliding-window
 *                    UCB of the non-stationary appendix) and the next round's selection.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless the parameter name starts with host_.
 *   - Logit tensors are dense, row-major, innermost dimension V (the vocabulary).  Rows whose
 *     byte length and base address are multiples of 16 take the vectorised path; anything else
 *     is still correct through a scalar path.
 *   - The caller owns every input and output buffer.  The library owns the context, the bandit
 *     state and its scratch; nothing is allocated after metasd_init.
 *   - Calls are asynchronous on the CUDA stream passed as `stream` (a cudaStream_t, typed void*
 *     so that this header needs no CUDA include); calls on one context must be stream-ordered.
 *     metasd_select, metasd_verify and metasd_reset only launch kernels: they may be captured into
 *     a CUDA graph.  A replay is the context's next round on whatever the captured buffers then
 *     hold (the round counter that keys the random numbers is device state, not a launch argument).
 *   - A context belongs to the device named in its configuration.  Every call that takes a context
 *     makes that device current for its own duration and restores the caller's current device before
 *     it returns; `stream` must be a stream of the context's device (or NULL).
 *   - Every function returns 0 (METASD_OK) or a negative metasd_error.  Device-side anomalies
 *     never trap: they set bits in the context's status word and produce the defined outputs
 *     described at metasd_last_status.
 *   - There is no CPU fallback: without a CUDA device metasd_init fails with METASD_ERR_CUDA.
 */
#ifndef METASD_H
#define METASD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct metasd_ctx metasd_ctx;

enum metasd_error {
    METASD_OK = 0,
    METASD_ERR_INVALID_ARGUMENT = -1,
    METASD_ERR_UNSUPPORTED = -2,
    METASD_ERR_CUDA = -3,
    METASD_ERR_NO_MEMORY = -4,
    METASD_ERR_BAD_STATE_BLOB = -5
};

enum metasd_dtype { METASD_BF16 = 0, METASD_FP32 = 1 };
enum metasd_bandit {
    METASD_UCB = 0,   /* Algorithm 2 */
    METASD_DUCB = 1,  /* Discounted UCB (non-stationary appendix) */
    METASD_SWUCB = 2, /* Sliding-window UCB (non-stationary appendix) */
    METASD_EXP3 = 3,  /* MetaSD-EXP3 (the algorithm box of that name): arms drawn from
                         p_t(i) = (1 - gamma) w_i / sum w + gamma / K, w_a <- w_a exp(gamma (r / p_t(a)) / K) */
    METASD_RAND = 4,  /* the uniformly random baseline of the paper's tables */
    METASD_PETC = 5   /* Pure exploration-then-commit (the algorithm box of that name): one Sequential Halving run
                         (the box of that name) over `window` rounds, then the surviving drafter only.
                         ceil(log2 K) phases; every surviving drafter is played floor(window / (survivors * phases))
                         times per phase (at least once), in index order, one block of rounds each; the half with the
                         larger phase sums survives, the lower index on equal sums */
};
enum metasd_reward { METASD_REWARD_BD = 0, METASD_REWARD_BE = 1 };

/* How the row-statistics kernel of the streaming path brings logit rows on chip (16-byte aligned rows; rows
 * that are not take plain scalar loads whatever is asked for). */
enum metasd_row_kernel {
    METASD_ROWS_AUTO = 0,    /* the fastest measured variant for the dtype */
    METASD_ROWS_PLAIN = 1,   /* ld.global straight into registers */
    METASD_ROWS_STAGED = 2,  /* per-thread cp.async into shared-memory slots, several trips ahead */
    METASD_ROWS_BULK = 3     /* a persistent CTA per SM: one warp issues TMA bulk copies (cp.async.bulk, mbarrier
                                completion) into a shared-memory ring, the other warps consume it */
};

/* Which kernels metasd_verify launches. */
enum metasd_path {
    METASD_PATH_AUTO = 0,      /* the fastest measured path for the shape (currently: streaming) */
    METASD_PATH_STREAMING = 1, /* row-statistics kernel + per-sequence epilogue kernel; any shape */
    METASD_PATH_FUSED = 2      /* one persistent thread-block-cluster kernel per call: every logit is read
                                  from HBM once; needs 16-byte aligned rows that fit its geometry, else
                                  metasd_init returns METASD_ERR_UNSUPPORTED */
};

/* Status bits (OR-accumulated on the device until read). */
#define METASD_STATUS_NONFINITE 1u /* a row held NaN / +Inf or no finite entry */
#define METASD_STATUS_TOKEN_OOR 2u /* a drafted token id was outside [0, V) */
#define METASD_STATUS_Q_ZERO    4u /* the drafter gave probability 0 to its own drafted token */
#define METASD_STATUS_TIMEOUT   8u /* a bounded device-side wait on an asynchronous copy ran out (see wait_poll_limit): the
                                      call still ends, its outputs are undefined, the context stays usable */
#define METASD_STATUS_BAD_LENGTH 32u /* a registered per-sequence draft length was outside 1 .. k: it was clamped */
#define METASD_STATUS_BAD_POINTER 16u /* the drafter table of a call held a NULL or misaligned entry: its rows are never
                                        read and the outputs of the sequences that played that drafter are meaningless */

/* Hyper-parameters of metasd_init.  Paper notation: n_drafters = K, max_draft = N_max, beta = the
 * exploration strength of Algorithm 2 (experiments: 0.01), gamma = the D-UCB decay or, for METASD_EXP3, its
 * mixing parameter (both are called gamma in the paper), window = the SW-UCB window tau or, for METASD_PETC, its
 * exploration budget in rounds (none of these values
 * is given in the paper; 0.975 / 50 are this library's defaults).
 * The randomised policies draw the arm of round t from word 2 of the Philox block keyed by the seed of the
 * latest metasd_verify call (0 before the first one) at counter (sequence_base + b, t, 0xFFFFFFFF, 0):
 * EXP3 by inverse CDF in arm order over the 24-bit uniform, RAND as floor(uniform * K). */
typedef struct metasd_config {
    int32_t max_batch;          /* B: sequences, 1 .. 65535 */
    int32_t n_drafters;         /* K: 1 .. 16 */
    int32_t max_draft;          /* N_max: 1 .. 16 */
    int32_t vocab;              /* V >= 1 */
    int32_t logit_dtype;        /* metasd_dtype */
    int32_t bandit;             /* metasd_bandit */
    int32_t reward;             /* metasd_reward */
    int32_t window;             /* tau >= 1 (METASD_SWUCB), exploration rounds (METASD_PETC) */
    int32_t device;             /* CUDA device ordinal */
    int32_t path;               /* metasd_path */
    uint32_t sequence_base;     /* id of sequence 0 in the random-number key (batch sharding) */
    int32_t host_staging;       /* != 0: also allocate device staging for metasd_verify_host */
    double beta;
    double gamma;
    double reward_temperature;  /* softmax temperature of the reward when verifying greedily */
    /* Tuning and test fields; 0 everywhere (what metasd_default_config writes) selects the measured defaults. */
    int32_t row_kernel;         /* metasd_row_kernel */
    int32_t row_threads;        /* threads per CTA of the row-statistics kernel; only the built shapes are accepted */
    int32_t row_stages;         /* depth of its shared-memory staging; only the built shapes are accepted */
    int32_t keep_permille;      /* share (its end, in 1/1000) of every row that the first sweep asks L2 to keep for the
                                   second; 0 = default, negative = keep nothing */
    int32_t fused_cluster;      /* METASD_PATH_FUSED: CTAs per cluster (0 = the smallest that fits) */
    int32_t fused_threads;      /* METASD_PATH_FUSED: threads per CTA (0 = chosen from the slice length) */
    int32_t wait_poll_limit;    /* polls after which a device-side wait on an asynchronous copy gives up and sets
                                   METASD_STATUS_TIMEOUT (0 = 2^18 polls of up to 4 us each: about a second).  For tests of that path. */
    int32_t row_cluster;        /* METASD_ROWS_STAGED: CTAs (a thread-block cluster) that share one row pair, each a
                                   contiguous part of it; 0 or 1 = one CTA per row pair; only the built shapes are accepted */
} metasd_config;

/* Optional per-position diagnostics of metasd_verify, [B, k]. */
typedef struct metasd_diag {
    float p_x;      /* target probability of the drafted token */
    float q_x;      /* drafter probability of the drafted token */
    float D;        /* d_TV(p_j, q_j) */
    float u;        /* the uniform of the accept test */
    int32_t accept; /* 1 = the accept test passed at this position */
} metasd_diag;

/* Fills *cfg with the defaults (UCB, BD reward, beta 0.01, gamma 0.975, window 50, bf16, auto path). */
void metasd_default_config(metasd_config *cfg);

/* Creates a context on cfg->device: validates cfg, allocates bandit state, scratch and (optionally)
 * staging, and resets every sequence (Algorithm 2, initialisation: t <- 0).  *out is NULL on failure. */
int metasd_init(metasd_ctx **out, const metasd_config *cfg);

/* Frees everything metasd_init allocated.  NULL is accepted. */
void metasd_destroy(metasd_ctx *ctx);

/* Per-query re-initialisation (experimental setup section: one bandit run per query):
 * t <- 0 and cleared arm statistics for the n sequences listed in seq_ids (device int32),
 * or for all sequences when seq_ids is NULL.  Ids outside [0, max_batch) are ignored. */
int metasd_reset(metasd_ctx *ctx, const int32_t *seq_ids, int32_t n, void *stream);

/* Algorithm 2, round-robin start and selection rule: arm_out[b] = the drafter sequence b plays this round, b < batch.
 * Rounds t < K play arm t (the initial sweep); afterwards argmax_i mu_i + beta sqrt(2 ln t / n_i),
 * lowest index on ties; an arm with no pull inside the SW-UCB window scores +infinity.  METASD_EXP3 and
 * METASD_RAND: the arm drawn as described at metasd_config. */
int metasd_select(metasd_ctx *ctx, int32_t batch, int32_t *arm_out, void *stream);

/* One verification round for sequences 0 .. batch-1 (Algorithm 4 verification loop, Definition 2,
 * Algorithm 2 statistics update, then the next selection).
 *
 *   target_logits  [batch, k+1, V]  target logits at the k drafted positions and the bonus position
 *   draft_logits   [batch, k, V]    the played drafter's logits, already gathered by arm; or NULL and
 *   drafter_ptrs   device table of K pointers, each [batch, k, V]; the kernel reads table[arm[b]]
 *   draft_tokens   [batch, k] int32 when token_arm_stride == 0, else [K, ...] with
 *                  token_arm_stride int32 elements between consecutive drafters' [batch, k] blocks
 *   temperature    T > 0: accept iff u < min(1, p(x)/q(x)) with p, q = softmax(logits / T);
 *                  T == 0: greedy, accept iff x == argmax of the target row (lowest id on ties) and
 *                  the reward uses softmax(logits / reward_temperature)
 *   seed           key of the counter-based Philox4x32-10 stream; the counter is
 *                  (sequence_base + b, round t of sequence b, position j, 0); word 0 drives the
 *                  accept test, word 1 the residual / bonus draw; uniform = top 24 bits * 2^-24
 *   accepted_len   [batch] int32, N_acc in [0, k]
 *   next_token     [batch] int32, drawn from max(0, p - q) at the first rejection (inverse CDF in
 *                  token order), or from p at position k if all accepted; greedy: the argmax;
 *                  -1 when the row it needs is flagged non-finite
 *   reward         [batch] fp32, BD: 1 - mean_j d_TV(p_j, q_j) over all k positions; BE: N_acc / k
 *   diag           optional [batch, k]
 *
 * On return (stream order) each sequence's round counter is t+1 and its statistics include the
 * reward.  Errors: invalid sizes / NULL pointers / both or neither draft source -> INVALID_ARGUMENT. */
int metasd_verify(metasd_ctx *ctx, int32_t batch, int32_t k, const void *target_logits,
                  const void *draft_logits, const void *const *drafter_ptrs,
                  const int32_t *draft_tokens, int64_t token_arm_stride, float temperature,
                  uint64_t seed, int32_t *accepted_len, int32_t *next_token, float *reward,
                  metasd_diag *diag, void *stream);

/* Per-sequence draft lengths (the paper fixes N_max per run and sweeps it as an ablation; a serving batch mixes
 * lengths): draft_len is a DEVICE array [max_batch] of int32 that metasd_verify reads on every later call, or NULL
 * to go back to "every sequence drafted k tokens".  Sequence b then uses target rows 0 .. draft_len[b] (the last one
 * is its bonus row) and draft rows / tokens 0 .. draft_len[b]-1 of its k-padded slots; nothing behind them is read,
 * accepted_len[b] <= draft_len[b], and both rewards are normalised by draft_len[b].  The layout of every buffer is
 * unchanged.  A length outside 1 .. k is clamped and sets METASD_STATUS_BAD_LENGTH.  The caller owns the array and
 * keeps it valid (its contents may change between calls, in stream order).  Streaming path only: with lengths
 * registered, a context whose path is METASD_PATH_FUSED returns METASD_ERR_UNSUPPORTED from metasd_verify. */
int metasd_set_draft_lengths(metasd_ctx *ctx, const int32_t *draft_len);

/* The same round with HOST buffers (gathered draft logits only): copies the inputs to the context's
 * staging memory, runs metasd_verify, copies the three outputs (and host_arm_next, optional: the
 * next round's selection) back, and synchronises the stream.  Needs cfg.host_staging != 0.
 * Pinned host memory makes the copies asynchronous. */
int metasd_verify_host(metasd_ctx *ctx, int32_t batch, int32_t k, const void *host_target_logits,
                       const void *host_draft_logits, const int32_t *host_draft_tokens,
                       float temperature, uint64_t seed, int32_t *host_accepted_len,
                       int32_t *host_next_token, float *host_reward, int32_t *host_arm_next,
                       void *stream);

/* Bandit state as a flat blob in HOST memory (round counters, current arms, arm statistics,
 * SW-UCB windows, and a header that import checks against the context's configuration).
 * Both calls synchronise the stream. */
size_t metasd_state_bytes(const metasd_ctx *ctx);
int metasd_state_export(metasd_ctx *ctx, void *host_buf, size_t bytes, void *stream);
int metasd_state_import(metasd_ctx *ctx, const void *host_buf, size_t bytes, void *stream);

/* The check metasd_state_import makes before anything reaches the device, as a host-only call (no CUDA): the header
 * must match cfg, every round counter must be >= 0, every current arm and every arm recorded in an SW-UCB window
 * must lie in [0, K), every statistic must be finite and every count non-negative -- the kernels index and divide
 * with these values.  Returns METASD_OK, METASD_ERR_BAD_STATE_BLOB, or METASD_ERR_INVALID_ARGUMENT (NULL, short
 * buffer, invalid cfg). */
int metasd_state_validate(const metasd_config *cfg, const void *host_buf, size_t bytes);

/* Reads and clears the status word (synchronises the stream).  Defined outputs: a non-finite row
 * pair is rejected with d_TV = 1; an out-of-range token is rejected; q(x) = 0 < p(x) is accepted. */
int metasd_last_status(metasd_ctx *ctx, uint32_t *host_flags, void *stream);

/* Number of kernels this context has launched so far. */
uint64_t metasd_kernel_launches(const metasd_ctx *ctx);

/* The path metasd_verify takes for draft length k with the context's configuration
 * (METASD_PATH_STREAMING or METASD_PATH_FUSED). */
int metasd_resolved_path(const metasd_ctx *ctx, int32_t k);

/* The row-statistics variant the streaming path of this context launches for 16-byte aligned rows
 * (a metasd_row_kernel other than METASD_ROWS_AUTO). */
int metasd_resolved_row_kernel(const metasd_ctx *ctx);

/* One verification round for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging of the stateless part of metasd_verify -- Algorithm 4's verification loop
 * and the reward -- for hosts where cudaMalloc is not available to this code: a serving process whose
 * memory pool already owns the whole device, a plugin that may not allocate after start-up, or a
 * latency-critical thread that must stay clear of the allocator.  Such callers cannot create a
 * context, so there is no bandit here and nothing persists between calls.)
 *
 * It launches the kernels of a default streaming context (the staged row-statistics kernel for 16-byte aligned
 * rows, the plain-load one otherwise, then the epilogue).  Their scratch lives in a fixed array inside the library image (about 0.7 MB, held
 * by every GPU that loads the library until the process exits), which bounds the sizes:
 * batch <= METASD_NOALLOC_MAX_BATCH and batch * (k + 1) <= METASD_NOALLOC_MAX_ROWS; beyond that the
 * call returns METASD_ERR_UNSUPPORTED and launches nothing.  The call makes no cudaMalloc / cudaFree
 * and calls no allocating library routine.
 *
 * Runs on the calling thread's current device.  The first call on each device looks up the array's
 * device address, and the first call per device and logit type sets the launch attribute its row-statistics
 * kernel needs (one-time runtime queries, no allocation): make those first calls before any stream capture begins.
 * All calls on a device share the one array and it keeps the previous call's contents; every field
 * the kernels read is rewritten at the start of each call, so calls in stream order are independent,
 * but two calls that overlap on the GPU (different streams, no ordering between them) race on it.
 *
 *   target_logits [batch, k+1, V], draft_logits [batch, k, V] (gathered), draft_tokens [batch, k]:
 *   as for metasd_verify; logit_dtype is a metasd_dtype, reward_kind a metasd_reward;
 *   reward_temperature is used only when temperature == 0 (greedy);
 *   round is the counter that keys the uniforms with (sequence_base + b, round, position);
 *   status_out: optional device uint32 that receives this call's METASD_STATUS_* bits. */
#define METASD_NOALLOC_MAX_BATCH 4096
#define METASD_NOALLOC_MAX_ROWS 16384
int metasd_verify_noalloc(int32_t batch, int32_t k, int32_t vocab, int32_t logit_dtype,
                          const void *target_logits, const void *draft_logits,
                          const int32_t *draft_tokens, float temperature, float reward_temperature,
                          int32_t reward_kind, uint64_t seed, uint32_t sequence_base, uint32_t round,
                          int32_t *accepted_len, int32_t *next_token, float *reward,
                          uint32_t *status_out, void *stream);

const char *metasd_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* METASD_H */
