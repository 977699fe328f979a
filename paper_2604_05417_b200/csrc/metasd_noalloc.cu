// metasd_verify_noalloc: one verification round for callers that cannot allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- a serving loop whose memory pool
// owns the whole device and hands out no more, a plugin loaded into a host process that forbids
// allocations after start-up, or a latency-critical thread that must not take the allocator's
// device-wide lock.  Such a caller cannot create a metasd context (metasd_init allocates the bandit
// state and the row-statistics scratch), so this entry point keeps the scratch in a fixed array that
// is part of the library image: every GPU that loads the library holds it until the process exits.
//
// The round it runs is the stateless part of metasd_verify: softmax statistics, accept tests, first
// rejection, correction/bonus draw and the reward, launched as the two streaming kernels a context
// with the default configuration launches for the same logit type (the staged row-statistics kernel
// for 16-byte aligned rows, the plain-load one otherwise, then the epilogue).  There is no bandit here
// (nothing persists between calls); the caller passes the round counter that keys the random numbers.
#include <mutex>

#include "metasd_internal.h"

using namespace metasd;

namespace {

constexpr int NOALLOC_MAX_ROWS = METASD_NOALLOC_MAX_ROWS;    // batch * (k + 1)
constexpr int NOALLOC_MAX_BATCH = METASD_NOALLOC_MAX_BATCH;

// Everything the two kernels keep in global memory besides the caller's inputs and outputs.
struct StaticScratch {
    RowStats rows[NOALLOC_MAX_ROWS];       // written by the row-statistics kernel, read by the epilogue
    double stat_a[NOALLOC_MAX_BATCH];      // a one-armed dummy bandit per sequence: the epilogue kernel
    double stat_b[NOALLOC_MAX_BATCH];      // updates it and nobody reads it
    double win_reward[NOALLOC_MAX_BATCH];
    int32_t t[NOALLOC_MAX_BATCH];          // round counter the epilogue keys the uniforms with
    int32_t arm[NOALLOC_MAX_BATCH];
    int32_t win_arm[NOALLOC_MAX_BATCH];
    uint32_t status;
};

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a
// device address and must never be passed to a kernel.
static __device__ __align__(256) StaticScratch g_noalloc_scratch[1];

// Device code may name the array directly: start every call from a clean dummy-bandit block.
__global__ void noalloc_prepare_kernel(int batch, int32_t round)
{
    StaticScratch &s = g_noalloc_scratch[0];
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) s.status = 0u;
    if (b < batch) {
        s.t[b] = round;
        s.arm[b] = 0;
        s.stat_a[b] = 0.0;
        s.stat_b[b] = 0.0;
        s.win_arm[b] = 0;
        s.win_reward[b] = 0.0;
    }
}

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_lock;
StaticScratch *g_scratch_ptr[MAX_DEVICES];   // device address of the array on each device, once known
RowGeometry g_geometry[MAX_DEVICES][2];      // launch shape of the row-statistics kernel per device and logit type
bool g_geometry_ready[MAX_DEVICES][2];

// Once per device, with that device current: ask the runtime where the array lives there.
cudaError_t scratch_address(int device, StaticScratch **out)
{
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_scratch_ptr[device]) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[device] = static_cast<StaticScratch *>(ptr);
    }
    *out = g_scratch_ptr[device];
    return cudaSuccess;
}

// Once per device and logit type: the default launch shape and the function attribute (a larger dynamic
// shared-memory window) its kernel needs.  Neither allocates device memory.
cudaError_t default_geometry(int device, int dtype, RowGeometry *out)
{
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_geometry_ready[device][dtype]) {
        metasd_config cfg;
        metasd_default_config(&cfg);
        cudaError_t e = streaming_prepare(device, dtype, cfg, &g_geometry[device][dtype]);
        if (e != cudaSuccess) return e;
        g_geometry_ready[device][dtype] = true;
    }
    *out = g_geometry[device][dtype];
    return cudaSuccess;
}

}  // namespace

extern "C" int metasd_verify_noalloc(int32_t batch, int32_t k, int32_t vocab, int32_t logit_dtype,
                                     const void *target_logits, const void *draft_logits,
                                     const int32_t *draft_tokens, float temperature, float reward_temperature,
                                     int32_t reward_kind, uint64_t seed, uint32_t sequence_base, uint32_t round,
                                     int32_t *accepted_len, int32_t *next_token, float *reward,
                                     uint32_t *status_out, void *stream)
{
    if (batch < 1 || k < 1 || k > 16 || vocab < 1) return METASD_ERR_INVALID_ARGUMENT;
    if (batch > NOALLOC_MAX_BATCH || (int64_t)batch * (k + 1) > NOALLOC_MAX_ROWS) return METASD_ERR_UNSUPPORTED;
    if ((uint64_t)vocab * (uint64_t)(k + 1) >= (1ull << 31)) return METASD_ERR_UNSUPPORTED;
    if (logit_dtype != METASD_BF16 && logit_dtype != METASD_FP32) return METASD_ERR_UNSUPPORTED;
    if (reward_kind != METASD_REWARD_BD && reward_kind != METASD_REWARD_BE) return METASD_ERR_UNSUPPORTED;
    if (!target_logits || !draft_logits || !draft_tokens || !accepted_len || !next_token || !reward)
        return METASD_ERR_INVALID_ARGUMENT;
    if (!(temperature >= 0.f) || !(temperature < INFINITY) || round > 0x7FFFFFFFu) return METASD_ERR_INVALID_ARGUMENT;
    if (temperature == 0.f && !(reward_temperature > 0.f && reward_temperature < INFINITY))
        return METASD_ERR_INVALID_ARGUMENT;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= MAX_DEVICES) return METASD_ERR_CUDA;
    StaticScratch *scratch = nullptr;
    if (scratch_address(device, &scratch) != cudaSuccess) return METASD_ERR_CUDA;
    RowGeometry geo;
    if (default_geometry(device, logit_dtype, &geo) != cudaSuccess) return METASD_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;

    VerifyParams p = {};
    p.batch = batch; p.k = k; p.V = vocab;
    p.K = 1; p.bandit = METASD_UCB; p.reward_kind = reward_kind; p.tau = 1;
    p.sequence_base = sequence_base;
    p.target = target_logits; p.draft = draft_logits; p.drafter_ptrs = nullptr;
    p.tokens = draft_tokens; p.token_arm_stride = 0;
    p.greedy = temperature == 0.f;
    p.c = (float)(1.4426950408889634 / (p.greedy ? (double)reward_temperature : (double)temperature));
    p.seed = seed; p.beta = 0.0; p.gamma = 1.0;
    p.accepted_len = accepted_len; p.next_token = next_token; p.reward = reward; p.diag = nullptr;
    p.st.t = scratch->t; p.st.arm = scratch->arm;
    p.st.stat_a = scratch->stat_a; p.st.stat_b = scratch->stat_b;
    p.st.win_arm = scratch->win_arm; p.st.win_reward = scratch->win_reward;
    p.stats = scratch->rows;
    p.status = &scratch->status;
    const size_t row_bytes = (size_t)vocab * (logit_dtype == METASD_BF16 ? 2 : 4);
    p.vector_ok = row_bytes % 16 == 0 && ((uintptr_t)target_logits % 16) == 0 && ((uintptr_t)draft_logits % 16) == 0;
    {   // the share of every row that L2 is asked to keep between the sweeps: as in a default context
        const long long nvec = (long long)row_bytes / 16;
        p.keep_from_vec = (int32_t)(nvec - nvec * (logit_dtype == METASD_BF16 ? 750 : 900) / 1000);
    }
    p.poll_limit = 1u << 18;

    noalloc_prepare_kernel<<<(batch + 255) / 256, 256, 0, s>>>(batch, (int32_t)round);
    cudaError_t e = cudaGetLastError();
    uint64_t launches = 0;
    if (e == cudaSuccess) e = launch_streaming(p, logit_dtype, geo, s, &launches);
    if (e == cudaSuccess && status_out)
        e = cudaMemcpyAsync(status_out, &scratch->status, sizeof(uint32_t), cudaMemcpyDeviceToDevice, s);
    return e == cudaSuccess ? METASD_OK : METASD_ERR_CUDA;
}
