// Internal declarations shared by the translation units of libmetasd (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "metasd.h"

namespace metasd {

// Per-(sequence, position) result of the row-statistics pass; the scratch the streaming path keeps
// between its two kernels.  Softmax terms are held relative to the raw row maximum:
//   p_v = 2^((x_v - max_a) * c) / sum_a,  c = log2(e) / T.
struct RowStats {
    float max_a, sum_a;   // target row
    float max_b, sum_b;   // draft row (unused at the bonus position); max_b is the reference sum_b is relative to:
                          // the row's maximum, or the target row's where the staged kernels could share it
    double sum_min;       // sum_v min(p_v, q_v) = 1 - d_TV(p, q)
    int32_t argmax_a;     // first index of the target row's maximum
    uint32_t flags;       // METASD_STATUS_* of this row pair
};

// Bandit state of all sequences, structure of arrays in device memory.
struct BanditState {
    int32_t *t;          // [B] rounds completed
    int32_t *arm;        // [B] arm to play in round t
    double *stat_a;      // [B, K] UCB: mu_hat;  D-UCB: discounted reward sum
    double *stat_b;      // [B, K] UCB: n;       D-UCB: discounted count
    int32_t *win_arm;    // [B, tau] SW-UCB: arm of round s in slot s mod tau
    double *win_reward;  // [B, tau]
};

// Shape of the row-statistics launch, resolved from the configuration once per context.
struct RowGeometry {
    int32_t kernel;     // metasd_row_kernel, never AUTO
    int32_t threads;    // threads per CTA
    int32_t stages;     // staging depth (0 for plain loads)
    int32_t per_sm;     // CTAs per SM the shape is built for
    int32_t n_sm;       // SMs of the device (persistent kernels size their grid with it)
    int32_t cluster;    // CTAs that share one row pair (1: none)
};

struct VerifyParams {
    // shapes
    int32_t batch, k, V;
    int32_t K, bandit, reward_kind, tau;
    uint32_t sequence_base;
    // inputs
    const void *target;
    const void *draft;                 // gathered, or nullptr
    const void *const *drafter_ptrs;   // table, or nullptr
    const int32_t *tokens;
    const int32_t *draft_len;          // [batch] tokens drafted per sequence this round, or nullptr = k for all
    int64_t token_arm_stride;
    // math
    float c;           // log2(e) / softmax temperature
    int32_t greedy;
    uint64_t seed;
    double beta, gamma;
    // outputs
    int32_t *accepted_len;
    int32_t *next_token;
    float *reward;
    metasd_diag *diag;
    // state + scratch
    BanditState st;
    RowStats *stats;   // [batch, k+1]
    uint32_t *status;
    int32_t vector_ok; // rows are 16-byte aligned and a whole number of 16-byte vectors
    int32_t keep_from_vec;   // first 16-byte vector of a row in the share that the first sweep asks L2 to keep
    uint32_t poll_limit;     // polls after which a wait on an asynchronous copy gives up
    uint32_t table_mask;     // pointer-table mode: low address bits that must be clear in every entry
};

// streaming path (metasd_streaming.cu, metasd_bulk.cu)
cudaError_t streaming_prepare(int device, int dtype, const metasd_config &cfg, RowGeometry *geo);
cudaError_t launch_streaming(const VerifyParams &p, int dtype, const RowGeometry &geo, cudaStream_t stream, uint64_t *launches);
cudaError_t bulk_prepare(int dtype, RowGeometry *geo);
cudaError_t launch_row_stats_bulk(const VerifyParams &p, int dtype, const RowGeometry &geo, cudaStream_t stream);
// fused cluster path (metasd_fused.cu)
struct FusedPlan {
    int32_t cluster;       // CTAs per cluster (0: no plan)
    int32_t threads;       // threads per CTA
    int32_t n_vec_row;     // 16-byte vectors per logit row
    int32_t n_vec_cta;     // vectors of a row owned by one CTA
    int32_t n_slot;        // log2 of the vectors per chunk of a slice
    int32_t slot_bytes;
    int32_t max_clusters;  // co-resident clusters on the device
    size_t smem_bytes;     // dynamic shared memory of the launch
    long work_per_item;    // threads x vectors per thread
};
bool fused_supported(int dtype, int V, int k);
cudaError_t fused_prepare(int device, int dtype, int V, int max_batch, int pin_cluster, int pin_threads, FusedPlan *plan);
cudaError_t launch_fused(const VerifyParams &p, int dtype, const FusedPlan &plan, cudaStream_t stream,
                         uint64_t *launches);
// small state kernels (metasd_streaming.cu)
cudaError_t launch_select(const BanditState &st, int batch, int32_t *arm_out, cudaStream_t stream);
cudaError_t launch_reset(const BanditState &st, int max_batch, int K, int tau, int variant, double gamma,
                         uint32_t sequence_base, const int32_t *seq_ids, int n, cudaStream_t stream);

// Host-side check of a state blob's payload against what the kernels index with (metasd_api.cu).
int validate_state_payload(const metasd_config &cfg, const void *payload);

}  // namespace metasd
