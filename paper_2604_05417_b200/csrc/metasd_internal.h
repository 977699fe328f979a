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
                          // the row's maximum, or the target row's where the staged kernel could share it
    double sum_min;       // sum_v min(p_v, q_v) = 1 - d_TV(p, q)
    int32_t argmax_a;     // first index of the target row's maximum
    uint32_t flags;       // METASD_STATUS_* of this row pair
};

// What one CTA of a group publishes about its part of a row pair (split streaming path).
struct GroupRecord {
    float max_a, sum_a, max_b, sum_b;
    int32_t argmax_a;
    int32_t pad[3];
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
    int32_t keep_permille;   // share of every row (its end) that the first sweep asks L2 to keep
    int32_t keep_from_vec;   // the same as an index: first 16-byte vector of a row in the kept share
    int32_t k1_stages;       // depth of the row-statistics kernel's cp.async pipeline (0 or 1: plain loads)
    // split streaming path: grp_size CTAs share a row pair (0: one CTA per row pair)
    int32_t grp_size;
    int32_t grp_ctas;        // CTAs of the launch (co-resident)
    GroupRecord *grp_rec;    // [batch * (k + 1), grp_size]
    double *grp_min;         // [batch * (k + 1), grp_size] partial sums of min(p, q)
    uint32_t *grp_count;     // [batch * (k + 1)] arrivals, cleared before every launch
};

// streaming path (metasd_streaming.cu)
cudaError_t launch_streaming(const VerifyParams &p, int dtype, cudaStream_t stream, uint64_t *launches);
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
cudaError_t fused_prepare(int device, int dtype, int V, int max_batch, FusedPlan *plan);
cudaError_t launch_fused(const VerifyParams &p, int dtype, const FusedPlan &plan, cudaStream_t stream,
                         uint64_t *launches);
// how many CTAs of the split kernel are co-resident, and how many of them should share a row pair so that
// the rows in flight stay inside L2 (1: not worth splitting)
cudaError_t split_prepare(int device, int dtype, int V, int *resident_ctas, int *group_size);
// copies the drafter table, flagging and replacing entries that must not be dereferenced (metasd_streaming.cu)
cudaError_t launch_sanitize_table(const void *const *table, int K, const void *target, uint32_t mask, const void **clean,
                                  uint32_t *status, cudaStream_t stream);
// small state kernels (metasd_streaming.cu)
cudaError_t launch_select(const BanditState &st, int batch, int32_t *arm_out, cudaStream_t stream);
cudaError_t launch_reset(const BanditState &st, int max_batch, int K, int tau, int variant, double gamma,
                         uint32_t sequence_base, const int32_t *seq_ids, int n, cudaStream_t stream);

}  // namespace metasd
