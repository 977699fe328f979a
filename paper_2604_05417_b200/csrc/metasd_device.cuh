// Device-side building blocks of the MetaSD hot path: Philox4x32-10, fast exp2, 16-byte logit
// vectors, warp/block reductions and the fp64 bandit arithmetic.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "metasd_internal.h"

namespace metasd {

// A finite stand-in for "no maximum yet": keeps (x - max) * c finite for masked (-inf) logits.
#define METASD_NEG_BIG (-1.0e30f)

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and key bumps.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, uint2 key)
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(M0, ctr.x), lo0 = M0 * ctr.x;
        uint32_t hi1 = __umulhi(M1, ctr.z), lo1 = M1 * ctr.z;
        ctr = make_uint4(hi1 ^ ctr.y ^ key.x, lo1, hi0 ^ ctr.w ^ key.y, lo0);
        key.x += 0x9E3779B9u;
        key.y += 0xBB67AE85u;
    }
    return ctr;
}

// Uniform in [0, 1) from the top 24 bits of a word (exact in fp32).
__device__ __forceinline__ float uniform24(uint32_t w) { return (float)(w >> 8) * (1.0f / 16777216.0f); }

// The random words of (seed, sequence, round, position): .x accept test, .y residual / bonus draw.
__device__ __forceinline__ uint4 round_words(uint64_t seed, uint32_t sequence, uint32_t round, uint32_t position)
{
    return philox4x32_10(make_uint4(sequence, round, position, 0u),
                         make_uint2((uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)));
}

// ---------------------------------------------------------------------------------------------
// exp2 on the special-function unit (flushes denormals; relative error about 2^-22)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---------------------------------------------------------------------------------------------
// Logit element types: 16-byte vectors of bf16 (8 per vector) or fp32 (4 per vector)
// ---------------------------------------------------------------------------------------------
template <typename LT> struct Logit;

template <> struct Logit<__nv_bfloat16> {
    static constexpr int VEC = 8;
    __device__ static __forceinline__ void unpack(const uint4 &raw, float (&x)[8])
    {
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static __forceinline__ float scalar(const __nv_bfloat16 *p, size_t i)
    {
        return __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(p)[i] << 16);
    }
};

template <> struct Logit<float> {
    static constexpr int VEC = 4;
    __device__ static __forceinline__ void unpack(const uint4 &raw, float (&x)[4])
    {
        x[0] = __uint_as_float(raw.x);
        x[1] = __uint_as_float(raw.y);
        x[2] = __uint_as_float(raw.z);
        x[3] = __uint_as_float(raw.w);
    }
    __device__ static __forceinline__ float scalar(const float *p, size_t i) { return p[i]; }
};

// Tokens sequence b drafted this round: the call's k unless the caller registered per-sequence lengths, which are
// clamped to 1 .. k (the epilogue flags a length outside that range).
__device__ __forceinline__ int drafted(const int32_t *draft_len, int b, int k)
{
    if (!draft_len) return k;
    const int kb = draft_len[b];
    return kb < 1 ? 1 : (kb > k ? k : kb);
}

// Rows of the drafter sequence b plays: the gathered tensor, or the entry of the caller's pointer table for the
// sequence's arm.  An entry that is NULL or not aligned like the target (table_mask: 15 on the vector path, else
// the element size minus one) is never dereferenced: the target tensor stands in for it, so that the outputs of the
// sequences that play that drafter are defined (if meaningless); the epilogue flags such a table once per call.
template <typename LT>
__device__ __forceinline__ const LT *draft_rows(const VerifyParams &p, int b)
{
    if (p.draft) return reinterpret_cast<const LT *>(p.draft);
    const void *q = p.drafter_ptrs[p.st.arm[b]];
    if (q == nullptr || (reinterpret_cast<uintptr_t>(q) & p.table_mask) != 0) q = p.target;
    return reinterpret_cast<const LT *>(q);
}

// Streaming 16-byte load that does not allocate in L1.
__device__ __forceinline__ uint4 ld_stream(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// The same load with an L2 eviction policy (from createpolicy): evict_last keeps the line for a later re-read,
// evict_first gives it up early.
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint4 ld_stream_hint(const void *p, uint64_t policy)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(policy));
    return v;
}

// ---------------------------------------------------------------------------------------------
// Online softmax statistics relative to the raw maximum m: s = sum 2^((x - m) c)
// ---------------------------------------------------------------------------------------------
struct MaxSum {
    float m, s;
};

__device__ __forceinline__ MaxSum merge(MaxSum a, MaxSum b, float c)
{
    MaxSum r;
    r.m = fmaxf(a.m, b.m);
    r.s = a.s * ex2((a.m - r.m) * c) + b.s * ex2((b.m - r.m) * c);
    return r;
}

__device__ __forceinline__ MaxSum warp_merge(MaxSum v, float c)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MaxSum w;
        w.m = __shfl_xor_sync(0xFFFFFFFFu, v.m, o);
        w.s = __shfl_xor_sync(0xFFFFFFFFu, v.s, o);
        v = merge(v, w, c);
    }
    return v;
}

// Offsets and scale of the second sweep: min(p, q) = 2^min(ya, yb + lg) / sum_a = 2^min(ya - lg, yb) / sum_b with
// ya = (a - max_a) c, yb = (b - max_b) c, lg = log2(sum_a / sum_b).  lg is folded into the offset of the row whose
// reference is smaller in magnitude: added to a large offset it would be rounded at that offset's size (logits
// near +-300 would cost 1e-5 of every term).  out = {offset of the target row, offset of the draft row, scale}.
__device__ __forceinline__ void second_sweep_offsets(MaxSum a, MaxSum b, float c, float *out)
{
    const float lg = log2f(a.s / b.s);
    const bool on_a = fabsf(a.m) < fabsf(b.m);
    out[0] = on_a ? -a.m * c - lg : -a.m * c;
    out[1] = on_a ? -b.m * c : -b.m * c + lg;
    out[2] = 1.0f / (on_a ? b.s : a.s);
}

struct ArgMax {
    float v;
    int32_t i;
};

__device__ __forceinline__ ArgMax better(ArgMax a, ArgMax b)
{
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

__device__ __forceinline__ ArgMax warp_argmax(ArgMax a)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ArgMax b;
        b.v = __shfl_xor_sync(0xFFFFFFFFu, a.v, o);
        b.i = __shfl_xor_sync(0xFFFFFFFFu, a.i, o);
        a = better(a, b);
    }
    return a;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// ---------------------------------------------------------------------------------------------
// Thread-block clusters: identity, barrier, distributed shared memory
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_size()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_id()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
// Every thread of every CTA of the cluster arrives and waits; release/acquire at cluster scope.
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of that barrier on their own (every thread of every CTA of the cluster runs both, in this order).
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// Address of the same shared-memory variable in the CTA of the given cluster rank.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster(uint32_t addr, int32_t v)
{
    asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void st_cluster(uint32_t addr, double v)
{
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bulk asynchronous copy global -> this CTA's shared memory; both addresses and the size are
// multiples of 16 bytes.  Completion is signalled on the mbarrier as transferred bytes.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// 16 bytes from this CTA's shared memory.
__device__ __forceinline__ uint4 lds16(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// Programmatic dependent launch: lets the next kernel in the stream be set up while this grid still runs.  That
// kernel waits for this whole grid (griddepcontrol.wait) before it touches anything this one reads or writes.
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
// Warp-wide maximum in one instruction (sm_100a).
__device__ __forceinline__ float warp_max_f(float v)
{
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}

// ---------------------------------------------------------------------------------------------
// Bandit arithmetic in fp64 (Algorithm 2; Discounted UCB; Sliding-window UCB)
// ---------------------------------------------------------------------------------------------
// Position index of the random-number block that draws a randomised policy's arm.
#define METASD_SELECT_POSITION 0xFFFFFFFFu

// MetaSD-EXP3: p_t(i) = (1 - gamma) w_i / sum_j w_j + gamma / K.
__device__ inline double exp3_probability(int K, double gamma, const double *w, double sum, int i)
{
    return (1.0 - gamma) * (w[i] / sum) + gamma / (double)K;
}

// Arm of round t for the randomised policies: word 2 of the block (seed; sequence, t, METASD_SELECT_POSITION, 0).
// EXP3: inverse CDF in arm order over the 24-bit uniform; RAND: floor(uniform * K) in integers.
__device__ inline int random_select(int variant, int K, double gamma, int t, const double *w, uint64_t seed,
                                    uint32_t sequence)
{
    const uint4 words = round_words(seed, sequence, (uint32_t)t, METASD_SELECT_POSITION);
    if (variant == METASD_RAND) return (int)(((uint64_t)(words.z >> 8) * (uint64_t)K) >> 24);
    const double u = (double)(words.z >> 8) * (1.0 / 16777216.0);
    double sum = 0.0, cum = 0.0;
    for (int i = 0; i < K; ++i) sum += w[i];
    for (int i = 0; i < K; ++i) {
        cum += exp3_probability(K, gamma, w, sum, i);
        if (cum > u) return i;
    }
    return K - 1;
}

// Pure exploration-then-commit with Sequential Halving (the algorithm boxes of those names): one halving run over
// `budget` rounds, then the surviving drafter.  ceil(log2 K) phases; in a phase every member of the surviving set
// is played floor(budget / (members * phases)) times (at least once), members in index order, each in one block.
// sa: the current phase's reward sums; sb: membership of the surviving set (1 or 0).
struct HalvingPhase {
    int index, n_phases, first, members, pulls;   // index == n_phases: exploration is over
};
__device__ inline HalvingPhase halving_phase(int K, int budget, int t)
{
    HalvingPhase ph;
    ph.n_phases = K > 1 ? 32 - __clz(K - 1) : 0;
    ph.first = 0;
    ph.members = K;
    for (ph.index = 0; ph.index < ph.n_phases; ++ph.index) {
        ph.pulls = max(budget / (ph.members * ph.n_phases), 1);
        const int length = ph.pulls * ph.members;
        if (t - ph.first < length) return ph;
        ph.first += length;
        ph.members = (ph.members + 1) >> 1;
    }
    ph.pulls = 0;
    return ph;
}
__device__ inline int petc_select(int K, int budget, int t, const double *sb)
{
    const HalvingPhase ph = halving_phase(K, budget, t);
    int skip = ph.index < ph.n_phases ? (t - ph.first) / ph.pulls : 0;
    for (int i = 0; i < K; ++i)
        if (sb[i] > 0.0 && skip-- == 0) return i;
    return K - 1;
}
__device__ inline void petc_update(int K, int budget, int t, double *sa, double *sb, int a, double r)
{
    sa[a] += r;
    const HalvingPhase ph = halving_phase(K, budget, t);
    if (ph.index >= ph.n_phases || t + 1 != ph.first + ph.pulls * ph.members) return;
    // the round closed a phase: the better half stays (larger sum; the lower index on equal sums)
    uint32_t in = 0, out = 0;
    for (int i = 0; i < K; ++i)
        if (sb[i] > 0.0) in |= 1u << i;
    for (int c = (ph.members + 1) >> 1; c > 0; --c) {
        int best = -1;
        for (int i = 0; i < K; ++i)
            if (((in >> i) & 1u) && (best < 0 || sa[i] > sa[best])) best = i;
        in &= ~(1u << best);
        out |= 1u << best;
    }
    for (int i = 0; i < K; ++i) { sb[i] = (out >> i) & 1u ? 1.0 : 0.0; sa[i] = 0.0; }
}

// Arm for round t of one sequence.  sa/sb: this sequence's [K] statistics; wa/wr: its window.
__device__ inline int bandit_select(int variant, int K, double beta, double gamma, int tau, int t, const double *sa,
                                    const double *sb, const int32_t *wa, const double *wr, uint64_t seed,
                                    uint32_t sequence)
{
    if (variant == METASD_EXP3 || variant == METASD_RAND) return random_select(variant, K, gamma, t, sa, seed, sequence);
    if (variant == METASD_PETC) return petc_select(K, tau, t, sb);   // tau carries the exploration budget
    if (t < K) return t;  // initial sweep: every drafter once, in order
    double mu[16], n[16];
    if (variant == METASD_SWUCB) {
        for (int i = 0; i < K; ++i) { mu[i] = 0.0; n[i] = 0.0; }
        int first = t - tau > 0 ? t - tau : 0;
        for (int s = first; s < t; ++s) {  // oldest first
            int slot = s % tau;
            int i = wa[slot];
            mu[i] += wr[slot];
            n[i] += 1.0;
        }
        for (int i = 0; i < K; ++i)
            if (n[i] > 0.0) mu[i] /= n[i];
    } else if (variant == METASD_DUCB) {
        for (int i = 0; i < K; ++i) { n[i] = sb[i]; mu[i] = sa[i] / sb[i]; }
    } else {
        for (int i = 0; i < K; ++i) { mu[i] = sa[i]; n[i] = sb[i]; }
    }
    const double two_ln_t = 2.0 * log((double)t);
    int best = 0;
    double best_score = -INFINITY;
    for (int i = 0; i < K; ++i) {
        double score = n[i] > 0.0 ? mu[i] + beta * sqrt(two_ln_t / n[i]) : INFINITY;
        if (score > best_score) { best_score = score; best = i; }
    }
    return best;
}

// Folds reward r of arm a into the statistics and advances the round counter.
__device__ inline void bandit_update(int variant, int K, double gamma, int tau, int32_t *t, double *sa,
                                     double *sb, int32_t *wa, double *wr, int a, double r)
{
    if (variant == METASD_UCB) {
        double n = sb[a];
        sa[a] = (sa[a] * n + r) / (n + 1.0);
        sb[a] = n + 1.0;
    } else if (variant == METASD_DUCB) {
        for (int i = 0; i < K; ++i) { sa[i] *= gamma; sb[i] *= gamma; }
        sa[a] += r;
        sb[a] += 1.0;
    } else if (variant == METASD_EXP3) {
        // r_hat = r / p_t(a); w_a <- w_a exp(gamma r_hat / K); then all weights are divided by the largest one
        // (the probabilities do not change and nothing overflows)
        double sum = 0.0, top = 0.0;
        for (int i = 0; i < K; ++i) sum += sa[i];
        sa[a] *= exp(gamma * (r / exp3_probability(K, gamma, sa, sum, a)) / (double)K);
        for (int i = 0; i < K; ++i) top = sa[i] > top ? sa[i] : top;
        for (int i = 0; i < K; ++i) sa[i] /= top;
    } else if (variant == METASD_RAND) {
        // no statistics
    } else if (variant == METASD_PETC) {
        petc_update(K, tau, *t, sa, sb, a, r);
    } else {
        int slot = *t % tau;
        wa[slot] = a;
        wr[slot] = r;
    }
    *t = *t + 1;
}

// bandit_update followed by bandit_select for one sequence, by one whole warp: for the UCB family (Algorithm 2, its
// discounted and its sliding-window form) lane i holds arm i, so the fp64 divisions, square roots and the window
// scan of the K arms run side by side; the arithmetic per arm, the order of the window's additions and the
// lowest-index tie-break are those of the serial functions.  The other policies run on lane 0.  Returns the next arm
// (the same value in every lane) after storing it and the advanced round counter.
__device__ inline int warp_bandit_step(int variant, int K, double beta, double gamma, int tau, int32_t *t_ptr, int32_t *arm_ptr,
                                       double *sa, double *sb, int32_t *wa, double *wr, int a, double r, uint64_t seed,
                                       uint32_t sequence)
{
    const int lane = threadIdx.x & 31;
    const int t = *t_ptr;
    int next = 0;
    if (variant != METASD_UCB && variant != METASD_DUCB && variant != METASD_SWUCB) {
        if (lane == 0) {
            int32_t tt = t;
            bandit_update(variant, K, gamma, tau, &tt, sa, sb, wa, wr, a, r);
            next = bandit_select(variant, K, beta, gamma, tau, tt, sa, sb, wa, wr, seed, sequence);
            *t_ptr = tt;
            *arm_ptr = next;
        }
        return __shfl_sync(0xFFFFFFFFu, next, 0);
    }
    double a_i = 0.0, b_i = 0.0;
    if (variant == METASD_UCB) {
        if (lane < K) { a_i = sa[lane]; b_i = sb[lane]; }
        if (lane == a) {
            a_i = (a_i * b_i + r) / (b_i + 1.0);
            b_i = b_i + 1.0;
            sa[lane] = a_i;
            sb[lane] = b_i;
        }
    } else if (variant == METASD_DUCB) {
        if (lane < K) {
            a_i = sa[lane] * gamma;
            b_i = sb[lane] * gamma;
            if (lane == a) { a_i += r; b_i += 1.0; }
            sa[lane] = a_i;
            sb[lane] = b_i;
        }
    } else {
        if (lane == 0) {
            const int slot = t % tau;
            wa[slot] = a;
            wr[slot] = r;
        }
        __syncwarp();
    }
    const int t1 = t + 1;
    next = t1;   // initial sweep: every drafter once, in order
    if (t1 >= K) {
        double mu = 0.0, n = 0.0;
        if (variant == METASD_SWUCB) {
            if (lane < K) {
                const int first = t1 - tau > 0 ? t1 - tau : 0;
                for (int s = first; s < t1; ++s) {   // oldest first
                    const int slot = s % tau;
                    if (wa[slot] == lane) { mu += wr[slot]; n += 1.0; }
                }
                if (n > 0.0) mu /= n;
            }
        } else if (variant == METASD_DUCB) {
            n = b_i;
            mu = a_i / b_i;
        } else {
            mu = a_i;
            n = b_i;
        }
        const double two_ln_t = 2.0 * log((double)t1);
        double score = -INFINITY;
        if (lane < K) score = n > 0.0 ? mu + beta * sqrt(two_ln_t / n) : INFINITY;
        int best = lane;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double os = __shfl_xor_sync(0xFFFFFFFFu, score, o);
            const int ob = __shfl_xor_sync(0xFFFFFFFFu, best, o);
            if (os > score || (os == score && ob < best)) { score = os; best = ob; }
        }
        next = best;
    }
    if (lane == 0) {
        *t_ptr = t1;
        *arm_ptr = next;
    }
    return next;
}

}  // namespace metasd
