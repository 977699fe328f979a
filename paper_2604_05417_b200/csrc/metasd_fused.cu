// Fused cluster path of the MetaSD verify round: ONE persistent kernel per call.
//
// A thread-block cluster of C CTAs owns one sequence at a time and walks its k+1 positions in order.
// Every CTA owns a contiguous 1/C slice of each logit row.  The slices arrive in shared memory through
// a ring of bulk asynchronous copies (TMA, completion on an mbarrier) that runs several rows ahead of
// the arithmetic, so each logit is read from HBM exactly once.  A thread turns its logits into
// exponentials relative to its own maximum and keeps them in registers; the cluster exchanges
// (max, sum, arg-max) records through distributed shared memory, after which the same registers give
//   - sum_v min(p_v, q_v) = 1 - d_TV(p_j, q_j)                                (Definition 2, Eq. 4),
//   - the accept test u q(x) < p(x) of the drafted token                      (Algorithm 4, lines 7-8),
//   - at the first rejection (or at the bonus position) the inverse-CDF draw from max(0, p - q)
//     (or from p), a prefix search in token order across the cluster          (Algorithm 4, lines 11-12).
// Rank 0 of the cluster then writes the outputs, forms the reward and a warp updates the bandit and
// selects the next arm with one lane per drafter                             (Algorithm 2, lines 7-10).
//
// One exponential is evaluated per logit (the special-function pipe is the second roof of this path).
#include <limits.h>
#include <stdio.h>
#include <stdlib.h>

#include "metasd_device.cuh"

namespace metasd {

namespace {

constexpr int FUSED_MAX_THREADS = 512;
constexpr int FUSED_MAX_WARPS = FUSED_MAX_THREADS / 32;
constexpr int FUSED_MAX_CLUSTER = 16;
constexpr int FUSED_MAX_SLOTS = 8;
constexpr int FUSED_MAX_POS = 17;                 // k + 1 <= 17
constexpr int FUSED_SMEM_RESERVE = 12 * 1024;     // static shared memory + slack kept out of the ring
constexpr uint32_t WAIT_FAST_POLLS = 4096u;
constexpr uint32_t WAIT_SLOW_POLLS = 1u << 21;    // with a back-off of 128 ns each: a few tenths of a second

// ---------------------------------------------------------------------------------------------
// PTX wrappers: cluster identity and barrier, distributed shared memory, mbarrier, bulk copy
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
// 16 bytes into a peer CTA's shared memory; the peer's mbarrier counts them as transferred bytes.
__device__ __forceinline__ void st_async_16(uint32_t remote_addr, uint32_t remote_bar, uint32_t a, uint32_t b, uint32_t c,
                                            uint32_t d)
{
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(remote_addr), "r"(a), "r"(b), "r"(c), "r"(d), "r"(remote_bar)
                 : "memory");
}

// ---------------------------------------------------------------------------------------------
// Shared-memory state of one CTA (besides the ring)
// ---------------------------------------------------------------------------------------------
struct __align__(16) Exchange {   // (max, sum) of both rows and the first arg-max of the target row
    float max_a, sum_a, max_b, sum_b;
    int32_t idx_a;
    int32_t pad[3];
};
constexpr uint32_t EXCHANGE_BYTES = 32;

struct FusedShared {
    uint64_t full[FUSED_MAX_SLOTS];                      // one mbarrier per ring slot
    uint64_t xbar[2];                                    // arrival of the peers' records, by item parity
    Exchange exch[2][FUSED_MAX_CLUSTER];                 // [item parity][sender rank]
    Exchange wrec[2][FUSED_MAX_WARPS];                   // [item parity][warp]: the warps' records
    double tot[10 * FUSED_MAX_WARPS];                    // draw: weight of (vector index i, warp)
    double pre[10 * FUSED_MAX_WARPS];                    // draw: exclusive prefix of tot
    double cta_tot[FUSED_MAX_CLUSTER];                   // draw: weight of each CTA's slice
    double cta_min[16][FUSED_MAX_CLUSTER];               // rank 0: sum of min(p, q) per position and sender
    float pmin[16][FUSED_MAX_WARPS];                     // sum of min(p, q) per position and warp
    const void *table[16];                               // the drafter pointer table
    // header of the current sequence
    int32_t h_tok[16];
    float h_xa[16], h_xb[16], h_u[16], h_ud[FUSED_MAX_POS];
    int32_t h_t, h_arm;
    // per-position results of the current sequence
    int32_t r_acc[16];
    float r_px[16], r_qx[16];
    uint32_t r_rowflag[16];
    int32_t nstar, nlast, token;
    int32_t dead;       // a wait ran out: later waits do not spin again
};

struct FusedGeom {
    int32_t n_vec_row;   // 16-byte vectors per logit row
    int32_t n_vec_cta;   // vectors of a row owned by one CTA (the last ranks may own fewer)
    int32_t n_slot;      // ring slots
    int32_t slot_bytes;  // n_vec_cta * 16
};

// Waits for a phase of an mbarrier.  Bounded: after the limit the CTA is marked dead, the status word
// gets the time-out bit and every later wait returns at once, so all barriers stay matched, every CTA
// still sends its records and the kernel ends.
__device__ __forceinline__ void wait_bar(FusedShared &sh, uint64_t *bar, uint32_t parity, uint32_t *status)
{
    if (mbar_try_wait(bar, parity)) return;
    if (*(volatile int32_t *)&sh.dead) return;
    for (uint32_t it = 0; it < WAIT_FAST_POLLS + WAIT_SLOW_POLLS; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if (it >= WAIT_FAST_POLLS) __nanosleep(128);
    }
    *(volatile int32_t *)&sh.dead = 1;
    atomicOr(status, METASD_STATUS_TIMEOUT);
}

// Element q of a register array of pairs.
template <int N>
__device__ __forceinline__ float elem(const float2 (&a)[N], int q) { return (q & 1) ? a[q >> 1].y : a[q >> 1].x; }

// One row slice from shared memory into registers: e_q = 2^((x_q - m_t) c) with the thread's own
// maximum m_t, s_t = sum_q e_q.  Vector i of the thread is vector i * nthr + tid of the slice.
template <typename LT, int VPT>
__device__ __forceinline__ void load_row(const unsigned char *slot, int my_vecs, int tid, int nthr, float c,
                                         float2 (&e)[VPT * Logit<LT>::VEC / 2], float &m_t, float &s_t)
{
    constexpr int NP = VPT * Logit<LT>::VEC / 2;
    float m = METASD_NEG_BIG;
    if constexpr (sizeof(LT) == 2) {
        // every lane of a vector outside the slice reads as -inf: weight 0, never the maximum
        uint32_t w[NP];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = i * nthr + tid;
            uint4 raw = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
            if (v < my_vecs) raw = *reinterpret_cast<const uint4 *>(slot + (size_t)v * 16);
            w[4 * i] = raw.x; w[4 * i + 1] = raw.y; w[4 * i + 2] = raw.z; w[4 * i + 3] = raw.w;
        }
        // the maximum on the packed words, two logits per instruction
        __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162 *>(&w[0]);
#pragma unroll
        for (int n = 1; n < NP; ++n) m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&w[n]));
        m = fmaxf(m, fmaxf(__low2float(m2), __high2float(m2)));
#pragma unroll
        for (int n = 0; n < NP; ++n) e[n] = make_float2(__uint_as_float(w[n] << 16), __uint_as_float(w[n] & 0xFFFF0000u));
    } else {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int v = i * nthr + tid;
            uint4 raw = make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);
            if (v < my_vecs) raw = *reinterpret_cast<const uint4 *>(slot + (size_t)v * 16);
            e[2 * i] = make_float2(__uint_as_float(raw.x), __uint_as_float(raw.y));
            e[2 * i + 1] = make_float2(__uint_as_float(raw.z), __uint_as_float(raw.w));
            m = fmaxf(m, fmaxf(fmaxf(e[2 * i].x, e[2 * i].y), fmaxf(e[2 * i + 1].x, e[2 * i + 1].y)));
        }
    }
    const float nm = -m * c;
    const float2 cc = make_float2(c, c), nn = make_float2(nm, nm);
    float2 s2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int n = 0; n < NP; ++n) {
        const float2 y = __ffma2_rn(e[n], cc, nn);
        e[n] = make_float2(ex2(y.x), ex2(y.y));
        s2 = __fadd2_rn(s2, e[n]);
    }
    m_t = m;
    s_t = s2.x + s2.y;
}

// First index (in the row) of value m among this thread's logits of a slice, INT_MAX if absent.
template <typename LT, int VPT>
__device__ __forceinline__ int first_index_of(const unsigned char *slot, int my_vecs, int tid, int nthr, int vec0, float m)
{
    constexpr int VEC = Logit<LT>::VEC;
    int found = INT_MAX;
#pragma unroll
    for (int i = VPT - 1; i >= 0; --i) {
        const int v = i * nthr + tid;
        if (v < my_vecs) {
            float x[VEC];
            Logit<LT>::unpack(*reinterpret_cast<const uint4 *>(slot + (size_t)v * 16), x);
#pragma unroll
            for (int q = VEC - 1; q >= 0; --q)
                if (x[q] == m) found = (vec0 + v) * VEC + q;
        }
    }
    return found;
}

// Merges up to 32 records held one per lane (lanes >= n hold nothing): row maxima, row sums relative
// to them, the first arg-max of the target row, and each lane's own rescaling factors.
struct Merged {
    float Ma, Sa, Mb, Sb;
    int idx;
    float ta, tb;   // this lane's 2^((m_lane - M) c)
};
__device__ __forceinline__ Merged merge_records(const Exchange *rec, int n, int lane, float c)
{
    float ma = METASD_NEG_BIG, sa = 0.f, mb = METASD_NEG_BIG, sb = 0.f;
    int ia = INT_MAX;
    if (lane < n) {
        const Exchange x = rec[lane];
        ma = x.max_a; sa = x.sum_a; mb = x.max_b; sb = x.sum_b; ia = x.idx_a;
    }
    Merged r;
    r.Ma = warp_max_f(ma);
    r.Mb = warp_max_f(mb);
    r.ta = ex2((ma - r.Ma) * c);
    r.tb = ex2((mb - r.Mb) * c);
    r.Sa = warp_sum_f(sa * r.ta);
    r.Sb = warp_sum_f(sb * r.tb);
    r.idx = __reduce_min_sync(0xFFFFFFFFu, (lane < n && ma == r.Ma) ? ia : INT_MAX);
    return r;
}

// Weight of element q in the draw: mode 1 = max(0, p - q) (correction), mode 2 = p (bonus).
__device__ __forceinline__ float draw_weight(int mode, float ea, float fa, float eb, float fb)
{
    const float pv = ea * fa;
    return mode == 1 ? fmaxf(pv - eb * fb, 0.f) : pv;
}

// Inverse CDF in token order over one row (pair) that lives in the registers of the whole cluster:
// the smallest v with sum_{w <= v} weight_w > u * total.  Token order is (rank, vector i, thread, lane
// of the vector).  Totals and offsets are carried in fp64.  Returns false (for every thread of the
// cluster alike) when the row has no mass; otherwise the token lands in sh.token of rank 0.
template <int VPT, int VEC>
__device__ bool cluster_draw(FusedShared &sh, const float2 (&ea)[VPT * VEC / 2], const float2 (&eb)[VPT * VEC / 2], float fa,
                             float fb, int mode, float u, int rank, int csize, int vec0, int nthr)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nw = nthr >> 5, ne = VPT * nw;
    float vs[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        float s = 0.f;
#pragma unroll
        for (int q = 0; q < VEC; ++q) s += draw_weight(mode, elem(ea, i * VEC + q), fa, elem(eb, i * VEC + q), fb);
        vs[i] = s;
    }
    if (tid == 0) { sh.nstar = INT_MAX; sh.nlast = -1; }
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const double d = warp_sum((double)vs[i]);
        if (lane == 0) sh.tot[i * nw + warp] = d;
    }
    __syncthreads();
    if (warp == 0) {
        // exclusive prefix over the ne entries, `per` consecutive entries per lane
        const int per = (ne + 31) >> 5;
        double loc[5], sum = 0.0;
#pragma unroll
        for (int q = 0; q < 5; ++q) {
            const int n = lane * per + q;
            loc[q] = (q < per && n < ne) ? sh.tot[n] : 0.0;
            sum += loc[q];
        }
        double incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        double run = incl - sum;
#pragma unroll
        for (int q = 0; q < 5; ++q) {
            const int n = lane * per + q;
            if (q < per && n < ne) { sh.pre[n] = run; run += loc[q]; }
        }
        const double total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        if (lane < csize) st_cluster(map_to_rank(smem_addr(&sh.cta_tot[rank]), lane), total);
    }
    cluster_sync_all();
    double R = 0.0, mybase = 0.0;
    int rlast = -1;
    for (int r = 0; r < csize; ++r) {
        const double t = sh.cta_tot[r];
        if (r == rank) mybase = R;
        if (t > 0.0) rlast = r;
        R += t;
    }
    if (!(R > 0.0)) return false;
    const double thr = (double)u * R;
    int rstar = -1;
    {
        double run = 0.0;
        for (int r = 0; r < csize; ++r) {
            const double t = sh.cta_tot[r];
            if (rstar < 0 && run + t > thr) rstar = r;
            run += t;
        }
    }
    if (rstar < 0) rstar = rlast;   // rounding left the total a hair under the threshold
    if (rank == rstar) {
        const double th = thr - mybase;
        if (tid < ne) {
            const double t = sh.tot[tid];
            if (t > 0.0) atomicMax(&sh.nlast, tid);
            if (sh.pre[tid] + t > th) atomicMin(&sh.nstar, tid);
        }
        __syncthreads();
        const int n = sh.nstar != INT_MAX ? sh.nstar : sh.nlast;
        const int istar = n / nw, wstar = n - istar * nw;
        if (warp == wstar) {
            float v = 0.f;
#pragma unroll
            for (int i = 0; i < VPT; ++i)
                if (i == istar) v = vs[i];
            const double dv = (double)v;
            double incl = dv;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            const double pre = sh.pre[n];
            const unsigned crossing = __ballot_sync(0xFFFFFFFFu, pre + incl > th);
            const unsigned mass = __ballot_sync(0xFFFFFFFFu, v > 0.f);
            const int src = crossing ? __ffs(crossing) - 1 : (mass ? 31 - __clz(mass) : 0);
            if (lane == src) {
                double cum = pre + incl - dv;
                int tok_q = -1, last_q = -1;
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    if (i == istar) {
#pragma unroll
                        for (int q = 0; q < VEC; ++q) {
                            const float w = draw_weight(mode, elem(ea, i * VEC + q), fa, elem(eb, i * VEC + q), fb);
                            cum += (double)w;
                            if (w > 0.f) last_q = q;
                            if (tok_q < 0 && cum > th) tok_q = q;
                        }
                    }
                }
                if (tok_q < 0) tok_q = last_q;
                const int token = tok_q < 0 ? -1 : (vec0 + istar * nthr + tid) * VEC + tok_q;
                st_cluster(map_to_rank(smem_addr(&sh.token), 0), (int32_t)token);
            }
        }
    }
    return true;
}

// Bandit update and next selection by one warp, lane i = drafter i (Algorithm 2 lines 7-10; Discounted
// UCB; Sliding-window UCB).  Same fp64 expressions as the one-thread routines in metasd_device.cuh.
__device__ void warp_bandit(const VerifyParams &p, int b, int t, int arm, double r)
{
    const int lane = threadIdx.x & 31;
    const int K = p.K, tau = p.tau;
    double *sa = p.st.stat_a + (size_t)b * K, *sb = p.st.stat_b + (size_t)b * K;
    int32_t *wa = p.st.win_arm + (size_t)b * tau;
    double *wr = p.st.win_reward + (size_t)b * tau;
    double a_i = 0.0, b_i = 0.0;
    if (lane < K) { a_i = sa[lane]; b_i = sb[lane]; }
    if (p.bandit == METASD_UCB) {
        if (lane == arm) {
            const double n = b_i;
            a_i = (a_i * n + r) / (n + 1.0);
            b_i = n + 1.0;
            sa[lane] = a_i; sb[lane] = b_i;
        }
    } else if (p.bandit == METASD_DUCB) {
        a_i *= p.gamma; b_i *= p.gamma;
        if (lane == arm) { a_i += r; b_i += 1.0; }
        if (lane < K) { sa[lane] = a_i; sb[lane] = b_i; }
    } else if (lane == 0) {
        const int slot = t % tau;
        wa[slot] = arm;
        wr[slot] = r;
    }
    __syncwarp();
    const int t1 = t + 1;
    int next = t1;   // initial sweep: every drafter once, in order
    if (t1 >= K) {
        double mu = 0.0, n = 0.0;
        if (p.bandit == METASD_SWUCB) {
            if (lane < K) {
                const int first = t1 - tau > 0 ? t1 - tau : 0;
                for (int s = first; s < t1; ++s) {   // oldest first
                    const int slot = s % tau;
                    if (wa[slot] == lane) { mu += wr[slot]; n += 1.0; }
                }
                if (n > 0.0) mu /= n;
            }
        } else if (p.bandit == METASD_DUCB) {
            n = b_i; mu = a_i / b_i;
        } else {
            mu = a_i; n = b_i;
        }
        const double two_ln_t = 2.0 * log((double)t1);
        double score = -INFINITY;
        if (lane < K) score = n > 0.0 ? mu + p.beta * sqrt(two_ln_t / n) : INFINITY;
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
        p.st.t[b] = t1;
        p.st.arm[b] = next;
    }
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <typename LT, int VPT>
__global__ void __launch_bounds__(FUSED_MAX_THREADS, 1) fused_round_kernel(const VerifyParams p, const FusedGeom g)
{
    constexpr int VEC = Logit<LT>::VEC;
    constexpr int NP = VPT * VEC / 2;
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ FusedShared sh;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthr = blockDim.x, nw = nthr >> 5;
    const int rank = (int)cluster_rank(), csize = (int)cluster_size();
    const int cid = (int)cluster_id(), ncl = (int)cluster_count();
    const int k = p.k, V = p.V;
    const float c = p.c;
    const size_t row_bytes = (size_t)V * sizeof(LT);
    const int vec0 = rank * g.n_vec_cta;
    const int my_vecs = max(0, min(g.n_vec_cta, g.n_vec_row - vec0));
    const uint32_t my_bytes = (uint32_t)my_vecs * 16u;

    if (tid == 0) {
        for (int s = 0; s < g.n_slot; ++s) mbar_init(&sh.full[s], 1);
        mbar_init(&sh.xbar[0], 1);
        mbar_init(&sh.xbar[1], 1);
        sh.dead = 0;
        sh.token = -1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 16) sh.table[tid] = (p.drafter_ptrs && tid < p.K) ? p.drafter_ptrs[tid] : nullptr;
    cluster_sync_all();   // every CTA of the cluster is running, its barriers initialised, before a peer writes to it

    // ---- producer (thread 0): the order of loads is sequence-major, position, target then draft
    int ld_b = cid, ld_j = 0, ld_row = 0, ld_slot = 0, ld_arm_next = 0;
    uint32_t ld_issued = 0, consumed = 0;
    const unsigned char *ld_draft = nullptr;
    auto draft_base = [&](int arm) -> const unsigned char * {
        return reinterpret_cast<const unsigned char *>(p.draft ? p.draft : sh.table[arm & 15]);
    };
    auto issue_one = [&]() {
        if (ld_b >= p.batch || *(volatile int32_t *)&sh.dead) return;   // after a time-out nothing more is armed
        const unsigned char *base = ld_row == 0 ? reinterpret_cast<const unsigned char *>(p.target) : ld_draft;
        const unsigned char *src =
            base + (ld_row == 0 ? ((size_t)ld_b * (k + 1) + ld_j) : ((size_t)ld_b * k + ld_j)) * row_bytes + (size_t)vec0 * 16;
        uint64_t *bar = &sh.full[ld_slot];
        if (my_bytes == 0) {
            mbar_arrive(bar);
        } else if (base == nullptr || (reinterpret_cast<uintptr_t>(src) & 15u) != 0) {
            atomicOr(p.status, METASD_STATUS_BAD_POINTER);   // never hand a misaligned address to the copy engine
            mbar_arrive(bar);
        } else {
            mbar_arrive_expect_tx(bar, my_bytes);
            bulk_load(ring + (size_t)ld_slot * g.slot_bytes, src, my_bytes, bar);
        }
        ++ld_issued;
        ld_slot = ld_slot + 1 == g.n_slot ? 0 : ld_slot + 1;
        if (ld_row == 0 && ld_j < k) {
            ld_row = 1;
        } else {
            ld_row = 0;
            if (++ld_j > k) {
                ld_j = 0;
                ld_b += ncl;
                if (ld_b < p.batch) {
                    ld_draft = draft_base(ld_arm_next);
                    if (!p.draft && ld_b + ncl < p.batch) ld_arm_next = p.st.arm[ld_b + ncl];
                }
            }
        }
    };
    if (tid == 0 && cid < p.batch) {
        ld_draft = draft_base(p.draft ? 0 : p.st.arm[cid]);
        if (!p.draft && cid + ncl < p.batch) ld_arm_next = p.st.arm[cid + ncl];
        for (int s = 0; s < g.n_slot; ++s) issue_one();
    }

    // ---- header of a sequence (warp 0, lane j = position j): round counter, arm, drafted token and
    // its two logits.  Fetched one sequence ahead, in three steps spread over the item loop.
    int nx_t = 0, nx_arm = 0, nx_tok = -1;
    float nx_xa = 0.f, nx_xb = 0.f;
    auto fetch_step = [&](int b, int step) {
        if (step == 0) {
            nx_t = p.st.t[b];
            nx_arm = p.st.arm[b];
        } else if (step == 1) {
            nx_tok = -1;
            if (lane < k) {
                const int32_t *tokens = p.tokens + (p.token_arm_stride ? (size_t)nx_arm * p.token_arm_stride : 0) + (size_t)b * k;
                nx_tok = tokens[lane];
            }
        } else {
            nx_xa = 0.f; nx_xb = 0.f;
            if (lane < k && nx_tok >= 0 && nx_tok < V) {
                const LT *ta = reinterpret_cast<const LT *>(p.target) + ((size_t)b * (k + 1) + lane) * V;
                const LT *td = reinterpret_cast<const LT *>(draft_base(nx_arm));
                nx_xa = Logit<LT>::scalar(ta, nx_tok);
                if (td) nx_xb = Logit<LT>::scalar(td + ((size_t)b * k + lane) * V, nx_tok);
            }
        }
    };
    if (warp == 0 && cid < p.batch) {
        fetch_step(cid, 0);
        fetch_step(cid, 1);
        fetch_step(cid, 2);
    }

    int cs = 0;              // ring slot the consumers read next
    uint32_t cpar = 0;       // and its phase parity
    uint32_t item = 0;       // items done by this cluster: bit 0 selects the exchange buffers, bit 1 their phase

    for (int b = cid; b < p.batch; b += ncl) {
        // ---- publish the header of sequence b
        if (warp == 0) {
            if (lane == 0) { sh.h_t = nx_t; sh.h_arm = nx_arm; }
            if (lane <= k) {
                const uint4 w = round_words(p.seed, p.sequence_base + (uint32_t)b, (uint32_t)nx_t, (uint32_t)lane);
                sh.h_ud[lane] = uniform24(w.y);
                if (lane < k) {
                    sh.h_u[lane] = uniform24(w.x);
                    sh.h_tok[lane] = nx_tok;
                    sh.h_xa[lane] = nx_xa;
                    sh.h_xb[lane] = nx_xb;
                }
            }
        }
        const int b_next = b + ncl;
        int n_acc = -1;          // undecided
        int token = -1;
        bool drew = false;       // the token sits in sh.token of rank 0
        uint32_t seq_flags = 0;

        for (int j = 0; j <= k; ++j, ++item) {
            const bool pair = j < k;
            const int par = item & 1;
            if (warp == 0) {
                if (b_next < p.batch) {
                    if (j == 0) fetch_step(b_next, 0);
                    if (j == 1) fetch_step(b_next, 1);
                    if (j == (k < 2 ? k : 2)) fetch_step(b_next, 2);
                }
                // expect one record of 32 bytes from every CTA of the cluster (this one included)
                if (lane == 0 && !*(volatile int32_t *)&sh.dead)
                    mbar_arrive_expect_tx(&sh.xbar[par], (uint32_t)csize * EXCHANGE_BYTES);
            }

            // ---- this item's slices: shared memory -> registers, exponentials relative to the thread maximum,
            //      then the warp's record: maxima, sums relative to them, first arg-max of the target row
            float2 ea[NP], eb[NP];
            float mta, mtb = METASD_NEG_BIG;
            Exchange wr;
            {
                float sta;
                const unsigned char *slot = ring + (size_t)cs * g.slot_bytes;
                wait_bar(sh, &sh.full[cs], cpar, p.status);
                load_row<LT, VPT>(slot, my_vecs, tid, nthr, c, ea, mta, sta);
                if (++cs == g.n_slot) { cs = 0; cpar ^= 1u; }
                wr.max_a = warp_max_f(mta);
                wr.sum_a = warp_sum_f(sta * ex2((mta - wr.max_a) * c));
                int cand = INT_MAX;
                if (p.greedy && mta == wr.max_a && mta > METASD_NEG_BIG)
                    cand = first_index_of<LT, VPT>(slot, my_vecs, tid, nthr, vec0, mta);
                wr.idx_a = p.greedy ? __reduce_min_sync(0xFFFFFFFFu, cand) : INT_MAX;
            }
            if (pair) {
                float stb;
                wait_bar(sh, &sh.full[cs], cpar, p.status);
                load_row<LT, VPT>(ring + (size_t)cs * g.slot_bytes, my_vecs, tid, nthr, c, eb, mtb, stb);
                if (++cs == g.n_slot) { cs = 0; cpar ^= 1u; }
                wr.max_b = warp_max_f(mtb);
                wr.sum_b = warp_sum_f(stb * ex2((mtb - wr.max_b) * c));
            } else {
#pragma unroll
                for (int n = 0; n < NP; ++n) eb[n] = make_float2(0.f, 0.f);
                wr.max_b = METASD_NEG_BIG;
                wr.sum_b = 0.f;
            }
            if (lane == 0) {
                wr.pad[0] = wr.pad[1] = wr.pad[2] = 0;
                sh.wrec[par][warp] = wr;
            }
            __syncthreads();

            // ---- the slots of this item are free: refill them
            if (tid == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                consumed += pair ? 2u : 1u;
                issue_one();
                if (pair) issue_one();
            }
            // ---- the CTA's record goes to every CTA of the cluster (asynchronous stores that complete on
            //      the receiver's barrier); then wait for all the records addressed to this CTA
            if (warp == 0) {
                const Merged mc = merge_records(sh.wrec[par], nw, lane, c);
                if (lane < csize) {
                    const uint32_t dst = map_to_rank(smem_addr(&sh.exch[par][rank]), (uint32_t)lane);
                    const uint32_t bar = map_to_rank(smem_addr(&sh.xbar[par]), (uint32_t)lane);
                    st_async_16(dst, bar, __float_as_uint(mc.Ma), __float_as_uint(mc.Sa), __float_as_uint(mc.Mb),
                                __float_as_uint(mc.Sb));
                    st_async_16(dst + 16, bar, (uint32_t)mc.idx, 0u, 0u, 0u);
                }
            }
            wait_bar(sh, &sh.xbar[par], (item >> 1) & 1u, p.status);
            const Merged mg = merge_records(sh.exch[par], csize, lane, c);
            const float Ma = mg.Ma, Sa = mg.Sa, Mb = mg.Mb, Sb = mg.Sb;
            const int argidx = mg.idx;

            // NaN or +Inf anywhere makes the sum NaN; an all -Inf row leaves it 0
            const bool bad_a = !(Sa > 0.f) || !(Sa < INFINITY) || !(Ma < INFINITY);
            const bool bad_b = pair && (!(Sb > 0.f) || !(Sb < INFINITY) || !(Mb < INFINITY));
            const uint32_t rowflag = (bad_a || bad_b) ? METASD_STATUS_NONFINITE : 0u;
            // p_v = e_v * fa with fa = 2^((m_t - M) c) / S
            const float fa = rowflag ? 0.f : ex2((mta - Ma) * c) / Sa;
            const float fb = (rowflag || !pair) ? 0.f : ex2((mtb - Mb) * c) / Sb;

            // ---- sum_v min(p_v, q_v) of this warp's logits
            bool accepted = false;
            if (pair) {
                float2 acc2 = make_float2(0.f, 0.f);
                const float2 fa2 = make_float2(fa, fa), fb2 = make_float2(fb, fb);
#pragma unroll
                for (int n = 0; n < NP; ++n) {
                    const float2 pv = __fmul2_rn(ea[n], fa2), qv = __fmul2_rn(eb[n], fb2);
                    acc2 = __fadd2_rn(acc2, make_float2(fminf(pv.x, qv.x), fminf(pv.y, qv.y)));
                }
                const float acc = warp_sum_f(acc2.x + acc2.y);
                if (lane == 0) sh.pmin[j][warp] = acc;

                // ---- the accept test of Algorithm 4 (lines 7-8), evaluated alike by every thread of the cluster
                const int x = sh.h_tok[j];
                float p_x = 0.f, q_x = 0.f;
                uint32_t fl = rowflag;
                if (!rowflag) {
                    if (x < 0 || x >= V) {
                        fl |= METASD_STATUS_TOKEN_OOR;
                    } else {
                        p_x = ex2(fmaf(sh.h_xa[j], c, -Ma * c)) / Sa;
                        q_x = ex2(fmaf(sh.h_xb[j], c, -Mb * c)) / Sb;
                        if (p.greedy) {
                            accepted = x == argidx;
                        } else {
                            if (q_x == 0.f) fl |= METASD_STATUS_Q_ZERO;
                            accepted = sh.h_u[j] * q_x < p_x;   // u < min(1, p/q) without the division
                        }
                    }
                }
                seq_flags |= fl;
                if (tid == 0) {
                    sh.r_acc[j] = accepted ? 1 : 0;
                    sh.r_px[j] = p_x;
                    sh.r_qx[j] = q_x;
                    sh.r_rowflag[j] = rowflag;
                }
            }

            // ---- first rejection (Algorithm 4, "exit for loop") or the bonus position: emit the next token
            int mode = 0;
            if (n_acc < 0) {
                if (pair && !accepted) { n_acc = j; mode = 1; }
                if (!pair) { n_acc = k; mode = 2; seq_flags |= rowflag; }
                if (mode) {
                    if (rowflag) {
                        mode = 0;
                    } else if (p.greedy) {
                        token = argidx;
                        mode = 0;
                    }
                }
            }
            if (mode) {
                const float u = sh.h_ud[j];
                bool ok = cluster_draw<VPT, VEC>(sh, ea, eb, fa, fb, mode, u, rank, csize, vec0, nthr);
                if (!ok && mode == 1)   // p == q in fp32 yet rejected: draw from p
                    ok = cluster_draw<VPT, VEC>(sh, ea, eb, fa, fb, 2, u, rank, csize, vec0, nthr);
                drew = ok;
            }
        }

        // ---- end of the sequence: gather sum_v min(p, q) per position in rank 0
        __syncthreads();
        if (warp == 0 && lane < k) {
            double s = 0.0;
            for (int w = 0; w < nw; ++w) s += (double)sh.pmin[lane][w];
            st_cluster(map_to_rank(smem_addr(&sh.cta_min[lane][rank]), 0), s);
        }
        cluster_sync_all();
        if (rank == 0 && warp == 0) {
            double smin = 0.0;
            uint32_t rf = 0;
            if (lane < k) {
                for (int r = 0; r < csize; ++r) smin += sh.cta_min[lane][r];
                rf = sh.r_rowflag[lane];
                if (rf) smin = 0.0;
            }
            double sum_align = 0.0;
            for (int j = 0; j < k; ++j) sum_align += __shfl_sync(0xFFFFFFFFu, smin, j);
            // Definition 2: 1 - mean_j d_TV; block efficiency: N_acc / N_max
            const double r = p.reward_kind == METASD_REWARD_BE ? (double)n_acc / (double)k : sum_align / (double)k;
            if (p.diag && lane < k) {
                metasd_diag dg;
                dg.p_x = sh.r_px[lane];
                dg.q_x = sh.r_qx[lane];
                dg.D = rf ? 1.f : (float)(1.0 - smin);
                dg.u = sh.h_u[lane];
                dg.accept = sh.r_acc[lane];
                p.diag[(size_t)b * k + lane] = dg;
            }
            if (lane == 0) {
                p.accepted_len[b] = n_acc;
                p.next_token[b] = drew ? sh.token : token;
                p.reward[b] = (float)r;
                if (seq_flags) atomicOr(p.status, seq_flags);
            }
            warp_bandit(p, b, sh.h_t, sh.h_arm, r);
        }
    }

    // ---- no CTA leaves while a copy into its shared memory may be in flight or a peer may still write to it
    if (tid == 0) {
        while (consumed < ld_issued) {
            wait_bar(sh, &sh.full[cs], cpar, p.status);
            if (++cs == g.n_slot) { cs = 0; cpar ^= 1u; }
            ++consumed;
        }
    }
    cluster_sync_all();
}

// ---------------------------------------------------------------------------------------------
// Host side: geometry, occupancy, launch
// ---------------------------------------------------------------------------------------------
template <typename LT, int VPT>
const void *kernel_ptr() { return reinterpret_cast<const void *>(&fused_round_kernel<LT, VPT>); }

const void *kernel_for(int dtype)
{
    return dtype == METASD_BF16 ? kernel_ptr<__nv_bfloat16, 5>() : kernel_ptr<float, 10>();
}

int vectors_per_thread_max(int dtype) { return dtype == METASD_BF16 ? 5 : 10; }

// Geometry for cluster size C, or false when the row does not fit.
bool geometry(int dtype, int V, int C, int smem_optin, FusedPlan *pl)
{
    const size_t row_bytes = (size_t)V * (dtype == METASD_BF16 ? 2 : 4);
    if (row_bytes % 16 != 0) return false;
    const int n_vec_row = (int)(row_bytes / 16);
    if (C > n_vec_row) return false;
    const int n_vec_cta = (n_vec_row + C - 1) / C;
    if ((size_t)(C - 1) * n_vec_cta >= (size_t)n_vec_row) return false;   // an empty last rank: a smaller C serves better
    const int vpt_max = vectors_per_thread_max(dtype);
    if (n_vec_cta > FUSED_MAX_THREADS * vpt_max) return false;
    // threads: the multiple of 32 with the least padding, the larger one on ties
    int best_t = 0;
    long best_cost = 0;
    for (int t = FUSED_MAX_THREADS; t >= 64; t -= 32) {
        const int vpt = (n_vec_cta + t - 1) / t;
        if (vpt > vpt_max) break;
        const long cost = (long)t * vpt;
        if (!best_t || cost < best_cost) { best_t = t; best_cost = cost; }
    }
    if (!best_t) return false;
    const int slot_bytes = n_vec_cta * 16;
    int n_slot = (smem_optin - FUSED_SMEM_RESERVE) / slot_bytes;
    if (n_slot > FUSED_MAX_SLOTS) n_slot = FUSED_MAX_SLOTS;
    if (n_slot < 3) return false;
    pl->cluster = C;
    pl->threads = best_t;
    pl->n_vec_row = n_vec_row;
    pl->n_vec_cta = n_vec_cta;
    pl->n_slot = n_slot;
    pl->slot_bytes = slot_bytes;
    pl->smem_bytes = (size_t)n_slot * slot_bytes;
    pl->work_per_item = best_cost;
    pl->max_clusters = 0;
    return true;
}

int env_int(const char *name, int fallback)
{
    const char *s = getenv(name);
    return s && *s ? atoi(s) : fallback;
}

}  // namespace

bool fused_supported(int dtype, int V, int k)
{
    if (k < 1 || k > 16) return false;
    FusedPlan pl;
    for (int C = 1; C <= FUSED_MAX_CLUSTER; ++C)
        if (geometry(dtype, V, C, 227 * 1024, &pl)) return true;
    return false;
}

// Chooses the cluster size for this device: for every size that fits, ask the occupancy calculator how
// many clusters are co-resident (GPC shapes decide) and take the least estimated time for a full batch.
// METASD_FUSED_CLUSTER / METASD_FUSED_THREADS (environment) pin the choice for tuning runs.
cudaError_t fused_prepare(int device, int dtype, int V, int max_batch, FusedPlan *plan)
{
    plan->cluster = 0;
    int smem_optin = 0;
    cudaError_t e = cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e != cudaSuccess) return e;
    const void *fn = kernel_for(dtype);
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin - FUSED_SMEM_RESERVE);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    const int pin_c = env_int("METASD_FUSED_CLUSTER", 0), pin_t = env_int("METASD_FUSED_THREADS", 0);
    double best = 0.0;
    for (int C = 1; C <= FUSED_MAX_CLUSTER; ++C) {
        if (pin_c && C != pin_c) continue;
        FusedPlan pl;
        if (!geometry(dtype, V, C, smem_optin, &pl)) continue;
        if (pin_t >= 64 && pin_t <= FUSED_MAX_THREADS && pin_t % 32 == 0 &&
            (pl.n_vec_cta + pin_t - 1) / pin_t <= vectors_per_thread_max(dtype)) {
            pl.threads = pin_t;
            pl.work_per_item = (long)pin_t * ((pl.n_vec_cta + pin_t - 1) / pin_t);
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(C);
        cfg.blockDim = dim3(pl.threads);
        cfg.dynamicSmemBytes = pl.smem_bytes;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeClusterDimension;
        at.val.clusterDim.x = C; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, fn, &cfg) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            continue;
        }
        pl.max_clusters = n;
        const int used = n < max_batch ? n : max_batch;
        const double waves = (double)((max_batch + used - 1) / used);
        // per item: the arithmetic of the slice plus a fixed cost for its barriers and exchanges
        const double cost = waves * ((double)pl.work_per_item + 400.0);
        if (!plan->cluster || cost < best) { *plan = pl; best = cost; }
    }
    if (plan->cluster && env_int("METASD_FUSED_VERBOSE", 0))
        fprintf(stderr, "metasd fused plan: V=%d cluster=%d threads=%d vectors/cta=%d slots=%d x %d B, %d clusters co-resident\n",
                V, plan->cluster, plan->threads, plan->n_vec_cta, plan->n_slot, plan->slot_bytes, plan->max_clusters);
    return plan->cluster ? cudaSuccess : cudaErrorNotSupported;
}

cudaError_t launch_fused(const VerifyParams &p, int dtype, const FusedPlan &plan, cudaStream_t stream, uint64_t *launches)
{
    FusedGeom g;
    g.n_vec_row = plan.n_vec_row;
    g.n_vec_cta = plan.n_vec_cta;
    g.n_slot = plan.n_slot;
    g.slot_bytes = plan.slot_bytes;
    const int n_clusters = p.batch < plan.max_clusters ? p.batch : plan.max_clusters;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_clusters * plan.cluster));
    cfg.blockDim = dim3((unsigned)plan.threads);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeClusterDimension;
    at.val.clusterDim.x = (unsigned)plan.cluster; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
    cfg.attrs = &at;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (dtype == METASD_BF16)
        e = cudaLaunchKernelEx(&cfg, fused_round_kernel<__nv_bfloat16, 5>, p, g);
    else
        e = cudaLaunchKernelEx(&cfg, fused_round_kernel<float, 10>, p, g);
    *launches += 1;
    return e;
}

}  // namespace metasd
