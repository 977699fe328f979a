// Fused cluster path of the MetaSD verify round: ONE persistent kernel per call.
//
// A thread-block cluster of C CTAs owns one sequence at a time and walks its k+1 positions in order.
// Every CTA owns a contiguous 1/C slice of each logit row.  The slices arrive in shared memory through
// a ring of bulk asynchronous copies (TMA, completion on an mbarrier) that runs ahead of the arithmetic,
// so each logit is read from HBM exactly once and stays on chip for both passes over it:
//
//   pass 1 (row statistics)  per row: running maximum and sum_v 2^((x_v - max) c); the CTA's record
//                            (max, sum, first arg-max) goes to every CTA of the cluster as asynchronous
//                            distributed-shared-memory stores that complete on the receiver's mbarrier;
//   pass 2 (one item later)  with the merged records of the whole row pair:
//                              sum_v min(p_v, q_v) = 1 - d_TV(p_j, q_j)            (Definition 2, Eq. 4)
//                            evaluated as sum_v 2^min(log2 p_v, log2 q_v): one exponential per PAIR;
//                            the accept test u q(x) < p(x) of the drafted token     (Algorithm 4, l. 7-8);
//                            at the first rejection (or the bonus position) the inverse-CDF draw from
//                            max(0, p - q) (or p), a prefix search in token order across the cluster
//                                                                                    (Algorithm 4, l. 11-12).
//
// Pass 2 of item n-1 runs after pass 1 of item n, so the latency of the record exchange hides behind a
// full pass.  Warp 0 of every CTA is a control warp (lane j = position j of the sequence): it issues the
// copies, merges and sends records, runs the accept tests, and in rank 0 writes the outputs, forms the
// reward and updates the bandit with one lane per drafter (Algorithm 2, lines 7-10).  The other warps
// only stream logits out of shared memory.
#include <limits.h>
#include <stdio.h>
#include <stdlib.h>

#include "metasd_device.cuh"

namespace metasd {

namespace {

constexpr int FUSED_MAX_THREADS = 1024;
constexpr int FUSED_MAX_WARPS = FUSED_MAX_THREADS / 32;
constexpr int FUSED_MAX_CLUSTER = 16;
constexpr int FUSED_MAX_SLOTS = 8;
constexpr int FUSED_MIN_SLOTS = 5;                // two items of two rows each, plus one copy in flight
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

// What the control warp hands to the streaming warps for pass 2 of one item.
struct RowConst {
    float nma, nmb;      // -max c of the target / draft row
    float nmb_rel;       // nmb + log2(sum_a / sum_b): the draft row on the target row's scale
    float inv_sa, inv_sb;
    float u_draw;        // uniform of the residual / bonus draw
    int32_t mode;        // 0 none, 1 draw from max(0, p - q), 2 draw from p
    int32_t valid;       // 0: the row pair is flagged non-finite, its sum of minima is 0
};

struct FusedShared {
    uint64_t full[FUSED_MAX_SLOTS];                      // one mbarrier per ring slot
    uint64_t xbar[3];                                    // arrival of the peers' records, by item mod 3
    uint64_t wbar[2];                                    // the streaming warps' records are written, by step parity
    uint64_t rcbar[2];                                   // pass 2's row constants are written, by item parity
    uint64_t ebar[2];                                    // the streaming warps are done with pass 2's slots, by item parity
    Exchange exch[3][FUSED_MAX_CLUSTER];                 // [item mod 3][sender rank]
    Exchange wrec[2][FUSED_MAX_WARPS];                   // the streaming warps' records of the item in pass 1
    RowConst rc[2];
    double tot[FUSED_MAX_WARPS];                         // draw: weight of each streaming warp's range
    double pre[FUSED_MAX_WARPS];                         // draw: exclusive prefix of tot
    double cta_tot[FUSED_MAX_CLUSTER];                   // draw: weight of each CTA's slice
    double cta_min[16][FUSED_MAX_CLUSTER];               // rank 0: sum of min(p, q) per position and sender
    float pmin[16][FUSED_MAX_WARPS];                     // sum of min(p, q) per position and streaming warp
    const void *table[16];                               // the drafter pointer table
    int32_t token;                                       // rank 0: the drawn token
    int32_t dead;                                        // a wait ran out: later waits do not spin again
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

// Largest of the 16 bytes of logits (NaN entries are ignored).
template <typename LT>
__device__ __forceinline__ float vector_max(const uint4 &raw)
{
    if constexpr (sizeof(LT) == 2) {
        const __nv_bfloat162 *w = reinterpret_cast<const __nv_bfloat162 *>(&raw);
        const __nv_bfloat162 m2 = __hmax2(__hmax2(w[0], w[1]), __hmax2(w[2], w[3]));   // two logits per instruction
        return fmaxf(__low2float(m2), __high2float(m2));
    } else {
        return fmaxf(fmaxf(__uint_as_float(raw.x), __uint_as_float(raw.y)), fmaxf(__uint_as_float(raw.z), __uint_as_float(raw.w)));
    }
}

// Pass 1 over one item's row slices in shared memory, by one warp: running maxima shared by the whole
// warp (so that the rare rescaling branch never diverges), sums 2^((x - max) c) per lane, and per lane the
// vector in which it first met the target row's maximum.  Thread ct of ncomp takes vectors ct, ct + ncomp, ...;
// every lane makes the same number of trips, a vector beyond the slice reads as -inf.
template <typename LT, bool PAIR>
__device__ __forceinline__ void stats_rows(const unsigned char *slot_a, const unsigned char *slot_b, int my_vecs, int ct,
                                           int ncomp, int trips, float c, bool want_argmax, float &max_a, float &sum_a,
                                           int &vec_a, float &max_b, float &sum_b)
{
    constexpr int VEC = Logit<LT>::VEC;
    const uint32_t ninf = sizeof(LT) == 2 ? 0xFF80FF80u : 0xFF800000u;
    float ma = METASD_NEG_BIG, mb = METASD_NEG_BIG;
    float sa0 = 0.f, sa1 = 0.f, sb0 = 0.f, sb1 = 0.f;
    int bv = -1;
    for (int i = 0, v = ct; i < trips; ++i, v += ncomp) {
        uint4 ra = make_uint4(ninf, ninf, ninf, ninf), rb = ra;
        if (v < my_vecs) {
            ra = *reinterpret_cast<const uint4 *>(slot_a + (size_t)v * 16);
            if (PAIR) rb = *reinterpret_cast<const uint4 *>(slot_b + (size_t)v * 16);
        }
        {
            const float vm = vector_max<LT>(ra);
            const float wm = warp_max_f(vm);
            if (wm > ma) {   // warp-uniform, rare after the first vectors: rescale the sums to the new maximum
                const float r = ex2((ma - wm) * c);
                sa0 *= r; sa1 *= r;
                ma = wm;
                bv = -1;
            }
            if (want_argmax && bv < 0 && vm == ma) bv = v;
            const float nm = -ma * c;
            float x[VEC];
            Logit<LT>::unpack(ra, x);
#pragma unroll
            for (int q = 0; q < VEC; q += 2) {
                sa0 += ex2(fmaf(x[q], c, nm));
                sa1 += ex2(fmaf(x[q + 1], c, nm));
            }
        }
        if (PAIR) {
            const float vm = vector_max<LT>(rb);
            const float wm = warp_max_f(vm);
            if (wm > mb) {
                const float r = ex2((mb - wm) * c);
                sb0 *= r; sb1 *= r;
                mb = wm;
            }
            const float nm = -mb * c;
            float x[VEC];
            Logit<LT>::unpack(rb, x);
#pragma unroll
            for (int q = 0; q < VEC; q += 2) {
                sb0 += ex2(fmaf(x[q], c, nm));
                sb1 += ex2(fmaf(x[q + 1], c, nm));
            }
        }
    }
    max_a = ma; sum_a = sa0 + sa1; vec_a = bv;
    max_b = mb; sum_b = sb0 + sb1;
}

// Pass 2 over one row pair in shared memory: sum_v 2^min(ya_v, yb_v) with ya = x_a c + nma, yb = x_b c + nmb_rel,
// i.e. sum_v min(p_v, q_v) * sum_a.
template <typename LT>
__device__ __forceinline__ float min_rows(const unsigned char *slot_a, const unsigned char *slot_b, int my_vecs, int ct,
                                          int ncomp, float c, float nma, float nmb_rel)
{
    constexpr int VEC = Logit<LT>::VEC;
    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll 2
    for (int v = ct; v < my_vecs; v += ncomp) {
        float xa[VEC], xb[VEC];
        Logit<LT>::unpack(*reinterpret_cast<const uint4 *>(slot_a + (size_t)v * 16), xa);
        Logit<LT>::unpack(*reinterpret_cast<const uint4 *>(slot_b + (size_t)v * 16), xb);
#pragma unroll
        for (int q = 0; q < VEC; q += 2) {
            acc0 += ex2(fminf(fmaf(xa[q], c, nma), fmaf(xb[q], c, nmb_rel)));
            acc1 += ex2(fminf(fmaf(xa[q + 1], c, nma), fmaf(xb[q + 1], c, nmb_rel)));
        }
    }
    return acc0 + acc1;
}

// Weights of the draw for one vector: mode 1 = max(0, p - q) (correction), mode 2 = p (bonus).
template <typename LT>
__device__ __forceinline__ void draw_weights(const unsigned char *slot_a, const unsigned char *slot_b, int v, int mode,
                                             float c, const RowConst &rc, float (&w)[Logit<LT>::VEC])
{
    constexpr int VEC = Logit<LT>::VEC;
    float xa[VEC], xb[VEC];
    Logit<LT>::unpack(*reinterpret_cast<const uint4 *>(slot_a + (size_t)v * 16), xa);
    if (mode == 1) Logit<LT>::unpack(*reinterpret_cast<const uint4 *>(slot_b + (size_t)v * 16), xb);
#pragma unroll
    for (int q = 0; q < VEC; ++q) {
        const float pv = ex2(fmaf(xa[q], c, rc.nma)) * rc.inv_sa;
        if (mode == 1) {
            const float qv = ex2(fmaf(xb[q], c, rc.nmb)) * rc.inv_sb;
            w[q] = fmaxf(pv - qv, 0.f);
        } else {
            w[q] = pv;
        }
    }
}

// Inverse CDF in token order over one row (pair) that lives in the shared memory of the whole cluster:
// the smallest v with sum_{w <= v} weight_w > u * total.  Every streaming warp owns a contiguous range
// of its CTA's slice; totals and offsets are carried in fp64.  Returns false (for every thread of the
// cluster alike) when the row has no mass; otherwise the token lands in sh.token of rank 0.
template <typename LT>
__device__ bool cluster_draw(FusedShared &sh, const RowConst &rc, const unsigned char *slot_a, const unsigned char *slot_b,
                             int mode, float c, int my_vecs, int vec0, int rank, int csize, int ncw)
{
    constexpr int VEC = Logit<LT>::VEC;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per_warp = (my_vecs + ncw - 1) / ncw;
    const int cw = warp - 1;   // streaming warp index; the control warp has none
    const int v0 = cw >= 0 ? min(cw * per_warp, my_vecs) : 0, v1 = cw >= 0 ? min(v0 + per_warp, my_vecs) : 0;
    if (cw >= 0) {
        double acc = 0.0;
        for (int v = v0 + lane; v < v1; v += 32) {
            float w[VEC];
            draw_weights<LT>(slot_a, slot_b, v, mode, c, rc, w);
            float s = 0.f;
#pragma unroll
            for (int q = 0; q < VEC; ++q) s += w[q];
            acc += (double)s;
        }
        acc = warp_sum(acc);
        if (lane == 0) sh.tot[cw] = acc;
    }
    __syncthreads();
    if (warp == 0) {
        const double t = lane < ncw ? sh.tot[lane] : 0.0;
        double incl = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double x = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += x;
        }
        if (lane < ncw) sh.pre[lane] = incl - t;
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
    const double thr = (double)rc.u_draw * R;
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
    if (rank == rstar && cw >= 0) {
        const double th = thr - mybase;
        // the warp whose range holds the crossing; rounding may leave none: then the last warp with mass
        const double t = lane < ncw ? sh.tot[lane] : 0.0;
        const double pr = lane < ncw ? sh.pre[lane] : 0.0;
        const unsigned crossing = __ballot_sync(0xFFFFFFFFu, lane < ncw && pr + t > th);
        const unsigned mass = __ballot_sync(0xFFFFFFFFu, lane < ncw && t > 0.0);
        const int wstar = crossing ? __ffs(crossing) - 1 : 31 - __clz(mass);
        if (cw == wstar) {
            int found = -1, last_pos = -1;
            double run_base = sh.pre[wstar];
            for (int i0 = v0; i0 < v1 && found < 0; i0 += 32) {
                const int v = i0 + lane;
                float w[VEC];
#pragma unroll
                for (int q = 0; q < VEC; ++q) w[q] = 0.f;
                if (v < v1) draw_weights<LT>(slot_a, slot_b, v, mode, c, rc, w);
                float s = 0.f;
#pragma unroll
                for (int q = 0; q < VEC; ++q) s += w[q];
                double incl = (double)s;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double x = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += x;
                }
                const unsigned ballot = __ballot_sync(0xFFFFFFFFu, run_base + incl > th);
#pragma unroll
                for (int q = 0; q < VEC; ++q)
                    if (w[q] > 0.f) last_pos = (vec0 + v) * VEC + q;
                if (ballot) {
                    const int src = __ffs(ballot) - 1;
                    if (lane == src) {
                        double cum = run_base + incl - (double)s;
                        int tok = -1;
#pragma unroll
                        for (int q = 0; q < VEC; ++q) {
                            cum += (double)w[q];
                            if (tok < 0 && cum > th) tok = (vec0 + v) * VEC + q;
                        }
                        // the vector's own sum crossed, so an element does unless rounding interferes
                        if (tok < 0) {
#pragma unroll
                            for (int q = 0; q < VEC; ++q)
                                if (w[q] > 0.f) tok = (vec0 + v) * VEC + q;
                        }
                        found = tok;
                    }
                    found = __shfl_sync(0xFFFFFFFFu, found, src);
                }
                run_base += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
            if (found < 0) {   // rounding left the running sum a hair under the threshold
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xFFFFFFFFu, last_pos, o));
                found = last_pos;
            }
            if (lane == 0) st_cluster(map_to_rank(smem_addr(&sh.token), 0), (int32_t)found);
        }
    }
    return true;
}

// Merges up to 32 records held one per lane (lanes >= n hold nothing): row maxima, row sums relative
// to them and the first arg-max of the target row.
struct Merged {
    float Ma, Sa, Mb, Sb;
    int idx;
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
    r.Sa = warp_sum_f(sa * ex2((ma - r.Ma) * c));
    r.Sb = warp_sum_f(sb * ex2((mb - r.Mb) * c));
    r.idx = __reduce_min_sync(0xFFFFFFFFu, (lane < n && ma == r.Ma) ? ia : INT_MAX);
    return r;
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
template <typename LT>
__global__ void __launch_bounds__(FUSED_MAX_THREADS, 1) fused_round_kernel(const VerifyParams p, const FusedGeom g)
{
    constexpr int VEC = Logit<LT>::VEC;
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ FusedShared sh;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ncw = (blockDim.x >> 5) - 1;            // streaming warps
    const int ncomp = ncw * 32, ct = tid - 32;        // streaming threads and this thread's index among them
    const bool control = warp == 0;
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
        for (int s = 0; s < 3; ++s) mbar_init(&sh.xbar[s], 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&sh.wbar[s], (uint32_t)ncw);
            mbar_init(&sh.rcbar[s], 1);
            mbar_init(&sh.ebar[s], (uint32_t)ncw);
        }
        sh.dead = 0;
        sh.token = -1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 16) sh.table[tid] = (p.drafter_ptrs && tid < p.K) ? p.drafter_ptrs[tid] : nullptr;
    cluster_sync_all();   // every CTA of the cluster is running, its barriers initialised, before a peer writes to it

    const int n_seq = cid < p.batch ? (p.batch - cid + ncl - 1) / ncl : 0;   // sequences of this cluster
    const int n_items = n_seq * (k + 1);

    // ---- producer (thread 0): the order of loads is sequence-major, position, target then draft
    int ld_b = cid, ld_j = 0, ld_row = 0, ld_slot = 0, ld_arm_next = 0;
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
    if (tid == 0 && n_seq > 0) {
        ld_draft = draft_base(p.draft ? 0 : p.st.arm[cid]);
        if (!p.draft && cid + ncl < p.batch) ld_arm_next = p.st.arm[cid + ncl];
        for (int s = 0; s < g.n_slot; ++s) issue_one();
    }

    // ---- control warp, lane j = position j: header of a sequence (round counter, arm, drafted token, its
    // two logits), fetched one sequence ahead in three steps spread over the items
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
    if (control && n_seq > 0) {
        fetch_step(cid, 0);
        fetch_step(cid, 1);
        fetch_step(cid, 2);
    }
    // header and results of the sequence in pass 2 (control warp registers, lane j = position j)
    int h_t = 0, h_arm = 0, h_tok = -1, r_acc = 0;
    float h_xa = 0.f, h_xb = 0.f, h_u = 0.f, h_ud = 0.f, r_px = 0.f, r_qx = 0.f;
    uint32_t r_rowflag = 0, seq_flags = 0;
    int n_acc = -1, token = -1;   // n_acc < 0: no rejection yet
    bool drew = false;            // the token sits in sh.token of rank 0

    // cursors: pass 1 consumes ring slots c1, pass 2 (one item behind) reads slots c2 and then frees them
    int j1 = 0, c1 = 0, b2 = cid, j2 = 0, c2 = 0;
    uint32_t c1par = 0;
    int u1 = 0, u2 = 0;            // item mod 3 of pass 1 / pass 2: which exchange buffer
    uint32_t x2par = 0;            // phase parity of xbar[u2]
    const int trips = (my_vecs + ncomp - 1) / ncomp;   // vectors per streaming thread and row slice

    // The streaming warps never meet a CTA-wide barrier in the steady state.  Per step n they hand their
    // records of item n to the control warp (wbar), pick up the row constants of item n-1 (rcbar) and give
    // back its slots (ebar); each hand-over is an mbarrier with two buffers, used by alternate steps.
    for (int step = 0; step <= n_items; ++step) {
        const bool do1 = step < n_items, do2 = step >= 1;
        const bool pair1 = j1 < k, pair2 = j2 < k;
        const int s1 = step & 1, s2 = (step - 1) & 1;                          // buffers of pass 1 / pass 2
        const uint32_t ph1 = (uint32_t)(step >> 1) & 1u, ph2 = (uint32_t)((step - 1) >> 1) & 1u;   // their phases
        const unsigned char *a2 = ring + (size_t)c2 * g.slot_bytes;
        const unsigned char *d2 = ring + (size_t)(c2 + 1 == g.n_slot ? 0 : c2 + 1) * g.slot_bytes;

        if (control) {
            // ---- expect one record of 32 bytes from every CTA of the cluster (this one included) for pass 1's item
            if (do1 && lane == 0 && !*(volatile int32_t *)&sh.dead)
                mbar_arrive_expect_tx(&sh.xbar[u1], (uint32_t)csize * EXCHANGE_BYTES);
            if (do2) {
                // ---- pass 2's item: merged records, flags, the accept test of Algorithm 4 (lines 7-8), what to draw
                if (j2 == 0) {   // a new sequence enters pass 2
                    h_t = nx_t; h_arm = nx_arm; h_tok = nx_tok; h_xa = nx_xa; h_xb = nx_xb;
                    const uint4 w = round_words(p.seed, p.sequence_base + (uint32_t)b2, (uint32_t)h_t, (uint32_t)lane);
                    h_u = uniform24(w.x);
                    h_ud = uniform24(w.y);
                    n_acc = -1; token = -1; drew = false; seq_flags = 0; r_acc = 0; r_px = 0.f; r_qx = 0.f; r_rowflag = 0;
                }
                const int b_next = b2 + ncl;
                if (b_next < p.batch) {
                    if (j2 == 0) fetch_step(b_next, 0);
                    if (j2 == 1) fetch_step(b_next, 1);
                    if (j2 == (k < 2 ? k : 2)) fetch_step(b_next, 2);
                }
                wait_bar(sh, &sh.xbar[u2], x2par, p.status);
                const Merged mg = merge_records(sh.exch[u2], csize, lane, c);
                // NaN or +Inf anywhere makes the sum NaN; an all -Inf row leaves it 0
                const bool bad_a = !(mg.Sa > 0.f) || !(mg.Sa < INFINITY) || !(mg.Ma < INFINITY);
                const bool bad_b = pair2 && (!(mg.Sb > 0.f) || !(mg.Sb < INFINITY) || !(mg.Mb < INFINITY));
                const uint32_t rowflag = (bad_a || bad_b) ? METASD_STATUS_NONFINITE : 0u;
                const float nma = -mg.Ma * c, nmb = -mg.Mb * c;
                bool accepted = false;
                if (pair2) {
                    // lane j2 holds this position's token; every lane evaluates it on the broadcast values
                    const int x = __shfl_sync(0xFFFFFFFFu, h_tok, j2);
                    const float xa = __shfl_sync(0xFFFFFFFFu, h_xa, j2), xb = __shfl_sync(0xFFFFFFFFu, h_xb, j2);
                    const float u = __shfl_sync(0xFFFFFFFFu, h_u, j2);
                    float p_x = 0.f, q_x = 0.f;
                    uint32_t fl = rowflag;
                    if (!rowflag) {
                        if (x < 0 || x >= V) {
                            fl |= METASD_STATUS_TOKEN_OOR;
                        } else {
                            p_x = ex2(fmaf(xa, c, nma)) / mg.Sa;
                            q_x = ex2(fmaf(xb, c, nmb)) / mg.Sb;
                            if (p.greedy) {
                                accepted = x == mg.idx;
                            } else {
                                if (q_x == 0.f) fl |= METASD_STATUS_Q_ZERO;
                                accepted = u * q_x < p_x;   // u < min(1, p/q) without the division
                            }
                        }
                    }
                    seq_flags |= fl;
                    if (lane == j2) { r_acc = accepted ? 1 : 0; r_px = p_x; r_qx = q_x; r_rowflag = rowflag; }
                }
                // first rejection (Algorithm 4, "exit for loop") or the bonus position: the next token comes from here
                int mode = 0;
                if (n_acc < 0) {
                    if (pair2 && !accepted) { n_acc = j2; mode = 1; }
                    if (!pair2) { n_acc = k; mode = 2; seq_flags |= rowflag; }
                    if (mode) {
                        if (rowflag) {
                            mode = 0;
                        } else if (p.greedy) {
                            token = mg.idx;
                            mode = 0;
                        }
                    }
                }
                const float ud = __shfl_sync(0xFFFFFFFFu, h_ud, j2);
                if (lane == 0) {
                    RowConst rc;
                    rc.nma = nma;
                    rc.nmb = nmb;
                    // q_v / p_v = 2^(yb - ya) sum_a / sum_b: the ratio of the sums folds into the draft row's offset
                    rc.nmb_rel = nmb + log2f(mg.Sa / mg.Sb);
                    rc.inv_sa = 1.0f / mg.Sa;
                    rc.inv_sb = 1.0f / mg.Sb;
                    rc.u_draw = ud;
                    rc.mode = mode;
                    rc.valid = rowflag ? 0 : 1;
                    sh.rc[s2] = rc;
                    mbar_arrive(&sh.rcbar[s2]);   // release: the streaming warps may start pass 2 of this item
                }
            }
            // ---- the CTA's record of pass 1's item goes to every CTA of the cluster
            if (do1) {
                wait_bar(sh, &sh.wbar[s1], ph1, p.status);
                const Merged mc = merge_records(sh.wrec[s1], ncw, lane, c);
                if (lane < csize) {
                    const uint32_t dst = map_to_rank(smem_addr(&sh.exch[u1][rank]), (uint32_t)lane);
                    const uint32_t bar = map_to_rank(smem_addr(&sh.xbar[u1]), (uint32_t)lane);
                    st_async_16(dst, bar, __float_as_uint(mc.Ma), __float_as_uint(mc.Sa), __float_as_uint(mc.Mb),
                                __float_as_uint(mc.Sb));
                    st_async_16(dst + 16, bar, (uint32_t)mc.idx, 0u, 0u, 0u);
                }
            }
        } else {
            if (do1) {
                // ---- pass 1: statistics of this item's row slices out of shared memory
                Exchange wr;
                int v_t;
                const int cb = c1 + 1 == g.n_slot ? 0 : c1 + 1;
                const unsigned char *slot_a = ring + (size_t)c1 * g.slot_bytes, *slot_b = ring + (size_t)cb * g.slot_bytes;
                wait_bar(sh, &sh.full[c1], c1par, p.status);
                if (pair1) {
                    wait_bar(sh, &sh.full[cb], cb == 0 ? c1par ^ 1u : c1par, p.status);
                    stats_rows<LT, true>(slot_a, slot_b, my_vecs, ct, ncomp, trips, c, p.greedy != 0, wr.max_a, wr.sum_a, v_t,
                                         wr.max_b, wr.sum_b);
                } else {
                    stats_rows<LT, false>(slot_a, slot_b, my_vecs, ct, ncomp, trips, c, p.greedy != 0, wr.max_a, wr.sum_a, v_t,
                                          wr.max_b, wr.sum_b);
                }
                int cand = INT_MAX;
                if (v_t >= 0) {   // first index of the maximum inside the vector in which this lane met it
                    float x[VEC];
                    Logit<LT>::unpack(*reinterpret_cast<const uint4 *>(slot_a + (size_t)v_t * 16), x);
#pragma unroll
                    for (int q = VEC - 1; q >= 0; --q)
                        if (x[q] == wr.max_a) cand = (vec0 + v_t) * VEC + q;
                }
                wr.idx_a = p.greedy ? __reduce_min_sync(0xFFFFFFFFu, cand) : INT_MAX;
                wr.sum_a = warp_sum_f(wr.sum_a);   // the lanes share one maximum per row
                wr.sum_b = warp_sum_f(wr.sum_b);
                if (lane == 0) {
                    wr.pad[0] = wr.pad[1] = wr.pad[2] = 0;
                    sh.wrec[s1][warp - 1] = wr;
                    mbar_arrive(&sh.wbar[s1]);
                }
            }
            if (do2) {
                // ---- pass 2: sum_v min(p_v, q_v) of this warp's logits
                wait_bar(sh, &sh.rcbar[s2], ph2, p.status);
                if (pair2) {
                    const RowConst rc = sh.rc[s2];
                    float acc = 0.f;
                    if (rc.valid) acc = min_rows<LT>(a2, d2, my_vecs, ct, ncomp, c, rc.nma, rc.nmb_rel) * rc.inv_sa;
                    acc = warp_sum_f(acc);
                    if (lane == 0) sh.pmin[j2][warp - 1] = acc;
                }
            }
        }
        if (do2) {
            const int mode = sh.rc[s2].mode;   // alike in every thread of the cluster; the control warp wrote it
            if (mode) {
                bool ok = cluster_draw<LT>(sh, sh.rc[s2], a2, d2, mode, c, my_vecs, vec0, rank, csize, ncw);
                if (!ok && mode == 1)   // p == q in fp32 yet rejected: draw from p
                    ok = cluster_draw<LT>(sh, sh.rc[s2], a2, d2, 2, c, my_vecs, vec0, rank, csize, ncw);
                drew = ok;
            }
            if (!pair2) {
                // ---- end of the sequence: gather sum_v min(p, q) per position in rank 0
                __syncthreads();
                if (control && lane < k) {
                    double s = 0.0;
                    for (int w = 0; w < ncw; ++w) s += (double)sh.pmin[lane][w];
                    st_cluster(map_to_rank(smem_addr(&sh.cta_min[lane][rank]), 0), s);
                }
                cluster_sync_all();
                if (rank == 0 && control) {
                    double smin = 0.0;
                    if (lane < k) {
                        for (int r = 0; r < csize; ++r) smin += sh.cta_min[lane][r];
                        if (r_rowflag) smin = 0.0;
                    }
                    double sum_align = 0.0;
                    for (int j = 0; j < k; ++j) sum_align += __shfl_sync(0xFFFFFFFFu, smin, j);
                    // Definition 2: 1 - mean_j d_TV; block efficiency: N_acc / N_max
                    const double r = p.reward_kind == METASD_REWARD_BE ? (double)n_acc / (double)k : sum_align / (double)k;
                    if (p.diag && lane < k) {
                        metasd_diag dg;
                        dg.p_x = r_px;
                        dg.q_x = r_qx;
                        dg.D = r_rowflag ? 1.f : (float)(1.0 - smin);
                        dg.u = h_u;
                        dg.accept = r_acc;
                        p.diag[(size_t)b2 * k + lane] = dg;
                    }
                    if (lane == 0) {
                        p.accepted_len[b2] = n_acc;
                        p.next_token[b2] = drew ? sh.token : token;
                        p.reward[b2] = (float)r;
                        if (seq_flags) atomicOr(p.status, seq_flags);
                    }
                    warp_bandit(p, b2, h_t, h_arm, r);
                }
            }
            // ---- pass 2's slots go back to the ring: the streaming warps sign off, the control warp refills
            if (!control) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.ebar[s2]);
            } else {
                wait_bar(sh, &sh.ebar[s2], ph2, p.status);
                if (lane == 0) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    issue_one();
                    if (pair2) issue_one();
                }
                __syncwarp();
            }
            c2 += pair2 ? 2 : 1;
            if (c2 >= g.n_slot) c2 -= g.n_slot;
            if (++u2 == 3) { u2 = 0; x2par ^= 1u; }
            if (++j2 > k) { j2 = 0; b2 += ncl; }
        }
        if (do1) {
            c1 += pair1 ? 2 : 1;
            if (c1 >= g.n_slot) { c1 -= g.n_slot; c1par ^= 1u; }
            if (++u1 == 3) u1 = 0;
            if (++j1 > k) j1 = 0;
        }
    }

    // ---- No CTA leaves while a copy into its shared memory may be in flight or a peer may still write to it.
    // Pass 1 has waited for every copy that was issued, unless a wait ran out: then give the copies one more
    // bounded delay before the shared memory is given up.
    if (tid == 0 && *(volatile int32_t *)&sh.dead) {
        for (uint32_t it = 0; it < (1u << 18); ++it) __nanosleep(256);
    }
    cluster_sync_all();
}

// ---------------------------------------------------------------------------------------------
// Host side: geometry, occupancy, launch
// ---------------------------------------------------------------------------------------------
const void *kernel_for(int dtype)
{
    return dtype == METASD_BF16 ? reinterpret_cast<const void *>(&fused_round_kernel<__nv_bfloat16>)
                                : reinterpret_cast<const void *>(&fused_round_kernel<float>);
}

// Geometry for cluster size C, or false when the row does not fit.
bool geometry(int dtype, int V, int C, int smem_optin, FusedPlan *pl)
{
    const size_t row_bytes = (size_t)V * (dtype == METASD_BF16 ? 2 : 4);
    if (row_bytes % 16 != 0) return false;
    const int n_vec_row = (int)(row_bytes / 16);
    if (C > n_vec_row) return false;
    const int n_vec_cta = (n_vec_row + C - 1) / C;
    if ((size_t)(C - 1) * n_vec_cta >= (size_t)n_vec_row) return false;   // an empty last rank: a smaller C serves better
    const int slot_bytes = n_vec_cta * 16;
    int n_slot = (smem_optin - FUSED_SMEM_RESERVE) / slot_bytes;
    if (n_slot > FUSED_MAX_SLOTS) n_slot = FUSED_MAX_SLOTS;
    if (n_slot < FUSED_MIN_SLOTS) return false;
    // streaming warps: the count that divides the slice with the least padding (the larger count on ties),
    // plus the control warp
    int best_w = 0;
    long best_cost = 0;
    for (int w = FUSED_MAX_WARPS - 1; w >= 1; --w) {
        const long cost = (long)(w * 32) * ((n_vec_cta + w * 32 - 1) / (w * 32));
        if (!best_w || cost < best_cost) { best_w = w; best_cost = cost; }
    }
    pl->cluster = C;
    pl->threads = (best_w + 1) * 32;
    pl->n_vec_row = n_vec_row;
    pl->n_vec_cta = n_vec_cta;
    pl->n_slot = n_slot;
    pl->slot_bytes = slot_bytes;
    pl->smem_bytes = (size_t)n_slot * slot_bytes;
    pl->work_per_item = n_vec_cta;
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
        if (pin_t >= 64 && pin_t <= FUSED_MAX_THREADS && pin_t % 32 == 0) pl.threads = pin_t;
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
        // per item: the two passes over the slice plus a fixed cost for barriers and exchanges
        const double cost = waves * ((double)pl.work_per_item + 300.0);
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
        e = cudaLaunchKernelEx(&cfg, fused_round_kernel<__nv_bfloat16>, p, g);
    else
        e = cudaLaunchKernelEx(&cfg, fused_round_kernel<float>, p, g);
    *launches += 1;
    return e;
}

}  // namespace metasd
