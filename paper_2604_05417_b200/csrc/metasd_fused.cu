// Fused cluster path of the MetaSD verify round: ONE persistent kernel per call.
//
// A thread-block cluster of C CTAs owns one sequence at a time and walks its k+1 positions in order.
// Every CTA owns a contiguous 1/C slice of each logit row; C is the smallest size for which a slice
// pair (target + draft) fits half an SM's shared memory, so that TWO CTAs (of different clusters) live
// on every SM and fill each other's waits.  Per position a CTA
//   - receives its two slices through bulk asynchronous copies (TMA), a few chunks per slice, each
//     completing on its own mbarrier: every logit is read from HBM exactly once;
//   - pass 1, chunk by chunk as they land: running maximum and sum_v 2^((x_v - max) c) of both rows, the
//     first arg-max of the target row; the CTA's record goes to every CTA of the cluster as asynchronous
//     distributed-shared-memory stores that complete on the receiver's mbarrier;
//   - pass 2, over the same bytes still in shared memory, with the merged records of the whole row pair:
//       sum_v min(p_v, q_v) = 1 - d_TV(p_j, q_j)  (Definition 2, Eq. 4), evaluated as
//       sum_v 2^min(log2 p_v, log2 q_v): one exponential per PAIR;
//     the accept test u q(x) < p(x) of the drafted token (Algorithm 4, the accept step), evaluated alike by
//     every thread of the cluster; at the first rejection (or the bonus position) the inverse-CDF draw
//     from max(0, p - q) (or p), a prefix search in token order across the cluster (Algorithm 4, 11-12).
// Rank 0 of the cluster then writes the outputs, forms the reward, and one warp updates the bandit and
// selects the next arm with one lane per drafter (Algorithm 2, update and selection steps).
#include <limits.h>

#include "metasd_device.cuh"

namespace metasd {

namespace {

constexpr int FUSED_MAX_THREADS = 640;            // two CTAs per SM: 1280 threads, about 50 registers each
constexpr int FUSED_MAX_WARPS = 32;
constexpr int FUSED_MAX_CLUSTER = 16;
constexpr int FUSED_CHUNKS = 4;                   // bulk copies (and mbarriers) per row slice
constexpr int FUSED_STATIC_SMEM = 9 * 1024;       // static shared memory of one CTA, rounded up
constexpr uint32_t WAIT_FAST_POLLS = 4096u;
constexpr uint32_t WAIT_SLOW_POLLS = 1u << 21;    // with a back-off of 128 ns each: a few tenths of a second

// ---------------------------------------------------------------------------------------------
// PTX wrappers: cluster identity and barrier, distributed shared memory, mbarrier, bulk copy
// ---------------------------------------------------------------------------------------------
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

// Constants of one row pair, known once the cluster's records are merged.
struct RowConst {
    float nma, nmb;      // -max c of the target / draft row
    float nmb_rel;       // nmb + log2(sum_a / sum_b): the draft row on the target row's scale
    float inv_sa, inv_sb;
    float u_draw;        // uniform of the residual / bonus draw
};

struct FusedShared {
    uint64_t full[2][FUSED_CHUNKS];                      // [row][chunk]: the chunk's bytes have landed
    uint64_t xbar[2];                                    // arrival of the peers' records, by item parity
    Exchange exch[2][FUSED_MAX_CLUSTER];                 // [item parity][sender rank]
    Exchange wrec[FUSED_MAX_WARPS];                      // the warps' records of the item
    double tot[FUSED_MAX_WARPS];                         // draw: weight of each warp's range
    double pre[FUSED_MAX_WARPS];                         // draw: exclusive prefix of tot
    double cta_tot[FUSED_MAX_CLUSTER];                   // draw: weight of each CTA's slice
    double cta_min[16][FUSED_MAX_CLUSTER];               // rank 0: sum of min(p, q) per position and sender
    float pmin[16][FUSED_MAX_WARPS];                     // sum of min(p, q) per position and warp
    const void *table[16];                               // the drafter pointer table
    // header of the current sequence
    int32_t h_tok[16];
    float h_xa[16], h_xb[16], h_u[16], h_ud[17];
    int32_t h_t, h_arm;
    // per-position results of the current sequence
    int32_t r_acc[16];
    float r_px[16], r_qx[16];
    uint32_t r_rowflag[16];
    int32_t token;                                       // rank 0: the drawn token
    int32_t dead;                                        // a wait ran out: later waits do not spin again
};

struct FusedGeom {
    int32_t n_vec_row;    // 16-byte vectors per logit row
    int32_t n_vec_cta;    // vectors of a row owned by one CTA (the last ranks may own fewer)
    int32_t slot_bytes;   // n_vec_cta * 16
    int32_t chunk_shift;  // a chunk is 1 << chunk_shift vectors
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
// vector in which it first met the target row's maximum.  Thread ct of nthr takes vectors ct, ct + nthr, ...;
// every lane makes the same number of trips, a vector beyond the slice reads as -inf.  A lane waits for the
// chunk that holds its vector before it reads it.
template <typename LT, bool PAIR>
__device__ __forceinline__ void stats_rows(FusedShared &sh, uint32_t *status, const unsigned char *slot_a,
                                           const unsigned char *slot_b, uint32_t par_a, uint32_t par_b, int chunk_shift,
                                           int my_vecs, int ct, int nthr, int trips, float c, float &max_a, float &sum_a,
                                           int &vec_a, float &max_b, float &sum_b)
{
    constexpr int VEC = Logit<LT>::VEC;
    const uint32_t ninf = sizeof(LT) == 2 ? 0xFF80FF80u : 0xFF800000u;
    float ma = METASD_NEG_BIG, mb = METASD_NEG_BIG;
    float sa0 = 0.f, sa1 = 0.f, sb0 = 0.f, sb1 = 0.f;
    int bv = -1, ready = 0;   // chunks [0, ready) of both rows are known to have landed
    for (int i = 0, v = ct; i < trips; ++i, v += nthr) {
        uint4 ra = make_uint4(ninf, ninf, ninf, ninf), rb = ra;
        if (v < my_vecs) {
            const int need = v >> chunk_shift;
            while (ready <= need) {
                wait_bar(sh, &sh.full[0][ready], par_a, status);
                if (PAIR) wait_bar(sh, &sh.full[1][ready], par_b, status);
                ++ready;
            }
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
            if (bv < 0 && vm == ma) bv = v;
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
// the smallest v with sum_{w <= v} weight_w > u * total.  Every warp owns a contiguous range of its
// CTA's slice; totals and offsets are carried in fp64.  Returns false (for every thread of the
// cluster alike) when the row has no mass; otherwise the token lands in sh.token of rank 0.
template <typename LT>
__device__ bool cluster_draw(FusedShared &sh, const RowConst &rc, const unsigned char *slot_a, const unsigned char *slot_b,
                             int mode, float c, int my_vecs, int vec0, int rank, int csize, int ncw)
{
    constexpr int VEC = Logit<LT>::VEC;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per_warp = (my_vecs + ncw - 1) / ncw;
    const int cw = warp;
    const int v0 = min(cw * per_warp, my_vecs), v1 = min(v0 + per_warp, my_vecs);
    {
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
    if (rank == rstar) {
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

// Bandit update and next selection by one warp, lane i = drafter i (Algorithm 2, update and selection steps; Discounted
// UCB; Sliding-window UCB).  Same fp64 expressions as the one-thread routines in metasd_device.cuh.
__device__ void warp_bandit(const VerifyParams &p, int b, int t, int arm, double r)
{
    const int lane = threadIdx.x & 31;
    const int K = p.K, tau = p.tau;
    double *sa = p.st.stat_a + (size_t)b * K, *sb = p.st.stat_b + (size_t)b * K;
    int32_t *wa = p.st.win_arm + (size_t)b * tau;
    double *wr = p.st.win_reward + (size_t)b * tau;
    if (p.bandit == METASD_EXP3 || p.bandit == METASD_RAND || p.bandit == METASD_PETC) {   // not an index arg-max: one lane does it
        if (lane == 0) {
            int32_t tt = t;
            bandit_update(p.bandit, K, p.gamma, tau, &tt, sa, sb, wa, wr, arm, r);
            p.st.t[b] = tt;
            p.st.arm[b] = bandit_select(p.bandit, K, p.beta, p.gamma, tau, tt, sa, sb, wa, wr, p.seed,
                                        p.sequence_base + (uint32_t)b);
        }
        return;
    }
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
__global__ void __launch_bounds__(FUSED_MAX_THREADS, 2) fused_round_kernel(const VerifyParams p, const FusedGeom g)
{
    constexpr int VEC = Logit<LT>::VEC;
    extern __shared__ __align__(128) unsigned char slices[];   // target slice, then draft slice
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
    const int chunk_vecs = 1 << g.chunk_shift;
    const int n_chunk = (my_vecs + chunk_vecs - 1) >> g.chunk_shift;
    const int trips = (my_vecs + nthr - 1) / nthr;   // vectors per thread and row slice
    unsigned char *slot_a = slices, *slot_b = slices + g.slot_bytes;

    if (tid == 0) {
        for (int r = 0; r < 2; ++r)
            for (int ch = 0; ch < FUSED_CHUNKS; ++ch) mbar_init(&sh.full[r][ch], 1);
        mbar_init(&sh.xbar[0], 1);
        mbar_init(&sh.xbar[1], 1);
        sh.dead = 0;
        sh.token = -1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 16) {
        const void *q = (p.drafter_ptrs && tid < p.K) ? p.drafter_ptrs[tid] : nullptr;
        sh.table[tid] = q;
        // a table entry that must not be read (NULL, misaligned) is flagged once per call, played or not
        if (p.drafter_ptrs && tid < p.K && blockIdx.x == 0 && (q == nullptr || (reinterpret_cast<uintptr_t>(q) & 15u) != 0))
            atomicOr(p.status, METASD_STATUS_BAD_POINTER);
    }
    cluster_sync_all();   // every CTA of the cluster is running, its barriers initialised, before a peer writes to it

    // ---- producer (thread 0): one item = the chunks of a target slice and, below the bonus position, of a draft slice
    int ld_b = cid, ld_j = 0, ld_arm_next = 0;
    const unsigned char *ld_draft = nullptr;
    auto draft_base = [&](int arm) -> const unsigned char * {
        return reinterpret_cast<const unsigned char *>(p.draft ? p.draft : sh.table[arm & 15]);
    };
    auto issue_row = [&](int row, const unsigned char *base, size_t row_index) {
        const unsigned char *src = base + row_index * row_bytes + (size_t)vec0 * 16;
        const bool bad = base == nullptr || (reinterpret_cast<uintptr_t>(src) & 15u) != 0;
        if (bad) atomicOr(p.status, METASD_STATUS_BAD_POINTER);   // never hand a misaligned address to the copy engine
        unsigned char *dst = row == 0 ? slot_a : slot_b;
        for (int ch = 0; ch < n_chunk; ++ch) {
            const int v_lo = ch << g.chunk_shift;
            const uint32_t bytes = (uint32_t)(min(my_vecs, v_lo + chunk_vecs) - v_lo) * 16u;
            uint64_t *bar = &sh.full[row][ch];
            if (bad) {
                mbar_arrive(bar);
            } else {
                mbar_arrive_expect_tx(bar, bytes);
                bulk_load(dst + (size_t)v_lo * 16, src + (size_t)v_lo * 16, bytes, bar);
            }
        }
    };
    auto issue_item = [&]() {
        if (ld_b >= p.batch || *(volatile int32_t *)&sh.dead) return;   // after a time-out nothing more is armed
        issue_row(0, reinterpret_cast<const unsigned char *>(p.target), (size_t)ld_b * (k + 1) + ld_j);
        if (ld_j < k) issue_row(1, ld_draft, (size_t)ld_b * k + ld_j);
        if (++ld_j > k) {
            ld_j = 0;
            ld_b += ncl;
            if (ld_b < p.batch) {
                ld_draft = draft_base(ld_arm_next);
                if (!p.draft && ld_b + ncl < p.batch) ld_arm_next = p.st.arm[ld_b + ncl];
            }
        }
    };
    if (tid == 0 && cid < p.batch) {
        ld_draft = draft_base(p.draft ? 0 : p.st.arm[cid]);
        if (!p.draft && cid + ncl < p.batch) ld_arm_next = p.st.arm[cid + ncl];
        issue_item();
    }

    // ---- header of a sequence (warp 0, lane j = position j): round counter, arm, drafted token and
    // its two logits.  Fetched one sequence ahead, in three steps spread over the items.
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

    uint32_t item = 0;       // items done by this cluster: bit 0 selects the exchange buffers, bit 1 their phase
    uint32_t par_a = 0, par_b = 0;   // phase parities of the target / draft chunk barriers

    for (int b = cid; b < p.batch; b += ncl) {
        // ---- publish the header of sequence b (read after the next CTA barrier)
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

            // ---- pass 1: statistics of this item's slices, chunk by chunk as the copies land
            {
                Exchange wr;
                int v_t;
                if (pair)
                    stats_rows<LT, true>(sh, p.status, slot_a, slot_b, par_a, par_b, g.chunk_shift, my_vecs, tid, nthr, trips, c,
                                         wr.max_a, wr.sum_a, v_t, wr.max_b, wr.sum_b);
                else
                    stats_rows<LT, false>(sh, p.status, slot_a, slot_b, par_a, par_b, g.chunk_shift, my_vecs, tid, nthr, trips, c,
                                          wr.max_a, wr.sum_a, v_t, wr.max_b, wr.sum_b);
                int cand = INT_MAX;
                if (p.greedy && v_t >= 0) {   // first index of the maximum inside the vector in which this lane met it
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
                    sh.wrec[warp] = wr;
                }
            }
            par_a ^= 1u;
            if (pair) par_b ^= 1u;
            __syncthreads();

            // ---- the CTA's record goes to every CTA of the cluster (asynchronous stores that complete on
            //      the receiver's barrier); then wait for all the records addressed to this CTA
            if (warp == 0) {
                const Merged mc = merge_records(sh.wrec, nw, lane, c);
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
            // NaN or +Inf anywhere makes the sum NaN; an all -Inf row leaves it 0
            const bool bad_a = !(mg.Sa > 0.f) || !(mg.Sa < INFINITY) || !(mg.Ma < INFINITY);
            const bool bad_b = pair && (!(mg.Sb > 0.f) || !(mg.Sb < INFINITY) || !(mg.Mb < INFINITY));
            const uint32_t rowflag = (bad_a || bad_b) ? METASD_STATUS_NONFINITE : 0u;
            RowConst rc;
            rc.nma = -mg.Ma * c;
            rc.nmb = -mg.Mb * c;
            // q_v / p_v = 2^(yb - ya) sum_a / sum_b: the ratio of the sums folds into the draft row's offset
            rc.nmb_rel = rc.nmb + log2f(mg.Sa / mg.Sb);
            rc.inv_sa = 1.0f / mg.Sa;
            rc.inv_sb = 1.0f / mg.Sb;
            rc.u_draw = sh.h_ud[j];

            // ---- pass 2: sum_v min(p_v, q_v) of this warp's logits; the accept test of Algorithm 4,
            //      evaluated alike by every thread of the cluster
            bool accepted = false;
            if (pair) {
                float acc = 0.f;
                if (!rowflag) acc = min_rows<LT>(slot_a, slot_b, my_vecs, tid, nthr, c, rc.nma, rc.nmb_rel) * rc.inv_sa;
                acc = warp_sum_f(acc);
                if (lane == 0) sh.pmin[j][warp] = acc;

                const int x = sh.h_tok[j];
                float p_x = 0.f, q_x = 0.f;
                uint32_t fl = rowflag;
                if (!rowflag) {
                    if (x < 0 || x >= V) {
                        fl |= METASD_STATUS_TOKEN_OOR;
                    } else {
                        p_x = ex2(fmaf(sh.h_xa[j], c, rc.nma)) / mg.Sa;
                        q_x = ex2(fmaf(sh.h_xb[j], c, rc.nmb)) / mg.Sb;
                        if (p.greedy) {
                            accepted = x == mg.idx;
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
                        token = mg.idx;
                        mode = 0;
                    }
                }
            }
            if (mode) {
                // the draw reads vectors this thread has not read before: see every chunk's copy complete first
                for (int ch = 0; ch < n_chunk; ++ch) {
                    wait_bar(sh, &sh.full[0][ch], par_a ^ 1u, p.status);
                    if (pair) wait_bar(sh, &sh.full[1][ch], par_b ^ 1u, p.status);
                }
                bool ok = cluster_draw<LT>(sh, rc, slot_a, slot_b, mode, c, my_vecs, vec0, rank, csize, nw);
                if (!ok && mode == 1)   // p == q in fp32 yet rejected: draw from p
                    ok = cluster_draw<LT>(sh, rc, slot_a, slot_b, 2, c, my_vecs, vec0, rank, csize, nw);
                drew = ok;
            }
            __syncthreads();   // every warp is done with the slices: the next item's copies may overwrite them
            if (tid == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                issue_item();
            }
        }

        // ---- end of the sequence: gather sum_v min(p, q) per position in rank 0
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

// Geometry for cluster size C, or false when a slice pair does not fit half an SM's shared memory.
bool geometry(int dtype, int V, int C, int smem_per_sm, FusedPlan *pl)
{
    const size_t row_bytes = (size_t)V * (dtype == METASD_BF16 ? 2 : 4);
    if (row_bytes % 16 != 0) return false;
    const int n_vec_row = (int)(row_bytes / 16);
    if (C > n_vec_row) return false;
    const int n_vec_cta = (n_vec_row + C - 1) / C;
    if ((size_t)(C - 1) * n_vec_cta >= (size_t)n_vec_row) return false;   // an empty last rank: a smaller C serves better
    const int slot_bytes = n_vec_cta * 16;
    // two CTAs per SM; each CTA also pays 1 KB that the system reserves
    const int budget = smem_per_sm / 2 - 1024 - FUSED_STATIC_SMEM;
    if (2 * slot_bytes > budget) return false;
    // warps: the count that covers the slice with the least padding (the larger count on ties)
    int best_w = 0;
    long best_cost = 0;
    for (int w = FUSED_MAX_THREADS / 32; w >= 2; --w) {
        const long cost = (long)(w * 32) * ((n_vec_cta + w * 32 - 1) / (w * 32));
        if (!best_w || cost < best_cost) { best_w = w; best_cost = cost; }
    }
    int shift = 0;
    while ((FUSED_CHUNKS << shift) < n_vec_cta) ++shift;
    pl->cluster = C;
    pl->threads = best_w * 32;
    pl->n_vec_row = n_vec_row;
    pl->n_vec_cta = n_vec_cta;
    pl->n_slot = shift;   // log2 of the vectors per chunk
    pl->slot_bytes = slot_bytes;
    pl->smem_bytes = (size_t)2 * slot_bytes;
    pl->work_per_item = n_vec_cta;
    pl->max_clusters = 0;
    return true;
}

}  // namespace

bool fused_supported(int dtype, int V, int k)
{
    if (k < 1 || k > 16) return false;
    FusedPlan pl;
    for (int C = 1; C <= FUSED_MAX_CLUSTER; ++C)
        if (geometry(dtype, V, C, 228 * 1024, &pl)) return true;
    return false;
}

// Chooses the cluster size for this device: the smallest for which two CTAs fit an SM, and asks the occupancy
// calculator how many clusters are co-resident (GPC shapes decide).
// pin_c / pin_t (the configuration's fused_cluster / fused_threads; 0 = free) pin the choice for tuning runs.
cudaError_t fused_prepare(int device, int dtype, int V, int max_batch, int pin_c, int pin_t, FusedPlan *plan)
{
    plan->cluster = 0;
    int smem_per_sm = 0;
    cudaError_t e = cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, device);
    if (e != cudaSuccess) return e;
    const void *fn = kernel_for(dtype);
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_per_sm / 2 - 1024 - FUSED_STATIC_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    double best = 0.0;
    for (int C = 1; C <= FUSED_MAX_CLUSTER; ++C) {
        if (pin_c && C != pin_c) continue;
        FusedPlan pl;
        if (!geometry(dtype, V, C, smem_per_sm, &pl)) continue;
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
        if (!pin_c) break;   // the smallest size that fits: the largest slices, the fewest exchange partners
    }
    return plan->cluster ? cudaSuccess : cudaErrorNotSupported;
}

cudaError_t launch_fused(const VerifyParams &p, int dtype, const FusedPlan &plan, cudaStream_t stream, uint64_t *launches)
{
    FusedGeom g;
    g.n_vec_row = plan.n_vec_row;
    g.n_vec_cta = plan.n_vec_cta;
    g.slot_bytes = plan.slot_bytes;
    g.chunk_shift = plan.n_slot;
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
