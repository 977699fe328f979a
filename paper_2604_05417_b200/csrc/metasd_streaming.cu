// Streaming path of the MetaSD verify round: works for every shape.
//
//   K1s split_row_stats_kernel  the same statistics as K1 with grp_size co-resident CTAs per row pair, each on its
//                          own part of the vocabulary: they exchange (max, sum, arg-max) records through global
//                          memory between the two sweeps.  Few enough row pairs are then in flight for the second
//                          sweep to be served by L2 instead of HBM.  Used for 16-byte aligned rows when splitting pays.
//   K1  row_stats_kernel   one CTA per (sequence b, position j): softmax statistics of the target
//                          row and the draft row with an online maximum, the target arg-max, then
//                          sum_v min(p_v, q_v) = 1 - d_TV(p_j, q_j) (Definition 2) in a second
//                          sweep over the same rows.  Writes one RowStats record.
//   K2  epilogue_kernel    one CTA per sequence: accept tests with the Philox uniforms (Algorithm 4,
//                          lines 7-8), first rejection, inverse-CDF draw of the correction token from
//                          max(0, p - q) or of the bonus token from p (lines 11-12), the reward, the
//                          bandit update and the next round's arm (Algorithm 2, lines 7-10).
#include <stdlib.h>

#include "metasd_device.cuh"

namespace metasd {

constexpr int K1_THREADS = 512;

template <typename LT>
__device__ __forceinline__ const LT *draft_rows(const VerifyParams &p, int b)
{
    if (p.draft) return reinterpret_cast<const LT *>(p.draft);
    return reinterpret_cast<const LT *>(p.drafter_ptrs[p.st.arm[b]]);   // the table was checked by sanitize_table_kernel
}

// -------------------------------------------------------------------------------------------
// K1
// -------------------------------------------------------------------------------------------
template <typename LT, bool VECTOR>
__global__ void __launch_bounds__(K1_THREADS) row_stats_kernel(const VerifyParams p)
{
    constexpr int VEC = VECTOR ? Logit<LT>::VEC : 1;
    constexpr int NWARP = K1_THREADS / 32;
    const int j = blockIdx.x, b = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = p.V;
    const float c = p.c;
    const bool pair = j < p.k;

    const LT *a = reinterpret_cast<const LT *>(p.target) + ((size_t)b * (p.k + 1) + j) * V;
    const LT *d = pair ? draft_rows<LT>(p, b) + ((size_t)b * p.k + j) * V : nullptr;
    const int nvec = V / VEC;

    // ---- sweep 1: online (max, sum) of both rows, arg-max of the target row
    MaxSum sa = {METASD_NEG_BIG, 0.f}, sb = {METASD_NEG_BIG, 0.f};
    ArgMax am = {METASD_NEG_BIG, 0x7FFFFFFF};
    const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
    const int keep_from = nvec - (int)((long long)nvec * p.keep_permille / 1000);
    for (int i = tid; i < nvec; i += K1_THREADS) {
        float xa[VEC], xb[VEC];
        if constexpr (VECTOR) {
            // the end of the rows is asked to stay in L2 until the second sweep (which starts there) re-reads it
            const uint64_t pol = i >= keep_from ? keep : drop;
            Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(a) + i, pol), xa);
            if (pair) Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(d) + i, pol), xb);
        } else {
            xa[0] = Logit<LT>::scalar(a, i);
            if (pair) xb[0] = Logit<LT>::scalar(d, i);
        }
        float cm = xa[0];
#pragma unroll
        for (int e = 1; e < VEC; ++e) cm = fmaxf(cm, xa[e]);
        if (cm > sa.m) {
            sa.s *= ex2((sa.m - cm) * c);
            sa.m = cm;
            int first = 0;
#pragma unroll
            for (int e = VEC - 1; e >= 0; --e)
                if (xa[e] == cm) first = e;
            am.v = cm;
            am.i = i * VEC + first;
        }
        const float nma = -sa.m * c;
#pragma unroll
        for (int e = 0; e < VEC; ++e) sa.s += ex2(fmaf(xa[e], c, nma));
        if (pair) {
            float bm = xb[0];
#pragma unroll
            for (int e = 1; e < VEC; ++e) bm = fmaxf(bm, xb[e]);
            if (bm > sb.m) {
                sb.s *= ex2((sb.m - bm) * c);
                sb.m = bm;
            }
            const float nmb = -sb.m * c;
#pragma unroll
            for (int e = 0; e < VEC; ++e) sb.s += ex2(fmaf(xb[e], c, nmb));
        }
    }

    __shared__ MaxSum sh_a[NWARP], sh_b[NWARP];
    __shared__ ArgMax sh_am[NWARP];
    __shared__ double sh_min[NWARP];
    __shared__ float sh_bcast[5];

    sa = warp_merge(sa, c);
    sb = warp_merge(sb, c);
    am = warp_argmax(am);
    if (lane == 0) { sh_a[warp] = sa; sh_b[warp] = sb; sh_am[warp] = am; }
    __syncthreads();
    if (warp == 0) {
        MaxSum ra = lane < NWARP ? sh_a[lane] : MaxSum{METASD_NEG_BIG, 0.f};
        MaxSum rb = lane < NWARP ? sh_b[lane] : MaxSum{METASD_NEG_BIG, 0.f};
        ArgMax rm = lane < NWARP ? sh_am[lane] : ArgMax{METASD_NEG_BIG, 0x7FFFFFFF};
        ra = warp_merge(ra, c);
        rb = warp_merge(rb, c);
        rm = warp_argmax(rm);
        if (lane == 0) {
            sh_bcast[0] = ra.m; sh_bcast[1] = ra.s; sh_bcast[2] = rb.m; sh_bcast[3] = rb.s;
            // q_v / p_v = 2^(yb - ya) sum_a / sum_b: the ratio of the sums folds into the draft row's offset
            sh_bcast[4] = -rb.m * c + log2f(ra.s / rb.s);
            sh_am[0] = rm;
        }
    }
    __syncthreads();
    const float max_a = sh_bcast[0], sum_a = sh_bcast[1], max_b = sh_bcast[2], sum_b = sh_bcast[3];

    // ---- sweep 2: sum_v min(p_v, q_v) = (1 / sum_a) sum_v 2^min(ya_v, yb_v): one exponential per pair
    double total_min = 0.0;
    if (pair) {
        const float nma = -max_a * c, nmb = sh_bcast[4];
        const float ia = 1.0f / sum_a;
        float acc = 0.f;
        // backwards: the end of the rows was read last in sweep 1 and is the part most likely still in L2
        for (int i = nvec - 1 - tid; i >= 0; i -= K1_THREADS) {
            float xa[VEC], xb[VEC];
            if constexpr (VECTOR) {
                Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(a) + i, drop), xa);
                Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(d) + i, drop), xb);
            } else {
                xa[0] = Logit<LT>::scalar(a, i);
                xb[0] = Logit<LT>::scalar(d, i);
            }
#pragma unroll
            for (int e = 0; e < VEC; ++e)
                acc += ex2(fminf(fmaf(xa[e], c, nma), fmaf(xb[e], c, nmb)));
        }
        double w = warp_sum((double)(acc * ia));
        if (lane == 0) sh_min[warp] = w;
        __syncthreads();
        if (tid == 0) {
            for (int i = 0; i < NWARP; ++i) total_min += sh_min[i];
        }
    }

    if (tid == 0) {
        RowStats r;
        r.max_a = max_a; r.sum_a = sum_a; r.max_b = max_b; r.sum_b = sum_b;
        r.argmax_a = sh_am[0].i;
        uint32_t flags = 0;
        // NaN or +Inf anywhere makes the sum NaN; an all -Inf row leaves it 0
        const bool bad_a = !(sum_a > 0.f) || !(sum_a < INFINITY) || !(max_a < INFINITY);
        const bool bad_b = pair && (!(sum_b > 0.f) || !(sum_b < INFINITY) || !(max_b < INFINITY));
        if (bad_a || bad_b) flags |= METASD_STATUS_NONFINITE;
        r.sum_min = flags ? 0.0 : total_min;
        r.flags = flags;
        p.stats[(size_t)b * (p.k + 1) + j] = r;
    }
}

// -------------------------------------------------------------------------------------------
// K1s
// -------------------------------------------------------------------------------------------
constexpr int KS_THREADS = 512;
constexpr uint32_t KS_SPIN_LIMIT = 1u << 22;   // polls of 64 ns: a quarter of a second

// Adds 1 without waiting for the result; the thread's earlier writes are visible to whoever sees the new count.
__device__ __forceinline__ void red_release_inc(uint32_t *p)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Warp 0 of every CTA only communicates: it publishes the CTA's record of a row pair (a release increment, no
// round trip), waits (bounded) for the group's records, merges them for the second sweep, and afterwards
// publishes the CTA's partial sum of min(p, q); the CTAs of a group take turns in adding the parts up.
template <typename LT>
__global__ void __launch_bounds__(KS_THREADS, 3) split_row_stats_kernel(const VerifyParams p)
{
    constexpr int VEC = Logit<LT>::VEC;
    constexpr int NWARP = KS_THREADS / 32;          // warp 0 + NWARP - 1 sweeping warps
    constexpr int NSWEEP = KS_THREADS - 32;         // sweeping threads
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int st = tid - 32;                        // index among the sweeping threads
    const int V = p.V, G = p.grp_size;
    const float c = p.c;
    const int n_groups = gridDim.x / G, grp = blockIdx.x / G, g = blockIdx.x - grp * G;
    const int nvec = V / VEC, per = (nvec + G - 1) / G;
    const int v_lo = min(g * per, nvec), v_hi = min(v_lo + per, nvec);   // this CTA's part of every row
    const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
    const int keep_from = v_hi - (int)((long long)(v_hi - v_lo) * p.keep_permille / 1000);
    __shared__ MaxSum sh_a[NWARP], sh_b[NWARP];
    __shared__ ArgMax sh_am[NWARP];
    __shared__ double sh_min[NWARP];
    __shared__ float sh_bcast[5];      // merged statistics of the row pair in its second sweep
    __shared__ int sh_arg;
    const int n_items = p.batch * (p.k + 1);

    auto row_ptrs = [&](int item, const LT *&a, const LT *&d, bool &pair) {
        const int b = item / (p.k + 1), j = item - b * (p.k + 1);
        pair = j < p.k;
        a = reinterpret_cast<const LT *>(p.target) + ((size_t)b * (p.k + 1) + j) * V;
        d = pair ? draft_rows<LT>(p, b) + ((size_t)b * p.k + j) * V : nullptr;
    };
    // ---- sweeping warps: online (max, sum) of both rows, arg-max of the target row, over this CTA's part
    auto first_sweep = [&](int item) {
        const LT *a, *d;
        bool pair;
        row_ptrs(item, a, d, pair);
        MaxSum sa = {METASD_NEG_BIG, 0.f}, sb = {METASD_NEG_BIG, 0.f};
        ArgMax am = {METASD_NEG_BIG, 0x7FFFFFFF};
        for (int i = v_lo + st; i < v_hi; i += NSWEEP) {
            float xa[VEC], xb[VEC];
            // the end of this CTA's part is asked to stay in L2 until the second sweep (which starts there)
            const uint64_t pol = i >= keep_from ? keep : drop;
            Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(a) + i, pol), xa);
            if (pair) Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(d) + i, pol), xb);
            float cm = xa[0];
#pragma unroll
            for (int e = 1; e < VEC; ++e) cm = fmaxf(cm, xa[e]);
            if (cm > sa.m) {
                sa.s *= ex2((sa.m - cm) * c);
                sa.m = cm;
                int first = 0;
#pragma unroll
                for (int e = VEC - 1; e >= 0; --e)
                    if (xa[e] == cm) first = e;
                am.v = cm;
                am.i = i * VEC + first;
            }
            const float nma = -sa.m * c;
#pragma unroll
            for (int e = 0; e < VEC; ++e) sa.s += ex2(fmaf(xa[e], c, nma));
            if (pair) {
                float bm = xb[0];
#pragma unroll
                for (int e = 1; e < VEC; ++e) bm = fmaxf(bm, xb[e]);
                if (bm > sb.m) {
                    sb.s *= ex2((sb.m - bm) * c);
                    sb.m = bm;
                }
                const float nmb = -sb.m * c;
#pragma unroll
                for (int e = 0; e < VEC; ++e) sb.s += ex2(fmaf(xb[e], c, nmb));
            }
        }
        sa = warp_merge(sa, c);
        sb = warp_merge(sb, c);
        am = warp_argmax(am);
        if (lane == 0) { sh_a[warp] = sa; sh_b[warp] = sb; sh_am[warp] = am; }
    };
    // ---- sweeping warps: sum_v min(p_v, q_v) = (1 / sum_a) sum_v 2^min(ya_v, yb_v) over this CTA's part
    auto second_sweep = [&](int item) {
        const LT *a, *d;
        bool pair;
        row_ptrs(item, a, d, pair);
        double w = 0.0;
        if (pair) {
            const float nma = -sh_bcast[0] * c, nmb = sh_bcast[4], sum_a = sh_bcast[1];
            float acc = 0.f;
            for (int i = v_hi - 1 - st; i >= v_lo; i -= NSWEEP) {   // backwards: the end was read last
                float xa[VEC], xb[VEC];
                Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(a) + i, drop), xa);
                Logit<LT>::unpack(ld_stream_hint(reinterpret_cast<const uint4 *>(d) + i, drop), xb);
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc += ex2(fminf(fmaf(xa[e], c, nma), fmaf(xb[e], c, nmb)));
            }
            w = warp_sum((double)(acc / sum_a));
        }
        if (lane == 0) sh_min[warp] = w;
    };
    // ---- warp 0: the CTA's record of a first sweep goes to global memory
    auto publish_record = [&](int item) {
        MaxSum ra = (lane >= 1 && lane < NWARP) ? sh_a[lane] : MaxSum{METASD_NEG_BIG, 0.f};
        MaxSum rb = (lane >= 1 && lane < NWARP) ? sh_b[lane] : MaxSum{METASD_NEG_BIG, 0.f};
        ArgMax rm = (lane >= 1 && lane < NWARP) ? sh_am[lane] : ArgMax{METASD_NEG_BIG, 0x7FFFFFFF};
        ra = warp_merge(ra, c);
        rb = warp_merge(rb, c);
        rm = warp_argmax(rm);
        if (lane == 0) {
            GroupRecord r;
            r.max_a = ra.m; r.sum_a = ra.s; r.max_b = rb.m; r.sum_b = rb.s; r.argmax_a = rm.i;
            r.pad[0] = r.pad[1] = r.pad[2] = 0;
            p.grp_rec[(size_t)item * G + g] = r;
            red_release_inc(&p.grp_count[item]);
        }
    };
    // ---- warp 0: wait (bounded) for the group's records of a row pair and merge them for its second sweep
    auto merge_group = [&](int item) {
        if (lane == 0) {
            uint32_t it = 0;
            while (ld_acquire(&p.grp_count[item]) < (uint32_t)G) {
                if (++it > KS_SPIN_LIMIT) { atomicOr(p.status, METASD_STATUS_TIMEOUT); break; }
                __nanosleep(64);
            }
        }
        __syncwarp();
        MaxSum ga = {METASD_NEG_BIG, 0.f}, gb = {METASD_NEG_BIG, 0.f};
        ArgMax gm = {METASD_NEG_BIG, 0x7FFFFFFF};
        if (lane < G) {
            const int4 *src = reinterpret_cast<const int4 *>(p.grp_rec + (size_t)item * G + lane);
            const int4 lo = __ldcg(src), hi = __ldcg(src + 1);
            ga.m = __int_as_float(lo.x); ga.s = __int_as_float(lo.y);
            gb.m = __int_as_float(lo.z); gb.s = __int_as_float(lo.w);
            gm.v = ga.m; gm.i = hi.x;
        }
        ga = warp_merge(ga, c);
        gb = warp_merge(gb, c);
        gm = warp_argmax(gm);
        if (lane == 0) {
            sh_bcast[0] = ga.m; sh_bcast[1] = ga.s; sh_bcast[2] = gb.m; sh_bcast[3] = gb.s;
            // q_v / p_v = 2^(yb - ya) sum_a / sum_b: the ratio of the sums folds into the draft row's offset
            sh_bcast[4] = -gb.m * c + log2f(ga.s / gb.s);
            sh_arg = gm.i;
        }
    };
    // ---- warp 0: this CTA's part of sum min(p, q)
    auto publish_min = [&](int item) {
        if (lane == 0) {
            double part = 0.0;
            for (int i = 1; i < NWARP; ++i) part += sh_min[i];
            p.grp_min[(size_t)item * G + g] = part;
            red_release_inc(&p.grp_count[item]);
        }
    };
    // ---- warp 0 of one CTA of the group (they take turns): once every part is in, add the parts up and write the
    //      row pair's statistics
    auto finalise = [&](int item, float max_a, float sum_a, float max_b, float sum_b, int arg) {
        if (lane == 0) {
            uint32_t it = 0;
            while (ld_acquire(&p.grp_count[item]) < 2u * (uint32_t)G) {
                if (++it > KS_SPIN_LIMIT) { atomicOr(p.status, METASD_STATUS_TIMEOUT); break; }
                __nanosleep(64);
            }
            const bool pair = item % (p.k + 1) < p.k;
            double total = 0.0;
            for (int i = 0; i < G; ++i) total += __ldcg(p.grp_min + (size_t)item * G + i);
            RowStats r;
            r.max_a = max_a; r.sum_a = sum_a; r.max_b = max_b; r.sum_b = sum_b;
            r.argmax_a = arg;
            uint32_t flags = 0;
            // NaN or +Inf anywhere makes the sum NaN; an all -Inf row leaves it 0
            const bool bad_a = !(sum_a > 0.f) || !(sum_a < INFINITY) || !(max_a < INFINITY);
            const bool bad_b = pair && (!(sum_b > 0.f) || !(sum_b < INFINITY) || !(max_b < INFINITY));
            if (bad_a || bad_b) flags |= METASD_STATUS_NONFINITE;
            r.sum_min = flags ? 0.0 : total;
            r.flags = flags;
            p.stats[item] = r;
        }
    };

    // Group grp takes row pairs grp, grp + n_groups, ... in (sequence, position) order: both sweeps of a row pair
    // back to back (the second finds the first's bytes in L2), the group's exchange in between.
    float m_a = 0.f, s_a = 0.f, m_b = 0.f, s_b = 0.f;
    int arg = 0, turn = 0;
    for (int item = grp; item < n_items; item += n_groups, ++turn) {
        if (warp != 0) first_sweep(item);
        __syncthreads();
        if (warp == 0) {
            publish_record(item);
            merge_group(item);
            m_a = sh_bcast[0]; s_a = sh_bcast[1]; m_b = sh_bcast[2]; s_b = sh_bcast[3]; arg = sh_arg;
        }
        __syncthreads();
        if (warp != 0) second_sweep(item);
        __syncthreads();
        if (warp == 0) {
            publish_min(item);
            if (turn % G == g) finalise(item, m_a, s_a, m_b, s_b, arg);   // the CTAs of a group take turns
        }
    }
}

// -------------------------------------------------------------------------------------------
// K2
// -------------------------------------------------------------------------------------------
// weight of token v in the draw: mode 1 = max(0, p_v - q_v) (correction), mode 2 = p_v (bonus)
template <typename LT, int VEC>
__device__ __forceinline__ void draw_weights(const LT *a, const LT *d, int i, int mode, float c, float nma,
                                             float ia, float nmb, float ib, float (&w)[VEC])
{
    float xa[VEC], xb[VEC];
    if constexpr (VEC > 1) {
        Logit<LT>::unpack(ld_stream(reinterpret_cast<const uint4 *>(a) + i), xa);
        if (mode == 1) Logit<LT>::unpack(ld_stream(reinterpret_cast<const uint4 *>(d) + i), xb);
    } else {
        xa[0] = Logit<LT>::scalar(a, i);
        if (mode == 1) xb[0] = Logit<LT>::scalar(d, i);
    }
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        float pv = ex2(fmaf(xa[e], c, nma)) * ia;
        if (mode == 1) {
            float qv = ex2(fmaf(xb[e], c, nmb)) * ib;
            w[e] = fmaxf(pv - qv, 0.f);
        } else {
            w[e] = pv;
        }
    }
}

// Inverse CDF in token order over one row (pair): the smallest v with sum_{w<=v} weight_w > u * total.
// Every warp owns a contiguous range of vectors; totals and offsets are carried in fp64.
template <typename LT, bool VECTOR, int K2_THREADS>
__device__ int block_inverse_cdf(const LT *a, const LT *d, int V, int mode, float u, float c, float max_a,
                                 float sum_a, float max_b, float sum_b, double *sh_tot, double *sh_sub, int *sh_tok,
                                 int rank, int csize)
{
    constexpr int VEC = VECTOR ? Logit<LT>::VEC : 1;
    constexpr int NWARP = K2_THREADS / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec = V / VEC;
    const int nwt = NWARP * csize, gw = rank * NWARP + warp;   // warps of the whole cluster, this warp among them
    const int per_warp = (nvec + nwt - 1) / nwt;
    const int v0 = min(gw * per_warp, nvec), v1 = min(v0 + per_warp, nvec);
    const float nma = -max_a * c, nmb = -max_b * c;
    const float ia = 1.0f / sum_a, ib = 1.0f / sum_b;

    double acc = 0.0;
    for (int i = v0 + lane; i < v1; i += 32) {
        float w[VEC];
        draw_weights<LT, VEC>(a, d, i, mode, c, nma, ia, nmb, ib, w);
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < VEC; ++e) s += w[e];
        acc += (double)s;
    }
    acc = warp_sum(acc);
    // Every CTA of the cluster is running (a peer's shared memory may not be written before that) and has
    // finished reading the slots of an earlier call.
    cluster_sync_all();
    // every CTA of the cluster gets every warp's total
    if (lane < csize) st_cluster(map_to_rank(smem_addr(&sh_tot[gw]), (uint32_t)lane), acc);
    if (tid == 0) *sh_tok = -1;
    cluster_sync_all();
    double total = 0.0;
    for (int w = 0; w < nwt; ++w) total += sh_tot[w];
    if (!(total > 0.0)) { cluster_sync_all(); return -1; }
    const double threshold = (double)u * total;
    // the warp whose range holds the crossing; rounding may leave none: then the last warp with mass
    int wstar = -1, wlast = -1;
    double base = 0.0, run = 0.0, base_last = 0.0;
    for (int w = 0; w < nwt; ++w) {
        if (sh_tot[w] > 0.0) { wlast = w; base_last = run; }
        if (wstar < 0 && run + sh_tot[w] > threshold) { wstar = w; base = run; }
        run += sh_tot[w];
    }
    if (wstar < 0) { wstar = wlast; base = base_last; }
    // second level, in the CTA that owns that range: each of its warps takes a part of it, so that the final scan
    // is a trip or two instead of a long chain of dependent loads in one warp
    if (rank == wstar / NWARP) {
    const int r0 = min(wstar * per_warp, nvec), r1 = min(r0 + per_warp, nvec);
    const int per_sub = (r1 - r0 + NWARP - 1) / NWARP;
    const int s0 = min(r0 + warp * per_sub, r1), s1 = min(s0 + per_sub, r1);
    {
        double acc2 = 0.0;
        for (int i = s0 + lane; i < s1; i += 32) {
            float w[VEC];
            draw_weights<LT, VEC>(a, d, i, mode, c, nma, ia, nmb, ib, w);
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < VEC; ++e) s += w[e];
            acc2 += (double)s;
        }
        acc2 = warp_sum(acc2);
        if (lane == 0) sh_sub[warp] = acc2;
    }
    __syncthreads();
    int sstar = -1, slast = -1;
    {
        double run2 = base, base2 = base, base2_last = base;
        for (int w = 0; w < NWARP; ++w) {
            if (sh_sub[w] > 0.0) { slast = w; base2_last = run2; }
            if (sstar < 0 && run2 + sh_sub[w] > threshold) { sstar = w; base2 = run2; }
            run2 += sh_sub[w];
        }
        if (sstar < 0) { sstar = slast; base2 = base2_last; }
        base = base2;
    }
    if (warp == sstar) {
        const int v0 = s0, v1 = s1;
        int found = -1, last_pos = -1;
        double run_base = base;
        for (int i0 = v0; i0 < v1 && found < 0; i0 += 32) {
            const int i = i0 + lane;
            float w[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) w[e] = 0.f;
            if (i < v1) draw_weights<LT, VEC>(a, d, i, mode, c, nma, ia, nmb, ib, w);
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < VEC; ++e) s += w[e];
            double incl = (double)s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                double t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            const bool crosses = run_base + incl > threshold;
            const unsigned ballot = __ballot_sync(0xFFFFFFFFu, crosses);
#pragma unroll
            for (int e = 0; e < VEC; ++e)
                if (w[e] > 0.f) last_pos = i * VEC + e;
            if (ballot) {
                const int src = __ffs(ballot) - 1;
                if (lane == src) {
                    double cum = run_base + incl - (double)s;
                    int tok = -1;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        cum += (double)w[e];
                        if (tok < 0 && cum > threshold) tok = i * VEC + e;
                    }
                    // the vector's own sum crossed, so an element does unless rounding interferes
                    if (tok < 0) {
#pragma unroll
                        for (int e = 0; e < VEC; ++e)
                            if (w[e] > 0.f) tok = i * VEC + e;
                    }
                    found = tok;
                }
                found = __shfl_sync(0xFFFFFFFFu, found, src);
            }
            run_base += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
        if (found < 0) {  // rounding left the running sum a hair under the threshold
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xFFFFFFFFu, last_pos, o));
            found = last_pos;
        }
        // every CTA of the cluster gets the token: they must all agree on whether the draw found one
        if (lane < csize) st_cluster(map_to_rank(smem_addr(sh_tok), (uint32_t)lane), (int32_t)found);
    }
    }
    cluster_sync_all();
    return *sh_tok;
}

// K2_THREADS: the draw walks one row pair per sequence, so a small batch wants large CTAs (many warps keep the
// load chains short) and a large batch wants many small ones.
template <typename LT, bool VECTOR, int K2_THREADS>
__global__ void __launch_bounds__(K2_THREADS) epilogue_kernel(const VerifyParams p)
{
    // A cluster of CTAs per sequence (1 when the batch alone fills the GPU): they share the draw's walk over a row
    // pair; everything else is evaluated alike by each of them and written by rank 0.
    const int rank = (int)cluster_rank(), csize = (int)cluster_size();
    const int b = (int)cluster_id(), tid = threadIdx.x;
    const int k = p.k, V = p.V, K = p.K;
    const float c = p.c;
    const LT *target = reinterpret_cast<const LT *>(p.target) + (size_t)b * (k + 1) * V;
    const LT *draft = draft_rows<LT>(p, b) + (size_t)b * k * V;
    const RowStats *stats = p.stats + (size_t)b * (k + 1);

    __shared__ int sh_nacc, sh_mode, sh_tok;
    __shared__ float sh_u;
    __shared__ uint32_t sh_flags;
    __shared__ double sh_reward;
    __shared__ double sh_tot[64], sh_sub[K2_THREADS / 32];   // warp totals of the cluster / of the second level
    __shared__ int sh_accept[16];
    __shared__ double sh_align[16];

    if (tid == 0) sh_flags = 0;
    __syncthreads();
    const int t = p.st.t[b];
    const int arm = p.st.arm[b];
    if (tid < k) {
        // position j = tid: the accept test of Algorithm 4 (lines 7-8)
        const int j = tid;
        const int32_t *tokens = p.tokens + (p.token_arm_stride ? (size_t)arm * p.token_arm_stride : 0) + (size_t)b * k;
        const RowStats r = stats[j];
        const uint4 words = round_words(p.seed, p.sequence_base + (uint32_t)b, (uint32_t)t, (uint32_t)j);
        const float u = uniform24(words.x);
        const int x = tokens[j];
        const bool in_range = x >= 0 && x < V;
        float p_x = 0.f, q_x = 0.f, D = 1.f;
        bool accepted = false;
        uint32_t flags = r.flags;
        double align = 0.0;
        if (!r.flags) {
            D = (float)(1.0 - r.sum_min);
            align = r.sum_min;
            if (!in_range) {
                flags |= METASD_STATUS_TOKEN_OOR;
            } else {
                p_x = ex2(fmaf(Logit<LT>::scalar(target + (size_t)j * V, x), c, -r.max_a * c)) / r.sum_a;
                q_x = ex2(fmaf(Logit<LT>::scalar(draft + (size_t)j * V, x), c, -r.max_b * c)) / r.sum_b;
                if (p.greedy) {
                    accepted = x == r.argmax_a;
                } else {
                    if (q_x == 0.f) flags |= METASD_STATUS_Q_ZERO;
                    accepted = u * q_x < p_x;  // u < min(1, p/q) without the division
                }
            }
        }
        sh_accept[j] = accepted ? 1 : 0;
        sh_align[j] = align;
        if (flags) atomicOr(&sh_flags, flags);
        if (p.diag && rank == 0) {
            metasd_diag dg;
            dg.p_x = p_x; dg.q_x = q_x; dg.D = D; dg.u = u; dg.accept = accepted ? 1 : 0;
            p.diag[(size_t)b * k + j] = dg;
        }
    }
    __syncthreads();
    if (tid == 0) {
        // first rejection (Algorithm 4, "exit for loop"), reward (Definition 2), what to draw
        int n_acc = k;
        double sum_align = 0.0;
        for (int j = k - 1; j >= 0; --j)
            if (!sh_accept[j]) n_acc = j;
        for (int j = 0; j < k; ++j) sum_align += sh_align[j];
        int mode = n_acc == k ? 2 : 1;  // 2: bonus token from p_k, 1: correction from the residual
        int tok = -1;
        const RowStats rs = stats[n_acc];
        if (n_acc == k && rs.flags) sh_flags |= rs.flags;
        if (rs.flags) {
            mode = 0;
        } else if (p.greedy) {
            mode = 0;
            tok = rs.argmax_a;
        }
        sh_nacc = n_acc;
        sh_mode = mode;
        sh_tok = tok;
        sh_u = uniform24(round_words(p.seed, p.sequence_base + (uint32_t)b, (uint32_t)t, (uint32_t)n_acc).y);
        sh_reward = p.reward_kind == METASD_REWARD_BE ? (double)n_acc / (double)k : sum_align / (double)k;
    }
    __syncthreads();

    int token = sh_tok;
    const int mode = sh_mode, n_acc = sh_nacc;
    __syncthreads();
    if (mode != 0) {
        const RowStats rs = stats[n_acc];
        const LT *a = target + (size_t)n_acc * V;
        const LT *d = mode == 1 ? draft + (size_t)n_acc * V : nullptr;
        token = block_inverse_cdf<LT, VECTOR, K2_THREADS>(a, d, V, mode, sh_u, c, rs.max_a, rs.sum_a, rs.max_b, rs.sum_b,
                                              sh_tot, sh_sub, &sh_tok, rank, csize);
        if (token < 0 && mode == 1)  // p == q in fp32 yet rejected: draw from p
            token = block_inverse_cdf<LT, VECTOR, K2_THREADS>(a, nullptr, V, 2, sh_u, c, rs.max_a, rs.sum_a, rs.max_b,
                                                  rs.sum_b, sh_tot, sh_sub, &sh_tok, rank, csize);
    }

    // Rank 0 is about to advance the sequence's round counter and arm: every CTA of the cluster must have read
    // the old ones first (they key its random numbers and pick its drafter), or the cluster would disagree.
    cluster_sync_all();
    if (tid == 0 && rank == 0) {
        const double r = sh_reward;
        p.accepted_len[b] = n_acc;
        p.next_token[b] = token;
        p.reward[b] = (float)r;
        double *sa = p.st.stat_a + (size_t)b * K, *sb = p.st.stat_b + (size_t)b * K;
        int32_t *wa = p.st.win_arm + (size_t)b * p.tau;
        double *wr = p.st.win_reward + (size_t)b * p.tau;
        bandit_update(p.bandit, K, p.gamma, p.tau, &p.st.t[b], sa, sb, wa, wr, arm, r);
        p.st.arm[b] = bandit_select(p.bandit, K, p.beta, p.gamma, p.tau, p.st.t[b], sa, sb, wa, wr, p.seed,
                                    p.sequence_base + (uint32_t)b);
        if (sh_flags) atomicOr(p.status, sh_flags);
    }
}

// -------------------------------------------------------------------------------------------
// launchers
// -------------------------------------------------------------------------------------------
template <typename LT>
static cudaError_t launch_streaming_t(const VerifyParams &p, cudaStream_t stream, uint64_t *launches)
{
    dim3 g1(p.k + 1, p.batch);
    const bool big_ctas = p.batch <= 320;   // up to about two sequences per SM
    if (p.vector_ok && p.grp_size > 1) {
        const int n_items = p.batch * (p.k + 1);
        int n_groups = p.grp_ctas / p.grp_size;
        if (n_groups > n_items) n_groups = n_items;
        cudaError_t e = cudaMemsetAsync(p.grp_count, 0, (size_t)n_items * sizeof(uint32_t), stream);
        if (e != cudaSuccess) return e;
        // the CTAs of a group wait on one another: a cooperative launch guarantees that they are co-resident
        VerifyParams q = p;
        void *args[] = {&q};
        e = cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(&split_row_stats_kernel<LT>), dim3(n_groups * p.grp_size),
                                        dim3(KS_THREADS), args, 0, stream);
        if (e != cudaSuccess) return e;
    } else if (p.vector_ok) {
        row_stats_kernel<LT, true><<<g1, K1_THREADS, 0, stream>>>(p);
    } else {
        row_stats_kernel<LT, false><<<g1, K1_THREADS, 0, stream>>>(p);
    }
    {
        // small batch: 4 CTAs of 512 threads per sequence; large batch: one CTA of 256 threads
        const unsigned csize = big_ctas ? 4u : 1u, threads = big_ctas ? 512u : 256u;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)p.batch * csize);
        cfg.blockDim = dim3(threads);
        cfg.stream = stream;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeClusterDimension;
        at.val.clusterDim.x = csize; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        cudaError_t e;
        if (!p.vector_ok) e = big_ctas ? cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, false, 512>, p)
                                       : cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, false, 256>, p);
        else e = big_ctas ? cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, true, 512>, p)
                          : cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, true, 256>, p);
        if (e != cudaSuccess) return e;
    }
    *launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_streaming(const VerifyParams &p, int dtype, cudaStream_t stream, uint64_t *launches)
{
    if (dtype == METASD_BF16) return launch_streaming_t<__nv_bfloat16>(p, stream, launches);
    return launch_streaming_t<float>(p, stream, launches);
}

cudaError_t split_prepare(int device, int dtype, int V, int *resident_ctas, int *group_size)
{
    *resident_ctas = 0;
    *group_size = 1;
    int per_sm = 0, n_sm = 0, l2 = 0, coop = 0;
    cudaError_t e;
    if (dtype == METASD_BF16)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, split_row_stats_kernel<__nv_bfloat16>, KS_THREADS, 0);
    else
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, split_row_stats_kernel<float>, KS_THREADS, 0);
    if (e != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device)) != cudaSuccess) return e;
    if (!coop || per_sm < 1) return cudaSuccess;
    const int resident = per_sm * n_sm;
    // row-pair bytes in flight = resident CTAs x (row pair / group size); keep them within a third of L2
    const double pair_bytes = 2.0 * V * (dtype == METASD_BF16 ? 2 : 4);
    const char *pin = getenv("METASD_SPLIT_GROUP");
    // measured on B200: the exchange costs more than the saved HBM traffic gains, so splitting is opt-in
    // (METASD_SPLIT_GROUP); the L2-sized default would be ceil(resident * pair_bytes / (l2 / 3))
    (void)pair_bytes; (void)l2;
    int G = pin && *pin ? atoi(pin) : 1;
    if (G < 1) G = 1;
    if (G > 16) G = 16;
    *resident_ctas = resident - resident % G;
    *group_size = G;
    return cudaSuccess;
}

// -------------------------------------------------------------------------------------------
// drafter table check
// -------------------------------------------------------------------------------------------
// Copies the caller's table of K drafter pointers into the context's own table.  An entry that is NULL or not
// aligned like the target (16 bytes on the vector path, else the element size) must never be dereferenced: it is
// flagged and replaced by the target pointer, so that the outputs of the sequences that play that drafter are
// defined (if meaningless) and nothing faults.
__global__ void sanitize_table_kernel(const void *const *table, int K, const void *target, uint32_t mask,
                                      const void **clean, uint32_t *status)
{
    const int i = threadIdx.x;
    if (i >= K) return;
    const void *q = table[i];
    if (q == nullptr || (reinterpret_cast<uintptr_t>(q) & mask) != 0) {
        atomicOr(status, METASD_STATUS_BAD_POINTER);
        q = target;
    }
    clean[i] = q;
}

cudaError_t launch_sanitize_table(const void *const *table, int K, const void *target, uint32_t mask, const void **clean,
                                  uint32_t *status, cudaStream_t stream)
{
    sanitize_table_kernel<<<1, 32, 0, stream>>>(table, K, target, mask, clean, status);
    return cudaGetLastError();
}

// -------------------------------------------------------------------------------------------
// select / reset
// -------------------------------------------------------------------------------------------
__global__ void select_kernel(BanditState st, int batch, int32_t *arm_out)
{
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) arm_out[b] = st.arm[b];
}

__global__ void reset_kernel(BanditState st, int max_batch, int K, int tau, int variant, double gamma,
                             uint32_t sequence_base, const int32_t *seq_ids, int n)
{
    int i = blockIdx.x;
    if (i >= n) return;
    int b = seq_ids ? seq_ids[i] : i;
    if (b < 0 || b >= max_batch) return;
    const double first = variant == METASD_EXP3 ? 1.0 : 0.0;   // EXP3 starts from w(i) = 1
    for (int a = threadIdx.x; a < K; a += blockDim.x) {
        st.stat_a[(size_t)b * K + a] = first;
        st.stat_b[(size_t)b * K + a] = 0.0;
    }
    for (int s = threadIdx.x; s < tau; s += blockDim.x) {
        st.win_arm[(size_t)b * tau + s] = 0;
        st.win_reward[(size_t)b * tau + s] = 0.0;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        st.t[b] = 0;
        // round 0: arm 0 of the initial sweep, or the randomised policies' draw (keyed by seed 0: no verify yet)
        st.arm[b] = bandit_select(variant, K, 0.0, gamma, tau, 0, st.stat_a + (size_t)b * K, st.stat_b + (size_t)b * K,
                                  st.win_arm + (size_t)b * tau, st.win_reward + (size_t)b * tau, 0ull,
                                  sequence_base + (uint32_t)b);
    }
}

cudaError_t launch_select(const BanditState &st, int batch, int32_t *arm_out, cudaStream_t stream)
{
    select_kernel<<<(batch + 255) / 256, 256, 0, stream>>>(st, batch, arm_out);
    return cudaGetLastError();
}

cudaError_t launch_reset(const BanditState &st, int max_batch, int K, int tau, int variant, double gamma,
                         uint32_t sequence_base, const int32_t *seq_ids, int n, cudaStream_t stream)
{
    if (n <= 0) return cudaSuccess;
    reset_kernel<<<n, 64, 0, stream>>>(st, max_batch, K, tau, variant, gamma, sequence_base, seq_ids, n);
    return cudaGetLastError();
}

}  // namespace metasd
