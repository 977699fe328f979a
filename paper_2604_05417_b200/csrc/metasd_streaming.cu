// Streaming path of the MetaSD verify round: works for every shape.
//
//   K1  row_stats_kernel   one CTA per (sequence b, position j): softmax statistics of the target
//                          row and the draft row with an online maximum, the target arg-max, then
//                          sum_v min(p_v, q_v) = 1 - d_TV(p_j, q_j) (Definition 2) in a second
//                          sweep over the same rows.  Writes one RowStats record.  Plain loads: any alignment.
//   K1p row_stats_staged_kernel  K1 for 16-byte aligned rows: every thread stages its own
//                          vectors through shared memory with cp.async, several trips ahead, and the second
//                          sweep starts on the trips that are still staged instead of reading them again.
//   K1t row_stats_bulk_kernel    (metasd_bulk.cu) the same two sweeps by persistent CTAs whose rows arrive as TMA
//                          bulk copies issued by one warp into a shared-memory ring.
//   K2  epilogue_kernel    one CTA per sequence: accept tests with the Philox uniforms (Algorithm 4,
//                          accept step), first rejection, inverse-CDF draw of the correction token from
//                          max(0, p - q) or of the bonus token from p (its resampling step), the reward, the
//                          bandit update and the next round's arm (Algorithm 2, update and selection steps).
#include "metasd_device.cuh"

namespace metasd {

constexpr int K1_THREADS = 512;

// -------------------------------------------------------------------------------------------
// K1
// -------------------------------------------------------------------------------------------
template <typename LT, bool VECTOR>
__global__ void __launch_bounds__(K1_THREADS) row_stats_kernel(const VerifyParams p)
{
    constexpr int VEC = VECTOR ? Logit<LT>::VEC : 1;
    constexpr int NWARP = K1_THREADS / 32;
    launch_dependents();   // the epilogue may be set up while this kernel runs; it waits for the whole grid before it reads
    const int j = blockIdx.x, b = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = p.V;
    const float c = p.c;
    const int kb = drafted(p.draft_len, b, p.k);
    if (j > kb) return;   // behind this sequence's bonus row: nothing to read
    const bool pair = j < kb;

    const LT *a = reinterpret_cast<const LT *>(p.target) + ((size_t)b * (p.k + 1) + j) * V;
    const LT *d = pair ? draft_rows<LT>(p, b) + ((size_t)b * p.k + j) * V : nullptr;
    const int nvec = V / VEC;

    // ---- sweep 1: online (max, sum) of both rows, arg-max of the target row
    MaxSum sa = {METASD_NEG_BIG, 0.f}, sb = {METASD_NEG_BIG, 0.f};
    ArgMax am = {METASD_NEG_BIG, 0x7FFFFFFF};
    const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
    const int keep_from = p.keep_from_vec;   // first 16-byte vector of a row that L2 is asked to keep (set by the host)
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
    __shared__ float sh_bcast[7];

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
            second_sweep_offsets(ra, rb, c, sh_bcast + 4);
            sh_am[0] = rm;
        }
    }
    __syncthreads();
    const float max_a = sh_bcast[0], sum_a = sh_bcast[1], max_b = sh_bcast[2], sum_b = sh_bcast[3];

    // ---- sweep 2: sum_v min(p_v, q_v) = (1 / sum_a) sum_v 2^min(ya_v, yb_v): one exponential per pair
    double total_min = 0.0;
    if (pair) {
        const float nma = sh_bcast[4], nmb = sh_bcast[5], ia = sh_bcast[6];
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
// K1p
// -------------------------------------------------------------------------------------------
// K1 with its loads staged through shared memory.  Every thread copies its own vectors D - 1 trips ahead with
// cp.async and reads them back when their group has landed; a slot is written and read by the same thread only, so
// there is no barrier and no register cost.  The second sweep visits the thread's trips in reverse: the last D trips
// of the first sweep are still in their slots and are not read from memory again, and each slot is refilled with the
// trip D further down as soon as it has been used.  Vectors and their order per thread in sweep 1 are K1's; in
// sweep 2 the partition of the row among threads differs from K1's, which only regroups an fp32 sum.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint64_t policy)
{
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

//
// CL > 1: a thread-block cluster of CL CTAs shares one row (pair), every CTA a contiguous CL-th of it.  The CTAs
// exchange their sweep-1 records through distributed shared memory (every CTA gets every record and merges them in
// rank order, so all hold the same normalisers), sweep their own part again, and rank 0 adds up the parts of
// sum min(p, q).  The same number of threads then holds a CL-th of the row pairs in flight.
template <typename LT, int D, int THREADS, int MINB, bool BONUS_LAST, int CL>
__global__ void __launch_bounds__(THREADS, MINB) row_stats_staged_kernel(const VerifyParams p)
{
    static_assert(D >= 2, "at least two stages");
    constexpr int VEC = Logit<LT>::VEC;
    constexpr int NWARP = THREADS / 32;
    constexpr uint32_t ROW_STRIDE = THREADS * 16, STAGE_STRIDE = 2 * ROW_STRIDE;
    extern __shared__ __align__(16) unsigned char stage_mem[];   // [D][2 rows][THREADS] 16-byte slots
    launch_dependents();   // the epilogue may be set up while this kernel runs; it waits for the whole grid before it reads
    // Blocks are dispatched in index order.  BONUS_LAST: the row pairs come first and the bonus rows (one row, half
    // the work) last, so that the launch ends on its shortest items (measured: better for the bf16 geometry, worse
    // for the fp32 one, which keeps the bonus rows interleaved).
    const int unit = (int)blockIdx.x / CL;                        // the row (pair) of this CTA or cluster
    const int rank = CL > 1 ? (int)cluster_rank() : 0;
    const int first_bonus = BONUS_LAST ? p.batch * p.k : 0x7FFFFFFF;
    const int b = BONUS_LAST ? (unit < first_bonus ? unit / p.k : unit - first_bonus) : unit / (p.k + 1);
    const int kb = drafted(p.draft_len, b, p.k);
    const int j = BONUS_LAST ? (unit < first_bonus ? unit - b * p.k : kb) : unit - b * (p.k + 1);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float c = p.c;
    // nothing to do behind the sequence's bonus row; with BONUS_LAST the bonus row belongs to its own late block
    // (the same for every CTA of a cluster: none of them reaches a cluster barrier)
    if (j > kb || (BONUS_LAST && unit < first_bonus && j == kb)) return;
    const bool pair = j < kb;
    // a peer's shared memory may be written once that peer is running: every CTA says so here and checks it after sweep 1
    if (CL > 1) cluster_arrive();

    const int nvec_row = p.V / VEC;
    const int v_lo = (int)((long long)nvec_row * rank / CL), v_hi = (int)((long long)nvec_row * (rank + 1) / CL);
    const uint4 *a4 = reinterpret_cast<const uint4 *>(reinterpret_cast<const LT *>(p.target) + ((size_t)b * (p.k + 1) + j) * p.V) + v_lo;
    const uint4 *d4 = pair ? reinterpret_cast<const uint4 *>(draft_rows<LT>(p, b) + ((size_t)b * p.k + j) * p.V) + v_lo : nullptr;
    const int nvec = v_hi - v_lo;   // vectors of this CTA, numbered from 0
    const int n_trip = tid < nvec ? (nvec - tid + THREADS - 1) / THREADS : 0;   // vectors of this thread
    const uint32_t slot0 = smem_addr(stage_mem) + (uint32_t)tid * 16u;

    // ---- sweep 1: online (max, sum) of the target row and its arg-max; the draft row's sum is taken relative to
    // the SAME running reference (the target's maximum so far): a softmax sum may be taken relative to any
    // reference that neither overflows nor underflows it, and sharing one spares the draft row its own maximum
    // search (the kernel is bound by instruction issue).  Whether the reference suited the draft row is checked
    // after the sweep; if not, that row's statistics are redone relative to its own maximum.
    MaxSum sa = {METASD_NEG_BIG, 0.f}, sb = {METASD_NEG_BIG, 0.f};
    ArgMax am = {METASD_NEG_BIG, 0x7FFFFFFF};
    // a bonus row is read once: nothing of it is worth keeping in L2
    const uint64_t drop = l2_policy_evict_first(), keep = pair ? l2_policy_evict_last() : drop;
    const int keep_from = p.keep_from_vec / CL;   // first 16-byte vector of this CTA's part that L2 is asked to keep
    // One group of copies per call, empty past the end: the group count stays in step with the trips.
    auto request1 = [&](int m, int slot, uint64_t pol) {
        if (m < n_trip) {
            const int i = tid + m * THREADS;
            const uint32_t dst = slot0 + (uint32_t)slot * STAGE_STRIDE;
            cp_async16(dst, a4 + i, pol);
            if (pair) cp_async16(dst + ROW_STRIDE, d4 + i, pol);
        }
        cp_async_commit();
    };
    // Trip n of sweep 1 (its vectors sit in slot n mod D): first ask for the trip D - 1 ahead.
    auto trip1 = [&](int n, int slot, uint64_t pol) {
        request1(n + D - 1, (slot + D - 1) % D, pol);
        cp_async_wait<D - 1>();   // all but the D - 1 youngest groups have landed: trip n's is among them
        const uint32_t src = slot0 + (uint32_t)slot * STAGE_STRIDE;
        const int i = tid + n * THREADS;
        float xa[VEC];
        Logit<LT>::unpack(lds16(src), xa);
        float cm = xa[0];
#pragma unroll
        for (int e = 1; e < VEC; ++e) cm = fmaxf(cm, xa[e]);
        if (cm > sa.m) {
            const float shrink = ex2((sa.m - cm) * c);
            sa.s *= shrink;
            sb.s *= shrink;
            sa.m = cm;
            int first = 0;
#pragma unroll
            for (int e = VEC - 1; e >= 0; --e)
                if (xa[e] == cm) first = e;
            am.v = cm;
            am.i = (v_lo + i) * VEC + first;
        }
        const float nma = -sa.m * c;
#pragma unroll
        for (int e = 0; e < VEC; ++e) sa.s += ex2(fmaf(xa[e], c, nma));
        if (pair) {
            float xb[VEC];
            Logit<LT>::unpack(lds16(src + ROW_STRIDE), xb);
#pragma unroll
            for (int e = 0; e < VEC; ++e) sb.s += ex2(fmaf(xb[e], c, nma));
        }
    };
    // The trips run in groups of D so that the slot of every copy and read is a constant, and in two phases so that
    // the L2 policy is one too: requests below the kept share of the row ask L2 to drop the line, the rest to keep it
    // (the boundary is rounded down to a whole group: a few vectors more are kept).
    const int m_keep = keep_from > tid ? (keep_from - tid + THREADS - 1) / THREADS : 0;   // first request that is kept
    const int groups = n_trip / D;
    int groups_drop = (m_keep - (D - 1)) / D;
    groups_drop = groups_drop < 0 ? 0 : (groups_drop > groups ? groups : groups_drop);
#pragma unroll
    for (int m = 0; m < D - 1; ++m) request1(m, m, m >= m_keep ? keep : drop);
    int n = 0;
    for (int g = 0; g < groups_drop; ++g, n += D) {
#pragma unroll
        for (int u = 0; u < D; ++u) trip1(n + u, u, drop);
    }
    for (int g = groups_drop; g < groups; ++g, n += D) {
#pragma unroll
        for (int u = 0; u < D; ++u) trip1(n + u, u, keep);
    }
#pragma unroll
    for (int u = 0; u < D - 1; ++u)
        if (n + u < n_trip) trip1(n + u, u, keep);
    cp_async_wait<0>();
    if (CL > 1) cluster_wait();
    sb.m = sa.m;   // the draft row's sum is relative to the target row's maximum

    __shared__ MaxSum sh_a[NWARP], sh_b[NWARP];
    __shared__ ArgMax sh_am[NWARP];
    __shared__ double sh_min[NWARP];
    __shared__ float sh_bcast[7];

    // records of the cluster's CTAs, written by their owners: of sweep 1, of a redone draft row, of sweep 2
    __shared__ float sh_xrec[CL][6];
    __shared__ float sh_xredo[CL][2];
    __shared__ double sh_xmin[CL];

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
        if (CL > 1) {
            // lane r hands this CTA's record to the CTA of rank r (every lane holds the merged values)
            if (lane < CL) {
                const uint32_t dst = map_to_rank(smem_addr(&sh_xrec[rank][0]), (uint32_t)lane);
                st_cluster(dst, __float_as_int(ra.m));      st_cluster(dst + 4, __float_as_int(ra.s));
                st_cluster(dst + 8, __float_as_int(rb.m));  st_cluster(dst + 12, __float_as_int(rb.s));
                st_cluster(dst + 16, __float_as_int(rm.v)); st_cluster(dst + 20, rm.i);
            }
        } else if (lane == 0) {
            sh_bcast[0] = ra.m; sh_bcast[1] = ra.s; sh_bcast[2] = rb.m; sh_bcast[3] = rb.s;
            second_sweep_offsets(ra, rb, c, sh_bcast + 4);
            sh_am[0] = rm;
        }
    }
    if (CL > 1) {
        cluster_sync_all();   // every CTA's record has arrived in every CTA
        if (tid == 0) {
            MaxSum ra = {sh_xrec[0][0], sh_xrec[0][1]}, rb = {sh_xrec[0][2], sh_xrec[0][3]};
            ArgMax rm = {sh_xrec[0][4], __float_as_int(sh_xrec[0][5])};
            for (int r = 1; r < CL; ++r) {
                ra = merge(ra, MaxSum{sh_xrec[r][0], sh_xrec[r][1]}, c);
                rb = merge(rb, MaxSum{sh_xrec[r][2], sh_xrec[r][3]}, c);
                rm = better(rm, ArgMax{sh_xrec[r][4], __float_as_int(sh_xrec[r][5])});
            }
            sh_bcast[0] = ra.m; sh_bcast[1] = ra.s; sh_bcast[2] = rb.m; sh_bcast[3] = rb.s;
            second_sweep_offsets(ra, rb, c, sh_bcast + 4);
            sh_am[0] = rm;
        }
    }
    __syncthreads();
    // The shared reference suits the draft row when its sum is neither flushed nor overflowed: 2^-60 .. finite
    // leaves every term that matters in fp32 range.  Otherwise (draft logits far from the target's, or a row
    // that is not finite) the draft row is swept again relative to its own running maximum.
    if (pair && !(sh_bcast[3] >= 0x1p-60f && sh_bcast[3] < INFINITY)) {
        __syncthreads();   // everybody has read the first verdict
        MaxSum own = {METASD_NEG_BIG, 0.f};
        for (int i = tid; i < nvec; i += THREADS) {
            float xb[VEC];
            Logit<LT>::unpack(ld_stream(d4 + i), xb);
            float bm = xb[0];
#pragma unroll
            for (int e = 1; e < VEC; ++e) bm = fmaxf(bm, xb[e]);
            if (bm > own.m) {
                own.s *= ex2((own.m - bm) * c);
                own.m = bm;
            }
            const float nmb = -own.m * c;
#pragma unroll
            for (int e = 0; e < VEC; ++e) own.s += ex2(fmaf(xb[e], c, nmb));
        }
        own = warp_merge(own, c);
        if (lane == 0) sh_b[warp] = own;
        __syncthreads();
        if (warp == 0) {
            MaxSum rb = lane < NWARP ? sh_b[lane] : MaxSum{METASD_NEG_BIG, 0.f};
            rb = warp_merge(rb, c);
            if (CL > 1) {
                if (lane < CL) {
                    const uint32_t dst = map_to_rank(smem_addr(&sh_xredo[rank][0]), (uint32_t)lane);
                    st_cluster(dst, __float_as_int(rb.m));
                    st_cluster(dst + 4, __float_as_int(rb.s));
                }
            } else if (lane == 0) {
                sh_bcast[2] = rb.m; sh_bcast[3] = rb.s;
                second_sweep_offsets(MaxSum{sh_bcast[0], sh_bcast[1]}, rb, c, sh_bcast + 4);
            }
        }
        if (CL > 1) {
            cluster_sync_all();   // the verdict above came from the merged records: every CTA of the cluster is here
            if (tid == 0) {
                MaxSum rb = {sh_xredo[0][0], sh_xredo[0][1]};
                for (int r = 1; r < CL; ++r) rb = merge(rb, MaxSum{sh_xredo[r][0], sh_xredo[r][1]}, c);
                sh_bcast[2] = rb.m; sh_bcast[3] = rb.s;
                second_sweep_offsets(MaxSum{sh_bcast[0], sh_bcast[1]}, rb, c, sh_bcast + 4);
            }
        }
        __syncthreads();
    }
    const float max_a = sh_bcast[0], sum_a = sh_bcast[1], max_b = sh_bcast[2], sum_b = sh_bcast[3];

    // ---- sweep 2, this thread's trips in reverse: sum_v 2^min(ya_v, yb_v), one exponential per pair
    double total_min = 0.0;
    if (pair) {
        const float nma = sh_bcast[4], nmb = sh_bcast[5], ia = sh_bcast[6];
        float acc = 0.f;
        // Trip n of sweep 2 from its slot; the slot is then refilled with the trip D further down.
        auto trip2 = [&](int n, int slot) {
            // the first D trips are still in their slots from sweep 1; the group of a later one was committed D trips
            // ago, so at most D - 1 younger groups may still be pending
            cp_async_wait<D - 1>();
            const uint32_t src = slot0 + (uint32_t)slot * STAGE_STRIDE;
            float xa[VEC], xb[VEC];
            Logit<LT>::unpack(lds16(src), xa);
            Logit<LT>::unpack(lds16(src + ROW_STRIDE), xb);
#pragma unroll
            for (int e = 0; e < VEC; ++e)
                acc += ex2(fminf(fmaf(xa[e], c, nma), fmaf(xb[e], c, nmb)));
            if (n >= D) {   // refill the slot just used with the trip D further down
                const int i = tid + (n - D) * THREADS;
                cp_async16(src, a4 + i, drop);
                cp_async16(src + ROW_STRIDE, d4 + i, drop);
            }
            cp_async_commit();
        };
        // the ragged top first, then whole groups downwards with constant slots
        int n = n_trip - 1;
        for (; n >= 0 && (n + 1) % D != 0; --n) trip2(n, n % D);
        for (; n >= D; n -= D) {   // n + 1 is a multiple of D and a whole group lies below: every refill is real
#pragma unroll
            for (int u = 0; u < D; ++u) trip2(n - u, D - 1 - u);
        }
        if (n >= 0) {
#pragma unroll
            for (int u = 0; u < D; ++u) trip2(n - u, D - 1 - u);
        }
        cp_async_wait<0>();
        double w = warp_sum((double)(acc * ia));
        if (lane == 0) sh_min[warp] = w;
        __syncthreads();
        if (tid == 0) {
            for (int i = 0; i < NWARP; ++i) total_min += sh_min[i];
            if (CL > 1) st_cluster(map_to_rank(smem_addr(&sh_xmin[rank]), 0u), total_min);
        }
        if (CL > 1) {
            cluster_sync_all();   // rank 0 holds every part; no CTA leaves while a peer may still write to it
            if (tid == 0) {
                total_min = 0.0;
                for (int r = 0; r < CL; ++r) total_min += sh_xmin[r];
            }
        }
    }

    if (tid == 0 && rank == 0) {
        RowStats r;
        r.max_a = max_a; r.sum_a = sum_a; r.max_b = max_b; r.sum_b = sum_b;
        r.argmax_a = sh_am[0].i;
        uint32_t flags = 0;
        const bool bad_a = !(sum_a > 0.f) || !(sum_a < INFINITY) || !(max_a < INFINITY);
        const bool bad_b = pair && (!(sum_b > 0.f) || !(sum_b < INFINITY) || !(max_b < INFINITY));
        if (bad_a || bad_b) flags |= METASD_STATUS_NONFINITE;
        r.sum_min = flags ? 0.0 : total_min;
        r.flags = flags;
        p.stats[(size_t)b * (p.k + 1) + j] = r;
    }
}

template <typename LT, int D, int THREADS, int MINB, bool BONUS_LAST, int CL>
static cudaError_t launch_staged(const VerifyParams &p, unsigned units, cudaStream_t stream)
{
    const size_t smem = (size_t)D * 2 * THREADS * 16;   // the attribute that allows it was set by streaming_prepare
    if (CL == 1) {
        row_stats_staged_kernel<LT, D, THREADS, MINB, BONUS_LAST, CL><<<units, THREADS, smem, stream>>>(p);
        return cudaSuccess;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(units * CL);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeClusterDimension;
    at.val.clusterDim.x = CL; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
    cfg.attrs = &at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, row_stats_staged_kernel<LT, D, THREADS, MINB, BONUS_LAST, CL>, p);
}

// -------------------------------------------------------------------------------------------
// K2
// -------------------------------------------------------------------------------------------
// weight of token v in the draw: MODE 1 = max(0, p_v - q_v) (correction), MODE 2 = p_v (bonus)
template <typename LT, int VEC, int MODE>
__device__ __forceinline__ void weights_of(const float (&xa)[VEC], const float (&xb)[VEC], float c, float nma, float ia,
                                           float nmb, float ib, float (&w)[VEC])
{
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const float pv = ex2(fmaf(xa[e], c, nma)) * ia;
        if (MODE == 1) {
            const float qv = ex2(fmaf(xb[e], c, nmb)) * ib;
            w[e] = fmaxf(pv - qv, 0.f);
        } else {
            w[e] = pv;
        }
    }
}

// one vector of logits as loaded (unpacked to fp32 only where it is used: registers)
template <typename LT, int VEC> struct RawVec { uint4 v; };
template <typename LT> struct RawVec<LT, 1> { float v; };

template <typename LT, int VEC>
__device__ __forceinline__ RawVec<LT, VEC> load_raw(const LT *row, int i)
{
    RawVec<LT, VEC> r;
    if constexpr (VEC > 1) r.v = ld_stream(reinterpret_cast<const uint4 *>(row) + i);
    else r.v = Logit<LT>::scalar(row, i);
    return r;
}

template <typename LT, int VEC>
__device__ __forceinline__ void unpack_raw(const RawVec<LT, VEC> &r, float (&x)[VEC])
{
    if constexpr (VEC > 1) Logit<LT>::unpack(r.v, x);
    else x[0] = r.v;
}

template <typename LT, int VEC>
__device__ __forceinline__ void draw_weights(const LT *a, const LT *d, int i, int mode, float c, float nma,
                                             float ia, float nmb, float ib, float (&w)[VEC])
{
    float xa[VEC], xb[VEC];
    unpack_raw<LT, VEC>(load_raw<LT, VEC>(a, i), xa);
    if (mode == 1) {
        unpack_raw<LT, VEC>(load_raw<LT, VEC>(d, i), xb);
        weights_of<LT, VEC, 1>(xa, xb, c, nma, ia, nmb, ib, w);
    } else {
        weights_of<LT, VEC, 2>(xa, xa, c, nma, ia, nmb, ib, w);
    }
}

// Sum of the draw's weights over the vectors [lo, hi), by one warp: lane l takes lo + l, lo + l + 32, ... and adds
// each vector's fp32 sum to its fp64 total in that order.  U vectors' loads are issued before the first is used.
template <typename LT, int VEC, int MODE, int U>
__device__ __forceinline__ double warp_range_sum_m(const LT *a, const LT *d, int lo, int hi, float c, float nma,
                                                   float ia, float nmb, float ib)
{
    const int lane = threadIdx.x & 31;
    double acc = 0.0;
    for (int i0 = lo + lane; i0 < hi; i0 += 32 * U) {
        RawVec<LT, VEC> ra[U], rb[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + 32 * u;
            if (i < hi) {
                ra[u] = load_raw<LT, VEC>(a, i);
                if (MODE == 1) rb[u] = load_raw<LT, VEC>(d, i);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + 32 * u;
            if (i < hi) {
                float xa[VEC], xb[VEC], w[VEC];
                unpack_raw<LT, VEC>(ra[u], xa);
                if (MODE == 1) unpack_raw<LT, VEC>(rb[u], xb);
                weights_of<LT, VEC, MODE>(xa, MODE == 1 ? xb : xa, c, nma, ia, nmb, ib, w);
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < VEC; ++e) s += w[e];
                acc += (double)s;
            }
        }
    }
    return warp_sum(acc);
}

template <typename LT, int VEC, int U = 4>
__device__ __forceinline__ double warp_range_sum(const LT *a, const LT *d, int lo, int hi, int mode, float c,
                                                 float nma, float ia, float nmb, float ib)
{
    return mode == 1 ? warp_range_sum_m<LT, VEC, 1, U>(a, d, lo, hi, c, nma, ia, nmb, ib)
                     : warp_range_sum_m<LT, VEC, 2, U>(a, d, lo, hi, c, nma, ia, nmb, ib);
}

// Given n <= 64 non-negative parts x[0..n) laid end to end after base0, finds the first part whose end lies beyond
// the threshold; rounding may leave none, then the last part with mass (-1 if there is none).  FRACTION: the
// threshold comes in as a fraction of the parts' sum and goes out absolute.  Returns the part, the sum of the parts
// before it plus base0 in `base`, and the sum of all parts in `total`.  Every lane of the calling warp takes part
// and gets the same answers.
template <bool FRACTION>
__device__ __forceinline__ int warp_find_part(const double *x, int n, double base0, double &threshold, double &base,
                                              double &total)
{
    const unsigned FULL = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31;
    const double x0 = lane < n ? x[lane] : 0.0, x1 = lane + 32 < n ? x[lane + 32] : 0.0;
    double i0 = x0, i1 = x1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t0 = __shfl_up_sync(FULL, i0, o), t1 = __shfl_up_sync(FULL, i1, o);
        if (lane >= o) { i0 += t0; i1 += t1; }
    }
    const double tot0 = __shfl_sync(FULL, i0, 31);
    i1 += tot0;
    total = __shfl_sync(FULL, i1, 31);
    if (FRACTION) threshold *= total;
    double e0 = __shfl_up_sync(FULL, i0, 1), e1 = __shfl_up_sync(FULL, i1, 1);
    if (lane == 0) { e0 = 0.0; e1 = tot0; }
    const unsigned c0 = __ballot_sync(FULL, lane < n && base0 + i0 > threshold);
    const unsigned c1 = __ballot_sync(FULL, lane + 32 < n && base0 + i1 > threshold);
    const unsigned m0 = __ballot_sync(FULL, x0 > 0.0), m1 = __ballot_sync(FULL, x1 > 0.0);
    int part, src;
    bool upper;
    if (c0)      { src = __ffs(c0) - 1;    upper = false; }
    else if (c1) { src = __ffs(c1) - 1;    upper = true; }
    else if (m1) { src = 31 - __clz(m1);   upper = true; }
    else if (m0) { src = 31 - __clz(m0);   upper = false; }
    else { base = base0; return -1; }
    part = src + (upper ? 32 : 0);
    const double b0 = __shfl_sync(FULL, e0, src), b1 = __shfl_sync(FULL, e1, src);
    base = base0 + (upper ? b1 : b0);
    return part;
}

// Shared-memory work space of the draw.
template <int NWARP> struct DrawShared {
    double tot[NWARP], sub[NWARP];   // warp totals of the two search levels
    double before;                   // weight in front of the token that was found
    int tok;
};

// Inverse CDF in token order over the vectors [0, v_end) of one row (pair): the smallest token v with
// sum_{w <= v} weight_w > threshold.  Every warp owns a contiguous range of vectors and sums it (fp32 weights, fp64
// sums); one warp-parallel scan finds the range that holds the crossing, the same two steps repeat inside that range,
// and the owning warp finishes with a lane scan.  FRACTION: the threshold comes in as a fraction of the range's total
// (the walk's own total, when the range is the whole row) and rounding may leave no crossing: then the last token
// with mass.  Otherwise it is absolute, and -2 says that the crossing lies behind the range.  Returns the token (-1:
// the range has no mass), the weight in front of it in `before` and the weight of the range in `total`.
template <typename LT, int VEC, int NWARP, bool FRACTION>
__device__ __forceinline__ int range_inverse_cdf(const LT *a, const LT *d, int v_end, int mode, double threshold, float c,
                                                 float nma, float ia, float nmb, float ib, DrawShared<NWARP> &sh,
                                                 double &before, double &total)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per_warp = (v_end + NWARP - 1) / NWARP;
    const int v0 = min(warp * per_warp, v_end), v1 = min(v0 + per_warp, v_end);
    const double acc = warp_range_sum<LT, VEC>(a, d, v0, v1, mode, c, nma, ia, nmb, ib);
    if (lane == 0) sh.tot[warp] = acc;
    if (tid == 0) { sh.tok = -1; sh.before = 0.0; }
    __syncthreads();
    double base;
    const int wstar = warp_find_part<FRACTION>(sh.tot, NWARP, 0.0, threshold, base, total);
    if (!(total > 0.0) || wstar < 0) { before = 0.0; return -1; }
    if (!FRACTION && !(total > threshold)) { before = total; return -2; }   // the crossing is not inside the range
    const int r0 = min(wstar * per_warp, v_end), r1 = min(r0 + per_warp, v_end);
    const int per_sub = (r1 - r0 + NWARP - 1) / NWARP;
    const int s0 = min(r0 + warp * per_sub, r1), s1 = min(s0 + per_sub, r1);
    {
        const double acc2 = warp_range_sum<LT, VEC>(a, d, s0, s1, mode, c, nma, ia, nmb, ib);
        if (lane == 0) sh.sub[warp] = acc2;
    }
    __syncthreads();
    double total2;
    const int sstar = warp_find_part<false>(sh.sub, NWARP, base, threshold, base, total2);
    if (warp == sstar) {
        int found = -1, last_pos = -1;
        double found_before = base, last_before = base;
        double run_base = base;
        for (int i0 = s0; i0 < s1 && found < 0; i0 += 32) {
            const int i = i0 + lane;
            float w[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) w[e] = 0.f;
            if (i < s1) draw_weights<LT, VEC>(a, d, i, mode, c, nma, ia, nmb, ib, w);
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
            {
                double cum = run_base + incl - (double)s;
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    if (w[e] > 0.f) { last_pos = i * VEC + e; last_before = cum; }
                    cum += (double)w[e];
                }
            }
            if (ballot) {
                const int src = __ffs(ballot) - 1;
                if (lane == src) {
                    double cum = run_base + incl - (double)s;
                    int tok = -1;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        if (tok < 0 && cum + (double)w[e] > threshold) { tok = i * VEC + e; found_before = cum; }
                        cum += (double)w[e];
                    }
                    if (tok < 0) { tok = last_pos; found_before = last_before; }
                    found = tok;
                }
                found = __shfl_sync(0xFFFFFFFFu, found, src);
                found_before = __shfl_sync(0xFFFFFFFFu, found_before, src);
            }
            run_base += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
        if (found < 0) {
            int best = last_pos;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xFFFFFFFFu, best, o));
            const unsigned who = __ballot_sync(0xFFFFFFFFu, best >= 0 && last_pos == best);
            found = best;
            if (who) found_before = __shfl_sync(0xFFFFFFFFu, last_before, __ffs(who) - 1);
        }
        if (lane == 0) { sh.tok = found; sh.before = found_before; }
    }
    __syncthreads();
    before = sh.before;
    return sh.tok;
}

// The draw of one sequence: the smallest v with sum_{w<=v} weight_w > u * total, total being the sum of all the weights
// as the walk over the whole row adds them up.  `approx_total` is the same total as the row statistics already give
// it (1 - sum_v min(p_v, q_v) for the residual, 1 for the bonus row); the two are fp32 evaluations of one sum and
// agree to within `guard` (they were never seen further apart than 2e-6, typically 2e-7, over millions of rows).
// So the first eighth of the vocabulary is searched first, with the upper end of the band u * (approx_total +- guard)
// as the threshold: a token found there whose weight in front does not reach the lower end of the band is the answer
// for every total in the band, hence the full walk's answer, and the rest of the row is never read.  Otherwise (the
// crossing lies further back, a CDF edge falls inside the band, or the total is too small for the band to mean
// anything) the whole row is walked and its own total decides.  With a frequency-sorted vocabulary most draws end in
// the probe; with the likely tokens at the end of the vocabulary none does, and the probe costs an eighth more.
template <typename LT, bool VECTOR, int K2_THREADS>
__device__ __forceinline__ int block_inverse_cdf(const LT *a, const LT *d, int V, int mode, float u, float c, float max_a, float sum_a,
                                 float max_b, float sum_b, double approx_total, DrawShared<K2_THREADS / 32> &sh)
{
    constexpr int VEC = VECTOR ? Logit<LT>::VEC : 1;
    constexpr int NWARP = K2_THREADS / 32;
    constexpr double guard = 5.0e-6;
    const int nvec = V / VEC;
    const float nma = -max_a * c, nmb = -max_b * c;
    const float ia = 1.0f / sum_a, ib = 1.0f / sum_b;
    const double lo = (double)u * (approx_total - guard), hi = (double)u * (approx_total + guard);
    double before, total;
    const int probe = (nvec / 8 + 31) & ~31;
    if (approx_total > 16.0 * guard && probe >= NWARP * 32 && probe < nvec) {
        const int tok = range_inverse_cdf<LT, VEC, NWARP, false>(a, d, probe, mode, hi, c, nma, ia, nmb, ib, sh, before, total);
        if (tok >= 0 && before <= lo) return tok;
        __syncthreads();
    }
    return range_inverse_cdf<LT, VEC, NWARP, true>(a, d, nvec, mode, (double)u, c, nma, ia, nmb, ib, sh, before, total);
}

// The draw from p alone over the whole row, for the one case that needs a second draw: the residual of a rejected
// position has no mass in fp32 (p == q to rounding).  Rare, so it is a call and not a second inlined copy.
template <typename LT, bool VECTOR, int K2_THREADS>
__device__ __noinline__ int draw_from_target(const LT *a, int V, float u, float c, float max_a, float sum_a,
                                             DrawShared<K2_THREADS / 32> &sh)
{
    constexpr int VEC = VECTOR ? Logit<LT>::VEC : 1;
    double before, total;
    return range_inverse_cdf<LT, VEC, K2_THREADS / 32, true>(a, nullptr, V / VEC, 2, (double)u, c, -max_a * c, 1.0f / sum_a, 0.f,
                                                             0.f, sh, before, total);
}

// Blocks until the kernel launched before this one in the stream has finished and its writes are visible (a no-op
// when this kernel was launched without programmatic stream serialisation).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// K2_THREADS: the draw walks (part of) one row pair per sequence, so a small batch wants large CTAs (many warps keep the
// load chains short) and a large batch wants many small ones.  512 threads per SM in either shape: the draw keeps a
// dozen fp64 running values next to its loads in flight and wants about 100 registers per thread.
template <typename LT, bool VECTOR, int K2_THREADS>
__global__ void __launch_bounds__(K2_THREADS, 1024 / K2_THREADS) epilogue_kernel(const VerifyParams p)
{
    const int b = blockIdx.x, tid = threadIdx.x;
    const int k_slots = p.k, V = p.V, K = p.K;   // rows and tokens are laid out for k_slots positions per sequence
    const float c = p.c;

    __shared__ int sh_nacc, sh_mode, sh_tok;
    __shared__ float sh_u;
    __shared__ uint32_t sh_flags;
    __shared__ double sh_reward;
    __shared__ DrawShared<K2_THREADS / 32> sh_draw;
    __shared__ int sh_accept[16];
    __shared__ double sh_align[16];

    // The row-statistics kernel may still be running when this kernel starts (programmatic stream serialisation):
    // nothing it writes is read, and nothing it reads is written, before this wait.
    grid_dependency_wait();

    const int k = drafted(p.draft_len, b, k_slots);   // positions this sequence drafted this round
    const LT *target = reinterpret_cast<const LT *>(p.target) + (size_t)b * (k_slots + 1) * V;
    const LT *draft = draft_rows<LT>(p, b) + (size_t)b * k_slots * V;
    const RowStats *stats = p.stats + (size_t)b * (k_slots + 1);

    if (tid == 0) sh_flags = (p.draft_len && p.draft_len[b] != k) ? METASD_STATUS_BAD_LENGTH : 0u;
    __syncthreads();
    // pointer-table mode: an entry that must not be dereferenced is flagged once per call, played or not
    if (b == 0 && p.drafter_ptrs && tid < K) {
        const void *q = p.drafter_ptrs[tid];
        if (q == nullptr || (reinterpret_cast<uintptr_t>(q) & p.table_mask) != 0) atomicOr(&sh_flags, METASD_STATUS_BAD_POINTER);
    }
    const int t = p.st.t[b];
    const int arm = p.st.arm[b];
    if (tid < k) {
        // position j = tid: the accept test of Algorithm 4
        const int j = tid;
        const int32_t *tokens = p.tokens + (p.token_arm_stride ? (size_t)arm * p.token_arm_stride : 0) + (size_t)b * k_slots;
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
        if (p.diag) {
            metasd_diag dg;
            dg.p_x = p_x; dg.q_x = q_x; dg.D = D; dg.u = u; dg.accept = accepted ? 1 : 0;
            p.diag[(size_t)b * k_slots + j] = dg;
        }
    }
    __syncthreads();
    if (tid == 0) {
        // first rejection (Algorithm 4, the rejection step ends the loop), reward (Definition 2), what to draw
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
    if (mode != 0) {
        const RowStats rs = stats[n_acc];
        const LT *a = target + (size_t)n_acc * V;
        const LT *d = mode == 1 ? draft + (size_t)n_acc * V : nullptr;
        // the total of the draw's weights as the row statistics give it: sum max(0, p - q) = 1 - sum min(p, q); sum p = 1
        const double known = mode == 1 ? 1.0 - rs.sum_min : 1.0;
        token = block_inverse_cdf<LT, VECTOR, K2_THREADS>(a, d, V, mode, sh_u, c, rs.max_a, rs.sum_a, rs.max_b, rs.sum_b,
                                                          known, sh_draw);
        if (token < 0 && mode == 1) {  // p == q in fp32 yet rejected (the residual has no mass): draw from p
            __syncthreads();   // every thread has read the first draw's answer before the work space is reused
            token = draw_from_target<LT, VECTOR, K2_THREADS>(a, V, sh_u, c, rs.max_a, rs.sum_a, sh_draw);
        }
    }

    if (tid < 32) {
        // the bandit of this sequence: update with the reward, then the next round's arm (one lane per drafter)
        const double r = sh_reward;
        double *sa = p.st.stat_a + (size_t)b * K, *sb = p.st.stat_b + (size_t)b * K;
        int32_t *wa = p.st.win_arm + (size_t)b * p.tau;
        double *wr = p.st.win_reward + (size_t)b * p.tau;
        warp_bandit_step(p.bandit, K, p.beta, p.gamma, p.tau, &p.st.t[b], &p.st.arm[b], sa, sb, wa, wr, arm, r, p.seed,
                         p.sequence_base + (uint32_t)b);
        if (tid == 0) {
            p.accepted_len[b] = n_acc;
            p.next_token[b] = token;
            p.reward[b] = (float)r;
            if (sh_flags) atomicOr(p.status, sh_flags);
        }
    }
}

// -------------------------------------------------------------------------------------------
// launchers
// -------------------------------------------------------------------------------------------
// The built shapes of the staged kernel, per logit type: (threads, stages, CTAs per SM, bonus rows last, CTAs per row).
#define METASD_STAGED_SHAPES(X) \
    X(512, 4, 3, true, 1) X(1024, 6, 1, false, 1) X(1024, 4, 1, true, 1) X(768, 4, 2, true, 1) X(384, 4, 4, true, 1) \
    X(512, 4, 3, true, 3) X(512, 4, 3, true, 2) X(768, 4, 2, true, 2)

template <typename LT, int D, int THREADS, int MINB, bool BONUS_LAST, int CL>
static cudaError_t prepare_staged()
{
    return cudaFuncSetAttribute(row_stats_staged_kernel<LT, D, THREADS, MINB, BONUS_LAST, CL>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, D * 2 * THREADS * 16);
}

template <typename LT>
static cudaError_t prepare_staged_t(int threads, int stages, int cluster, int *per_sm)
{
#define X(T, D, M, BL, C) if (threads == T && stages == D && cluster == C) { *per_sm = M; return prepare_staged<LT, D, T, M, BL, C>(); }
    METASD_STAGED_SHAPES(X)
#undef X
    return cudaErrorNotSupported;
}

template <typename LT>
static cudaError_t launch_staged_t(const VerifyParams &p, const RowGeometry &geo, cudaStream_t stream)
{
    const unsigned units = (unsigned)p.batch * (unsigned)(p.k + 1);
#define X(T, D, M, BL, C) if (geo.threads == T && geo.stages == D && geo.cluster == C) return launch_staged<LT, D, T, M, BL, C>(p, units, stream);
    METASD_STAGED_SHAPES(X)
#undef X
    return cudaErrorNotSupported;
}

// Resolves the row-statistics shape for a context and sets the launch attributes its kernels need, once.
// Measured on B200: bf16 rows (8 logits per 16 bytes) are bound by arithmetic as much as by memory, fp32 rows (4 logits
// per 16 bytes) by memory: they want few row pairs in flight and a large share of each kept in shared memory.
cudaError_t streaming_prepare(int device, int dtype, const metasd_config &cfg, RowGeometry *geo)
{
    cudaError_t e = cudaDeviceGetAttribute(&geo->n_sm, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return e;
    geo->kernel = cfg.row_kernel == METASD_ROWS_AUTO ? METASD_ROWS_STAGED : cfg.row_kernel;
    geo->threads = cfg.row_threads;
    geo->stages = cfg.row_stages;
    geo->per_sm = 1;
    geo->cluster = 1;
    if (cfg.row_cluster > 1 && geo->kernel != METASD_ROWS_STAGED) return cudaErrorNotSupported;   // only the staged kernel has a cluster form
    if (geo->kernel == METASD_ROWS_PLAIN) {
        if (geo->threads && geo->threads != K1_THREADS) return cudaErrorNotSupported;
        geo->threads = K1_THREADS;
        geo->stages = 0;
        geo->per_sm = 3;
        return cudaSuccess;
    }
    if (geo->kernel == METASD_ROWS_BULK) {
        if (!geo->threads) geo->threads = 1024;
        if (!geo->stages) geo->stages = 6;
        return bulk_prepare(dtype, geo);
    }
    if (geo->kernel != METASD_ROWS_STAGED) return cudaErrorNotSupported;
    if (!geo->threads) geo->threads = dtype == METASD_BF16 ? 512 : 1024;
    if (!geo->stages) geo->stages = dtype == METASD_BF16 ? 4 : 6;
    geo->cluster = cfg.row_cluster > 1 ? cfg.row_cluster : 1;
    return dtype == METASD_BF16 ? prepare_staged_t<__nv_bfloat16>(geo->threads, geo->stages, geo->cluster, &geo->per_sm)
                                : prepare_staged_t<float>(geo->threads, geo->stages, geo->cluster, &geo->per_sm);
}

template <typename LT>
static cudaError_t launch_streaming_t(const VerifyParams &p, const RowGeometry &geo, cudaStream_t stream, uint64_t *launches)
{
    cudaError_t e = cudaSuccess;
    if (!p.vector_ok) {
        row_stats_kernel<LT, false><<<dim3(p.k + 1, p.batch), K1_THREADS, 0, stream>>>(p);
    } else if (geo.kernel == METASD_ROWS_BULK) {
        e = launch_row_stats_bulk(p, sizeof(LT) == 2 ? METASD_BF16 : METASD_FP32, geo, stream);
    } else if (geo.kernel == METASD_ROWS_STAGED) {
        e = launch_staged_t<LT>(p, geo, stream);
    } else {
        row_stats_kernel<LT, true><<<dim3(p.k + 1, p.batch), K1_THREADS, 0, stream>>>(p);
    }
    if (e != cudaSuccess) return e;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // The epilogue is launched with programmatic stream serialisation: its blocks may be set up while the
    // row-statistics kernel drains, and wait (griddepcontrol.wait) for its completion before they read anything.
    const bool big_ctas = p.batch <= 320;   // up to about one sequence per SM
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.batch);
    cfg.blockDim = dim3(big_ctas ? 512u : 256u);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &at;
    cfg.numAttrs = 1;
    if (!p.vector_ok) {
        if (big_ctas) e = cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, false, 512>, p);
        else e = cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, false, 256>, p);
    } else {
        if (big_ctas) e = cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, true, 512>, p);
        else e = cudaLaunchKernelEx(&cfg, epilogue_kernel<LT, true, 256>, p);
    }
    *launches += 2;
    return e;
}

cudaError_t launch_streaming(const VerifyParams &p, int dtype, const RowGeometry &geo, cudaStream_t stream, uint64_t *launches)
{
    if (dtype == METASD_BF16) return launch_streaming_t<__nv_bfloat16>(p, geo, stream, launches);
    return launch_streaming_t<float>(p, geo, stream, launches);
}

// -------------------------------------------------------------------------------------------
// select / reset
// -------------------------------------------------------------------------------------------
// The arm of the coming round was chosen at the end of the previous epilogue: selecting is a copy.  (A kernel, not a
// device-to-device cudaMemcpyAsync: measured on the launch-bound configurations the copy-engine hop cost more.)
__global__ void select_kernel(const int32_t *arm, int batch, int32_t *arm_out)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) arm_out[b] = arm[b];
}

cudaError_t launch_select(const BanditState &st, int batch, int32_t *arm_out, cudaStream_t stream)
{
    select_kernel<<<(batch + 255) / 256, 256, 0, stream>>>(st.arm, batch, arm_out);
    return cudaGetLastError();
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
        st.stat_b[(size_t)b * K + a] = variant == METASD_PETC ? 1.0 : 0.0;   // PETC: every drafter starts in the set
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

cudaError_t launch_reset(const BanditState &st, int max_batch, int K, int tau, int variant, double gamma,
                         uint32_t sequence_base, const int32_t *seq_ids, int n, cudaStream_t stream)
{
    if (n <= 0) return cudaSuccess;
    reset_kernel<<<n, 64, 0, stream>>>(st, max_batch, K, tau, variant, gamma, sequence_base, seq_ids, n);
    return cudaGetLastError();
}

}  // namespace metasd
