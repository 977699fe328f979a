// K1t, the row-statistics kernel with TMA-staged rows (METASD_ROWS_BULK).
//
// One persistent CTA per SM walks the launch's row pairs (sequence b, position j).  Its last warp is the producer: one
// lane issues bulk asynchronous copies (cp.async.bulk, global -> this CTA's shared memory, completion counted in bytes
// on an mbarrier; no tensor map, no multicast, this GPU's memory only) that bring a row pair on chip chunk by chunk
// into a ring of S stages.  The other warps consume the ring: every thread reads its own 16-byte vector of both rows
// from the stage, so a chunk is CT = 32 x (consumer warps) vectors of each row.
//
// Per row pair the consumers make the two sweeps of the streaming path (softmax statistics and target arg-max, then
// sum_v min(p_v, q_v) = 1 - d_TV(p_j, q_j), Definition 2 / Eq. 4):
//   sweep 1 takes chunks 0 .. n-1 as they land and gives every stage back except the last R = min(n, S) chunks;
//   sweep 2 starts on those R chunks, which are still in the ring, and goes on with chunks 0 .. n-R-1, which the
//   producer fetches again (from L2 where the rows in flight fit it) as stages come free.
// Both sweeps consume the ring in the order it was filled, so the ring is a plain FIFO: fill f sits in stage f mod S,
// the producer waits on the stage's `empty` barrier before refilling it, the consumers on its `full` barrier before
// reading it.  The copies of the next row pair start while sweep 2 of the current one drains, so the only exposed
// memory latency is that of the first chunk of a launch.
//
// Every wait is bounded: when one runs out, the CTA sets METASD_STATUS_TIMEOUT, stops waiting (and arming copies)
// everywhere and runs to its end with every barrier matched; the producer leaves only after all copies it issued
// have landed, so nothing is written into the shared memory of a CTA that has gone.
#include "metasd_device.cuh"

namespace metasd {

namespace {

struct BulkShared {
    uint64_t full[8], empty[8];
    MaxSum rec_a[2][32], rec_b[2][32];   // per consumer warp, by item parity
    ArgMax rec_am[2][32];
    MaxSum rec_own[32];                  // draft-row statistics redone relative to the row's own maximum
    double rec_min[2][32];
    int arrived[2];                      // consumer warps that have delivered their part of sum min, by item parity
    int dead;                            // a wait ran out: nobody waits any more
};

__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// The suspending form of the wait with a time hint: the hardware parks the warp until the phase is over or about
// `ns` nanoseconds have passed, so a warp that is ahead of its data costs one instruction, not a polling loop.
__device__ __forceinline__ bool mbar_try_wait_for(uint64_t *bar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// Waits until the barrier's phase of the given parity is over, for at most `limit` polls.  Limits below 16 poll
// without suspending the warp (so that a test can make a wait run out for certain); larger ones park the warp for up
// to 4 us per poll (the default limit of 2^18 polls, about a second, is far beyond any real wait and still ends).  After a time-out
// every later wait of the CTA returns at once.
__device__ __forceinline__ void wait_phase(uint64_t *bar, uint32_t parity, uint32_t limit, BulkShared &sh, uint32_t *status)
{
    if (mbar_test_wait(bar, parity)) return;
    if (*(volatile int *)&sh.dead) return;
    const bool tiny = limit < 16u;
    for (uint32_t it = 0; it < limit; ++it) {
        if (tiny ? mbar_test_wait(bar, parity) : mbar_try_wait_for(bar, parity, 4000u)) return;
    }
    *(volatile int *)&sh.dead = 1;
    atomicOr(status, METASD_STATUS_TIMEOUT);
}

__device__ __forceinline__ void bulk_load_hint(uint32_t dst, const void *src, uint32_t bytes, uint64_t *bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
        : "memory");
}

// Barrier among the consumer threads only (the producer warp never joins it).
template <int COUNT> __device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(COUNT) : "memory"); }

// Largest of the 16 bytes of logits (NaN entries are ignored, as fmaxf does).
template <typename LT>
__device__ __forceinline__ float vector_max(const uint4 &raw, const float (&x)[Logit<LT>::VEC])
{
    if constexpr (sizeof(LT) == 2) {
        const __nv_bfloat162 *w = reinterpret_cast<const __nv_bfloat162 *>(&raw);
        const __nv_bfloat162 m2 = __hmax2(__hmax2(w[0], w[1]), __hmax2(w[2], w[3]));   // two logits per instruction
        return fmaxf(__low2float(m2), __high2float(m2));
    } else {
        return fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    }
}

}  // namespace

template <typename LT, int NCW, int S, int MINB>
__global__ void __launch_bounds__((NCW + 1) * 32, MINB) row_stats_bulk_kernel(const VerifyParams p)
{
    static_assert(S >= 2 && S <= 8 && NCW >= 1 && NCW <= 31, "ring and warp counts");
    constexpr int VEC = Logit<LT>::VEC;
    constexpr int CT = NCW * 32;                       // consumer threads = vectors of a row per chunk
    constexpr uint32_t ROW_BYTES = CT * 16u, STAGE_BYTES = 2u * ROW_BYTES;
    extern __shared__ __align__(128) unsigned char ring[];   // [S][2 rows][CT] 16-byte vectors
    __shared__ BulkShared sh;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float c = p.c;
    const int nvec = p.V / VEC;
    const int n_chunk = (nvec + CT - 1) / CT;
    const int n_pairs = p.batch * p.k, n_items = n_pairs + p.batch;
    const uint32_t limit = p.poll_limit;
    const size_t row_bytes = (size_t)p.V * sizeof(LT);

    launch_dependents();   // the epilogue may be set up while this kernel runs; it waits for the whole grid before it reads
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&sh.full[s], 1);        // the producer's arrival; the copies' bytes complete the phase
            mbar_init(&sh.empty[s], NCW);     // one arrival per consumer warp
        }
        sh.arrived[0] = sh.arrived[1] = 0;
        sh.dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // Items in dispatch order: the row pairs of every sequence first, the (half-size) bonus rows last, so that the
    // launch ends on its shortest items.  false: nothing to do (a position behind the sequence's draft length).
    auto decode = [&](int it, int &b, int &j, bool &pair) -> bool {
        if (it < n_pairs) {
            b = it / p.k;
            j = it - b * p.k;
            pair = true;
            return j < drafted(p.draft_len, b, p.k);
        }
        b = it - n_pairs;
        j = drafted(p.draft_len, b, p.k);
        pair = false;
        return true;
    };

    // ------------------------------------------------------------------------------------------ producer
    if (warp == NCW) {
        if (lane != 0) return;
        const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
        const uint32_t ring_addr = smem_addr(ring);
        uint32_t fill = 0, slot = 0, phase = 0;   // fill counter, its stage and the stage's phase parity
        bool armed = true;
        for (int it = blockIdx.x; it < n_items && armed; it += gridDim.x) {
            int b, j;
            bool pair;
            if (!decode(it, b, j, pair)) continue;
            const unsigned char *a = reinterpret_cast<const unsigned char *>(p.target) + ((size_t)b * (p.k + 1) + j) * row_bytes;
            const unsigned char *d =
                pair ? reinterpret_cast<const unsigned char *>(draft_rows<LT>(p, b)) + ((size_t)b * p.k + j) * row_bytes : nullptr;
            const int retained = pair ? min(n_chunk, S) : 0;
            const int n_fill = n_chunk + (pair ? n_chunk - retained : 0);
            for (int f = 0; f < n_fill; ++f) {
                const bool first_sweep = f < n_chunk;
                const int ch = first_sweep ? f : f - n_chunk;
                wait_phase(&sh.empty[slot], phase ^ 1u, limit, sh, p.status);   // the stage's previous chunk was given back
                if (*(volatile int *)&sh.dead) { armed = false; break; }        // after a time-out nothing more is armed
                const int v0 = ch * CT;
                const uint32_t bytes = (uint32_t)(min(nvec, v0 + CT) - v0) * 16u;
                // a bonus row is read once, and so is everything the second sweep fetches: nothing of it is worth
                // keeping; of the first sweep L2 is asked to keep the end of the row, which the second fetches first
                const uint64_t pol = (first_sweep && pair && v0 >= p.keep_from_vec) ? keep : drop;
                const uint32_t dst = ring_addr + slot * STAGE_BYTES;
                mbar_arrive_expect_tx(&sh.full[slot], pair ? 2u * bytes : bytes);
                bulk_load_hint(dst, a + (size_t)v0 * 16, bytes, &sh.full[slot], pol);
                if (pair) bulk_load_hint(dst + ROW_BYTES, d + (size_t)v0 * 16, bytes, &sh.full[slot], pol);
                ++fill;
                if (++slot == S) { slot = 0; phase ^= 1u; }
            }
        }
        // No copy may still be in flight when the CTA's shared memory is given up: see the last (up to S) fills land.
        // (Without a time-out the consumers have waited for every one of them already.)
        const uint32_t outstanding = fill < (uint32_t)S ? fill : (uint32_t)S;
        for (uint32_t g = fill - outstanding; g < fill; ++g) {
            uint64_t *bar = &sh.full[g % S];
            const uint32_t par = (g / S) & 1u;
            for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(bar, par); ++it) __nanosleep(64);
        }
        return;
    }

    // ------------------------------------------------------------------------------------------ consumers
    const uint32_t my_slot_off = smem_addr(ring) + (uint32_t)tid * 16u;
    uint32_t slot = 0, phase = 0;     // stage and phase parity of the next fill to consume
    uint32_t ord = 0;                 // items this CTA has worked on: its parity selects the record buffers
    auto release = [&](uint32_t s) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[s]);
    };
    for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
        int b, j;
        bool pair;
        if (!decode(it, b, j, pair)) continue;
        const int par = ord & 1;
        ++ord;
        const int retained = pair ? min(n_chunk, S) : 0;

        // ---- sweep 1: online (max, sum) of the target row and its arg-max; the draft row's sum is taken relative to
        // the SAME running reference (a softmax sum may be taken relative to any reference that neither overflows nor
        // flushes it; whether it suited the draft row is checked after the sweep)
        MaxSum sa = {METASD_NEG_BIG, 0.f}, sb = {METASD_NEG_BIG, 0.f};
        ArgMax am = {METASD_NEG_BIG, 0x7FFFFFFF};
        uint32_t slot_r = slot, phase_r = phase;   // where the retained chunks begin (set below)
        for (int ch = 0; ch < n_chunk; ++ch) {
            if (ch == n_chunk - retained) { slot_r = slot; phase_r = phase; }
            wait_phase(&sh.full[slot], phase, limit, sh, p.status);
            const int v = ch * CT + tid;
            if (v < nvec) {
                const uint32_t src = my_slot_off + slot * STAGE_BYTES;
                const uint4 raw = lds16(src);
                float xa[VEC];
                Logit<LT>::unpack(raw, xa);
                const float cm = vector_max<LT>(raw, xa);
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
                    am.i = v * VEC + first;
                }
                const float nma = -sa.m * c;
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int e = 0; e < VEC; e += 2) {
                    s0 += ex2(fmaf(xa[e], c, nma));
                    s1 += ex2(fmaf(xa[e + 1], c, nma));
                }
                sa.s += s0 + s1;
                if (pair) {
                    float xb[VEC];
                    Logit<LT>::unpack(lds16(src + ROW_BYTES), xb);
                    float t0 = 0.f, t1 = 0.f;
#pragma unroll
                    for (int e = 0; e < VEC; e += 2) {
                        t0 += ex2(fmaf(xb[e], c, nma));
                        t1 += ex2(fmaf(xb[e + 1], c, nma));
                    }
                    sb.s += t0 + t1;
                }
            }
            if (ch < n_chunk - retained) release(slot);
            if (++slot == S) { slot = 0; phase ^= 1u; }
        }
        sb.m = sa.m;   // the draft row's sum is relative to the target row's maximum

        sa = warp_merge(sa, c);
        sb = warp_merge(sb, c);
        am = warp_argmax(am);
        if (lane == 0) { sh.rec_a[par][warp] = sa; sh.rec_b[par][warp] = sb; sh.rec_am[par][warp] = am; }
        consumer_sync<CT>();
        // every warp merges the warps' records for itself: no second barrier
        MaxSum ra = lane < NCW ? sh.rec_a[par][lane] : MaxSum{METASD_NEG_BIG, 0.f};
        MaxSum rb = lane < NCW ? sh.rec_b[par][lane] : MaxSum{METASD_NEG_BIG, 0.f};
        ArgMax rm = lane < NCW ? sh.rec_am[par][lane] : ArgMax{METASD_NEG_BIG, 0x7FFFFFFF};
        ra = warp_merge(ra, c);
        rb = warp_merge(rb, c);
        rm = warp_argmax(rm);
        // The shared reference suits the draft row when its sum is neither flushed nor overflowed: 2^-60 .. finite
        // leaves every term that matters in fp32 range.  Otherwise (draft logits far from the target's, or a row
        // that is not finite) the draft row is swept again, from memory, relative to its own running maximum.
        if (pair && !(rb.s >= 0x1p-60f && rb.s < INFINITY)) {
            const uint4 *d4 = reinterpret_cast<const uint4 *>(draft_rows<LT>(p, b) + ((size_t)b * p.k + j) * p.V);
            MaxSum own = {METASD_NEG_BIG, 0.f};
            for (int i = tid; i < nvec; i += CT) {
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
            if (lane == 0) sh.rec_own[warp] = own;
            consumer_sync<CT>();
            rb = lane < NCW ? sh.rec_own[lane] : MaxSum{METASD_NEG_BIG, 0.f};
            rb = warp_merge(rb, c);
        }
        const float max_a = ra.m, sum_a = ra.s, max_b = rb.m, sum_b = rb.s;
        const bool bad_a = !(sum_a > 0.f) || !(sum_a < INFINITY) || !(max_a < INFINITY);
        const bool bad_b = pair && (!(sum_b > 0.f) || !(sum_b < INFINITY) || !(max_b < INFINITY));
        const uint32_t flags = (bad_a || bad_b) ? METASD_STATUS_NONFINITE : 0u;
        auto write_stats = [&](double total_min) {
            RowStats r;
            r.max_a = max_a; r.sum_a = sum_a; r.max_b = max_b; r.sum_b = sum_b;
            r.argmax_a = rm.i;
            r.sum_min = flags ? 0.0 : total_min;
            r.flags = flags;
            p.stats[(size_t)b * (p.k + 1) + j] = r;
        };
        if (!pair) {
            if (tid == 0) write_stats(0.0);
            continue;
        }

        // ---- sweep 2: sum_v 2^min(ya_v, yb_v), one exponential per pair; first the chunks still in the ring, then
        // chunks 0 .. n - retained - 1 as the producer brings them back
        float offs[3];
        second_sweep_offsets(ra, rb, c, offs);
        const float nma2 = offs[0], nmb2 = offs[1], ia = offs[2];
        float acc0 = 0.f, acc1 = 0.f;
        uint32_t slot2 = slot_r, phase2 = phase_r;
        for (int i = 0; i < n_chunk; ++i) {
            const int ch = i < retained ? n_chunk - retained + i : i - retained;
            wait_phase(&sh.full[slot2], phase2, limit, sh, p.status);
            const int v = ch * CT + tid;
            if (v < nvec) {
                const uint32_t src = my_slot_off + slot2 * STAGE_BYTES;
                float xa[VEC], xb[VEC];
                Logit<LT>::unpack(lds16(src), xa);
                Logit<LT>::unpack(lds16(src + ROW_BYTES), xb);
#pragma unroll
                for (int e = 0; e < VEC; e += 2) {
                    acc0 += ex2(fminf(fmaf(xa[e], c, nma2), fmaf(xb[e], c, nmb2)));
                    acc1 += ex2(fminf(fmaf(xa[e + 1], c, nma2), fmaf(xb[e + 1], c, nmb2)));
                }
            }
            release(slot2);
            if (++slot2 == S) { slot2 = 0; phase2 ^= 1u; }
        }
        slot = slot2;
        phase = phase2;
        // the warp that delivers its part last adds the parts up, in warp order
        const double w = warp_sum((double)((acc0 + acc1) * ia));
        int last = 0;
        if (lane == 0) {
            sh.rec_min[par][warp] = w;
            __threadfence_block();
            last = atomicAdd(&sh.arrived[par], 1) == NCW - 1;
        }
        last = __shfl_sync(0xFFFFFFFFu, last, 0);
        if (last && lane == 0) {
            __threadfence_block();
            sh.arrived[par] = 0;
            double total_min = 0.0;
            for (int i = 0; i < NCW; ++i) total_min += ((volatile double *)sh.rec_min[par])[i];
            write_stats(total_min);
        }
    }
}

// ---------------------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------------------
// The built shapes: (threads per CTA including the producer warp, ring stages, CTAs per SM).
#define METASD_BULK_SHAPES(X) X(1024, 6, 1) X(1024, 7, 1) X(1024, 4, 1) X(768, 8, 1) X(512, 6, 2) X(512, 4, 2) X(512, 3, 3)

template <typename LT, int THREADS, int S, int M>
static cudaError_t prepare_shape()
{
    return cudaFuncSetAttribute(row_stats_bulk_kernel<LT, THREADS / 32 - 1, S, M>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                S * 2 * (THREADS - 32) * 16);
}

cudaError_t bulk_prepare(int dtype, RowGeometry *geo)
{
#define X(T, S, M)                                                                                       \
    if (geo->threads == T && geo->stages == S) {                                                         \
        geo->per_sm = M;                                                                                 \
        return dtype == METASD_BF16 ? prepare_shape<__nv_bfloat16, T, S, M>() : prepare_shape<float, T, S, M>(); \
    }
    METASD_BULK_SHAPES(X)
#undef X
    return cudaErrorNotSupported;
}

template <typename LT, int THREADS, int S, int M>
static cudaError_t launch_shape(const VerifyParams &p, int n_sm, cudaStream_t stream)
{
    const size_t smem = (size_t)S * 2 * (THREADS - 32) * 16;
    const long long n_items = (long long)p.batch * (p.k + 1);
    const long long resident = (long long)n_sm * M;
    const unsigned grid = (unsigned)(n_items < resident ? n_items : resident);
    row_stats_bulk_kernel<LT, THREADS / 32 - 1, S, M><<<grid, THREADS, smem, stream>>>(p);
    return cudaSuccess;
}

cudaError_t launch_row_stats_bulk(const VerifyParams &p, int dtype, const RowGeometry &geo, cudaStream_t stream)
{
#define X(T, S, M)                                                                                  \
    if (geo.threads == T && geo.stages == S)                                                        \
        return dtype == METASD_BF16 ? launch_shape<__nv_bfloat16, T, S, M>(p, geo.n_sm, stream)     \
                                    : launch_shape<float, T, S, M>(p, geo.n_sm, stream);
    METASD_BULK_SHAPES(X)
#undef X
    return cudaErrorNotSupported;
}

}  // namespace metasd
