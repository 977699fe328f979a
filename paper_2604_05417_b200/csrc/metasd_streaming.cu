// Streaming path of the MetaSD verify round: works for every shape.
//
//   K1  row_stats_kernel   one CTA per (sequence b, position j): softmax statistics of the target
//                          row and the draft row with an online maximum, the target arg-max, then
//                          sum_v min(p_v, q_v) = 1 - d_TV(p_j, q_j) (Definition 2) in a second
//                          sweep over the same rows.  Writes one RowStats record.
//   K2  epilogue_kernel    one CTA per sequence: accept tests with the Philox uniforms (Algorithm 4,
//                          lines 7-8), first rejection, inverse-CDF draw of the correction token from
//                          max(0, p - q) or of the bonus token from p (lines 11-12), the reward, the
//                          bandit update and the next round's arm (Algorithm 2, lines 7-10).
#include "metasd_device.cuh"

namespace metasd {

constexpr int K1_THREADS = 512;
constexpr int K2_THREADS = 256;

template <typename LT>
__device__ __forceinline__ const LT *draft_rows(const VerifyParams &p, int b)
{
    if (p.draft) return reinterpret_cast<const LT *>(p.draft);
    return reinterpret_cast<const LT *>(p.drafter_ptrs[p.st.arm[b]]);
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
    for (int i = tid; i < nvec; i += K1_THREADS) {
        float xa[VEC], xb[VEC];
        if constexpr (VECTOR) {
            Logit<LT>::unpack(ld_stream(reinterpret_cast<const uint4 *>(a) + i), xa);
            if (pair) Logit<LT>::unpack(ld_stream(reinterpret_cast<const uint4 *>(d) + i), xb);
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
    __shared__ float sh_bcast[4];

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
            sh_am[0] = rm;
        }
    }
    __syncthreads();
    const float max_a = sh_bcast[0], sum_a = sh_bcast[1], max_b = sh_bcast[2], sum_b = sh_bcast[3];

    // ---- sweep 2: sum_v min(p_v, q_v)
    double total_min = 0.0;
    if (pair) {
        const float nma = -max_a * c, nmb = -max_b * c;
        const float ia = 1.0f / sum_a, ib = 1.0f / sum_b;
        float acc = 0.f;
        for (int i = tid; i < nvec; i += K1_THREADS) {
            float xa[VEC], xb[VEC];
            if constexpr (VECTOR) {
                Logit<LT>::unpack(ld_stream(reinterpret_cast<const uint4 *>(a) + i), xa);
                Logit<LT>::unpack(ld_stream(reinterpret_cast<const uint4 *>(d) + i), xb);
            } else {
                xa[0] = Logit<LT>::scalar(a, i);
                xb[0] = Logit<LT>::scalar(d, i);
            }
#pragma unroll
            for (int e = 0; e < VEC; ++e)
                acc += fminf(ex2(fmaf(xa[e], c, nma)) * ia, ex2(fmaf(xb[e], c, nmb)) * ib);
        }
        double w = warp_sum((double)acc);
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
template <typename LT, bool VECTOR>
__device__ int block_inverse_cdf(const LT *a, const LT *d, int V, int mode, float u, float c, float max_a,
                                 float sum_a, float max_b, float sum_b, double *sh_tot, int *sh_tok)
{
    constexpr int VEC = VECTOR ? Logit<LT>::VEC : 1;
    constexpr int NWARP = K2_THREADS / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec = V / VEC;
    const int per_warp = (nvec + NWARP - 1) / NWARP;
    const int v0 = min(warp * per_warp, nvec), v1 = min(v0 + per_warp, nvec);
    const float nma = -max_a * c, nmb = -max_b * c;
    const float ia = 1.0f / sum_a, ib = 1.0f / sum_b;

    __syncthreads();  // the shared slots may still be read from an earlier call
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
    if (lane == 0) sh_tot[warp] = acc;
    if (tid == 0) *sh_tok = -1;
    __syncthreads();
    double total = 0.0;
    for (int w = 0; w < NWARP; ++w) total += sh_tot[w];
    if (!(total > 0.0)) { __syncthreads(); return -1; }
    const double threshold = (double)u * total;
    // the warp whose range holds the crossing; rounding may leave none: then the last warp with mass
    int wstar = -1, wlast = -1;
    double base = 0.0, run = 0.0, base_last = 0.0;
    for (int w = 0; w < NWARP; ++w) {
        if (sh_tot[w] > 0.0) { wlast = w; base_last = run; }
        if (wstar < 0 && run + sh_tot[w] > threshold) { wstar = w; base = run; }
        run += sh_tot[w];
    }
    if (wstar < 0) { wstar = wlast; base = base_last; }
    if (warp == wstar) {
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
        if (lane == 0) *sh_tok = found;
    }
    __syncthreads();
    return *sh_tok;
}

template <typename LT, bool VECTOR>
__global__ void __launch_bounds__(K2_THREADS) epilogue_kernel(const VerifyParams p)
{
    const int b = blockIdx.x, tid = threadIdx.x;
    const int k = p.k, V = p.V, K = p.K;
    const float c = p.c;
    const LT *target = reinterpret_cast<const LT *>(p.target) + (size_t)b * (k + 1) * V;
    const LT *draft = draft_rows<LT>(p, b) + (size_t)b * k * V;
    const RowStats *stats = p.stats + (size_t)b * (k + 1);

    __shared__ int sh_nacc, sh_mode, sh_tok;
    __shared__ float sh_u;
    __shared__ uint32_t sh_flags;
    __shared__ double sh_reward;
    __shared__ double sh_tot[K2_THREADS / 32];
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
        if (p.diag) {
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
        token = block_inverse_cdf<LT, VECTOR>(a, d, V, mode, sh_u, c, rs.max_a, rs.sum_a, rs.max_b, rs.sum_b,
                                              sh_tot, &sh_tok);
        if (token < 0 && mode == 1)  // p == q in fp32 yet rejected: draw from p
            token = block_inverse_cdf<LT, VECTOR>(a, nullptr, V, 2, sh_u, c, rs.max_a, rs.sum_a, rs.max_b,
                                                  rs.sum_b, sh_tot, &sh_tok);
    }

    if (tid == 0) {
        const double r = sh_reward;
        p.accepted_len[b] = n_acc;
        p.next_token[b] = token;
        p.reward[b] = (float)r;
        double *sa = p.st.stat_a + (size_t)b * K, *sb = p.st.stat_b + (size_t)b * K;
        int32_t *wa = p.st.win_arm + (size_t)b * p.tau;
        double *wr = p.st.win_reward + (size_t)b * p.tau;
        bandit_update(p.bandit, K, p.gamma, p.tau, &p.st.t[b], sa, sb, wa, wr, arm, r);
        p.st.arm[b] = bandit_select(p.bandit, K, p.beta, p.tau, p.st.t[b], sa, sb, wa, wr);
        if (sh_flags) atomicOr(p.status, sh_flags);
    }
}

// -------------------------------------------------------------------------------------------
// launchers
// -------------------------------------------------------------------------------------------
template <typename LT>
static cudaError_t launch_streaming_t(const VerifyParams &p, cudaStream_t stream, uint64_t *launches)
{
    dim3 g1(p.k + 1, p.batch), g2(p.batch);
    if (p.vector_ok) {
        row_stats_kernel<LT, true><<<g1, K1_THREADS, 0, stream>>>(p);
        epilogue_kernel<LT, true><<<g2, K2_THREADS, 0, stream>>>(p);
    } else {
        row_stats_kernel<LT, false><<<g1, K1_THREADS, 0, stream>>>(p);
        epilogue_kernel<LT, false><<<g2, K2_THREADS, 0, stream>>>(p);
    }
    *launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_streaming(const VerifyParams &p, int dtype, cudaStream_t stream, uint64_t *launches)
{
    if (dtype == METASD_BF16) return launch_streaming_t<__nv_bfloat16>(p, stream, launches);
    return launch_streaming_t<float>(p, stream, launches);
}

// -------------------------------------------------------------------------------------------
// select / reset
// -------------------------------------------------------------------------------------------
__global__ void select_kernel(BanditState st, int batch, int32_t *arm_out)
{
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) arm_out[b] = st.arm[b];
}

__global__ void reset_kernel(BanditState st, int max_batch, int K, int tau, const int32_t *seq_ids, int n)
{
    int i = blockIdx.x;
    if (i >= n) return;
    int b = seq_ids ? seq_ids[i] : i;
    if (b < 0 || b >= max_batch) return;
    if (threadIdx.x == 0) { st.t[b] = 0; st.arm[b] = 0; }
    for (int a = threadIdx.x; a < K; a += blockDim.x) {
        st.stat_a[(size_t)b * K + a] = 0.0;
        st.stat_b[(size_t)b * K + a] = 0.0;
    }
    for (int s = threadIdx.x; s < tau; s += blockDim.x) {
        st.win_arm[(size_t)b * tau + s] = 0;
        st.win_reward[(size_t)b * tau + s] = 0.0;
    }
}

cudaError_t launch_select(const BanditState &st, int batch, int32_t *arm_out, cudaStream_t stream)
{
    select_kernel<<<(batch + 255) / 256, 256, 0, stream>>>(st, batch, arm_out);
    return cudaGetLastError();
}

cudaError_t launch_reset(const BanditState &st, int max_batch, int K, int tau, const int32_t *seq_ids, int n,
                         cudaStream_t stream)
{
    if (n <= 0) return cudaSuccess;
    reset_kernel<<<n, 64, 0, stream>>>(st, max_batch, K, tau, seq_ids, n);
    return cudaGetLastError();
}

}  // namespace metasd
