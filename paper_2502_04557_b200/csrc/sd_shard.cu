// sd_verify for logits that arrive split along the vocabulary (a tensor-parallel LM head):
// every GPU holds columns [v0, v0 + Vs) of each p and q row.  Four local kernels, with one
// small all-gather between them (done by the caller):
//   1 shard_stats    per row and shard: (max, sum exp) of p and of q, and the logits of the
//                    draft token if it falls into this shard            -> 24 B per row
//   2 shard_decide   merges the G shard records of every row in rank order, runs the
//                    min(1, p/q) test and the first-rejection scan (same result on every GPU)
//   3 shard_weights  per sequence: this shard's share of the correction draw's weights
//                    (residual of Eq. 1 with the global normalisation, or softmax of the
//                    bonus row)                                          -> 16 B per sequence
//   4 shard_draw     every GPU finds the shard in which u * total falls; that shard's GPU
//                    locates the token, the others report -1
// No kernel waits on another CTA or on another GPU.
#include "draw_common.cuh"

namespace spr {

constexpr int kStatRecord = 6;   // floats per (row, shard): m_p, s_p, m_q, s_q, l_p[x], l_q[x]

// ------------------------------------------------------------------ 1: shard statistics
template <typename T, int ITERS, bool HAS_Q>
__device__ __forceinline__ void shard_segment(const T *prow, const T *qrow, int V, int c, MS &mp, MS &mq)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    constexpr int kSegment = kWarps * ITERS * kStep;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int first_p = c * kSegment + warp * kStep - row_pad(prow);
    const int first_q = HAS_Q ? c * kSegment + warp * kStep - row_pad(qrow) : first_p;
    stream_segment<T, ITERS, HAS_Q>(prow, qrow, first_p, first_q, V, lane, mp, mq);
}

template <typename T>
__device__ __forceinline__ float logit_at(const T *row, int x)
{
    if (sizeof(T) == 4) return reinterpret_cast<const float *>(row)[x];
    return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(row)[x]);
}

// the record of row (b, k): merged statistics and, if the draft token falls into this shard, its two logits
template <typename T>
__device__ __forceinline__ void write_record(const ShardStatsParams &prm, int64_t row, int b, int k, bool has_q,
                                             const T *prow, const T *qrow, float m_p, double z_p, float m_q, double z_q)
{
    float lpx = neg_inf(), lqx = neg_inf();
    if (has_q) {
        const int x = prm.draft_tokens[(int64_t)b * prm.K + k] - prm.v0;   // index inside the shard
        if (x >= 0 && x < prm.V) {
            lpx = logit_at<T>(prow, x);
            lqx = logit_at<T>(qrow, x);
        }
    }
    float *rec = prm.stats + row * kStatRecord;
    rec[0] = m_p;
    rec[1] = (float)z_p;
    rec[2] = m_q;
    rec[3] = (float)z_q;
    rec[4] = lpx;
    rec[5] = lqx;
}

// One CTA per (row, segment); row r = b*Kr + k (the first Kr <= Kp positions of every
// sequence) reads p row b*Kp + k and, when k < K, q row b*K + k (the bonus row k = K has no q
// row).  The CTA that finishes a row last merges its segments in segment order and writes
// the row's record.
// kSplit (many waves of CTAs): the CTA writes its segment's partial and leaves, the records
// are formed by shard_finish_kernel behind this grid (see sd_row_stats_kernel for why).
template <typename T, int ITERS, bool kSplit>
__global__ void __launch_bounds__(kThreads, 4) shard_stats_kernel(const ShardStatsParams prm)
{
    __shared__ float4 s_part[kWarps];
    __shared__ int s_last;
    const int C = prm.chunks;
    const int64_t row = blockIdx.x / C;
    const int c = blockIdx.x % C;
    const int b = (int)(row / prm.Kr), k = (int)(row % prm.Kr);
    const bool has_q = k < prm.K;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const T *prow = static_cast<const T *>(prm.p) + ((int64_t)b * prm.Kp + k) * prm.ldv;
    const T *qrow = has_q ? static_cast<const T *>(prm.q) + ((int64_t)b * prm.K + k) * prm.ldv : prow;

    MS mp{neg_inf(), 0.f}, mq{neg_inf(), 0.f};
    if (has_q) shard_segment<T, ITERS, true>(prow, qrow, prm.V, c, mp, mq);
    else shard_segment<T, ITERS, false>(prow, qrow, prm.V, c, mp, mq);
    if (kSplit) pdl_trigger();           // the finish grid may be scheduled behind this one
    mp = warp_ms(mp);
    mq = warp_ms(mq);
    if (lane == 0) s_part[warp] = make_float4(mp.m, mp.s, mq.m, mq.s);
    __syncthreads();
    if (warp != 0) return;
    {
        const float4 v = lane < kWarps ? s_part[lane] : make_float4(neg_inf(), 0.f, neg_inf(), 0.f);
        mp = warp_ms(MS{v.x, v.y});
        mq = warp_ms(MS{v.z, v.w});
    }
    if (kSplit) {
        if (lane == 0) prm.part[row * C + c] = make_float4(mp.m, mp.s, mq.m, mq.s);
        return;
    }
    float m_p = mp.m, m_q = mq.m;
    double z_p = mp.s, z_q = mq.s;
    if (C > 1) {   // (a row that one CTA covers needs no ticket and no trip through global memory)
    if (lane == 0) {
        prm.part[row * C + c] = make_float4(mp.m, mp.s, mq.m, mq.s);
        __threadfence();
        s_last = (atomicAdd(&prm.row_counters[row], 1) == C - 1);
    }
    __syncwarp();
    if (!s_last) return;

    // ---- last segment of the row: merge in segment order (fp64), write the record
    __threadfence();
    m_p = m_q = neg_inf();
    for (int cc = lane; cc < C; cc += 32) {
        const float4 v = __ldcg(&prm.part[row * C + cc]);
        m_p = fmaxf(m_p, v.x);
        m_q = fmaxf(m_q, v.z);
    }
    m_p = warp_max(m_p);
    m_q = warp_max(m_q);
    z_p = z_q = 0.0;
    for (int c0 = 0; c0 < C; c0 += 32) {
        const int cc = c0 + lane;
        double a = 0.0, bq = 0.0;
        if (cc < C) {
            const float4 v = __ldcg(&prm.part[row * C + cc]);
            a = v.y > 0.f ? (double)v.y * exp((double)v.x - (double)m_p) : 0.0;
            bq = v.w > 0.f ? (double)v.w * exp((double)v.z - (double)m_q) : 0.0;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, o);
            bq += __shfl_xor_sync(0xffffffffu, bq, o);
        }
        z_p += a;
        z_q += bq;
    }
    }
    if (lane == 0) write_record<T>(prm, row, b, k, has_q, prow, qrow, m_p, z_p, m_q, z_q);
}

// Behind a kSplit statistics grid: one thread per row merges the row's segment partials in
// segment order and writes the record.
template <typename T>
__global__ void __launch_bounds__(kThreads) shard_finish_kernel(const ShardStatsParams prm, int64_t rows)
{
    pdl_wait();                          // every partial of the statistics grid is written
    const int64_t row = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (row >= rows) return;
    const int C = prm.chunks;
    const int b = (int)(row / prm.Kr), k = (int)(row % prm.Kr);
    const bool has_q = k < prm.K;
    const T *prow = static_cast<const T *>(prm.p) + ((int64_t)b * prm.Kp + k) * prm.ldv;
    const T *qrow = has_q ? static_cast<const T *>(prm.q) + ((int64_t)b * prm.K + k) * prm.ldv : prow;
    const float4 *part = prm.part + row * C;
    float m_p = neg_inf(), m_q = neg_inf();
    for (int cc = 0; cc < C; ++cc) {
        const float4 v = __ldcg(&part[cc]);
        m_p = fmaxf(m_p, v.x);
        m_q = fmaxf(m_q, v.z);
    }
    double z_p = 0.0, z_q = 0.0;
    for (int cc = 0; cc < C; ++cc) {
        const float4 v = __ldcg(&part[cc]);
        z_p += v.y > 0.f ? (double)v.y * exp((double)v.x - (double)m_p) : 0.0;
        z_q += v.w > 0.f ? (double)v.w * exp((double)v.z - (double)m_q) : 0.0;
    }
    write_record<T>(prm, row, b, k, has_q, prow, qrow, m_p, z_p, m_q, z_q);
}

cudaError_t launch_shard_stats(const ShardStatsParams &sp, int64_t rows, int dt, cudaStream_t st)
{
    const int64_t grid = rows * sp.chunks;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (grid == 0) return cudaSuccess;
#define SPR_SHARD(T_, I_) shard_stats_kernel<T_, I_, false><<<(unsigned)grid, kThreads, 0, st>>>(sp)
    // several waves of four-step CTAs with more than one segment per row: partials only, then the finish grid
    const bool split = sp.iters == 4 && sp.chunks > 1 && grid >= 4 * 4 * 148;
    if (split) {
        if (dt == SPR_F32) shard_stats_kernel<float, 4, true><<<(unsigned)grid, kThreads, 0, st>>>(sp);
        else shard_stats_kernel<__nv_bfloat16, 4, true><<<(unsigned)grid, kThreads, 0, st>>>(sp);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((rows + kThreads - 1) / kThreads));
        cfg.blockDim = dim3(kThreads);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // scheduled while the statistics grid drains
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return dt == SPR_F32 ? cudaLaunchKernelEx(&cfg, shard_finish_kernel<float>, sp, rows)
                             : cudaLaunchKernelEx(&cfg, shard_finish_kernel<__nv_bfloat16>, sp, rows);
    }
    if (dt == SPR_F32) {
        if (sp.iters == 4) SPR_SHARD(float, 4);
        else if (sp.iters == 2) SPR_SHARD(float, 2);
        else SPR_SHARD(float, 1);
    } else {
        if (sp.iters == 4) SPR_SHARD(__nv_bfloat16, 4);
        else if (sp.iters == 2) SPR_SHARD(__nv_bfloat16, 2);
        else SPR_SHARD(__nv_bfloat16, 1);
    }
#undef SPR_SHARD
    return cudaGetLastError();
}

// ------------------------------------------------------------------ 2: decision
// (max, ln Z) of a whole row from its G shard records, in rank order
__device__ __forceinline__ void merge_shards(const float *all_stats, int64_t rows, int G, int64_t row, int off,
                                             float &M, double &lnZ)
{
    M = neg_inf();
    for (int g = 0; g < G; ++g) M = fmaxf(M, all_stats[((int64_t)g * rows + row) * kStatRecord + off]);
    double Z = 0.0;
    for (int g = 0; g < G; ++g) {
        const float *rec = all_stats + ((int64_t)g * rows + row) * kStatRecord + off;
        if (rec[1] > 0.f) Z += (double)rec[1] * exp((double)rec[0] - (double)M);
    }
    lnZ = log(Z);
}

// Whole CTA, for sequence b of B: threads take the Kp rows, then warp 0 scans the accept bits.
// Several CTAs may do this for the same sequence: they write the same values.
__device__ __forceinline__ void decide_sequence(const ShardDecideParams &prm, int b, int B)
{
    const int tid = threadIdx.x, lane = tid & 31;
    const int64_t rows = (int64_t)B * prm.Kp;
    for (int k = tid; k < prm.Kp; k += blockDim.x) {
        const int64_t row = (int64_t)b * prm.Kp + k;
        float m_p, m_q = neg_inf();
        double lnz_p, lnz_q = 0.0;
        merge_shards(prm.all_stats, rows, prm.G, row, 0, m_p, lnz_p);
        if (k < prm.K) merge_shards(prm.all_stats, rows, prm.G, row, 2, m_q, lnz_q);
        prm.rowstats[row] = make_double2((double)m_p + lnz_p, (double)m_q + lnz_q);
        if (k >= prm.K) continue;
        const int64_t tok = (int64_t)b * prm.K + k;
        const int x = prm.draft_tokens[tok];
        unsigned char acc;
        float P = -1.f, Q = -1.f;
        if (x < 0 || x >= prm.V) {
            raise_status(prm.status, SPR_ERR_BAD_TOKEN);
            acc = 2;
        } else {
            float lpx = neg_inf(), lqx = neg_inf();   // exactly one shard holds the token
            for (int g = 0; g < prm.G; ++g) {
                const float *rec = prm.all_stats + ((int64_t)g * rows + row) * kStatRecord;
                lpx = fmaxf(lpx, rec[4]);
                lqx = fmaxf(lqx, rec[5]);
            }
            const double logP = (double)lpx - (double)m_p - lnz_p;
            const double logQ = (double)lqx - (double)m_q - lnz_q;
            const double ratio = exp(logP - logQ);
            const double u = (double)prm.uniforms[(int64_t)b * (prm.K + 1) + k];
            acc = (u <= fmin(1.0, ratio)) ? 1 : 0;
            P = (float)exp(logP);
            Q = (float)exp(logQ);
        }
        prm.acc[tok] = acc;
        if (prm.accept) prm.accept[tok] = acc == 1 ? 1 : 0;
        if (prm.p_tok) prm.p_tok[tok] = P;
        if (prm.q_tok) prm.q_tok[tok] = Q;
    }
    __syncthreads();   // the CTA's own global writes are visible to it after the barrier
    if (tid >= 32) return;
    int first = prm.K;
    bool bad = false;
    for (int k0 = 0; k0 < prm.K; k0 += 32) {
        const int kk = k0 + lane;
        const unsigned v = kk < prm.K ? (unsigned)prm.acc[(int64_t)b * prm.K + kk] : 1u;
        const unsigned rej = __ballot_sync(0xffffffffu, v != 1u);
        bad |= __ballot_sync(0xffffffffu, v == 2u) != 0u;
        if (rej != 0u && first == prm.K) first = k0 + __ffs(rej) - 1;
    }
    if (lane == 0) {
        prm.accepted_len[b] = bad ? -1 : first;
        if (bad && prm.accept)
            for (int kk = 0; kk < prm.K; ++kk) prm.accept[(int64_t)b * prm.K + kk] = 0;
    }
}

__global__ void __launch_bounds__(128) shard_decide_kernel(const ShardDecideParams prm)
{
    decide_sequence(prm, blockIdx.x, gridDim.x);
}

cudaError_t launch_shard_decide(const ShardDecideParams &dp, int B, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    shard_decide_kernel<<<B, 128, 0, st>>>(dp);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ 3, 4: correction draw
// The draw of sequence b on this shard: residual at the first rejected position (weights
// normalised with the whole row's max and ln Z, so that shards add up), softmax of the
// bonus row, or none.
template <typename T>
__device__ __forceinline__ Job<T> shard_job(const ShardDrawParams &prm, int b)
{
    Job<T> job;
    job.mode = MODE_NONE;
    job.p_row = job.q_row = nullptr;
    job.cp = job.cq = job.dc = 0.f;
    job.sp = job.sq = 1.f;
    job.u = prm.uniforms[(int64_t)b * (prm.K + 1) + prm.K];
    const int nb = prm.accepted_len[b];
    const T *p = static_cast<const T *>(prm.p);
    if (nb >= 0 && nb < prm.K) {
        const double2 rs = prm.rowstats[(int64_t)b * prm.Kp + nb];
        job.mode = MODE_RESIDUAL;
        job.p_row = p + ((int64_t)b * prm.Kp + nb) * prm.ldv;
        job.q_row = static_cast<const T *>(prm.q) + ((int64_t)b * prm.K + nb) * prm.ldv;
        set_residual_scales(job, rs);
    } else if (nb == prm.K && prm.Kp == prm.K + 1) {
        job.mode = MODE_SOFTMAX;
        job.p_row = p + ((int64_t)b * prm.Kp + prm.K) * prm.ldv;
    }
    return job;
}

// One CTA per (sequence, segment) writes the step partials; the last CTA of a sequence adds
// them up: weights[b] = (largest step maximum, total weight relative to it); (0, total) for
// residual draws, (0, 0) when the sequence has no draw.
// kDecide: the kernel first takes the decision of its sequence itself (every CTA of a sequence
// does, with identical results), which saves the separate decision launch.
template <typename T, bool kDecide>
__global__ void __launch_bounds__(kThreads, 3) shard_weights_kernel(const ShardDrawParams prm,
                                                                    const ShardDecideParams dec)
{
    __shared__ DrawSmem sm;
    const int C = prm.chunks;
    const int b = blockIdx.x / C;
    const int c = blockIdx.x % C;
    const int tid = threadIdx.x;
    if (kDecide) {
        decide_sequence(dec, b, (int)(gridDim.x / C));
        __syncthreads();   // accepted_len[b] and the row statistics this CTA wrote are visible to all its threads
    }
    const Job<T> job = shard_job<T>(prm, b);
    if (job.mode == MODE_NONE) {
        if (c == 0 && tid == 0) prm.weights[b] = make_double2(0.0, 0.0);
        return;
    }
    float2 *part = prm.part + (int64_t)b * prm.steps;
    segment_pass<T>(job, job.mode, prm.V, c, prm.steps, prm.iters, part);
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        sm.last = (atomicAdd(&prm.counters[b], 1) == C - 1);
    }
    __syncthreads();
    if (!sm.last || tid >= 32) return;
    __threadfence();
    steps_total(part, prm.steps, sm);
    if (tid == 0) prm.weights[b] = make_double2(job.mode == MODE_SOFTMAX ? (double)sm.row_max : 0.0, sm.total);
}

struct OwnerSmem {
    int mode;        // MODE_NONE: this GPU reports -1
    int fallback;    // residual weights vanished on every shard: draw from p
    double target;   // what is left of u * total inside this shard, in units of exp(l - ref)
    double ref;      // softmax draws: the maximum the target is relative to
};

// One CTA per sequence.  Thread 0 adds the G shard weights in rank order and finds the shard
// where the running sum crosses u * total; only that shard's GPU goes on to locate the token.
template <typename T>
__global__ void __launch_bounds__(kThreads, 3) shard_draw_kernel(const ShardDrawParams prm)
{
    __shared__ DrawSmem sm;
    __shared__ OwnerSmem own;
    const int b = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int B = gridDim.x, G = prm.G;
    Job<T> job = shard_job<T>(prm, b);
    if (job.mode == MODE_NONE) {
        if (tid == 0) {
            prm.tokens[b] = -1;
            if (prm.residual_mass) prm.residual_mass[b] = 0.f;
        }
        return;
    }
    if (tid == 0) {
        const int nb = prm.accepted_len[b];
        int mode = job.mode, fallback = 0;
        double total = 0.0, M = 0.0;
        if (mode == MODE_RESIDUAL) {
            for (int g = 0; g < G; ++g) total += prm.all_weights[(int64_t)g * B + b].y;
            if (prm.residual_mass) prm.residual_mass[b] = (float)total;
            if (!(total > 0.0)) {   // max(0, p - q) vanished: Eq. 1 is undefined, draw from p itself
                fallback = 1;
                mode = MODE_SOFTMAX;
            }
        } else if (prm.residual_mass) {
            prm.residual_mass[b] = 0.f;
        }
        // (max, weight) of shard g for a softmax draw: from the weights pass, or, in the
        // fallback, from the row statistics every GPU already holds
        const int64_t rows = (int64_t)B * prm.Kp, row = (int64_t)b * prm.Kp + nb;
        auto shard_ms = [&](int g, double &m, double &s) {
            if (fallback) {
                const float *rec = prm.all_stats + ((int64_t)g * rows + row) * kStatRecord;
                m = (double)rec[0];
                s = (double)rec[1];
            } else {
                const double2 w = prm.all_weights[(int64_t)g * B + b];
                m = w.x;
                s = w.y;
            }
        };
        auto shard_weight = [&](int g) -> double {
            if (mode == MODE_RESIDUAL) return prm.all_weights[(int64_t)g * B + b].y;
            double m, s;
            shard_ms(g, m, s);
            return s > 0.0 ? s * exp(m - M) : 0.0;
        };
        if (mode == MODE_SOFTMAX) {
            M = -INFINITY;
            for (int g = 0; g < G; ++g) {
                double m, s;
                shard_ms(g, m, s);
                if (s > 0.0) M = fmax(M, m);
            }
            total = 0.0;
            for (int g = 0; g < G; ++g) total += shard_weight(g);
        }
        const double target = (double)job.u * total;
        double run = 0.0, before = 0.0;
        int owner = -1, last_pos = -1;
        for (int g = 0; g < G; ++g) {
            const double w = shard_weight(g);
            if (w > 0.0) last_pos = g;
            if (owner < 0 && run + w > target) {
                owner = g;
                before = run;
            }
            run += w;
        }
        double t_in = target - before;
        if (owner < 0) {   // rounding, or u >= 1: the last token with positive weight
            owner = last_pos;
            t_in = INFINITY;
        }
        own.mode = owner == prm.rank ? mode : MODE_NONE;
        own.fallback = fallback;
        own.target = t_in;
        own.ref = M;
    }
    __syncthreads();
    if (own.mode == MODE_NONE) {
        if (tid == 0) prm.tokens[b] = -1;
        return;
    }
    const int mode = own.mode;
    float2 *part = prm.part + (int64_t)b * prm.steps;
    if (own.fallback) {   // no softmax partials yet for this row: one CTA, rare
        const int C = (prm.steps + kWarps * kStatIters - 1) / (kWarps * kStatIters);
        for (int cc = 0; cc < C; ++cc) segment_pass<T>(job, mode, prm.V, cc, prm.steps, kStatIters, part);
        __syncthreads();
    }
    if (warp != 0) return;
    steps_total(part, prm.steps, sm);
    // the step partials are relative to this shard's own maximum
    const double target = mode == MODE_SOFTMAX ? own.target * exp(own.ref - (double)sm.row_max) : own.target;
    steps_cross(part, prm.steps, target, sm);
    int token = -1;
    if (sm.step >= 0) token = step_locate<T>(job, mode, prm.V, sm.step, sm.t_in, sm.ref);
    if (tid == 0) prm.tokens[b] = token >= 0 ? token + prm.v0 : -1;
}

cudaError_t launch_shard_weights(const ShardDrawParams &dp, const ShardDecideParams *dec, int B, int dt,
                                 cudaStream_t st)
{
    const int64_t grid = (int64_t)B * dp.chunks;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (grid == 0) return cudaSuccess;
    const ShardDecideParams none = {};
    if (dec) {
        if (dt == SPR_F32) shard_weights_kernel<float, true><<<(unsigned)grid, kThreads, 0, st>>>(dp, *dec);
        else shard_weights_kernel<__nv_bfloat16, true><<<(unsigned)grid, kThreads, 0, st>>>(dp, *dec);
    } else {
        if (dt == SPR_F32) shard_weights_kernel<float, false><<<(unsigned)grid, kThreads, 0, st>>>(dp, none);
        else shard_weights_kernel<__nv_bfloat16, false><<<(unsigned)grid, kThreads, 0, st>>>(dp, none);
    }
    return cudaGetLastError();
}

cudaError_t launch_shard_draw(const ShardDrawParams &dp, int B, int dt, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    if (dt == SPR_F32) shard_draw_kernel<float><<<B, kThreads, 0, st>>>(dp);
    else shard_draw_kernel<__nv_bfloat16><<<B, kThreads, 0, st>>>(dp);
    return cudaGetLastError();
}

}  // namespace spr
