// sd_verify, stage 1: softmax statistics of every (p, q) row pair, the min(1, p/q) accept test
// and the first-rejection scan.  Streams each logits row from HBM exactly once in 16-byte
// vectors; per-segment partial results go to the last CTA that finishes a row ("last block
// done" tickets: nothing ever waits on another CTA).
#include "vocab_common.cuh"

namespace spr {

// The accept test of draft position (b, k) from the merged statistics of its two rows:
// ln p(x) and ln q(x) of the draft token x in double precision, u <= min(1, p/q); writes the
// row's outputs and returns the code kept in prm.acc (1 accept, 0 reject, 2 bad token).
template <typename T>
__device__ __forceinline__ int decide_row(const SdParams &prm, int64_t row, int b, int k, const T *prow, const T *qrow,
                                          float m_p, double z_p, float m_q, double z_q)
{
    const double lnz_p = log(z_p), lnz_q = log(z_q);
    const int x = prm.draft_tokens[row];
    unsigned char acc;
    float P = -1.f, Q = -1.f;
    if (x < 0 || x >= prm.V) {
        raise_status(prm.status, SPR_ERR_BAD_TOKEN);
        acc = 2;
    } else {
        float lpx, lqx;
        if (sizeof(T) == 4) {
            lpx = reinterpret_cast<const float *>(prow)[x];
            lqx = reinterpret_cast<const float *>(qrow)[x];
        } else {
            lpx = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(prow)[x]);
            lqx = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(qrow)[x]);
        }
        const double logP = (double)lpx - (double)m_p - lnz_p;
        const double logQ = (double)lqx - (double)m_q - lnz_q;
        const double ratio = exp(logP - logQ);
        const double u = (double)prm.uniforms[(int64_t)b * (prm.K + 1) + k];
        acc = (u <= fmin(1.0, ratio)) ? 1 : 0;
        P = (float)exp(logP);
        Q = (float)exp(logQ);
    }
    prm.acc[row] = acc;
    if (prm.accept) prm.accept[row] = acc == 1 ? 1 : 0;
    if (prm.p_tok) prm.p_tok[row] = P;
    if (prm.q_tok) prm.q_tok[row] = Q;
    prm.rowstats[row] = make_double2((double)m_p + lnz_p, (double)m_q + lnz_q);
    return acc;
}

// One CTA per (row, segment): statistics of the p row and the q row over a segment of
// kWarps*kStatIters warp steps (warp w takes steps w, w+8, ...; loads for a warp's next step
// are issued before the current one is consumed).  The CTA that finishes a row last merges
// the segments, runs the accept test for that position, and the row that finishes a
// sequence last runs the first-rejection scan.
//
// kSplit (many waves of CTAs): the CTA only writes its segment's partial and leaves; the
// merge, the accept test and the scan run in sd_finish_kernel behind this grid.  In the fused
// form warp 0 of every CTA holds the CTA's registers and warp slots through a fence and an
// atomic round trip - and, for the CTA that finishes a row, two dependent trips to memory for
// the draft token's logits - during which no new CTA can start streaming on that slot: 4 % of
// the pass at the llama3 size.
template <typename T, int ITERS, bool kSplit>
__global__ void __launch_bounds__(kThreads, 4) sd_row_stats_kernel(const SdParams prm)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    constexpr int kSegment = kWarps * ITERS * kStep;      // ITERS steps per warp: 4, fewer for small batches
    __shared__ float4 s_part[kWarps];
    __shared__ int s_last;

    const int C = prm.chunks;            // segments per row
    const int64_t row = blockIdx.x / C;  // = b*K + k
    const int c = blockIdx.x % C;
    const int b = (int)(row / prm.K), k = (int)(row % prm.K);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const T *prow = static_cast<const T *>(prm.p) + ((int64_t)b * prm.Kp + k) * prm.ldv;
    const T *qrow = static_cast<const T *>(prm.q) + row * prm.ldv;
    // element index (may be negative) of this warp's first step in each row
    const int first_p = c * kSegment + warp * kStep - row_pad(prow);
    const int first_q = c * kSegment + warp * kStep - row_pad(qrow);
    const int V = prm.V;

    MS mp{neg_inf(), 0.f}, mq{neg_inf(), 0.f};
    stream_segment<T, ITERS, true>(prow, qrow, first_p, first_q, V, lane, mp, mq);
    pdl_trigger();                       // the correction draw may be scheduled behind this grid
    mp = warp_ms(mp);
    mq = warp_ms(mq);
    if (lane == 0) s_part[warp] = make_float4(mp.m, mp.s, mq.m, mq.s);
    __syncthreads();
    if (warp != 0) return;               // the other warps leave before the ticket's round trip
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
        s_last = take_ticket(&prm.row_counters[row], C);
    }
    __syncwarp();
    if (!s_last) return;

    // ---- this CTA saw the last chunk of the row: merge chunks in chunk order (warp 0)
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
    for (int c0 = 0; c0 < C; c0 += 32) {  // fixed order: chunk groups ascending, butterfly inside
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
    int last_row = 0;
    if (lane == 0) {
        decide_row<T>(prm, row, b, k, prow, qrow, m_p, z_p, m_q, z_q);
        __threadfence();
        last_row = take_ticket(&prm.seq_counters[b], prm.K);
    }
    last_row = __shfl_sync(0xffffffffu, last_row, 0);
    if (!last_row) return;

    // ---- last row of the sequence: first rejection = lowest set bit of the reject ballot
    __threadfence();
    int first = prm.K;
    bool bad = false;
    for (int k0 = 0; k0 < prm.K; k0 += 32) {
        const int kk = k0 + lane;
        const unsigned v = kk < prm.K ? (unsigned)__ldcg(&prm.acc[(int64_t)b * prm.K + kk]) : 1u;
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

// Behind a kSplit statistics grid: one warp per sequence, lane k takes draft position k (in
// rounds of 32): merges the row's segment partials in segment order, runs the accept test,
// and the warp's reject ballot gives the first rejection.  No tickets.
template <typename T>
__global__ void __launch_bounds__(kThreads) sd_finish_kernel(const SdParams prm, int B)
{
    pdl_trigger();                       // the correction draw may be scheduled behind this grid
    pdl_wait();                          // every partial of the statistics grid is written
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b >= B) return;
    const int C = prm.chunks;
    int first = prm.K;
    bool bad = false;
    for (int k0 = 0; k0 < prm.K; k0 += 32) {
        const int k = k0 + lane;
        unsigned code = 1u;
        if (k < prm.K) {
            const int64_t row = (int64_t)b * prm.K + k;
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
            const T *prow = static_cast<const T *>(prm.p) + ((int64_t)b * prm.Kp + k) * prm.ldv;
            const T *qrow = static_cast<const T *>(prm.q) + row * prm.ldv;
            code = (unsigned)decide_row<T>(prm, row, b, k, prow, qrow, m_p, z_p, m_q, z_q);
        }
        const unsigned rej = __ballot_sync(0xffffffffu, code != 1u);
        bad |= __ballot_sync(0xffffffffu, code == 2u) != 0u;
        if (rej != 0u && first == prm.K) first = k0 + __ffs(rej) - 1;
    }
    if (bad && prm.accept)
        for (int k = lane; k < prm.K; k += 32) prm.accept[(int64_t)b * prm.K + k] = 0;
    if (lane == 0) prm.accepted_len[b] = bad ? -1 : first;
}

// Optional CUDA events recorded right before and after the row-statistics kernel (the
// launch that moves almost all the bytes), so a caller can time it inside a longer step.
static thread_local cudaEvent_t g_stage_before = nullptr, g_stage_after = nullptr;
void set_stage_events(cudaEvent_t before, cudaEvent_t after)
{
    g_stage_before = before;
    g_stage_after = after;
}

constexpr int64_t kSplitMinCtas = 4 * 4 * 148;   // four waves of resident CTAs

// several waves of four-step CTAs with more than one segment per row: partials only, then the finish grid
static bool stats_split(int64_t grid, int chunks, int iters) { return iters == 4 && chunks > 1 && grid >= kSplitMinCtas; }
int sd_row_stats_launches(int B, int K, int chunks, int iters)
{
    return stats_split((int64_t)B * K * chunks, chunks, iters) ? 2 : 1;
}

cudaError_t launch_sd_row_stats(const SdParams &sp, int B, int K, int dt, cudaStream_t st)
{
    const int64_t grid = (int64_t)B * K * sp.chunks;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (grid == 0) return cudaSuccess;
    if (g_stage_before) cudaEventRecord(g_stage_before, st);
#define SPR_STATS(T_, I_) sd_row_stats_kernel<T_, I_, false><<<(unsigned)grid, kThreads, 0, st>>>(sp)
    const bool split = stats_split(grid, sp.chunks, sp.iters);
    if (split) {
        if (dt == SPR_F32) sd_row_stats_kernel<float, 4, true><<<(unsigned)grid, kThreads, 0, st>>>(sp);
        else sd_row_stats_kernel<__nv_bfloat16, 4, true><<<(unsigned)grid, kThreads, 0, st>>>(sp);
    } else if (dt == SPR_F32) {
        if (sp.iters == 4) SPR_STATS(float, 4);
        else if (sp.iters == 2) SPR_STATS(float, 2);
        else SPR_STATS(float, 1);
    } else {
        if (sp.iters == 4) SPR_STATS(__nv_bfloat16, 4);
        else if (sp.iters == 2) SPR_STATS(__nv_bfloat16, 2);
        else SPR_STATS(__nv_bfloat16, 1);
    }
#undef SPR_STATS
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && g_stage_after) cudaEventRecord(g_stage_after, st);
    if (e == cudaSuccess && split) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((B + kWarps - 1) / kWarps));
        cfg.blockDim = dim3(kThreads);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // scheduled while the statistics grid drains
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = g_stage_after ? 0 : 1;    // (an event record in between: plain stream order)
        e = dt == SPR_F32 ? cudaLaunchKernelEx(&cfg, sd_finish_kernel<float>, sp, B)
                          : cudaLaunchKernelEx(&cfg, sd_finish_kernel<__nv_bfloat16>, sp, B);
    }
    return e;
}

}  // namespace spr
