// Vocabulary-wide kernels: softmax statistics, the min(1, p/q) accept test, the
// first-rejection scan, and inverse-CDF draws from softmax(l) or from the residual
// norm(max(0, p - q)) of Eq. 1.  All of them stream each logits row from HBM once in
// 16-byte vectors, keep probabilities in registers only, and hand per-chunk partial
// results to the last CTA that finishes a row ("last block done" tickets: nothing ever
// waits on another CTA).
#include <limits.h>

#include "common.cuh"
#include "launch.h"

namespace spr {

// ---------------------------------------------------------------- 16-byte vectors
template <typename T>
struct Vec;

template <>
struct Vec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[N])
    {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ float vmax(const uint4 &v)
    {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)),
                     fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    // elements i0 .. i0+3 of the row, -inf where the index falls outside [0, V)
    static __device__ __forceinline__ uint4 gather(const float *row, int i0, int V)
    {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int i = i0 + e;
            w[e] = (i >= 0 && i < V) ? __float_as_uint(row[i]) : 0xff800000u;
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

template <>
struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[N])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            f[2 * j] = __uint_as_float(w[j] << 16);
            f[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ float vmax(const uint4 &v)
    {
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&v.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&v.y);
        const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162 *>(&v.z);
        const __nv_bfloat162 d = *reinterpret_cast<const __nv_bfloat162 *>(&v.w);
        const __nv_bfloat162 m = __hmax2(__hmax2(a, b), __hmax2(c, d));
        return fmaxf(__low2float(m), __high2float(m));
    }
    static __device__ __forceinline__ uint4 gather(const __nv_bfloat16 *row, int i0, int V)
    {
        const unsigned short *r = reinterpret_cast<const unsigned short *>(row);
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int a = i0 + 2 * j, b = a + 1;
            const uint32_t lo = (a >= 0 && a < V) ? (uint32_t)r[a] : 0xff80u;
            const uint32_t hi = (b >= 0 && b < V) ? (uint32_t)r[b] : 0xff80u;
            w[j] = lo | (hi << 16);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Elements i0 .. i0+N-1 of a row as one vector.  One 16-byte load when the vector lies
// inside the row and its address is 16-byte aligned, element loads with -inf fill otherwise.
template <typename T>
__device__ __forceinline__ uint4 load_vec(const T *__restrict__ row, int i0, int V)
{
    constexpr int N = Vec<T>::N;
    if (i0 >= 0 && i0 + N <= V && (reinterpret_cast<uintptr_t>(row + i0) & 15) == 0)
        return ld_stream(reinterpret_cast<const uint4 *>(row + i0));
    if (i0 + N <= 0 || i0 >= V) {
        const uint32_t f = sizeof(T) == 4 ? 0xff800000u : 0xff80ff80u;
        return make_uint4(f, f, f, f);
    }
    return Vec<T>::gather(row, i0, V);
}

// Number of elements by which the row start lies past a 16-byte boundary.  Vector j of
// thread t in chunk c starts at element (c*CH + (j*256 + t)*N) - pad of the row, which makes
// every interior vector 16-byte aligned whatever the row's own alignment.
template <typename T>
__device__ __forceinline__ int row_pad(const T *row)
{
    return (int)((reinterpret_cast<uintptr_t>(row) & 15) / sizeof(T));
}

template <typename T>
__device__ __forceinline__ int vec_start(int c, int j, int tid, int pad)
{
    constexpr int N = Vec<T>::N;
    return c * (kThreads * kUnroll * N) + (j * kThreads + tid) * N - pad;
}

// (max, sum of exp(x - max)) over the kUnroll vectors a thread holds
template <typename T>
__device__ __forceinline__ MS thread_ms(const uint4 (&raw)[kUnroll])
{
    constexpr int N = Vec<T>::N;
    float m = Vec<T>::vmax(raw[0]);
#pragma unroll
    for (int j = 1; j < kUnroll; ++j) m = fmaxf(m, Vec<T>::vmax(raw[j]));
    const float ref = (m == neg_inf()) ? 0.f : m;
    const float off = -ref * kLog2e;
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float f[N];
        Vec<T>::unpack(raw[j], f);
#pragma unroll
        for (int e = 0; e < N; ++e) s += ex2(fmaf(f[e], kLog2e, off));
    }
    MS r;
    r.m = m;
    r.s = s;
    return r;
}

// ================================================================ sd_verify, stage 1
// Lane-local online softmax statistics: folds kUnroll vectors into a running (max, sum of
// exp(x - max)).  When the maximum grows the old sum is rescaled once per call.
template <typename T>
__device__ __forceinline__ void online_update(const uint4 (&raw)[kUnroll], float &m, float &s)
{
    constexpr int N = Vec<T>::N;
    float g = Vec<T>::vmax(raw[0]);
#pragma unroll
    for (int j = 1; j < kUnroll; ++j) g = fmaxf(g, Vec<T>::vmax(raw[j]));
    const float mn = fmaxf(m, g);
    const float ref = (mn == neg_inf()) ? 0.f : mn;
    const float off = -ref * kLog2e;
    float acc[kUnroll];
    acc[0] = s * ex2(fmaf(m, kLog2e, off));   // m = -inf: exp2(-inf) = 0
#pragma unroll
    for (int j = 1; j < kUnroll; ++j) acc[j] = 0.f;
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float f[N];
        Vec<T>::unpack(raw[j], f);
#pragma unroll
        for (int e = 0; e < N; ++e) acc[j] += ex2(fmaf(f[e], kLog2e, off));
    }
    m = mn;
    s = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

// The kUnroll vectors of one warp step: vector j of lane l starts at element
// first + (j*32 + l)*N of the row (first may be negative or run past V at the row's ends).
template <typename T>
__device__ __forceinline__ void load_step(const T *__restrict__ row, int first, int V, int lane,
                                          uint4 (&raw)[kUnroll])
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    if (first >= 0 && first + kStep <= V) {   // interior: aligned by construction
        const uint4 *p = reinterpret_cast<const uint4 *>(row + first) + lane;
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) raw[j] = ld_stream(p + j * 32);
    } else {
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) raw[j] = load_vec<T>(row, first + (j * 32 + lane) * N, V);
    }
}

// One CTA per (row, segment): statistics of the p row and the q row over a segment of
// kWarps*kStatIters warp steps (warp w takes steps w, w+8, ...; loads for a warp's next step
// are issued before the current one is consumed).  The CTA that finishes a row last merges
// the segments, runs the accept test for that position, and the row that finishes a
// sequence last runs the first-rejection scan.
template <typename T>
__global__ void __launch_bounds__(kThreads) sd_row_stats_kernel(const SdParams prm)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    constexpr int kSegment = kWarps * kStatIters * kStep;
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
    uint4 rp[kUnroll], rq[kUnroll];
    load_step<T>(prow, first_p, V, lane, rp);
    load_step<T>(qrow, first_q, V, lane, rq);
#pragma unroll
    for (int it = 0; it < kStatIters; ++it) {
        const int nxt = (it + 1) * kWarps * kStep;
        const bool more = it + 1 < kStatIters && min(first_p, first_q) + nxt < V;   // warp-uniform
        online_update<T>(rp, mp.m, mp.s);
        if (more) load_step<T>(prow, first_p + nxt, V, lane, rp);
        online_update<T>(rq, mq.m, mq.s);
        if (more) load_step<T>(qrow, first_q + nxt, V, lane, rq);
        if (!more) break;
    }
    mp = warp_ms(mp);
    mq = warp_ms(mq);
    if (lane == 0) s_part[warp] = make_float4(mp.m, mp.s, mq.m, mq.s);
    __syncthreads();
    if (warp == 0) {
        float4 v = lane < kWarps ? s_part[lane] : make_float4(neg_inf(), 0.f, neg_inf(), 0.f);
        mp = warp_ms(MS{v.x, v.y});
        mq = warp_ms(MS{v.z, v.w});
        if (lane == 0) {
            prm.part[row * C + c] = make_float4(mp.m, mp.s, mq.m, mq.s);
            __threadfence();
            const int ticket = atomicAdd(&prm.row_counters[row], 1);
            s_last = (ticket == C - 1);
        }
    }
    __syncthreads();
    if (!s_last || warp != 0) return;

    // ---- this CTA saw the last chunk of the row: merge chunks in chunk order (warp 0)
    __threadfence();
    float m_p = neg_inf(), m_q = neg_inf();
    for (int cc = lane; cc < C; cc += 32) {
        const float4 v = __ldcg(&prm.part[row * C + cc]);
        m_p = fmaxf(m_p, v.x);
        m_q = fmaxf(m_q, v.z);
    }
    m_p = warp_max(m_p);
    m_q = warp_max(m_q);
    double z_p = 0.0, z_q = 0.0;
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
    int last_row = 0;
    if (lane == 0) {
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
        prm.rowstats[row] = make_float4(m_p, (float)lnz_p, m_q, (float)lnz_q);
        __threadfence();
        last_row = (atomicAdd(&prm.seq_counters[b], 1) == prm.K - 1);
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

// ================================================================ inverse-CDF draws
enum { MODE_NONE = 0, MODE_SOFTMAX = 1, MODE_RESIDUAL = 2 };

template <typename T>
struct Job {
    int mode;
    const T *p_row;
    const T *q_row;
    float cp, cq;  // residual: (max + ln Z) * log2(e) of the p row and of the q row
    float u;
};

template <typename T>
__device__ __forceinline__ Job<T> resolve_job(const DrawParams &prm, int i)
{
    Job<T> job;
    job.mode = MODE_NONE;
    job.p_row = job.q_row = nullptr;
    job.cp = job.cq = 0.f;
    job.u = 0.f;
    const T *p = static_cast<const T *>(prm.p);
    if (prm.kind == DRAW_REPLACE) {
        int off = 0;
        if (prm.gate) {
            off = prm.gate[i];
            if (off >= prm.K) return job;  // verifier kept every token: the target is not called
        }
        const int64_t row = (prm.rows ? (int64_t)prm.rows[i] : (int64_t)i * prm.seq_stride) + off;
        if (row < 0 || row >= prm.R) {
            raise_status(prm.status, SPR_ERR_BAD_ROW);
            return job;
        }
        job.mode = MODE_SOFTMAX;
        job.p_row = p + row * prm.ldv;
        job.u = prm.uniforms[i];
    } else {
        const int nb = prm.accepted_len[i];
        if (nb < 0) return job;  // invalid draft token in this sequence
        if (nb < prm.K) {
            const float4 st = prm.rowstats[(int64_t)i * prm.K + nb];
            job.mode = MODE_RESIDUAL;
            job.p_row = p + ((int64_t)i * prm.Kp + nb) * prm.ldv;
            job.q_row = static_cast<const T *>(prm.q) + ((int64_t)i * prm.K + nb) * prm.ldv;
            job.cp = (st.x + st.y) * kLog2e;
            job.cq = (st.z + st.w) * kLog2e;
        } else if (prm.Kp == prm.K + 1) {
            job.mode = MODE_SOFTMAX;
            job.p_row = p + ((int64_t)i * prm.Kp + prm.K) * prm.ldv;
        } else {
            return job;
        }
        job.u = prm.uniforms[(int64_t)i * (prm.K + 1) + prm.K];
    }
    return job;
}

// residual weights max(0, p_i - q_i) of one vector (probabilities, already normalised)
template <typename T>
__device__ __forceinline__ void residual_weights(const uint4 &vp, const uint4 &vq, float cp, float cq,
                                                 float (&w)[Vec<T>::N])
{
    constexpr int N = Vec<T>::N;
    float fp[N], fq[N];
    Vec<T>::unpack(vp, fp);
    Vec<T>::unpack(vq, fq);
#pragma unroll
    for (int e = 0; e < N; ++e)
        w[e] = fmaxf(0.f, ex2(fmaf(fp[e], kLog2e, -cp)) - ex2(fmaf(fq[e], kLog2e, -cq)));
}

static_assert(kWarps * kStatIters == 32, "a segment must hold exactly one warp's worth of steps");

struct DrawSmem {
    float4 red[kWarps];
    double step_sum[32];   // weight of each warp step of the rescanned segment
    double base;           // weight before the crossing step
    double t_in;
    double total;
    float ref;
    int segment;
    int step;
    int lastpos;
    int token;
    int last;
};

__device__ __forceinline__ double warp_sum_f64(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// inclusive prefix sum over the lanes of a warp, in lane order
__device__ __forceinline__ double warp_scan_f64(double v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += up;
    }
    return v;
}

// like load_step, for a row whose vectors need not be 16-byte aligned at `first`
template <typename T>
__device__ __forceinline__ void load_step_any(const T *__restrict__ row, int first, int V, int lane,
                                              uint4 (&raw)[kUnroll])
{
    constexpr int N = Vec<T>::N;
    if ((reinterpret_cast<uintptr_t>(row + first) & 15) == 0) {
        load_step<T>(row, first, V, lane, raw);
    } else {
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) raw[j] = load_vec<T>(row, first + (j * 32 + lane) * N, V);
    }
}

// lane-local sum of the residual weights of one warp step
template <typename T>
__device__ __forceinline__ float residual_step_sum(const uint4 (&rp)[kUnroll], const uint4 (&rq)[kUnroll],
                                                   float cp, float cq)
{
    constexpr int N = Vec<T>::N;
    float acc[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float w[N];
        residual_weights<T>(rp[j], rq[j], cp, cq, w);
        acc[j] = 0.f;
#pragma unroll
        for (int e = 0; e < N; ++e) acc[j] += w[e];
    }
    return (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

// (segment max, segment sum) of softmax weights, or (0, segment sum) of residual weights over
// segment c of the job's row(s); same step interleaving and prefetch as the row-statistics
// kernel.  The result is valid in thread 0.
template <typename T>
__device__ __forceinline__ MS segment_stats(const Job<T> &job, int mode, int V, int c, DrawSmem &sm)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    constexpr int kSegment = 32 * kStep;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int first = c * kSegment + warp * kStep - row_pad(job.p_row);
    MS v{neg_inf(), 0.f};
    uint4 rp[kUnroll];
    load_step<T>(job.p_row, first, V, lane, rp);
    if (mode == MODE_SOFTMAX) {
#pragma unroll
        for (int it = 0; it < kStatIters; ++it) {
            const int nxt = (it + 1) * kWarps * kStep;
            const bool more = it + 1 < kStatIters && first + nxt < V;
            online_update<T>(rp, v.m, v.s);
            if (!more) break;
            load_step<T>(job.p_row, first + nxt, V, lane, rp);
        }
        v = warp_ms(v);
    } else {
        uint4 rq[kUnroll];
        load_step_any<T>(job.q_row, first, V, lane, rq);
        float s = 0.f;
#pragma unroll
        for (int it = 0; it < kStatIters; ++it) {
            const int nxt = (it + 1) * kWarps * kStep;
            const bool more = it + 1 < kStatIters && first + nxt < V;
            s += residual_step_sum<T>(rp, rq, job.cp, job.cq);
            if (!more) break;
            load_step<T>(job.p_row, first + nxt, V, lane, rp);
            load_step_any<T>(job.q_row, first + nxt, V, lane, rq);
        }
        v.m = 0.f;
        v.s = warp_sum(s);
    }
    __syncthreads();  // sm.red may still be read by the previous use
    if (lane == 0) sm.red[warp] = make_float4(v.m, v.s, 0.f, 0.f);
    __syncthreads();
    if (warp == 0) {
        const float4 r = lane < kWarps ? sm.red[lane] : make_float4(neg_inf(), 0.f, 0.f, 0.f);
        if (mode == MODE_SOFTMAX) {
            v = warp_ms(MS{r.x, r.y});
        } else {
            v.m = 0.f;
            v.s = warp_sum(lane < kWarps ? r.y : 0.f);
        }
    }
    return v;
}

// weights of one vector of a step (softmax relative to `ref`, or residual)
template <typename T>
__device__ __forceinline__ void step_weights(const Job<T> &job, int mode, float off, const uint4 &vp,
                                             const uint4 &vq, float (&w)[Vec<T>::N])
{
    constexpr int N = Vec<T>::N;
    if (mode == MODE_SOFTMAX) {
        float f[N];
        Vec<T>::unpack(vp, f);
#pragma unroll
        for (int e = 0; e < N; ++e) w[e] = ex2(fmaf(f[e], kLog2e, off));
    } else {
        residual_weights<T>(vp, vq, job.cp, job.cq, w);
    }
}

// Finds, inside segment c, the first element whose running weight sum exceeds t_in (softmax
// weights are taken relative to `ref`).  Three phases: per-step sums of the whole segment,
// the step that holds the crossing (one warp scan), then the element inside that step (its
// owner warp).  Falls back to the last positive-weight element of the segment when rounding
// leaves no crossing; -1 if the segment has no weight.
template <typename T>
__device__ int segment_locate(const Job<T> &job, int mode, int V, int c, double t_in, float ref,
                              DrawSmem &sm)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    constexpr int kSegment = 32 * kStep;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int first = c * kSegment + warp * kStep - row_pad(job.p_row);
    const float off = -ref * kLog2e;
    if (tid == 0) {
        sm.lastpos = -1;
        sm.token = -1;
        sm.step = -1;
        sm.base = 0.0;
    }
    __syncthreads();
    int lp = -1;
    for (int it = 0; it < kStatIters; ++it) {
        const int f0 = first + it * kWarps * kStep;
        uint4 rp[kUnroll], rq[kUnroll] = {};
        load_step<T>(job.p_row, f0, V, lane, rp);
        if (mode == MODE_RESIDUAL) load_step_any<T>(job.q_row, f0, V, lane, rq);
        double ts = 0.0;
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            float w[N];
            step_weights<T>(job, mode, off, rp[j], rq[j], w);
#pragma unroll
            for (int e = 0; e < N; ++e) {
                ts += (double)w[e];
                if (w[e] > 0.f) lp = f0 + (j * 32 + lane) * N + e;
            }
        }
        ts = warp_sum_f64(ts);
        if (lane == 0) sm.step_sum[it * kWarps + warp] = ts;
    }
    lp = (int)__reduce_max_sync(0xffffffffu, lp);
    if (lane == 0 && lp >= 0) atomicMax(&sm.lastpos, lp);
    __syncthreads();
    if (warp == 0) {
        const double v = sm.step_sum[lane];
        const double incl = warp_scan_f64(v, lane);
        const unsigned cross = __ballot_sync(0xffffffffu, incl > t_in);
        if (cross != 0u && lane == __ffs(cross) - 1) {
            sm.step = lane;
            sm.base = incl - v;
        }
    }
    __syncthreads();
    const int step = sm.step;
    if (step < 0) return sm.lastpos;
    if (warp == step % kWarps) {
        const int f0 = first + (step / kWarps) * kWarps * kStep;
        uint4 rp[kUnroll], rq[kUnroll] = {};
        load_step<T>(job.p_row, f0, V, lane, rp);
        if (mode == MODE_RESIDUAL) load_step_any<T>(job.q_row, f0, V, lane, rq);
        double run = sm.base;
        int tok = -1;
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            float w[N];
            step_weights<T>(job, mode, off, rp[j], rq[j], w);
            double ts = 0.0;
#pragma unroll
            for (int e = 0; e < N; ++e) ts += (double)w[e];
            const double incl = run + warp_scan_f64(ts, lane);
            const unsigned cross = tok < 0 ? __ballot_sync(0xffffffffu, incl > t_in) : 0u;
            if (tok < 0 && cross != 0u) {
                const int owner = __ffs(cross) - 1;
                int mine = -1;
                if (lane == owner) {
                    double r = incl - ts;
                    int last_pos = -1;
#pragma unroll
                    for (int e = 0; e < N; ++e) {
                        r += (double)w[e];
                        if (w[e] > 0.f) last_pos = e;
                        if (mine < 0 && r > t_in && w[e] > 0.f) mine = e;
                    }
                    if (mine < 0) mine = last_pos;   // rounding inside the vector
                    if (mine >= 0) mine += f0 + (j * 32 + lane) * N;
                }
                tok = __shfl_sync(0xffffffffu, mine, owner);
                if (tok < 0) tok = -2;   // crossing vector had no positive weight: use the fallback
            }
            run = __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) sm.token = tok >= 0 ? tok : sm.lastpos;
    }
    __syncthreads();
    return sm.token;
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 4) draw_kernel(const DrawParams prm)
{
    __shared__ DrawSmem sm;
    const int C = prm.chunks;   // segments per row
    const int i = blockIdx.x / C;
    const int c = blockIdx.x % C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    Job<T> job = resolve_job<T>(prm, i);
    if (job.mode == MODE_NONE) {
        if (c == 0 && tid == 0) {
            prm.tokens[i] = -1;
            if (prm.residual_mass) prm.residual_mass[i] = 0.f;
        }
        return;
    }
    int mode = job.mode;
    float *part_m = prm.part_m + (int64_t)i * C;
    double *part_s = prm.part_s + (int64_t)i * C;

    const MS v = segment_stats<T>(job, mode, prm.V, c, sm);
    if (tid == 0) {
        part_m[c] = v.m;
        part_s[c] = (double)v.s;
        __threadfence();
        sm.last = (atomicAdd(&prm.counters[i], 1) == C - 1);
    }
    __syncthreads();
    if (!sm.last) return;
    __threadfence();

    // ---- last CTA of this draw: total weight and crossing segment (warp 0, segments in
    //      order, 32 at a time), then the token inside that segment (whole CTA)
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (warp == 0) {
            float M = neg_inf();
            for (int cc = lane; cc < C; cc += 32) M = fmaxf(M, __ldcg(&part_m[cc]));
            M = warp_max(M);
            double carry = 0.0, before = 0.0;
            int seg = -1, last_seg = -1;
            for (int c0 = 0; c0 < C; c0 += 32) {      // pass 1: total
                const int cc = c0 + lane;
                double S = 0.0;
                if (cc < C) {
                    const double s = __ldcg(&part_s[cc]);
                    if (s > 0.0) S = s * exp((double)__ldcg(&part_m[cc]) - (double)M);
                }
                carry += __shfl_sync(0xffffffffu, warp_scan_f64(S, lane), 31);
            }
            const double total = carry;
            const double target = (double)job.u * total;
            carry = 0.0;
            for (int c0 = 0; c0 < C; c0 += 32) {      // pass 2: same sums, find the crossing
                const int cc = c0 + lane;
                double S = 0.0;
                if (cc < C) {
                    const double s = __ldcg(&part_s[cc]);
                    if (s > 0.0) S = s * exp((double)__ldcg(&part_m[cc]) - (double)M);
                }
                const double incl = carry + warp_scan_f64(S, lane);
                const unsigned pos = __ballot_sync(0xffffffffu, S > 0.0);
                if (pos != 0u) last_seg = c0 + 31 - __clz(pos);
                const unsigned cross = __ballot_sync(0xffffffffu, incl > target);
                if (seg < 0 && cross != 0u) {
                    const int owner = __ffs(cross) - 1;
                    seg = c0 + owner;
                    before = __shfl_sync(0xffffffffu, incl - S, owner);
                }
                carry = __shfl_sync(0xffffffffu, incl, 31);
            }
            if (lane == 0) {
                sm.total = total;
                if (seg >= 0) {
                    const float mc = __ldcg(&part_m[seg]);
                    sm.segment = seg;
                    sm.ref = mc;
                    sm.t_in = (target - before) * exp((double)M - (double)mc);
                } else {  // u*total not below total (rounding, or u >= 1): last positive weight
                    sm.segment = last_seg;
                    sm.ref = last_seg >= 0 ? __ldcg(&part_m[last_seg]) : 0.f;
                    sm.t_in = __longlong_as_double(0x7ff0000000000000LL);
                }
            }
        }
        __syncthreads();
        if (attempt == 0 && prm.kind == DRAW_SD && tid == 0 && prm.residual_mass)
            prm.residual_mass[i] = mode == MODE_RESIDUAL ? (float)sm.total : 0.f;
        if (mode == MODE_RESIDUAL && !(sm.total > 0.0)) {
            // max(0, p - q) vanished: Eq. 1 is undefined, draw from p itself (one CTA, rare)
            mode = MODE_SOFTMAX;
            for (int cc = 0; cc < C; ++cc) {
                const MS r = segment_stats<T>(job, mode, prm.V, cc, sm);
                if (tid == 0) {
                    part_m[cc] = r.m;
                    part_s[cc] = (double)r.s;
                }
            }
            __threadfence();
            __syncthreads();
            continue;
        }
        break;
    }
    int token = -1;
    if (sm.segment >= 0) {
        const int seg = sm.segment;
        const double t_in = sm.t_in;
        const float ref = sm.ref;
        token = segment_locate<T>(job, mode, prm.V, seg, t_in, ref, sm);
    }
    if (tid == 0) prm.tokens[i] = token;
}

// ================================================================ host launchers
// Optional CUDA events recorded right before and after the row-statistics kernel (the
// launch that moves almost all the bytes), so a caller can time it inside a longer step.
static thread_local cudaEvent_t g_stage_before = nullptr, g_stage_after = nullptr;
void set_stage_events(cudaEvent_t before, cudaEvent_t after)
{
    g_stage_before = before;
    g_stage_after = after;
}

template <typename T>
static cudaError_t launch_sd_t(const SdParams &sp, const DrawParams &dp, int B, int K, cudaStream_t st)
{
    const int64_t grid_a = (int64_t)B * K * sp.chunks;
    const int64_t grid_b = (int64_t)B * dp.chunks;
    if (grid_a > 0x7fffffffLL || grid_b > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (grid_a == 0) return cudaSuccess;
    if (g_stage_before) cudaEventRecord(g_stage_before, st);
    sd_row_stats_kernel<T><<<(unsigned)grid_a, kThreads, 0, st>>>(sp);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (g_stage_after) cudaEventRecord(g_stage_after, st);
    draw_kernel<T><<<(unsigned)grid_b, kThreads, 0, st>>>(dp);
    return cudaGetLastError();
}

cudaError_t launch_sd_verify(const SdParams &sp, const DrawParams &dp, int B, int K, int dt,
                             cudaStream_t st)
{
    return dt == SPR_F32 ? launch_sd_t<float>(sp, dp, B, K, st)
                         : launch_sd_t<__nv_bfloat16>(sp, dp, B, K, st);
}

cudaError_t launch_draw(const DrawParams &dp, int n, int dt, cudaStream_t st)
{
    const int64_t grid = (int64_t)n * dp.chunks;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (grid == 0) return cudaSuccess;
    if (dt == SPR_F32)
        draw_kernel<float><<<(unsigned)grid, kThreads, 0, st>>>(dp);
    else
        draw_kernel<__nv_bfloat16><<<(unsigned)grid, kThreads, 0, st>>>(dp);
    return cudaGetLastError();
}

}  // namespace spr
