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

constexpr int kCachedSteps = 512;   // step weights the last CTA of a draw keeps in shared memory

struct DrawSmem {
    double weight[kCachedSteps];   // weight of each step, relative to the row maximum
    double base;                   // weight before the crossing step
    double t_in;
    double total;
    float row_max;
    float ref;
    int step;
    int token;
    int last;
};

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

// (max, sum of exp(x - max)) of one warp step of a softmax draw, in every lane
template <typename T>
__device__ __forceinline__ MS softmax_step(const uint4 (&raw)[kUnroll])
{
    const MS t = thread_ms<T>(raw);
    MS r;
    r.m = warp_max(t.m);
    const float ref = (r.m == neg_inf()) ? 0.f : r.m;
    r.s = warp_sum(t.s * ex2((t.m - ref) * kLog2e));
    return r;
}

// Step partials (max, weight) of segment c of the job's row(s), written to part[step] for the
// steps this CTA owns; same step interleaving and prefetch as the row-statistics kernel.
// Residual draws store (0, sum of max(0, p - q)).
template <typename T>
__device__ __forceinline__ void segment_pass(const Job<T> &job, int mode, int V, int c, int steps,
                                             float2 *__restrict__ part)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int step0 = c * 32 + warp;                      // this warp's steps: step0 + it*kWarps
    const int first = step0 * kStep - row_pad(job.p_row);
    uint4 rp[kUnroll], rq[kUnroll];
    if (step0 >= steps) return;
    load_step<T>(job.p_row, first, V, lane, rp);
    if (mode == MODE_RESIDUAL) load_step_any<T>(job.q_row, first, V, lane, rq);
#pragma unroll
    for (int it = 0; it < kStatIters; ++it) {
        const int step = step0 + it * kWarps;
        const int nxt = (it + 1) * kWarps * kStep;
        const bool more = it + 1 < kStatIters && step + kWarps < steps;
        MS v;
        if (mode == MODE_SOFTMAX) {
            uint4 cur[kUnroll];
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) cur[j] = rp[j];
            if (more) load_step<T>(job.p_row, first + nxt, V, lane, rp);   // in flight during the math
            v = softmax_step<T>(cur);
        } else {
            v.m = 0.f;
            v.s = warp_sum(residual_step_sum<T>(rp, rq, job.cp, job.cq));
            if (more) {
                load_step<T>(job.p_row, first + nxt, V, lane, rp);
                load_step_any<T>(job.q_row, first + nxt, V, lane, rq);
            }
        }
        if (lane == 0) part[step] = make_float2(v.m, v.s);
        if (!more) break;
    }
    __threadfence();
}

// Inside step `step` of the row, the first element whose running weight exceeds t_in (softmax
// weights relative to `ref`); the last positive-weight element of the step if rounding
// leaves no crossing, -1 if the step has no weight.  One warp; result in every lane.
template <typename T>
__device__ int step_locate(const Job<T> &job, int mode, int V, int step, double t_in, float ref)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    const int lane = threadIdx.x & 31;
    const int f0 = step * kStep - row_pad(job.p_row);
    const float off = -ref * kLog2e;
    uint4 rp[kUnroll], rq[kUnroll] = {};
    load_step<T>(job.p_row, f0, V, lane, rp);
    if (mode == MODE_RESIDUAL) load_step_any<T>(job.q_row, f0, V, lane, rq);
    double run = 0.0;
    int tok = -1, lastpos = -1;
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float w[N];
        if (mode == MODE_SOFTMAX) {
            float f[N];
            Vec<T>::unpack(rp[j], f);
#pragma unroll
            for (int e = 0; e < N; ++e) w[e] = ex2(fmaf(f[e], kLog2e, off));
        } else {
            residual_weights<T>(rp[j], rq[j], job.cp, job.cq, w);
        }
        const int e0 = f0 + (j * 32 + lane) * N;
        double ts = 0.0;
#pragma unroll
        for (int e = 0; e < N; ++e) {
            ts += (double)w[e];
            if (w[e] > 0.f) lastpos = e0 + e;
        }
        const double incl = run + warp_scan_f64(ts, lane);
        const unsigned cross = __ballot_sync(0xffffffffu, incl > t_in);
        if (tok < 0 && cross != 0u) {
            const int owner = __ffs(cross) - 1;
            int mine = -1;
            if (lane == owner) {
                double r = incl - ts;
                int last_e = -1;
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    r += (double)w[e];
                    if (w[e] > 0.f) last_e = e;
                    if (mine < 0 && r > t_in && w[e] > 0.f) mine = e;
                }
                if (mine < 0) mine = last_e;       // rounding inside the vector
                if (mine >= 0) mine += e0;
            }
            tok = __shfl_sync(0xffffffffu, mine, owner);
            if (tok < 0) tok = -2;                 // no weight in the crossing vector: fall back
        }
        run = __shfl_sync(0xffffffffu, incl, 31);
    }
    lastpos = (int)__reduce_max_sync(0xffffffffu, lastpos);
    return tok >= 0 ? tok : lastpos;
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 3) draw_kernel(const DrawParams prm)
{
    __shared__ DrawSmem sm;
    const int C = prm.chunks;   // segments (CTAs) per row
    const int steps = prm.steps;
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
    float2 *part = prm.part + (int64_t)i * steps;

    segment_pass<T>(job, mode, prm.V, c, steps, part);
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        sm.last = (atomicAdd(&prm.counters[i], 1) == C - 1);
    }
    __syncthreads();
    if (!sm.last) return;
    __threadfence();

    // ---- last CTA of this draw: warp 0 adds the step weights in step order, finds the step
    //      where the running sum crosses u * total, and then the token inside that step
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (warp == 0) {
            float M = neg_inf();
            for (int t = lane; t < steps; t += 32) M = fmaxf(M, __ldcg(&part[t]).x);
            M = warp_max(M);
            double carry = 0.0;
            for (int t0 = 0; t0 < steps; t0 += 32) {      // pass 1: weights and their total
                const int t = t0 + lane;
                double S = 0.0;
                if (t < steps) {
                    const float2 ms = __ldcg(&part[t]);
                    if (ms.y > 0.f) S = (double)ms.y * exp((double)ms.x - (double)M);
                    if (t < kCachedSteps) sm.weight[t] = S;
                }
                carry += __shfl_sync(0xffffffffu, warp_scan_f64(S, lane), 31);
            }
            const double total = carry;
            const double target = (double)job.u * total;
            __syncwarp();
            carry = 0.0;
            double before = 0.0;
            int hit = -1, last_pos = -1;
            for (int t0 = 0; t0 < steps && hit < 0; t0 += 32) {   // pass 2: the crossing step
                const int t = t0 + lane;
                double S = 0.0;
                if (t < steps) {
                    if (t < kCachedSteps) {
                        S = sm.weight[t];
                    } else {
                        const float2 ms = __ldcg(&part[t]);
                        if (ms.y > 0.f) S = (double)ms.y * exp((double)ms.x - (double)M);
                    }
                }
                const double incl = carry + warp_scan_f64(S, lane);
                const unsigned pos = __ballot_sync(0xffffffffu, S > 0.0);
                if (pos != 0u) last_pos = t0 + 31 - __clz(pos);
                const unsigned cross = __ballot_sync(0xffffffffu, incl > target);
                if (cross != 0u) {
                    const int owner = __ffs(cross) - 1;
                    hit = t0 + owner;
                    before = __shfl_sync(0xffffffffu, incl - S, owner);
                }
                carry = __shfl_sync(0xffffffffu, incl, 31);
            }
            if (lane == 0) {
                sm.total = total;
                sm.row_max = M;
                if (hit >= 0) {
                    const float mc = __ldcg(&part[hit]).x;
                    sm.step = hit;
                    sm.ref = mc;
                    sm.t_in = (target - before) * exp((double)M - (double)mc);
                } else {  // u*total not below total (rounding, or u >= 1): last positive weight
                    sm.step = last_pos;
                    sm.ref = last_pos >= 0 ? __ldcg(&part[last_pos]).x : 0.f;
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
            for (int cc = 0; cc < C; ++cc) segment_pass<T>(job, mode, prm.V, cc, steps, part);
            __syncthreads();
            continue;
        }
        break;
    }
    if (warp != 0) return;
    int token = -1;
    if (sm.step >= 0) token = step_locate<T>(job, mode, prm.V, sm.step, sm.t_in, sm.ref);
    if (lane == 0) prm.tokens[i] = token;
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
