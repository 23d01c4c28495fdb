// Inverse-CDF draws from softmax(l) or from the residual norm(max(0, p - q)) of Eq. 1: the
// device code shared by the draw kernel and by the vocabulary-sharded correction draw.
#pragma once

#include <limits.h>

#include "vocab_common.cuh"

namespace spr {

// MODE_RESIDUAL forms max(0, p - q) in the ratio form below, accurate however close p and q are;
// MODE_RESIDUAL_FAST as the plain difference of the two probabilities, which costs a third of the
// instructions and is accurate enough whenever the residual mass is not tiny (see kResidualRedo).
enum { MODE_NONE = 0, MODE_SOFTMAX = 1, MODE_RESIDUAL = 2, MODE_RESIDUAL_FAST = 3 };

// The plain difference carries an absolute error of about 5e-7 of the probability mass passed
// (ex2.approx, two per element).  Where the draw falls is decided in units of the residual mass
// R, so that error counts 5e-7 / R there: two orders under the 1e-4 a decision must keep from
// its boundary as long as R >= 0.02.  A draw whose plain-difference mass comes out below that is
// redone in the ratio form by the warp that finishes it.
constexpr float kResidualRedo = 0.02f;

template <typename T>
struct Job {
    int mode;
    const T *p_row;
    const T *q_row;
    float cp, cq;  // residual: (max + ln Z) * log2(e) of the p row and of the q row, rounded
    float sp, sq;  // residual: 2^-(what the rounding of cp, cq dropped), factors next to 1
    float dc;      // residual: cq - cp, formed in double precision before rounding
    float u;
};

// Normalisers of both rows of a residual draw from the row statistics st = (max + ln Z of the p
// row, the same of the q row).  A probability is 2^(l * log2(e) - c) with c = (max + ln Z) *
// log2(e) of order 10..30: rounded to float c is off by up to 1e-6, a common factor on every
// probability of the row that would show in the residual mass; the factor is kept beside it.
template <typename T>
__device__ __forceinline__ void set_residual_scales(Job<T> &job, const double2 &st)
{
    constexpr double kL = 1.4426950408889634;
    const double cp = st.x * kL, cq = st.y * kL;
    job.cp = (float)cp;
    job.cq = (float)cq;
    job.sp = (float)exp2((double)job.cp - cp);
    job.sq = (float)exp2((double)job.cq - cq);
    job.dc = (float)(cq - cp);
}

// Residual weights max(0, p_i - q_i) of one vector (probabilities, already normalised).
// Where p_i and q_i nearly agree the difference of two rounded exponentials would be mostly
// rounding noise (or exactly zero), so there it is formed as q_i * (2^D - 1) with
// D = log2(p_i / q_i) = (lp_i - lq_i) * log2(e) + (cq - cp): the logit difference is exact and the
// normaliser difference comes from double precision, so D keeps its relative accuracy however
// small it is, and 2^D - 1 is a short series.  From ratio 2^(1/4) on the plain difference is used.
template <typename T>
__device__ __forceinline__ void residual_weights(const uint4 &vp, const uint4 &vq, const Job<T> &job,
                                                 float (&w)[Vec<T>::N])
{
    constexpr int N = Vec<T>::N;
    constexpr float kLn2 = 0.6931471805599453f;
    float fp[N], fq[N];
    Vec<T>::unpack(vp, fp);
    Vec<T>::unpack(vq, fq);
#pragma unroll
    for (int e = 0; e < N; ++e) {
        const float qv = ex2(fmaf(fq[e], kLog2e, -job.cq)) * job.sq;
        const float direct = fmaf(ex2(fmaf(fp[e], kLog2e, -job.cp)), job.sp, -qv);
        const float D = fmaf(fp[e] - fq[e], kLog2e, job.dc);   // NaN where both logits are -inf
        const float x = D * kLn2;
        // e^x - 1 for 0 < x < ln(2)/4: relative error below x^5/720 < 3e-7
        const float em1 = x * fmaf(x, fmaf(x, fmaf(x, fmaf(x, 1.f / 120.f, 1.f / 24.f), 1.f / 6.f), 0.5f), 1.f);
        const float r = D < 0.25f ? qv * em1 : direct;
        w[e] = D > 0.f ? r : 0.f;
    }
}

// max(0, p_i - q_i) of one vector as the plain difference of the probabilities
template <typename T>
__device__ __forceinline__ void residual_weights_fast(const uint4 &vp, const uint4 &vq, const Job<T> &job,
                                                      float (&w)[Vec<T>::N])
{
    constexpr int N = Vec<T>::N;
    float fp[N], fq[N];
    Vec<T>::unpack(vp, fp);
    Vec<T>::unpack(vq, fq);
    const uint64_t l2 = pack2(kLog2e, kLog2e), cp2 = pack2(-job.cp, -job.cp), cq2 = pack2(-job.cq, -job.cq);
    const uint64_t sp2 = pack2(job.sp, job.sp), nsq2 = pack2(-job.sq, -job.sq);
#pragma unroll
    for (int e = 0; e < N; e += 2) {
        float a0, a1, b0, b1, d0, d1;
        unpack2(fma2(pack2(fp[e], fp[e + 1]), l2, cp2), a0, a1);
        unpack2(fma2(pack2(fq[e], fq[e + 1]), l2, cq2), b0, b1);
        const uint64_t qs = mul2(pack2(ex2(b0), ex2(b1)), nsq2);          // -q
        unpack2(fma2(pack2(ex2(a0), ex2(a1)), sp2, qs), d0, d1);          // p - q
        w[e] = fmaxf(d0, 0.f);                                            // (-inf) - (-inf): both terms are 0
        w[e + 1] = fmaxf(d1, 0.f);
    }
}

// lane-local sum of those weights over one warp step
template <typename T>
__device__ __forceinline__ float residual_step_sum_fast(const uint4 (&rp)[kUnroll], const uint4 (&rq)[kUnroll],
                                                        const Job<T> &job)
{
    constexpr int N = Vec<T>::N;
    uint64_t acc[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float w[N];
        residual_weights_fast<T>(rp[j], rq[j], job, w);
        acc[j] = pack2(w[0], w[1]);
#pragma unroll
        for (int e = 2; e < N; e += 2) acc[j] = add2(acc[j], pack2(w[e], w[e + 1]));
    }
    float a0, a1, b0, b1;
    unpack2(add2(acc[0], acc[1]), a0, a1);
    unpack2(add2(acc[2], acc[3]), b0, b1);
    return (a0 + a1) + (b0 + b1);
}

// Scratch of whoever finishes a draw (a CTA in the sharded kernels, one warp in draw_kernel);
// CACHED = how many step weights it keeps in shared memory between the two passes over them.
template <int CACHED>
struct DrawSmemT {
    static constexpr int kCached = CACHED;
    double weight[CACHED];         // weight of each step, relative to the row maximum
    double base;                   // weight before the crossing step
    double t_in;
    double total;
    float row_max;
    float ref;
    int step;
    int token;
    int last;
};
using DrawSmem = DrawSmemT<512>;

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
                                                   const Job<T> &job)
{
    constexpr int N = Vec<T>::N;
    float acc[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float w[N];
        residual_weights<T>(rp[j], rq[j], job, w);
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
// steps this CTA owns (iters per warp; fewer when there are few draws, so that more CTAs
// share a row); same step interleaving and prefetch as the row-statistics kernel.
// Residual draws store (0, sum of max(0, p - q)).
template <typename T>
__device__ __forceinline__ void segment_pass(const Job<T> &job, int mode, int V, int c, int steps, int iters,
                                             float2 *__restrict__ part)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int step0 = c * kWarps * iters + warp;          // this warp's steps: step0 + it*kWarps
    const int first = step0 * kStep - row_pad(job.p_row);
    uint4 rp[kUnroll], rq[kUnroll];
    if (step0 >= steps) return;
    load_step<T>(job.p_row, first, V, lane, rp);
    if (mode == MODE_RESIDUAL) load_step_any<T>(job.q_row, first, V, lane, rq);
#pragma unroll
    for (int it = 0; it < kStatIters; ++it) {
        const int step = step0 + it * kWarps;
        const int nxt = (it + 1) * kWarps * kStep;
        const bool more = it + 1 < iters && step + kWarps < steps;
        MS v;
        if (mode == MODE_SOFTMAX) {
            uint4 cur[kUnroll];
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) cur[j] = rp[j];
            if (more) load_step<T>(job.p_row, first + nxt, V, lane, rp);   // in flight during the math
            v = softmax_step<T>(cur);
        } else {
            v.m = 0.f;
            v.s = warp_sum(residual_step_sum<T>(rp, rq, job));
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
    if (mode != MODE_SOFTMAX) load_step_any<T>(job.q_row, f0, V, lane, rq);
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
        } else if (mode == MODE_RESIDUAL_FAST) {
            residual_weights_fast<T>(rp[j], rq[j], job, w);
        } else {
            residual_weights<T>(rp[j], rq[j], job, w);
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

// weight of a step relative to the row maximum M: its own sum, rescaled from its own maximum
__device__ __forceinline__ double step_weight(float2 ms, float M)
{
    return ms.y > 0.f ? (double)(ms.y * ex2((ms.x - M) * kLog2e)) : 0.0;
}

// One warp, once every step partial of a draw is in part[0 .. steps): adds the step weights in
// step order (fp64 sums of fp32 weights relative to the largest step maximum) -> sm.total,
// sm.row_max; the first CACHED weights stay in sm.weight for steps_cross.
template <int CACHED>
__device__ __forceinline__ void steps_total(const float2 *part, int steps, DrawSmemT<CACHED> &sm)
{
    const int lane = threadIdx.x & 31;
    float2 *raw = reinterpret_cast<float2 *>(sm.weight);   // one trip to L2: the pairs wait here
    float M = neg_inf();
    for (int t = lane; t < steps; t += 32) {
        const float2 ms = __ldcg(&part[t]);
        if (t < CACHED) raw[t] = ms;
        M = fmaxf(M, ms.x);
    }
    M = warp_max(M);
    double carry = 0.0;
    for (int t0 = 0; t0 < steps; t0 += 32) {
        const int t = t0 + lane;
        double S = 0.0;
        if (t < steps) {
            S = step_weight(t < CACHED ? raw[t] : __ldcg(&part[t]), M);
            if (t < CACHED) sm.weight[t] = S;   // same lane, same slot: the pair is no longer needed
        }
        carry += __shfl_sync(0xffffffffu, warp_scan_f64(S, lane), 31);
    }
    if (lane == 0) {
        sm.total = carry;
        sm.row_max = M;
    }
    __syncwarp();
}

// Warp 0, after steps_total: the step where the running weight first exceeds `target` (same
// scale as sm.total) -> sm.step, with sm.t_in = what is left of the target inside that step,
// relative to that step's own maximum sm.ref.  If rounding (or u >= 1) leaves no crossing:
// the last step with positive weight and an infinite t_in; sm.step = -1 if there is none.
template <int CACHED>
__device__ __forceinline__ void steps_cross(const float2 *part, int steps, double target, DrawSmemT<CACHED> &sm)
{
    const int lane = threadIdx.x & 31;
    const float M = sm.row_max;
    double carry = 0.0, before = 0.0;
    int hit = -1, last_pos = -1;
    for (int t0 = 0; t0 < steps && hit < 0; t0 += 32) {
        const int t = t0 + lane;
        double S = 0.0;
        if (t < steps) {
            if (t < CACHED) {
                S = sm.weight[t];
            } else {
                S = step_weight(__ldcg(&part[t]), M);
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
        if (hit >= 0) {
            const float mc = __ldcg(&part[hit]).x;
            sm.step = hit;
            sm.ref = mc;
            sm.t_in = (target - before) * exp((double)M - (double)mc);
        } else {
            sm.step = last_pos;
            sm.ref = last_pos >= 0 ? __ldcg(&part[last_pos]).x : 0.f;
            sm.t_in = __longlong_as_double(0x7ff0000000000000LL);
        }
    }
    __syncwarp();
}

// ---------------------------------------------------------------- one-warp finish, short chain
// The finish of a draw is a chain of dependent steps on one warp while everybody else is done:
// the versions below keep it short for rows of at most kFastSteps warp steps.  Lane l owns
// steps 4l .. 4l+3 (and, inside the crossing step, vectors 4l .. 4l+3), so a lane adds its own
// items serially and ONE warp scan joins the lanes, where the general routines above scan once
// per 32 items; nothing is read twice.
constexpr int kFastSteps = 128;

struct Crossing {
    double total;     // weight of the row, relative to its maximum
    double t_in;      // what is left of the target inside the crossing step, in that step's own scale
    float ref;        // maximum of the crossing step
    int step;         // crossing step; the last step with weight if rounding leaves none; -1: no weight
};

// steps <= kFastSteps step partials -> where u * total falls.  Same arithmetic per item as
// step_weight / steps_total / steps_cross; the scale between the row's units and the crossing
// step's is the very factor its weight was formed with.
__device__ __forceinline__ Crossing warp_crossing(const float2 *part, int steps, float u)
{
    const int lane = threadIdx.x & 31;
    float2 ms[4];
    float M = neg_inf();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int t = 4 * lane + k;
        ms[k] = t < steps ? __ldcg(&part[t]) : make_float2(neg_inf(), 0.f);
        M = fmaxf(M, ms[k].x);
    }
    M = warp_max(M);
    float f[4];
    double incl[4];
    double run = 0.0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        f[k] = ms[k].y > 0.f ? ex2((ms[k].x - M) * kLog2e) : 0.f;
        run += ms[k].y > 0.f ? (double)(ms[k].y * f[k]) : 0.0;
        incl[k] = run;
    }
    const double lanes = warp_scan_f64(run, lane);    // inclusive over the lanes
    const double before_lane = lanes - run;
    Crossing c;
    c.total = __shfl_sync(0xffffffffu, lanes, 31);
    const double target = (double)u * c.total;
    // first own step whose running weight passes the target, last own step with weight
    // (selected without indexing the register arrays by a run-time value)
    int kfirst = 4, klast = -1;
    double before_first = 0.0;
    float f_first = 1.f, ref_first = 0.f, ref_last = 0.f;
#pragma unroll
    for (int k = 3; k >= 0; --k) {
        const bool has = ms[k].y > 0.f && f[k] > 0.f;
        if (has && before_lane + incl[k] > target) {
            kfirst = k;
            before_first = before_lane + (k > 0 ? incl[k > 0 ? k - 1 : 0] : 0.0);
            f_first = f[k];
            ref_first = ms[k].x;
        }
        if (has && klast < 0) {
            klast = k;
            ref_last = ms[k].x;
        }
    }
    const unsigned cross = __ballot_sync(0xffffffffu, kfirst < 4);
    const unsigned pos = __ballot_sync(0xffffffffu, klast >= 0);
    if (cross != 0u) {
        const int owner = __ffs(cross) - 1;
        c.step = __shfl_sync(0xffffffffu, 4 * lane + kfirst, owner);
        c.t_in = __shfl_sync(0xffffffffu, (target - before_first) / (double)f_first, owner);
        c.ref = __shfl_sync(0xffffffffu, ref_first, owner);
    } else if (pos != 0u) {
        const int owner = 31 - __clz(pos);
        c.step = __shfl_sync(0xffffffffu, 4 * lane + klast, owner);
        c.ref = __shfl_sync(0xffffffffu, ref_last, owner);
        c.t_in = __longlong_as_double(0x7ff0000000000000LL);
    } else {
        c.step = -1;
        c.ref = 0.f;
        c.t_in = 0.0;
    }
    return c;
}

// the ratio-form weights as a call: rare in warp_locate (only the redo of a draw with a tiny
// residual mass gets there), so it is kept out of line there
template <typename T>
__device__ __noinline__ void residual_weights_call(const uint4 &vp, const uint4 &vq, const Job<T> &job,
                                                   float (&w)[Vec<T>::N])
{
    residual_weights<T>(vp, vq, job, w);
}

// Inside step `step`: the first element whose running weight exceeds t_in, as step_locate
// finds it, with the step's 128 vectors dealt to the lanes four in a row.
template <typename T, bool kUnrolled>
__device__ __forceinline__ int warp_locate(const Job<T> &job, int mode, int V, int step, double t_in, float ref)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    static_assert(kUnroll == 4, "four vectors per lane");
    const int lane = threadIdx.x & 31;
    const int f0 = step * kStep - row_pad(job.p_row) + 4 * lane * N;    // this lane's first element
    const float off = -ref * kLog2e;
    uint4 rp[4], rq[4] = {};
#pragma unroll
    for (int j = 0; j < 4; ++j) rp[j] = load_vec<T>(job.p_row, f0 + j * N, V);
    if (mode != MODE_SOFTMAX) {
#pragma unroll
        for (int j = 0; j < 4; ++j) rq[j] = load_vec<T>(job.q_row, f0 + j * N, V);
    }
    // The finish of a draw is cold code that one warp runs once; much of what it costs is
    // fetching its instructions.  Where the weight formulas are long (a kernel that knows the
    // residual modes: !kUnrolled) the loops over the lane's four vectors are NOT unrolled (one
    // copy of the formulas each); the vector is picked with selects, since registers cannot be
    // indexed by a run-time value.
    auto pick = [](const uint4 (&r)[4], int j) { return j == 0 ? r[0] : j == 1 ? r[1] : j == 2 ? r[2] : r[3]; };
    auto weights = [&](int j, float (&w)[N]) {
        const uint4 vp = pick(rp, j);
        if (mode == MODE_SOFTMAX) {
            float f[N];
            Vec<T>::unpack(vp, f);
#pragma unroll
            for (int e = 0; e < N; ++e) w[e] = ex2(fmaf(f[e], kLog2e, off));
        } else if (mode == MODE_RESIDUAL_FAST) {
            residual_weights_fast<T>(vp, pick(rq, j), job, w);
        } else {
            residual_weights_call<T>(vp, pick(rq, j), job, w);
        }
    };
    double vs0 = 0.0, vs1 = 0.0, vs2 = 0.0, vs3 = 0.0;      // weight of each of the lane's vectors
    int lastpos = -1;
#pragma unroll(kUnrolled ? 4 : 1)
    for (int j = 0; j < 4; ++j) {
        float w[N];
        weights(j, w);
        double ts = 0.0;
#pragma unroll
        for (int e = 0; e < N; ++e) {
            ts += (double)w[e];
            if (w[e] > 0.f) lastpos = f0 + j * N + e;
        }
        vs0 = j == 0 ? ts : vs0;
        vs1 = j == 1 ? ts : vs1;
        vs2 = j == 2 ? ts : vs2;
        vs3 = j == 3 ? ts : vs3;
    }
    const double mine = (vs0 + vs1) + (vs2 + vs3);
    const double incl = warp_scan_f64(mine, lane);
    const unsigned cross = __ballot_sync(0xffffffffu, incl > t_in);
    int tok = -1;
    if (cross != 0u) {
        const int owner = __ffs(cross) - 1;
        int found = -1;
        if (lane == owner) {
            double r = incl - mine;
            int last_e = -1;       // last element with weight up to and including the crossing vector
#pragma unroll(kUnrolled ? 4 : 1)
            for (int j = 0; j < 4 && found == -1; ++j) {
                const double vsj = j == 0 ? vs0 : j == 1 ? vs1 : j == 2 ? vs2 : vs3;
                float w[N];
                weights(j, w);
                const bool here = r + vsj > t_in;
                double rr = r;
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    rr += (double)w[e];
                    if (w[e] > 0.f) last_e = f0 + j * N + e;
                    if (here && found < 0 && rr > t_in && w[e] > 0.f) found = f0 + j * N + e;
                }
                if (here && found < 0) found = last_e >= 0 ? last_e : -2;   // rounding inside the vector
                r += vsj;
            }
        }
        tok = __shfl_sync(0xffffffffu, found, owner);
    }
    lastpos = (int)__reduce_max_sync(0xffffffffu, lastpos);
    return tok >= 0 ? tok : lastpos;
}

// Whole CTA, once every step partial of a draw is in part[0 .. steps): the token where the
// running weight crosses u * total.  A residual draw whose weights vanish (Eq. 1 undefined)
// is redone as a draw from p.  The token is returned in warp 0 (other warps get -1);
// *residual_mass, if given, receives the total residual weight (0 for softmax draws).
template <typename T>
__device__ int finish_draw(const Job<T> &job, int mode, int V, int steps, int iters, float2 *part, DrawSmem &sm,
                           float *residual_mass)
{
    const int tid = threadIdx.x, warp = tid >> 5;
    const int C = (steps + kWarps * iters - 1) / (kWarps * iters);
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (warp == 0) {
            steps_total(part, steps, sm);
            steps_cross(part, steps, (double)job.u * sm.total, sm);
        }
        __syncthreads();
        if (attempt == 0 && tid == 0 && residual_mass) *residual_mass = mode == MODE_RESIDUAL ? (float)sm.total : 0.f;
        if (mode == MODE_RESIDUAL && !(sm.total > 0.0)) {
            // max(0, p - q) vanished: Eq. 1 is undefined, draw from p itself (one CTA, rare)
            mode = MODE_SOFTMAX;
            for (int cc = 0; cc < C; ++cc) segment_pass<T>(job, mode, V, cc, steps, iters, part);
            __syncthreads();
            continue;
        }
        break;
    }
    if (warp != 0) return -1;
    return sm.step >= 0 ? step_locate<T>(job, mode, V, sm.step, sm.t_in, sm.ref) : -1;
}

}  // namespace spr
