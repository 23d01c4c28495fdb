// Inverse-CDF draws from softmax(l) (replacement token, bonus token) or from the residual
// norm(max(0, p - q)) of Eq. 1 (correction token).  One read of the row(s); probabilities live
// in registers only; per-step partial weights go to the last CTA that finishes a draw, which
// finds the crossing step and re-reads just that step (2 KB) to pick the token.
#include <limits.h>

#include "vocab_common.cuh"

namespace spr {

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
    // the uniform does not depend on the row choice: fetch it alongside the gate
    job.u = prm.kind == DRAW_REPLACE ? prm.uniforms[i] : prm.uniforms[(int64_t)i * (prm.K + 1) + prm.K];
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
    const int C = prm.chunks;   // segments (CTAs) per row, of kWarps * prm.iters steps each
    const int steps = prm.steps;
    const int i = blockIdx.x / C;
    const int c = blockIdx.x % C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    pdl_wait();   // the kernel before this one may still be writing first_reject / accepted_len
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

    segment_pass<T>(job, mode, prm.V, c, steps, prm.iters, part);
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
            for (int cc = 0; cc < C; ++cc) segment_pass<T>(job, mode, prm.V, cc, steps, prm.iters, part);
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

cudaError_t launch_draw(const DrawParams &dp, int n, int dt, cudaStream_t st, bool after_kernel)
{
    const int64_t grid = (int64_t)n * dp.chunks;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (grid == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (after_kernel) {   // overlap this launch with the tail of the kernel that feeds it
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    return dt == SPR_F32 ? cudaLaunchKernelEx(&cfg, draw_kernel<float>, dp)
                         : cudaLaunchKernelEx(&cfg, draw_kernel<__nv_bfloat16>, dp);
}

}  // namespace spr
