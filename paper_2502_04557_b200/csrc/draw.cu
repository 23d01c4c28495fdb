// Inverse-CDF draws from softmax(l) (replacement token, bonus token) or from the residual
// norm(max(0, p - q)) of Eq. 1 (correction token).  One read of the row(s); probabilities live
// in registers only.
//
// The unit of work is one warp step (2 KB of one row, 4 KB of a row pair).  Every CTA first
// finds out which draws are live (a draw gated off by first_reject, or a sequence without a
// correction token, costs nothing), then the live draws' steps, laid end to end, are cut into
// equal contiguous runs, one per warp of a grid sized to the GPU: no CTA is launched for a dead
// draw and every warp streams the same number of bytes, with the loads of its next steps in
// flight while it works on the current one.  A warp writes one (max, weight) pair per step and
// takes tickets on the draw for the steps it did; the warp that takes the last ticket adds the
// step weights in step order, finds the step where the running sum crosses u * total and
// re-reads just that step to pick the token.  Warps never wait for each other.
#include "draw_common.cuh"

namespace spr {

// Development aid (compiled only with -DSPR_DRAW_STAMPS): SM-clock stamps of the phases of the
// first CTAs of a launch, read back with spr_debug_draw_stamps().
#ifdef SPR_DRAW_STAMPS
__device__ long long g_draw_stamps[1024][8];
#define SPR_DSTAMP(i)                                                         \
    do {                                                                      \
        if (blockIdx.x < 1024) g_draw_stamps[blockIdx.x][i] = clock64();      \
    } while (0)
extern "C" int spr_debug_draw_stamps(long long *host_out)   // reads the stamps and clears them
{
    cudaError_t e = cudaMemcpyFromSymbol(host_out, g_draw_stamps, sizeof(long long) * 1024 * 8);
    void *p = nullptr;
    if (e == cudaSuccess) e = cudaGetSymbolAddress(&p, g_draw_stamps);
    if (e == cudaSuccess) e = cudaMemset(p, 0, sizeof(long long) * 1024 * 8);
    return (int)e;
}
#else
#define SPR_DSTAMP(i)
#endif

namespace {

constexpr int kMaxCompact = 4096;   // draws whose live list a CTA builds in shared memory
// CTAs per SM: what the registers of the streaming loops (three steps of one row, or two steps
// of a row pair, in flight per warp) leave room for
constexpr int kDrawCtasSoftmax = 3, kDrawCtasResidual = 2;
using WarpSmem = DrawSmemT<128>;    // per-warp scratch of a finishing warp

// does draw i need any work?  (a negative first_reject is live: it is reported as a bad row)
__device__ __forceinline__ bool draw_is_live(const DrawParams &prm, int i)
{
    if (prm.kind == DRAW_REPLACE) return !prm.gate || prm.gate[i] < prm.K;
    const int nb = prm.accepted_len[i];
    return nb >= 0 && (nb < prm.K || prm.Kp == prm.K + 1);
}

template <typename T>
__device__ __forceinline__ Job<T> resolve_job(const DrawParams &prm, int i)
{
    Job<T> job;
    job.mode = MODE_NONE;
    job.p_row = job.q_row = nullptr;
    job.cp = job.cq = job.dc = 0.f;
    job.sp = job.sq = 1.f;
    job.u = prm.kind == DRAW_REPLACE ? prm.uniforms[i] : prm.uniforms[(int64_t)i * (prm.K + 1) + prm.K];
    const T *p = static_cast<const T *>(prm.p);
    if (prm.kind == DRAW_REPLACE) {
        int off = 0;
        if (prm.gate) {
            off = prm.gate[i];
            if (off >= prm.K) return job;  // verifier kept every token: the target is not called
        }
        const int64_t row = (prm.rows ? (int64_t)prm.rows[i] : (int64_t)i * prm.seq_stride) + off;
        if (off < 0 || row < 0 || row >= prm.R) {
            raise_status(prm.status, SPR_ERR_BAD_ROW);
            return job;
        }
        job.mode = MODE_SOFTMAX;
        job.p_row = p + row * prm.ldv;
    } else {
        const int nb = prm.accepted_len[i];
        if (nb < 0) return job;  // invalid draft token in this sequence
        if (nb < prm.K) {
            job.mode = MODE_RESIDUAL_FAST;
            job.p_row = p + ((int64_t)i * prm.Kp + nb) * prm.ldv;
            job.q_row = static_cast<const T *>(prm.q) + ((int64_t)i * prm.K + nb) * prm.ldv;
            set_residual_scales(job, prm.rowstats[(int64_t)i * prm.K + nb]);
        } else if (prm.Kp == prm.K + 1) {
            job.mode = MODE_SOFTMAX;
            job.p_row = p + ((int64_t)i * prm.Kp + prm.K) * prm.ldv;
        }
    }
    return job;
}

// One warp: (max, weight) of steps [s0, s1) of the job's row(s) -> part[step]; the loads of
// the following step(s) are issued before the current step is consumed.
template <typename T, bool kSoftmaxOnly>
__device__ __forceinline__ void warp_steps(const Job<T> &job, int mode, int V, int s0, int s1,
                                           float2 *__restrict__ part)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    const int lane = threadIdx.x & 31;
    const int pad = row_pad(job.p_row);
    if (kSoftmaxOnly || mode == MODE_SOFTMAX) {
        // two steps in flight behind the one being summed; the three buffers swap roles by
        // position in an unrolled loop instead of being copied
        uint4 a[kUnroll], b[kUnroll], c[kUnroll];
        auto emit = [&](const uint4 (&src)[kUnroll], int s) {
            const MS v = softmax_step<T>(src);
            if (lane == 0) part[s] = make_float2(v.m, v.s);
        };
        auto run = [&](auto fetch) {
            fetch(a, s0);
            if (s0 + 1 < s1) fetch(b, s0 + 1);
            for (int s = s0;;) {
                if (s + 2 < s1) fetch(c, s + 2);
                emit(a, s);
                if (++s >= s1) break;
                if (s + 2 < s1) fetch(a, s + 2);
                emit(b, s);
                if (++s >= s1) break;
                if (s + 2 < s1) fetch(b, s + 2);
                emit(c, s);
                if (++s >= s1) break;
            }
        };
        const int64_t f0 = (int64_t)s0 * kStep - pad;
        if (f0 >= 0 && (int64_t)s1 * kStep - pad <= V) {
            // every step of the run is whole aligned vectors inside the row: loads without checks
            const uint4 *pp = reinterpret_cast<const uint4 *>(job.p_row + f0) + lane;
            run([&](uint4 (&dst)[kUnroll], int s) {
#pragma unroll
                for (int j = 0; j < kUnroll; ++j) dst[j] = ld_stream(pp + (s - s0) * (kStep / N) + j * 32);
            });
        } else {
            run([&](uint4 (&dst)[kUnroll], int s) { load_step<T>(job.p_row, s * kStep - pad, V, lane, dst); });
        }
    } else {
        uint4 rp[kUnroll], rq[kUnroll], np[kUnroll], nq[kUnroll];
        load_step<T>(job.p_row, s0 * kStep - pad, V, lane, rp);
        load_step_any<T>(job.q_row, s0 * kStep - pad, V, lane, rq);
        for (int s = s0; s < s1; ++s) {
            if (s + 1 < s1) {
                load_step<T>(job.p_row, (s + 1) * kStep - pad, V, lane, np);
                load_step_any<T>(job.q_row, (s + 1) * kStep - pad, V, lane, nq);
            }
            const float w = warp_sum(residual_step_sum_fast<T>(rp, rq, job));
            if (lane == 0) part[s] = make_float2(0.f, w);
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                rp[j] = np[j];
                rq[j] = nq[j];
            }
        }
    }
}

// One warp: softmax partials of every step of the row, one step at a time (the rare redo of a
// residual draw whose weights vanished; kept small on purpose)
template <typename T>
__device__ __noinline__ void warp_softmax_row(const T *row, int V, int steps, float2 *part)
{
    constexpr int kStep = 32 * kUnroll * Vec<T>::N;
    const int lane = threadIdx.x & 31;
    const int pad = row_pad(row);
    for (int s = 0; s < steps; ++s) {
        uint4 a[kUnroll];
        load_step<T>(row, s * kStep - pad, V, lane, a);
        const MS v = softmax_step<T>(a);
        if (lane == 0) part[s] = make_float2(v.m, v.s);
    }
    __syncwarp();   // lane 0's partials are read by the other lanes next
}

// One warp: the residual partials of every step of a row pair in the ratio form (the rare redo
// of a draw whose residual mass is too small for plain differences; kept small on purpose)
template <typename T>
__device__ __noinline__ void warp_residual_row(const Job<T> &job, int V, int steps, float2 *part)
{
    constexpr int kStep = 32 * kUnroll * Vec<T>::N;
    const int lane = threadIdx.x & 31;
    const int pad = row_pad(job.p_row);
    for (int s = 0; s < steps; ++s) {
        uint4 rp[kUnroll], rq[kUnroll];
        load_step<T>(job.p_row, s * kStep - pad, V, lane, rp);
        load_step_any<T>(job.q_row, s * kStep - pad, V, lane, rq);
        const float w = warp_sum(residual_step_sum<T>(rp, rq, job));
        if (lane == 0) part[s] = make_float2(0.f, w);
    }
    __syncwarp();
}

// One warp, once every step partial of the draw is in part[0 .. steps): the token where the
// running weight crosses u * total.  A residual draw whose mass (from plain differences) is
// below kResidualRedo is first redone by this warp in the ratio form.  A residual draw whose weights vanish (Eq. 1 undefined) is
// redone by this warp as a draw from p.  *residual_mass, if given, receives the total residual
// weight (0 for softmax draws).
template <typename T, bool kSoftmaxOnly>
__device__ __noinline__ int warp_finish(const Job<T> &job, int mode, int V, int steps, float2 *part, WarpSmem &sm,
                                        float *residual_mass)
{
    const int lane = threadIdx.x & 31;
    const bool fast = steps <= kFastSteps;     // the short chain: everything in registers
    Crossing c;
    auto cross = [&]() {
        if (fast) {
            c = warp_crossing(part, steps, job.u);
        } else {
            steps_total(part, steps, sm);
            c.total = sm.total;
        }
    };
    cross();
    if (!kSoftmaxOnly && mode == MODE_RESIDUAL_FAST && !(c.total >= (double)kResidualRedo)) {
        mode = MODE_RESIDUAL;
        warp_residual_row<T>(job, V, steps, part);
        cross();
    }
    if (lane == 0 && residual_mass) *residual_mass = mode == MODE_SOFTMAX ? 0.f : (float)c.total;
    if (!kSoftmaxOnly && mode != MODE_SOFTMAX && !(c.total > 0.0)) {
        mode = MODE_SOFTMAX;
        warp_softmax_row<T>(job.p_row, V, steps, part);
        cross();
    }
    if (fast) return c.step >= 0 ? warp_locate<T, kSoftmaxOnly>(job, mode, V, c.step, c.t_in, c.ref) : -1;
    steps_cross(part, steps, (double)job.u * sm.total, sm);
    return sm.step >= 0 ? step_locate<T>(job, mode, V, sm.step, sm.t_in, sm.ref) : -1;
}

// kSoftmaxOnly: replacement draws never take the residual branch; compiled without it the
// kernel needs fewer registers.
template <typename T, bool kSoftmaxOnly>
__global__ void __launch_bounds__(kThreads, kSoftmaxOnly ? kDrawCtasSoftmax : kDrawCtasResidual)
draw_kernel(const DrawParams prm)
{
    // live draws in ascending order: those that read two rows (residual draws: twice the bytes
    // and more than twice the arithmetic per step) and those that read one
    __shared__ unsigned short s_live[kMaxCompact];
    __shared__ unsigned short s_light[kSoftmaxOnly ? 1 : kMaxCompact];
    __shared__ int s_count[2][kWarps];
    __shared__ WarpSmem s_fin[kWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = prm.n, steps = prm.steps;
    if (tid == 0) SPR_DSTAMP(0);

    pdl_wait();   // the kernel before this one may still be writing first_reject / accepted_len
    if (tid == 0) SPR_DSTAMP(1);

    // ---- which draws are live?  Every CTA builds the same lists.
    const bool compact = n <= kMaxCompact;
    int nheavy = n, nlight = 0;
    if (compact) {
        // Rounds of 1024 draws: warp w looks at draws w*128 .. w*128+127 of the round, four per
        // lane with their loads in flight together, so a round costs one trip to memory.
        nheavy = 0;
        for (int base = 0; base < n; base += kWarps * 128) {
            bool heavy[4], light[4];
            unsigned mh[4], ml[4];
            int mine_h = 0, mine_l = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = base + warp * 128 + j * 32 + lane;
                const bool live = i < n && draw_is_live(prm, i);
                // a correction draw from the residual reads the p row and the q row
                heavy[j] = live;
                light[j] = false;
                if constexpr (!kSoftmaxOnly) {
                    heavy[j] = live && (prm.kind != DRAW_SD || prm.accepted_len[i] < prm.K);
                    light[j] = live && !heavy[j];
                }
                if (i < n && !live && blockIdx.x == 0) {
                    prm.tokens[i] = -1;
                    if (prm.residual_mass) prm.residual_mass[i] = 0.f;
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                mh[j] = __ballot_sync(0xffffffffu, heavy[j]);
                mine_h += __popc(mh[j]);
                ml[j] = 0u;
                if constexpr (!kSoftmaxOnly) {
                    ml[j] = __ballot_sync(0xffffffffu, light[j]);
                    mine_l += __popc(ml[j]);
                }
            }
            if (lane == 0) {
                s_count[0][warp] = mine_h;
                if constexpr (!kSoftmaxOnly) s_count[1][warp] = mine_l;
            }
            __syncthreads();
            int before_h = nheavy, all_h = nheavy, before_l = nlight, all_l = nlight;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                if (w < warp) before_h += s_count[0][w];
                all_h += s_count[0][w];
                if constexpr (!kSoftmaxOnly) {
                    if (w < warp) before_l += s_count[1][w];
                    all_l += s_count[1][w];
                }
            }
            const unsigned below = (1u << lane) - 1u;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const unsigned short i = (unsigned short)(base + warp * 128 + j * 32 + lane);
                if (heavy[j]) s_live[before_h + __popc(mh[j] & below)] = i;
                before_h += __popc(mh[j]);
                if constexpr (!kSoftmaxOnly) {
                    if (light[j]) s_light[before_l + __popc(ml[j] & below)] = i;
                    before_l += __popc(ml[j]);
                }
            }
            nheavy = all_h;
            nlight = all_l;
            __syncthreads();
        }
    }

    if (tid == 0) SPR_DSTAMP(2);
    // ---- this warp's run of the live draws' steps.  The steps of the two-row draws, then those
    // of the one-row draws, laid end to end and cut into runs of equal COST, a two-row step
    // counting twice: a cut at cost x lies at step ceil(x / 2) inside the first part.
    const int64_t heavy_steps = (int64_t)nheavy * steps, all_steps = heavy_steps + (int64_t)nlight * steps;
    const int64_t cost = 2 * heavy_steps + (int64_t)nlight * steps;
    const int64_t warps = (int64_t)gridDim.x * kWarps, gw = (int64_t)blockIdx.x * kWarps + warp;
    auto cut = [&](int64_t g) {     // first step of warp g's run
        if (kSoftmaxOnly) return all_steps / warps * g + min(g, all_steps % warps);   // every step costs the same
        const int64_t x = cost / warps * g + min(g, cost % warps);
        return x <= 2 * heavy_steps ? (x + 1) / 2 : x - heavy_steps;
    };
    int64_t u = cut(gw);
    const int64_t u_end = gw + 1 == warps ? all_steps : cut(gw + 1);
    while (u < u_end) {
        int64_t j = u / steps;
        const int s0 = (int)(u - j * steps);
        const int s1 = (int)min((int64_t)steps, s0 + (u_end - u));
        u += s1 - s0;
        // Each list is gone through last to first: the statistics pass has just streamed the
        // rows in ascending order, so the highest ones are the ones still in L2.
        int i;
        if (j < nheavy) {
            j = kSoftmaxOnly ? j : nheavy - 1 - j;
            i = compact ? (int)s_live[j] : (int)j;
        } else {
            i = (int)s_light[nlight - 1 - (j - nheavy)];
        }
        const Job<T> job = resolve_job<T>(prm, i);
        if (job.mode == MODE_NONE) {   // gated off (when no list was built), or a bad row
            if (s0 == 0 && lane == 0) {
                prm.tokens[i] = -1;
                if (prm.residual_mass) prm.residual_mass[i] = 0.f;
            }
            continue;
        }
        const int mode = kSoftmaxOnly ? (int)MODE_SOFTMAX : job.mode;
        float2 *part = prm.part + (int64_t)i * steps;
        warp_steps<T, kSoftmaxOnly>(job, mode, prm.V, s0, s1, part);
        if (tid == 0) SPR_DSTAMP(3);
        int last = 0;
        if (lane == 0) {
            __threadfence();
            last = take_ticket(&prm.counters[i], steps, s1 - s0);
        }
        if (tid == 0) SPR_DSTAMP(4);
        if (!__shfl_sync(0xffffffffu, last, 0)) continue;
        __threadfence();
        const int token = warp_finish<T, kSoftmaxOnly>(job, mode, prm.V, steps, part, s_fin[warp],
                                                       prm.kind == DRAW_SD && prm.residual_mass
                                                           ? prm.residual_mass + i : nullptr);
        if (lane == 0) prm.tokens[i] = token;
        if (lane == 0) SPR_DSTAMP(5);
    }
    if (tid == 0) SPR_DSTAMP(6);
}

}  // namespace

// CTAs of a launch: enough warps for one step each, at most what the GPU holds at once
int draw_grid(int n, int steps, bool softmax_only)
{
    const int64_t units = (int64_t)n * steps;
    const int64_t resident = 148 * (softmax_only ? kDrawCtasSoftmax : kDrawCtasResidual);
    const int64_t ctas = (units + kWarps - 1) / kWarps;
    return (int)(ctas < resident ? ctas : resident);
}

cudaError_t launch_draw(const DrawParams &dp, int dt, cudaStream_t st, bool after_kernel)
{
    if (dp.n == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)draw_grid(dp.n, dp.steps, dp.kind == DRAW_REPLACE));
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (after_kernel) {   // overlap this launch with the tail of the kernel that feeds it
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    if (dp.kind == DRAW_REPLACE)
        return dt == SPR_F32 ? cudaLaunchKernelEx(&cfg, draw_kernel<float, true>, dp)
                             : cudaLaunchKernelEx(&cfg, draw_kernel<__nv_bfloat16, true>, dp);
    return dt == SPR_F32 ? cudaLaunchKernelEx(&cfg, draw_kernel<float, false>, dp)
                         : cudaLaunchKernelEx(&cfg, draw_kernel<__nv_bfloat16, false>, dp);
}

}  // namespace spr
