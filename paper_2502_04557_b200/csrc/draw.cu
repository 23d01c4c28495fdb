// Inverse-CDF draws from softmax(l) (replacement token, bonus token) or from the residual
// norm(max(0, p - q)) of Eq. 1 (correction token).  One read of the row(s); probabilities live
// in registers only; per-step partial weights go to the last CTA that finishes a draw, which
// finds the crossing step and re-reads just that step (2 KB) to pick the token.
#include "draw_common.cuh"

namespace spr {

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

// kSoftmaxOnly: replacement draws never take the residual branch; compiled without it the
// kernel needs fewer registers and four CTAs fit an SM.
template <typename T, bool kSoftmaxOnly>
__global__ void __launch_bounds__(kThreads, kSoftmaxOnly ? 4 : 3) draw_kernel(const DrawParams prm)
{
    __shared__ DrawSmem sm;
    const int C = prm.chunks;   // segments (CTAs) per row, of kWarps * prm.iters steps each
    const int steps = prm.steps;
    // correction draws go through the sequences last to first: the statistics pass has just
    // streamed the rows in ascending order, so the highest ones are the ones still in L2
    const int i = kSoftmaxOnly ? blockIdx.x / C : (int)(gridDim.x / C) - 1 - (int)(blockIdx.x / C);
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
    const int mode = kSoftmaxOnly ? (int)MODE_SOFTMAX : job.mode;
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

    const int token = finish_draw<T>(job, mode, prm.V, steps, prm.iters, part, sm,
                                     prm.kind == DRAW_SD && prm.residual_mass ? prm.residual_mass + i : nullptr);
    if (warp == 0 && lane == 0) prm.tokens[i] = token;
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
    if (dp.kind == DRAW_REPLACE)
        return dt == SPR_F32 ? cudaLaunchKernelEx(&cfg, draw_kernel<float, true>, dp)
                             : cudaLaunchKernelEx(&cfg, draw_kernel<__nv_bfloat16, true>, dp);
    return dt == SPR_F32 ? cudaLaunchKernelEx(&cfg, draw_kernel<float, false>, dp)
                         : cudaLaunchKernelEx(&cfg, draw_kernel<__nv_bfloat16, false>, dp);
}

}  // namespace spr
