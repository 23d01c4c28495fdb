// Inverse-CDF draws from softmax(l) (replacement token, bonus token) or from the residual
// norm(max(0, p - q)) of Eq. 1 (correction token).  One read of the row(s); probabilities live
// in registers only; per-step partial weights go to the last CTA that finishes a draw, which
// finds the crossing step and re-reads just that step (2 KB) to pick the token.
#include "draw_common.cuh"

namespace spr {

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
