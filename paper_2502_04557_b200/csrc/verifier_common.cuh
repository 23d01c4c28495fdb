// Shared tail of the verifier kernels.
#pragma once

#include "common.cuh"
#include "launch.h"

namespace spr {

// Last CTA: z = b2 + sum over slices (ascending), sigmoid, threshold, then the scan: one
// warp per sequence, first rejection = lowest set bit of the reject ballot.
__device__ inline void finalise_scores(const VerifyParams &prm)
{
    const int M = prm.B * prm.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const double tau = (double)prm.threshold;
    const float b2 = prm.b2[0];
    for (int m = tid; m < M; m += blockDim.x) {
        float z = b2;
        for (int s = 0; s < prm.slices; ++s) z += __ldcg(&prm.part_z[(int64_t)s * M + m]);
        const double score = 1.0 / (1.0 + exp(-(double)z));
        if (prm.scores) prm.scores[m] = (float)score;
        prm.accept[m] = score >= tau ? 1 : 0;
    }
    __syncthreads();
    if (!prm.first_reject) return;
    const int nwarps = blockDim.x >> 5;
    for (int b = warp; b < prm.B; b += nwarps) {
        int first = prm.K;
        for (int k0 = 0; k0 < prm.K; k0 += 32) {
            const int k = k0 + lane;
            const unsigned a = k < prm.K ? (unsigned)prm.accept[(int64_t)b * prm.K + k] : 1u;
            const unsigned rej = __ballot_sync(0xffffffffu, a == 0u);
            if (rej != 0u) {
                first = k0 + __ffs(rej) - 1;
                break;
            }
        }
        if (lane == 0) prm.first_reject[b] = first;
    }
}


}  // namespace spr
