// Shared tail of the verifier kernels.
#pragma once

#include "common.cuh"
#include "launch.h"

namespace spr {

// first rejection of sequence b = lowest set bit of the reject ballot (one warp per call)
__device__ inline void scan_sequence(const VerifyParams &prm, int b, int lane)
{
    int first = prm.K;
    for (int k0 = 0; k0 < prm.K; k0 += 32) {
        const int k = k0 + lane;
        const unsigned a = k < prm.K ? (unsigned)__ldcg(&prm.accept[(int64_t)b * prm.K + k]) : 1u;
        const unsigned rej = __ballot_sync(0xffffffffu, a == 0u);
        if (rej != 0u) {
            first = k0 + __ffs(rej) - 1;
            break;
        }
    }
    if (lane == 0) prm.first_reject[b] = first;
}

// Tokens [m_lo, m_hi): z = b2 + sum over slices (ascending), sigmoid, threshold; then the
// scan of every sequence that lies completely inside the range, one warp per sequence.
__device__ inline void finalise_tile(const VerifyParams &prm, int m_lo, int m_hi)
{
    const int M = prm.B * prm.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const double tau = (double)prm.threshold;
    const float b2 = prm.b2[0];
    for (int m = m_lo + tid; m < m_hi; m += blockDim.x) {
        float z = b2;
        for (int s = 0; s < prm.slices; ++s) z += __ldcg(&prm.part_z[(int64_t)s * M + m]);
        const double score = 1.0 / (1.0 + exp(-(double)z));
        if (prm.scores) prm.scores[m] = (float)score;
        prm.accept[m] = score >= tau ? 1 : 0;
    }
    __threadfence();
    __syncthreads();
    if (!prm.first_reject) return;
    const int nwarps = blockDim.x >> 5;
    const int b_lo = (m_lo + prm.K - 1) / prm.K, b_hi = m_hi / prm.K;
    for (int b = b_lo + warp; b < b_hi; b += nwarps) scan_sequence(prm, b, lane);
}

// Sequences cut by a tile boundary (multiples of `tile` tokens): scanned by whoever finishes
// last overall, once every tile has written its accept bits.
__device__ inline void finalise_straddlers(const VerifyParams &prm, int tile)
{
    if (!prm.first_reject) return;
    const int M = prm.B * prm.K;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int t = 1 + warp; (int64_t)t * tile < M; t += nwarps) {
        const int edge = t * tile;
        if (edge % prm.K == 0) continue;                 // boundary falls between sequences
        const int b = edge / prm.K;
        if ((int64_t)b * prm.K < edge - tile) continue;  // already handled at an earlier boundary
        scan_sequence(prm, b, lane);
    }
}

// whole batch in one CTA
__device__ inline void finalise_scores(const VerifyParams &prm) { finalise_tile(prm, 0, prm.B * prm.K); }

}  // namespace spr
