// Shared tail of the verifier kernels: logit -> score -> accept bit, and the first-rejection
// scan, from global memory or from a tile's accept codes kept in shared memory.
#pragma once

#include "common.cuh"
#include "launch.h"

namespace spr {

// accept codes a finishing CTA keeps in shared memory
enum { ACC_REJECT = 0, ACC_ACCEPT = 1, ACC_INVALID = 2 };

// A kernel whose bounded wait ran out hands on NaN instead of a partial sum: the token's score
// is then reported as -1, its accept bit as 0 and its sequence's first_reject as -1.
__device__ __forceinline__ float poisoned_z() { return __int_as_float(0x7fc00000); }

// score, accept bit and (optionally) the score output of token m from its logit z
__device__ __forceinline__ int classify_token(const VerifyParams &prm, float z, int m)
{
    if (z != z) {
        if (prm.scores) prm.scores[m] = -1.f;
        prm.accept[m] = 0;
        return ACC_INVALID;
    }
    const double score = 1.0 / (1.0 + exp(-(double)z));
    if (prm.scores) prm.scores[m] = (float)score;
    const int a = score >= (double)prm.threshold ? ACC_ACCEPT : ACC_REJECT;
    prm.accept[m] = (uint8_t)a;
    return a;
}

// first rejection of sequence b = lowest set bit of the reject ballot (one warp per call);
// accept bits from global memory.  poisoned: a bounded wait ran out somewhere in this launch.
__device__ inline void scan_sequence(const VerifyParams &prm, int b, int lane, bool poisoned = false)
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
    if (lane == 0) prm.first_reject[b] = poisoned ? -1 : first;
}

// the same scan over accept codes in shared memory: codes[k] for the K tokens of the sequence
__device__ inline void scan_sequence_smem(const VerifyParams &prm, int b, const unsigned char *codes, int lane)
{
    int first = prm.K;
    bool invalid = false;
    for (int k0 = 0; k0 < prm.K; k0 += 32) {
        const int k = k0 + lane;
        const unsigned a = k < prm.K ? (unsigned)codes[k] : (unsigned)ACC_ACCEPT;
        invalid |= __any_sync(0xffffffffu, a == (unsigned)ACC_INVALID);
        const unsigned rej = __ballot_sync(0xffffffffu, a != (unsigned)ACC_ACCEPT);
        if (rej != 0u && first == prm.K) first = k0 + __ffs(rej) - 1;
    }
    if (lane == 0) prm.first_reject[b] = invalid ? -1 : first;
}

__device__ __forceinline__ bool launch_poisoned(const VerifyParams &prm)
{
    return *reinterpret_cast<volatile int *>(prm.status) == SPR_ERR_TIMEOUT;
}

// Tokens [m_lo, m_hi): z = b2 + sum over slices (ascending), sigmoid, threshold; then the
// scan of every sequence that lies completely inside the range, one warp per sequence.
// codes: shared memory for m_hi - m_lo accept codes (the scan then needs no trip through
// global memory), or null.
__device__ inline void finalise_tile(const VerifyParams &prm, int m_lo, int m_hi, unsigned char *codes = nullptr)
{
    const int M = prm.B * prm.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float b2 = prm.b2[0];
    for (int m = m_lo + tid; m < m_hi; m += blockDim.x) {
        float z = b2;
        for (int s = 0; s < prm.slices; ++s) z += __ldcg(&prm.part_z[(int64_t)s * M + m]);
        const int a = classify_token(prm, z, m);
        if (codes) codes[m - m_lo] = (unsigned char)a;
    }
    if (!codes) __threadfence();
    __syncthreads();
    if (!prm.first_reject) return;
    const int nwarps = blockDim.x >> 5;
    const int b_lo = (m_lo + prm.K - 1) / prm.K, b_hi = m_hi / prm.K;
    if (codes) {
        for (int b = b_lo + warp; b < b_hi; b += nwarps) scan_sequence_smem(prm, b, codes + (b * prm.K - m_lo), lane);
    } else {
        const bool poisoned = launch_poisoned(prm);
        for (int b = b_lo + warp; b < b_hi; b += nwarps) scan_sequence(prm, b, lane, poisoned);
    }
}

// Sequences cut by a tile boundary (multiples of `tile` tokens): scanned by whoever finishes
// last overall, once every tile has written its accept bits.
__device__ inline void finalise_straddlers(const VerifyParams &prm, int tile)
{
    if (!prm.first_reject) return;
    const int M = prm.B * prm.K;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const bool poisoned = launch_poisoned(prm);
    for (int t = 1 + warp; (int64_t)t * tile < M; t += nwarps) {
        const int edge = t * tile;
        if (edge % prm.K == 0) continue;                 // boundary falls between sequences
        const int b = edge / prm.K;
        if ((int64_t)b * prm.K < edge - tile) continue;  // already handled at an earlier boundary
        scan_sequence(prm, b, lane, poisoned);
    }
}

// whole batch in one CTA
__device__ inline void finalise_scores(const VerifyParams &prm) { finalise_tile(prm, 0, prm.B * prm.K); }

}  // namespace spr
