// Monte-Carlo of the run length N of Theorems 2 and 3: how many draft tokens in a row an
// i.i.d. verifier accepts when the first r are acceptable (accepted with probability eta_TP)
// and the rest are not (accepted with probability eta_FP).  One Philox4x32-10 stream per run,
// so every run is reproducible on its own; pure integer/ALU work, no memory traffic beyond
// the optional per-run output.
#include "common.cuh"
#include "launch.h"

namespace spr {

namespace {

constexpr int kSimThreads = 256;
constexpr int kSimMaxBins = 1024;   // histogram bins kept in shared memory

// Philox4x32-10 (Salmon et al., SC'11): 10 rounds of two 32x32->64 multiplies and a key bump
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t (&out)[4])
{
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

__global__ void __launch_bounds__(kSimThreads) simulate_kernel(const SimParams prm)
{
    __shared__ unsigned int s_hist[kSimMaxBins];
    const int bins = prm.max_tokens + 1;
    const bool smem_hist = prm.histogram != nullptr && bins <= kSimMaxBins;
    if (smem_hist)
        for (int i = threadIdx.x; i < bins; i += kSimThreads) s_hist[i] = 0u;
    __syncthreads();
    const uint32_t k0 = (uint32_t)prm.seed, k1 = (uint32_t)(prm.seed >> 32);
    for (int64_t j = (int64_t)blockIdx.x * kSimThreads + threadIdx.x; j < prm.runs;
         j += (int64_t)gridDim.x * kSimThreads) {
        const uint64_t run = (uint64_t)(prm.first_run + j);
        int n = 0;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        while (n < prm.max_tokens) {
            if ((n & 3) == 0) philox4x32_10((uint32_t)run, (uint32_t)(run >> 32), (uint32_t)(n >> 2), 0u, k0, k1, w);
            const uint32_t word = (n & 3) == 0 ? w[0] : (n & 3) == 1 ? w[1] : (n & 3) == 2 ? w[2] : w[3];
            const float u = (float)(word >> 8) * 5.9604644775390625e-8f;   // 24 bits -> [0, 1)
            const float eta = n < prm.r ? prm.eta_tp : prm.eta_fp;
            if (!(u < eta)) break;
            ++n;
        }
        if (prm.n_accepted) prm.n_accepted[j] = n;
        if (prm.histogram) {
            if (smem_hist)
                atomicAdd(&s_hist[n], 1u);
            else
                atomicAdd(&prm.histogram[n], 1ull);
        }
    }
    __syncthreads();
    if (smem_hist)
        for (int i = threadIdx.x; i < bins; i += kSimThreads)
            if (s_hist[i]) atomicAdd(&prm.histogram[i], (unsigned long long)s_hist[i]);
}

}  // namespace

cudaError_t launch_simulate(const SimParams &sp, cudaStream_t st)
{
    if (sp.runs == 0) return cudaSuccess;
    // at most a few waves of CTAs, each thread striding over runs
    int64_t blocks = (sp.runs + kSimThreads - 1) / kSimThreads;
    if (blocks > 148 * 32) blocks = 148 * 32;
    simulate_kernel<<<(unsigned)blocks, kSimThreads, 0, st>>>(sp);
    return cudaGetLastError();
}

}  // namespace spr
