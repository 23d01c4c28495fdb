// SIMT verifiers.  MLP: score = sigmoid(b2 + W2 . relu(W1 s + b1)) for any element type and
// shape - the path for float32 inputs and for batches too small for a tensor-core tile, where
// the work is a bandwidth-bound sweep over W1.  Linear: the paper's single layer,
// score = sigmoid(b + w . s).  Both end with the threshold test and the first-rejection scan.
#include "common.cuh"
#include "launch.h"
#include "verifier_common.cuh"

namespace spr {

constexpr int kTokTile = 8;  // tokens processed per sweep over a W1 row

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__device__ __forceinline__ void unpack16(const uint4 &v, float (&f)[16 / sizeof(T)]);
template <>
__device__ __forceinline__ void unpack16<float>(const uint4 &v, float (&f)[4])
{
    f[0] = __uint_as_float(v.x);
    f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z);
    f[3] = __uint_as_float(v.w);
}
template <>
__device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4 &v, float (&f)[8])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        f[2 * j] = __uint_as_float(w[j] << 16);
        f[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
}

// dot products of one weight row with up to kTokTile hidden rows, result in every lane
template <typename T>
__device__ __forceinline__ void warp_dots(const T *__restrict__ wrow, const T *__restrict__ hid, int d,
                                          int m0, int M, bool vec_ok, float (&acc)[kTokTile])
{
    constexpr int N = 16 / sizeof(T);
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int t = 0; t < kTokTile; ++t) acc[t] = 0.f;
    if (vec_ok) {
#pragma unroll 4
        for (int i = lane * N; i < d; i += 32 * N) {   // several weight vectors in flight per lane
            float w[N];
            unpack16<T>(__ldg(reinterpret_cast<const uint4 *>(wrow + i)), w);
#pragma unroll
            for (int t = 0; t < kTokTile; ++t) {
                if (m0 + t < M) {
                    float x[N];
                    unpack16<T>(__ldg(reinterpret_cast<const uint4 *>(hid + (int64_t)(m0 + t) * d + i)), x);
#pragma unroll
                    for (int e = 0; e < N; ++e) acc[t] = fmaf(w[e], x[e], acc[t]);
                }
            }
        }
    } else {
        for (int i = lane; i < d; i += 32) {
            const float w = to_f32<T>(wrow[i]);
#pragma unroll
            for (int t = 0; t < kTokTile; ++t)
                if (m0 + t < M) acc[t] = fmaf(w, to_f32<T>(hid[(int64_t)(m0 + t) * d + i]), acc[t]);
        }
    }
#pragma unroll
    for (int t = 0; t < kTokTile; ++t) acc[t] = warp_sum(acc[t]);
}

template <typename T>
__global__ void __launch_bounds__(kThreads) verifier_simt_kernel(const VerifyParams prm)
{
    __shared__ float s_z[kWarps][kTokTile];
    __shared__ int s_last;
    pdl_trigger();   // a replacement draw launched behind this grid may be scheduled now
    const int M = prm.B * prm.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *hid = static_cast<const T *>(prm.hidden);
    const T *W1 = static_cast<const T *>(prm.W1);
    constexpr int N = 16 / sizeof(T);
    const bool vec_ok = (prm.d % N == 0) && ((reinterpret_cast<uintptr_t>(hid) & 15) == 0) &&
                        ((reinterpret_cast<uintptr_t>(W1) & 15) == 0);

    if (prm.h > 0) {
        // slice = kWarps consecutive hidden units, one per warp
        const int slice = blockIdx.x;
        const int j = slice * kWarps + warp;
        float b1j = 0.f, w2j = 0.f;
        if (j < prm.h) {
            b1j = prm.b1[j];
            w2j = to_f32<T>(static_cast<const T *>(prm.W2)[j]);
        }
        for (int m0 = 0; m0 < M; m0 += kTokTile) {
            float acc[kTokTile];
            if (j < prm.h) {
                warp_dots<T>(W1 + (int64_t)j * prm.d, hid, prm.d, m0, M, vec_ok, acc);
            } else {
#pragma unroll
                for (int t = 0; t < kTokTile; ++t) acc[t] = 0.f;
            }
            if (lane == 0) {
#pragma unroll
                for (int t = 0; t < kTokTile; ++t)
                    s_z[warp][t] = (j < prm.h) ? w2j * fmaxf(acc[t] + b1j, 0.f) : 0.f;
            }
            __syncthreads();
            if (tid < kTokTile && m0 + tid < M) {
                float z = 0.f;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) z += s_z[w][tid];
                prm.part_z[(int64_t)slice * M + m0 + tid] = z;
            }
            __syncthreads();
        }
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = take_ticket(prm.counter, (int)gridDim.x);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    finalise_scores(prm);
}

// The paper's verifier: one linear layer and a sigmoid.  A bandwidth-bound sweep over the hidden
// states: one warp per token reads its row once with 16-byte loads (the weight vector stays in
// L1), forms the score and the accept bit on the spot, and takes a ticket on its sequence;
// the warp that completes a sequence runs the first-rejection scan.  No partial sums, no
// single-CTA tail.
template <typename T>
__global__ void __launch_bounds__(kThreads) verifier_linear_kernel(const VerifyParams prm)
{
    pdl_trigger();   // a replacement draw launched behind this grid may be scheduled now
    constexpr int N = 16 / sizeof(T);
    const int M = prm.B * prm.K;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int m = blockIdx.x * kWarps + warp;
    if (m >= M) return;
    const T *w = static_cast<const T *>(prm.W1);
    const T *x = static_cast<const T *>(prm.hidden) + (int64_t)m * prm.d;
    const bool vec_ok = (prm.d % N == 0) && ((reinterpret_cast<uintptr_t>(prm.hidden) & 15) == 0) &&
                        ((reinterpret_cast<uintptr_t>(w) & 15) == 0);
    float acc = 0.f;
    if (vec_ok) {
#pragma unroll 4
        for (int i = lane * N; i < prm.d; i += 32 * N) {
            float wv[N], xv[N];
            unpack16<T>(__ldg(reinterpret_cast<const uint4 *>(w + i)), wv);
            unpack16<T>(__ldg(reinterpret_cast<const uint4 *>(x + i)), xv);
#pragma unroll
            for (int e = 0; e < N; ++e) acc = fmaf(wv[e], xv[e], acc);
        }
    } else {
        for (int i = lane; i < prm.d; i += 32) acc = fmaf(to_f32<T>(w[i]), to_f32<T>(x[i]), acc);
    }
    const float z = warp_sum(acc) + prm.b2[0];
    const int b = m / prm.K;
    int ticket = 0;
    if (lane == 0) {
        const double score = 1.0 / (1.0 + exp(-(double)z));
        if (prm.scores) prm.scores[m] = (float)score;
        prm.accept[m] = score >= (double)prm.threshold ? 1 : 0;
        __threadfence();
        ticket = take_ticket(&prm.counter[1 + b], prm.K);
    }
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (!ticket || !prm.first_reject) return;
    __threadfence();
    scan_sequence(prm, b, lane);
}

int verifier_simt_slices(int h) { return h > 0 ? (h + kWarps - 1) / kWarps : 1; }

cudaError_t launch_verifier_simt(const VerifyParams &vp, int dt, cudaStream_t st)
{
    if (vp.h == 0) {   // single linear layer
        const int64_t grid = ((int64_t)vp.B * vp.K + kWarps - 1) / kWarps;
        if (grid <= 0) return cudaSuccess;
        if (dt == SPR_F32)
            verifier_linear_kernel<float><<<(unsigned)grid, kThreads, 0, st>>>(vp);
        else
            verifier_linear_kernel<__nv_bfloat16><<<(unsigned)grid, kThreads, 0, st>>>(vp);
        return cudaGetLastError();
    }
    const int grid = verifier_simt_slices(vp.h);
    if (dt == SPR_F32)
        verifier_simt_kernel<float><<<grid, kThreads, 0, st>>>(vp);
    else
        verifier_simt_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(vp);
    return cudaGetLastError();
}

}  // namespace spr
