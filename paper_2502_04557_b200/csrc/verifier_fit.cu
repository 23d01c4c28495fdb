// Preparing and fitting the verifier (Section 3.2): training labels 1[q(x)/p(x) <= lambda]
// from the two models' logits, and optimiser steps (binary cross-entropy + Adam) for the
// linear-layer + sigmoid verifier on the draft model's hidden states.
#include <string.h>

#include "host_util.h"
#include "launch.h"
#include "vocab_common.cuh"

namespace spr {

namespace {

constexpr int kStatRecord = 6;       // floats per row from shard_stats_kernel
constexpr int kMaxLambdas = 8;
constexpr int kTrainMaxVpl = 16;     // 16-byte vectors per lane: d <= 4096 (bf16) or 2048 (fp32)

// ---------------------------------------------------------------------------- labels
struct LabelParams {
    const float *stats;            // [M, 6] whole-row records (one shard covering the vocabulary)
    int64_t M;
    int V;
    const int32_t *draft_tokens;   // [M]
    int n_lambda;
    float lambdas[kMaxLambdas];
    uint8_t *labels;               // [n_lambda, M]
    float *ratio;                  // [M] or null
    int *status;
};

__global__ void __launch_bounds__(256) labels_kernel(const LabelParams prm)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= prm.M) return;
    const float *rec = prm.stats + i * kStatRecord;
    const int x = prm.draft_tokens[i];
    double ratio = -1.0;
    const bool valid = x >= 0 && x < prm.V;
    if (valid) {
        const double logP = (double)rec[4] - (double)rec[0] - log((double)rec[1]);
        const double logQ = (double)rec[5] - (double)rec[2] - log((double)rec[3]);
        ratio = exp(logQ - logP);
    } else {
        raise_status(prm.status, SPR_ERR_BAD_TOKEN);
    }
    for (int l = 0; l < prm.n_lambda; ++l)
        prm.labels[(int64_t)l * prm.M + i] = (valid && ratio <= (double)prm.lambdas[l]) ? 1 : 0;
    if (prm.ratio) prm.ratio[i] = (float)ratio;
}

// ---------------------------------------------------------------------------- training
struct TrainParams {
    const void *hidden;      // [N, d]
    const uint8_t *labels;   // [N]
    int64_t N;
    int d;
    float *theta, *m, *v;    // [d+1]: weights, then the bias
    int t;
    float lr, beta1, beta2, eps;
    float *loss;             // [1] or null
    float *part;             // [ctas, d+2]: per-CTA sums of the gradient terms, then of the loss
    int ctas;
    int stages;              // rows a warp keeps in flight (queue variant)
};

// Gradient pass (one resident wave of CTAs): one warp per sample, samples dealt to warps in a
// fixed pattern; a lane keeps
// its columns of the row in registers, so every hidden state is read from HBM exactly once.
//   z = b + w.s,  r = sigma(z) - y,  grad_w += r s,  grad_b += r,  loss += ln(1 + e^z) - y z
// The warps of a CTA add their sums in warp order; the CTA's sums go to part[blockIdx.x].
template <typename T, int VPL>
__global__ void __launch_bounds__(kThreads, VPL <= 3 ? 3 : (VPL <= 8 ? 2 : 1)) train_grad_kernel(const TrainParams prm)
{
    constexpr int N = Vec<T>::N;
    extern __shared__ float smem[];
    const int d = prm.d;
    float *sw = smem;              // [d] weights
    float *red = smem + d;         // [d + 2] CTA sums
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nv = d / N;          // vectors per row
    for (int j = tid; j < d; j += kThreads) sw[j] = prm.theta[j];
    const float bias = prm.theta[d];
    __syncthreads();

    uint64_t acc[VPL * N / 2];       // packed pairs of fp32 sums (two columns each)
#pragma unroll
    for (int e = 0; e < VPL * N / 2; ++e) acc[e] = pack2(0.f, 0.f);
    double acc_b = 0.0, acc_loss = 0.0;   // same-signed addends: fp32 sums would drift
    const T *base = static_cast<const T *>(prm.hidden);
    constexpr bool kPrefetch = VPL <= 4;   // short rows: keep the next row in flight as well
    auto load_row = [&](int64_t row, uint4 (&dst)[VPL], float &y) {
        const uint4 *x = reinterpret_cast<const uint4 *>(base + row * d);
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int vi = j * 32 + lane;
            dst[j] = vi < nv ? ld_stream(x + vi) : make_uint4(0u, 0u, 0u, 0u);
        }
        y = (float)prm.labels[row];
    };
    const int64_t stride = (int64_t)gridDim.x * kWarps;
    int64_t row = (int64_t)blockIdx.x * kWarps + warp;
    uint4 raw[VPL];
    float y = 0.f;
    if (row < prm.N) load_row(row, raw, y);
    for (; row < prm.N; row += stride) {
        uint4 nxt[VPL];
        float y_nxt = 0.f;
        const bool more = row + stride < prm.N;
        if (kPrefetch && more) load_row(row + stride, nxt, y_nxt);
        uint64_t dot2 = pack2(0.f, 0.f);   // even and odd columns apart
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int vi = j * 32 + lane;
            if (vi < nv) {
                float f[N];
                Vec<T>::unpack(raw[j], f);
#pragma unroll
                for (int e = 0; e < N; e += 2)
                    dot2 = fma2(pack2(f[e], f[e + 1]), *reinterpret_cast<const uint64_t *>(&sw[vi * N + e]), dot2);
            }
        }
        float d_even, d_odd;
        unpack2(dot2, d_even, d_odd);
        const float z = warp_sum(d_even + d_odd) + bias;
        const float r = 1.f / (1.f + expf(-z)) - y;
        const uint64_t r2 = pack2(r, r);
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            float f[N];
            Vec<T>::unpack(raw[j], f);     // zero beyond the row
#pragma unroll
            for (int e = 0; e < N; e += 2)
                acc[(j * N + e) / 2] = fma2(r2, pack2(f[e], f[e + 1]), acc[(j * N + e) / 2]);
        }
        acc_b += (double)r;
        acc_loss += (double)(fmaxf(z, 0.f) + log1pf(expf(-fabsf(z))) - y * z);
        if (kPrefetch) {
#pragma unroll
            for (int j = 0; j < VPL; ++j) raw[j] = nxt[j];
            y = y_nxt;
        } else if (more) {
            load_row(row + stride, raw, y);
        }
    }

    for (int w = 0; w < kWarps; ++w) {     // fixed order: warp 0 stores, the others add
        if (warp == w) {
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const int vi = j * 32 + lane;
                if (vi < nv) {
#pragma unroll
                    for (int e = 0; e < N; e += 2) {
                        float lo, hi;
                        unpack2(acc[(j * N + e) / 2], lo, hi);
                        float *dst = red + vi * N + e;
                        dst[0] = w == 0 ? lo : dst[0] + lo;
                        dst[1] = w == 0 ? hi : dst[1] + hi;
                    }
                }
            }
            if (lane == 0) {
                red[d] = w == 0 ? (float)acc_b : red[d] + (float)acc_b;
                red[d + 1] = w == 0 ? (float)acc_loss : red[d + 1] + (float)acc_loss;
            }
        }
        __syncthreads();
    }
    float *out = prm.part + (int64_t)blockIdx.x * (d + 2);
    for (int j = tid; j < d + 2; j += kThreads) out[j] = red[j];
}

// Short rows (at most 4 vectors per lane, d <= 1024 bf16): the same pass, but a warp's next
// `depth` rows are already on their way into shared memory (cp.async, 16 bytes per lane per
// copy) while it works on the current one, and the weights stay in registers.  A lane reads back
// only what it copied itself, so the queue needs no barrier: cp.async.wait_group orders a lane's
// own copies.  With 16 warps and 8 rows each an SM has ~190 KB of hidden states in flight.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
                 "l"(gmem_src)
                 : "memory");
}

template <typename T, int VPL>
__global__ void __launch_bounds__(kThreads, 2) train_grad_queue_kernel(const TrainParams prm)
{
    constexpr int N = Vec<T>::N;
    extern __shared__ __align__(16) unsigned char qsmem[];
    const int d = prm.d, depth = prm.stages;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nv = d / N;                     // vectors per row
    const int slot_vecs = VPL * 32;           // vectors per queue slot
    uint4 *queue = reinterpret_cast<uint4 *>(qsmem) + (size_t)warp * depth * slot_vecs;
    float *red = reinterpret_cast<float *>(qsmem + (size_t)kWarps * depth * slot_vecs * 16);   // [d + 2] CTA sums

    uint64_t w2[VPL * N / 2];                 // this lane's columns of the weight vector
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        const int vi = j * 32 + lane;
#pragma unroll
        for (int e = 0; e < N; e += 2)
            w2[(j * N + e) / 2] = vi < nv ? pack2(prm.theta[vi * N + e], prm.theta[vi * N + e + 1]) : pack2(0.f, 0.f);
    }
    const float bias = prm.theta[d];
    uint64_t acc[VPL * N / 2];
#pragma unroll
    for (int e = 0; e < VPL * N / 2; ++e) acc[e] = pack2(0.f, 0.f);
    double acc_b = 0.0, acc_loss = 0.0;

    const T *base = static_cast<const T *>(prm.hidden);
    const int64_t stride = (int64_t)gridDim.x * kWarps;
    const int64_t first = (int64_t)blockIdx.x * kWarps + warp;
    const int64_t n = first < prm.N ? (prm.N - first + stride - 1) / stride : 0;   // this warp's rows
    auto enqueue = [&](int64_t i, int slot) {       // row i of this warp -> queue slot (one commit group)
        if (i < n) {
            const uint4 *x = reinterpret_cast<const uint4 *>(base + (first + i * stride) * d);
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const int vi = j * 32 + lane;
                if (vi < nv) cp_async16(queue + slot * slot_vecs + vi, x + vi);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    for (int s = 0; s < depth; ++s) enqueue(s, s);
    float y = n > 0 ? (float)prm.labels[first] : 0.f;
    int slot = 0;
    for (int64_t i = 0; i < n; ++i) {
        const float y_next = i + 1 < n ? (float)prm.labels[first + (i + 1) * stride] : 0.f;
        // all but the newest depth-1 groups are complete: row i has landed
        if (depth == 8) asm volatile("cp.async.wait_group 7;" ::: "memory");
        else if (depth == 4) asm volatile("cp.async.wait_group 3;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        uint4 raw[VPL];
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int vi = j * 32 + lane;
            raw[j] = vi < nv ? queue[slot * slot_vecs + vi] : make_uint4(0u, 0u, 0u, 0u);
        }
        enqueue(i + depth, slot);               // the slot is free again: its values are in registers
        uint64_t dot2 = pack2(0.f, 0.f);
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            float f[N];
            Vec<T>::unpack(raw[j], f);
#pragma unroll
            for (int e = 0; e < N; e += 2) dot2 = fma2(pack2(f[e], f[e + 1]), w2[(j * N + e) / 2], dot2);
        }
        float d_even, d_odd;
        unpack2(dot2, d_even, d_odd);
        const float z = warp_sum(d_even + d_odd) + bias;
        const float r = 1.f / (1.f + expf(-z)) - y;
        const uint64_t r2 = pack2(r, r);
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            float f[N];
            Vec<T>::unpack(raw[j], f);
#pragma unroll
            for (int e = 0; e < N; e += 2)
                acc[(j * N + e) / 2] = fma2(r2, pack2(f[e], f[e + 1]), acc[(j * N + e) / 2]);
        }
        acc_b += (double)r;
        acc_loss += (double)(fmaxf(z, 0.f) + log1pf(expf(-fabsf(z))) - y * z);
        y = y_next;
        if (++slot == depth) slot = 0;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    for (int w = 0; w < kWarps; ++w) {     // fixed order: warp 0 stores, the others add
        if (warp == w) {
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const int vi = j * 32 + lane;
                if (vi < nv) {
#pragma unroll
                    for (int e = 0; e < N; e += 2) {
                        float lo, hi;
                        unpack2(acc[(j * N + e) / 2], lo, hi);
                        float *dst = red + vi * N + e;
                        dst[0] = w == 0 ? lo : dst[0] + lo;
                        dst[1] = w == 0 ? hi : dst[1] + hi;
                    }
                }
            }
            if (lane == 0) {
                red[d] = w == 0 ? (float)acc_b : red[d] + (float)acc_b;
                red[d + 1] = w == 0 ? (float)acc_loss : red[d + 1] + (float)acc_loss;
            }
        }
        __syncthreads();
    }
    float *out = prm.part + (int64_t)blockIdx.x * (d + 2);
    for (int j = tid; j < d + 2; j += kThreads) out[j] = red[j];
}

// One thread per parameter: sums the CTA partials in CTA order, divides by N, applies the
// bias-corrected Adam update (arithmetic in double, state kept in float).
__global__ void __launch_bounds__(256) train_adam_kernel(const TrainParams prm)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int d = prm.d;
    if (j > d + 1) return;
    double sum = 0.0;
    for (int c = 0; c < prm.ctas; ++c) sum += (double)prm.part[(int64_t)c * (d + 2) + j];
    sum /= (double)prm.N;
    if (j == d + 1) {
        if (prm.loss) *prm.loss = (float)sum;
        return;
    }
    const double b1 = (double)prm.beta1, b2 = (double)prm.beta2;
    const double m = b1 * (double)prm.m[j] + (1.0 - b1) * sum;
    const double v = b2 * (double)prm.v[j] + (1.0 - b2) * sum * sum;
    const double m_hat = m / (1.0 - pow(b1, (double)prm.t));
    const double v_hat = v / (1.0 - pow(b2, (double)prm.t));
    prm.m[j] = (float)m;
    prm.v[j] = (float)v;
    prm.theta[j] = (float)((double)prm.theta[j] - (double)prm.lr * m_hat / (sqrt(v_hat) + (double)prm.eps));
}

template <typename T, int VPL>
cudaError_t launch_grad(const TrainParams &tp, cudaStream_t st)
{
    const size_t smem = sizeof(float) * (2 * (size_t)tp.d + 2);
    cudaError_t e = cudaFuncSetAttribute(train_grad_kernel<T, VPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    // one full wave: as many CTAs as are resident at once, so that all of them finish together
    int per_sm = 0, dev = 0, sms = 0;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, train_grad_kernel<T, VPL>, kThreads, smem)) !=
            cudaSuccess ||
        (e = cudaGetDevice(&dev)) != cudaSuccess ||
        (e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return e;
    TrainParams p = tp;
    p.ctas = (int)max((int64_t)1, min((int64_t)min(kTrainMaxCtas, per_sm * sms), (tp.N + kWarps - 1) / kWarps));
    train_grad_kernel<T, VPL><<<p.ctas, kThreads, smem, st>>>(p);
    train_adam_kernel<<<(tp.d + 2 + 255) / 256, 256, 0, st>>>(p);
    return cudaGetLastError();
}

template <typename T, int VPL>
cudaError_t launch_grad_queue(const TrainParams &tp, cudaStream_t st)
{
    TrainParams p = tp;
    const size_t slot_bytes = (size_t)kWarps * VPL * 32 * 16;       // one queue slot of every warp
    p.stages = slot_bytes * 8 <= 96 * 1024 ? 8 : 4;
    const size_t smem = slot_bytes * p.stages + sizeof(float) * ((size_t)tp.d + 2);
    cudaError_t e = cudaFuncSetAttribute(train_grad_queue_kernel<T, VPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    int per_sm = 0, dev = 0, sms = 0;
    if (e != cudaSuccess ||
        (e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, train_grad_queue_kernel<T, VPL>, kThreads, smem)) !=
            cudaSuccess ||
        (e = cudaGetDevice(&dev)) != cudaSuccess ||
        (e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return e;
    if (per_sm < 1) return cudaErrorInvalidConfiguration;
    p.ctas = (int)max((int64_t)1, min((int64_t)min(kTrainMaxCtas, per_sm * sms), (tp.N + kWarps - 1) / kWarps));
    train_grad_queue_kernel<T, VPL><<<p.ctas, kThreads, smem, st>>>(p);
    train_adam_kernel<<<(tp.d + 2 + 255) / 256, 256, 0, st>>>(p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_grad_any(const TrainParams &tp, cudaStream_t st)
{
    const int vpl = (tp.d / Vec<T>::N + 31) / 32;
    if (vpl <= 1) return launch_grad_queue<T, 1>(tp, st);
    if (vpl <= 2) return launch_grad_queue<T, 2>(tp, st);
    if (vpl <= 3) return launch_grad_queue<T, 3>(tp, st);
    if (vpl <= 4) return launch_grad_queue<T, 4>(tp, st);
    if (vpl <= 8) return launch_grad<T, 8>(tp, st);
    return launch_grad<T, 16>(tp, st);
}


}  // namespace

}  // namespace spr

using namespace spr;

extern "C" {

int verifier_labels(const void *p_logits, const void *q_logits, int64_t ldv, const int32_t *draft_tokens, int B,
                    int K, int Kp, int V, int dt, const float *lambdas, int n_lambda, uint8_t *labels, float *ratio,
                    void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!dtype_ok(dt)) return SPR_ERR_UNSUPPORTED;
    if (B < 0 || K <= 0 || Kp < K || V <= 0 || V > (1 << 30) || ldv < V || (int64_t)B * K > 0x7fffffff ||
        n_lambda <= 0 || n_lambda > kMaxLambdas || !lambdas)
        return SPR_ERR_INVALID_ARG;
    if (B == 0) return SPR_OK;
    if (!p_logits || !q_logits || !draft_tokens || !labels) return SPR_ERR_INVALID_ARG;
    const size_t es = elem_size(dt);
    if (!aligned(p_logits, es) || !aligned(q_logits, es) || !aligned(draft_tokens, 4) || (ratio && !aligned(ratio, 4)))
        return SPR_ERR_INVALID_ARG;
    Carver cv = carve(ws_bytes);
    const LabelWs lay = label_ws_layout(cv, B, K, stat_max_segments_per_row(V, dt));
    if (!ws || !aligned(ws, 256) || !cv.fits()) return SPR_ERR_WORKSPACE;
    int rc = device_supported();
    if (rc != SPR_OK) return rc;

    const int64_t M = (int64_t)B * K;
    ShardStatsParams sp;
    memset(&sp, 0, sizeof sp);
    sp.p = p_logits;
    sp.q = q_logits;
    sp.ldv = ldv;
    sp.V = V;
    sp.v0 = 0;
    sp.K = K;
    sp.Kp = Kp;
    sp.Kr = K;   // the bonus row has no draft token
    draw_geometry((int)M, stat_steps_per_row(V, dt), &sp.chunks, &sp.iters);
    sp.draft_tokens = draft_tokens;
    sp.stats = at<float>(ws, lay.stats);
    sp.row_counters = at<int>(ws, lay.row_counters);
    sp.part = at<float4>(ws, lay.part);
    LabelParams lp;
    memset(&lp, 0, sizeof lp);
    lp.stats = sp.stats;
    lp.M = M;
    lp.V = V;
    lp.draft_tokens = draft_tokens;
    lp.n_lambda = n_lambda;
    for (int l = 0; l < n_lambda; ++l) lp.lambdas[l] = lambdas[l];
    lp.labels = labels;
    lp.ratio = ratio;
    lp.status = at<int>(ws, 0);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(sp.row_counters, 0, sizeof(int) * (size_t)M, st);
    if (e == cudaSuccess) e = launch_shard_stats(sp, M, dt, st);
    if (e == cudaSuccess) {
        labels_kernel<<<(unsigned)((M + 255) / 256), 256, 0, st>>>(lp);
        e = cudaGetLastError();
    }
    return finish(e);
}

int verifier_train_step(const void *hidden, const uint8_t *labels, int64_t N, int d, int dt, float *theta,
                        float *adam_m, float *adam_v, int t, float lr, float beta1, float beta2, float eps,
                        float *loss, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!dtype_ok(dt)) return SPR_ERR_UNSUPPORTED;
    if (N < 0 || d <= 0 || t < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) ||
        !(eps >= 0.f) || !(lr == lr))
        return SPR_ERR_INVALID_ARG;
    const int vec = vec_elems(dt);
    if (d % vec != 0 || d / vec > 32 * kTrainMaxVpl) return SPR_ERR_UNSUPPORTED;
    if (N == 0) return SPR_OK;
    if (!hidden || !labels || !theta || !adam_m || !adam_v) return SPR_ERR_INVALID_ARG;
    if (!aligned(hidden, 16) || !aligned(theta, 4) || !aligned(adam_m, 4) || !aligned(adam_v, 4) ||
        (loss && !aligned(loss, 4)))
        return SPR_ERR_INVALID_ARG;
    Carver cv = carve(ws_bytes);
    const size_t part_off = train_ws_layout(cv, d);
    if (!ws || !aligned(ws, 256) || !cv.fits()) return SPR_ERR_WORKSPACE;
    int rc = device_supported();
    if (rc != SPR_OK) return rc;

    TrainParams tp;
    memset(&tp, 0, sizeof tp);
    tp.hidden = hidden;
    tp.labels = labels;
    tp.N = N;
    tp.d = d;
    tp.theta = theta;
    tp.m = adam_m;
    tp.v = adam_v;
    tp.t = t;
    tp.lr = lr;
    tp.beta1 = beta1;
    tp.beta2 = beta2;
    tp.eps = eps;
    tp.loss = loss;
    tp.part = at<float>(ws, part_off);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    return finish(dt == SPR_F32 ? launch_grad_any<float>(tp, st) : launch_grad_any<__nv_bfloat16>(tp, st));
}

}  // extern "C"
