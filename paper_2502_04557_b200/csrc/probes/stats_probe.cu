// Measurement aid, not part of the library: the streaming loop of the row-statistics pass
// (online softmax of a p step and a q step per warp turn, the library's own online_update) on
// plain arrays, and the same with the features of the real kernel added one at a time - the
// CTA's epilogue chain, row addressing with run-time checks, rows at the pitch of a 128256-entry
// vocabulary - so that the gap between the kernel and the bare loop can be read off in parts.
// The table in profiles/sd_row_stats_kernel_llama3.md comes from this program
// (python -m paper_2502_04557_b200.stream_probes).
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include "vocab_common.cuh"
using namespace spr;
typedef __nv_bfloat16 T;
#define CK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("err %s line %d\n", cudaGetErrorString(e), __LINE__); return 1; } } while (0)

constexpr int kStepVecs = 32 * kUnroll;   // uint4 per step (2 KB)

// A: the kernel's structure on plain arrays: CTA = 32 steps, warp takes steps w, w+8, w+16, w+24
__global__ void __launch_bounds__(256, 4) kernel_a(const uint4 *p, const uint4 *q, float4 *out)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t base = ((size_t)blockIdx.x * 32 + warp) * kStepVecs + lane;
    MS mp{neg_inf(), 0.f}, mq{neg_inf(), 0.f};
    uint4 rp[kUnroll], rq[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) { rp[j] = ld_stream(p + base + j * 32); rq[j] = ld_stream(q + base + j * 32); }
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const size_t nx = base + (size_t)(it + 1) * 8 * kStepVecs;
        online_update<T>(rp, mp.m, mp.s);
        if (it < 3) {
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) rp[j] = ld_stream(p + nx + j * 32);
        }
        online_update<T>(rq, mq.m, mq.s);
        if (it < 3) {
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) rq[j] = ld_stream(q + nx + j * 32);
        }
    }
    mp = warp_ms(mp); mq = warp_ms(mq);
    if (lane == 0) out[(size_t)blockIdx.x * 8 + warp] = make_float4(mp.m, mp.s, mq.m, mq.s);
}


// A2: A plus the fused kernel's epilogue chain: CTA partial -> fence + ticket -> (last of 4) merge,
// two scattered logit reads, fp64 log/exp, store, fence + second ticket -> (last of 16) scan
__global__ void __launch_bounds__(256, 4) kernel_a2(const uint4 *p, const uint4 *q, float4 *part, int *row_cnt, int *seq_cnt,
                                                     unsigned char *acc, int *lens, const int *tok, int mode)
{
    __shared__ float4 s_part[8];
    __shared__ int s_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t base = ((size_t)blockIdx.x * 32 + warp) * kStepVecs + lane;
    MS mp{neg_inf(), 0.f}, mq{neg_inf(), 0.f};
    uint4 rp[kUnroll], rq[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) { rp[j] = ld_stream(p + base + j * 32); rq[j] = ld_stream(q + base + j * 32); }
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const size_t nx = base + (size_t)(it + 1) * 8 * kStepVecs;
        online_update<T>(rp, mp.m, mp.s);
        if (it < 3) {
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) rp[j] = ld_stream(p + nx + j * 32);
        }
        online_update<T>(rq, mq.m, mq.s);
        if (it < 3) {
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) rq[j] = ld_stream(q + nx + j * 32);
        }
    }
    mp = warp_ms(mp); mq = warp_ms(mq);
    if (lane == 0) s_part[warp] = make_float4(mp.m, mp.s, mq.m, mq.s);
    __syncthreads();
    if (warp != 0) return;
    const float4 v = lane < 8 ? s_part[lane] : make_float4(neg_inf(), 0.f, neg_inf(), 0.f);
    mp = warp_ms(MS{v.x, v.y}); mq = warp_ms(MS{v.z, v.w});
    const int row = blockIdx.x >> 2;
    if (lane == 0) {
        part[blockIdx.x] = make_float4(mp.m, mp.s, mq.m, mq.s);
        if (mode == 0) return;          // partials only: the CTA is done here
        __threadfence();
        s_last = atomicAdd(&row_cnt[row], 1) == 3;
        if (s_last) row_cnt[row] = 0;
    }
    if (mode == 0) return;
    __syncwarp();
    if (!s_last) return;
    __threadfence();
    double zp = 0, zq = 0; float m_p = neg_inf(), m_q = neg_inf();
    if (lane < 4) { const float4 w = __ldcg(&part[row * 4 + lane]); m_p = w.x; m_q = w.z; zp = w.y; zq = w.w; }
    m_p = warp_max(m_p); m_q = warp_max(m_q);
    for (int o = 16; o > 0; o >>= 1) { zp += __shfl_xor_sync(0xffffffffu, zp, o); zq += __shfl_xor_sync(0xffffffffu, zq, o); }
    int last_row = 0;
    if (lane == 0) {
        const int x = tok[row];
        const size_t rb = (size_t)row * 128 * kStepVecs * 8;    // elements
        const float lpx = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p)[rb + x]);
        const float lqx = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(q)[rb + x]);
        const double logP = (double)lpx - m_p - log(zp), logQ = (double)lqx - m_q - log(zq);
        acc[row] = exp(logP - logQ) > 0.5 ? 1 : 0;
        __threadfence();
        last_row = atomicAdd(&seq_cnt[row >> 4], 1) == 15;
        if (last_row) seq_cnt[row >> 4] = 0;
    }
    last_row = __shfl_sync(0xffffffffu, last_row, 0);
    if (!last_row) return;
    __threadfence();
    const unsigned a = lane < 16 ? (unsigned)__ldcg(&acc[(row & ~15) + lane]) : 1u;
    const unsigned rej = __ballot_sync(0xffffffffu, a != 1u);
    if (lane == 0) lens[row >> 4] = rej ? __ffs(rej) - 1 : 16;
}


// A3: A2's partial-only variant with the kernel's addressing: rows of V = 128256 elements
// (pitch not a multiple of a step), 4 segments of 32 steps per row of which 126 exist, p rows
// in groups of 17 of which 16 are read; the ragged last step is read as whole vectors (the
// buffer is padded) - only addressing and layout differ from A2 mode 0.
__global__ void __launch_bounds__(256, 4) kernel_a3(const T *p, const T *q, float4 *part, int V, int64_t ldv, int mode)
{
    __shared__ float4 s_part[8];
    constexpr int kStep = 1024, kSegment = 8 * 4 * kStep;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = blockIdx.x >> 2; const int c = blockIdx.x & 3;
    const int b = (int)(row >> 4), k = (int)(row & 15);
    const T *prow = p + ((int64_t)b * 17 + k) * ldv, *qrow = q + row * ldv;
    const int first = c * kSegment + warp * kStep;
    MS mp{neg_inf(), 0.f}, mq{neg_inf(), 0.f};
    uint4 rp[kUnroll], rq[kUnroll];
    auto ld = [&](const T *r, int f, uint4 (&dst)[kUnroll]) {
        const uint4 *x = reinterpret_cast<const uint4 *>(r + f) + lane;
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) dst[j] = (mode == 1 && f + (j * 32 + lane) * 8 >= V) ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u) : ld_stream(x + j * 32);
    };
    ld(prow, first, rp); ld(qrow, first, rq);
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int nxt = (it + 1) * 8 * kStep;
        const bool more = it + 1 < 4 && first + nxt < V;
        online_update<T>(rp, mp.m, mp.s);
        if (more) ld(prow, first + nxt, rp);
        online_update<T>(rq, mq.m, mq.s);
        if (more) ld(qrow, first + nxt, rq);
        if (!more) break;
    }
    mp = warp_ms(mp); mq = warp_ms(mq);
    if (lane == 0) s_part[warp] = make_float4(mp.m, mp.s, mq.m, mq.s);
    __syncthreads();
    if (warp != 0) return;
    const float4 v = lane < 8 ? s_part[lane] : make_float4(neg_inf(), 0.f, neg_inf(), 0.f);
    mp = warp_ms(MS{v.x, v.y}); mq = warp_ms(MS{v.z, v.w});
    if (lane == 0) part[blockIdx.x] = make_float4(mp.m, mp.s, mq.m, mq.s);
}

__device__ __forceinline__ uint32_t sa(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// B: persistent, per-warp ring of SLOTS slots (p step + q step each) fed by bulk copies
template <int SLOTS, int CPS>
__global__ void __launch_bounds__(256, CPS) kernel_b(const uint4 *p, const uint4 *q, float4 *out, int64_t n_steps, int *err)
{
    extern __shared__ __align__(128) unsigned char sm[];
    __shared__ __align__(8) uint64_t bars[8][SLOTS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint4 *ring = reinterpret_cast<uint4 *>(sm) + (size_t)warp * SLOTS * 2 * kStepVecs;
    uint64_t *bar = bars[warp];
    const int64_t stride = (int64_t)gridDim.x * 8, first = (int64_t)blockIdx.x * 8 + warp;
    const int n = first < n_steps ? (int)((n_steps - first + stride - 1) / stride) : 0;
    auto fetch = [&](int i, int s) {
        const size_t off = (size_t)(first + (int64_t)i * stride) * kStepVecs;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sa(&bar[s])), "r"(4096) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sa(ring + (2 * s) * kStepVecs)),
                     "l"(p + off), "r"(2048), "r"(sa(&bar[s])) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sa(ring + (2 * s + 1) * kStepVecs)),
                     "l"(q + off), "r"(2048), "r"(sa(&bar[s])) : "memory");
    };
    if (lane == 0) {
        for (int s = 0; s < SLOTS; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sa(&bar[s])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < SLOTS && i < n; ++i) fetch(i, i);
    }
    __syncwarp();
    MS mp{neg_inf(), 0.f}, mq{neg_inf(), 0.f};
    int s = 0; uint32_t par = 0;
    for (int i = 0; i < n; ++i) {
        bool ok = false;
        for (int k = 0; k < (1 << 22) && !ok; ++k) {
            uint32_t d;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(d) : "r"(sa(&bar[s])), "r"(par) : "memory");
            ok = d != 0;
        }
        if (!ok) { if (lane == 0) atomicExch(err, 1); break; }
        uint4 rp[kUnroll], rq[kUnroll];
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) { rp[j] = ring[(2 * s) * kStepVecs + j * 32 + lane]; rq[j] = ring[(2 * s + 1) * kStepVecs + j * 32 + lane]; }
        __syncwarp();
        if (lane == 0 && i + SLOTS < n) fetch(i + SLOTS, s);
        online_update<T>(rp, mp.m, mp.s);
        online_update<T>(rq, mq.m, mq.s);
        if ((i & 3) == 3) {   // a segment ends: reduce and write, as the kernel does per CTA
            const MS a = warp_ms(mp), b = warp_ms(mq);
            if (lane == 0) out[(first + (int64_t)i * stride) >> 2] = make_float4(a.m, a.s, b.m, b.s);
            mp = MS{neg_inf(), 0.f}; mq = MS{neg_inf(), 0.f};
        }
        if (++s == SLOTS) { s = 0; par ^= 1; }
    }
}

template <typename F>
float time_it(F f)
{
    cudaEvent_t a, b;
    cudaEventCreate(&a); cudaEventCreate(&b);
    for (int i = 0; i < 3; ++i) f();
    cudaEventRecord(a);
    for (int i = 0; i < 10; ++i) f();
    cudaEventRecord(b);
    cudaEventSynchronize(b);
    float ms; cudaEventElapsedTime(&ms, a, b);
    return ms / 10;
}

__global__ void fill(uint4 *x, size_t n, unsigned seed)
{
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        unsigned h = (unsigned)i * 2654435761u + seed;
        // bf16 values around [-4, 4): exponent bits of 1.0..4.0 with random mantissa and sign
        auto v = [&](unsigned r) { return (unsigned)(((r & 0x8000u)) | 0x3f80u + ((r >> 3) & 0xffu)) & 0xffffu; };
        uint4 o;
        o.x = v(h) | (v(h >> 7) << 16); h = h * 1664525u + 1013904223u;
        o.y = v(h) | (v(h >> 7) << 16); h = h * 1664525u + 1013904223u;
        o.z = v(h) | (v(h >> 7) << 16); h = h * 1664525u + 1013904223u;
        o.w = v(h) | (v(h >> 7) << 16);
        x[i] = o;
    }
}

int main()
{
    const int64_t n_steps = 1 << 19;            // 2 KB each for p and for q: 2.1 GB in all
    const size_t vecs = (size_t)n_steps * kStepVecs;
    uint4 *p, *q; float4 *out; int *err;
    CK(cudaMalloc(&p, vecs * 16)); CK(cudaMalloc(&q, vecs * 16)); CK(cudaMalloc(&out, (size_t)n_steps * 16)); CK(cudaMalloc(&err, 4));
    CK(cudaMemset(err, 0, 4));
    fill<<<1184, 256>>>(p, vecs, 1u); fill<<<1184, 256>>>(q, vecs, 77u);
    CK(cudaDeviceSynchronize());
    const double bytes = 2.0 * vecs * 16;
    float ms = time_it([&] { kernel_a<<<(unsigned)(n_steps / 32), 256>>>(p, q, out); });
    printf("A (CTA per 32 steps, register loads, 4 CTAs/SM): %.1f us  %.0f GB/s\n", ms * 1e3, bytes / ms / 1e6);
    {
        int *row_cnt, *seq_cnt, *lens, *tok; unsigned char *acc; float4 *part;
        const int rows = (int)(n_steps / 128);
        CK(cudaMalloc(&row_cnt, rows * 4)); CK(cudaMalloc(&seq_cnt, rows / 16 * 4)); CK(cudaMalloc(&lens, rows / 16 * 4));
        CK(cudaMalloc(&tok, rows * 4)); CK(cudaMalloc(&acc, rows)); CK(cudaMalloc(&part, (size_t)rows * 4 * 16));
        CK(cudaMemset(row_cnt, 0, rows * 4)); CK(cudaMemset(seq_cnt, 0, rows / 16 * 4)); CK(cudaMemset(tok, 0, rows * 4));
        for (int mode = 0; mode < 2; ++mode) {
            ms = time_it([&] { kernel_a2<<<(unsigned)(n_steps / 32), 256>>>(p, q, part, row_cnt, seq_cnt, acc, lens, tok, mode); });
            printf("A2 mode %d (%s): %.1f us  %.0f GB/s\n", mode, mode ? "ticket chain in the CTA" : "partials only", ms * 1e3, bytes / ms / 1e6);
        }
        CK(cudaGetLastError());
    }
    for (int cfg = 0; cfg < 4; ++cfg) {
        const int V = cfg == 0 ? 131072 : 128256, rows = 4096;
        const int64_t ldv = cfg == 3 ? 128256 : (cfg == 2 ? 128256 + 768 : 131072);
        T *p3, *q3; float4 *part;
        const size_t pe = (size_t)(rows / 16) * 17 * ldv + 4096, qe = (size_t)rows * ldv + 4096;
        CK(cudaMalloc(&p3, pe * 2)); CK(cudaMalloc(&q3, qe * 2)); CK(cudaMalloc(&part, (size_t)rows * 4 * 16));
        fill<<<1184, 256>>>(reinterpret_cast<uint4 *>(p3), pe / 8, 5u); fill<<<1184, 256>>>(reinterpret_cast<uint4 *>(q3), qe / 8, 9u);
        CK(cudaDeviceSynchronize());
        const double b3 = 2.0 * rows * V * 2;
        for (int mode = 0; mode < 2; ++mode) {
            ms = time_it([&] { kernel_a3<<<rows * 4, 256>>>(p3, q3, part, V, ldv, mode); });
            printf("A3 (row addressing with run-time checks%s) V=%d pitch=%lld elements: %.1f us  %.0f GB/s\n", mode ? ", vectors past V not read" : "", V, (long long)ldv, ms * 1e3, b3 / ms / 1e6);
        }
        CK(cudaGetLastError());
        CK(cudaFree(p3)); CK(cudaFree(q3)); CK(cudaFree(part));
    }
#define RUN_B(SL, CPS) { CK(cudaFuncSetAttribute(kernel_b<SL, CPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * SL * 4096)); \
        ms = time_it([&] { kernel_b<SL, CPS><<<148 * CPS, 256, 8 * SL * 4096>>>(p, q, out, n_steps, err); }); \
        printf("B ring %d slots, %d CTAs/SM (persistent): %.1f us  %.0f GB/s\n", SL, CPS, ms * 1e3, bytes / ms / 1e6); }
    RUN_B(1, 4) RUN_B(2, 3) RUN_B(2, 2)
    CK(cudaDeviceSynchronize());
    int h = 0; CK(cudaMemcpy(&h, err, 4, cudaMemcpyDeviceToHost));
    printf("err flag %d\n", h);
    return 0;
}
