// Building blocks shared by the vocabulary kernels: 16-byte vectors of logits, row addressing
// that keeps every interior load aligned whatever the row's own alignment, and the lane-local
// softmax statistics.
#pragma once

#include "common.cuh"
#include "launch.h"

namespace spr {

// ---------------------------------------------------------------- 16-byte vectors
template <typename T>
struct Vec;

template <>
struct Vec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[N])
    {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ float vmax(const uint4 &v)
    {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)),
                     fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    // elements i0 .. i0+3 of the row, -inf where the index falls outside [0, V)
    static __device__ __forceinline__ uint4 gather(const float *row, int i0, int V)
    {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int i = i0 + e;
            w[e] = (i >= 0 && i < V) ? __float_as_uint(row[i]) : 0xff800000u;
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

template <>
struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[N])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            f[2 * j] = __uint_as_float(w[j] << 16);
            f[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ float vmax(const uint4 &v)
    {
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&v.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&v.y);
        const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162 *>(&v.z);
        const __nv_bfloat162 d = *reinterpret_cast<const __nv_bfloat162 *>(&v.w);
        const __nv_bfloat162 m = __hmax2(__hmax2(a, b), __hmax2(c, d));
        return fmaxf(__low2float(m), __high2float(m));
    }
    static __device__ __forceinline__ uint4 gather(const __nv_bfloat16 *row, int i0, int V)
    {
        const unsigned short *r = reinterpret_cast<const unsigned short *>(row);
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int a = i0 + 2 * j, b = a + 1;
            const uint32_t lo = (a >= 0 && a < V) ? (uint32_t)r[a] : 0xff80u;
            const uint32_t hi = (b >= 0 && b < V) ? (uint32_t)r[b] : 0xff80u;
            w[j] = lo | (hi << 16);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Elements i0 .. i0+N-1 of a row as one vector.  One 16-byte load when the vector lies
// inside the row and its address is 16-byte aligned, element loads with -inf fill otherwise.
template <typename T>
__device__ __forceinline__ uint4 load_vec(const T *__restrict__ row, int i0, int V)
{
    constexpr int N = Vec<T>::N;
    if (i0 >= 0 && i0 + N <= V && (reinterpret_cast<uintptr_t>(row + i0) & 15) == 0)
        return ld_stream(reinterpret_cast<const uint4 *>(row + i0));
    if (i0 + N <= 0 || i0 >= V) {
        const uint32_t f = sizeof(T) == 4 ? 0xff800000u : 0xff80ff80u;
        return make_uint4(f, f, f, f);
    }
    return Vec<T>::gather(row, i0, V);
}

// Number of elements by which the row start lies past a 16-byte boundary.  Warp steps start at
// element step*kStep - pad of the row, which makes every interior vector 16-byte aligned
// whatever the row's own alignment.
template <typename T>
__device__ __forceinline__ int row_pad(const T *row)
{
    return (int)((reinterpret_cast<uintptr_t>(row) & 15) / sizeof(T));
}

// Two fp32 lanes per instruction (sm_100 packed fp32): halves the issue slots of the multiply-
// add and of the accumulation, which matter here because the exp pipe and the issue rate are
// the co-limiters of the streaming kernels.
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// (max, sum of exp(x - max)) over the kUnroll vectors a thread holds; the multiply-add and the
// accumulation run on pairs of fp32 lanes (the issue rate is a co-limiter of the streaming loops)
template <typename T>
__device__ __forceinline__ MS thread_ms(const uint4 (&raw)[kUnroll])
{
    constexpr int N = Vec<T>::N;
    float m = Vec<T>::vmax(raw[0]);
#pragma unroll
    for (int j = 1; j < kUnroll; ++j) m = fmaxf(m, Vec<T>::vmax(raw[j]));
    const float ref = (m == neg_inf()) ? 0.f : m;
    const float off = -ref * kLog2e;
    const uint64_t scale2 = pack2(kLog2e, kLog2e), off2 = pack2(off, off);
    uint64_t acc[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float f[N];
        Vec<T>::unpack(raw[j], f);
        acc[j] = pack2(0.f, 0.f);
#pragma unroll
        for (int e = 0; e < N; e += 2) {
            float t0, t1;
            unpack2(fma2(pack2(f[e], f[e + 1]), scale2, off2), t0, t1);
            acc[j] = add2(acc[j], pack2(ex2(t0), ex2(t1)));
        }
    }
    float a0, a1, b0, b1;
    unpack2(add2(acc[0], acc[1]), a0, a1);
    unpack2(add2(acc[2], acc[3]), b0, b1);
    MS r;
    r.m = m;
    r.s = (a0 + a1) + (b0 + b1);
    return r;
}

// Lane-local online softmax statistics: folds kUnroll vectors into a running (max, sum of
// exp(x - max)).  When the maximum grows the old sum is rescaled once per call.
template <typename T>
__device__ __forceinline__ void online_update(const uint4 (&raw)[kUnroll], float &m, float &s)
{
    constexpr int N = Vec<T>::N;
    float g = Vec<T>::vmax(raw[0]);
#pragma unroll
    for (int j = 1; j < kUnroll; ++j) g = fmaxf(g, Vec<T>::vmax(raw[j]));
    const float mn = fmaxf(m, g);
    const float ref = (mn == neg_inf()) ? 0.f : mn;
    const float off = -ref * kLog2e;
    const uint64_t scale2 = pack2(kLog2e, kLog2e), off2 = pack2(off, off);
    uint64_t acc[kUnroll];
    acc[0] = pack2(s * ex2(fmaf(m, kLog2e, off)), 0.f);   // m = -inf: exp2(-inf) = 0
#pragma unroll
    for (int j = 1; j < kUnroll; ++j) acc[j] = pack2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        float f[N];
        Vec<T>::unpack(raw[j], f);
#pragma unroll
        for (int e = 0; e < N; e += 2) {
            float t0, t1;
            unpack2(fma2(pack2(f[e], f[e + 1]), scale2, off2), t0, t1);
            acc[j] = add2(acc[j], pack2(ex2(t0), ex2(t1)));
        }
    }
    m = mn;
    float a0, a1, b0, b1;
    unpack2(add2(acc[0], acc[1]), a0, a1);
    unpack2(add2(acc[2], acc[3]), b0, b1);
    s = (a0 + a1) + (b0 + b1);
}

// The kUnroll vectors of one warp step: vector j of lane l starts at element
// first + (j*32 + l)*N of the row (first may be negative or run past V at the row's ends).
template <typename T>
__device__ __forceinline__ void load_step(const T *__restrict__ row, int first, int V, int lane,
                                          uint4 (&raw)[kUnroll])
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    if (first >= 0 && first + kStep <= V) {   // interior: aligned by construction
        const uint4 *p = reinterpret_cast<const uint4 *>(row + first) + lane;
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) raw[j] = ld_stream(p + j * 32);
    } else {
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) raw[j] = load_vec<T>(row, first + (j * 32 + lane) * N, V);
    }
}

// One warp's share of a row segment: its ITERS steps (warp steps are kWarps steps apart),
// starting at element first_p of the p row and first_q of the q row (HAS_Q), folded into the
// lane-local statistics.  The loads of a warp's next step are issued before the current one is
// consumed.  When every step is made of whole aligned vectors inside the row(s) - warp-uniform,
// and true for all but the warps at a row's ends - the loop carries no condition at all, which
// the compiler unrolls and schedules freely (4 % of the row-statistics pass); same arithmetic in
// the same order either way.
template <typename T, int ITERS, bool HAS_Q>
__device__ __forceinline__ void stream_segment(const T *__restrict__ prow, const T *__restrict__ qrow, int first_p,
                                               int first_q, int V, int lane, MS &mp, MS &mq)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    constexpr int kLast = (ITERS - 1) * kWarps * kStep;
    uint4 rp[kUnroll], rq[kUnroll];
    if (first_p >= 0 && first_q >= 0 && first_p + kLast + kStep <= V && first_q + kLast + kStep <= V) {
        const uint4 *pp = reinterpret_cast<const uint4 *>(prow + first_p) + lane;
        const uint4 *qq = reinterpret_cast<const uint4 *>(qrow + first_q) + lane;
        constexpr int kNext = kWarps * kStep / N;     // vectors from one step of a warp to its next
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            rp[j] = ld_stream(pp + j * 32);
            if (HAS_Q) rq[j] = ld_stream(qq + j * 32);
        }
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            online_update<T>(rp, mp.m, mp.s);
            if (it + 1 < ITERS) {
#pragma unroll
                for (int j = 0; j < kUnroll; ++j) rp[j] = ld_stream(pp + (it + 1) * kNext + j * 32);
            }
            if (HAS_Q) {
                online_update<T>(rq, mq.m, mq.s);
                if (it + 1 < ITERS) {
#pragma unroll
                    for (int j = 0; j < kUnroll; ++j) rq[j] = ld_stream(qq + (it + 1) * kNext + j * 32);
                }
            }
        }
        return;
    }
    load_step<T>(prow, first_p, V, lane, rp);
    if (HAS_Q) load_step<T>(qrow, first_q, V, lane, rq);
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        const int nxt = (it + 1) * kWarps * kStep;
        const bool more = it + 1 < ITERS && min(first_p, first_q) + nxt < V;   // warp-uniform
        online_update<T>(rp, mp.m, mp.s);
        if (more) load_step<T>(prow, first_p + nxt, V, lane, rp);
        if (HAS_Q) {
            online_update<T>(rq, mq.m, mq.s);
            if (more) load_step<T>(qrow, first_q + nxt, V, lane, rq);
        }
        if (!more) break;
    }
}

}  // namespace spr
