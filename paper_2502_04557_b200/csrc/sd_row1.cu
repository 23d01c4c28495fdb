// sd_verify for one draft position per sequence (K = 1, no bonus row): the keep-or-resample
// rule of Section 3 ("Algorithm") on a token the verifier rejected.  Here the correction draw
// would re-read half of all rows, so the row pair is kept on chip instead: a cluster of eight
// CTAs takes one (p, q) row pair, every CTA stages an eighth of both rows in shared memory with
// two bulk asynchronous copies, computes its softmax statistics from there, the eight CTAs
// exchange them through distributed shared memory, and on a rejection each CTA forms the
// residual weights of Eq. 1 of its part from the same staged data.  HBM is read once.
#include <cooperative_groups.h>

#include "draw_common.cuh"

namespace cg = cooperative_groups;

namespace spr {

namespace {

constexpr int kCluster = 8;                 // CTAs per row pair (the portable cluster size)
constexpr int kMaxSegSteps = 16;            // warp steps (2 KB each) a CTA stages per row: 32 KB + 32 KB
constexpr uint32_t kSpinLimit = 1u << 22;   // polls of mbarrier.try_wait before giving up

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait: false when the phase did not complete within kSpinLimit polls
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> shared copy of `bytes` (a multiple of 16, both addresses 16-byte aligned) that
// completes on `bar`
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

struct Row1Params {
    const void *p;   // [B, ldv]
    const void *q;   // [B, ldv]
    int64_t ldv;
    int V, steps, seg_steps;       // warp steps per row, and per CTA
    const int32_t *draft_tokens;   // [B]
    const float *uniforms;         // [B, 2]
    int32_t *accepted_len, *correction_token;
    uint8_t *accept;
    float *p_tok, *q_tok, *residual_mass;
    int *status;
    float2 *part;                  // [B * steps] step weights of the residual
};

struct Slot {   // what a CTA tells its cluster about its part of the row pair
    float m_p, s_p, m_q, s_q, lpx, lqx;
};

struct Decision {
    int acc;          // 0 reject, 1 accept, 2 invalid draft token
    float cp, cq;     // (max + ln Z) * log2(e) of the whole p row and q row
};

// One warp step out of the staged segment: vector j of lane l is vector step*128 + j*32 + l of
// the segment; vectors past the end of the row read as -inf (V is a multiple of the vector).
template <typename T>
__device__ __forceinline__ void staged_step(const uint4 *seg, int step, int first_elem, int V, int lane,
                                            uint4 (&raw)[kUnroll])
{
    constexpr int N = Vec<T>::N;
    const uint32_t f = sizeof(T) == 4 ? 0xff800000u : 0xff80ff80u;
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) {
        const int v = j * 32 + lane;
        raw[j] = first_elem + v * N < V ? seg[step * (32 * kUnroll) + v] : make_uint4(f, f, f, f);
    }
}

template <typename T>
__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads, 3) sd_row1_kernel(const Row1Params prm)
{
    constexpr int N = Vec<T>::N;
    constexpr int kStep = 32 * kUnroll * N;
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(128) unsigned char staged[];   // this CTA's part of the p row, then of the q row
    __shared__ __align__(8) uint64_t bar;
    __shared__ float4 s_part[kWarps];
    __shared__ Slot slot;
    __shared__ Decision dec;
    __shared__ DrawSmem sm;

    const int rank = (int)cluster.block_rank();
    const int b = blockIdx.x / kCluster;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = prm.V, S = prm.seg_steps;
    const int step0 = rank * S;                                       // this CTA's first step of the row
    const int my_steps = max(0, min(S, prm.steps - step0));
    const int e0 = step0 * kStep;                                     // ... and first element
    const int n_el = max(0, min(V - e0, S * kStep));
    const uint32_t bytes = (uint32_t)n_el * sizeof(T);
    const T *prow = static_cast<const T *>(prm.p) + (int64_t)b * prm.ldv;
    const T *qrow = static_cast<const T *>(prm.q) + (int64_t)b * prm.ldv;
    uint4 *sp = reinterpret_cast<uint4 *>(staged);
    uint4 *sq = reinterpret_cast<uint4 *>(staged + (size_t)S * kStep * sizeof(T));

    if (tid == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0 && bytes) {
        mbar_expect_tx(&bar, 2 * bytes);
        bulk_load(sp, prow + e0, bytes, &bar);
        bulk_load(sq, qrow + e0, bytes, &bar);
    }
    const float u_acc = prm.uniforms[(int64_t)b * 2], u_draw = prm.uniforms[(int64_t)b * 2 + 1];
    const int x = prm.draft_tokens[b];
    // every thread polls; a wait that runs out is reported and the CTA goes on with empty
    // statistics, so that it still meets its cluster at every barrier below
    const int landed = __syncthreads_and(bytes == 0 || mbar_wait(&bar, 0));
    if (!landed && tid == 0) raise_status(prm.status, SPR_ERR_TIMEOUT);

    // ---- statistics of this CTA's part, from shared memory
    MS mp{neg_inf(), 0.f}, mq{neg_inf(), 0.f};
    if (landed) {
        for (int s = warp; s < my_steps; s += kWarps) {
            uint4 rp[kUnroll], rq[kUnroll];
            staged_step<T>(sp, s, e0 + s * kStep, V, lane, rp);
            staged_step<T>(sq, s, e0 + s * kStep, V, lane, rq);
            online_update<T>(rp, mp.m, mp.s);
            online_update<T>(rq, mq.m, mq.s);
        }
    }
    mp = warp_ms(mp);
    mq = warp_ms(mq);
    if (lane == 0) s_part[warp] = make_float4(mp.m, mp.s, mq.m, mq.s);
    __syncthreads();
    if (warp == 0) {
        const float4 v = lane < kWarps ? s_part[lane] : make_float4(neg_inf(), 0.f, neg_inf(), 0.f);
        mp = warp_ms(MS{v.x, v.y});
        mq = warp_ms(MS{v.z, v.w});
        if (lane == 0) {
            slot.m_p = mp.m;
            slot.s_p = mp.s;
            slot.m_q = mq.m;
            slot.s_q = mq.s;
            slot.lpx = slot.lqx = neg_inf();
            if (landed && x >= e0 && x < e0 + n_el) {   // the draft token's logits are staged here
                const T *tp = reinterpret_cast<const T *>(sp), *tq = reinterpret_cast<const T *>(sq);
                if (sizeof(T) == 4) {
                    slot.lpx = reinterpret_cast<const float *>(tp)[x - e0];
                    slot.lqx = reinterpret_cast<const float *>(tq)[x - e0];
                } else {
                    slot.lpx = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(tp)[x - e0]);
                    slot.lqx = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(tq)[x - e0]);
                }
            }
        }
    }
    cluster.sync();

    // ---- every CTA merges the eight parts in rank order (fp64) and takes the same decision
    if (warp == 0) {
        Slot v = {neg_inf(), 0.f, neg_inf(), 0.f, neg_inf(), neg_inf()};
        if (lane < kCluster) v = *cluster.map_shared_rank(&slot, lane);
        const float m_p = warp_max(v.m_p), m_q = warp_max(v.m_q);
        const float lpx = warp_max(v.lpx), lqx = warp_max(v.lqx);
        double z_p = 0.0, z_q = 0.0;
        for (int g = 0; g < kCluster; ++g) {
            const float a_m = __shfl_sync(0xffffffffu, v.m_p, g), a_s = __shfl_sync(0xffffffffu, v.s_p, g);
            const float b_m = __shfl_sync(0xffffffffu, v.m_q, g), b_s = __shfl_sync(0xffffffffu, v.s_q, g);
            if (a_s > 0.f) z_p += (double)a_s * exp((double)a_m - (double)m_p);
            if (b_s > 0.f) z_q += (double)b_s * exp((double)b_m - (double)m_q);
        }
        if (lane == 0) {
            const double lnz_p = log(z_p), lnz_q = log(z_q);
            int acc;
            float P = -1.f, Q = -1.f;
            if (x < 0 || x >= V) {
                acc = 2;
                if (rank == 0) raise_status(prm.status, SPR_ERR_BAD_TOKEN);
            } else {
                const double logP = (double)lpx - (double)m_p - lnz_p;
                const double logQ = (double)lqx - (double)m_q - lnz_q;
                acc = ((double)u_acc <= fmin(1.0, exp(logP - logQ))) ? 1 : 0;
                P = (float)exp(logP);
                Q = (float)exp(logQ);
            }
            dec.acc = acc;
            dec.cp = (m_p + (float)lnz_p) * kLog2e;
            dec.cq = (m_q + (float)lnz_q) * kLog2e;
            if (rank == 0) {
                prm.accepted_len[b] = acc == 2 ? -1 : acc;
                if (prm.accept) prm.accept[b] = acc == 1 ? 1 : 0;
                if (prm.p_tok) prm.p_tok[b] = P;
                if (prm.q_tok) prm.q_tok[b] = Q;
                if (acc != 0) {
                    prm.correction_token[b] = -1;
                    if (prm.residual_mass) prm.residual_mass[b] = 0.f;
                }
            }
        }
    }
    __syncthreads();

    // ---- rejected: residual weights of this CTA's steps, again from shared memory
    const bool rejected = dec.acc == 0;
    float2 *part = prm.part + (int64_t)b * prm.steps;
    if (rejected) {
        for (int s = warp; s < my_steps; s += kWarps) {
            uint4 rp[kUnroll], rq[kUnroll];
            float w = 0.f;
            if (landed) {
                staged_step<T>(sp, s, e0 + s * kStep, V, lane, rp);
                staged_step<T>(sq, s, e0 + s * kStep, V, lane, rq);
                w = warp_sum(residual_step_sum<T>(rp, rq, dec.cp, dec.cq));
            }
            if (lane == 0) part[step0 + s] = make_float2(0.f, w);
        }
        __threadfence();
    }
    cluster.sync();   // also the last use of the other CTAs' shared memory is behind us here

    // ---- the first CTA adds the step weights in step order and locates the token (the one
    //      2 KB step it needs comes from L2)
    if (rejected && rank == 0) {
        Job<T> job;
        job.mode = MODE_RESIDUAL;
        job.p_row = prow;
        job.q_row = qrow;
        job.cp = dec.cp;
        job.cq = dec.cq;
        job.u = u_draw;
        const int token = finish_draw<T>(job, MODE_RESIDUAL, V, prm.steps, kStatIters, part, sm,
                                         prm.residual_mass ? prm.residual_mass + b : nullptr);
        if (tid == 0) prm.correction_token[b] = token;
    }
}

}  // namespace

// Takes sd_verify calls with K = Kp = 1 whose rows can be staged: 16-byte aligned rows of
// whole vectors, at most kCluster * kMaxSegSteps warp steps long.
bool sd_row1_applies(const void *p, const void *q, int64_t ldv, int K, int Kp, int V, int dt)
{
    const size_t es = elem_size(dt);
    if (K != 1 || Kp != 1) return false;
    if ((reinterpret_cast<uintptr_t>(p) | reinterpret_cast<uintptr_t>(q)) & 15) return false;
    if (((size_t)ldv * es) % 16 != 0 || ((size_t)V * es) % 16 != 0) return false;
    return stat_steps_per_row(V, dt) <= kCluster * kMaxSegSteps;
}

cudaError_t launch_sd_row1(const SdParams &sp, float2 *part, int32_t *correction_token, float *residual_mass, int B,
                           int dt, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    if ((int64_t)B * kCluster > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    Row1Params rp;
    rp.p = sp.p;
    rp.q = sp.q;
    rp.ldv = sp.ldv;
    rp.V = sp.V;
    rp.steps = stat_steps_per_row(sp.V, dt);
    rp.seg_steps = (rp.steps + kCluster - 1) / kCluster;
    rp.draft_tokens = sp.draft_tokens;
    rp.uniforms = sp.uniforms;
    rp.accepted_len = sp.accepted_len;
    rp.correction_token = correction_token;
    rp.accept = sp.accept;
    rp.p_tok = sp.p_tok;
    rp.q_tok = sp.q_tok;
    rp.residual_mass = residual_mass;
    rp.status = sp.status;
    rp.part = part;
    const size_t smem = 2 * (size_t)rp.seg_steps * stat_step_elems(dt) * elem_size(dt);
    cudaError_t e;
    if (dt == SPR_F32) {
        e = cudaFuncSetAttribute(sd_row1_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) sd_row1_kernel<float><<<(unsigned)(B * kCluster), kThreads, smem, st>>>(rp);
    } else {
        e = cudaFuncSetAttribute(sd_row1_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e == cudaSuccess) sd_row1_kernel<__nv_bfloat16><<<(unsigned)(B * kCluster), kThreads, smem, st>>>(rp);
    }
    return e == cudaSuccess ? cudaGetLastError() : e;
}

}  // namespace spr
