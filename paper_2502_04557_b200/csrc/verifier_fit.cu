// Preparing and fitting the verifier (Section 3.2): training labels 1[q(x)/p(x) <= lambda]
// from the two models' logits, and optimiser steps (binary cross-entropy + Adam) for the
// linear-layer + sigmoid verifier on the draft model's hidden states.
#include <string.h>

#include <type_traits>

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
    int *status;             // the workspace's status word
    uint32_t spin_limit;     // polls of one mbarrier before the gradient kernel gives up
    int test_flags;          // TRAIN_TEST_NO_FETCH
};
enum { TRAIN_TEST_NO_FETCH = 1 };   // test hook: no row is ever fetched, so the first wait of every team runs out

// Gradient pass (one resident wave of CTAs), every hidden state read from HBM exactly once:
//   z = b + w.s,  r = sigma(z) - y,  grad_w += r s,  grad_b += r,  loss += ln(1 + e^z) - y z
// Rows are dealt to teams of warps in a fixed pattern, the teams of a CTA add their sums in team
// order and the CTA's sums go to part[blockIdx.x]: the result does not depend on timing.
// Rows go through shared memory.  A team of WPR warps (one warp, or two for rows
// of more than 8 vectors per lane) owns a ring of SLOTS row buffers, each filled by ONE
// bulk copy (a row is contiguous) that signals the slot's mbarrier.  The team works on R rows
// at a time straight out of the ring - their logits are independent chains (dot product, warp
// sum, sigmoid), which hides those latencies with few warps on the SM - while the other
// SLOTS - R rows are on their way.  A lane keeps its columns of the weights and of the
// gradient sums in registers; with two warps per row each warp has half of the columns and the
// two halves of a dot product meet in shared memory.  A slot is refilled as soon as both
// passes over it are done.
constexpr uint32_t kRingSpin = 1u << 22;      // polls of one mbarrier before the kernel gives up

__device__ __forceinline__ uint32_t ring_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool ring_poll(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(ring_addr(bar)), "r"(parity)
        : "memory");
    return done != 0u;
}
__device__ __forceinline__ bool ring_wait(uint64_t *bar, uint32_t parity, uint32_t limit)
{
    for (uint32_t n = 0; n < limit; ++n)
        if (ring_poll(bar, parity)) return true;
    return false;
}
// one row: global -> shared, completion counted in bytes on the slot's mbarrier (one lane calls)
__device__ __forceinline__ void ring_fetch(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(ring_addr(bar)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     ring_addr(dst)),
                 "l"(src), "r"(bytes), "r"(ring_addr(bar))
                 : "memory");
}
__device__ __forceinline__ bool feeder_team_has_copies(const TrainParams &prm) { return !(prm.test_flags & TRAIN_TEST_NO_FETCH); }
// the warps of one team meet (a warp alone: its lanes)
template <int WPR>
__device__ __forceinline__ void team_sync(int team)
{
    if (WPR == 1) __syncwarp();
    else asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(WPR * 32) : "memory");
}

__host__ __device__ constexpr int ring_ctas_per_sm(int vpl, int wpr, int g) { return g > 1 ? 2 : (wpr == 1 && vpl <= 4 ? 2 : 1); }

// G: consecutive rows per slot and per bulk copy (short rows: a copy of 4 KB instead of 512 bytes);
// a team then takes blocks of G rows, and R divides G so that the rows a team works on together
// lie in one slot.
template <typename T, int VPL, int WPR, int R, int SLOTS, int G>
__global__ void __launch_bounds__(kThreads, ring_ctas_per_sm(VPL, WPR, G)) train_grad_ring_kernel(const TrainParams prm)
{
    static_assert(G == 1 || (G % R == 0 && WPR == 1), "the rows of a group share a slot");
    constexpr int N = Vec<T>::N;
    constexpr int kTeams = kWarps / WPR;
    constexpr int kSlotVecs = VPL * WPR * 32 * G;
    extern __shared__ __align__(128) unsigned char rsmem[];
    __shared__ __align__(8) uint64_t bars[kTeams][SLOTS];
    __shared__ float halves[kTeams][R][2];    // WPR = 2: the two warps' parts of the R dot products
    __shared__ int team_fail[kTeams];         // WPR = 2: a wait of one of the team's warps ran out
    const int d = prm.d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int team = warp / WPR, half = warp % WPR;
    const int nv = d / N;
    const uint32_t row_bytes = (uint32_t)d * (uint32_t)sizeof(T);   // a multiple of 16: d is a multiple of N
    uint4 *ring = reinterpret_cast<uint4 *>(rsmem) + (size_t)team * SLOTS * kSlotVecs;
    float *red = reinterpret_cast<float *>(rsmem + (size_t)kTeams * SLOTS * kSlotVecs * 16);   // [d + 2]
    uint64_t *bar = bars[team];
    const int v0 = half * VPL * 32 + lane;    // this lane's vectors of a row: v0 + 32 j

    uint64_t w2[VPL * N / 2];                 // this lane's columns of the weight vector
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        const int vi = v0 + j * 32;
#pragma unroll
        for (int e = 0; e < N; e += 2)
            w2[(j * N + e) / 2] = vi < nv ? pack2(prm.theta[vi * N + e], prm.theta[vi * N + e + 1]) : pack2(0.f, 0.f);
    }
    const float bias = prm.theta[d];
    uint64_t acc[VPL * N / 2];
#pragma unroll
    for (int e = 0; e < VPL * N / 2; ++e) acc[e] = pack2(0.f, 0.f);
    double acc_b = 0.0, acc_loss = 0.0;       // per lane: see the note on z_keep below
    float z_keep = 0.f, y_keep = 0.f, r_keep = 0.f;
    int kept = 0;

    // Blocks of G consecutive rows are dealt to the teams in a fixed pattern; block k of this team
    // is block first + k * stride of the data, goes to slot k % SLOTS and is its (k / SLOTS)-th fill.
    const T *base = static_cast<const T *>(prm.hidden);
    const int64_t blocks = (prm.N + G - 1) / G;
    const int64_t stride = (int64_t)gridDim.x * kTeams;
    const int64_t first = (int64_t)blockIdx.x * kTeams + team;
    const int nb = first < blocks ? (int)((blocks - first + stride - 1) / stride) : 0;   // this team's blocks
    // only the last block of the data can be short, and it is the last of its team
    const int rows_last = nb > 0 ? (int)min((int64_t)G, prm.N - (first + (int64_t)(nb - 1) * stride) * G) : 0;
    const int n = nb > 0 ? (nb - 1) * G + rows_last : 0;                                 // this team's rows
    auto rows_in = [&](int k) { return k == nb - 1 ? rows_last : G; };
    auto row_of = [&](int i) { return (first + (int64_t)(i / G) * stride) * G + i % G; };   // row i of this team
    const bool feeder = half == 0 && lane == 0 && !(prm.test_flags & TRAIN_TEST_NO_FETCH);
    auto fetch_block = [&](int k) {
        ring_fetch(ring + (k % SLOTS) * kSlotVecs, base + (first + (int64_t)k * stride) * G * d,
                   (uint32_t)rows_in(k) * row_bytes, &bar[k % SLOTS]);
    };
    const uint32_t limit = prm.spin_limit;
    if (half == 0 && lane == 0) {
        team_fail[team] = 0;
        for (int s = 0; s < SLOTS; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(ring_addr(&bar[s])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int k = 0; feeder && k < SLOTS && k < nb; ++k) fetch_block(k);
    }
    team_sync<WPR>(team);

    // Labels: lane l holds the label of row (32 b + l) of this team, the batch after it is on its
    // way - a label fetched next to its row would cost a full trip to memory per group of rows.
    auto label_batch = [&](int i0) { return i0 + lane < n ? (float)prm.labels[row_of(i0 + lane)] : 0.f; };
    float y_batch = label_batch(0), y_batch_next = label_batch(32);
    bool ok = true;
    int fail_at = 0;                          // first row of the group whose wait ran out

    // rows [i, i + RR) of this team, RR <= R
    auto group = [&](auto rr_tag, int i) {
        constexpr int RR = decltype(rr_tag)::value;
        int s[RR];                             // where row i + r starts in the ring, in vectors
        int blk[RR];
        float y[RR];
#pragma unroll
        for (int r = 0; r < RR; ++r) {
            blk[r] = (i + r) / G;
            s[r] = (blk[r] % SLOTS) * kSlotVecs + ((i + r) % G) * (G > 1 ? nv : 0);
            const int idx = i + r;
            if ((idx & 31) == 0 && idx > 0) {
                y_batch = y_batch_next;
                y_batch_next = label_batch(idx + 32);
            }
            y[r] = __shfl_sync(0xffffffffu, y_batch, idx & 31);
        }
#pragma unroll
        for (int r = 0; r < RR; ++r)
            if (G == 1 || r == 0) ok = ok && ring_wait(&bar[blk[r] % SLOTS], (uint32_t)(blk[r] / SLOTS) & 1u, limit);
        if (WPR > 1) {
            // a team leaves together: the barriers below need both of its warps
            if (lane == 0 && !ok) team_fail[team] = 1;
        }
        if (WPR == 1 && !ok) {
            fail_at = i;
            return;
        }
        uint64_t dot[RR][2];
#pragma unroll
        for (int r = 0; r < RR; ++r) dot[r][0] = dot[r][1] = pack2(0.f, 0.f);
        if (ok) {
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const int vi = v0 + j * 32;
#pragma unroll
                for (int r = 0; r < RR; ++r) {
                    const uint4 x = vi < nv ? ring[s[r] + vi] : make_uint4(0u, 0u, 0u, 0u);
                    float f[N];
                    Vec<T>::unpack(x, f);
#pragma unroll
                    for (int e = 0; e < N; e += 2)
                        dot[r][j & 1] = fma2(pack2(f[e], f[e + 1]), w2[(j * N + e) / 2], dot[r][j & 1]);
                }
            }
        }
        float zs[RR];
#pragma unroll
        for (int r = 0; r < RR; ++r) {
            float a0, a1, b0, b1;
            unpack2(dot[r][0], a0, a1);
            unpack2(dot[r][1], b0, b1);
            zs[r] = warp_sum((a0 + a1) + (b0 + b1));
        }
        if (WPR > 1) {
            if (lane == 0 && ok) {
#pragma unroll
                for (int r = 0; r < RR; ++r) halves[team][r][half] = zs[r];
            }
            team_sync<WPR>(team);
#pragma unroll
            for (int r = 0; r < RR; ++r) zs[r] = halves[team][r][0] + halves[team][r][1];
            if (team_fail[team] != 0) ok = false;
            if (!ok) {
                fail_at = i;
                return;
            }
        }
        uint64_t res2[RR];
#pragma unroll
        for (int r = 0; r < RR; ++r) {
            const float z = zs[r] + bias;
            const float res = 1.f / (1.f + expf(-z)) - y[r];
            res2[r] = pack2(res, res);
            // The bias-gradient and loss terms of a row are one lane's business: lane (row count
            // mod 32) keeps z and y, and every 32 rows each lane works off the row it kept.
            if (lane == (kept & 31)) {
                z_keep = z;
                y_keep = y[r];
                r_keep = res;
            }
            if ((++kept & 31) == 0) {
                acc_b += (double)r_keep;
                acc_loss += (double)(fmaxf(z_keep, 0.f) + log1pf(expf(-fabsf(z_keep))) - y_keep * z_keep);
            }
        }
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int vi = v0 + j * 32;
#pragma unroll
            for (int r = 0; r < RR; ++r) {
                const uint4 x = vi < nv ? ring[s[r] + vi] : make_uint4(0u, 0u, 0u, 0u);
                float f[N];
                Vec<T>::unpack(x, f);
#pragma unroll
                for (int e = 0; e < N; e += 2)
                    acc[(j * N + e) / 2] = fma2(res2[r], pack2(f[e], f[e + 1]), acc[(j * N + e) / 2]);
            }
        }
        team_sync<WPR>(team);                  // the whole team is done with the slots: refill them
        if (feeder) {
#pragma unroll
            for (int r = 0; r < RR; ++r) {     // a block whose last row was just used makes room for block + SLOTS
                if ((i + r) % G == rows_in(blk[r]) - 1 && blk[r] + SLOTS < nb) fetch_block(blk[r] + SLOTS);
            }
        }
    };
    int i = 0;
    for (; ok && i + R <= n; i += R) group(std::integral_constant<int, R>{}, i);
    for (; ok && i < n; ++i) group(std::integral_constant<int, 1>{}, i);
    if (!ok) {
        // A wait ran out: report it, then give the copies still on their way the same bounded
        // time to land before the CTA's shared memory goes away: the blocks from fail_at's on.
        if (lane == 0) raise_status(prm.status, SPR_ERR_TIMEOUT);
        for (int k = fail_at / G; feeder_team_has_copies(prm) && k < nb && k < fail_at / G + SLOTS; ++k)
            ring_wait(&bar[k % SLOTS], (uint32_t)(k / SLOTS) & 1u, limit);
    }

    if (lane < (kept & 31)) {      // rows kept since the last full round of 32
        acc_b += (double)r_keep;
        acc_loss += (double)(fmaxf(z_keep, 0.f) + log1pf(expf(-fabsf(z_keep))) - y_keep * z_keep);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {   // lanes in a fixed (butterfly) order
        acc_b += __shfl_xor_sync(0xffffffffu, acc_b, o);
        acc_loss += __shfl_xor_sync(0xffffffffu, acc_loss, o);
    }
    __syncthreads();
    for (int t = 0; t < kTeams; ++t) {     // fixed order: team 0 stores, the others add
        if (team == t) {
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const int vi = v0 + j * 32;
                if (vi < nv) {
#pragma unroll
                    for (int e = 0; e < N; e += 2) {
                        float lo, hi;
                        unpack2(acc[(j * N + e) / 2], lo, hi);
                        float *dst = red + vi * N + e;
                        dst[0] = t == 0 ? lo : dst[0] + lo;
                        dst[1] = t == 0 ? hi : dst[1] + hi;
                    }
                }
            }
            if (half == 0 && lane == 0) {
                red[d] = t == 0 ? (float)acc_b : red[d] + (float)acc_b;
                red[d + 1] = t == 0 ? (float)acc_loss : red[d + 1] + (float)acc_loss;
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
    if (*reinterpret_cast<volatile int *>(prm.status) == SPR_ERR_TIMEOUT) {
        // the gradient pass gave up: no step is taken, the loss reads NaN
        if (j == d + 1 && prm.loss) *prm.loss = __int_as_float(0x7fc00000);
        return;
    }
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

template <typename T, int VPL, int WPR, int R, int SLOTS, int G = 1>
cudaError_t launch_grad_ring(const TrainParams &tp, cudaStream_t st)
{
    TrainParams p = tp;
    constexpr int kTeams = kWarps / WPR;
    const size_t smem = (size_t)kTeams * SLOTS * VPL * WPR * 32 * G * 16 + sizeof(float) * ((size_t)tp.d + 2);
    auto kernel = train_grad_ring_kernel<T, VPL, WPR, R, SLOTS, G>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    int per_sm = 0, dev = 0, sms = 0;
    if (e != cudaSuccess ||
        (e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, smem)) != cudaSuccess ||
        (e = cudaGetDevice(&dev)) != cudaSuccess ||
        (e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return e;
    if (per_sm < 1) return cudaErrorInvalidConfiguration;
    // one full wave: as many CTAs as are resident at once, so that all of them finish together
    const int64_t blocks = (tp.N + G - 1) / G;
    p.ctas = (int)max((int64_t)1, min((int64_t)min(kTrainMaxCtas, per_sm * sms), (blocks + kTeams - 1) / kTeams));
    kernel<<<p.ctas, kThreads, smem, st>>>(p);
    train_adam_kernel<<<(tp.d + 2 + 255) / 256, 256, 0, st>>>(p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_grad_any(const TrainParams &tp, cudaStream_t st)
{
    const int vpl = (tp.d / Vec<T>::N + 31) / 32;
    // rows per group and ring slots: about 190 KB of ring per SM (two CTAs share it up to 4 vectors per lane)
    if (vpl <= 1) return launch_grad_ring<T, 1, 1, 4, 3, 8>(tp, st);     // eight rows (4 KB) per copy
    if (vpl <= 2) return launch_grad_ring<T, 2, 1, 4, 3, 4>(tp, st);     // four rows per copy
    if (vpl <= 3) return launch_grad_ring<T, 3, 1, 4, 8>(tp, st);
    if (vpl <= 4) return launch_grad_ring<T, 4, 1, 3, 6>(tp, st);
    if (vpl <= 6) return launch_grad_ring<T, 6, 1, 3, 8>(tp, st);
    if (vpl <= 8) return launch_grad_ring<T, 8, 1, 2, 6>(tp, st);
    if (vpl <= 12) return launch_grad_ring<T, 6, 2, 3, 8>(tp, st);
    return launch_grad_ring<T, 8, 2, 2, 6>(tp, st);
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

static int train_step(const void *hidden, const uint8_t *labels, int64_t N, int d, int dt, float *theta,
                      float *adam_m, float *adam_v, int t, float lr, float beta1, float beta2, float eps,
                      float *loss, void *ws, size_t ws_bytes, void *cuda_stream, int flags, unsigned spin_limit)
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
    tp.status = at<int>(ws, 0);
    tp.spin_limit = spin_limit ? spin_limit : kRingSpin;
    tp.test_flags = flags;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    return finish(dt == SPR_F32 ? launch_grad_any<float>(tp, st) : launch_grad_any<__nv_bfloat16>(tp, st));
}

int verifier_train_step(const void *hidden, const uint8_t *labels, int64_t N, int d, int dt, float *theta,
                        float *adam_m, float *adam_v, int t, float lr, float beta1, float beta2, float eps,
                        float *loss, void *ws, size_t ws_bytes, void *cuda_stream)
{
    return train_step(hidden, labels, N, d, dt, theta, adam_m, adam_v, t, lr, beta1, beta2, eps, loss, ws, ws_bytes,
                      cuda_stream, 0, 0u);
}

int spr_test_verifier_train_step(const void *hidden, const uint8_t *labels, int64_t N, int d, int dt, float *theta,
                                 float *adam_m, float *adam_v, int t, float lr, float beta1, float beta2, float eps,
                                 float *loss, void *ws, size_t ws_bytes, void *cuda_stream, int flags,
                                 unsigned spin_limit)
{
    if (flags & ~TRAIN_TEST_NO_FETCH) return SPR_ERR_INVALID_ARG;
    return train_step(hidden, labels, N, d, dt, theta, adam_m, adam_v, t, lr, beta1, beta2, eps, loss, ws, ws_bytes,
                      cuda_stream, flags, spin_limit);
}

}  // extern "C"
