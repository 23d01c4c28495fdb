// Tensor-core verifier for bf16 MLPs on sm_100a.
//
//   A = relu(H W1^T + b1)   -> tcgen05.mma (bf16 x bf16 -> fp32 in TMEM), operands staged in
//                              shared memory by TMA with the 128-byte swizzle
//   z = A W2                -> fused epilogue: each epilogue thread owns one token (one TMEM
//                              lane), reads its accumulator row with tcgen05.ld and folds
//                              bias, ReLU and the W2 dot product in registers; A never
//                              reaches HBM
// One CTA computes a BM-token x BN-hidden-unit tile (BM, BN in {64, 128}) and writes one
// partial z per token.
// The CTA that completes a token tile adds its partials in slice order, applies the sigmoid
// and the threshold and scans the sequences inside the tile (same tail as the SIMT kernel).
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue (warp w reads TMEM lanes 32*(w%4) .. +31).
// Every wait on an mbarrier is bounded: when a wait runs out the kernel records
// SPR_ERR_TIMEOUT in the status word, all roles leave their loops, TMEM is released and
// the CTA exits.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "launch.h"
#include "verifier_common.cuh"

namespace spr {

namespace {

constexpr int kAtomK = 64;      // bf16 elements of one 128-byte swizzle row (one TMA box)
constexpr int kAtoms = 2;       // swizzle atoms per pipeline stage
constexpr int kBK = kAtomK * kAtoms;   // bf16 elements per k-block (pipeline stage)
constexpr int kUmmaK = 16;      // K of one tcgen05.mma for 16-bit operands
constexpr int kTcThreads = 192;
constexpr int kMaxStages = 12;
constexpr uint32_t kSpinLimit = 1u << 24;   // polls of mbarrier.try_wait before giving up

template <int BM, int BN>
struct TileCfg {
    static constexpr int kBytesA = BM * kBK * 2;
    static constexpr int kBytesB = BN * kBK * 2;
    static constexpr int kStageBytes = kBytesA + kBytesB;
    // The k-loop is bound by the time a stage takes to come round again (MMA done -> commit ->
    // producer -> TMA -> full, about 2 us), so throughput is stages / that time: use all the
    // shared memory there is (one CTA per SM either way).
    static constexpr int kStages = (220 * 1024) / kStageBytes < kMaxStages ? (220 * 1024) / kStageBytes : kMaxStages;
    static constexpr int kTmemCols = BN < 32 ? 32 : BN;
    // stages, slack to align them to 1024 bytes, control block
    static constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 1024 + 3072;
};

struct Control {                 // lives behind the stages in dynamic shared memory
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full;
    uint32_t tmem_base;
    int abort;
    int last;
    float b1[128];
    float w2[128];
};
static_assert(sizeof(Control) <= 3072, "control block must fit its reservation");

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
// Bounded wait.  Returns false (and flags the CTA) if the phase never completes or another
// role already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Control *ctl, int *status)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int *>(&ctl->abort)) return false;
    }
    *reinterpret_cast<volatile int *>(&ctl->abort) = 1;
    raise_status(status, SPR_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
        : "memory");
}

// Shared-memory matrix descriptor: K-major tile whose rows are one 128-byte swizzle span;
// 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3ffffu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                          // leading-dimension offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride between 8-row groups
    d |= (uint64_t)1 << 46;                          // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                          // 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = BM, N = BN.
template <int BM, int BN>
__device__ __forceinline__ constexpr uint32_t umma_instr_desc()
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

template <int BM, int BN>
__global__ void __launch_bounds__(kTcThreads, 1)
verifier_tcgen05_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                        const VerifyParams prm)
{
    using Cfg = TileCfg<BM, BN>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *stages = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Control *ctl = reinterpret_cast<Control *>(stages + (size_t)Cfg::kStages * Cfg::kStageBytes);

    pdl_trigger();   // a replacement draw launched behind this grid may be scheduled now
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int M = prm.B * prm.K;
    const int n0 = blockIdx.x * BN;      // first hidden unit of this slice
    const int m0 = blockIdx.y * BM;      // first token of this tile
    const int num_kb = (prm.d + kBK - 1) / kBK;

    if (tid == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->tmem_full, 1);
        ctl->abort = 0;
        ctl->last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int j = tid; j < BN; j += kTcThreads) {
        const int n = n0 + j;
        ctl->b1[j] = n < prm.h ? prm.b1[n] : 0.f;
        ctl->w2[j] = n < prm.h ? __bfloat162float(static_cast<const __nv_bfloat16 *>(prm.W2)[n]) : 0.f;
    }
    if (warp == 1) {   // TMEM: BN fp32 accumulator columns x 128 lanes
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                     "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = ctl->tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % Cfg::kStages;
                const uint32_t round = (uint32_t)(kb / Cfg::kStages);
                if (!mbar_wait(&ctl->empty[s], (round & 1u) ^ 1u, ctl, prm.status)) break;
                unsigned char *a_dst = stages + (size_t)s * Cfg::kStageBytes;
                unsigned char *b_dst = a_dst + Cfg::kBytesA;
                mbar_expect_tx(&ctl->full[s], (uint32_t)Cfg::kStageBytes);
#pragma unroll
                for (int a = 0; a < kAtoms; ++a) {   // one box per 64-wide swizzle atom
                    tma_load_2d(a_dst + a * (Cfg::kBytesA / kAtoms), &map_h, kb * kBK + a * kAtomK, m0, &ctl->full[s]);
                    tma_load_2d(b_dst + a * (Cfg::kBytesB / kAtoms), &map_w, kb * kBK + a * kAtomK, n0, &ctl->full[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_instr_desc<BM, BN>();
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % Cfg::kStages;
                const uint32_t round = (uint32_t)(kb / Cfg::kStages);
                ok = mbar_wait(&ctl->full[s], round & 1u, ctl, prm.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(stages + (size_t)s * Cfg::kStageBytes);
                const uint32_t b_addr = a_addr + Cfg::kBytesA;
#pragma unroll
                for (int a = 0; a < kAtoms; ++a) {
                    const uint64_t da = umma_smem_desc(a_addr + a * (Cfg::kBytesA / kAtoms));
                    const uint64_t db = umma_smem_desc(b_addr + a * (Cfg::kBytesB / kAtoms));
#pragma unroll
                    for (int k = 0; k < kAtomK / kUmmaK; ++k) {
                        // next 16 elements along K: 32 bytes further inside the swizzle row
                        const uint64_t adv = (uint64_t)((k * kUmmaK * 2) >> 4);
                        umma_bf16(tmem_acc, da + adv, db + adv, idesc, (kb | a | k) != 0 ? 1u : 0u);
                    }
                }
                umma_commit(&ctl->empty[s]);       // stage is free once these MMAs have read it
            }
            if (ok) umma_commit(&ctl->tmem_full);  // accumulator complete
        }
    } else {
        // ---------------- epilogue: thread = token, TMEM lane = 32*(warp%4) + lane
        // BM = 128: accumulator row r lives in TMEM lane r.  BM = 64: the 64 rows use lanes
        // 0-15 of each 32-lane quarter (row r in lane 32*(r/16) + r%16).
        const int quarter = warp & 3;
        const bool has_row = BM == 128 || lane < 16;
        const int row = m0 + (BM == 128 ? quarter * 32 + lane : quarter * 16 + lane);
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&ctl->tmem_full, 0, ctl, prm.status));
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            float z = 0.f;
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 16) {
                float v[16];
                tmem_ld16(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) z = fmaf(ctl->w2[c0 + j], fmaxf(v[j] + ctl->b1[c0 + j], 0.f), z);
            }
            if (has_row && row < M) prm.part_z[(int64_t)blockIdx.x * M + row] = z;
        }
    }

    // ---------------- teardown: release TMEM, then the ticket for the final reduction
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
    }
    // Tickets: the CTA that completes a token tile (all slices written) turns its 128 partial
    // sums into scores, accept bits and the scan of the sequences inside the tile; sequences
    // cut by a tile boundary wait for the CTA that completes the last tile.
    if (tid == 0) {
        __threadfence();
        ctl->last = take_ticket(&prm.counter[1 + blockIdx.y], (int)gridDim.x);
    }
    __syncthreads();
    if (!ctl->last) return;
    __threadfence();
    finalise_tile(prm, m0, min(m0 + BM, M));
    if (BM % prm.K == 0) return;   // no sequence straddles a tile boundary
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        ctl->last = take_ticket(&prm.counter[0], (int)gridDim.y);
    }
    __syncthreads();
    if (!ctl->last) return;
    __threadfence();
    finalise_straddlers(prm, BM);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [rows, cols] bf16 row-major tensor, boxes of box_rows x 64 elements, 128-byte swizzle,
// out-of-range elements read as zero.
bool make_map(CUtensorMap *map, const void *base, int rows, int cols, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kAtomK, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BM, int BN>
int launch_tile(const CUtensorMap &mh, const CUtensorMap &mw, VerifyParams vp, int tiles_m, cudaStream_t st)
{
    using Cfg = TileCfg<BM, BN>;
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(verifier_tcgen05_kernel<BM, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)Cfg::kSmemBytes);
        if (e != cudaSuccess) return (int)e;
        attr_set[dev] = true;
    }
    vp.slices = (vp.h + BN - 1) / BN;
    dim3 grid((unsigned)vp.slices, (unsigned)tiles_m);
    verifier_tcgen05_kernel<BM, BN><<<grid, kTcThreads, Cfg::kSmemBytes, st>>>(mh, mw, vp);
    return (int)cudaGetLastError();
}

}  // namespace

int launch_verifier_tensor(const VerifyParams &vp, int dt, int min_tokens, cudaStream_t st)
{
    const int64_t M = (int64_t)vp.B * vp.K;
    if (dt != SPR_BF16 || vp.h <= 0 || vp.d % 8 != 0 || M < min_tokens) return -1;
    if ((reinterpret_cast<uintptr_t>(vp.hidden) & 15) || (reinterpret_cast<uintptr_t>(vp.W1) & 15)) return -1;
    // Measured on B200: a CTA's k-loop costs about the same per tcgen05.mma (140-250 cycles)
    // whatever the tile shape up to 128 x 128, so time is set by the d/16 instructions each CTA
    // issues in a row and by how many CTAs run at once.  Take the largest of the four tile
    // shapes that still gives the GPU about a wave of CTAs; 64 x 64 if none does, 128 x 128
    // once even that exceeds a wave.
    auto ctas = [&](int m, int n) { return ((M + m - 1) / m) * (int64_t)((vp.h + n - 1) / n); };
    static const int kShapes[4][2] = {{128, 128}, {64, 128}, {128, 64}, {64, 64}};
    int bm = 64, bn = 64;
    for (const auto &sh : kShapes) {
        if (ctas(sh[0], sh[1]) >= 96) {
            bm = sh[0];
            bn = sh[1];
            break;
        }
    }
    // tuning aids: SPR_VERIFIER_BM=64|128, SPR_VERIFIER_BN=64|128
    if (const char *env = getenv("SPR_VERIFIER_BM")) {
        const int v = atoi(env);
        if (v == 64 || v == 128) bm = v;
    }
    if (const char *env = getenv("SPR_VERIFIER_BN")) {
        const int v = atoi(env);
        if (v == 64 || v == 128) bn = v;
    }
    const int64_t tiles64 = (M + bm - 1) / bm;
    if (tiles64 > 65535) return -1;
    const int tiles_m = (int)tiles64;
    CUtensorMap mh, mw;
    if (!make_map(&mh, vp.hidden, (int)M, vp.d, bm)) return -1;
    if (!make_map(&mw, vp.W1, vp.h, vp.d, bn)) return -1;
#define SPR_TILE(BM_, BN_) \
    if (bm == BM_ && bn == BN_) return launch_tile<BM_, BN_>(mh, mw, vp, tiles_m, st)
    SPR_TILE(64, 64);
    SPR_TILE(64, 128);
    SPR_TILE(128, 64);
    SPR_TILE(128, 128);
#undef SPR_TILE
    return -1;
}

}  // namespace spr
