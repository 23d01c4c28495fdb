// Tensor-core verifier for bf16 MLPs on sm_100a.
//
//   A = relu(H W1^T + b1)   -> tcgen05.mma (bf16 x bf16 -> fp32 in TMEM), operands staged in
//                              shared memory by TMA with the 128-byte swizzle
//   z = A W2                -> fused epilogue: each epilogue thread owns one token (one TMEM
//                              lane) and folds bias, ReLU and the W2 dot product in registers;
//                              A never reaches HBM
//
// Grid (S, slices, tiles): a CTA computes a BM-token x BN-hidden-unit tile over one of S equal
// ranges of d.  The S CTAs of a tile form a cluster (along x) and add their accumulators
// through distributed shared memory BEFORE the ReLU: CTA r receives, from every CTA of the
// tile, the BN/S accumulator columns it owns (asynchronous remote stores that count bytes on
// the receiver's mbarrier), adds them in CTA order and applies bias, ReLU and W2 to those
// columns.  Small batches thereby spread the sweep over W1 (the only real traffic they
// have) over many SMs.  The per-token partial z of the S CTAs go, the same way, to the CTA
// with split 0, which adds them in order.
// Where S x slices <= 8 the cluster also spans the hidden-unit slices of the tile (along y):
// every CTA sends its partial z to the cluster's first CTA, which adds them in rank order,
// applies sigmoid and threshold and scans the sequences inside the tile out of shared memory
// - no trip through global memory.  Otherwise one partial z per slice goes to the workspace
// and the CTA that takes the tile's last ticket finishes it.
// Cluster barriers are used only as handshakes whose two halves lie far apart: "started"
// (arrive at the start, wait before the first remote store) and "done with my peers" (arrive
// when nothing more is sent or expected, wait before exit), so nobody stands at one.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue (warp w reads TMEM lanes 32*(w%4) .. +31).
// Every wait on an mbarrier is bounded: when a wait runs out the kernel records
// SPR_ERR_TIMEOUT in the status word, all roles leave their loops, the CTA still goes through
// every cluster barrier (so its peers never wait for it), hands on NaN instead of its partial
// results (the tile's tokens then report score -1, accept 0, first_reject -1), waits - again
// bounded - for what it has in flight, releases TMEM and exits.
#include <cuda.h>

#include <atomic>

#include "common.cuh"
#include "launch.h"
#include "verifier_common.cuh"

namespace spr {

// Development aid (compiled only with -DSPR_VERIFIER_STAMPS): SM-clock stamps of the phases of
// the first CTAs of a launch, read back with spr_debug_verifier_stamps().
#ifdef SPR_VERIFIER_STAMPS
__device__ long long g_stamps[512][64];
#define SPR_STAMP(i)                                                                                     \
    do {                                                                                                 \
        const unsigned cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);            \
        if (cta_ < 512) g_stamps[cta_][i] = clock64();                                                   \
    } while (0)
#else
#define SPR_STAMP(i)
#endif

namespace {

constexpr int kAtomK = 64;      // bf16 elements of one 128-byte swizzle row: one TMA box, one "atom" of d
constexpr int kUmmaK = 16;      // K of one tcgen05.mma for 16-bit operands
constexpr int kTcThreads = 192;
constexpr int kMaxStages = 4;
constexpr int kMaxClusterCtas = 8;          // portable cluster size
constexpr uint32_t kSpinLimit = 1u << 24;   // polls of mbarrier.try_wait before giving up

struct Control {                 // lives behind the ring in dynamic shared memory
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full;
    uint64_t drain;
    uint64_t xchg;               // counts the bytes of accumulator columns received from the tile's CTAs
    uint64_t zgather;            // counts the bytes of partial z received (receiving CTA only)
    uint32_t tmem_base;
    int abort;
    int last;
    int consumed;                // stages whose operands the MMA issuer saw arrive
    float b1[128];
    float w2[128];
    float zbuf[kMaxClusterCtas][128];   // first CTA of a cluster: partial z of every CTA, per token
    unsigned char codes[128];           // accept codes of the tile, for the scan
};

template <int BM, int BN>
struct TileCfg {
    static constexpr int kBytesA = BM * kAtomK * 2;     // one atom of the hidden-state tile
    static constexpr int kBytesB = BN * kAtomK * 2;     // one atom of the W1 tile
    // A pipeline stage costs the two threads that run it (producer, MMA issuer) about 0.25 us
    // of barrier and issue latency whatever it holds, so a stage holds several atoms: 48-64 KB.
    static constexpr int kAtoms = (BM + BN == 128) ? 4 : 2;
    static constexpr int kStageBytes = kAtoms * (kBytesA + kBytesB);
    static constexpr int kStages = (200 * 1024) / kStageBytes;
    static_assert(kStages >= 2 && kStages <= kMaxStages, "stage count");
    static constexpr int kRingBytes = kStages * kStageBytes;
    // after the k-loop the ring is reused for the accumulator columns received from the
    // other CTAs of the tile: [S][BN/S/4][BM] float4
    static_assert(BM * BN * 4 <= kRingBytes, "ring must hold the exchanged accumulator columns");
    static constexpr int kTmemCols = BN < 32 ? 32 : BN;
    // ring, slack to align it to 1024 bytes, control block
    static constexpr size_t kSmemBytes = (size_t)kRingBytes + 1024 + ((sizeof(Control) + 255) / 256) * 256;
};

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
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Control *ctl, int *status, uint32_t limit)
{
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u && *reinterpret_cast<volatile int *>(&ctl->abort)) return false;
    }
    *reinterpret_cast<volatile int *>(&ctl->abort) = 1;
    raise_status(status, SPR_ERR_TIMEOUT);
    return false;
}
// the same without side effects: used on the way out, when the CTA has already given up
__device__ __forceinline__ void mbar_wait_quiet(uint64_t *bar, uint32_t parity, uint32_t limit)
{
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
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
// 32 accumulator columns of this thread's TMEM lane; the registers are valid after tmem_ld_wait()
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- thread-block cluster: barrier over all threads of all CTAs, shared memory of a peer CTA
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.aligned;" ::: "memory"); }   // release
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }       // acquire
__device__ __forceinline__ void cluster_sync()
{
    cluster_arrive();
    cluster_wait();
}
// address, in the cluster's shared window, of this CTA's shared address `saddr` in CTA `rank`
__device__ __forceinline__ uint32_t peer_smem(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
// Asynchronous stores into a peer's shared memory; each adds its size to the transaction count
// of the mbarrier `bar` (an address in the same peer), whose waiters then see the data.
__device__ __forceinline__ void st_async_b32(uint32_t addr, uint32_t v, uint32_t bar)
{
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(addr), "r"(v), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void st_async_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t bar)
{
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
                 "r"(a), "r"(b), "r"(c), "r"(d), "r"(bar)
                 : "memory");
}

// One epilogue thread (= accumulator row r_in): its BN accumulator columns, four at a time, to
// the CTAs that own them.  Receiver layout: recv4[source split][group of 4 owned columns][row].
template <int BM, int BN, int S>
__device__ __forceinline__ void send_columns(uint32_t lane_base, const float4 *recv4, uint64_t *xchg, int split,
                                             uint32_t row_rank0, int r_in, bool live_row)
{
    constexpr int kColsPer = BN / S, kGroups = kColsPer / 4;
    static_assert(kColsPer >= 8 && kColsPer % 4 == 0, "columns per owner");
    uint32_t base[S], bar[S];    // where this CTA's block of rows starts in every owner's buffer; its mbarrier
#pragma unroll
    for (int o = 0; o < S; ++o) {
        base[o] = peer_smem(smem_u32(recv4 + ((size_t)split * kGroups * BM + r_in)), row_rank0 + (uint32_t)o);
        bar[o] = peer_smem(smem_u32(xchg), row_rank0 + (uint32_t)o);
    }
#pragma unroll
    for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(lane_base + (uint32_t)c0, r);
        tmem_ld_wait();
        if (live_row) {
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const int c = c0 + 4 * g;
                const int owner = c / kColsPer, cg = (c % kColsPer) / 4;
                st_async_v4(base[owner] + (uint32_t)(cg * BM * 16), r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3],
                            bar[owner]);
            }
        }
    }
}

// the same thread, after the exchange: sum over the source CTAs (in order), bias, ReLU and W2
// for the columns this CTA owns
template <int BM, int BN, int S>
__device__ __forceinline__ float owned_columns_z(const float4 *recv4, const Control *ctl, int split, int r_in)
{
    constexpr int kColsPer = BN / S, kGroups = kColsPer / 4;
    float z = 0.f;
#pragma unroll
    for (int cg = 0; cg < kGroups; ++cg) {
        float4 a = recv4[(size_t)cg * BM + r_in];
#pragma unroll
        for (int s = 1; s < S; ++s) {
            const float4 b = recv4[((size_t)s * kGroups + cg) * BM + r_in];
            a.x += b.x;
            a.y += b.y;
            a.z += b.z;
            a.w += b.w;
        }
        const int c = split * kColsPer + 4 * cg;
        z = fmaf(ctl->w2[c], fmaxf(a.x + ctl->b1[c], 0.f), z);
        z = fmaf(ctl->w2[c + 1], fmaxf(a.y + ctl->b1[c + 1], 0.f), z);
        z = fmaf(ctl->w2[c + 2], fmaxf(a.z + ctl->b1[c + 2], 0.f), z);
        z = fmaf(ctl->w2[c + 3], fmaxf(a.w + ctl->b1[c + 3], 0.f), z);
    }
    return z;
}

// K = 1 (one token per sequence, so a token can be finished on its own): a slice's partial
// logit is added to the token's 64-bit word with ONE atomic - bits 0-7 count the slices that
// have arrived, bits 8-15 those that arrived poisoned, bits 16-63 hold the sum in fixed point
// (2^-24; a partial is clamped to +-32768, far beyond where the sigmoid saturates).  Integer
// addition commutes, so the sum does not depend on who comes first; the thread whose addition
// completes the count holds the whole sum in its register, finishes the token and sets the
// word back to zero.  No fence, no ticket, no second trip to read partial sums.
__device__ __forceinline__ void add_partial_and_finish(const VerifyParams &prm, float z, int m, int slices)
{
    const bool bad = !(z == z);
    const float zc = fminf(fmaxf(bad ? 0.f : z, -32768.f), 32768.f);
    const long long fix = __double2ll_rn((double)zc * 16777216.0);
    const unsigned long long add = ((unsigned long long)fix << 16) + (bad ? 0x101ull : 0x1ull);
    const unsigned long long now = atomicAdd(&prm.zacc[m], add) + add;
    if ((int)(now & 0xffull) != slices) return;
    *reinterpret_cast<volatile unsigned long long *>(&prm.zacc[m]) = 0ull;
    const bool poisoned = ((now >> 8) & 0xffull) != 0ull;
    const double zsum = (double)((long long)now >> 16) * (1.0 / 16777216.0) + (double)prm.b2[0];
    const int a = classify_token(prm, poisoned ? poisoned_z() : (float)zsum, m);
    if (prm.first_reject) prm.first_reject[m] = a == ACC_INVALID ? -1 : (a == ACC_ACCEPT ? 1 : 0);
}

template <int BM, int BN>
__global__ void __launch_bounds__(kTcThreads, 1)
verifier_tcgen05_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                        const VerifyParams prm)
{
    using Cfg = TileCfg<BM, BN>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *ring = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Control *ctl = reinterpret_cast<Control *>(ring + Cfg::kRingBytes);

    pdl_trigger();   // a replacement draw launched behind this grid may be scheduled now
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) SPR_STAMP(0);
    const int M = prm.B * prm.K;
    const int S = (int)gridDim.x, split = (int)blockIdx.x;   // CTAs sharing this tile along d
    const int n0 = blockIdx.y * BN;      // first hidden unit of this slice
    const int m0 = blockIdx.z * BM;      // first token of this tile
    const int atom0 = split * prm.kb_per;                                          // first atom of d of this CTA
    const int num_atoms = min(prm.kb_per, (prm.d + kAtomK - 1) / kAtomK - atom0);  // >= 1: the host sees to it
    const int num_stages = (num_atoms + Cfg::kAtoms - 1) / Cfg::kAtoms;
    const int cluster_ctas = S * prm.cluster_n;
    const bool clustered = cluster_ctas > 1;
    // rank inside the cluster (x runs fastest) and the rank of the tile's CTA with split 0
    const uint32_t my_rank = (uint32_t)split + (blockIdx.y % (unsigned)prm.cluster_n) * (uint32_t)S;
    const uint32_t row_rank0 = my_rank - (uint32_t)split;
    const uint32_t limit = prm.spin_limit;
    const int ring_stages = prm.ring_stages;     // the last stage's room may be lent to the exchange
    const int live_rows = min(BM, M - m0);       // tokens of this tile
    // which CTA adds up partial z: the cluster's first CTA when the cluster holds the whole
    // tile, else the tile's CTA with split 0 (nobody when d is not split)
    const bool gather_z = clustered;
    const uint32_t z_rank = prm.final_in_cluster ? 0u : row_rank0;
    const int z_sources = prm.final_in_cluster ? cluster_ctas : S;

    if (tid == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->tmem_full, 1);
        mbar_init(&ctl->drain, 1);
        mbar_init(&ctl->xchg, 1);
        mbar_init(&ctl->zgather, 1);
        // what this CTA is going to receive from its peers (and from itself)
        if (S > 1) mbar_expect_tx(&ctl->xchg, (uint32_t)(live_rows * BN * 4));
        if (gather_z && my_rank == z_rank) mbar_expect_tx(&ctl->zgather, (uint32_t)(z_sources * live_rows * 4));
        ctl->abort = 0;
        ctl->last = 0;
        ctl->consumed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0 && lane < 2)   // descriptor fetch off the critical path of the first copy
        asm volatile("prefetch.tensormap [%0];" ::"l"(lane == 0 ? &map_h : &map_w) : "memory");
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
    if (tid == 0) SPR_STAMP(1);
    // A peer's shared memory may be written once that CTA has started and set up its
    // barriers: each thread says so here and checks for everybody's word only where the first
    // remote store is made.  Where the exchange buffer overlays the ring, the peers must be
    // through their k-loops as well: that handshake is made in one piece after the loop.
    const bool early_arrive = clustered && (S == 1 || prm.recv_dedicated);
    if (early_arrive) cluster_arrive();

    int issued = 0;       // producer: stages whose copies are on their way
    bool ok = true;       // epilogue: the accumulator is complete
    if (warp == 0) {
        // ---------------- TMA producer: one lane per box of a stage (even lanes: hidden-state
        // atoms, odd lanes: W1 atoms), so one instruction issues all copies of a stage
        if (lane < 2 * Cfg::kAtoms && !(prm.test_flags & VERIFIER_TEST_NO_LOADS)) {
            const int atom = lane >> 1;
            const bool is_w = lane & 1;
            const CUtensorMap *map = is_w ? &map_w : &map_h;
            const int row0 = is_w ? n0 : m0;
            const uint32_t off = is_w ? (uint32_t)(Cfg::kAtoms * Cfg::kBytesA + atom * Cfg::kBytesB)
                                      : (uint32_t)(atom * Cfg::kBytesA);
            const uint32_t atom_bytes = (uint32_t)prm.a_box_rows * (kAtomK * 2) + (uint32_t)Cfg::kBytesB;
            for (int st = 0; st < num_stages; ++st) {
                const int s = st % ring_stages;
                const uint32_t round = (uint32_t)(st / ring_stages);
                const int n_at = min(Cfg::kAtoms, num_atoms - st * Cfg::kAtoms);
                if (!mbar_wait(&ctl->empty[s], (round & 1u) ^ 1u, ctl, prm.status, limit)) break;
                if (lane == 0) mbar_expect_tx(&ctl->full[s], (uint32_t)n_at * atom_bytes);
                if (atom < n_at)
                    tma_load_2d(smem_u32(ring + (size_t)s * Cfg::kStageBytes) + off, map,
                                (atom0 + st * Cfg::kAtoms + atom) * kAtomK, row0, &ctl->full[s]);
                issued = st + 1;
                if (st == 0) SPR_STAMP(2);
                if (st < 24 && lane == 0) SPR_STAMP(40 + st);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_instr_desc<BM, BN>();
            bool fed = true;
            int st = 0;
            for (; st < num_stages; ++st) {
                const int s = st % ring_stages;
                const uint32_t round = (uint32_t)(st / ring_stages);
                const int n_at = min(Cfg::kAtoms, num_atoms - st * Cfg::kAtoms);
                fed = mbar_wait(&ctl->full[s], round & 1u, ctl, prm.status, limit);
                if (!fed) break;
                if (st == 0) SPR_STAMP(3);
                if (st < 24) SPR_STAMP(16 + st);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(ring + (size_t)s * Cfg::kStageBytes);
                const uint32_t b_addr = a_addr + Cfg::kAtoms * Cfg::kBytesA;
#pragma unroll
                for (int a = 0; a < Cfg::kAtoms; ++a) {
                    if (a < n_at) {
                        const uint64_t da = umma_smem_desc(a_addr + a * Cfg::kBytesA);
                        const uint64_t db = umma_smem_desc(b_addr + a * Cfg::kBytesB);
#pragma unroll
                        for (int k = 0; k < kAtomK / kUmmaK; ++k) {
                            // next 16 elements along K: 32 bytes further inside the swizzle row
                            const uint64_t adv = (uint64_t)((k * kUmmaK * 2) >> 4);
                            umma_bf16(tmem_acc, da + adv, db + adv, idesc, (st | a | k) != 0 ? 1u : 0u);
                        }
                    }
                }
                umma_commit(&ctl->empty[s]);       // stage is free once these MMAs have read it
            }
            ctl->consumed = st;
            SPR_STAMP(4);
            if (fed) {
                umma_commit(&ctl->tmem_full);      // accumulator complete
            } else {
                umma_commit(&ctl->drain);          // what was issued is waited for on the way out
            }
        }
    } else {
        // ---------------- epilogue threads: layer-2 constants of this slice into shared memory
        // (read again only after a barrier below), then wait for the accumulator
        for (int j = tid - 64; j < BN; j += kTcThreads - 64) {
            const int n = n0 + j;
            ctl->b1[j] = n < prm.h ? prm.b1[n] : 0.f;
            ctl->w2[j] = n < prm.h ? __bfloat162float(static_cast<const __nv_bfloat16 *>(prm.W2)[n]) : 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");   // the four epilogue warps
        ok = mbar_wait(&ctl->tmem_full, 0, ctl, prm.status, limit);
        if (tid == 64) SPR_STAMP(5);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    __syncwarp();

    // thread = token: TMEM lane 32*(warp%4) + lane.  BM = 128: accumulator row r lives in TMEM
    // lane r.  BM = 64: the 64 rows use lanes 0-15 of each 32-lane quarter.
    const int quarter = warp & 3;
    const int r_in = BM == 128 ? quarter * 32 + lane : quarter * 16 + (lane & 15);   // row inside the tile
    const int row = m0 + r_in;
    const bool live_row = warp >= 2 && (BM == 128 || lane < 16) && row < M;
    const uint32_t lane_base = tmem_acc + ((uint32_t)(quarter * 32) << 16);
    const float4 *recv4 = reinterpret_cast<const float4 *>(
        ring + (prm.recv_dedicated ? (size_t)ring_stages * Cfg::kStageBytes : 0));

    if (clustered) {
        if (early_arrive) cluster_wait();
        else cluster_sync();
    }
    if (tid == 64) SPR_STAMP(6);

    if (S > 1 && warp >= 2) {
        // ---------------- accumulator columns to their owners; then wait for the columns owned here
        if (S == 2) send_columns<BM, BN, 2>(lane_base, recv4, &ctl->xchg, split, row_rank0, r_in, live_row);
        if (S == 4) send_columns<BM, BN, 4>(lane_base, recv4, &ctl->xchg, split, row_rank0, r_in, live_row);
        if (S == 8) send_columns<BM, BN, 8>(lane_base, recv4, &ctl->xchg, split, row_rank0, r_in, live_row);
        ok &= mbar_wait(&ctl->xchg, 0, ctl, prm.status, limit);
    }
    if (tid == 64) SPR_STAMP(7);

    // ---------------- bias, ReLU, W2 over the columns this CTA owns
    float z = 0.f;
    if (warp >= 2) {
        if (S == 1) {
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 64) {
                uint32_t v[2][32];
                tmem_ld32(lane_base + (uint32_t)c0, v[0]);
                tmem_ld32(lane_base + (uint32_t)(c0 + 32), v[1]);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 64; ++j)
                    z = fmaf(ctl->w2[c0 + j], fmaxf(__uint_as_float(v[j >> 5][j & 31]) + ctl->b1[c0 + j], 0.f), z);
            }
        } else if (live_row) {
            if (S == 2) z = owned_columns_z<BM, BN, 2>(recv4, ctl, split, r_in);
            if (S == 4) z = owned_columns_z<BM, BN, 4>(recv4, ctl, split, r_in);
            if (S == 8) z = owned_columns_z<BM, BN, 8>(recv4, ctl, split, r_in);
        }
        if (!ok || *reinterpret_cast<volatile int *>(&ctl->abort)) z = poisoned_z();
    }
    if (tid == 64) SPR_STAMP(8);

    // ---------------- partial z to whoever adds them up
    const bool z_receiver = my_rank == z_rank;
    if (gather_z) {
        if (live_row) {
            const int src = prm.final_in_cluster ? (int)my_rank : split;
            st_async_b32(peer_smem(smem_u32(&ctl->zbuf[src][r_in]), z_rank), __float_as_uint(z),
                         peer_smem(smem_u32(&ctl->zgather), z_rank));
        }
        if (z_receiver && warp >= 2) {
            const bool got = mbar_wait(&ctl->zgather, 0, ctl, prm.status, limit);
            if (!prm.final_in_cluster && live_row) {   // one partial per slice leaves the cluster
                float zs = 0.f;
                for (int i = 0; i < z_sources; ++i) zs += ctl->zbuf[i][r_in];
                if (!got) zs = poisoned_z();
                if (prm.atomic_finish) add_partial_and_finish(prm, zs, row, (int)gridDim.y);
                else prm.part_z[(int64_t)blockIdx.y * M + row] = zs;
            } else if (!got && live_row) {
                ctl->zbuf[0][r_in] = poisoned_z();
            }
        }
    } else if (prm.final_in_cluster) {      // a tile with a single CTA
        if (live_row) ctl->zbuf[0][r_in] = z;
    } else if (live_row) {
        if (prm.atomic_finish) add_partial_and_finish(prm, z, row, (int)gridDim.y);
        else prm.part_z[(int64_t)blockIdx.y * M + row] = z;
    }
    __syncwarp();
    // this CTA sends nothing more and expects nothing more: its peers may leave
    if (clustered) cluster_arrive();

    // ---------------- teardown: nothing in flight, release TMEM
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (*reinterpret_cast<volatile int *>(&ctl->abort)) {   // the same for every thread by now
        if (warp == 0) {   // copies issued but never consumed
            int last = issued;     // a lane may be one stage ahead of lane 0
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
            if (lane == 0) {
                for (int st = ctl->consumed; st < last; ++st)
                    mbar_wait_quiet(&ctl->full[st % ring_stages], (uint32_t)(st / ring_stages) & 1u, limit);
            }
        }
        if (warp == 1 && lane == 0 && ctl->consumed < num_stages) mbar_wait_quiet(&ctl->drain, 0, limit);
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
    }
    if (tid == 64) SPR_STAMP(9);

    // ---------------- finish: the receiver of the partial z when the cluster holds the whole
    // tile, else whoever takes the tile's last ticket (one ticket per slice)
    const int m_hi = min(m0 + BM, M);
    bool finisher = false;
    if (prm.final_in_cluster) {
        finisher = z_receiver;
        if (finisher) {
            const float b2 = prm.b2[0];
            for (int t = tid; t < m_hi - m0; t += kTcThreads) {
                float zt = b2;
                for (int i = 0; i < z_sources; ++i) zt += ctl->zbuf[i][t];
                ctl->codes[t] = (unsigned char)classify_token(prm, zt, m0 + t);
            }
            __syncthreads();
            if (prm.first_reject) {
                const int b_lo = (m0 + prm.K - 1) / prm.K, b_hi = m_hi / prm.K;
                for (int b = b_lo + warp; b < b_hi; b += kTcThreads / 32)
                    scan_sequence_smem(prm, b, ctl->codes + (b * prm.K - m0), lane);
            }
        }
    } else if (!prm.atomic_finish && (!gather_z || z_receiver)) {
        if (tid == 0) {
            __threadfence();
            ctl->last = take_ticket(&prm.counter[1 + blockIdx.z], (int)gridDim.y);
        }
        __syncthreads();
        finisher = ctl->last != 0;
        if (finisher) {
            __threadfence();
            finalise_tile(prm, m0, m_hi, ctl->codes);
        }
    }
    if (tid == 64) SPR_STAMP(10);
    // sequences cut by a tile boundary wait for the CTA that completes the last tile
    if (finisher && BM % prm.K != 0 && gridDim.z > 1) {
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            ctl->last = take_ticket(&prm.counter[0], (int)gridDim.z);
        }
        __syncthreads();
        if (ctl->last) {
            __threadfence();
            finalise_straddlers(prm, BM);
        }
    }
    if (clustered) cluster_wait();   // no peer is still sending to this CTA
}

// ---------------------------------------------------------------- CTA pairs (large batches)
// With many tokens the k-loop is bound by how fast one SM takes operands in (about one 128-byte
// row per two clocks).  Two CTAs of a cluster then share one 256-token x 128-hidden-unit tile:
// each stages its own 128 token rows but only HALF of the W1 tile (64 rows), and one thread of
// the even CTA issues tcgen05.mma.cta_group::2, which reads both CTAs' shared memory and writes
// both CTAs' TMEM - a quarter fewer operand bytes per SM and per FLOP.  The copies of both CTAs
// count on the even CTA's "full" barriers; its commits free the stage in both CTAs.  Every
// CTA then runs the same epilogue as above on its own 128 accumulator rows.  The cluster is
// (2, n, 1): the pair along x, and along y all slices of the token tiles when they fit (finish
// out of shared memory, one receiver per token tile), else one slice (tickets).
constexpr int kPairBM = 128, kPairBN = 128;
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;   // clears the bit that tells the two CTAs of a pair apart

struct PairCfg {
    static constexpr int kBytesA = kPairBM * kAtomK * 2;          // 128 token rows of one atom
    static constexpr int kBytesB = (kPairBN / 2) * kAtomK * 2;    // this CTA's 64 W1 rows of one atom
    static constexpr int kAtoms = 2;
    static constexpr int kStageBytes = kAtoms * (kBytesA + kBytesB);
    static constexpr int kStages = 4;
    static constexpr int kRingBytes = kStages * kStageBytes;
    static constexpr int kTmemCols = kPairBN;
    static constexpr size_t kSmemBytes = (size_t)kRingBytes + 1024 + ((sizeof(Control) + 255) / 256) * 256;
};

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(0u)
        : "memory");
}
// arrives, once the MMAs issued so far are complete, on the barrier at this address in every CTA of `mask`
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar, uint16_t mask)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask)
                 : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1)
verifier_pair_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                     const VerifyParams prm)
{
    using Cfg = PairCfg;
    constexpr int BM = kPairBM, BN = kPairBN;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *ring = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Control *ctl = reinterpret_cast<Control *>(ring + Cfg::kRingBytes);

    pdl_trigger();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) SPR_STAMP(0);
    const int M = prm.B * prm.K;
    const int half = (int)blockIdx.x;                  // 0: the CTA that issues the MMAs, 1: its peer
    const int n0 = blockIdx.y * BN;
    const int tile = (int)blockIdx.z * 2 + half;       // token tile of this CTA
    const int m0 = tile * BM;
    const int num_atoms = (prm.d + kAtomK - 1) / kAtomK;
    const int num_stages = (num_atoms + Cfg::kAtoms - 1) / Cfg::kAtoms;
    const uint32_t cy = blockIdx.y % (unsigned)prm.cluster_n;
    const uint32_t my_rank = (uint32_t)half + 2u * cy;             // x runs fastest inside the cluster
    const uint32_t limit = prm.spin_limit;
    const int live_rows = max(0, min(BM, M - m0));                 // the odd tile may lie past the batch
    const bool z_receiver = prm.final_in_cluster && cy == 0;       // one per token tile

    if (tid == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->tmem_full, 1);
        mbar_init(&ctl->drain, 1);
        mbar_init(&ctl->zgather, 1);
        if (z_receiver && live_rows > 0) mbar_expect_tx(&ctl->zgather, (uint32_t)(prm.cluster_n * live_rows * 4));
        ctl->abort = 0;
        ctl->last = 0;
        ctl->consumed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0 && lane < 2)
        asm volatile("prefetch.tensormap [%0];" ::"l"(lane == 0 ? &map_h : &map_w) : "memory");
    if (warp == 1) {   // both CTAs of the pair allocate the same columns
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                     "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = ctl->tmem_base;
    // "started, barriers set up": the peer's copies count on the even CTA's barriers and its
    // commits arrive on the peer's, so both sides check for this word before their loops
    cluster_arrive();
    if (tid == 0) SPR_STAMP(1);

    int issued = 0;
    bool ok = true;
    if (warp == 0) {
        // ---------------- TMA producer (both CTAs): even lanes hidden-state atoms, odd lanes W1 atoms
        cluster_wait();
        if (lane < 2 * Cfg::kAtoms && !(prm.test_flags & VERIFIER_TEST_NO_LOADS)) {
            const int atom = lane >> 1;
            const bool is_w = lane & 1;
            const CUtensorMap *map = is_w ? &map_w : &map_h;
            const int row0 = is_w ? n0 + half * (BN / 2) : m0;
            const uint32_t off = is_w ? (uint32_t)(Cfg::kAtoms * Cfg::kBytesA + atom * Cfg::kBytesB)
                                      : (uint32_t)(atom * Cfg::kBytesA);
            for (int st = 0; st < num_stages; ++st) {
                const int s = st % Cfg::kStages;
                const uint32_t round = (uint32_t)(st / Cfg::kStages);
                const int n_at = min(Cfg::kAtoms, num_atoms - st * Cfg::kAtoms);
                if (!mbar_wait(&ctl->empty[s], (round & 1u) ^ 1u, ctl, prm.status, limit)) break;
                // the even CTA expects the bytes of both
                if (lane == 0 && half == 0)
                    mbar_expect_tx(&ctl->full[s], (uint32_t)(2 * n_at * (Cfg::kBytesA + Cfg::kBytesB)));
                if (atom < n_at)
                    tma_load_2d_pair(smem_u32(ring + (size_t)s * Cfg::kStageBytes) + off, map,
                                     (st * Cfg::kAtoms + atom) * kAtomK, row0, smem_u32(&ctl->full[s]) & kPeerBitMask);
                issued = st + 1;
                if (st == 0) SPR_STAMP(2);
                if (st < 24 && lane == 0) SPR_STAMP(40 + st);
            }
        }
    } else if (warp == 1) {
        cluster_wait();
        // ---------------- MMA issuer: one thread of the even CTA, for both
        if (lane == 0 && half == 0) {
            constexpr uint32_t idesc = umma_instr_desc<2 * BM, BN>();
            const uint16_t both = (uint16_t)(3u << my_rank);
            bool fed = true;
            int st = 0;
            for (; st < num_stages; ++st) {
                const int s = st % Cfg::kStages;
                const uint32_t round = (uint32_t)(st / Cfg::kStages);
                const int n_at = min(Cfg::kAtoms, num_atoms - st * Cfg::kAtoms);
                fed = mbar_wait(&ctl->full[s], round & 1u, ctl, prm.status, limit);
                if (!fed) break;
                if (st == 0) SPR_STAMP(3);
                if (st < 24) SPR_STAMP(16 + st);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(ring + (size_t)s * Cfg::kStageBytes);
                const uint32_t b_addr = a_addr + Cfg::kAtoms * Cfg::kBytesA;
#pragma unroll
                for (int a = 0; a < Cfg::kAtoms; ++a) {
                    if (a < n_at) {
                        const uint64_t da = umma_smem_desc(a_addr + a * Cfg::kBytesA);
                        const uint64_t db = umma_smem_desc(b_addr + a * Cfg::kBytesB);
#pragma unroll
                        for (int k = 0; k < kAtomK / kUmmaK; ++k) {
                            const uint64_t adv = (uint64_t)((k * kUmmaK * 2) >> 4);
                            umma_bf16_pair(tmem_acc, da + adv, db + adv, idesc, (st | a | k) != 0 ? 1u : 0u);
                        }
                    }
                }
                umma_commit_pair(&ctl->empty[s], both);     // the stage is free in both CTAs
            }
            ctl->consumed = st;
            SPR_STAMP(4);
            if (fed) umma_commit_pair(&ctl->tmem_full, both);   // both epilogues may read
            else umma_commit_pair(&ctl->drain, (uint16_t)(1u << my_rank));
        }
    } else {
        for (int j = tid - 64; j < BN; j += kTcThreads - 64) {
            const int n = n0 + j;
            ctl->b1[j] = n < prm.h ? prm.b1[n] : 0.f;
            ctl->w2[j] = n < prm.h ? __bfloat162float(static_cast<const __nv_bfloat16 *>(prm.W2)[n]) : 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        cluster_wait();
        ok = mbar_wait(&ctl->tmem_full, 0, ctl, prm.status, limit);
        if (tid == 64) SPR_STAMP(5);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    __syncwarp();

    const int quarter = warp & 3;
    const int r_in = quarter * 32 + lane;
    const int row = m0 + r_in;
    const bool live_row = warp >= 2 && row < M;
    const uint32_t lane_base = tmem_acc + ((uint32_t)(quarter * 32) << 16);

    float z = 0.f;
    if (warp >= 2) {
#pragma unroll
        for (int c0 = 0; c0 < BN; c0 += 64) {
            uint32_t v[2][32];
            tmem_ld32(lane_base + (uint32_t)c0, v[0]);
            tmem_ld32(lane_base + (uint32_t)(c0 + 32), v[1]);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 64; ++j)
                z = fmaf(ctl->w2[c0 + j], fmaxf(__uint_as_float(v[j >> 5][j & 31]) + ctl->b1[c0 + j], 0.f), z);
        }
        if (!ok || *reinterpret_cast<volatile int *>(&ctl->abort)) z = poisoned_z();
        if (prm.final_in_cluster) {
            // to the CTA that finishes this token tile: same half of the pair, first slice
            if (live_row)
                st_async_b32(peer_smem(smem_u32(&ctl->zbuf[cy][r_in]), (uint32_t)half), __float_as_uint(z),
                             peer_smem(smem_u32(&ctl->zgather), (uint32_t)half));
            if (z_receiver && live_rows > 0) {
                const bool got = mbar_wait(&ctl->zgather, 0, ctl, prm.status, limit);
                if (!got && live_row) ctl->zbuf[0][r_in] = poisoned_z();
            }
        } else if (live_row) {
            prm.part_z[(int64_t)blockIdx.y * M + row] = z;
        }
    }
    __syncwarp();
    if (tid == 64) SPR_STAMP(8);
    cluster_arrive();   // done with the peers: TMEM read, nothing more sent or expected

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (*reinterpret_cast<volatile int *>(&ctl->abort)) {
        if (warp == 0) {
            int last = issued;
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
            // the copies of both CTAs count on the even CTA's barriers: it waits for them
            if (lane == 0 && half == 0) {
                for (int st = ctl->consumed; st < last; ++st)
                    mbar_wait_quiet(&ctl->full[st % Cfg::kStages], (uint32_t)(st / Cfg::kStages) & 1u, limit);
            }
        }
        if (warp == 1 && lane == 0 && half == 0 && ctl->consumed < num_stages) mbar_wait_quiet(&ctl->drain, 0, limit);
        __syncthreads();
    }

    if (tid == 64) SPR_STAMP(9);
    // ---------------- finish (as in the single-CTA kernel)
    const int m_hi = min(m0 + BM, M);
    bool finisher = false;
    if (live_rows > 0) {
        if (prm.final_in_cluster) {
            finisher = z_receiver;
            if (finisher) {
                const float b2 = prm.b2[0];
                for (int t = tid; t < m_hi - m0; t += kTcThreads) {
                    float zt = b2;
                    for (int i = 0; i < prm.cluster_n; ++i) zt += ctl->zbuf[i][t];
                    ctl->codes[t] = (unsigned char)classify_token(prm, zt, m0 + t);
                }
                __syncthreads();
                if (prm.first_reject) {
                    const int b_lo = (m0 + prm.K - 1) / prm.K, b_hi = m_hi / prm.K;
                    for (int b = b_lo + warp; b < b_hi; b += kTcThreads / 32)
                        scan_sequence_smem(prm, b, ctl->codes + (b * prm.K - m0), lane);
                }
            }
        } else {
            if (tid == 0) {
                __threadfence();
                ctl->last = take_ticket(&prm.counter[1 + tile], (int)gridDim.y);
            }
            __syncthreads();
            finisher = ctl->last != 0;
            if (finisher) {
                __threadfence();
                finalise_tile(prm, m0, m_hi, ctl->codes);
            }
        }
    }
    // sequences cut by a tile boundary wait for the CTA that completes the last tile
    if (finisher && BM % prm.K != 0 && M > BM) {
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            ctl->last = take_ticket(&prm.counter[0], (M + BM - 1) / BM);
        }
        __syncthreads();
        if (ctl->last) {
            __threadfence();
            finalise_straddlers(prm, BM);
        }
    }
    if (tid == 64) SPR_STAMP(10);
    // Both CTAs are through with the accumulator (and nobody is still sending here): release it
    cluster_wait();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static const EncodeTiledFn fn = [] {   // initialised once, thread-safe
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
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

struct Shape {
    int bm, bn, splits, cluster_n;
};

int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// k-blocks per CTA when d is cut S ways, or 0 if some CTA would get none
int kb_per_split(int d, int S)
{
    const int kb_all = ceil_div(d, kAtomK), per = ceil_div(kb_all, S);
    return (int64_t)(S - 1) * per < kb_all ? per : 0;
}

bool shape_usable(const Shape &s, int64_t M, int d, int h)
{
    if (s.bm == 2 * kPairBM) {   // a pair of CTAs per 256 x 128 tile
        const int slices = ceil_div(h, kPairBN);
        return s.bn == kPairBN && s.splits == 1 && (s.cluster_n == 1 || (s.cluster_n == slices && 2 * slices <= kMaxClusterCtas)) &&
               slices <= 65535 && ceil_div(M, 2 * kPairBM) <= 65535;
    }
    if ((s.bm != 64 && s.bm != 128) || (s.bn != 64 && s.bn != 128)) return false;
    if (s.splits != 1 && s.splits != 2 && s.splits != 4 && s.splits != 8) return false;
    if (s.bn / s.splits < 8 || kb_per_split(d, s.splits) == 0) return false;
    const int slices = ceil_div(h, s.bn);
    if (s.cluster_n != 1 && s.cluster_n != slices) return false;
    if (s.splits * s.cluster_n > kMaxClusterCtas) return false;
    if (slices > 65535 || ceil_div(M, s.bm) > 65535) return false;
    return true;
}

// Estimated microseconds of a launch with this shape: a model with a handful of constants
// fitted to CUDA-graph timings of every usable shape on the library's workload sizes (B200).
//   per CTA: set-up and first data; the k-loop, whose stages each cost the larger of a fixed
//            barrier/issue latency, the rows they fetch (one 128-byte row per ~2 clocks) and
//            their tensor-pipe time; the exchange of accumulator columns when d is split;
//            the epilogue
//   per launch: waves of clusters (a cluster of c CTAs fits the GPU 148, 74, 33, 15 times for
//            c = 1, 2, 4, 8) and the finish - cheap inside a cluster, two trips through
//            global memory otherwise.
double shape_cost(const Shape &s, int64_t M, int K, int d, int h)
{
    const bool pair = s.bm == 2 * kPairBM;
    const int slices = ceil_div(h, s.bn), tiles = ceil_div(M, s.bm);
    const int cluster_ctas = (pair ? 2 : s.splits) * s.cluster_n;
    const int64_t clusters = (int64_t)tiles * slices * (pair ? 2 : s.splits) / cluster_ctas;
    const int capacity = cluster_ctas == 1 ? 148 : cluster_ctas == 2 ? 74 : cluster_ctas <= 4 ? 33 : 15;
    const double waves = (double)((clusters + capacity - 1) / capacity);
    const int atoms_per_stage = s.bm + s.bn == 128 ? 4 : 2;
    const int stage_bytes = atoms_per_stage * (pair ? kPairBM + kPairBN / 2 : s.bm + s.bn) * kAtomK * 2;
    const int ring = (200 * 1024) / stage_bytes;
    const int stages = ceil_div(kb_per_split(d, s.splits), atoms_per_stage);
    const double rows_a = pair ? (double)kPairBM : tiles == 1 ? (double)((M + 7) / 8 * 8) : (double)s.bm;
    const double rows = rows_a + (pair ? (double)(kPairBN / 2) : (double)(h < s.bn ? h : s.bn));
    // (all SMs together take about 13 TB/s from L2: a pair fetches fewer rows, each a little slower)
    const double feed = rows * atoms_per_stage * (pair ? 0.00153 : 0.00135);
    const double mma = (double)(pair ? kPairBM : s.bm) * s.bn * atoms_per_stage * kAtomK / 8192.0 / 1965.0;
    double stage = 0.483;
    if (feed > stage) stage = feed;
    if (mma > stage) stage = mma;
    double loop = stages * stage, exchange = 0.0;
    if (s.splits > 1) {
        const double rows_live = (double)(M < s.bm ? M : s.bm);
        exchange = 2 * 0.314 + rows_live * s.bn * 4 / 1000.0 * 0.0124;
        const bool dedicated = s.bm * s.bn * 4 <= stage_bytes && ring - 1 >= (stages < 3 ? stages : 3);
        if (!dedicated) exchange += 1.32;           // the hand-shake after the k-loop
        else if (stages > ring - 1) loop += 0.83;   // one stage fewer in flight
    }
    const double finish = s.cluster_n == slices ? 0.314 : (K == 1 && slices <= 255 ? 0.0 : 1.94);
    return 1.12 + waves * ((pair ? 2.6 : 2.15) + loop + exchange + 2.03) + finish;
}

Shape choose_shape(int64_t M, int K, int d, int h)
{
    Shape best = {64, 64, 1, 1};
    double best_cost = -1.0;
    for (int bm = 64; bm <= 128; bm += 64) {
        if (bm == 128 && M <= 64) continue;
        for (int bn = 64; bn <= 128; bn += 64) {
            if (bn == 128 && h <= 64) continue;
            for (int S = 1; S <= 8; S *= 2) {
                const int slices = ceil_div(h, bn);
                for (int all = 0; all < 2; ++all) {
                    const Shape s = {bm, bn, S, all ? slices : 1};
                    if (all && slices == 1) continue;
                    if (!shape_usable(s, M, d, h)) continue;
                    const double c = shape_cost(s, M, K, d, h);
                    if (best_cost < 0.0 || c < best_cost) {
                        best_cost = c;
                        best = s;
                    }
                }
            }
        }
    }
    // CTA pairs: once the batch has at least two 128-token tiles per pair of SMs
    if (M >= 512 && h > 64) {
        const int slices = ceil_div(h, kPairBN);
        for (int all = 0; all < 2; ++all) {
            const Shape s = {2 * kPairBM, kPairBN, 1, all ? slices : 1};
            if ((all && slices == 1) || !shape_usable(s, M, d, h)) continue;
            const double c = shape_cost(s, M, K, d, h);
            if (c < best_cost) {
                best_cost = c;
                best = s;
            }
        }
    }
    return best;
}

int launch_pair(const CUtensorMap &mh, const CUtensorMap &mw, VerifyParams vp, const Shape &s, cudaStream_t st)
{
    static std::atomic<bool> attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(verifier_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)PairCfg::kSmemBytes);
        if (e != cudaSuccess) return (int)e;
        attr_set[dev].store(true, std::memory_order_release);
    }
    const int slices = ceil_div(vp.h, kPairBN);
    const int64_t M = (int64_t)vp.B * vp.K;
    vp.slices = slices;
    vp.cluster_n = s.cluster_n;
    vp.final_in_cluster = s.cluster_n == slices ? 1 : 0;
    vp.atomic_finish = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u, (unsigned)slices, (unsigned)ceil_div(M, 2 * kPairBM));
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = PairCfg::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = (unsigned)s.cluster_n;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return (int)cudaLaunchKernelEx(&cfg, verifier_pair_kernel, mh, mw, vp);
}

template <int BM, int BN>
int launch_tile(const CUtensorMap &mh, const CUtensorMap &mw, VerifyParams vp, const Shape &s, int tiles_m,
                cudaStream_t st)
{
    using Cfg = TileCfg<BM, BN>;
    static std::atomic<bool> attr_set[64];   // host threads may race to set it: all of them store `true`
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(verifier_tcgen05_kernel<BM, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)Cfg::kSmemBytes);
        if (e != cudaSuccess) return (int)e;
        attr_set[dev].store(true, std::memory_order_release);
    }
    const int slices = ceil_div(vp.h, BN);
    vp.slices = slices;
    vp.kb_per = kb_per_split(vp.d, s.splits);
    // With d split, the accumulator columns that arrive from the other CTAs get the room of
    // the last pipeline stage if enough stages remain; else they overlay the ring after the k-loop.
    const int stages_needed = ceil_div(vp.kb_per, Cfg::kAtoms);
    const int spare = Cfg::kStages - 1;
    vp.recv_dedicated = s.splits > 1 && BM * BN * 4 <= Cfg::kStageBytes && spare >= (stages_needed < 3 ? stages_needed : 3);
    vp.ring_stages = vp.recv_dedicated ? spare : Cfg::kStages;
    vp.cluster_n = s.cluster_n;
    vp.final_in_cluster = s.cluster_n == slices ? 1 : 0;
    vp.atomic_finish = !vp.final_in_cluster && vp.K == 1 && vp.zacc && slices <= 255;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)s.splits, (unsigned)slices, (unsigned)tiles_m);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (s.splits * s.cluster_n > 1) {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)s.splits;
        attr[0].val.clusterDim.y = (unsigned)s.cluster_n;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    return (int)cudaLaunchKernelEx(&cfg, verifier_tcgen05_kernel<BM, BN>, mh, mw, vp);
}

}  // namespace

#ifdef SPR_VERIFIER_STAMPS
extern "C" int spr_debug_max_clusters(int cx, int cy)   // co-resident clusters of the 64 x 128 kernel
{
    using Cfg = TileCfg<64, 128>;
    cudaFuncSetAttribute(verifier_tcgen05_kernel<64, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmemBytes);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cx * 16, cy * 16, 1);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cx;
    attr[0].val.clusterDim.y = cy;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = -1;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&n, verifier_tcgen05_kernel<64, 128>, &cfg);
    return e == cudaSuccess ? n : -(int)e;
}
extern "C" int spr_debug_verifier_stamps(long long *host_out)   // [512][64]
{
    cudaError_t e = cudaMemcpyFromSymbol(host_out, g_stamps, sizeof(long long) * 512 * 64);   // reads, then clears
    void *p = nullptr;
    if (e == cudaSuccess) e = cudaGetSymbolAddress(&p, g_stamps);
    if (e == cudaSuccess) e = cudaMemset(p, 0, sizeof(long long) * 512 * 64);
    return (int)e;
}
#endif

int verifier_tensor_max_slices(int h) { return ceil_div(h > 0 ? h : 1, 128) * 16; }

int launch_verifier_tensor(const VerifyParams &vp_in, int dt, int min_tokens, const VerifierTune *tune,
                           cudaStream_t st)
{
    VerifyParams vp = vp_in;
    const int64_t M = (int64_t)vp.B * vp.K;
    if (dt != SPR_BF16 || vp.h <= 0 || vp.d % 8 != 0 || M < min_tokens) return -1;
    if ((reinterpret_cast<uintptr_t>(vp.hidden) & 15) || (reinterpret_cast<uintptr_t>(vp.W1) & 15)) return -1;
    Shape s = choose_shape(M, vp.K, vp.d, vp.h);
    vp.spin_limit = kSpinLimit;
    vp.test_flags = 0;
    if (tune) {
        if (tune->bm) s.bm = tune->bm;
        if (tune->bn) s.bn = tune->bn;
        if (tune->splits) s.splits = tune->splits;
        const int slices = ceil_div(vp.h, s.bn);
        if (tune->cluster_n) s.cluster_n = tune->cluster_n < 0 ? slices : 1;
        else if (tune->bm || tune->bn || tune->splits)
            s.cluster_n = (s.bm == 2 * kPairBM ? 2 : s.splits) * slices <= kMaxClusterCtas ? slices : 1;
        if (tune->spin_limit) vp.spin_limit = tune->spin_limit;
        vp.test_flags = tune->test_flags;
    }
    if (!shape_usable(s, M, vp.d, vp.h)) return -1;
    if (s.bm == 2 * kPairBM) {
        CUtensorMap mh, mw;
        if (!make_map(&mh, vp.hidden, (int)M, vp.d, kPairBM)) return -1;
        if (!make_map(&mw, vp.W1, vp.h, vp.d, kPairBN / 2)) return -1;
        return launch_pair(mh, mw, vp, s, st);
    }
    const int tiles_m = ceil_div(M, s.bm);
    // a batch that fills only part of its one tile fetches only the rows it has (the rest of
    // the operand tile stays as it is: accumulator rows that are never read)
    vp.a_box_rows = tiles_m == 1 ? (int)((M + 7) / 8 * 8) : s.bm;
    CUtensorMap mh, mw;
    if (!make_map(&mh, vp.hidden, (int)M, vp.d, vp.a_box_rows)) return -1;
    if (!make_map(&mw, vp.W1, vp.h, vp.d, s.bn)) return -1;
#define SPR_TILE(BM_, BN_) \
    if (s.bm == BM_ && s.bn == BN_) return launch_tile<BM_, BN_>(mh, mw, vp, s, tiles_m, st)
    SPR_TILE(64, 64);
    SPR_TILE(64, 128);
    SPR_TILE(128, 64);
    SPR_TILE(128, 128);
#undef SPR_TILE
    return -1;
}

}  // namespace spr
