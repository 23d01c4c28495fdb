// Measurement aid, not part of the library: what a B200 delivers to warps that each read one
// contiguous 4 KB row per turn (the access pattern of the verifier's training pass), with
// nothing computed but an XOR of the words - by vector loads into registers with 32 to 128 KB in
// flight per SM, and by one bulk copy per row into a per-warp ring of shared memory.  The
// figures quoted under profiles/ for the training pass come from this program
// (python -m paper_2502_04557_b200.stream_probes).
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("err %s line %d\n", cudaGetErrorString(e), __LINE__); return 1; } } while (0)

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// one 4 KB row per warp per iteration, 8 x 16 B per lane; ROWS rows in flight per warp
template <int ROWS>
__global__ void __launch_bounds__(256) reg_read(const uint4 *x, int64_t n_rows, unsigned *out)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t stride = (int64_t)gridDim.x * 8;
    unsigned acc = 0;
    for (int64_t row = (int64_t)blockIdx.x * 8 + warp; row < n_rows; row += stride * ROWS) {
        uint4 v[ROWS][8];
#pragma unroll
        for (int r = 0; r < ROWS; ++r)
#pragma unroll
            for (int j = 0; j < 8; ++j)
                v[r][j] = row + r * stride < n_rows ? ld_stream(x + (row + r * stride) * 256 + j * 32 + lane) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int r = 0; r < ROWS; ++r)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc ^= v[r][j].x ^ v[r][j].y ^ v[r][j].z ^ v[r][j].w;
    }
    if (acc == 0x12345678u) out[0] = acc;
}

__device__ __forceinline__ uint32_t sa(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// per-warp ring of SLOTS 4 KB slots filled by bulk copies
template <int SLOTS>
__global__ void __launch_bounds__(256, 1) ring_read(const uint4 *x, int64_t n_rows, unsigned *out, int *err)
{
    extern __shared__ __align__(128) unsigned char sm[];
    __shared__ __align__(8) uint64_t bars[8][SLOTS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint4 *ring = reinterpret_cast<uint4 *>(sm) + warp * SLOTS * 256;
    uint64_t *bar = bars[warp];
    const int64_t stride = (int64_t)gridDim.x * 8, first = (int64_t)blockIdx.x * 8 + warp;
    const int n = first < n_rows ? (int)((n_rows - first + stride - 1) / stride) : 0;
    auto fetch = [&](int i, int s) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sa(&bar[s])), "r"(4096) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sa(ring + s * 256)),
                     "l"(x + (first + (int64_t)i * stride) * 256), "r"(4096), "r"(sa(&bar[s])) : "memory");
    };
    if (lane == 0) {
        for (int s = 0; s < SLOTS; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sa(&bar[s])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < SLOTS && i < n; ++i) fetch(i, i);
    }
    __syncwarp();
    unsigned acc = 0;
    int s = 0;
    uint32_t par = 0;
    for (int i = 0; i < n; ++i) {
        bool ok = false;
        for (int k = 0; k < (1 << 22) && !ok; ++k) {
            uint32_t d;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(d) : "r"(sa(&bar[s])), "r"(par) : "memory");
            ok = d != 0;
        }
        if (!ok) { if (lane == 0) atomicExch(err, 1); break; }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint4 v = ring[s * 256 + j * 32 + lane];
            acc ^= v.x ^ v.y ^ v.z ^ v.w;
        }
        __syncwarp();
        if (lane == 0 && i + SLOTS < n) fetch(i + SLOTS, s);
        if (++s == SLOTS) { s = 0; par ^= 1; }
    }
    if (acc == 0x12345678u) out[0] = acc;
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

int main()
{
    const int64_t n_rows = 1 << 20;
    const size_t bytes = (size_t)n_rows * 4096;
    uint4 *x; unsigned *out; int *err;
    CK(cudaMalloc(&x, bytes)); CK(cudaMalloc(&out, 4)); CK(cudaMalloc(&err, 4));
    CK(cudaMemset(x, 1, bytes)); CK(cudaMemset(err, 0, 4));
    for (int ctas_per_sm = 1; ctas_per_sm <= 4; ++ctas_per_sm) {
        float ms = time_it([&] { reg_read<1><<<148 * ctas_per_sm, 256>>>(x, n_rows, out); });
        printf("reg_read<1 row>  %d CTAs/SM: %.1f us  %.0f GB/s\n", ctas_per_sm, ms * 1e3, bytes / ms / 1e6);
    }
    for (int ctas_per_sm = 1; ctas_per_sm <= 2; ++ctas_per_sm) {
        float ms = time_it([&] { reg_read<2><<<148 * ctas_per_sm, 256>>>(x, n_rows, out); });
        printf("reg_read<2 rows> %d CTAs/SM: %.1f us  %.0f GB/s\n", ctas_per_sm, ms * 1e3, bytes / ms / 1e6);
    }
    CK(cudaGetLastError());
    {
        CK(cudaFuncSetAttribute(ring_read<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * 2 * 4096));
        CK(cudaFuncSetAttribute(ring_read<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * 4 * 4096));
        CK(cudaFuncSetAttribute(ring_read<6>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * 6 * 4096));
        float ms = time_it([&] { ring_read<2><<<148, 256, 8 * 2 * 4096>>>(x, n_rows, out, err); });
        printf("ring_read<2 slots>: %.1f us  %.0f GB/s\n", ms * 1e3, bytes / ms / 1e6);
        ms = time_it([&] { ring_read<4><<<148, 256, 8 * 4 * 4096>>>(x, n_rows, out, err); });
        printf("ring_read<4 slots>: %.1f us  %.0f GB/s\n", ms * 1e3, bytes / ms / 1e6);
        ms = time_it([&] { ring_read<6><<<148, 256, 8 * 6 * 4096>>>(x, n_rows, out, err); });
        printf("ring_read<6 slots>: %.1f us  %.0f GB/s\n", ms * 1e3, bytes / ms / 1e6);
        ms = time_it([&] { ring_read<2><<<296, 256, 8 * 2 * 4096>>>(x, n_rows, out, err); });
        printf("ring_read<2 slots> 2 CTAs/SM: %.1f us  %.0f GB/s\n", ms * 1e3, bytes / ms / 1e6);
        ms = time_it([&] { ring_read<4><<<296, 256, 8 * 4 * 4096>>>(x, n_rows, out, err); });
        printf("ring_read<4 slots> 2 CTAs/SM: %.1f us  %.0f GB/s\n", ms * 1e3, bytes / ms / 1e6);
    }
    CK(cudaDeviceSynchronize());
    int h = 0; CK(cudaMemcpy(&h, err, 4, cudaMemcpyDeviceToHost));
    printf("err flag %d\n", h);
    return 0;
}
