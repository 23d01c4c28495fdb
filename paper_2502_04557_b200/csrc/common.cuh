// Shared device helpers and the workspace layout of libsprinter.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sprinter.h"

namespace spr {

// ---------------------------------------------------------------- constants
constexpr int kThreads = 256;           // CTA size of the vocabulary kernels
constexpr int kUnroll = 4;              // 16-byte vectors per lane per warp step
constexpr int kWarps = kThreads / 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kHeaderBytes = 256;       // workspace header; word 0 is the sticky status

__host__ __device__ constexpr int elem_size(int dt) { return dt == SPR_F32 ? 4 : 2; }
__host__ __device__ constexpr int vec_elems(int dt) { return 16 / elem_size(dt); }

// Vocabulary kernels: a warp consumes "steps" of 32 lanes x kUnroll vectors, kStatIters of
// them per CTA, so one CTA covers a segment of kWarps*kStatIters = 32 steps of a row (32768
// bf16 or 16384 fp32 elements).  Rows may start up to one vector minus one element past a
// 16-byte boundary, hence the vec_elems - 1 below.
constexpr int kStatIters = 4;
__host__ __device__ constexpr int stat_step_elems(int dt) { return 32 * kUnroll * vec_elems(dt); }
__host__ __device__ constexpr int stat_segment_elems(int dt) { return kWarps * kStatIters * stat_step_elems(dt); }
__host__ __device__ inline int stat_steps_per_row(int V, int dt)
{
    return (V + vec_elems(dt) - 1 + stat_step_elems(dt) - 1) / stat_step_elems(dt);
}
// most segments a row can be cut into (one step per warp)
__host__ __device__ inline int stat_max_segments_per_row(int V, int dt)
{
    return (stat_steps_per_row(V, dt) + kWarps - 1) / kWarps;
}
__host__ __device__ inline int stat_segments_per_row(int V, int dt)
{
    return (V + vec_elems(dt) - 1 + stat_segment_elems(dt) - 1) / stat_segment_elems(dt);
}

// With few rows to read, a row is spread over more CTAs (fewer steps per warp), which
// shortens the chain of dependent loads each CTA goes through.
inline void draw_geometry(int n, int steps, int *segments, int *iters)
{
    int it = kStatIters;
    while (it > 1 && (int64_t)n * ((steps + kWarps * it - 1) / (kWarps * it)) < 148) it /= 2;
    *iters = it;
    *segments = (steps + kWarps * it - 1) / (kWarps * it);
}

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---------------------------------------------------------------- workspace layouts
// All offsets are multiples of 256 bytes from the start of the workspace.  Every layout
// puts its ticket counters in one contiguous zone right after the header; the entry point
// clears that zone on the stream before its first kernel, so a workspace may be shared by
// calls of different ops and shapes.
struct DrawWs {              // replace_sample, and the correction draw of sd_verify
    size_t counters;         // int32 [n]      segments finished per draw
    size_t part;             // float2 [n*T]   (max, weight) of every warp step
    size_t end;
};
__host__ __device__ inline DrawWs draw_ws_layout(size_t counters, size_t scratch, int n, int T)
{
    DrawWs w;
    w.counters = counters;
    w.part = align_up(scratch, 256);
    w.end = align_up(w.part + 8 * (size_t)n * T, 256);
    return w;
}
// replace_sample alone: counters [n] directly after the header
__host__ __device__ inline DrawWs replace_ws_layout(int n, int T)
{
    return draw_ws_layout(kHeaderBytes, kHeaderBytes + align_up(sizeof(int32_t) * (size_t)n, 256), n, T);
}

struct SdWs {
    size_t row_counters;     // int32 [M]      segments finished per row
    size_t seq_counters;     // int32 [B]      rows finished per sequence
    size_t counters_end;     // end of the zone cleared per call (includes the draw counters)
    size_t acc;              // uint8 [M]      0 reject, 1 accept, 2 invalid token
    size_t part;             // float4 [M*S]   (max_p, sum_p, max_q, sum_q) per row segment
    size_t rowstats;         // float4 [M]     (max_p, ln Z_p, max_q, ln Z_q)
    DrawWs draw;             // correction draw, n = B
    size_t end;
};
__host__ __device__ inline SdWs sd_ws_layout(int B, int K, int S, int T)   // S segments, T steps per row
{
    const size_t M = (size_t)B * K;
    SdWs w;
    w.row_counters = kHeaderBytes;
    w.seq_counters = w.row_counters + 4 * M;
    const size_t draw_counters = w.seq_counters + 4 * (size_t)B;
    w.counters_end = align_up(draw_counters + 4 * (size_t)B, 256);
    w.acc = w.counters_end;
    w.part = align_up(w.acc + M, 256);
    w.rowstats = align_up(w.part + 16 * M * S, 256);
    w.draw = draw_ws_layout(draw_counters, align_up(w.rowstats + 16 * M, 256), B, T);
    w.end = w.draw.end;
    return w;
}

struct ShardWs {             // vocabulary-sharded sd_verify: the four passes share one workspace
    size_t row_counters;     // int32 [B*Kp]
    size_t draw_counters;    // int32 [B]
    size_t counters_end;
    size_t acc;              // uint8 [B*K]
    size_t part;             // float4 [B*Kp*S]
    size_t rowstats;         // float4 [B*Kp]  whole-row (max_p, ln Z_p, max_q, ln Z_q)
    size_t draw_part;        // float2 [B*T]
    size_t end;
};
__host__ __device__ inline ShardWs shard_ws_layout(int B, int K, int Kp, int S, int T)
{
    const size_t R = (size_t)B * Kp;
    ShardWs w;
    w.row_counters = kHeaderBytes;
    w.draw_counters = w.row_counters + 4 * R;
    w.counters_end = align_up(w.draw_counters + 4 * (size_t)B, 256);
    w.acc = w.counters_end;
    w.part = align_up(w.acc + (size_t)B * K, 256);
    w.rowstats = align_up(w.part + 16 * R * S, 256);
    w.draw_part = align_up(w.rowstats + 16 * R, 256);
    w.end = align_up(w.draw_part + 8 * (size_t)B * T, 256);
    return w;
}

struct LabelWs {             // verifier_labels: row records of the statistics pass
    size_t row_counters;     // int32 [M]
    size_t part;             // float4 [M*S]
    size_t stats;            // float [M*6]
    size_t end;
};
__host__ __device__ inline LabelWs label_ws_layout(int B, int K, int S)
{
    const size_t M = (size_t)B * K;
    LabelWs w;
    w.row_counters = kHeaderBytes;
    w.part = align_up(w.row_counters + 4 * M, 256);
    w.stats = align_up(w.part + 16 * M * S, 256);
    w.end = align_up(w.stats + 24 * M, 256);
    return w;
}

// verifier_train_step: per-CTA gradient sums, float [kTrainMaxCtas, d + 2]
constexpr int kTrainMaxCtas = 592;   // 148 SMs x 4
__host__ __device__ inline size_t train_ws_bytes(int d)
{
    return align_up(kHeaderBytes + 4 * (size_t)kTrainMaxCtas * ((size_t)d + 2), 256);
}

struct VerifyWs {
    size_t counter;          // int32 [1 + max(row tiles, B)]   CTAs finished per tile / tokens per sequence
    size_t counters_end;
    size_t part_z;           // float [slices * M]      per-slice partial of W2 . relu(...)
    size_t end;
};
__host__ __device__ inline VerifyWs verify_ws_layout(int M, int slices, int tiles)
{
    VerifyWs w;
    w.counter = kHeaderBytes;
    w.counters_end = align_up(w.counter + 4 * (size_t)(1 + tiles), 256);
    w.part_z = w.counters_end;
    w.end = align_up(w.part_z + 4 * (size_t)slices * M, 256);
    return w;
}

struct StepWs {              // sprinter_step: verifier and replacement draw in one call
    size_t verify_counter;   // int32 [1 + row tiles]
    size_t draw_counters;    // int32 [B]
    size_t counters_end;
    size_t part_z;           // float [slices * M]
    DrawWs draw;
    size_t end;
};
__host__ __device__ inline StepWs step_ws_layout(int B, int K, int slices, int tiles, int T)
{
    const size_t M = (size_t)B * K;
    StepWs w;
    w.verify_counter = kHeaderBytes;
    w.draw_counters = w.verify_counter + 4 * (size_t)(1 + tiles);
    w.counters_end = align_up(w.draw_counters + 4 * (size_t)B, 256);
    w.part_z = w.counters_end;
    w.draw = draw_ws_layout(w.draw_counters, align_up(w.part_z + 4 * (size_t)slices * M, 256), B, T);
    w.end = w.draw.end;
    return w;
}

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// Programmatic dependent launch: a kernel launched with the programmatic-serialisation
// attribute may start while the kernel before it in the stream is still running; it must
// call pdl_wait() before touching anything that kernel writes.  pdl_trigger() in the earlier
// kernel allows the next one to be scheduled as soon as every CTA has got this far.  Both are
// no-ops for ordinary launches.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// first error wins; the word stays set until the host clears it
__device__ __forceinline__ void raise_status(int *status, int code) { atomicCAS(status, 0, code); }

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// (m, s): s = sum of exp(x - m) over some set.  Merge of two sets, safe for empty ones (m = -inf).
struct MS {
    float m, s;
};
__device__ __forceinline__ MS ms_merge(MS a, MS b)
{
    const float m = fmaxf(a.m, b.m);
    const float ref = (m == neg_inf()) ? 0.f : m;
    MS r;
    r.m = m;
    r.s = a.s * ex2((a.m - ref) * kLog2e) + b.s * ex2((b.m - ref) * kLog2e);
    return r;
}
__device__ __forceinline__ MS warp_ms(MS v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MS other;
        other.m = __shfl_xor_sync(0xffffffffu, v.m, o);
        other.s = __shfl_xor_sync(0xffffffffu, v.s, o);
        v = ms_merge(v, other);
    }
    return v;
}

#endif  // __CUDACC__

}  // namespace spr
