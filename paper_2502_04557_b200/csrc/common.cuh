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
// A workspace of ws_bytes bytes is cut at a point that depends on ws_bytes alone:
//   [0, 256)                   header; word 0 is the sticky status
//   [256, 256 + Z)             ticket zone, Z = ticket_zone_bytes(ws_bytes): int32 counters only
//   [256 + Z, ws_bytes)        data zone: partial results, flags, everything else
// The kernels of sprinter_verify, replace_sample, sprinter_step and sd_verify take tickets from
// the ticket zone, and whoever takes the last ticket of a counter sets it back to zero
// (take_ticket below).  The zone is zero after spr_workspace_init and no call ever writes
// anything but tickets into it, so it is zero again whenever no call is in flight: these calls
// need no clearing pass, whatever ops and shapes the workspace served before.  The remaining
// ops keep their counters in the data zone and clear them on the stream at every call.
__host__ __device__ inline size_t ticket_zone_bytes(size_t ws_bytes)
{
    return ws_bytes <= (size_t)kHeaderBytes ? 0 : (ws_bytes - kHeaderBytes) / 4 / 256 * 256;
}
__host__ __device__ inline size_t data_zone_start(size_t ws_bytes) { return kHeaderBytes + ticket_zone_bytes(ws_bytes); }
// smallest workspace whose zones hold `tickets` bytes of counters and `data` bytes of the rest
__host__ __device__ inline size_t ws_bytes_for(size_t tickets, size_t data)
{
    const size_t a = align_up(tickets, 256), b = align_up((align_up(data, 256) + 2) / 3, 256);
    return kHeaderBytes + 4 * (a > b ? a : b);
}

// Cursor over the two zones.  Offsets are from the start of the workspace.
struct Carver {
    size_t tickets, data;        // next free byte of each zone
    size_t tickets_end, data_end;
    __host__ __device__ size_t take_tickets(size_t n)   // n int32 counters
    {
        const size_t o = tickets;
        tickets += 4 * n;
        return o;
    }
    __host__ __device__ size_t take_data(size_t bytes)  // 256-byte aligned block
    {
        const size_t o = data;
        data = align_up(data + bytes, 256);
        return o;
    }
    __host__ __device__ bool fits() const { return tickets <= tickets_end && data <= data_end; }
};
__host__ __device__ inline Carver carve(size_t ws_bytes)
{
    Carver c;
    c.tickets = kHeaderBytes;
    c.tickets_end = c.data = data_zone_start(ws_bytes);
    c.data_end = ws_bytes;
    return c;
}
// workspace size a layout needs: carve an unbounded workspace, measure both zones
template <typename F>
inline size_t ws_bytes_of(F layout)
{
    Carver c;
    c.tickets = c.data = 0;
    c.tickets_end = c.data_end = ~(size_t)0;
    layout(c);
    return ws_bytes_for(c.tickets, c.data);
}

struct DrawWs {              // replace_sample, and the correction draw of sd_verify
    size_t counters;         // int32 [n]      warp steps finished per draw (ticket zone)
    size_t part;             // float2 [n*T]   (max, weight) of every warp step
};
__host__ __device__ inline DrawWs draw_ws_layout(Carver &c, int n, int T)
{
    DrawWs w;
    w.counters = c.take_tickets((size_t)n);
    w.part = c.take_data(8 * (size_t)n * T);
    return w;
}

struct SdWs {
    size_t row_counters;     // int32 [M]      segments finished per row (ticket zone)
    size_t seq_counters;     // int32 [B]      rows finished per sequence (ticket zone)
    size_t acc;              // uint8 [M]      0 reject, 1 accept, 2 invalid token
    size_t part;             // float4 [M*S]   (max_p, sum_p, max_q, sum_q) per row segment
    size_t rowstats;         // double2 [M]    (max + ln Z) of the p row and of the q row
    DrawWs draw;             // correction draw, n = B
};
__host__ __device__ inline SdWs sd_ws_layout(Carver &c, int B, int K, int S, int T)   // S segments, T steps per row
{
    const size_t M = (size_t)B * K;
    SdWs w;
    w.row_counters = c.take_tickets(M);
    w.seq_counters = c.take_tickets((size_t)B);
    w.acc = c.take_data(M);
    w.part = c.take_data(16 * M * S);
    w.rowstats = c.take_data(16 * M);
    w.draw = draw_ws_layout(c, B, T);
    return w;
}

struct ShardWs {             // vocabulary-sharded sd_verify: the four passes share one workspace
    size_t row_counters;     // int32 [B*Kp]   (data zone, cleared per call)
    size_t draw_counters;    // int32 [B]      (data zone, cleared per call)
    size_t acc;              // uint8 [B*K]
    size_t part;             // float4 [B*Kp*S]
    size_t rowstats;         // double2 [B*Kp] whole-row (max + ln Z) of p and of q
    size_t draw_part;        // float2 [B*T]
};
__host__ __device__ inline ShardWs shard_ws_layout(Carver &c, int B, int K, int Kp, int S, int T)
{
    const size_t R = (size_t)B * Kp;
    ShardWs w;
    w.row_counters = c.take_data(4 * R);
    w.draw_counters = c.take_data(4 * (size_t)B);
    w.acc = c.take_data((size_t)B * K);
    w.part = c.take_data(16 * R * S);
    w.rowstats = c.take_data(16 * R);
    w.draw_part = c.take_data(8 * (size_t)B * T);
    return w;
}

struct LabelWs {             // verifier_labels: row records of the statistics pass
    size_t row_counters;     // int32 [M]      (data zone, cleared per call)
    size_t part;             // float4 [M*S]
    size_t stats;            // float [M*6]
};
__host__ __device__ inline LabelWs label_ws_layout(Carver &c, int B, int K, int S)
{
    const size_t M = (size_t)B * K;
    LabelWs w;
    w.row_counters = c.take_data(4 * M);
    w.part = c.take_data(16 * M * S);
    w.stats = c.take_data(24 * M);
    return w;
}

// verifier_train_step: per-CTA gradient sums, float [kTrainMaxCtas, d + 2] (data zone)
constexpr int kTrainMaxCtas = 592;   // 148 SMs x 4
__host__ __device__ inline size_t train_ws_layout(Carver &c, int d)
{
    return c.take_data(4 * (size_t)kTrainMaxCtas * ((size_t)d + 2));
}

struct VerifyWs {
    size_t zacc;             // uint64 [M], K = 1 only (ticket zone, first: 8-byte aligned): per-token sum of
                             //   partial logits in fixed point with an arrival count; zero between launches
    size_t counter;          // int32 [1 + tickets]   (ticket zone) see verify_tickets()
    size_t part_z;           // float [slices * M]    per-slice partial of W2 . relu(...)
};
__host__ __device__ inline VerifyWs verify_ws_layout(Carver &c, int M, int K, int slices, int tickets)
{
    VerifyWs w;
    w.zacc = K == 1 ? c.take_tickets(2 * (size_t)M) : 0;
    w.counter = c.take_tickets(1 + (size_t)tickets);
    w.part_z = c.take_data(4 * (size_t)slices * M);
    return w;
}

struct StepWs {              // sprinter_step: verifier and replacement draw in one call
    VerifyWs verify;
    DrawWs draw;
};
__host__ __device__ inline StepWs step_ws_layout(Carver &c, int B, int K, int slices, int tickets, int T)
{
    StepWs w;
    w.verify = verify_ws_layout(c, B * K, K, slices, tickets);
    w.draw = draw_ws_layout(c, B, T);
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

// One ticket of a counter that `total` parties take; true for whoever takes the last one, who
// also sets the counter back to zero so that the next launch finds it clean.  The caller orders
// its earlier global writes before the ticket (__threadfence) and its later reads after it.
__device__ __forceinline__ bool take_ticket(int *counter, int total, int n = 1)
{
    const int old = atomicAdd(counter, n);
    if (old + n != total) return false;
    *reinterpret_cast<volatile int *>(counter) = 0;
    return true;
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
