// Kernel parameter blocks and host-side launchers shared by the C-ABI layer.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace spr {

struct SdParams {
    const void *p;  // [B,Kp,ldv]
    const void *q;  // [B,K,ldv]
    int64_t ldv;
    int V, K, Kp, chunks;   // chunks = segments (CTAs) per row
    int iters;              // warp steps each warp of a CTA takes (1, 2 or 4)
    const int32_t *draft_tokens;  // [B,K]
    const float *uniforms;        // [B,K+1]
    // outputs
    int32_t *accepted_len;  // [B]
    uint8_t *accept;        // [B,K] or null
    float *p_tok, *q_tok;   // [B,K] or null
    // workspace
    int *status;
    int *row_counters;  // [B*K]
    int *seq_counters;  // [B]
    uint8_t *acc;       // [B*K]
    float4 *part;       // [B*K*chunks]
    double2 *rowstats;  // [B*K] (max + ln Z) of the p row and of the q row
};

enum { DRAW_REPLACE = 0, DRAW_SD = 1 };

struct DrawParams {
    int kind;
    const void *p;
    const void *q;
    int64_t ldv;
    int V, steps;           // warp steps per row
    int n;                  // draws
    // replace_sample
    int64_t R;
    const int32_t *rows;
    const int32_t *gate;
    int seq_stride;
    // sd_verify correction draw (K also bounds the gate of replace_sample)
    int K, Kp;
    const int32_t *accepted_len;
    const double2 *rowstats;
    const float *uniforms;
    int32_t *tokens;
    float *residual_mass;
    // workspace
    int *status;
    int *counters;   // [n] warp steps finished per draw; zero before and after the launch
    float2 *part;    // [n*steps] (max, weight) of every warp step
};

// Vocabulary-sharded sd_verify (sd_shard.cu): V is the width of this GPU's shard, v0 its
// first column; *_all arrays hold one block per rank, in rank order.
struct ShardStatsParams {
    const void *p;  // [B,Kp,ldv] shard columns
    const void *q;  // [B,K,ldv]
    int64_t ldv;
    int V, v0, K, Kp, chunks, iters;
    int Kr;                       // positions per sequence that get a record (Kp, or K without the bonus row)
    const int32_t *draft_tokens;  // [B,K] global token ids
    float *stats;                 // [B*Kr, 6]
    int *row_counters;            // [B*Kr]
    float4 *part;                 // [B*Kr*chunks]
};

struct ShardDecideParams {
    const float *all_stats;       // [G, B*Kp, 6]
    int G, K, Kp, V;              // V: the whole vocabulary
    const int32_t *draft_tokens;
    const float *uniforms;        // [B,K+1]
    int32_t *accepted_len;        // [B]
    uint8_t *accept;              // [B,K] or null
    float *p_tok, *q_tok;         // [B,K] or null
    int *status;
    uint8_t *acc;                 // [B*K]
    double2 *rowstats;            // [B*Kp] (max + ln Z) of the whole p row and q row
};

struct ShardDrawParams {
    const void *p;
    const void *q;
    int64_t ldv;
    int V, v0, K, Kp, chunks, steps, iters;
    int G, rank;
    const int32_t *accepted_len;
    const float *uniforms;
    const double2 *rowstats;
    double2 *weights;             // [B] this shard's (max, weight); weights pass only
    const double2 *all_weights;   // [G, B]; draw pass only
    const float *all_stats;       // [G, B*Kp, 6]; draw pass only
    int32_t *tokens;              // [B]
    float *residual_mass;         // [B] or null
    int *counters;                // [B]
    float2 *part;                 // [B*steps]
};
cudaError_t launch_shard_stats(const ShardStatsParams &sp, int64_t rows, int dt, cudaStream_t st);
cudaError_t launch_shard_decide(const ShardDecideParams &dp, int B, cudaStream_t st);
// dec != null: the decision pass runs inside the weights kernel
cudaError_t launch_shard_weights(const ShardDrawParams &dp, const ShardDecideParams *dec, int B, int dt,
                                 cudaStream_t st);
cudaError_t launch_shard_draw(const ShardDrawParams &dp, int B, int dt, cudaStream_t st);

struct VerifyParams {
    const void *hidden;  // [M,d]
    const void *W1;      // [h,d] (or [d] when h == 0)
    const float *b1;
    const void *W2;
    const float *b2;
    float threshold;
    int B, K, d, h;
    float *scores;
    uint8_t *accept;
    int32_t *first_reject;
    int *status;
    int *counter;
    float *part_z;  // [slices*M]
    unsigned long long *zacc;   // [M] when K == 1, else null (see VerifyWs)
    int slices;
    // tensor-core kernel only
    int kb_per;             // 64-element blocks of d each of the CTAs that share a tile takes
    int ring_stages;        // pipeline stages in use
    int recv_dedicated;     // the exchanged accumulator columns have room of their own beside the ring
    int a_box_rows;         // rows of hidden states one copy fetches (the tile height, or fewer for a small batch)
    int cluster_n;          // hidden-unit slices of one token tile per cluster (1, or all of them)
    int final_in_cluster;   // the CTAs of a token tile form one cluster: no tickets, no part_z
    int atomic_finish;      // K = 1, finish through zacc: one 64-bit atomic per token and slice
    uint32_t spin_limit;    // polls after which a bounded wait gives up
    int test_flags;         // VERIFIER_TEST_*
};

// test_flags: the TMA producer issues no copy, so that the first bounded wait runs out
enum { VERIFIER_TEST_NO_LOADS = 1 };

// Tile shape of the tensor-core verifier; zeros = chosen from the problem size.
struct VerifierTune {
    int bm, bn;         // tokens x hidden units per tile: 64 or 128 each
    int splits;         // CTAs sharing a tile along d: 1, 2, 4 or 8
    int cluster_n;      // 0: automatic; 1: one slice per cluster; -1: all slices of a tile in one cluster
    int test_flags;
    uint32_t spin_limit;   // 0: default
};

struct SimParams {
    uint64_t seed;
    int64_t first_run, runs;
    int r, max_tokens;
    float eta_tp, eta_fp;
    int32_t *n_accepted;              // [runs] or null
    unsigned long long *histogram;    // [max_tokens + 1] or null
};
cudaError_t launch_simulate(const SimParams &sp, cudaStream_t st);

cudaError_t launch_sd_row_stats(const SdParams &sp, int B, int K, int dt, cudaStream_t st);
// kernels that launch_sd_row_stats starts for this shape: 1, or 2 (statistics grid + finish grid)
int sd_row_stats_launches(int B, int K, int chunks, int iters);
int report_cuda_error(cudaError_t e);  // records the text, returns SPR_ERR_CUDA
int device_supported();                // SPR_OK on a compute-capability-10 device
void set_stage_events(cudaEvent_t before, cudaEvent_t after);
// everything of a replacement draw except the scratch pointers (status, counters, part)
DrawParams replace_params(const void *target_logits, int64_t ldv, int V, int64_t R, const int32_t *rows,
                          const int32_t *first_reject, int K, int seq_stride, int n, const float *uniforms,
                          int dt, int32_t *tokens);
// after_kernel: the launch directly follows, in the same stream, the kernel whose output
// selects the rows (programmatic dependent launch)
cudaError_t launch_draw(const DrawParams &dp, int dt, cudaStream_t st, bool after_kernel = false);

// SIMT verifier: any dtype and shape.  `slices` must equal verifier_simt_slices(h).
int verifier_simt_slices(int h);
cudaError_t launch_verifier_simt(const VerifyParams &vp, int dt, cudaStream_t st);

// Tensor-core (tcgen05) verifier for bf16 MLPs.  Returns 0 when launched, a negative
// value when it does not take this shape or dtype (nothing launched), or a positive
// cudaError_t.  It sets the slice count itself.  Batches of fewer than min_tokens tokens
// are left to the SIMT kernel.  tune (may be null) forces the tile shape: a shape that cannot
// be used for this problem gives a negative value.
int launch_verifier_tensor(const VerifyParams &vp, int dt, int min_tokens, const VerifierTune *tune,
                           cudaStream_t st);
// most partial sums per token the tensor-core kernel may write for h hidden units
int verifier_tensor_max_slices(int h);

}  // namespace spr
