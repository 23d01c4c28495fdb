// C ABI of the vocabulary-sharded sd_verify: argument validation, workspace carving, launches.
#include <string.h>

#include "common.cuh"
#include "host_util.h"
#include "launch.h"

using namespace spr;

namespace {

constexpr int kMaxVocab = 1 << 30;
constexpr int kMaxRanks = 1024;


constexpr int kProceed = -1;   // not a status: the arguments are fine and there is work to do

// sizes shared by the passes; kProceed, or the status to return
int check_sizes(int B, int K, int Kp, int Vs, int64_t ldv, int dt)
{
    if (!dtype_ok(dt)) return SPR_ERR_UNSUPPORTED;
    if (B < 0 || K <= 0 || Vs <= 0 || Vs > kMaxVocab || ldv < Vs || (Kp != K && Kp != K + 1) ||
        (int64_t)B * Kp > 0x7fffffff)
        return SPR_ERR_INVALID_ARG;
    return B == 0 ? SPR_OK : kProceed;
}

// the layout inside a workspace of ws_bytes bytes; *fits tells whether it has room
ShardWs layout(int B, int K, int Kp, int Vs, int dt, size_t ws_bytes, bool *fits)
{
    Carver cv = carve(ws_bytes);
    const ShardWs lay = shard_ws_layout(cv, B, K, Kp, stat_max_segments_per_row(Vs, dt), stat_steps_per_row(Vs, dt));
    *fits = cv.fits();
    return lay;
}

bool ws_ok(const void *ws, bool fits) { return ws && aligned(ws, 256) && fits; }

}  // namespace

extern "C" {

int sd_shard_stats(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, int v0,
                   const int32_t *draft_tokens, int B, int K, int Kp, int dt, float *stats, void *ws,
                   size_t ws_bytes, void *cuda_stream)
{
    int rc = check_sizes(B, K, Kp, Vs, ldv, dt);
    if (rc != kProceed) return rc;
    if (v0 < 0 || !p_shard || !q_shard || !draft_tokens || !stats) return SPR_ERR_INVALID_ARG;
    const size_t es = elem_size(dt);
    if (!aligned(p_shard, es) || !aligned(q_shard, es) || !aligned(draft_tokens, 4) || !aligned(stats, 4))
        return SPR_ERR_INVALID_ARG;
    bool fits;
    const ShardWs lay = layout(B, K, Kp, Vs, dt, ws_bytes, &fits);
    if (!ws_ok(ws, fits)) return SPR_ERR_WORKSPACE;
    if ((rc = device_supported()) != SPR_OK) return rc;

    ShardStatsParams sp;
    memset(&sp, 0, sizeof sp);
    sp.p = p_shard;
    sp.q = q_shard;
    sp.ldv = ldv;
    sp.V = Vs;
    sp.v0 = v0;
    sp.K = K;
    sp.Kp = Kp;
    sp.Kr = Kp;
    draw_geometry(B * Kp, stat_steps_per_row(Vs, dt), &sp.chunks, &sp.iters);
    sp.draft_tokens = draft_tokens;
    sp.stats = stats;
    sp.row_counters = at<int>(ws, lay.row_counters);
    sp.part = at<float4>(ws, lay.part);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(sp.row_counters, 0, sizeof(int) * (size_t)B * Kp, st);
    if (e == cudaSuccess) e = launch_shard_stats(sp, (int64_t)B * Kp, dt, st);
    return finish(e);
}

namespace {
// validation and parameters of the decision pass; kProceed, or the status to return
int decide_params(ShardDecideParams &dp, const float *all_stats, int G, const int32_t *draft_tokens,
                  const float *uniforms, int B, int K, int Kp, int V, int Vs, int dt, int32_t *accepted_len,
                  uint8_t *accept, float *p_tok, float *q_tok, void *ws, size_t ws_bytes)
{
    int rc = check_sizes(B, K, Kp, Vs, Vs, dt);
    if (rc != kProceed) return rc;
    if (G <= 0 || G > kMaxRanks || V <= 0 || V > kMaxVocab) return SPR_ERR_INVALID_ARG;
    if (!all_stats || !draft_tokens || !uniforms || !accepted_len) return SPR_ERR_INVALID_ARG;
    if (!aligned(all_stats, 4) || !aligned(draft_tokens, 4) || !aligned(uniforms, 4) || !aligned(accepted_len, 4) ||
        (p_tok && !aligned(p_tok, 4)) || (q_tok && !aligned(q_tok, 4)))
        return SPR_ERR_INVALID_ARG;
    bool fits;
    const ShardWs lay = layout(B, K, Kp, Vs, dt, ws_bytes, &fits);
    if (!ws_ok(ws, fits)) return SPR_ERR_WORKSPACE;
    memset(&dp, 0, sizeof dp);
    dp.all_stats = all_stats;
    dp.G = G;
    dp.K = K;
    dp.Kp = Kp;
    dp.V = V;
    dp.draft_tokens = draft_tokens;
    dp.uniforms = uniforms;
    dp.accepted_len = accepted_len;
    dp.accept = accept;
    dp.p_tok = p_tok;
    dp.q_tok = q_tok;
    dp.status = at<int>(ws, 0);
    dp.acc = at<uint8_t>(ws, lay.acc);
    dp.rowstats = at<double2>(ws, lay.rowstats);
    return kProceed;
}
}  // namespace

int sd_shard_decide(const float *all_stats, int G, const int32_t *draft_tokens, const float *uniforms, int B,
                    int K, int Kp, int V, int Vs, int dt, int32_t *accepted_len, uint8_t *accept, float *p_tok,
                    float *q_tok, void *ws, size_t ws_bytes, void *cuda_stream)
{
    ShardDecideParams dp;
    int rc = decide_params(dp, all_stats, G, draft_tokens, uniforms, B, K, Kp, V, Vs, dt, accepted_len, accept,
                           p_tok, q_tok, ws, ws_bytes);
    if (rc != kProceed) return rc;
    if ((rc = device_supported()) != SPR_OK) return rc;
    return finish(launch_shard_decide(dp, B, static_cast<cudaStream_t>(cuda_stream)));
}

namespace {
int draw_params(ShardDrawParams &dp, const void *p_shard, const void *q_shard, int64_t ldv, int Vs, int v0,
                const int32_t *accepted_len, const float *uniforms, int B, int K, int Kp, int dt, void *ws,
                size_t ws_bytes)
{
    int rc = check_sizes(B, K, Kp, Vs, ldv, dt);
    if (rc != kProceed) return rc;
    if (v0 < 0 || !p_shard || !q_shard || !accepted_len || !uniforms) return SPR_ERR_INVALID_ARG;
    const size_t es = elem_size(dt);
    if (!aligned(p_shard, es) || !aligned(q_shard, es) || !aligned(accepted_len, 4) || !aligned(uniforms, 4))
        return SPR_ERR_INVALID_ARG;
    bool fits;
    const ShardWs lay = layout(B, K, Kp, Vs, dt, ws_bytes, &fits);
    if (!ws_ok(ws, fits)) return SPR_ERR_WORKSPACE;
    memset(&dp, 0, sizeof dp);
    dp.p = p_shard;
    dp.q = q_shard;
    dp.ldv = ldv;
    dp.V = Vs;
    dp.v0 = v0;
    dp.K = K;
    dp.Kp = Kp;
    dp.steps = stat_steps_per_row(Vs, dt);
    draw_geometry(B, dp.steps, &dp.chunks, &dp.iters);
    dp.accepted_len = accepted_len;
    dp.uniforms = uniforms;
    dp.rowstats = at<double2>(ws, lay.rowstats);
    dp.counters = at<int>(ws, lay.draw_counters);
    dp.part = at<float2>(ws, lay.draw_part);
    return kProceed;
}
}  // namespace

int sd_shard_weights(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, const int32_t *accepted_len,
                     const float *uniforms, int B, int K, int Kp, int dt, double *weights, void *ws,
                     size_t ws_bytes, void *cuda_stream)
{
    ShardDrawParams dp;
    int rc = draw_params(dp, p_shard, q_shard, ldv, Vs, 0, accepted_len, uniforms, B, K, Kp, dt, ws, ws_bytes);
    if (rc != kProceed) return rc;
    if (!weights || !aligned(weights, 16)) return SPR_ERR_INVALID_ARG;
    if ((rc = device_supported()) != SPR_OK) return rc;
    dp.weights = reinterpret_cast<double2 *>(weights);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(dp.counters, 0, sizeof(int) * (size_t)B, st);
    if (e == cudaSuccess) e = launch_shard_weights(dp, nullptr, B, dt, st);
    return finish(e);
}

int sd_shard_decide_weights(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, const float *all_stats,
                            int G, const int32_t *draft_tokens, const float *uniforms, int B, int K, int Kp, int V,
                            int dt, int32_t *accepted_len, uint8_t *accept, float *p_tok, float *q_tok,
                            double *weights, void *ws, size_t ws_bytes, void *cuda_stream)
{
    ShardDecideParams dec;
    int rc = decide_params(dec, all_stats, G, draft_tokens, uniforms, B, K, Kp, V, Vs, dt, accepted_len, accept,
                           p_tok, q_tok, ws, ws_bytes);
    if (rc != kProceed) return rc;
    ShardDrawParams dp;
    rc = draw_params(dp, p_shard, q_shard, ldv, Vs, 0, accepted_len, uniforms, B, K, Kp, dt, ws, ws_bytes);
    if (rc != kProceed) return rc;
    if (!weights || !aligned(weights, 16)) return SPR_ERR_INVALID_ARG;
    if ((rc = device_supported()) != SPR_OK) return rc;
    dp.weights = reinterpret_cast<double2 *>(weights);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(dp.counters, 0, sizeof(int) * (size_t)B, st);
    if (e == cudaSuccess) e = launch_shard_weights(dp, &dec, B, dt, st);
    return finish(e);
}

int sd_shard_draw(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, int v0, const double *all_weights,
                  const float *all_stats, int G, int rank, const int32_t *accepted_len, const float *uniforms,
                  int B, int K, int Kp, int dt, int32_t *correction_token, float *residual_mass, void *ws,
                  size_t ws_bytes, void *cuda_stream)
{
    ShardDrawParams dp;
    int rc = draw_params(dp, p_shard, q_shard, ldv, Vs, v0, accepted_len, uniforms, B, K, Kp, dt, ws, ws_bytes);
    if (rc != kProceed) return rc;
    if (G <= 0 || G > kMaxRanks || rank < 0 || rank >= G || (int64_t)v0 + Vs > kMaxVocab) return SPR_ERR_INVALID_ARG;
    if (!all_weights || !all_stats || !correction_token || !aligned(all_weights, 16) || !aligned(all_stats, 4) ||
        !aligned(correction_token, 4) || (residual_mass && !aligned(residual_mass, 4)))
        return SPR_ERR_INVALID_ARG;
    if ((rc = device_supported()) != SPR_OK) return rc;
    dp.G = G;
    dp.rank = rank;
    dp.all_weights = reinterpret_cast<const double2 *>(all_weights);
    dp.all_stats = all_stats;
    dp.tokens = correction_token;
    dp.residual_mass = residual_mass;
    return finish(launch_shard_draw(dp, B, dt, static_cast<cudaStream_t>(cuda_stream)));
}

}  // extern "C"
