// C ABI of libsprinter: host-side argument validation, workspace carving, launches.
#include <stdio.h>
#include <string.h>

#include <atomic>

#include "common.cuh"
#include "host_util.h"
#include "launch.h"

using namespace spr;

namespace {

thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e)
{
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return SPR_ERR_CUDA;
}
}  // namespace

namespace spr {
int report_cuda_error(cudaError_t e) { return cuda_fail(e); }
}  // namespace spr
namespace {
int check_device();
}
namespace spr {
int device_supported() { return check_device(); }
}  // namespace spr

namespace {

// compute capability 10.x only; the answer is cached per device ordinal
int check_device()
{
    static std::atomic<int> cached[64];  // 0 unknown, 1 ok, 2 unsupported (racing threads store the same value)
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev >= 0 && dev < 64) {
        const int known = cached[dev].load(std::memory_order_relaxed);
        if (known) return known == 1 ? SPR_OK : SPR_ERR_UNSUPPORTED;
    }
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev >= 0 && dev < 64) cached[dev].store(major == 10 ? 1 : 2, std::memory_order_relaxed);
    return major == 10 ? SPR_OK : SPR_ERR_UNSUPPORTED;
}

// AUTO hands batches of at least this many tokens to the tensor-core verifier: with d split
// over the CTAs of a cluster it is the faster kernel even for a single token
constexpr int kTensorMinTokens = 1;

// row indices are 32-bit inside the kernels; leave room for the padding of the last step
constexpr int kMaxVocab = 1 << 30;


// tensor-core kernel where it applies (or is forced), SIMT kernel otherwise
int launch_verifier(VerifyParams &vp, int dt, int path, cudaStream_t st, const VerifierTune *tune = nullptr)
{
    if (path != SPR_VERIFIER_SIMT) {
        const int min_tokens = path == SPR_VERIFIER_TENSOR ? 1 : kTensorMinTokens;
        const int tensor_rc = launch_verifier_tensor(vp, dt, min_tokens, tune, st);  // < 0: shape not taken
        if (tensor_rc == 0) return SPR_OK;
        if (tensor_rc > 0) return cuda_fail((cudaError_t)tensor_rc);
        if (path == SPR_VERIFIER_TENSOR) return SPR_ERR_UNSUPPORTED;
    }
    vp.slices = verifier_simt_slices(vp.h);
    cudaError_t e = launch_verifier_simt(vp, dt, st);
    return e == cudaSuccess ? SPR_OK : cuda_fail(e);
}

VerifyParams verify_params(const void *hidden, const void *W1, const float *b1, const void *W2, const float *b2,
                           float threshold, int B, int K, int d, int h, float *scores, uint8_t *accept,
                           int32_t *first_reject)
{
    VerifyParams vp;
    memset(&vp, 0, sizeof vp);
    vp.hidden = hidden;
    vp.W1 = W1;
    vp.b1 = b1;
    vp.W2 = W2;
    vp.b2 = b2;
    vp.threshold = threshold;
    vp.B = B;
    vp.K = K;
    vp.d = d;
    vp.h = h;
    vp.scores = scores;
    vp.accept = accept;
    vp.first_reject = first_reject;
    return vp;
}

// sizes first (an empty batch may come with null pointers), then pointers and alignment
int check_verify_args(const VerifyParams &vp, int dt, int path)
{
    if (!dtype_ok(dt)) return SPR_ERR_UNSUPPORTED;
    if (path != SPR_VERIFIER_AUTO && path != SPR_VERIFIER_SIMT && path != SPR_VERIFIER_TENSOR)
        return SPR_ERR_UNSUPPORTED;
    if (vp.B < 0 || vp.K <= 0 || vp.d <= 0 || vp.h < 0 || (int64_t)vp.B * vp.K > 0x7fffffff)
        return SPR_ERR_INVALID_ARG;
    if (vp.B == 0) return SPR_OK;
    if (!vp.hidden || !vp.W1 || !vp.b2 || !vp.accept || !vp.first_reject) return SPR_ERR_INVALID_ARG;
    if (vp.h > 0 && (!vp.b1 || !vp.W2)) return SPR_ERR_INVALID_ARG;
    const size_t es = elem_size(dt);
    if (!aligned(vp.hidden, es) || !aligned(vp.W1, es) || (vp.W2 && !aligned(vp.W2, es)) || !aligned(vp.b2, 4) ||
        (vp.b1 && !aligned(vp.b1, 4)) || (vp.scores && !aligned(vp.scores, 4)) || !aligned(vp.first_reject, 4))
        return SPR_ERR_INVALID_ARG;
    return SPR_OK;
}

int check_replace_args(const DrawParams &dp, int n, int dt)
{
    if (!dtype_ok(dt)) return SPR_ERR_UNSUPPORTED;
    if (dp.V <= 0 || dp.V > kMaxVocab || dp.ldv < dp.V || dp.R < 0 || n < 0 || dp.seq_stride < 0)
        return SPR_ERR_INVALID_ARG;
    if (n == 0) return SPR_OK;
    if (!dp.p || !dp.uniforms || !dp.tokens || dp.R == 0) return SPR_ERR_INVALID_ARG;
    if (dp.gate && dp.K <= 0) return SPR_ERR_INVALID_ARG;
    // rows i*seq_stride + first_reject[i] of neighbouring sequences must not overlap
    if (dp.gate && !dp.rows && n > 1 && dp.seq_stride < dp.K) return SPR_ERR_INVALID_ARG;
    if (!aligned(dp.p, elem_size(dt)) || !aligned(dp.uniforms, 4) || !aligned(dp.tokens, 4) ||
        (dp.rows && !aligned(dp.rows, 4)) || (dp.gate && !aligned(dp.gate, 4)))
        return SPR_ERR_INVALID_ARG;
    return SPR_OK;
}

}  // namespace

namespace spr {
// everything of a replacement draw except the scratch pointers
DrawParams replace_params(const void *target_logits, int64_t ldv, int V, int64_t R, const int32_t *rows,
                          const int32_t *first_reject, int K, int seq_stride, int n, const float *uniforms,
                          int dt, int32_t *tokens)
{
    DrawParams dp;
    memset(&dp, 0, sizeof dp);
    dp.kind = DRAW_REPLACE;
    dp.p = target_logits;
    dp.ldv = ldv;
    dp.V = V;
    dp.R = R;
    dp.rows = rows;
    dp.gate = first_reject;
    dp.seq_stride = seq_stride;
    dp.K = K;
    dp.uniforms = uniforms;
    dp.tokens = tokens;
    dp.n = n;
    if (V > 0 && dtype_ok(dt)) dp.steps = stat_steps_per_row(V, dt);
    return dp;
}
}  // namespace spr

namespace {

// ticket counters of the verifier kernels: one per 64-token tile (MLP) or per sequence (linear)
int verify_counters(int B, int K) { return max((B * K + 63) / 64, B); }

// number of partial sums per token any of the verifier kernels may write for this shape
int verify_slices(int h) { return max(verifier_simt_slices(h), verifier_tensor_max_slices(h)); }

}  // namespace

extern "C" {

size_t spr_workspace_bytes(int op, int B, int K, int V, int d, int h, int dt)
{
    if (!dtype_ok(dt) || B < 0) return 0;
    switch (op) {
    case SPR_OP_SPRINTER_VERIFY:
        if (K <= 0 || d <= 0 || h < 0 || (int64_t)B * K > 0x7fffffff) return 0;
        return ws_bytes_of([&](Carver &c) { verify_ws_layout(c, B * K, K, verify_slices(h), verify_counters(B, K)); });
    case SPR_OP_REPLACE_SAMPLE:
        if (V <= 0) return 0;
        return ws_bytes_of([&](Carver &c) { draw_ws_layout(c, B, stat_steps_per_row(V, dt)); });
    case SPR_OP_SPRINTER_STEP:
        if (K <= 0 || d <= 0 || h < 0 || V <= 0 || (int64_t)B * K > 0x7fffffff) return 0;
        return ws_bytes_of([&](Carver &c) {
            step_ws_layout(c, B, K, verify_slices(h), verify_counters(B, K), stat_steps_per_row(V, dt));
        });
    case SPR_OP_SD_VERIFY:
        if (K <= 0 || V <= 0 || (int64_t)B * K > 0x7fffffff) return 0;
        return ws_bytes_of([&](Carver &c) {
            sd_ws_layout(c, B, K, stat_max_segments_per_row(V, dt), stat_steps_per_row(V, dt));
        });
    case SPR_OP_SD_SHARD:   // V = shard width; sized for a bonus row
        if (K <= 0 || V <= 0 || (int64_t)B * (K + 1) > 0x7fffffff) return 0;
        return ws_bytes_of([&](Carver &c) {
            shard_ws_layout(c, B, K, K + 1, stat_max_segments_per_row(V, dt), stat_steps_per_row(V, dt));
        });
    case SPR_OP_VERIFIER_LABELS:
        if (K <= 0 || V <= 0 || (int64_t)B * K > 0x7fffffff) return 0;
        return ws_bytes_of([&](Carver &c) { label_ws_layout(c, B, K, stat_max_segments_per_row(V, dt)); });
    case SPR_OP_VERIFIER_TRAIN:
        if (d <= 0) return 0;
        return ws_bytes_of([&](Carver &c) { train_ws_layout(c, d); });
    default:
        return 0;
    }
}

int spr_workspace_init(void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!ws || !aligned(ws, 256) || ws_bytes < (size_t)kHeaderBytes) return SPR_ERR_WORKSPACE;
    cudaError_t e = cudaMemsetAsync(ws, 0, ws_bytes, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? SPR_OK : cuda_fail(e);
}

int sprinter_verify(const void *hidden, const void *W1, const float *b1, const void *W2,
                    const float *b2, float threshold, int B, int K, int d, int h, int dt, int path,
                    float *scores, uint8_t *accept, int32_t *first_reject, void *ws, size_t ws_bytes,
                    void *cuda_stream)
{
    VerifyParams vp = verify_params(hidden, W1, b1, W2, b2, threshold, B, K, d, h, scores, accept, first_reject);
    int rc = check_verify_args(vp, dt, path);
    if (rc != SPR_OK || B == 0) return rc;  // empty batch: nothing to read or write
    Carver cv = carve(ws_bytes);
    const VerifyWs lay = verify_ws_layout(cv, B * K, K, verify_slices(h), verify_counters(B, K));
    if (!ws || !aligned(ws, 256) || !cv.fits()) return SPR_ERR_WORKSPACE;
    if ((rc = check_device()) != SPR_OK) return rc;

    vp.status = at<int>(ws, 0);
    vp.counter = at<int>(ws, lay.counter);
    vp.part_z = at<float>(ws, lay.part_z);
    vp.zacc = K == 1 ? at<unsigned long long>(ws, lay.zacc) : nullptr;
    return launch_verifier(vp, dt, path, static_cast<cudaStream_t>(cuda_stream));
}

int spr_test_sprinter_verify(const void *hidden, const void *W1, const float *b1, const void *W2,
                             const float *b2, float threshold, int B, int K, int d, int h, int dt,
                             float *scores, uint8_t *accept, int32_t *first_reject, void *ws, size_t ws_bytes,
                             void *cuda_stream, int bm, int bn, int splits, int cluster_n, int flags,
                             unsigned spin_limit)
{
    VerifyParams vp = verify_params(hidden, W1, b1, W2, b2, threshold, B, K, d, h, scores, accept, first_reject);
    int rc = check_verify_args(vp, dt, SPR_VERIFIER_TENSOR);
    if (rc != SPR_OK || B == 0) return rc;
    Carver cv = carve(ws_bytes);
    const VerifyWs lay = verify_ws_layout(cv, B * K, K, verify_slices(h), verify_counters(B, K));
    if (!ws || !aligned(ws, 256) || !cv.fits()) return SPR_ERR_WORKSPACE;
    if ((rc = check_device()) != SPR_OK) return rc;
    VerifierTune tune = {bm, bn, splits, cluster_n, flags, spin_limit};
    vp.status = at<int>(ws, 0);
    vp.counter = at<int>(ws, lay.counter);
    vp.part_z = at<float>(ws, lay.part_z);
    vp.zacc = K == 1 ? at<unsigned long long>(ws, lay.zacc) : nullptr;
    return launch_verifier(vp, dt, SPR_VERIFIER_TENSOR, static_cast<cudaStream_t>(cuda_stream), &tune);
}

int replace_sample(const void *target_logits, int64_t ldv, int V, int64_t R, const int32_t *rows,
                   const int32_t *first_reject, int K, int seq_stride, int n, const float *uniforms,
                   int dt, int32_t *tokens, void *ws, size_t ws_bytes, void *cuda_stream)
{
    DrawParams dp = replace_params(target_logits, ldv, V, R, rows, first_reject, K, seq_stride, n, uniforms, dt,
                                   tokens);
    int rc = check_replace_args(dp, n, dt);
    if (rc != SPR_OK || n == 0) return rc;  // no draws: pointers may be null
    Carver cv = carve(ws_bytes);
    const DrawWs lay = draw_ws_layout(cv, n, dp.steps);
    if (!ws || !aligned(ws, 256) || !cv.fits()) return SPR_ERR_WORKSPACE;
    if ((rc = check_device()) != SPR_OK) return rc;

    dp.status = at<int>(ws, 0);
    dp.counters = at<int>(ws, lay.counters);
    dp.part = at<float2>(ws, lay.part);
    const cudaError_t e = launch_draw(dp, dt, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? SPR_OK : cuda_fail(e);
}

int sprinter_step(const void *hidden, const void *W1, const float *b1, const void *W2, const float *b2,
                  float threshold, int B, int K, int d, int h, const void *target_logits, int64_t ldv,
                  int V, int seq_stride, const float *uniforms, int dt, int path, float *scores,
                  uint8_t *accept, int32_t *first_reject, int32_t *tokens, void *ws, size_t ws_bytes,
                  void *cuda_stream)
{
    VerifyParams vp = verify_params(hidden, W1, b1, W2, b2, threshold, B, K, d, h, scores, accept, first_reject);
    int rc = check_verify_args(vp, dt, path);
    if (rc != SPR_OK) return rc;
    if (seq_stride < K) return SPR_ERR_INVALID_ARG;
    DrawParams dp = replace_params(target_logits, ldv, V, (int64_t)B * seq_stride, nullptr, first_reject, K,
                                   seq_stride, B, uniforms, dt, tokens);
    rc = check_replace_args(dp, B, dt);
    if (rc != SPR_OK || B == 0) return rc;
    Carver cv = carve(ws_bytes);
    const StepWs lay = step_ws_layout(cv, B, K, verify_slices(h), verify_counters(B, K), dp.steps);
    if (!ws || !aligned(ws, 256) || !cv.fits()) return SPR_ERR_WORKSPACE;
    if ((rc = check_device()) != SPR_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    vp.status = dp.status = at<int>(ws, 0);
    vp.counter = at<int>(ws, lay.verify.counter);
    vp.part_z = at<float>(ws, lay.verify.part_z);
    vp.zacc = K == 1 ? at<unsigned long long>(ws, lay.verify.zacc) : nullptr;
    dp.counters = at<int>(ws, lay.draw.counters);
    dp.part = at<float2>(ws, lay.draw.part);
    // The draw is launched behind the verifier; programmatically (its launch overlapping the
    // verifier's tail) only for small batches: measured, that gains a few tenths of a
    // microsecond there and costs 1.5-2.5 us once the verifier's grid fills the GPU.
    if ((rc = launch_verifier(vp, dt, path, st)) != SPR_OK) return rc;
    const cudaError_t e = launch_draw(dp, dt, st, /*after_kernel=*/(int64_t)B * K <= 128);
    return e == cudaSuccess ? SPR_OK : cuda_fail(e);
}

int sd_verify(const void *p_logits, const void *q_logits, int64_t ldv, const int32_t *draft_tokens,
              const float *uniforms, int B, int K, int Kp, int V, int dt, int32_t *accepted_len,
              int32_t *correction_token, uint8_t *accept, float *p_tok, float *q_tok,
              float *residual_mass, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!dtype_ok(dt)) return SPR_ERR_UNSUPPORTED;
    if (B < 0 || K <= 0 || V <= 0 || V > kMaxVocab || ldv < V || (Kp != K && Kp != K + 1) ||
        (int64_t)B * K > 0x7fffffff)
        return SPR_ERR_INVALID_ARG;
    if (B == 0) return SPR_OK;  // empty batch: pointers may be null
    if (!p_logits || !q_logits || !draft_tokens || !uniforms || !accepted_len || !correction_token)
        return SPR_ERR_INVALID_ARG;
    const size_t es = elem_size(dt);
    if (!aligned(p_logits, es) || !aligned(q_logits, es) || !aligned(draft_tokens, 4) ||
        !aligned(uniforms, 4) || !aligned(accepted_len, 4) || !aligned(correction_token, 4) ||
        (p_tok && !aligned(p_tok, 4)) || (q_tok && !aligned(q_tok, 4)) ||
        (residual_mass && !aligned(residual_mass, 4)))
        return SPR_ERR_INVALID_ARG;
    const int T = stat_steps_per_row(V, dt);
    int C, stat_iters;
    draw_geometry(B * K, T, &C, &stat_iters);   // same rule for the row-statistics pass, over B*K rows
    Carver cv = carve(ws_bytes);
    const SdWs lay = sd_ws_layout(cv, B, K, stat_max_segments_per_row(V, dt), T);
    if (!ws || !aligned(ws, 256) || !cv.fits()) return SPR_ERR_WORKSPACE;
    int rc = check_device();
    if (rc != SPR_OK) return rc;
    if (B == 0) return SPR_OK;

    SdParams sp;
    memset(&sp, 0, sizeof sp);
    sp.p = p_logits;
    sp.q = q_logits;
    sp.ldv = ldv;
    sp.V = V;
    sp.K = K;
    sp.Kp = Kp;
    sp.chunks = C;
    sp.iters = stat_iters;
    sp.draft_tokens = draft_tokens;
    sp.uniforms = uniforms;
    sp.accepted_len = accepted_len;
    sp.accept = accept;
    sp.p_tok = p_tok;
    sp.q_tok = q_tok;
    sp.status = at<int>(ws, 0);
    sp.row_counters = at<int>(ws, lay.row_counters);
    sp.seq_counters = at<int>(ws, lay.seq_counters);
    sp.acc = at<uint8_t>(ws, lay.acc);
    sp.part = at<float4>(ws, lay.part);
    sp.rowstats = at<double2>(ws, lay.rowstats);

    DrawParams dp;
    memset(&dp, 0, sizeof dp);
    dp.kind = DRAW_SD;
    dp.p = p_logits;
    dp.q = q_logits;
    dp.ldv = ldv;
    dp.V = V;
    dp.n = B;
    dp.K = K;
    dp.Kp = Kp;
    dp.accepted_len = accepted_len;
    dp.rowstats = sp.rowstats;
    dp.uniforms = uniforms;
    dp.tokens = correction_token;
    dp.residual_mass = residual_mass;
    dp.status = sp.status;
    dp.counters = at<int>(ws, lay.draw.counters);
    dp.steps = T;
    dp.part = at<float2>(ws, lay.draw.part);

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = launch_sd_row_stats(sp, B, K, dt, st);
    if (e == cudaSuccess) e = launch_draw(dp, dt, st, /*after_kernel=*/true);
    return e == cudaSuccess ? SPR_OK : cuda_fail(e);
}

int sprinter_simulate(uint64_t seed, int64_t first_run, int64_t runs, int r, float eta_tp, float eta_fp,
                      int max_tokens, int32_t *n_accepted, uint64_t *histogram, void *cuda_stream)
{
    if (runs < 0 || first_run < 0 || r < 0 || max_tokens < 0 || (!n_accepted && !histogram))
        return SPR_ERR_INVALID_ARG;
    if (!(eta_tp >= 0.f && eta_tp <= 1.f) || !(eta_fp >= 0.f && eta_fp <= 1.f)) return SPR_ERR_INVALID_ARG;
    if ((n_accepted && !aligned(n_accepted, 4)) || (histogram && !aligned(histogram, 8)))
        return SPR_ERR_INVALID_ARG;
    int rc = check_device();
    if (rc != SPR_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (histogram) {
        cudaError_t e = cudaMemsetAsync(histogram, 0, sizeof(uint64_t) * ((size_t)max_tokens + 1), st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    SimParams sp;
    sp.seed = seed;
    sp.first_run = first_run;
    sp.runs = runs;
    sp.r = r;
    sp.max_tokens = max_tokens;
    sp.eta_tp = eta_tp;
    sp.eta_fp = eta_fp;
    sp.n_accepted = n_accepted;
    sp.histogram = reinterpret_cast<unsigned long long *>(histogram);
    cudaError_t e = launch_simulate(sp, st);
    return e == cudaSuccess ? SPR_OK : cuda_fail(e);
}

int spr_device_status(void *ws, void *cuda_stream)
{
    if (!ws) return SPR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof word, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (word != 0) {
        e = cudaMemsetAsync(ws, 0, sizeof word, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return word;
}

const char *spr_status_string(int status)
{
    switch (status) {
    case SPR_OK: return "ok";
    case SPR_ERR_INVALID_ARG: return "invalid argument";
    case SPR_ERR_UNSUPPORTED: return "unsupported dtype, op, path or device";
    case SPR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SPR_ERR_CUDA: return "CUDA runtime error";
    case SPR_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
    case SPR_ERR_BAD_TOKEN: return "draft token id outside the vocabulary";
    case SPR_ERR_BAD_ROW: return "logits row index outside the tensor";
    default: return "unknown status";
    }
}

const char *spr_last_cuda_error(void) { return g_cuda_error; }

void spr_set_stage_events(void *before, void *after)
{
    set_stage_events(static_cast<cudaEvent_t>(before), static_cast<cudaEvent_t>(after));
}

int spr_sd_verify_launches(int B, int K, int V, int dt)
{
    if (!dtype_ok(dt) || B <= 0 || K <= 0 || V <= 0 || (int64_t)B * K > 0x7fffffff) return 0;
    int C, iters;
    draw_geometry(B * K, stat_steps_per_row(V, dt), &C, &iters);
    return sd_row_stats_launches(B, K, C, iters) + 1;   // + the correction draw
}

int spr_version(void) { return 100; }

}  // extern "C"
