// Host-buffer variants of the three entry points: copy the inputs to a caller-supplied
// device arena, run the device entry point, copy the results back and synchronise.  Plumbing
// only - every step of the computation runs in the same kernels as the device-pointer calls.
#include <string.h>

#include "common.cuh"
#include "launch.h"

using namespace spr;

namespace {

struct Arena {
    char *base;
    size_t size, used;
    bool dry;  // only measure
    void *take(size_t bytes)
    {
        const size_t off = align_up(used, 256);
        used = off + bytes;
        if (dry || used > size) return nullptr;
        return base + off;
    }
};

size_t esz(int dt) { return dt == SPR_F32 ? 4 : 2; }

struct SdArena {
    void *p, *q, *x, *u, *len, *tok, *acc, *ptok, *qtok, *rm;
};
SdArena carve_sd(Arena &a, int64_t ldv, int B, int K, int Kp, int dt)
{
    SdArena s;
    const size_t M = (size_t)B * K;
    s.p = a.take((size_t)B * Kp * ldv * esz(dt));
    s.q = a.take(M * ldv * esz(dt));
    s.x = a.take(M * 4);
    s.u = a.take((size_t)B * (K + 1) * 4);
    s.len = a.take((size_t)B * 4);
    s.tok = a.take((size_t)B * 4);
    s.acc = a.take(M);
    s.ptok = a.take(M * 4);
    s.qtok = a.take(M * 4);
    s.rm = a.take((size_t)B * 4);
    return s;
}

struct VerifyArena {
    void *hid, *W1, *b1, *W2, *b2, *scores, *acc, *fr;
};
VerifyArena carve_verify(Arena &a, int B, int K, int d, int h, int dt)
{
    VerifyArena v;
    const size_t M = (size_t)B * K;
    v.hid = a.take(M * d * esz(dt));
    v.W1 = a.take((size_t)(h > 0 ? h : 1) * d * esz(dt));
    v.b1 = a.take((size_t)(h > 0 ? h : 1) * 4);
    v.W2 = a.take((size_t)(h > 0 ? h : 1) * esz(dt));
    v.b2 = a.take(4);
    v.scores = a.take(M * 4);
    v.acc = a.take(M);
    v.fr = a.take((size_t)B * 4);
    return v;
}

struct DrawArena {
    void *logits, *u, *tok;
};
DrawArena carve_draw(Arena &a, int64_t ldv, int n, int dt)
{
    DrawArena r;
    r.logits = a.take((size_t)n * ldv * esz(dt));
    r.u = a.take((size_t)n * 4);
    r.tok = a.take((size_t)n * 4);
    return r;
}

#define CK(call)                                           \
    do {                                                   \
        cudaError_t e_ = (call);                           \
        if (e_ != cudaSuccess) return report_cuda_error(e_); \
    } while (0)

}  // namespace

extern "C" {

size_t spr_host_arena_bytes(int op, int B, int K, int Kp, int64_t ldv, int d, int h, int dt)
{
    if ((dt != SPR_F32 && dt != SPR_BF16) || B < 0) return 0;
    Arena a{nullptr, 0, 0, true};
    switch (op) {
    case SPR_OP_SD_VERIFY: carve_sd(a, ldv, B, K, Kp, dt); break;
    case SPR_OP_SPRINTER_VERIFY: carve_verify(a, B, K, d, h, dt); break;
    case SPR_OP_REPLACE_SAMPLE: carve_draw(a, ldv, B, dt); break;
    default: return 0;
    }
    return align_up(a.used, 256);
}

int sd_verify_host(const void *p_logits, const void *q_logits, int64_t ldv, const int32_t *draft_tokens,
                   const float *uniforms, int B, int K, int Kp, int V, int dt, int32_t *accepted_len,
                   int32_t *correction_token, uint8_t *accept, float *p_tok, float *q_tok,
                   float *residual_mass, void *arena, size_t arena_bytes, void *ws, size_t ws_bytes,
                   void *cuda_stream)
{
    if (dt != SPR_F32 && dt != SPR_BF16) return SPR_ERR_UNSUPPORTED;
    if (B < 0 || K <= 0 || V <= 0 || ldv < V || (Kp != K && Kp != K + 1)) return SPR_ERR_INVALID_ARG;
    if (B == 0) return SPR_OK;
    if (!p_logits || !q_logits || !draft_tokens || !uniforms || !accepted_len || !correction_token)
        return SPR_ERR_INVALID_ARG;
    if (!arena || arena_bytes < spr_host_arena_bytes(SPR_OP_SD_VERIFY, B, K, Kp, ldv, 0, 0, dt))
        return SPR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Arena a{static_cast<char *>(arena), arena_bytes, 0, false};
    SdArena s = carve_sd(a, ldv, B, K, Kp, dt);
    const size_t M = (size_t)B * K;
    CK(cudaMemcpyAsync(s.p, p_logits, (size_t)B * Kp * ldv * esz(dt), cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(s.q, q_logits, M * ldv * esz(dt), cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(s.x, draft_tokens, M * 4, cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(s.u, uniforms, (size_t)B * (K + 1) * 4, cudaMemcpyHostToDevice, st));
    int rc = sd_verify(s.p, s.q, ldv, (const int32_t *)s.x, (const float *)s.u, B, K, Kp, V, dt,
                       (int32_t *)s.len, (int32_t *)s.tok, accept ? (uint8_t *)s.acc : nullptr,
                       p_tok ? (float *)s.ptok : nullptr, q_tok ? (float *)s.qtok : nullptr,
                       residual_mass ? (float *)s.rm : nullptr, ws, ws_bytes, cuda_stream);
    if (rc != SPR_OK) return rc;
    CK(cudaMemcpyAsync(accepted_len, s.len, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    CK(cudaMemcpyAsync(correction_token, s.tok, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    if (accept) CK(cudaMemcpyAsync(accept, s.acc, M, cudaMemcpyDeviceToHost, st));
    if (p_tok) CK(cudaMemcpyAsync(p_tok, s.ptok, M * 4, cudaMemcpyDeviceToHost, st));
    if (q_tok) CK(cudaMemcpyAsync(q_tok, s.qtok, M * 4, cudaMemcpyDeviceToHost, st));
    if (residual_mass) CK(cudaMemcpyAsync(residual_mass, s.rm, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    return spr_device_status(ws, cuda_stream);
}

int sprinter_verify_host(const void *hidden, const void *W1, const float *b1, const void *W2,
                         const float *b2, float threshold, int B, int K, int d, int h, int dt, int path,
                         float *scores, uint8_t *accept, int32_t *first_reject, void *arena,
                         size_t arena_bytes, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (dt != SPR_F32 && dt != SPR_BF16) return SPR_ERR_UNSUPPORTED;
    if (B < 0 || K <= 0 || d <= 0 || h < 0) return SPR_ERR_INVALID_ARG;
    if (B == 0) return SPR_OK;
    if (!hidden || !W1 || !b2 || !accept || !first_reject || (h > 0 && (!b1 || !W2)))
        return SPR_ERR_INVALID_ARG;
    if (!arena || arena_bytes < spr_host_arena_bytes(SPR_OP_SPRINTER_VERIFY, B, K, 0, 0, d, h, dt))
        return SPR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Arena a{static_cast<char *>(arena), arena_bytes, 0, false};
    VerifyArena v = carve_verify(a, B, K, d, h, dt);
    const size_t M = (size_t)B * K;
    CK(cudaMemcpyAsync(v.hid, hidden, M * d * esz(dt), cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(v.W1, W1, (size_t)(h > 0 ? h : 1) * d * esz(dt), cudaMemcpyHostToDevice, st));
    if (h > 0) {
        CK(cudaMemcpyAsync(v.b1, b1, (size_t)h * 4, cudaMemcpyHostToDevice, st));
        CK(cudaMemcpyAsync(v.W2, W2, (size_t)h * esz(dt), cudaMemcpyHostToDevice, st));
    }
    CK(cudaMemcpyAsync(v.b2, b2, 4, cudaMemcpyHostToDevice, st));
    int rc = sprinter_verify(v.hid, v.W1, h > 0 ? (const float *)v.b1 : nullptr, h > 0 ? v.W2 : nullptr,
                             (const float *)v.b2, threshold, B, K, d, h, dt, path,
                             scores ? (float *)v.scores : nullptr, (uint8_t *)v.acc, (int32_t *)v.fr, ws,
                             ws_bytes, cuda_stream);
    if (rc != SPR_OK) return rc;
    if (scores) CK(cudaMemcpyAsync(scores, v.scores, M * 4, cudaMemcpyDeviceToHost, st));
    CK(cudaMemcpyAsync(accept, v.acc, M, cudaMemcpyDeviceToHost, st));
    CK(cudaMemcpyAsync(first_reject, v.fr, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    return spr_device_status(ws, cuda_stream);
}

int replace_sample_host(const void *target_logits, int64_t ldv, int V, int64_t R, const int32_t *rows,
                        const int32_t *first_reject, int K, int seq_stride, int n,
                        const float *uniforms, int dt, int32_t *tokens, void *arena, size_t arena_bytes,
                        void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (dt != SPR_F32 && dt != SPR_BF16) return SPR_ERR_UNSUPPORTED;
    if (V <= 0 || ldv < V || R < 0 || n < 0 || seq_stride < 0) return SPR_ERR_INVALID_ARG;
    if (n == 0) return SPR_OK;
    if (!target_logits || !uniforms || !tokens || R == 0 || (first_reject && K <= 0))
        return SPR_ERR_INVALID_ARG;
    if (first_reject && !rows && n > 1 && seq_stride < K) return SPR_ERR_INVALID_ARG;
    if (!arena || arena_bytes < spr_host_arena_bytes(SPR_OP_REPLACE_SAMPLE, n, 0, 0, ldv, 0, 0, dt))
        return SPR_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Arena a{static_cast<char *>(arena), arena_bytes, 0, false};
    DrawArena r = carve_draw(a, ldv, n, dt);
    // The row choice is known on the host, so only the rows that are drawn from travel:
    // draw i of the device call reads arena row i.
    int bad_row = 0, live = 0;
    for (int i = 0; i < n; ++i) {
        tokens[i] = -1;
        if (first_reject && first_reject[i] >= K) continue;
        const int64_t row = (rows ? (int64_t)rows[i] : (int64_t)i * seq_stride) +
                            (first_reject ? first_reject[i] : 0);
        if ((first_reject && first_reject[i] < 0) || row < 0 || row >= R) {
            bad_row = 1;
            continue;
        }
        CK(cudaMemcpyAsync(static_cast<char *>(r.logits) + (size_t)live * ldv * esz(dt),
                           static_cast<const char *>(target_logits) + (size_t)row * ldv * esz(dt),
                           (size_t)V * esz(dt), cudaMemcpyHostToDevice, st));
        CK(cudaMemcpyAsync(static_cast<char *>(r.u) + (size_t)live * 4, uniforms + i, 4,
                           cudaMemcpyHostToDevice, st));
        tokens[i] = live++;  // slot, replaced by the token below
    }
    int rc = SPR_OK;
    if (live > 0) {
        rc = replace_sample(r.logits, ldv, V, live, nullptr, nullptr, 0, 1, live, (const float *)r.u, dt,
                            (int32_t *)r.tok, ws, ws_bytes, cuda_stream);
        if (rc != SPR_OK) return rc;
        // results come back compacted; scatter them on the host
        int32_t *tmp = new int32_t[live];
        cudaError_t e = cudaMemcpyAsync(tmp, r.tok, (size_t)live * 4, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e == cudaSuccess)
            for (int i = 0; i < n; ++i)
                if (tokens[i] >= 0) tokens[i] = tmp[tokens[i]];
        delete[] tmp;
        if (e != cudaSuccess) return report_cuda_error(e);
        rc = spr_device_status(ws, cuda_stream);
    }
    return rc != SPR_OK ? rc : (bad_row ? SPR_ERR_BAD_ROW : SPR_OK);
}

}  // extern "C"
