/*
 * libsprinter - the verification-and-replacement step of SPRINTER (sequential
 * approximate verification for speculative decoding) and, for comparison on
 * the same inputs, standard speculative decoding's exact verification, as
 * CUDA kernels for sm_100a behind a plain C ABI.
 *
 * Conventions shared by every entry point unless it says otherwise
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; tensors are
 *     dense, row-major, innermost dimension contiguous.  Element pointers must
 *     be aligned to the element size; rows need no further alignment (16-byte
 *     aligned rows take the fastest path).
 *   - `dt` selects the element type of the "dt" tensors (logits, hidden
 *     states, verifier weights): SPR_F32 or SPR_BF16.  Biases, uniforms,
 *     scores and probabilities are float32; token ids and indices int32;
 *     accept masks uint8.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL
 *     is the default stream) and the call returns without synchronising.
 *   - Arguments are validated on the host before anything is enqueued; on a
 *     non-zero return nothing was launched.
 *   - `ws` is caller-owned device scratch of at least spr_workspace_bytes()
 *     bytes, 256-byte aligned, cleared once with spr_workspace_init() after
 *     allocation (this zeroes the status word and the ticket counters).  The
 *     kernels leave every counter they use at zero again (or the call clears
 *     it on the stream first), so one workspace serves calls of any op and
 *     shape it is large enough for, one after the other.  Calls that may
 *     overlap on the GPU (different streams) need separate workspaces.
 *   - The library allocates nothing.  Its only state is per-process caches of
 *     device properties and kernel attributes, the calling thread's
 *     timing-event pair (spr_set_stage_events) and the fixed scratch array of
 *     replace_sample_static.
 *   - Problems a kernel detects (a draft token id outside [0,V), a row index
 *     outside the logits tensor, a bounded wait that ran out) never trap: the
 *     affected outputs are set to -1, a sticky status word in `ws` records the
 *     first such code, and spr_device_status() returns and clears it.
 *   - Outputs are fully overwritten and are bit-identical from run to run for
 *     identical inputs (fixed reduction orders, no floating-point atomics).
 *   - Logits must be finite or -inf; uniforms must lie in [0,1); V <= 2^30.
 *   - The library runs only on compute capability 10.x devices; there is no
 *     CPU or other fallback (SPR_ERR_UNSUPPORTED).
 */
#ifndef SPRINTER_H_
#define SPRINTER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SPR_OK = 0,
    SPR_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, ldv < V, misaligned pointer */
    SPR_ERR_UNSUPPORTED = 2, /* unknown dtype / op, or not a compute-capability-10 device     */
    SPR_ERR_WORKSPACE = 3,   /* ws is NULL, misaligned or smaller than spr_workspace_bytes()  */
    SPR_ERR_CUDA = 4,        /* a CUDA runtime call failed (see spr_last_cuda_error)          */
    SPR_ERR_TIMEOUT = 5,     /* device: a bounded wait inside a kernel expired                */
    SPR_ERR_BAD_TOKEN = 6,   /* device: draft token id outside [0, V)                         */
    SPR_ERR_BAD_ROW = 7      /* device: selected logits row outside [0, R)                    */
} spr_status;

typedef enum { SPR_F32 = 0, SPR_BF16 = 1 } spr_dtype;

typedef enum {
    SPR_OP_SPRINTER_VERIFY = 0,
    SPR_OP_REPLACE_SAMPLE = 1,
    SPR_OP_SD_VERIFY = 2,
    SPR_OP_SPRINTER_STEP = 3,
    SPR_OP_SD_SHARD = 4,
    SPR_OP_VERIFIER_LABELS = 5,
    SPR_OP_VERIFIER_TRAIN = 6
} spr_op;

/* Which verifier kernel sprinter_verify() uses.  AUTO picks the tensor-core
 * kernel for bf16 MLPs whose shapes it supports and the SIMT kernel otherwise. */
typedef enum { SPR_VERIFIER_AUTO = 0, SPR_VERIFIER_SIMT = 1, SPR_VERIFIER_TENSOR = 2 } spr_verifier_path;

/* Bytes of device scratch one call of `op` needs.  For SPR_OP_REPLACE_SAMPLE,
 * B is the number of draws n and K, d, h are ignored; for SPR_OP_SD_VERIFY d
 * and h are ignored; for SPR_OP_SPRINTER_VERIFY V is ignored; SPR_OP_SPRINTER_STEP
 * uses all of them; for SPR_OP_SD_SHARD V is the width of this GPU's vocabulary
 * shard and d, h are ignored; SPR_OP_VERIFIER_LABELS uses B, K, V; SPR_OP_VERIFIER_TRAIN
 * uses d only.  Returns 0 for invalid arguments.  A workspace sized for the
 * largest op serves all of them. */
size_t spr_workspace_bytes(int op, int B, int K, int V, int d, int h, int dt);

/* Clears a freshly allocated workspace (enqueues a memset on the stream). */
int spr_workspace_init(void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * sprinter_verify - verifier score, threshold test and first rejection.
 *
 * Defined by: Algorithm 2 (detailed SPRINTER), the while-loop: a draft token is
 * kept while V(s(x, prefix)) >= tau and generation stops at the first token
 * that fails; Section 3.2 "Verifier architecture": V is one linear layer and a
 * sigmoid on the draft model's last hidden state (tau = 0.5 in the experiments).
 *
 * hidden [B,K,d] dt : s(x, prefix) for the K draft positions of B sequences.
 * MLP mode (h > 0)  : W1 [h,d] dt, b1 [h] f32, W2 [h] dt, b2 [1] f32
 *                     score = sigmoid(b2 + W2 . relu(W1 hidden + b1))
 * paper's verifier (h == 0): W1 is the weight vector [d] dt, b1 = W2 = NULL,
 *                     score = sigmoid(b2 + W1 . hidden)
 * accept[b,k]      = score[b,k] >= threshold            (uint8, 0/1)
 * first_reject[b]  = min{k : accept[b,k] == 0}, K if every token passed
 *                    (= the number of draft tokens kept)
 * scores [B,K] f32 : optional (NULL to skip).
 * path             : spr_verifier_path.
 * Errors: SPR_ERR_INVALID_ARG (null / sizes), SPR_ERR_UNSUPPORTED (dtype, or
 * SPR_VERIFIER_TENSOR forced on a shape it cannot take), SPR_ERR_WORKSPACE.
 */
int sprinter_verify(const void *hidden, const void *W1, const float *b1, const void *W2,
                    const float *b2, float threshold, int B, int K, int d, int h, int dt, int path,
                    float *scores, uint8_t *accept, int32_t *first_reject, void *ws, size_t ws_bytes,
                    void *cuda_stream);

/*
 * replace_sample - the target model's replacement token for a rejected draft.
 *
 * Defined by: Algorithm 2, the part after the loop (the single call of the target
 * model): p' <- p, t ~ p'.  The draw is an inverse CDF in vocabulary order driven by a
 * caller-supplied uniform: with e_i = exp(l_i - max l),
 *   t = min{ j : sum_{i<=j} e_i > u * sum_i e_i }
 * (the last index with e_j > 0 if rounding leaves none).
 *
 * target_logits [R, ldv] dt, V <= ldv valid entries per row.
 * Draw i (0 <= i < n) reads row
 *   (rows ? rows[i] : i * seq_stride) + (first_reject ? first_reject[i] : 0)
 * and is skipped - tokens[i] = -1, no memory traffic - when first_reject is
 * given and first_reject[i] >= K (the verifier kept every draft token, so the
 * target is not called).  Passing sprinter_verify's first_reject output here
 * chains the two calls on one stream with no host synchronisation.
 * uniforms [n] f32, tokens [n] int32.  With first_reject and without rows, seq_stride >= K
 * (otherwise neighbouring sequences would share rows: SPR_ERR_INVALID_ARG).
 * Device-detected: row outside [0,R), or first_reject[i] < 0 -> tokens[i] = -1,
 * SPR_ERR_BAD_ROW.
 */
int replace_sample(const void *target_logits, int64_t ldv, int V, int64_t R, const int32_t *rows,
                   const int32_t *first_reject, int K, int seq_stride, int n, const float *uniforms,
                   int dt, int32_t *tokens, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * sprinter_step - one SPRINTER verification-and-replacement step in a single call.
 *
 * Defined by: Algorithm 2 as a whole: the verifier loop over the K draft positions
 * (sprinter_verify) followed by the single target call for the position where the
 * verifier stopped (replace_sample on row b*seq_stride + first_reject[b], skipped
 * when every token passed).  Same arguments, results and error behaviour as those
 * two calls made one after the other with first_reject passed along, on one
 * workspace; for small batches the replacement kernel is launched programmatically
 * behind the verifier kernel, so that its launch latency hides in the verifier's tail.
 *
 * target_logits [B, seq_stride, ldv] dt with seq_stride >= K rows per sequence (K, or
 * K+1 when a bonus row is kept); uniforms [B] f32; tokens [B] int32 (-1 where nothing
 * was rejected).  Workspace: spr_workspace_bytes(SPR_OP_SPRINTER_STEP, ...).
 */
int sprinter_step(const void *hidden, const void *W1, const float *b1, const void *W2, const float *b2,
                  float threshold, int B, int K, int d, int h, const void *target_logits, int64_t ldv,
                  int V, int seq_stride, const float *uniforms, int dt, int path, float *scores,
                  uint8_t *accept, int32_t *first_reject, int32_t *tokens, void *ws, size_t ws_bytes,
                  void *cuda_stream);

/*
 * sd_verify - exact verification of standard speculative decoding.
 *
 * Defined by: Section 2 (Preliminaries): draft token x is accepted with
 * probability min(1, p(x)/q(x)); at the first rejection the target resamples
 * from Eq. 1, p'(x) = norm(max(0, p(x) - q(x))).  With K = 1 on a token the
 * verifier rejected this is also the keep-or-resample rule of Section 3
 * ("Algorithm") that Theorem 1 analyses.
 *
 * p_logits [B,Kp,ldv] dt (Kp = K or K+1), q_logits [B,K,ldv] dt,
 * draft_tokens [B,K] int32, uniforms [B,K+1] f32.
 *   p(.), q(.)        = softmax of the rows (temperature 1)
 *   accept[b,k]       = uniforms[b,k] <= min(1, p(x)/q(x)), x = draft_tokens[b,k]
 *                       (every position is tested, also those after a rejection)
 *   accepted_len[b]   = n_b = min{k : accept[b,k] == 0}, K if none
 *   correction_token[b]:
 *       n_b < K            inverse-CDF draw with uniforms[b,K] from
 *                          norm(max(0, p - q)) at position n_b (from p itself
 *                          in the degenerate case max(0, p - q) == 0)
 *       n_b = K, Kp = K+1  draw with uniforms[b,K] from p at position K
 *       n_b = K, Kp = K    -1
 *   accept [B,K], p_tok [B,K] = p(x), q_tok [B,K] = q(x), residual_mass [B] =
 *   sum_i max(0, p_i - q_i) at position n_b (0 when n_b = K): optional, NULL to skip.
 * Device-detected: draft token outside [0,V) -> that sequence reports
 * accepted_len = correction_token = -1, accept bits 0, p_tok = q_tok = -1 at that
 * position, SPR_ERR_BAD_TOKEN.
 */
int sd_verify(const void *p_logits, const void *q_logits, int64_t ldv, const int32_t *draft_tokens,
              const float *uniforms, int B, int K, int Kp, int V, int dt, int32_t *accepted_len,
              int32_t *correction_token, uint8_t *accept, float *p_tok, float *q_tok,
              float *residual_mass, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * sd_shard_* - sd_verify for logits split along the vocabulary across G GPUs.
 *
 * Defined by: the same passages as sd_verify (Section 2, Eq. 1); the paper has no
 * multi-GPU form.  This is sd_verify for a tensor-parallel LM head: GPU g holds columns
 * [v0_g, v0_g + Vs_g) of every p and q row (shards in rank order tile [0, V) without gaps).
 * Results equal sd_verify's on the concatenated rows, on every GPU, except that
 * correction_token[b] is the token on the one GPU whose shard contains it and -1 on the
 * others (reduce with max).  The sequence of calls on each GPU, all on one stream and one
 * workspace of spr_workspace_bytes(SPR_OP_SD_SHARD, B, K, Vs, 0, 0, dt) bytes that nothing
 * else uses in between:
 *
 *   sd_shard_stats    reads the shard once.  stats [B*Kp, 6] f32 per row b*Kp + k:
 *                     (max, sum exp(l - max)) of the p shard row, the same of the q shard
 *                     row, and l_p[x], l_q[x] of the draft token x = draft_tokens[b,k] if
 *                     v0 <= x < v0 + Vs, else -inf (q entries of the bonus row k = K:
 *                     -inf, 0, -inf).
 *   -- all-gather stats -> all_stats [G, B*Kp, 6], rank order --
 *   sd_shard_decide   merges the G records of every row in rank order, then accept,
 *                     accepted_len, p_tok, q_tok exactly as sd_verify defines them
 *                     (identical on every GPU); keeps the whole-row statistics in ws.
 *                     V is the whole vocabulary (draft tokens outside [0,V) are reported
 *                     as in sd_verify); Vs and dt only size the workspace.
 *   sd_shard_weights  weights [B, 2] f64 per sequence: this shard's total weight of the
 *                     correction draw - (0, sum over the shard of max(0, p_i - q_i)) with
 *                     whole-row probabilities at position accepted_len[b] < K;
 *                     (shard max, sum exp(l - shard max)) of the bonus row when
 *                     accepted_len[b] = K and Kp = K+1; (0, 0) when there is no draw.
 *   (sd_shard_decide_weights does the two passes above in one launch: it takes the
 *   arguments of both and gives the results of sd_shard_decide followed by sd_shard_weights.)
 *   -- all-gather weights -> all_weights [G, B, 2], rank order --
 *   sd_shard_draw     adds the G shard weights in rank order, finds the shard in which
 *                     uniforms[b,K] * total falls, and on that GPU (rank) locates the token
 *                     by the inverse CDF of sd_verify, returned as a whole-vocabulary id.
 *                     residual_mass [B] (optional) is the total over all shards, on every
 *                     GPU.  If the residual vanishes on every shard the draw is from p at
 *                     that position, using the shard statistics in all_stats.
 *
 * p_shard [B,Kp,ldv] dt and q_shard [B,K,ldv] dt point at column v0 of the first row; ldv
 * is the row stride in elements (>= Vs).  Errors as for sd_verify; G <= 1024.
 */
int sd_shard_stats(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, int v0,
                   const int32_t *draft_tokens, int B, int K, int Kp, int dt, float *stats, void *ws,
                   size_t ws_bytes, void *cuda_stream);
int sd_shard_decide(const float *all_stats, int G, const int32_t *draft_tokens, const float *uniforms, int B,
                    int K, int Kp, int V, int Vs, int dt, int32_t *accepted_len, uint8_t *accept, float *p_tok,
                    float *q_tok, void *ws, size_t ws_bytes, void *cuda_stream);
int sd_shard_weights(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, const int32_t *accepted_len,
                     const float *uniforms, int B, int K, int Kp, int dt, double *weights, void *ws,
                     size_t ws_bytes, void *cuda_stream);
int sd_shard_decide_weights(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, const float *all_stats,
                            int G, const int32_t *draft_tokens, const float *uniforms, int B, int K, int Kp, int V,
                            int dt, int32_t *accepted_len, uint8_t *accept, float *p_tok, float *q_tok,
                            double *weights, void *ws, size_t ws_bytes, void *cuda_stream);
int sd_shard_draw(const void *p_shard, const void *q_shard, int64_t ldv, int Vs, int v0, const double *all_weights,
                  const float *all_stats, int G, int rank, const int32_t *accepted_len, const float *uniforms,
                  int B, int K, int Kp, int dt, int32_t *correction_token, float *residual_mass, void *ws,
                  size_t ws_bytes, void *cuda_stream);

/*
 * verifier_labels - training labels of the verifier.
 *
 * Defined by: Section 3.2 ("Verifier Training Methodology"): a (prefix, draft token x) pair
 * is labelled 1 if q(x)/p(x) <= lambda and 0 otherwise; lambda = 1 is the ideal verifier of
 * Section 3, the appendix on training details uses lambda in {1, 1.2, 1.5}.
 *
 * p_logits [B,Kp,ldv] dt (Kp >= K; only the first K rows of a sequence are read),
 * q_logits [B,K,ldv] dt, draft_tokens [B,K] int32 (device).  lambdas: HOST array of
 * n_lambda <= 8 thresholds (read during the call).  p, q = softmax of the rows; the ratio
 * is formed in log space in double precision from fp32 row statistics.
 *   labels [n_lambda,B,K] uint8 (device): labels[l,b,k] = (q(x)/p(x) <= lambdas[l])
 *   ratio  [B,K] f32 (device, optional):  q(x)/p(x), +inf where p(x) = 0
 * Each logits row is read once (2*V*es bytes per token).  Device-detected: draft token
 * outside [0,V) -> labels 0, ratio -1, SPR_ERR_BAD_TOKEN.
 * Workspace: spr_workspace_bytes(SPR_OP_VERIFIER_LABELS, B, K, V, 0, 0, dt).
 */
int verifier_labels(const void *p_logits, const void *q_logits, int64_t ldv, const int32_t *draft_tokens, int B,
                    int K, int Kp, int V, int dt, const float *lambdas, int n_lambda, uint8_t *labels, float *ratio,
                    void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * verifier_train_step - one optimiser step of the single-layer verifier.
 *
 * Defined by: Section 3.2 ("Verifier architecture used for evaluation"): V(s) = sigmoid(b +
 * w.s) on the draft model's last hidden state, trained with Adam on the binary
 * cross-entropy loss.  One call is one Adam step (Kingma & Ba, Algorithm 1, with bias
 * correction) on the mean loss over the N samples passed:
 *   z_i = b + w.s_i,  loss = (1/N) sum_i [ln(1 + e^{z_i}) - y_i z_i],
 *   g = (1/N) sum_i (sigmoid(z_i) - y_i) (s_i, 1),
 *   m <- beta1 m + (1-beta1) g,  v <- beta2 v + (1-beta2) g^2,
 *   theta <- theta - lr (m / (1-beta1^t)) / (sqrt(v / (1-beta2^t)) + eps).
 * The batch is whatever the caller passes; early stopping is the caller's loop over `loss`.
 *
 * hidden [N,d] dt (device, 16-byte aligned, d a multiple of 16/es and at most 4096 for
 * bf16, 2048 for fp32: otherwise SPR_ERR_UNSUPPORTED), labels [N] uint8 in {0,1} (device),
 * theta, adam_m, adam_v [d+1] f32 (device; weights then bias; updated in place; start m
 * and v at zero), t >= 1 the step number, loss [1] f32 (device, optional): the loss BEFORE
 * the update.  Every hidden state is read once (N*d*es bytes per step); sums have a fixed
 * order, so a step is reproducible bit for bit.
 * Errors on the device: the gradient kernel waits for its rows with a poll limit; if a wait
 * runs out the status word becomes SPR_ERR_TIMEOUT, no step is taken (theta, adam_m, adam_v
 * unchanged) and *loss is NaN.  While the status word still holds SPR_ERR_TIMEOUT (it is
 * cleared by spr_device_status) later steps on that workspace are not taken either.
 * Workspace: spr_workspace_bytes(SPR_OP_VERIFIER_TRAIN, 0, 0, 0, d, 0, dt).
 */
int verifier_train_step(const void *hidden, const uint8_t *labels, int64_t N, int d, int dt, float *theta,
                        float *adam_m, float *adam_v, int t, float lr, float beta1, float beta2, float eps,
                        float *loss, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * sprinter_simulate - run lengths of an i.i.d. verifier (Monte-Carlo of Theorems 2 and 3).
 *
 * Defined by: Section 3.1(b), the scenario of Theorem 2: the draft produces r acceptable
 * tokens followed by unacceptable ones; the verifier accepts an acceptable token with
 * probability eta_tp and an unacceptable one with probability eta_fp, independently;
 * N = number of consecutive tokens accepted before the first rejection (capped at
 * max_tokens).  Theorem 2 gives the law and mean of N, Theorem 3 the stopping time
 * t_d (N + 1).
 *
 * Run i (i = first_run .. first_run + runs - 1) owns one Philox4x32-10 stream: block j
 * = Philox(counter {lo(i), hi(i), j, 0}, key {lo(seed), hi(seed)}); token k uses word
 * k % 4 of block k / 4 with u = (word >> 8) * 2^-24 and is accepted iff
 * u < (k < r ? eta_tp : eta_fp).  Results therefore do not depend on the launch shape.
 * n_accepted [runs] int32 (device, optional), histogram [max_tokens + 1] uint64 (device,
 * optional, overwritten): at least one must be given.  No workspace.
 */
int sprinter_simulate(uint64_t seed, int64_t first_run, int64_t runs, int r, float eta_tp, float eta_fp,
                      int max_tokens, int32_t *n_accepted, uint64_t *histogram, void *cuda_stream);

/*
 * Host-buffer variants.  Same operations and arguments as the calls above, but every
 * tensor pointer is a HOST pointer (pinned memory makes the copies asynchronous and
 * fast).  Each call copies its inputs into `arena` - caller-owned device memory of at
 * least spr_host_arena_bytes() bytes, 256-byte aligned - runs the device entry point,
 * copies the outputs back, synchronises the stream and returns the device status
 * (so SPR_ERR_BAD_TOKEN / SPR_ERR_BAD_ROW come back directly).  replace_sample_host
 * resolves the row of every draw on the host and uploads only the rows that are
 * drawn from.  For spr_host_arena_bytes, B is the number of draws n for
 * SPR_OP_REPLACE_SAMPLE, and unused sizes may be 0.
 */
size_t spr_host_arena_bytes(int op, int B, int K, int Kp, int64_t ldv, int d, int h, int dt);

int sprinter_verify_host(const void *hidden, const void *W1, const float *b1, const void *W2,
                         const float *b2, float threshold, int B, int K, int d, int h, int dt, int path,
                         float *scores, uint8_t *accept, int32_t *first_reject, void *arena,
                         size_t arena_bytes, void *ws, size_t ws_bytes, void *cuda_stream);

int replace_sample_host(const void *target_logits, int64_t ldv, int V, int64_t R, const int32_t *rows,
                        const int32_t *first_reject, int K, int seq_stride, int n,
                        const float *uniforms, int dt, int32_t *tokens, void *arena, size_t arena_bytes,
                        void *ws, size_t ws_bytes, void *cuda_stream);

int sd_verify_host(const void *p_logits, const void *q_logits, int64_t ldv, const int32_t *draft_tokens,
                   const float *uniforms, int B, int K, int Kp, int V, int dt, int32_t *accepted_len,
                   int32_t *correction_token, uint8_t *accept, float *p_tok, float *q_tok,
                   float *residual_mass, void *arena, size_t arena_bytes, void *ws, size_t ws_bytes,
                   void *cuda_stream);

/*
 * replace_sample_static - replace_sample without a caller workspace.
 *
 * The paper has no counterpart: this exists for callers of this library that are not
 * allowed to allocate device memory around the call - code that runs inside someone
 * else's memory budget (a serving engine that has handed all free HBM to its KV-cache
 * pool, a plugin whose host forbids cudaMalloc), or that runs where cudaMalloc would
 * stall everything (it synchronises the device).  They have nowhere to get a `ws` from.
 * Same operation, arguments and results as replace_sample(), but the scratch is a fixed
 * array inside the library image (about 516 KB on every GPU that loads the library, held
 * until the process exits).  The call allocates and frees nothing.
 *
 * Limits: n <= SPR_STATIC_MAX_DRAWS and n * steps <= SPR_STATIC_MAX_DRAW_STEPS, where
 * steps = ceil((V + 7) / 1024) for bf16 and ceil((V + 3) / 512) for f32 (126 for
 * V = 128256 bf16, so up to 520 draws per call; 1024 draws up to V = 65529 bf16, 1008 draws at
 * V = 65536, where steps = 65).  Larger requests return
 * SPR_ERR_WORKSPACE and launch nothing; split them or use replace_sample().
 *
 * The device that owns the tensors must be the current device of the calling thread: the
 * scratch used is the current device's copy of the array.
 * First call on a device: looks up the device address of the array.  Make that first call
 * before starting any stream capture.
 * Sharing: every call on a GPU uses the same array.  Calls that can overlap on that GPU
 * (two streams, two host threads) race on it and give wrong tokens; issue them on one
 * stream or serialise them.  The array keeps the previous call's contents; the call clears
 * the part that must start at zero itself.
 * Device-detected bad rows still give tokens[i] = -1, but there is no status word to read
 * back.
 */
#define SPR_STATIC_MAX_DRAWS 1024
#define SPR_STATIC_MAX_DRAW_STEPS 65536
int replace_sample_static(const void *target_logits, int64_t ldv, int V, int64_t R, const int32_t *rows,
                          const int32_t *first_reject, int K, int seq_stride, int n,
                          const float *uniforms, int dt, int32_t *tokens, void *cuda_stream);

/* Timing aid: while set (non-NULL cudaEvent_t handles), sd_verify calls made by this
 * host thread record `before` / `after` on their stream around the row-statistics
 * kernel, the launch that reads the 2*B*K*V logits.  Pass NULL, NULL to stop. */
void spr_set_stage_events(void *before, void *after);

/*
 * spr_test_sprinter_verify - test hook, not part of the stable interface.
 *
 * The paper has no counterpart.  sprinter_verify on the tensor-core kernel (bf16 MLP, the
 * shapes SPR_VERIFIER_TENSOR takes) with the launch shape chosen by the caller instead of by
 * the library, so that tests reach every shape on small inputs: bm, bn in {64, 128} tokens x
 * hidden units per tile, splits in {1, 2, 4, 8} CTAs sharing a tile along d, cluster_n = 1
 * (finish through the workspace) or -1 (a tile's CTAs form one cluster; needs
 * splits * ceil(h / bn) <= 8); 0 leaves a value to the library.  bm = 256 (with bn = 128,
 * splits = 1) selects the kernel in which two CTAs share a 256 x 128 tile.  A combination
 * the problem does not allow returns SPR_ERR_UNSUPPORTED.
 * flags bit 0: the kernel's copy engine producer issues nothing, so that the first bounded
 * wait of every CTA runs out after spin_limit polls (0 = the library's limit): the call
 * returns SPR_OK, the status word reads SPR_ERR_TIMEOUT, scores are -1, accept bits 0 and
 * first_reject -1, nothing is left in flight and the workspace stays usable.
 */
int spr_test_sprinter_verify(const void *hidden, const void *W1, const float *b1, const void *W2,
                             const float *b2, float threshold, int B, int K, int d, int h, int dt,
                             float *scores, uint8_t *accept, int32_t *first_reject, void *ws, size_t ws_bytes,
                             void *cuda_stream, int bm, int bn, int splits, int cluster_n, int flags,
                             unsigned spin_limit);

/*
 * spr_test_verifier_train_step - test hook, not part of the stable interface.
 *
 * The paper has no counterpart.  verifier_train_step with flags bit 0 set: the gradient
 * kernel fetches no row, so the first bounded wait of every team of warps runs out after
 * spin_limit polls (0 = the library's limit).  The call returns SPR_OK, the status word reads
 * SPR_ERR_TIMEOUT, theta / adam_m / adam_v are left as they were, *loss is NaN, nothing is left
 * in flight and the workspace stays usable.  flags = 0 is verifier_train_step with that limit.
 */
int spr_test_verifier_train_step(const void *hidden, const uint8_t *labels, int64_t N, int d, int dt,
                                 float *theta, float *adam_m, float *adam_v, int t, float lr, float beta1,
                                 float beta2, float eps, float *loss, void *ws, size_t ws_bytes,
                                 void *cuda_stream, int flags, unsigned spin_limit);

/* Synchronises the stream, returns the sticky device status word of `ws`
 * (SPR_OK if nothing was detected) and clears it. */
int spr_device_status(void *ws, void *cuda_stream);

/* Text for a status code; the last CUDA runtime error string seen by this thread. */
const char *spr_status_string(int status);
const char *spr_last_cuda_error(void);

/* Kernels one sd_verify call launches for this shape (2, or 3 when the row-statistics pass is
 * followed by a separate finish grid; 0 for arguments sd_verify rejects).  The paper has no
 * counterpart: bookkeeping for callers that count launches. */
int spr_sd_verify_launches(int B, int K, int V, int dt);

/* Library version: major * 10000 + minor * 100 + patch. */
int spr_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPRINTER_H_ */
