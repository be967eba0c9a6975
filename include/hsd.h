/*
 * hsd.h -- C ABI of the B200 (sm_100a) hot path of Hierarchical Speculative Decoding.
 *
 * Method: "Fast Inference via Hierarchical Speculative Decoding" (arXiv 2510.19705).
 * Models M_0..M_K share a vocabulary; M_K is the target.  Only M_0 generates token by
 * token; every level i >= 1 verifies, in ONE multi-row forward pass, the tokens the level
 * below proposed, applies the speculative-sampling rule at every drafted position and hands
 * its verified tokens and its OWN distributions upward (Algorithm 1, Algorithm 2).
 *
 * Conventions
 *   - Every function returns HSD_OK (0) or a negative HSD_E_* code; nothing is printed, no
 *     exception crosses the boundary.  hsd_strerror() names a code.
 *   - "device" pointers are CUDA device memory of the current device, "host" pointers are
 *     ordinary host memory.  All buffers are caller-owned unless stated otherwise.  The
 *     library allocates no device memory: scratch comes from caller-provided workspaces.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - dtype: HSD_F32 or HSD_BF16 = storage type of weights, KV cache and logits.
 *   - Random numbers: Philox4x32-10, key = seed, counter = (position in call, call serial,
 *     level | purpose << 8, sequence index); the uniform is the top 24 bits of output word 0.
 *     A decision's uniform therefore does not depend on how many draws preceded it.
 *   - Decisions (accept / which token) are taken in integer arithmetic on 32-bit softmax
 *     numerators E_k = min(floor(exp(l_k - max l) * 2^32), 2^32 - 1), exp evaluated by a fixed
 *     sequence of IEEE fp32 operations, so results do not depend on summation order.
 */
#ifndef HSD_H_
#define HSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  HSD_OK = 0,
  HSD_E_INVALID_ARG = -1,
  HSD_E_WORKSPACE_TOO_SMALL = -2,
  HSD_E_OUT_OF_PAGES = -3,
  HSD_E_CUDA = -4,
  HSD_E_DEVICE_TIMEOUT = -5,
  HSD_E_UNSUPPORTED = -6,
  HSD_E_IO = -7,
  HSD_E_TOO_LARGE = -8
};
enum { HSD_F32 = 0, HSD_BF16 = 1 };

/* Text for a status code (static storage). */
const char *hsd_strerror(int status);

/* ---------------------------------------------------------------------------------------
 * Level-0 drafting, sampling step (Algorithm 1, base case: M_0 emits one token and its distribution at a time).
 * Token (b, j) is drawn from softmax(logits[b, j, :]) by inverse CDF in ascending token id
 * with the uniform addressed (j, call_serial, level 0, purpose 0, b).
 *   logits      device [batch, rows, vocab], dtype as given, row-major, read only
 *   out_tokens  device [batch, rows] int32
 * Errors: INVALID_ARG (null pointer, non-positive size, unknown dtype), CUDA (launch failed).
 */
int hsd_draft_sample(const void *logits, int batch, int rows, int vocab, int dtype,
                     uint64_t seed, uint64_t call_serial, void *stream, int32_t *out_tokens);

/* ---------------------------------------------------------------------------------------
 * Verification decision for one level on given logits (Algorithm 2 after its forward pass;
 * the rule of Section 2: accept x with probability min(1, p(x)/q(x)), otherwise resample from
 * norm(max(0, p - q))).  For every sequence b: positions j = 0..t-1 are tested in order with
 * uniforms (j, call_serial, level, purpose 1, b); n = number accepted before the first
 * rejection; the final token m is drawn with uniform (0, call_serial, level, purpose 2, b)
 * from the normalised residual of row n if n < t, else from target row t.
 *   target_logits  device [batch, t+1, vocab]   p_1..p_{t+1}
 *   draft_logits   device [batch, t,   vocab]   q_1..q_t
 *   draft_tokens   device [batch, t] int32      x_1..x_t, each in [0, vocab)
 *   workspace      device scratch of at least hsd_verify_workspace_bytes(batch, t) bytes,
 *                  16-byte aligned; contents on entry are ignored, on exit unspecified
 *   out_tokens     device [batch, t+1] int32: x_1..x_n, m, then -1 padding
 *   out_n_accepted device [batch] int32: n
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, CUDA.  Asynchronous on `stream`.
 */
size_t hsd_verify_workspace_bytes(int batch, int t);
int hsd_verify_level(int level, const void *target_logits, const void *draft_logits,
                     const int32_t *draft_tokens, int batch, int t, int vocab, int dtype,
                     uint64_t seed, uint64_t call_serial, void *workspace, size_t workspace_bytes,
                     void *stream, int32_t *out_tokens, int32_t *out_n_accepted);

/* ---------------------------------------------------------------------------------------
 * hsd_verify_level without a workspace argument and without any allocation.  (The paper has no
 * counterpart: this entry point exists for integration reasons only.)
 *
 * Who needs it: callers that get device buffers handed to them but cannot obtain more -- an
 * inference-server plugin or a custom op that receives only its input and output tensors, code
 * running under an allocator it must not re-enter, or a latency-critical thread for which an
 * allocating call (which may synchronise the whole device) is off limits.  hsd_verify_level
 * makes such callers find scratch memory somewhere; this variant brings its own.
 *
 * Same arguments, outputs and results as hsd_verify_level.  The scratch (row statistics, counters
 * and a queue of sequences) lives in a fixed device array of 98,560 bytes inside the library image (every GPU
 * that loads the library holds it until the process exits), which bounds the call:
 * batch * (2 t + 1) <= 4096, else HSD_E_TOO_LARGE (exactly 4096 is accepted).
 * The call performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *   - The first call on each device looks up the array's device address and keeps it; make that
 *     first call outside any stream capture.  The kept address does not survive cudaDeviceReset():
 *     do not use this entry point on a device after resetting it.
 *   - All calls share the one array and it keeps whatever the last call left in it.  The counters
 *     and the queue must start at zero and every call clears them on `stream` before its kernel; the statistics
 *     are overwritten before they are read.  Two calls that overlap on the GPU -- different streams,
 *     or different host threads -- race on the array: serialise them (one stream, or an event
 *     between them).
 * Errors: INVALID_ARG, TOO_LARGE, CUDA. */
int hsd_verify_level_static(int level, const void *target_logits, const void *draft_logits,
                            const int32_t *draft_tokens, int batch, int t, int vocab, int dtype,
                            uint64_t seed, uint64_t call_serial, void *stream, int32_t *out_tokens,
                            int32_t *out_n_accepted);

/* ---------------------------------------------------------------------------------------
 * The hierarchy: models M_0..M_K as early exits of one decoder-only transformer (Section 5.1:
 * level i = the first exit_layers[i] layers followed by the shared final norm and the shared
 * output head), parameters T_0..T_{K-1} (Algorithm 1).
 *
 * Network (the paper uses pretrained checkpoints and does not describe it; this is the
 * Llama-style decoder of the benchmark shapes): pre-norm residual blocks, RMSNorm with gain,
 * rotary embedding with half-split pairing, causal attention with grouped KV heads, SwiGLU MLP,
 * untied output head, softmax at temperature 1 over the whole vocabulary.  Matrices are stored
 * [out_features, in_features] row-major in `dtype`.
 */
typedef struct hsd_ctx hsd_ctx; /* opaque; owns host bookkeeping only */

typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
  int32_t dtype;                     /* HSD_F32 or HSD_BF16 */
  float rms_eps, rope_theta;
  int32_t max_batch, max_seq;        /* capacity: sequences, tokens per sequence (prompt + generated + drafts) */
  int32_t page_size;                 /* tokens per KV page (0 = 16) */
  const void *embed;                 /* device [vocab, d_model] */
  const void *final_norm;            /* device [d_model] */
  const void *lm_head;               /* device [vocab, d_model] */
  const void *const *layer_weights;  /* HOST array [n_layers * 9] of device pointers, per layer:
                                        attn_norm[d], wq[nq*hd, d], wk[nkv*hd, d], wv[nkv*hd, d], wo[d, nq*hd],
                                        mlp_norm[d], wg[ff, d], wu[ff, d], wd[d, ff] */
} hsd_model_desc;

/* Per-level counters accumulated over one hsd_generate call.  Level 0: calls = HSD(0) calls,
 * emitted = drafted tokens.  Level i >= 1: calls = Verify calls, drafted = tokens received,
 * tested = accept tests of Algorithm 2's sequential loop, accepted = sum of n, emitted = sum of n+1.
 * rows = token rows pushed through the level's forward passes (drafts + catch-up rows);
 * forwards = forward passes; ms = device time of those passes. */
typedef struct {
  int64_t calls, rows, drafted, tested, accepted, emitted, forwards;
  double ms;
} hsd_level_stats;

/* Device workspace needed by hsd_create for this model / hierarchy (KV pages, token buffers,
 * per-level logits rows, activations, scratch).  0 on invalid arguments. */
size_t hsd_workspace_bytes(const hsd_model_desc *model, const int32_t *exit_layers, int n_levels, const int32_t *T);

/* Build a context.  exit_layers [n_levels] ascending, last == n_layers; T [n_levels - 1], each >= 1
 * (n_levels == 1: plain autoregressive sampling from the target; n_levels == 2: single-draft
 * speculative decoding).  workspace: device, 256-byte aligned, >= hsd_workspace_bytes(), must
 * outlive the context, as must the weights.  The descriptor itself is only read during the call.
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, UNSUPPORTED (head_dim not in {32,64,128}, ...), CUDA. */
int hsd_create(const hsd_model_desc *model, const int32_t *exit_layers, int n_levels, const int32_t *T,
               void *workspace, size_t workspace_bytes, hsd_ctx **out);

/* The hierarchy as separate models (Section 3.1, "Preliminaries": M_0..M_K are arbitrary models over one
 * vocabulary, each with its own cost c_i; Section 5.1's early exits are one way to get them).  Level i is ALL
 * layers of models[i] with that model's own embedding, final norm and output head, and keeps a KV cache of its own:
 * a level's forward pass processes every position its own cache has not seen (the drafts it verifies plus the
 * tokens the other levels emitted since its last pass), the prompt pass runs every model over the prompt, and the
 * rollback after a verification cuts every model's cache to the accepted length.  Algorithm 1 and Algorithm 2 run
 * unchanged on top (hsd_generate, hsd_set_trace, hsd_set_iid_acceptance, hsd_set_exit_heads, hsd_destroy).
 *   models  host [n_levels], models[n_levels - 1] = the target.  All must agree on vocab, dtype, max_batch,
 *           max_seq and page_size; layer counts, widths, head counts and d_ff are free per model.
 *   T       host [n_levels - 1], each >= 1.
 * hsd_layer_logits on such a context runs the target model.
 * Errors: INVALID_ARG (also: the models disagree on a shared quantity), WORKSPACE_TOO_SMALL, UNSUPPORTED, CUDA. */
size_t hsd_models_workspace_bytes(const hsd_model_desc *models, int n_levels, const int32_t *T);
int hsd_create_models(const hsd_model_desc *models, int n_levels, const int32_t *T, void *workspace,
                      size_t workspace_bytes, hsd_ctx **out);

/* Decode passes of bf16 models fold two finish phases of the verification forward (Algorithm 2's multi-row pass)
 * into their consumers: the q / k / v finish into the attention phase, the gate / up finish into the down
 * projection; and the RMSNorm after each residual projection starts, on CTAs that hold no tile of that
 * projection, as soon as its partial sums are stored instead of after a grid-wide barrier.  fold_qkv = 0 /
 * fold_gate_up = 0 / early_norm = 0 keeps the separate phase or the barrier; the results are the same sums in
 * the same order either way (a test hook and a tuning knob; all on by default).  Errors: INVALID_ARG. */
int hsd_set_phase_folding(hsd_ctx *ctx, int fold_qkv, int fold_gate_up, int early_norm);

/* Which kernel path attention work items with long key ranges take (the paper gives no kernel design; its
 * verification pass of Algorithm 2 attends over the whole context).  enabled != 0 (the default): on models with
 * head size 128, an item with 8 or more query vectors whose key range has 2048 keys or more runs on the
 * fifth-generation tensor cores with its scores and outputs in tensor memory; enabled = 0: every item runs on the warp-level path.  Both paths compute the
 * same attention (softmax weights rounded to bf16 before the P V product on the tensor-memory path, to bf16 hi + lo
 * on the other), so results agree to rounding, not bit for bit.  enabled = 2 additionally keeps the key splits of
 * long contexts at 2048 keys or more, so that small test models reach that path too.  A test hook and a tuning knob.
 * Errors: INVALID_ARG. */
int hsd_set_tensor_attention(hsd_ctx *ctx, int enabled);

/* One output head per level instead of the shared one (Section 5.1: the setting in which every exit
 * layer has its own trained head, a linear map from the embedding dimension to the vocabulary, so that
 * memory grows with the number of levels; the shared head of the descriptor is the other setting).
 * Level i then computes its logits as lm_heads[i] x RMSNorm(hidden state after exit_layers[i]; gain
 * final_norms[i]).
 *   final_norms  host [n_levels] of device pointers [d_model] in the model's dtype, or NULL
 *   lm_heads     host [n_levels] of device pointers [vocab, d_model] row-major in the model's dtype,
 *                16-byte aligned, or NULL
 * A NULL array or entry keeps (or restores) the descriptor's shared tensor for that level.  The tensors
 * are not copied and must outlive the context.  Waits for the context's stream; must not overlap a
 * generation.  hsd_layer_logits keeps using the shared head.  Errors: INVALID_ARG, CUDA. */
int hsd_set_exit_heads(hsd_ctx *ctx, const void *const *final_norms, const void *const *lm_heads);

/* Ablation of the appendix "Examining the assumptions of HSD": the verification rule of Algorithm 2 is
 * replaced by a biased coin per drafted token.  Level i+1 then accepts a draft iff the 24-bit uniform of that
 * accept test is below round(alphas[i] * 2^24) (the same counter-addressed uniform the real test uses; logits
 * play no part in the test).  The token drawn after the last accepted draft is still Algorithm 2's (residual of
 * the first rejected position, or the target row after t acceptances), so the output is no longer distributed as
 * the target's: a measurement mode, not a decoding mode.  The other half of that ablation, a fixed artificial
 * cost per forward, needs no kernel: it is the sum over levels of hsd_level_stats.forwards times a cost.
 *   alphas host [n_levels - 1], each in [0, 1]; NULL restores the real rule.  Errors: INVALID_ARG. */
int hsd_set_iid_acceptance(hsd_ctx *ctx, const double *alphas);

/* Generate n_new tokens per sequence with Algorithm 1 called at idx = K until enough tokens exist
 * (the first n_new are returned).  Sequence b produces exactly the tokens it would produce alone
 * with the same seed (uniforms are keyed by b).
 *   prompt_ids  device int32 [batch, prompt_len], prompt_len >= 1
 *   out_tokens  device int32 [batch, n_new]
 *   stats       host [n_levels] or NULL; overwritten
 *   timing_ms   host [2] or NULL: device time of the prompt pass and of the generation loop
 * Blocks until done (the host reads one accept count per verification).  Requires
 * prompt_len + n_new + sum(T) + n_levels + 1 <= max_seq and batch <= max_batch.
 * Errors: INVALID_ARG, OUT_OF_PAGES, CUDA, IO (trace file), DEVICE_TIMEOUT (a kernel gave up one of its
 * bounded waits: it raises a status word in the workspace that every later call of the context reports too;
 * the word is sticky, so a context that has returned DEVICE_TIMEOUT must be destroyed). */
int hsd_generate(hsd_ctx *ctx, const int32_t *prompt_ids, int batch, int prompt_len, int n_new, uint64_t seed,
                 void *stream, int32_t *out_tokens, hsd_level_stats *stats, double *timing_ms);

/* Decision log for parity checks: every level-0 call and every verification appends one binary
 * record to `path` (NULL closes the log).  Record = 12 int32 {0x48534454, level, sequence, serial,
 * context length, t, n, forward rows, logit rows, has_logits, vocab, dtype} + t drafted tokens (level 0:
 * the T_0 sampled tokens) + [level >= 1: the final token m] + [the call's own logit rows, raw, if
 * has_logits].  Logits are included for the first `logit_calls` records only. */
int hsd_set_trace(hsd_ctx *ctx, const char *path, int logit_calls);

void hsd_destroy(hsd_ctx *ctx);

/* ---------------------------------------------------------------------------------------
 * Expected latency per token of the chain M_0..M_K (Theorem 3.2):
 *   cost(0) = T_0 c_0;  cost(k) = gamma(alpha_{k-1,k}, T_{k-1}, T_k) (cost(k-1) + c_k), 0 < k < K;
 *   L = (1 - a) / (1 - a^(T_{K-1}+1)) (cost(K-1) + c_K), a = alpha_{K-1,K}.
 * gamma = expected draft/verify rounds until T_k tokens are collected under IID acceptance (the
 * paper estimates it empirically; this is a renewal computation over the per-round yield).
 *   costs host [n_levels], alphas host [n_levels-1] (alphas[i] = rate level i -> i+1), T host [n_levels-1].
 * hsd_search_T minimises L over T in [1, T_max]^(n_levels-1); monotone != 0 keeps the search
 * graph's constraint T_k >= T_{k-1} (Section 4.2, edge list).  Ties keep the lexicographically
 * first T.  Host-only; Errors: INVALID_ARG. */
int hsd_expected_latency(const double *costs, const double *alphas, int n_levels, const int32_t *T, double *out);
/* The same quantity for Algorithm 1 run as printed, under the same assumptions (IID acceptance, constant costs):
 * Theorem 3.2 lets every verifier see exactly T_{k-1} drafts per round, the algorithm hands it everything the
 * level below collected (T_{k-1} up to T_{k-1} + that level's last batch).  Exact renewal computation: the
 * distribution of the number of tokens each level returns is carried upward, cost_k = E[rounds] (cost_{k-1} + c_k)
 * (Wald), L = (cost_{K-1} + c_K) / E[tokens per target verification].  Equal to Theorem 3.2 for n_levels <= 2,
 * below it otherwise.  Same arguments and errors as hsd_expected_latency (T[i] <= 4096). */
int hsd_expected_latency_literal(const double *costs, const double *alphas, int n_levels, const int32_t *T, double *out);
int hsd_search_T(const double *costs, const double *alphas, int n_levels, int T_max, int monotone, int32_t *out_T,
                 double *out_latency);

/* ---------------------------------------------------------------------------------------
 * Latency-optimal hierarchy (Section 4.2, Corollary 4.1): among the ordered subsets sigma of the models
 * 0 .. n_models-1 that end in the target (model n_models-1) and the draft lengths T_k in [1, T_max] with
 * T_k >= T_{k-1}, the pair (sigma, T) with the smallest expected latency per token L(sigma, T).  The
 * paper's reduction graph (vertices = (model, batch size)) is acyclic once its self-loops are dropped, so
 * the cheapest path is found by a cost-to-go recursion, O(n_models^2 T_max^2) evaluations of gamma.
 *   costs host [n_models]: c_i, cost of one forward of model i (any unit);
 *   alpha host [n_models * n_models], row-major: alpha[i * n_models + j] = acceptance rate of drafter i
 *     under verifier j; only entries with i < j are read;
 *   out_sigma host [n_models]: the chosen models in ascending order, the last one is the target;
 *   out_n_levels host [1]: how many models were chosen (1 = the target alone);
 *   out_T host [n_models-1]: T_0 .. T_{n_levels-2} for the chosen chain (may be null when n_models = 1);
 *   out_latency host [1] or null.
 * Ties keep the first candidate in the order (smaller drafter index, smaller batch).  Host-only.
 * Errors: INVALID_ARG (null pointers, n_models outside 1..64, T_max outside 1..64, a rate outside [0, 1],
 * a negative or NaN cost). */
int hsd_search_hierarchy(const double *costs, const double *alpha, int n_models, int T_max, int32_t *out_sigma,
                         int32_t *out_n_levels, int32_t *out_T, double *out_latency);

/* ---------------------------------------------------------------------------------------
 * Logits of chosen exit layers at every position of one token sequence (the candidates of Section 4.2's
 * hierarchy search are early exits that share the target's final norm and output head, Section 5): one
 * causal pass over tokens 0 .. n_tokens-1; after each layer in `layers` the shared final norm and head are
 * applied to all rows.  Feeds hsd_pairwise_alpha.
 *   ctx: a context from hsd_create (any hierarchy over the same model); the call uses its workspace and
 *     resets its sequences and KV cache as a generation does, so it must not overlap one;
 *   token_ids device [n_tokens], 1 <= n_tokens <= 128 (and <= max_seq);
 *   layers host [n_sel]: exit layers, strictly ascending, each in 1 .. n_layers (n_layers = the full model);
 *   out_logits device [n_sel, n_tokens, vocab] in the model's storage dtype, written by the call;
 *   stream: the call returns after its work on the stream has completed.
 * Errors: INVALID_ARG, OUT_OF_PAGES, CUDA, DEVICE_TIMEOUT. */
int hsd_layer_logits(hsd_ctx *ctx, const int32_t *token_ids, int n_tokens, const int32_t *layers, int n_sel,
                     void *out_logits, void *stream);

/* ---------------------------------------------------------------------------------------
 * Calibration for the hierarchy search (Section 4.2 takes the acceptance rate alpha_{i,j} of every drafter
 * i under every verifier j as given; Section 2: alpha = 1 - TV(p_i, p_j) = sum_x min(p_i(x), p_j(x))).
 * From the logits of n_models models (exit layers) at the same n_rows positions, the n_models x n_models
 * matrix of the rates averaged over the positions: alpha[i][j] = mean_r sum_x min(softmax(l_i[r])(x),
 * softmax(l_j[r])(x)); symmetric, diagonal 1.  fp32 softmax (exp by the hardware approximation), sums in
 * fixed order (fp32 per 128 tokens, fp64 across), no atomics: repeatable bit for bit.
 *   logits device: model m's rows at logits + m * model_stride elements, each [n_rows, vocab] row-major,
 *     dtype HSD_F32 or HSD_BF16; model_stride >= n_rows * vocab;
 *   workspace device, 256-byte aligned, at least hsd_pairwise_alpha_workspace_bytes(...) (0 = bad sizes);
 *   alpha device [n_models * n_models] doubles, row-major, written by the call (asynchronously on stream).
 * The caller owns every buffer.  n_models <= 32.  Errors: INVALID_ARG (null, sizes, alignment, workspace too
 * small), TOO_LARGE (n_models beyond what one block's shared memory holds), CUDA. */
size_t hsd_pairwise_alpha_workspace_bytes(int n_models, int n_rows, int vocab);
int hsd_pairwise_alpha(const void *logits, int dtype, int n_models, int n_rows, int vocab, long long model_stride,
                       void *workspace, size_t workspace_bytes, double *alpha, void *stream);

/* ---------------------------------------------------------------------------------------
 * One weight-streaming matrix product of the verifier forward in isolation (the contraction
 * behind every projection of Algorithm 2's multi-row forward pass): out[r, n] = sum_k A[r, k] W[n, k],
 * bf16 inputs, fp32 accumulation on the tensor cores, fp32 output.
 *   A    device bf16 [R, K] row-major, 1 <= R <= 256, K a multiple of 64
 *   W    device bf16 [N, K] row-major
 *   out  device fp32 [R, N]
 *   workspace  device, 256-byte aligned, >= hsd_gemm_workspace_bytes(R, N, K); ignored on entry
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, UNSUPPORTED (no tensor-map support), CUDA,
 * DEVICE_TIMEOUT is reported by hsd_gemm_status after synchronising. */
size_t hsd_gemm_workspace_bytes(int R, int N, int K);
int hsd_gemm_bf16(const void *A, int R, int K, const void *W, int N, float *out, void *workspace, size_t workspace_bytes,
                  void *stream);
/* Synchronises `stream` and returns DEVICE_TIMEOUT if a kernel using `workspace` gave up a bounded wait. */
int hsd_gemm_status(void *workspace, void *stream);

/* Measurement aid: one read-only pass over `bytes` (a multiple of 16 is read) of device memory at `buffer` (16-byte
 * aligned) with plain vector loads on every SM, nothing written (`sink`, a device word or NULL, is written only if a
 * checksum happens to match a constant).  Timed with events around it, bytes / time is the HBM rate a weight-streaming
 * verification forward (Algorithm 2's pass: every weight byte read once) could reach at best; bench.py reports the
 * forward's rate against it.  Asynchronous on `stream`.  Errors: INVALID_ARG, CUDA. */
int hsd_stream_read(const void *buffer, size_t bytes, void *sink, void *stream);

/* Number of CUDA kernels this library has launched in the calling process so far. */
uint64_t hsd_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* HSD_H_ */
