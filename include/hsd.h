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
  HSD_E_IO = -7
};
enum { HSD_F32 = 0, HSD_BF16 = 1 };

/* Text for a status code (static storage). */
const char *hsd_strerror(int status);

/* ---------------------------------------------------------------------------------------
 * Level-0 drafting, sampling step (Algorithm 1, base case: "new_token, new_prob <- M_0(...)").
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

#ifdef __cplusplus
}
#endif
#endif /* HSD_H_ */
