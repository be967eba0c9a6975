// Host-side interface of the sampling kernels (used by the C entry points and by the engine).
#pragma once
#include "common.cuh"

namespace hsd {

constexpr int kSampleThreads = 1024;
constexpr int kStatThreads = 512;

// One row to draft-sample: token = sample(softmax(logits[logit_row])) -> out[out_index].
struct SampleRow {
  long long logit_row;
  long long out_index;
  u32 j, serial, seq, level;
};

// One sequence of a verification call.  Target rows p_1..p_{t+1} are rows p_row0.. of the target
// logits buffer, draft rows q_1..q_t rows q_row0.. of the draft buffer, drafted tokens
// tokens[tok_off .. tok_off + t).
struct VerifySeq {
  long long p_row0, q_row0, tok_off;
  int t;
  u32 serial, seq, level;
};

struct __align__(16) RowStat {
  float m;     // row maximum
  u32 Ex;      // integer weight of the drafted token in this row
  u64 S;       // sum of the integer weights
};

size_t verify_scratch_bytes(int batch, int t_max);

int launch_draft_sample(const void *logits, int dtype, int V, const SampleRow *desc, int n_rows, int regular_rows,
                        u32 regular_serial, u64 seed, int32_t *out, cudaStream_t s);

// coin24 != kNoCoin: the ablation of Appendix "Examining the assumptions": every accept test becomes a biased
// coin, accepted iff the test's own 24-bit uniform is below coin24 (= acceptance probability x 2^24).
constexpr u32 kNoCoin = 0xFFFFFFFFu;
// scratch: verify_scratch_bytes(batch, t_max) bytes, 16-byte aligned.  It starts with the counters and the
// decision queue of the fused kernel, which are cleared on the stream before the kernel.
int launch_verify(const void *p, const void *q, int32_t *tokens, int dtype, int V, int batch, int t_max,
                  const VerifySeq *desc, int regular_t, u32 regular_serial, u32 regular_level, void *scratch,
                  u64 seed, int32_t *out_tokens, int32_t *out_n, int write_in_place, cudaStream_t s,
                  u32 coin24 = kNoCoin);

}  // namespace hsd
