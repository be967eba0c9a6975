// Sampling kernels of the HSD hot path: level-0 draft sampling (Algorithm 1, base case) and the
// fused softmax-statistics / acceptance / residual-resample step (Algorithm 2; rule of Section 2).
#include "sampling.cuh"
#include "sampling_api.cuh"
#include "tc_ptx.cuh"
#include <algorithm>
#include <atomic>

namespace hsd {

// ------------------------------------------------------------------------------ draft sampling
// One block per row: token = inverse-CDF sample of softmax(row) with the purpose-0 uniform.
template <typename T>
__global__ void __launch_bounds__(kSampleThreads)
draft_sample_kernel(const T *__restrict__ logits, int V, const SampleRow *__restrict__ desc,
                    int regular_rows, u32 regular_serial, u64 seed, int32_t *__restrict__ out) {
  __shared__ float shf[32];
  __shared__ u64 sh64[34];
  SampleRow d;
  if (desc) {
    d = desc[blockIdx.x];
  } else {
    d.logit_row = blockIdx.x;
    d.out_index = blockIdx.x;
    d.j = blockIdx.x % regular_rows;
    d.seq = blockIdx.x / regular_rows;
    d.serial = regular_serial;
    d.level = 0;
  }
  const T *row = logits + (size_t)d.logit_row * V;
  u32 U = uniform24(seed, d.j, d.serial, d.level, PURPOSE_DRAFT, d.seq);
  int tok;
  if (sizeof(T) == 2 && chunk_layout_ok(row, V, blockDim.x)) {
    const int k0 = threadIdx.x * kChunkTokens;
    const Chunk32 c = chunk_load(reinterpret_cast<const __nv_bfloat16 *>(row), V, k0);
    const float m = block_max(chunk_max(c, V, k0), shf);
    tok = block_inverse_cdf_chunk(V, k0, U, [&](int i) { return (u64)exp_weight(chunk_get(c, i), m); }, sh64, nullptr);
  } else {
    float m = row_max(row, V, shf);
    tok = block_inverse_cdf(V, U, [&](int k) { return (u64)exp_weight(to_f32(row[k]), m); }, sh64, nullptr);
  }
  if (threadIdx.x == 0) out[d.out_index] = tok;
}

// ------------------------------------------------------------------------------ row statistics
// grid (2 * t_max + 1, batch).  Block (r, b): r <= t_max -> target row r; else draft row
// r - t_max - 1.  Writes the row maximum, the integer total S and the weight of the drafted token.
template <typename T>
__global__ void __launch_bounds__(kStatThreads)
row_stats_kernel(const T *__restrict__ p_logits, const T *__restrict__ q_logits, const int32_t *__restrict__ tokens,
                 int V, int t_max, const VerifySeq *__restrict__ desc, int regular_t, RowStat *__restrict__ stats) {
  __shared__ float shf[32];
  __shared__ u64 sh64[33];
  int b = blockIdx.y, r = blockIdx.x;
  VerifySeq d;
  if (desc) d = desc[b];
  else { d.t = regular_t; d.p_row0 = (long long)b * (regular_t + 1); d.q_row0 = (long long)b * regular_t; d.tok_off = (long long)b * regular_t; }
  const T *row;
  int tok = -1;
  if (r <= t_max) {
    if (r > d.t) return;
    row = p_logits + (size_t)(d.p_row0 + r) * V;
    if (r < d.t) tok = tokens[d.tok_off + r];
  } else {
    int j = r - t_max - 1;
    if (j >= d.t) return;
    row = q_logits + (size_t)(d.q_row0 + j) * V;
    tok = tokens[d.tok_off + j];
  }
  float m = row_max(row, V, shf);
  u64 local = 0;
  for (int k = threadIdx.x; k < V; k += blockDim.x) local += exp_weight(to_f32(row[k]), m);
  u64 total;
  block_exclusive_scan(local, sh64, &total);
  if (threadIdx.x == 0) {
    RowStat s;
    s.m = m;
    s.S = total;
    s.Ex = (tok >= 0 && tok < V) ? exp_weight(to_f32(row[tok]), m) : 0u;
    stats[(size_t)b * (2 * t_max + 1) + r] = s;
  }
}

// Same statistics with the whole row held in registers: 16-byte loads, one pass over HBM, packed
// arithmetic.  Needs V a multiple of the vector width, V <= 8 vectors per thread and 16-byte rows.
template <typename T> struct StatVec;
template <> struct StatVec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void unpack(const uint4 &v, float *f) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
  }
};
template <> struct StatVec<float> {
  static constexpr int N = 4;
  __device__ static void unpack(const uint4 &v, float *f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
};
constexpr int kStatVecPerThread = 8;

template <typename T>
__global__ void __launch_bounds__(kStatThreads)
row_stats_vec_kernel(const T *__restrict__ p_logits, const T *__restrict__ q_logits, const int32_t *__restrict__ tokens,
                     int V, int t_max, const VerifySeq *__restrict__ desc, int regular_t, RowStat *__restrict__ stats) {
  constexpr int VN = StatVec<T>::N;
  __shared__ float shf[32];
  __shared__ u64 sh64[33];
  int b = blockIdx.y, r = blockIdx.x;
  VerifySeq d;
  if (desc) d = desc[b];
  else { d.t = regular_t; d.p_row0 = (long long)b * (regular_t + 1); d.q_row0 = (long long)b * regular_t; d.tok_off = (long long)b * regular_t; }
  const T *row;
  int tok = -1;
  if (r <= t_max) {
    if (r > d.t) return;
    row = p_logits + (size_t)(d.p_row0 + r) * V;
    if (r < d.t) tok = tokens[d.tok_off + r];
  } else {
    int j = r - t_max - 1;
    if (j >= d.t) return;
    row = q_logits + (size_t)(d.q_row0 + j) * V;
    tok = tokens[d.tok_off + j];
  }
  const int nvec = V / VN;
  const uint4 *row4 = reinterpret_cast<const uint4 *>(row);
  uint4 regs[kStatVecPerThread];
#pragma unroll
  for (int j = 0; j < kStatVecPerThread; ++j) {
    const int iv = threadIdx.x + kStatThreads * j;
    regs[j] = iv < nvec ? __ldg(row4 + iv) : make_uint4(0u, 0u, 0u, 0u);
  }
  float m = -INFINITY;
#pragma unroll
  for (int j = 0; j < kStatVecPerThread; ++j) {
    if ((int)threadIdx.x + kStatThreads * j < nvec) {
      float f[VN];
      StatVec<T>::unpack(regs[j], f);
#pragma unroll
      for (int e = 0; e < VN; ++e) m = fmaxf(m, f[e]);
    }
  }
  m = block_max(m, shf);
  u64 local = 0;
#pragma unroll
  for (int j = 0; j < kStatVecPerThread; ++j) {
    if ((int)threadIdx.x + kStatThreads * j < nvec) {
      float f[VN];
      StatVec<T>::unpack(regs[j], f);
#pragma unroll
      for (int e = 0; e < VN; e += 2) {
        u32 e0, e1;
        exp_weight2(f[e], f[e + 1], m, e0, e1);
        local += (u64)e0 + (u64)e1;
      }
    }
  }
  u64 total;
  block_exclusive_scan(local, sh64, &total);
  if (threadIdx.x == 0) {
    RowStat s;
    s.m = m;
    s.S = total;
    s.Ex = (tok >= 0 && tok < V) ? exp_weight(to_f32(row[tok]), m) : 0u;
    stats[(size_t)b * (2 * t_max + 1) + r] = s;
  }
}

// ------------------------------------------------------------------------------ decision
// One block per sequence: accept tests for all positions (each with its own counter-addressed
// uniform, so the parallel form equals Algorithm 2's sequential loop with break), n = index of the
// first rejection, then the final draw from the residual of row n (n < t) or from target row t.
template <typename T>
__global__ void __launch_bounds__(kSampleThreads)
decide_kernel(const T *__restrict__ p_logits, const T *__restrict__ q_logits, int32_t *__restrict__ tokens, int V,
              int t_max, const VerifySeq *__restrict__ desc, int regular_t, u32 regular_serial, u32 regular_level,
              const RowStat *__restrict__ stats, u64 seed, int32_t *__restrict__ out_tokens /*[B, t_max+1] or null*/,
              int32_t *__restrict__ out_n /*[B]*/, int write_in_place, u32 coin24) {
  __shared__ u64 sh64[34];
  __shared__ int sh_first_reject;
  int b = blockIdx.x;
  VerifySeq d;
  if (desc) d = desc[b];
  else {
    d.t = regular_t; d.p_row0 = (long long)b * (regular_t + 1); d.q_row0 = (long long)b * regular_t;
    d.tok_off = (long long)b * regular_t; d.serial = regular_serial; d.seq = b; d.level = regular_level;
  }
  const RowStat *st = stats + (size_t)b * (2 * t_max + 1);
  if (threadIdx.x == 0) sh_first_reject = d.t;
  __syncthreads();
  if ((int)threadIdx.x < d.t) {
    int j = threadIdx.x;
    RowStat sp = st[j], sq = st[t_max + 1 + j];
    u64 Pp = fixed_prob(sp.Ex, prob_scale(sp.S));
    u64 Pq = fixed_prob(sq.Ex, prob_scale(sq.S));
    u32 U = uniform24(seed, j, d.serial, d.level, PURPOSE_ACCEPT, d.seq);
    bool ok = (((u64)U * Pq) >> 24) < Pp;                 // u < p(x) / q(x)
    if (coin24 != kNoCoin) ok = U < coin24;               // ablation: IID acceptance with a fixed probability
    if (!ok) atomicMin(&sh_first_reject, j);
  }
  __syncthreads();
  int n = sh_first_reject;
  u32 U = uniform24(seed, 0, d.serial, d.level, PURPOSE_FINAL, d.seq);
  const T *prow = p_logits + (size_t)(d.p_row0 + n) * V;
  float mp = st[n].m;
  int m_tok = -1;
  const bool fast = sizeof(T) == 2 && chunk_layout_ok(prow, V, blockDim.x) &&
                    (n >= d.t || chunk_layout_ok(q_logits + (size_t)(d.q_row0 + n) * V, V, blockDim.x));
  if (fast) {
    const int k0 = threadIdx.x * kChunkTokens;
    const Chunk32 cp = chunk_load(reinterpret_cast<const __nv_bfloat16 *>(prow), V, k0);
    if (n < d.t) {
      const Chunk32 cq = chunk_load(reinterpret_cast<const __nv_bfloat16 *>(q_logits + (size_t)(d.q_row0 + n) * V), V, k0);
      const float mq = st[t_max + 1 + n].m;
      const ProbScale psp = prob_scale(st[n].S), psq = prob_scale(st[t_max + 1 + n].S);
      m_tok = block_inverse_cdf_chunk(V, k0, U, [&](int i) {
        u64 Pp = fixed_prob(exp_weight(chunk_get(cp, i), mp), psp);
        u64 Pq = fixed_prob(exp_weight(chunk_get(cq, i), mq), psq);
        return Pp > Pq ? Pp - Pq : 0ull;
      }, sh64, nullptr);
    }
    if (m_tok < 0)
      m_tok = block_inverse_cdf_chunk(V, k0, U, [&](int i) { return (u64)exp_weight(chunk_get(cp, i), mp); }, sh64, nullptr);
  } else if (n < d.t) {
    const T *qrow = q_logits + (size_t)(d.q_row0 + n) * V;
    float mq = st[t_max + 1 + n].m;
    ProbScale psp = prob_scale(st[n].S), psq = prob_scale(st[t_max + 1 + n].S);
    m_tok = block_inverse_cdf(V, U, [&](int k) {
      u64 Pp = fixed_prob(exp_weight(to_f32(prow[k]), mp), psp);
      u64 Pq = fixed_prob(exp_weight(to_f32(qrow[k]), mq), psq);
      return Pp > Pq ? Pp - Pq : 0ull;
    }, sh64, nullptr);
  }
  if (!fast && m_tok < 0)   // bonus token, or an all-zero residual: draw from the verifier's own row
    m_tok = block_inverse_cdf(V, U, [&](int k) { return (u64)exp_weight(to_f32(prow[k]), mp); }, sh64, nullptr);
  if (threadIdx.x == 0) {
    out_n[b] = n;
    if (write_in_place) tokens[d.tok_off + n] = m_tok;
  }
  if (out_tokens) {
    for (int j = threadIdx.x; j <= t_max; j += blockDim.x) {
      int v = -1;
      if (j < n) v = tokens[d.tok_off + j];
      else if (j == n) v = m_tok;
      out_tokens[(size_t)b * (t_max + 1) + j] = v;
    }
  }
}

// ------------------------------------------------------------------------------ fused verification
// Algorithm 2's decision in ONE launch for bf16 rows: statistics of all p and q rows, the accept tests and the
// final draw.  Persistent grid, one CTA per SM: a producer thread streams the CTA's rows into a shared-memory
// ring with bulk copies (so HBM latency hides under the other rows' arithmetic, which is what bounds this
// kernel: ~16 issue slots per logit for the unfused fp32 exp and the 64-bit sums); the 1024 threads take a row
// into registers, thread 0 refills the slot with the row three items ahead, and the row is reduced to (max,
// integer total, weight of the drafted token).
// Rows are dealt round-robin in sequence-major order, so a sequence's rows finish at about the same time on
// different SMs; the CTA that delivers a sequence's last row (a counter per sequence) takes that sequence's
// decision while the rows it needs are still in L2.  No CTA ever waits for another.
constexpr int kFusedConsumers = 1024;
constexpr int kFusedThreads = kFusedConsumers;
constexpr int kFusedSlots = 3;
constexpr int kFusedVecPerThread = 8;                      // 16-byte vectors of a row per thread of a 512-thread group
constexpr int kFusedMaxV = 512 * kFusedVecPerThread * 8;
constexpr uint32_t kFusedPiece = 4096;                     // bytes per bulk copy; 32 of them cover the largest row
using FusedGroup = WholeBlock;

struct FusedArgs {
  const __nv_bfloat16 *p, *q;
  int32_t *tokens;
  int V, t_max, batch;
  const VerifySeq *desc;
  int regular_t;
  u32 regular_serial, regular_level;
  RowStat *stats;
  unsigned *counters;            // zero on entry: [batch] rows delivered per sequence | queue length | tickets drawn |
                                 // [batch] queue of sequences ready for their decision (b + 1)
  u64 seed;
  int32_t *out_tokens, *out_n;
  int write_in_place;
  u32 coin24;
  int *status;                   // optional: set to 1 if a bounded wait gave up
};

__device__ __forceinline__ VerifySeq fused_seq(const FusedArgs &a, int b) {
  VerifySeq d;
  if (a.desc) return a.desc[b];
  d.t = a.regular_t; d.p_row0 = (long long)b * (a.regular_t + 1); d.q_row0 = (long long)b * a.regular_t;
  d.tok_off = (long long)b * a.regular_t; d.serial = a.regular_serial; d.seq = b; d.level = a.regular_level;
  return d;
}

__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Inverse CDF over weight(i) of the thread's own 32 tokens, as block_inverse_cdf_chunk, except that the walk
// through the owning thread's chunk is done by warp 0 together: lane i recomputes the weight of the chunk's
// token i from global memory (weight_at(k)), a warp scan finds the first token whose inclusive sum passes the
// threshold.  Integer weights, so the recomputed values are the same.
template <class WeightFn, class WeightAt>
__device__ __forceinline__ int fused_inverse_cdf(int V, int k0, u32 U, WeightFn weight, WeightAt weight_at, u64 *sh64 /*[34]*/,
                                                 int *sh_owner) {
  u64 local = 0;
#pragma unroll
  for (int i = 0; i < kChunkTokens; ++i)
    if (k0 + i < V) local += weight(i);
  u64 total;
  const u64 excl = block_exclusive_scan<FusedGroup>(local, sh64, &total);
  if (total == 0) return -1;                               // uniform
  const u64 tau = cdf_threshold(U, total);
  if (tau >= excl && tau < excl + local) {                 // exactly one thread
    *sh_owner = threadIdx.x;
    sh64[33] = excl;
  }
  FusedGroup::sync();
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x, k = *sh_owner * kChunkTokens + lane;
    u64 c = k < V ? weight_at(k) : 0ull;
    for (int o = 1; o < 32; o <<= 1) {
      const u64 n = __shfl_up_sync(0xFFFFFFFFu, c, o);
      if (lane >= o) c += n;
    }
    const unsigned hit = __ballot_sync(0xFFFFFFFFu, c + sh64[33] > tau && k < V);
    if (lane == 0) *sh_owner = *sh_owner * kChunkTokens + (__ffs(hit) - 1);
  }
  FusedGroup::sync();
  const int r = *sh_owner;
  FusedGroup::sync();
  return r;
}

// The decision of sequence b (the whole CTA): accept tests on the row statistics, then the final draw from the
// residual of the first rejected position, or from the last target row.
__device__ __forceinline__ void fused_decide(const FusedArgs &a, int b, const VerifySeq &d, u64 *sh64, int *sh_int /*[2]*/) {
  const int tid = threadIdx.x, V = a.V, t_max = a.t_max;
  const RowStat *st = a.stats + (size_t)b * (2 * t_max + 1);
  if (tid == 0) sh_int[1] = d.t;
  FusedGroup::sync();
  if (tid < d.t) {
    const int j = tid;
    const float4 rp = __ldcg(reinterpret_cast<const float4 *>(st + j)), rq = __ldcg(reinterpret_cast<const float4 *>(st + t_max + 1 + j));
    const RowStat sp = *reinterpret_cast<const RowStat *>(&rp), sq = *reinterpret_cast<const RowStat *>(&rq);
    const u64 Pp = fixed_prob(sp.Ex, prob_scale(sp.S)), Pq = fixed_prob(sq.Ex, prob_scale(sq.S));
    const u32 U = uniform24(a.seed, j, d.serial, d.level, PURPOSE_ACCEPT, d.seq);
    bool ok = (((u64)U * Pq) >> 24) < Pp;                  // u < p(x) / q(x)
    if (a.coin24 != kNoCoin) ok = U < a.coin24;            // ablation: IID acceptance with a fixed probability
    if (!ok) atomicMin(&sh_int[1], j);
  }
  FusedGroup::sync();
  const int n = sh_int[1];
  FusedGroup::sync();                                      // sh_int[1] is reused by the draw
  const u32 U = uniform24(a.seed, 0, d.serial, d.level, PURPOSE_FINAL, d.seq);
  const __nv_bfloat16 *prow = a.p + (size_t)(d.p_row0 + n) * V;
  const float4 rpn = __ldcg(reinterpret_cast<const float4 *>(st + n));
  const RowStat spn = *reinterpret_cast<const RowStat *>(&rpn);
  const float mp = spn.m;
  const int k0 = tid * kChunkTokens;
  const Chunk32 cp = chunk_load(prow, V, k0);
  int m_tok = -1;
  if (n < d.t) {
    const __nv_bfloat16 *qrow = a.q + (size_t)(d.q_row0 + n) * V;
    const Chunk32 cq = chunk_load(qrow, V, k0);
    const float4 rqn = __ldcg(reinterpret_cast<const float4 *>(st + t_max + 1 + n));
    const RowStat sqn = *reinterpret_cast<const RowStat *>(&rqn);
    const ProbScale psp = prob_scale(spn.S), psq = prob_scale(sqn.S);
    const float mq = sqn.m;
    auto residual = [&](float lp, float lq) {                // both rows' weights in one packed evaluation
      u32 ep, eq;
      exp_weight2m(lp, lq, mp, mq, ep, eq);
      const u64 Pp = fixed_prob(ep, psp), Pq = fixed_prob(eq, psq);
      return Pp > Pq ? Pp - Pq : 0ull;
    };
    m_tok = fused_inverse_cdf(V, k0, U, [&](int i) { return residual(chunk_get(cp, i), chunk_get(cq, i)); },
                              [&](int k) { return residual(__bfloat162float(prow[k]), __bfloat162float(qrow[k])); }, sh64, &sh_int[1]);
  }
  if (m_tok < 0)   // bonus token, or an all-zero residual: draw from the verifier's own row
    m_tok = fused_inverse_cdf(V, k0, U, [&](int i) { return (u64)exp_weight(chunk_get(cp, i), mp); },
                              [&](int k) { return (u64)exp_weight(__bfloat162float(prow[k]), mp); }, sh64, &sh_int[1]);
  if (tid == 0) {
    a.out_n[b] = n;
    if (a.write_in_place) a.tokens[d.tok_off + n] = m_tok;
  }
  if (a.out_tokens) {
    for (int j = tid; j <= t_max; j += kFusedConsumers) {
      int v = -1;
      if (j < n) v = a.tokens[d.tok_off + j];
      else if (j == n) v = m_tok;
      a.out_tokens[(size_t)b * (t_max + 1) + j] = v;
    }
  }
}

__global__ void __launch_bounds__(kFusedThreads, 1) verify_fused_kernel(const __grid_constant__ FusedArgs a) {
  extern __shared__ uint8_t fused_smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(fused_smem_raw) + 127) & ~(uintptr_t)127);
  const uint32_t row_bytes = (uint32_t)a.V * 2u, slot_bytes = (row_bytes + 127u) & ~127u;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)kFusedSlots * slot_bytes);   // full[S][2]
  __shared__ float shf[2][16];
  __shared__ u64 sh64[34];                   // row phase: [g * 16 + warp]; decisions: the block scan's scratch
  __shared__ int sh_flag[2];
  __shared__ int sh_abort;
  const uint32_t bar0 = ptx::smem_u32(bars);
  const int tid = threadIdx.x, lane = tid & 31;
  const int rows_per_seq = 2 * a.t_max + 1, n_items = a.batch * rows_per_seq;
  if (tid == 0) {
    for (int s = 0; s < 2 * kFusedSlots; ++s) ptx::mbar_init(bar0 + 8u * s, 1);
    sh_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int *abort_flag = &sh_abort;
  // item i = (sequence b, row r): r <= t_max: target row r (valid if r <= t_b); else draft row r - t_max - 1 (valid if < t_b)
  auto row_of = [&](int i, VerifySeq &d, int &b, int &r) -> const __nv_bfloat16 * {
    b = i / rows_per_seq; r = i - b * rows_per_seq;
    d = fused_seq(a, b);
    if (r <= a.t_max) return r <= d.t ? a.p + (size_t)(d.p_row0 + r) * a.V : nullptr;
    const int j = r - a.t_max - 1;
    return j < d.t ? a.q + (size_t)(d.q_row0 + j) * a.V : nullptr;
  };
  // Rows.  The CTA's valid items, numbered k = 0, 1, ..., go to its two groups of 512 threads in turn (group
  // k & 1) through ring slot k % 3; each group has its own barrier, so one group's reductions and global round
  // trips run under the other group's arithmetic.  The group that has taken item k out of its slot asks for item
  // k + 3 (4 KiB bulk copies, one per lane of the group's first warp: a single 64 KB copy runs at a fraction
  // of an SM's bandwidth).
  const int grp = tid >> 9, gtid = tid & 511, gwarp = gtid >> 5, bar_id = 1 + grp;
  auto group_sync = [&]() { asm volatile("bar.sync %0, 512;" ::"r"(bar_id) : "memory"); };
  // A slot's uses alternate between the groups, and a parity wait tells a barrier's phases apart only one phase
  // back, so each slot has two "full" barriers used in turn: a barrier's phases then all belong to one group, which
  // takes them in order.
  auto full_bar = [&](int k) { return bar0 + 8u * (uint32_t)((k % kFusedSlots) * 2 + ((k / kFusedSlots) & 1)); };
  int f_idx = blockIdx.x, f_ord = 0;                        // fetch cursor: next item index to look at, valid items passed so far
  auto fetch_ordinal = [&](int want) {                      // all lanes of a warp; asks for valid item number `want`, if it exists
    while (f_idx < n_items) {
      VerifySeq d; int b, r;
      const __nv_bfloat16 *row = row_of(f_idx, d, b, r);
      f_idx += gridDim.x;
      if (!row) continue;
      if (f_ord++ < want) continue;
      const int slot = want % kFusedSlots;
      const uint32_t bar = full_bar(want);
      if (lane == 0) ptx::mbar_expect_tx(bar, row_bytes);
      __syncwarp();
      const uint32_t off = (uint32_t)lane * kFusedPiece;
      if (off < row_bytes)
        bulk_load_row(ptx::smem_u32(smem + (size_t)slot * slot_bytes) + off, reinterpret_cast<const uint8_t *>(row) + off,
                      min(kFusedPiece, row_bytes - off), bar);
      return;
    }
  };
  if (tid < 32) {                                           // items 0, 1, 2; afterwards group 0 asks for 3, 5, ..., group 1 for 4, 6, ...
    for (int k = 0; k < kFusedSlots; ++k) fetch_ordinal(k);
    f_idx = blockIdx.x; f_ord = 0;                          // group 0's own cursor starts over (its next request is item 3)
  }
  const int nvec = a.V >> 3;
  int ord = 0;                                              // valid items of this CTA seen so far
  unsigned pending_before = 0u, pending_last = 0xFFFFFFFFu; // the row counter's old value of the group's previous item (thread 0 of the group)
  int pending_b = -1;
  auto settle = [&]() {                                     // group thread 0: was the previous item its sequence's last row?
    if (pending_b >= 0 && pending_before == pending_last) {
      // the sequence is ready for its decision: append it to the queue (entry = b + 1; 0 = not yet written)
      const unsigned at = atomicAdd(&a.counters[a.batch], 1u);
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(a.counters + a.batch + 2 + at), "r"((unsigned)pending_b + 1u) : "memory");
    }
    pending_b = -1;
  };
  for (int i = blockIdx.x; i < n_items; i += gridDim.x) {
    VerifySeq d; int b, r;
    const __nv_bfloat16 *row = row_of(i, d, b, r);
    if (!row) continue;
    const int k = ord++;
    if ((k & 1) != grp) continue;
    const int s = k % kFusedSlots;
    const uint32_t par = (uint32_t)(k / (2 * kFusedSlots)) & 1u;
    // the drafted token's logit (the group's thread 0 only), asked for before the wait
    int tok = -1;
    if (r < d.t) tok = a.tokens[d.tok_off + r];
    else if (r > a.t_max) tok = a.tokens[d.tok_off + (r - a.t_max - 1)];
    float l_tok = 0.f;
    const bool has_tok = tok >= 0 && tok < a.V;
    if (gtid == 0 && has_tok) l_tok = __bfloat162float(row[tok]);
    if (lane == 0) ptx::mbar_wait(full_bar(k), par, abort_flag);       // a give-up raises the CTA's abort flag
    __syncwarp();
    const uint4 *src = reinterpret_cast<const uint4 *>(smem + (size_t)s * slot_bytes);
    uint4 regs[kFusedVecPerThread];
#pragma unroll
    for (int j = 0; j < kFusedVecPerThread; ++j) {
      const int iv = gtid + 512 * j;
      regs[j] = iv < nvec ? src[iv] : make_uint4(0u, 0u, 0u, 0u);
    }
    group_sync();                                           // every thread holds its part of the row: the slot is free
    if (*abort_flag) break;                                 // uniform over the group: raised before the barrier
    if (gwarp == 0) fetch_ordinal(k + kFusedSlots);
    // the row maximum on the packed pairs (the maximum of bf16 values is one of them: exact)
    __nv_bfloat162 mx2 = __floats2bfloat162_rn(-INFINITY, -INFINITY);
#pragma unroll
    for (int j = 0; j < kFusedVecPerThread; ++j) {
      if (gtid + 512 * j < nvec) {
        const uint4 r4 = regs[j];
        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162 *>(&r4.x));
        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162 *>(&r4.y));
        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162 *>(&r4.z));
        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162 *>(&r4.w));
      }
    }
    float m = fmaxf(__low2float(mx2), __high2float(mx2));
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (lane == 0) shf[grp][gwarp] = m;
    group_sync();
    m = shf[grp][lane & 15];
    for (int o = 8; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    u64 local = 0;
#pragma unroll
    for (int j = 0; j < kFusedVecPerThread; ++j) {
      if (gtid + 512 * j < nvec) {
        float f[8];
        StatVec<__nv_bfloat16>::unpack(regs[j], f);
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          u32 e0, e1;
          exp_weight2(f[e], f[e + 1], m, e0, e1);
          local += (u64)e0 + (u64)e1;
        }
      }
    }
    for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xFFFFFFFFu, local, o);
    if (lane == 0) sh64[grp * 16 + gwarp] = local;
    group_sync();
    if (gtid == 0) {
      u64 total = 0;
#pragma unroll
      for (int w = 0; w < 16; ++w) total += sh64[grp * 16 + w];
      settle();                                             // the previous item's counter value has long arrived
      RowStat st;
      st.m = m; st.S = total; st.Ex = has_tok ? exp_weight(l_tok, m) : 0u;
      a.stats[(size_t)b * rows_per_seq + r] = st;
      // the statistics are ordered before the count by the release (and the other rows' statistics before whatever
      // follows a look at its old value, which happens one item later, by the acquire)
      asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(pending_before) : "l"(a.counters + b) : "memory");
      pending_b = b;
      pending_last = (unsigned)(2 * d.t);                   // 2 t + 1 rows per sequence
    }
    // (the next item's first barrier keeps the other threads from overwriting sh64 / shf before thread 0 has read them)
  }
  if (gtid == 0) settle();
  // Decisions.  Taking one where its last row arrives would chain: the CTA that decides delivers its next rows
  // late, so it is the last arriver of those sequences too.  Instead every CTA, once its rows are done, draws
  // tickets until all `batch` decisions are handed out; a ticket whose entry is not written yet waits for it
  // (bounded): the rows it waits for are never this CTA's own.
  for (;;) {
    __syncthreads();
    if (tid == 0) {
      int b = -1;
      if (!*abort_flag) {
        const unsigned t = atomicAdd(&a.counters[a.batch + 1], 1u);
        if (t < (unsigned)a.batch) {
          const unsigned *entry = a.counters + a.batch + 2 + t;
          unsigned v = 0;
          unsigned long long t0 = 0;
          for (uint32_t it = 0;; ++it) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(entry) : "memory");
            if (v != 0u) break;
            if ((it & 31u) == 31u) {
              const unsigned long long now = ptx::globaltimer_ns();
              if (t0 == 0) t0 = now;
              if (now - t0 > ptx::kWaitLimitNs) { *abort_flag = 1; break; }
            }
          }
          if (v != 0u) b = (int)v - 1;
        }
      }
      sh_flag[0] = b;
    }
    __syncthreads();
    const int b = sh_flag[0];
    if (b < 0) break;
    const VerifySeq d = fused_seq(a, b);
    fused_decide(a, b, d, sh64, sh_flag);
  }
  if (tid == 0 && sh_abort) {
    // copies already asked for must land before the CTA's shared memory goes away (bounded)
    const unsigned long long t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 20000ull) {}      // 20 us: far longer than a row's copy takes
    if (a.status) atomicExch(a.status, 1);
  }
}

// ------------------------------------------------------------------------------ host launchers
// Scratch of one verification call: [counter per sequence (fused kernel)] [RowStat per logits row].
static size_t verify_counter_bytes(int batch) { return ((size_t)(2 * batch + 2) * 4 + 255) / 256 * 256; }
size_t verify_scratch_bytes(int batch, int t_max) {
  return verify_counter_bytes(batch) + (size_t)batch * (2 * t_max + 1) * sizeof(RowStat);
}

template <typename T>
static int launch_draft_sample_t(const void *logits, int V, const SampleRow *desc, int n_rows, int regular_rows,
                                 u32 regular_serial, u64 seed, int32_t *out, cudaStream_t s) {
  draft_sample_kernel<T><<<n_rows, kSampleThreads, 0, s>>>((const T *)logits, V, desc, regular_rows, regular_serial, seed, out);
  hsd_count_launches(1);
  return hsd_launch_status();
}

int launch_draft_sample(const void *logits, int dtype, int V, const SampleRow *desc, int n_rows, int regular_rows,
                        u32 regular_serial, u64 seed, int32_t *out, cudaStream_t s) {
  if (n_rows == 0) return HSD_OK;
  return dtype == HSD_BF16
             ? launch_draft_sample_t<__nv_bfloat16>(logits, V, desc, n_rows, regular_rows, regular_serial, seed, out, s)
             : launch_draft_sample_t<float>(logits, V, desc, n_rows, regular_rows, regular_serial, seed, out, s);
}

template <typename T>
static int launch_verify_t(const void *p, const void *q, int32_t *tokens, int V, int batch, int t_max,
                           const VerifySeq *desc, int regular_t, u32 regular_serial, u32 regular_level, RowStat *stats,
                           u64 seed, int32_t *out_tokens, int32_t *out_n, int write_in_place, cudaStream_t s, u32 coin24) {
  dim3 grid(2 * t_max + 1, batch);
  constexpr int VN = StatVec<T>::N;
  const bool vec_ok = V % VN == 0 && V / VN <= kStatVecPerThread * kStatThreads && ((uintptr_t)p & 15) == 0 &&
                      (q == nullptr || ((uintptr_t)q & 15) == 0);
  if (vec_ok)
    row_stats_vec_kernel<T><<<grid, kStatThreads, 0, s>>>((const T *)p, (const T *)q, tokens, V, t_max, desc, regular_t, stats);
  else
    row_stats_kernel<T><<<grid, kStatThreads, 0, s>>>((const T *)p, (const T *)q, tokens, V, t_max, desc, regular_t, stats);
  if (cudaGetLastError() != cudaSuccess) return HSD_E_CUDA;
  decide_kernel<T><<<batch, kSampleThreads, 0, s>>>((const T *)p, (const T *)q, tokens, V, t_max, desc, regular_t,
                                                   regular_serial, regular_level, stats, seed, out_tokens, out_n,
                                                   write_in_place, coin24);
  hsd_count_launches(2);
  return hsd_launch_status();
}

static int fused_sm_count() {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    sms = n;
  }
  return sms;
}

int launch_verify(const void *p, const void *q, int32_t *tokens, int dtype, int V, int batch, int t_max,
                  const VerifySeq *desc, int regular_t, u32 regular_serial, u32 regular_level, void *scratch,
                  u64 seed, int32_t *out_tokens, int32_t *out_n, int write_in_place, cudaStream_t s,
                  u32 coin24) {
  if (batch == 0) return HSD_OK;
  unsigned *counters = (unsigned *)scratch;
  RowStat *stats = (RowStat *)((char *)scratch + verify_counter_bytes(batch));
  // bf16 rows that a bulk copy can fetch (16-byte multiples) and 1024 threads can hold: one fused launch
  const size_t slot = ((size_t)V * 2 + 127) / 128 * 128, smem = kFusedSlots * slot + 2 * kFusedSlots * 8 + 128;
  const bool fused = dtype == HSD_BF16 && V % 8 == 0 && V <= kFusedMaxV && smem <= 220 * 1024 && ((uintptr_t)p & 15) == 0 &&
                     (q == nullptr || ((uintptr_t)q & 15) == 0) && t_max < kFusedConsumers;
  if (fused) {
    static bool attr_set = false;
    if (!attr_set) {
      HSD_CUDA_OK(cudaFuncSetAttribute(verify_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
      attr_set = true;
    }
    HSD_CUDA_OK(cudaMemsetAsync(counters, 0, verify_counter_bytes(batch), s));
    FusedArgs a;
    a.p = (const __nv_bfloat16 *)p; a.q = (const __nv_bfloat16 *)q; a.tokens = tokens; a.V = V; a.t_max = t_max; a.batch = batch;
    a.desc = desc; a.regular_t = regular_t; a.regular_serial = regular_serial; a.regular_level = regular_level;
    a.stats = stats; a.counters = counters; a.seed = seed; a.out_tokens = out_tokens; a.out_n = out_n;
    a.write_in_place = write_in_place; a.coin24 = coin24; a.status = nullptr;
    const int n_items = batch * (2 * t_max + 1);
    verify_fused_kernel<<<std::min(fused_sm_count(), n_items), kFusedThreads, smem, s>>>(a);
    hsd_count_launches(1);
    return hsd_launch_status();
  }
  return dtype == HSD_BF16 ? launch_verify_t<__nv_bfloat16>(p, q, tokens, V, batch, t_max, desc, regular_t, regular_serial,
                                                            regular_level, stats, seed, out_tokens, out_n, write_in_place, s, coin24)
                           : launch_verify_t<float>(p, q, tokens, V, batch, t_max, desc, regular_t, regular_serial,
                                                    regular_level, stats, seed, out_tokens, out_n, write_in_place, s, coin24);
}

// ------------------------------------------------------------------------------ static scratch
// Scratch for hsd_verify_level_static: lives in the library image, so every GPU that loads the
// library holds these bytes until the process exits.  One RowStat per logits row of a call.
constexpr int kStaticStatRows = 4096;                       // 64 KiB of row statistics + 32.25 KiB of counters and queue
constexpr size_t kStaticScratchBytes = kStaticStatRows * sizeof(RowStat) + ((2 * kStaticStatRows + 2) * 4 + 255) / 256 * 256;
static __device__ __align__(256) unsigned char g_static_verify_scratch[kStaticScratchBytes];

// In host code the array's name is only a stand-in for the symbol, not a device address: the
// address has to be asked for, once per device, with that device current.  The answer is kept per
// device in an atomic (two host threads may make a device's first call at once: both look the
// symbol up and store the same value).  It does not survive cudaDeviceReset(): a process that
// resets a device must not use this entry point on it afterwards.
static std::atomic<void *> g_static_scratch_ptr[64];
static int static_scratch_address(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HSD_E_CUDA;
  void *p = g_static_scratch_ptr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_static_verify_scratch) != cudaSuccess || !p) return HSD_E_CUDA;
    g_static_scratch_ptr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return HSD_OK;
}

}  // namespace hsd

// ------------------------------------------------------------------------------ C ABI
unsigned long long g_hsd_launches = 0;

extern "C" {

uint64_t hsd_kernel_launches(void) { return g_hsd_launches; }

const char *hsd_strerror(int status) {
  switch (status) {
    case HSD_OK: return "ok";
    case HSD_E_INVALID_ARG: return "invalid argument";
    case HSD_E_WORKSPACE_TOO_SMALL: return "workspace too small";
    case HSD_E_OUT_OF_PAGES: return "out of KV pages";
    case HSD_E_CUDA: return "CUDA error";
    case HSD_E_DEVICE_TIMEOUT: return "device-side wait timed out";
    case HSD_E_UNSUPPORTED: return "unsupported configuration";
    case HSD_E_IO: return "I/O error";
    case HSD_E_TOO_LARGE: return "request exceeds the built-in scratch capacity";
    default: return "unknown status";
  }
}

int hsd_draft_sample(const void *logits, int batch, int rows, int vocab, int dtype, uint64_t seed,
                     uint64_t call_serial, void *stream, int32_t *out_tokens) {
  if (!logits || !out_tokens || batch <= 0 || rows <= 0 || vocab <= 0) return HSD_E_INVALID_ARG;
  if (dtype != HSD_F32 && dtype != HSD_BF16) return HSD_E_INVALID_ARG;
  if ((long long)batch * rows > 0x7FFFFFFFll) return HSD_E_INVALID_ARG;
  return hsd::launch_draft_sample(logits, dtype, vocab, nullptr, batch * rows, rows, (u32)call_serial, seed, out_tokens,
                                  (cudaStream_t)stream);
}

size_t hsd_verify_workspace_bytes(int batch, int t) {
  if (batch <= 0 || t < 0) return 0;
  return hsd::verify_scratch_bytes(batch, t);
}

int hsd_verify_level(int level, const void *target_logits, const void *draft_logits, const int32_t *draft_tokens,
                     int batch, int t, int vocab, int dtype, uint64_t seed, uint64_t call_serial, void *workspace,
                     size_t workspace_bytes, void *stream, int32_t *out_tokens, int32_t *out_n_accepted) {
  if (!target_logits || !out_tokens || !out_n_accepted || !workspace) return HSD_E_INVALID_ARG;
  if (batch <= 0 || t < 0 || vocab <= 0 || level < 0 || level > 255) return HSD_E_INVALID_ARG;
  if (t > 0 && (!draft_logits || !draft_tokens)) return HSD_E_INVALID_ARG;
  if (t >= hsd::kSampleThreads || batch > 65535) return HSD_E_INVALID_ARG;
  if (dtype != HSD_F32 && dtype != HSD_BF16) return HSD_E_INVALID_ARG;
  if (((uintptr_t)workspace & 15) != 0) return HSD_E_INVALID_ARG;
  if (workspace_bytes < hsd::verify_scratch_bytes(batch, t)) return HSD_E_WORKSPACE_TOO_SMALL;
  return hsd::launch_verify(target_logits, draft_logits, const_cast<int32_t *>(draft_tokens), dtype, vocab, batch, t,
                            nullptr, t, (u32)call_serial, (u32)level, workspace, seed, out_tokens, out_n_accepted, 0,
                            (cudaStream_t)stream);
}

int hsd_verify_level_static(int level, const void *target_logits, const void *draft_logits, const int32_t *draft_tokens,
                            int batch, int t, int vocab, int dtype, uint64_t seed, uint64_t call_serial, void *stream,
                            int32_t *out_tokens, int32_t *out_n_accepted) {
  if (!target_logits || !out_tokens || !out_n_accepted) return HSD_E_INVALID_ARG;
  if (batch <= 0 || t < 0 || vocab <= 0 || level < 0 || level > 255) return HSD_E_INVALID_ARG;
  if (t > 0 && (!draft_logits || !draft_tokens)) return HSD_E_INVALID_ARG;
  if (t >= hsd::kSampleThreads || batch > 65535) return HSD_E_INVALID_ARG;
  if (dtype != HSD_F32 && dtype != HSD_BF16) return HSD_E_INVALID_ARG;
  if ((long long)batch * (2 * t + 1) > hsd::kStaticStatRows) return HSD_E_TOO_LARGE;
  void *scratch = nullptr;
  int st = hsd::static_scratch_address(&scratch);          // first call on this device looks the symbol up
  if (st) return st;
  // every RowStat the decision reads is written by the same call first; the per-sequence counters have to start
  // at zero and are cleared on the stream inside launch_verify (a memset node, no allocation)
  return hsd::launch_verify(target_logits, draft_logits, const_cast<int32_t *>(draft_tokens), dtype, vocab, batch, t,
                            nullptr, t, (u32)call_serial, (u32)level, scratch, seed, out_tokens, out_n_accepted, 0,
                            (cudaStream_t)stream);
}

}  // extern "C"
