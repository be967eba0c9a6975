// Sampling kernels of the HSD hot path: level-0 draft sampling (Algorithm 1, base case) and the
// fused softmax-statistics / acceptance / residual-resample step (Algorithm 2; rule of Section 2).
#include "sampling.cuh"
#include "sampling_api.cuh"

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

// ------------------------------------------------------------------------------ host launchers
size_t verify_scratch_bytes(int batch, int t_max) { return (size_t)batch * (2 * t_max + 1) * sizeof(RowStat); }

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
                           const VerifySeq *desc, int regular_t, u32 regular_serial, u32 regular_level, void *scratch,
                           u64 seed, int32_t *out_tokens, int32_t *out_n, int write_in_place, cudaStream_t s, u32 coin24) {
  RowStat *stats = (RowStat *)scratch;
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

int launch_verify(const void *p, const void *q, int32_t *tokens, int dtype, int V, int batch, int t_max,
                  const VerifySeq *desc, int regular_t, u32 regular_serial, u32 regular_level, void *scratch, u64 seed,
                  int32_t *out_tokens, int32_t *out_n, int write_in_place, cudaStream_t s, u32 coin24) {
  if (batch == 0) return HSD_OK;
  return dtype == HSD_BF16 ? launch_verify_t<__nv_bfloat16>(p, q, tokens, V, batch, t_max, desc, regular_t, regular_serial,
                                                            regular_level, scratch, seed, out_tokens, out_n, write_in_place, s, coin24)
                           : launch_verify_t<float>(p, q, tokens, V, batch, t_max, desc, regular_t, regular_serial,
                                                    regular_level, scratch, seed, out_tokens, out_n, write_in_place, s, coin24);
}

// ------------------------------------------------------------------------------ static scratch
// Scratch for hsd_verify_level_static: lives in the library image, so every GPU that loads the
// library holds these bytes until the process exits.  One RowStat per logits row of a call.
constexpr int kStaticStatRows = 4096;                       // 64 KiB
static __device__ __align__(256) unsigned char g_static_verify_scratch[kStaticStatRows * sizeof(RowStat)];

// In host code the array's name is only a stand-in for the symbol, not a device address: the
// address has to be asked for, once per device, with that device current.
static void *g_static_scratch_ptr[64] = {nullptr};
static int static_scratch_address(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HSD_E_CUDA;
  if (!g_static_scratch_ptr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_verify_scratch) != cudaSuccess || !p) return HSD_E_CUDA;
    g_static_scratch_ptr[dev] = p;
  }
  *out = g_static_scratch_ptr[dev];
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
  // every RowStat the decision reads is written by the statistics kernel of the same call first,
  // so nothing left over from an earlier call needs clearing
  return hsd::launch_verify(target_logits, draft_logits, const_cast<int32_t *>(draft_tokens), dtype, vocab, batch, t,
                            nullptr, t, (u32)call_serial, (u32)level, scratch, seed, out_tokens, out_n_accepted, 0,
                            (cudaStream_t)stream);
}

}  // extern "C"
