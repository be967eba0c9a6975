// Device-side decision arithmetic of the speculative-sampling rule (Section 2, Algorithm 2):
// Philox4x32-10 uniforms, integer softmax numerators, fixed-point probabilities, block-wide
// inverse CDF.  Everything that decides an integer is integer arithmetic on values produced by a
// fixed sequence of IEEE fp32 operations, so the outcome does not depend on thread count or
// summation order.
#pragma once
#include "common.cuh"

namespace hsd {

enum { PURPOSE_DRAFT = 0, PURPOSE_ACCEPT = 1, PURPOSE_FINAL = 2 };

// ---- Philox4x32-10 (Salmon et al., SC'11): 10 rounds, key bumped by the Weyl constants.
__device__ __forceinline__ u32 philox_word0(u32 c0, u32 c1, u32 c2, u32 c3, u32 k0, u32 k1) {
  const u32 M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k0 += W0; k1 += W1; }
    u32 hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    u32 hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    u32 n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  return c0;
}

// 24-bit integer uniform of the decision addressed (j, serial, level, purpose, seq).
__device__ __forceinline__ u32 uniform24(u64 seed, u32 j, u32 serial, u32 level, u32 purpose, u32 seq) {
  return philox_word0(j, serial, (level & 0xFFu) | (purpose << 8), seq, (u32)seed, (u32)(seed >> 32)) >> 8;
}

// ---- E = min(floor(exp(l - m) * 2^32), 2^32 - 1): every step is one fp32 operation, never fused.
__device__ __forceinline__ u32 exp_weight(float l, float m) {
  float x = __fsub_rn(l, m);
  x = fmaxf(x, -32.0f);
  float t = __fmul_rn(x, __uint_as_float(0x3FB8AA3Bu));     // * log2(e), in [-46.2, 0]
  // rint(t), half to even, without the quarter-rate conversion instructions: at 1.5 * 2^23 the fp32 spacing is
  // 1, so the add rounds t to the nearest integer (ties to even), the subtraction is exact, and the integer
  // itself sits in the low mantissa bits of the sum
  const float magic = __uint_as_float(0x4B400000u);        // 12582912
  float tm = __fadd_rn(t, magic);
  float j = __fsub_rn(tm, magic);
  float f = __fsub_rn(t, j);                               // exact, in [-1/2, 1/2]
  float p = __uint_as_float(0x3AADDD0Au);
  p = __fadd_rn(__fmul_rn(p, f), __uint_as_float(0x3C1E7544u));
  p = __fadd_rn(__fmul_rn(p, f), __uint_as_float(0x3D635BA9u));
  p = __fadd_rn(__fmul_rn(p, f), __uint_as_float(0x3E75FCDEu));
  p = __fadd_rn(__fmul_rn(p, f), __uint_as_float(0x3F317215u));
  p = __fadd_rn(__fmul_rn(p, f), 1.0f);
  int e = (__float_as_int(tm) - 0x4B400000) + 32;          // (int)j + 32, in [-14, 32]
  float w = __fmul_rn(p, __int_as_float((e + 127) << 23)); // exact power-of-two scaling
  return __float2uint_rz(w);                               // floor; saturates at 2^32 - 1
}

// Two weights at once with the packed fp32 multiply / add of sm_100 (each half is an IEEE
// round-to-nearest operation, and t + (-j) equals t - j exactly, so the results are bit-identical
// to exp_weight); halves the instruction count of the vocabulary-wide pass.
__device__ __forceinline__ void exp_weight2m(float l0, float l1, float m0, float m1, u32 &e0, u32 &e1);
__device__ __forceinline__ void exp_weight2(float l0, float l1, float m, u32 &e0, u32 &e1) { exp_weight2m(l0, l1, m, m, e0, e1); }
// ... with a row maximum of its own for each half (two rows side by side)
__device__ __forceinline__ void exp_weight2m(float l0, float l1, float m0, float m1, u32 &e0, u32 &e1) {
  float2 x = __fadd2_rn(make_float2(l0, l1), make_float2(-m0, -m1));
  x.x = fmaxf(x.x, -32.0f);
  x.y = fmaxf(x.y, -32.0f);
  const float log2e = __uint_as_float(0x3FB8AA3Bu);
  const float2 t = __fmul2_rn(x, make_float2(log2e, log2e));
  const float magic = __uint_as_float(0x4B400000u);        // see exp_weight
  const float2 tm = __fadd2_rn(t, make_float2(magic, magic));
  const float2 jj = __fadd2_rn(tm, make_float2(-magic, -magic));
  const float2 f = __fadd2_rn(t, make_float2(-jj.x, -jj.y));
  float c = __uint_as_float(0x3AADDD0Au);
  float2 p = make_float2(c, c);
  c = __uint_as_float(0x3C1E7544u); p = __fadd2_rn(__fmul2_rn(p, f), make_float2(c, c));
  c = __uint_as_float(0x3D635BA9u); p = __fadd2_rn(__fmul2_rn(p, f), make_float2(c, c));
  c = __uint_as_float(0x3E75FCDEu); p = __fadd2_rn(__fmul2_rn(p, f), make_float2(c, c));
  c = __uint_as_float(0x3F317215u); p = __fadd2_rn(__fmul2_rn(p, f), make_float2(c, c));
  p = __fadd2_rn(__fmul2_rn(p, f), make_float2(1.0f, 1.0f));
  const float2 sc = make_float2(__int_as_float((__float_as_int(tm.x) - 0x4B400000 + 32 + 127) << 23),
                                __int_as_float((__float_as_int(tm.y) - 0x4B400000 + 32 + 127) << 23));
  const float2 w = __fmul2_rn(p, sc);
  e0 = __float2uint_rz(w.x);
  e1 = __float2uint_rz(w.y);
}

// Fixed-point probabilities in units of 2^-40: P = (E * rinv) >> shift.
struct ProbScale { u32 rinv; int shift; };
__device__ __forceinline__ ProbScale prob_scale(u64 S) {
  ProbScale ps;
  int z = __clzll((long long)S);
  u64 s_top = (S << z) >> 32;                              // in [2^31, 2^32)
  ps.rinv = (u32)(0x7FFFFFFFFFFFFFFFull / s_top);
  ps.shift = 55 - z;
  return ps;
}
__device__ __forceinline__ u64 fixed_prob(u32 E, ProbScale ps) { return ((u64)E * ps.rinv) >> ps.shift; }

// (U * total) >> 24 without overflow (U < 2^24, total < 2^64).
__device__ __forceinline__ u64 cdf_threshold(u32 U, u64 total) {
  return (u64)U * (total >> 24) + (((u64)U * (total & 0xFFFFFFull)) >> 24);
}

// ---- block-wide reductions over a group of threads: the whole block (blockDim.x a multiple of 32, at most
// 1024), or the first N threads of a block that has other warps besides (named barrier ID).
struct WholeBlock {
  __device__ static __forceinline__ void sync() { __syncthreads(); }
  __device__ static __forceinline__ int threads() { return blockDim.x; }
};
template <int ID, int N> struct FirstThreads {
  __device__ static __forceinline__ void sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(N) : "memory"); }
  __device__ static __forceinline__ int threads() { return N; }
};

template <class G = WholeBlock>
__device__ __forceinline__ float block_max(float v, float *sh /*[32]*/) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = G::threads() >> 5;
  G::sync();
  if (l == 0) sh[w] = v;
  G::sync();
  float r = (l < nw) ? sh[l] : -INFINITY;
  for (int o = 16; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xFFFFFFFFu, r, o));
  return r;
}

// Sum of one u64 per thread; every thread gets the total.
template <class G = WholeBlock>
__device__ __forceinline__ u64 block_sum(u64 v, u64 *sh /*[33]*/) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = G::threads() >> 5;
  G::sync();
  if (l == 0) sh[w] = v;
  G::sync();
  u64 r = (l < nw) ? sh[l] : 0ull;
  for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xFFFFFFFFu, r, o);
  return r;
}

// Exclusive prefix sum of one u64 per thread in thread order; *total receives the block sum.
template <class G = WholeBlock>
__device__ __forceinline__ u64 block_exclusive_scan(u64 v, u64 *sh /*[33]*/, u64 *total) {
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = G::threads() >> 5;
  u64 inc = v;
  for (int o = 1; o < 32; o <<= 1) {
    u64 n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (l >= o) inc += n;
  }
  G::sync();
  if (l == 31) sh[w] = inc;
  G::sync();
  if (w == 0) {
    u64 t = (l < nw) ? sh[l] : 0ull, ti = t;
    for (int o = 1; o < 32; o <<= 1) {
      u64 n = __shfl_up_sync(0xFFFFFFFFu, ti, o);
      if (l >= o) ti += n;
    }
    if (l < nw) sh[l] = ti - t;          // exclusive warp offsets
    if (l == 31) sh[32] = ti;            // block total
  }
  G::sync();
  *total = sh[32];
  return sh[w] + inc - v;
}

// Row maximum of stored logits (value only).
template <typename T>
__device__ __forceinline__ float row_max(const T *row, int V, float *sh) {
  float m = -INFINITY;
  for (int k = threadIdx.x; k < V; k += blockDim.x) m = fmaxf(m, to_f32(row[k]));
  return block_max(m, sh);
}

// Inverse CDF in ascending token id over integer weights weight(k), k in [0, V):
// returns the smallest k whose inclusive prefix sum exceeds (U * total) >> 24, or -1 if the
// total is zero.  Each thread owns a contiguous chunk of tokens.  All threads get the result.
template <class WeightFn>
__device__ __forceinline__ int block_inverse_cdf(int V, u32 U, WeightFn weight, u64 *sh64 /*[34]*/, u64 *total_out) {
  int chunk = (V + blockDim.x - 1) / blockDim.x;
  int k0 = threadIdx.x * chunk, k1 = min(V, k0 + chunk);
  u64 local = 0;
  for (int k = k0; k < k1; ++k) local += weight(k);
  u64 total;
  u64 excl = block_exclusive_scan(local, sh64, &total);
  if (total_out) *total_out = total;
  int *result = reinterpret_cast<int *>(&sh64[33]);
  if (threadIdx.x == 0) *result = -1;
  __syncthreads();
  if (total != 0) {
    u64 tau = cdf_threshold(U, total);
    if (tau >= excl && tau < excl + local) {       // exactly one thread
      u64 c = excl;
      for (int k = k0; k < k1; ++k) {
        c += weight(k);
        if (c > tau) { *result = k; break; }
      }
    }
  }
  __syncthreads();
  int r = *result;
  __syncthreads();
  return r;
}

// ---- fast path for bf16 rows: each thread owns 32 consecutive tokens, fetched with four 16-byte
// loads (all issued before the first use) and kept packed in registers.
constexpr int kChunkTokens = 32;
struct Chunk32 { uint4 v[4]; };
__device__ __forceinline__ bool chunk_layout_ok(const void *row, int V, int threads) {
  return (V % 8 == 0) && ((long long)threads * kChunkTokens >= V) && (((unsigned long long)row & 15ull) == 0);
}
__device__ __forceinline__ Chunk32 chunk_load(const __nv_bfloat16 *row, int V, int k0) {
  Chunk32 c;
#pragma unroll
  for (int j = 0; j < 4; ++j)
    c.v[j] = (k0 + 8 * j < V) ? __ldg(reinterpret_cast<const uint4 *>(row + k0) + j) : make_uint4(0u, 0u, 0u, 0u);
  return c;
}
__device__ __forceinline__ float chunk_get(const Chunk32 &c, int i) {      // i must be a compile-time constant
  const uint4 &q = c.v[i >> 3];
  const unsigned w = ((i >> 1) & 3) == 0 ? q.x : ((i >> 1) & 3) == 1 ? q.y : ((i >> 1) & 3) == 2 ? q.z : q.w;
  return (i & 1) ? __uint_as_float(w & 0xFFFF0000u) : __uint_as_float(w << 16);
}
__device__ __forceinline__ float chunk_max(const Chunk32 &c, int V, int k0) {
  float m = -INFINITY;
#pragma unroll
  for (int i = 0; i < kChunkTokens; ++i)
    if (k0 + i < V) m = fmaxf(m, chunk_get(c, i));
  return m;
}
// Inverse CDF over weights weight(i) of the thread's own 32 tokens (i = local index, compile-time in the
// unrolled loops).  Same result as block_inverse_cdf with the same weights.
template <class G = WholeBlock, class WeightFn>
__device__ __forceinline__ int block_inverse_cdf_chunk(int V, int k0, u32 U, WeightFn weight, u64 *sh64 /*[34]*/, u64 *total_out) {
  u64 local = 0;
#pragma unroll
  for (int i = 0; i < kChunkTokens; ++i)
    if (k0 + i < V) local += weight(i);
  u64 total;
  u64 excl = block_exclusive_scan<G>(local, sh64, &total);
  if (total_out) *total_out = total;
  int *result = reinterpret_cast<int *>(&sh64[33]);
  if (threadIdx.x == 0) *result = -1;
  G::sync();
  if (total != 0) {
    u64 tau = cdf_threshold(U, total);
    if (tau >= excl && tau < excl + local) {
      u64 c = excl;
      bool found = false;
#pragma unroll
      for (int i = 0; i < kChunkTokens; ++i) {
        if (!found && k0 + i < V) {
          c += weight(i);
          if (c > tau) { *result = k0 + i; found = true; }
        }
      }
    }
  }
  G::sync();
  int r = *result;
  G::sync();
  return r;
}

}  // namespace hsd
