// Calibration of the hierarchy search (Section 4.2 needs the acceptance rate alpha_{i,j} of every drafter i
// under every verifier j; Section 2: alpha = 1 - TV(p_i, p_j) = sum_x min(p_i(x), p_j(x))).  Given the logits of
// L models (exit layers) at the same R positions, the kernels below produce the L x L matrix of the rates
// averaged over the positions.
//   1. alpha_stats_kernel:   per (model, position): row maximum and sum of exp (fp32, fixed reduction order)
//   2. alpha_pairs_kernel:   per (position, 1024-token chunk): the L probabilities of the chunk in shared
//                            memory, every pair's sum of minima over the chunk -> one partial per pair
//   3. alpha_reduce_kernel:  per pair: the partials of all positions and chunks added in fixed order in fp64
// Deterministic (no atomics).  Model pairs are enumerated i < j, pair index = i L - i (i + 1) / 2 + (j - i - 1).
#include <cuda_bf16.h>
#include <math.h>

#include "../../include/hsd.h"
#include "common.cuh"

namespace hsd {
namespace {

constexpr int kAlphaThreads = 256;
constexpr int kAlphaChunk = 1024;      // tokens per block of the pair kernel
constexpr int kAlphaMaxModels = 32;

template <typename T>
__global__ void __launch_bounds__(kAlphaThreads)
alpha_stats_kernel(const T *__restrict__ logits, long long model_stride, int R, int V, float2 *__restrict__ stats) {
  __shared__ float sh[kAlphaThreads / 32];
  const int r = blockIdx.x, l = blockIdx.y;
  const T *row = logits + (size_t)l * model_stride + (size_t)r * V;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float m = -INFINITY;
  for (int k = threadIdx.x; k < V; k += kAlphaThreads) m = fmaxf(m, to_f32(row[k]));
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if (lane == 0) sh[warp] = m;
  __syncthreads();
  m = sh[0];
  for (int w = 1; w < kAlphaThreads / 32; ++w) m = fmaxf(m, sh[w]);
  __syncthreads();
  float s = 0.f;
  for (int k = threadIdx.x; k < V; k += kAlphaThreads) s += __expf(to_f32(row[k]) - m);
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if (lane == 0) sh[warp] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < kAlphaThreads / 32; ++w) tot += sh[w];
    stats[(size_t)l * R + r] = make_float2(m, tot);
  }
}

// grid (R, n_chunks).  Shared memory: prob[chunk token][L] (model index fastest: lanes that work on different
// pairs read different banks or the same word), then per-warp partials [8][n_pairs].
template <typename T>
__global__ void __launch_bounds__(kAlphaThreads)
alpha_pairs_kernel(const T *__restrict__ logits, long long model_stride, int L, int R, int V,
                   const float2 *__restrict__ stats, float *__restrict__ partials) {
  extern __shared__ float sm[];
  const int r = blockIdx.x, chunk = blockIdx.y, n_chunks = gridDim.y;
  const int v0 = chunk * kAlphaChunk, nv = min(kAlphaChunk, V - v0);
  const int n_pairs = L * (L - 1) / 2;
  float *prob = sm;                                   // [kAlphaChunk][L]
  float *wpart = sm + (size_t)kAlphaChunk * L;        // [8][n_pairs]
  for (int idx = threadIdx.x; idx < L * kAlphaChunk; idx += kAlphaThreads) {
    const int l = idx / kAlphaChunk, k = idx - l * kAlphaChunk;      // consecutive threads: consecutive tokens of one model
    float p = 0.f;
    if (k < nv) {
      const float2 st = stats[(size_t)l * R + r];
      p = __expf(to_f32(logits[(size_t)l * model_stride + (size_t)r * V + v0 + k]) - st.x) / st.y;
    }
    prob[(size_t)k * L + l] = p;
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int k0 = warp * (kAlphaChunk / 8);            // this warp's 128 tokens
  for (int pr = lane; pr < n_pairs; pr += 32) {
    int i = 0, rem = pr;                              // pair index -> (i, j)
    while (rem >= L - 1 - i) { rem -= L - 1 - i; ++i; }
    const int j = i + 1 + rem;
    float s = 0.f;
    for (int k = k0; k < k0 + kAlphaChunk / 8; ++k) s += fminf(prob[(size_t)k * L + i], prob[(size_t)k * L + j]);
    wpart[warp * n_pairs + pr] = s;
  }
  __syncthreads();
  for (int pr = threadIdx.x; pr < n_pairs; pr += kAlphaThreads) {
    float s = 0.f;
    for (int w = 0; w < 8; ++w) s += wpart[w * n_pairs + pr];
    partials[((size_t)r * n_chunks + chunk) * n_pairs + pr] = s;
  }
}

__global__ void __launch_bounds__(kAlphaThreads)
alpha_reduce_kernel(const float *__restrict__ partials, int L, int n_blocks, int R, double *__restrict__ alpha) {
  __shared__ double sh[kAlphaThreads];
  const int n_pairs = L * (L - 1) / 2;
  for (int pr = blockIdx.x; pr < n_pairs; pr += gridDim.x) {
    double s = 0.0;
    for (int b = threadIdx.x; b < n_blocks; b += kAlphaThreads) s += (double)partials[(size_t)b * n_pairs + pr];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int o = kAlphaThreads / 2; o > 0; o >>= 1) {
      if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      int i = 0, rem = pr;
      while (rem >= L - 1 - i) { rem -= L - 1 - i; ++i; }
      const int j = i + 1 + rem;
      const double a = sh[0] / (double)R;
      alpha[(size_t)i * L + j] = a;
      alpha[(size_t)j * L + i] = a;
    }
    __syncthreads();
  }
  if (blockIdx.x == 0 && (int)threadIdx.x < L) alpha[(size_t)threadIdx.x * L + threadIdx.x] = 1.0;
}

struct AlphaPlan { int n_chunks, n_pairs; size_t stats_off, partials_off, total; };
AlphaPlan alpha_plan(int L, int R, int V) {
  AlphaPlan p;
  p.n_chunks = (V + kAlphaChunk - 1) / kAlphaChunk;
  p.n_pairs = L * (L - 1) / 2;
  p.stats_off = 0;
  p.partials_off = ((size_t)L * R * sizeof(float2) + 255) / 256 * 256;
  p.total = p.partials_off + (size_t)R * p.n_chunks * (p.n_pairs > 0 ? p.n_pairs : 1) * sizeof(float);
  return p;
}

template <typename T>
int launch_alpha(const void *logits, long long model_stride, int L, int R, int V, void *ws, double *alpha, cudaStream_t s) {
  const AlphaPlan p = alpha_plan(L, R, V);
  float2 *stats = (float2 *)((char *)ws + p.stats_off);
  float *partials = (float *)((char *)ws + p.partials_off);
  alpha_stats_kernel<T><<<dim3(R, L), kAlphaThreads, 0, s>>>((const T *)logits, model_stride, R, V, stats);
  if (p.n_pairs > 0) {
    const size_t smem = ((size_t)kAlphaChunk * L + 8 * (size_t)p.n_pairs) * sizeof(float);
    if (smem > 48 * 1024) {
      static bool attr_set = false;
      if (!attr_set) {
        if (cudaFuncSetAttribute(alpha_pairs_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return HSD_E_CUDA;
        attr_set = true;
      }
    }
    alpha_pairs_kernel<T><<<dim3(R, p.n_chunks), kAlphaThreads, smem, s>>>((const T *)logits, model_stride, L, R, V, stats, partials);
  }
  alpha_reduce_kernel<<<p.n_pairs > 0 ? min(p.n_pairs, 148) : 1, kAlphaThreads, 0, s>>>(partials, L, R * p.n_chunks, R, alpha);
  hsd_count_launches(p.n_pairs > 0 ? 3 : 2);
  return hsd_launch_status();
}

}  // namespace
}  // namespace hsd

extern "C" {

size_t hsd_pairwise_alpha_workspace_bytes(int n_models, int n_rows, int vocab) {
  if (n_models < 1 || n_models > hsd::kAlphaMaxModels || n_rows < 1 || vocab < 1) return 0;
  return hsd::alpha_plan(n_models, n_rows, vocab).total;
}

int hsd_pairwise_alpha(const void *logits, int dtype, int n_models, int n_rows, int vocab, long long model_stride,
                       void *workspace, size_t workspace_bytes, double *alpha, void *stream) {
  if (!logits || !workspace || !alpha) return HSD_E_INVALID_ARG;
  if (dtype != HSD_BF16 && dtype != HSD_F32) return HSD_E_INVALID_ARG;
  if (n_models < 1 || n_models > hsd::kAlphaMaxModels || n_rows < 1 || vocab < 1) return HSD_E_INVALID_ARG;
  if (model_stride < (long long)n_rows * vocab) return HSD_E_INVALID_ARG;
  if (((uintptr_t)workspace & 255) != 0 || workspace_bytes < hsd::alpha_plan(n_models, n_rows, vocab).total) return HSD_E_INVALID_ARG;
  if (((size_t)hsd::kAlphaChunk * n_models + 8 * (size_t)(n_models * (n_models - 1) / 2)) * sizeof(float) > 200 * 1024)
    return HSD_E_TOO_LARGE;
  cudaStream_t s = (cudaStream_t)stream;
  return dtype == HSD_BF16
             ? hsd::launch_alpha<__nv_bfloat16>(logits, model_stride, n_models, n_rows, vocab, workspace, alpha, s)
             : hsd::launch_alpha<float>(logits, model_stride, n_models, n_rows, vocab, workspace, alpha, s);
}

}  // extern "C"
