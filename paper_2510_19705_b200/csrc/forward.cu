// Verifier-forward kernels, plain CUDA-core versions.  They serve fp32 models (no fp32 tensor-core
// path keeps fp32 accuracy) and every shape the tensor-core GEMM does not take.
#include "forward.cuh"

namespace hsd {

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ------------------------------------------------------------------------------ embedding gather
template <typename T>
__global__ void embed_kernel(const T *__restrict__ embed, const int *__restrict__ tokens, const int *__restrict__ row_seq,
                             const int *__restrict__ row_pos, int d, int max_seq, int V, float *__restrict__ x) {
  int r = blockIdx.x;
  // an id outside the vocabulary (only possible after non-finite logits) must not become an address
  int tok = min(max(tokens[(size_t)row_seq[r] * max_seq + row_pos[r]], 0), V - 1);
  const T *src = embed + (size_t)tok * d;
  for (int k = threadIdx.x; k < d; k += blockDim.x) x[(size_t)r * d + k] = to_f32(src[k]);
}

// ------------------------------------------------------------------------------ RMSNorm
template <typename T>
__global__ void rmsnorm_kernel(const float *__restrict__ x, const T *__restrict__ gain, const int *__restrict__ src, int d,
                               float eps, T *__restrict__ out) {
  __shared__ float sh[32];
  int i = blockIdx.x;
  const float *row = x + (size_t)(src ? src[i] : i) * d;
  float ss = 0.f;
  for (int k = threadIdx.x; k < d; k += blockDim.x) { float v = row[k]; ss += v * v; }
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += sh[w];
  float inv = rsqrtf(tot / (float)d + eps);
  for (int k = threadIdx.x; k < d; k += blockDim.x) out[(size_t)i * d + k] = from_f32<T>(row[k] * inv * to_f32(gain[k]));
}

// ------------------------------------------------------------------------------ SIMT skinny GEMM
// Each warp owns CPW output columns and streams their weight rows once with 16-byte loads; the
// activation rows are staged through shared memory in K-chunks.  acc[r][c] in fp32.
template <typename T> struct Vec16;
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void unpack16(const uint4 &v, float *f);
template <> __device__ __forceinline__ void unpack16<float>(const uint4 &v, float *f) {
  f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4 &v, float *f) {
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}

constexpr int kGemmWarps = 8;
constexpr int kGemmChunkBytes = 2048;   // bytes of one activation row per K-chunk

template <typename T, int RT, int CPW, int MODE>
__global__ void __launch_bounds__(kGemmWarps * 32)
gemm_simt_kernel(const T *__restrict__ A, int R, int r0, int K, GemmSegs segs, float *__restrict__ out_f32,
                 T *__restrict__ out_t, const long long *__restrict__ dst, int ldo) {
  constexpr int VN = Vec16<T>::N;
  constexpr int KC = kGemmChunkBytes / sizeof(T);          // elements per chunk
  __shared__ __align__(16) unsigned char sh_raw[RT * kGemmChunkBytes];
  T *shA = reinterpret_cast<T *>(sh_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rows = min(RT, R - r0);
  // column -> (segment, row within the segment's matrix)
  const int n_total = (MODE == GEMM_SWIGLU_T) ? segs.n[0] : (segs.n[0] + segs.n[1] + segs.n[2]);
  const int col0 = (blockIdx.x * kGemmWarps + warp) * CPW;
  constexpr int NW = (MODE == GEMM_SWIGLU_T) ? 2 * CPW : CPW;   // weight rows streamed per warp
  const T *wrow[NW];
#pragma unroll
  for (int c = 0; c < CPW; ++c) {
    int col = col0 + c;
    if (MODE == GEMM_SWIGLU_T) {
      bool ok = col < n_total;
      wrow[2 * c] = ok ? (const T *)segs.w[0] + (size_t)col * K : nullptr;
      wrow[2 * c + 1] = ok ? (const T *)segs.w[1] + (size_t)col * K : nullptr;
    } else {
      const T *p = nullptr;
      if (col < segs.n[0]) p = (const T *)segs.w[0] + (size_t)col * K;
      else if (col < segs.n[0] + segs.n[1]) p = (const T *)segs.w[1] + (size_t)(col - segs.n[0]) * K;
      else if (col < n_total) p = (const T *)segs.w[2] + (size_t)(col - segs.n[0] - segs.n[1]) * K;
      wrow[c] = p;
    }
  }
  float acc[RT][NW];
#pragma unroll
  for (int r = 0; r < RT; ++r)
#pragma unroll
    for (int c = 0; c < NW; ++c) acc[r][c] = 0.f;

  for (int kc = 0; kc < K; kc += KC) {
    const int klen = min(KC, K - kc);                       // multiple of VN (checked by the launcher)
    __syncthreads();
    for (int i = threadIdx.x; i < rows * (klen / VN); i += blockDim.x) {
      int r = i / (klen / VN), v = i % (klen / VN);
      *reinterpret_cast<uint4 *>(shA + r * KC + v * VN) =
          *reinterpret_cast<const uint4 *>(A + (size_t)(r0 + r) * K + kc + v * VN);
    }
    __syncthreads();
    for (int v = lane; v < klen / VN; v += 32) {
      float w[NW][VN];
#pragma unroll
      for (int c = 0; c < NW; ++c) {
        if (wrow[c]) {
          uint4 raw = __ldg(reinterpret_cast<const uint4 *>(wrow[c] + kc + v * VN));
          unpack16<T>(raw, w[c]);
        } else {
#pragma unroll
          for (int e = 0; e < VN; ++e) w[c][e] = 0.f;
        }
      }
#pragma unroll
      for (int r = 0; r < RT; ++r) {
        if (r < rows) {
          float a[VN];
          unpack16<T>(*reinterpret_cast<const uint4 *>(shA + r * KC + v * VN), a);
#pragma unroll
          for (int c = 0; c < NW; ++c)
#pragma unroll
            for (int e = 0; e < VN; ++e) acc[r][c] = fmaf(a[e], w[c][e], acc[r][c]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < RT; ++r)
#pragma unroll
    for (int c = 0; c < NW; ++c)
      for (int o = 16; o > 0; o >>= 1) acc[r][c] += __shfl_xor_sync(0xFFFFFFFFu, acc[r][c], o);
  if (lane == 0) {
#pragma unroll
    for (int r = 0; r < RT; ++r) {
      if (r >= rows) continue;
      int row = r0 + r;
#pragma unroll
      for (int c = 0; c < CPW; ++c) {
        int col = col0 + c;
        if (col >= n_total) continue;
        if (MODE == GEMM_STORE_F32) out_f32[(size_t)row * ldo + col] = acc[r][c];
        else if (MODE == GEMM_ADD_F32) out_f32[(size_t)row * ldo + col] += acc[r][c];
        else if (MODE == GEMM_STORE_T_SCATTER) out_t[(size_t)dst[row] * ldo + col] = from_f32<T>(acc[r][c]);
        else {
          float g = acc[r][2 * c], u = acc[r][2 * c + 1];
          out_t[(size_t)row * ldo + col] = from_f32<T>(g / (1.f + __expf(-g)) * u);
        }
      }
    }
  }
}

template <typename T, int RT, int MODE>
static void gemm_simt_launch(const T *A, int R, int K, const GemmSegs &segs, float *out_f32, T *out_t, const long long *dst,
                             int n_total, cudaStream_t s) {
  constexpr int CPW = 2;
  int grid = ceil_div(n_total, kGemmWarps * CPW);
  for (int r0 = 0; r0 < R; r0 += RT) {
    gemm_simt_kernel<T, RT, CPW, MODE><<<grid, kGemmWarps * 32, 0, s>>>(A, R, r0, K, segs, out_f32, out_t, dst, n_total);
    hsd_count_launches(1);
  }
}

template <typename T, int MODE>
static void gemm_simt_rows(const T *A, int R, int K, const GemmSegs &segs, float *out_f32, T *out_t, const long long *dst,
                           int n_total, cudaStream_t s) {
  if (R <= 4) gemm_simt_launch<T, 4, MODE>(A, R, K, segs, out_f32, out_t, dst, n_total, s);
  else if (R <= 8) gemm_simt_launch<T, 8, MODE>(A, R, K, segs, out_f32, out_t, dst, n_total, s);
  else gemm_simt_launch<T, kGemmRowTile, MODE>(A, R, K, segs, out_f32, out_t, dst, n_total, s);
}

template <typename T>
static int gemm_simt_t(const void *A, int R, int K, const GemmSegs &segs, int mode, float *out_f32, void *out_t,
                       const long long *dst, cudaStream_t s) {
  if (K % Vec16<T>::N != 0) return HSD_E_UNSUPPORTED;
  int n_total = (mode == GEMM_SWIGLU_T) ? segs.n[0] : segs.n[0] + segs.n[1] + segs.n[2];
  const T *a = (const T *)A;
  T *ot = (T *)out_t;
  switch (mode) {
    case GEMM_STORE_F32: gemm_simt_rows<T, GEMM_STORE_F32>(a, R, K, segs, out_f32, ot, dst, n_total, s); break;
    case GEMM_ADD_F32: gemm_simt_rows<T, GEMM_ADD_F32>(a, R, K, segs, out_f32, ot, dst, n_total, s); break;
    case GEMM_STORE_T_SCATTER: gemm_simt_rows<T, GEMM_STORE_T_SCATTER>(a, R, K, segs, out_f32, ot, dst, n_total, s); break;
    case GEMM_SWIGLU_T: gemm_simt_rows<T, GEMM_SWIGLU_T>(a, R, K, segs, out_f32, ot, dst, n_total, s); break;
    default: return HSD_E_INVALID_ARG;
  }
  return hsd_launch_status();
}

// ------------------------------------------------------------------------------ rotary + KV append
// grid (R, nq + 2 nkv): head h < nq -> rotated q; next nkv -> rotated k into its page; last nkv -> v.
template <typename T>
__global__ void rope_kv_kernel(const float *__restrict__ qkv, const int *__restrict__ row_seq, const int *__restrict__ row_pos,
                               const float *__restrict__ cos_tab, const float *__restrict__ sin_tab,
                               const int *__restrict__ page_table, T *__restrict__ k_pool, T *__restrict__ v_pool,
                               T *__restrict__ q_out, int nq, int nkv, int hd, int page, int pages_per_seq, int n_pages) {
  int r = blockIdx.x, h = blockIdx.y;
  int seq = row_seq[r], pos = row_pos[r];
  int half = hd >> 1;
  const float *src = qkv + (size_t)r * (nq + 2 * nkv) * hd + (size_t)h * hd;
  T *dst;
  bool rotate = h < nq + nkv;
  if (h < nq) {
    dst = q_out + ((size_t)r * nq + h) * hd;
  } else {
    int kvh = (h - nq) % nkv;
    int pg = page_table[(size_t)seq * pages_per_seq + pos / page];
    size_t off = (((size_t)kvh * n_pages + pg) * page + (pos % page)) * hd;
    dst = (h < nq + nkv ? k_pool : v_pool) + off;
  }
  if (rotate) {
    for (int k = threadIdx.x; k < half; k += blockDim.x) {
      float c = cos_tab[(size_t)pos * half + k], sn = sin_tab[(size_t)pos * half + k];
      float a = src[k], b = src[k + half];
      dst[k] = from_f32<T>(a * c - b * sn);
      dst[k + half] = from_f32<T>(b * c + a * sn);
    }
  } else {
    for (int k = threadIdx.x; k < hd; k += blockDim.x) dst[k] = from_f32<T>(src[k]);
  }
}

// ------------------------------------------------------------------------------ attention
// grid (n_splits, nkv, n_attn).  One block: the rows of one work item x the query heads of one KV
// head, over the keys of one split, with an online softmax per query; partial (m, l, o) per split.
constexpr int kAttnThreads = 128;

template <typename T, int HD>
__global__ void __launch_bounds__(kAttnThreads)
attn_split_kernel(const T *__restrict__ q, const int4 *__restrict__ items, const int *__restrict__ page_table,
                  const T *__restrict__ k_pool, const T *__restrict__ v_pool, float *__restrict__ partials, int nq, int nkv,
                  int page, int pages_per_seq, int n_pages, int keys_per_split, int n_splits, float scale) {
  constexpr int KT = kAttnKeyTile;
  constexpr int DPL = HD / 32;                         // output dims per lane
  extern __shared__ __align__(16) unsigned char smem[];
  const int group = nq / nkv;
  const int4 it = items[blockIdx.z];
  const int row0 = it.x, nrows = it.y, seq = it.z, pos0 = it.w;
  const int kvh = blockIdx.y, split = blockIdx.x;
  const int kv_len = pos0 + nrows;
  const int key_lo = split * keys_per_split, key_hi = min(kv_len, key_lo + keys_per_split);
  const int nqv = nrows * group;                       // query vectors of this block
  float *shQ = reinterpret_cast<float *>(smem);                               // [kAttnRows*group][HD]
  T *shK = reinterpret_cast<T *>(shQ + kAttnRows * group * HD);               // [KT][HD + 2]
  T *shV = shK + KT * (HD + 2);                                               // [KT][HD]
  float *shP = reinterpret_cast<float *>(shV + KT * HD);                      // [warps][KT]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = kAttnThreads / 32;

  for (int i = threadIdx.x; i < nqv * HD; i += blockDim.x) {
    int qi = i / HD, dd = i % HD;
    int r = qi / group, g = qi % group;
    shQ[i] = to_f32(q[((size_t)(row0 + r) * nq + kvh * group + g) * HD + dd]);
  }
  // per-warp query state: queries warp, warp + nwarps, ...
  constexpr int QPW = kAttnRows * 8 / (kAttnThreads / 32);   // queries per warp at most (group <= 8)
  float m_run[QPW], l_run[QPW], o_run[QPW][DPL];
#pragma unroll
  for (int i = 0; i < QPW; ++i) {
    m_run[i] = -INFINITY; l_run[i] = 0.f;
#pragma unroll
    for (int e = 0; e < DPL; ++e) o_run[i][e] = 0.f;
  }

  for (int kt = key_lo; kt < key_hi; kt += KT) {
    __syncthreads();
    // stage K and V tiles (zero-filled past key_hi)
    for (int i = threadIdx.x; i < KT * (HD / 2); i += blockDim.x) {
      int kk = i / (HD / 2), w2 = i % (HD / 2);
      int key = kt + kk;
      float2 kvv = make_float2(0.f, 0.f), vvv = make_float2(0.f, 0.f);
      if (key < key_hi) {
        int pg = page_table[(size_t)seq * pages_per_seq + key / page];
        size_t off = (((size_t)kvh * n_pages + pg) * page + (key % page)) * HD + 2 * w2;
        kvv = make_float2(to_f32(k_pool[off]), to_f32(k_pool[off + 1]));
        vvv = make_float2(to_f32(v_pool[off]), to_f32(v_pool[off + 1]));
      }
      shK[kk * (HD + 2) + 2 * w2] = from_f32<T>(kvv.x); shK[kk * (HD + 2) + 2 * w2 + 1] = from_f32<T>(kvv.y);
      shV[kk * HD + 2 * w2] = from_f32<T>(vvv.x); shV[kk * HD + 2 * w2 + 1] = from_f32<T>(vvv.y);
    }
    __syncthreads();
    int qslot = 0;
    for (int qi = warp; qi < nqv; qi += nwarps, ++qslot) {
      const int qpos = pos0 + qi / group;
      const int key = kt + lane;
      const float *qv = shQ + qi * HD;
      const T *kr = shK + lane * (HD + 2);
      float sc = 0.f;
#pragma unroll 8
      for (int dd = 0; dd < HD; ++dd) sc = fmaf(qv[dd], to_f32(kr[dd]), sc);
      sc *= scale;
      if (key >= key_hi || key > qpos) sc = -INFINITY;
      float mx = sc;
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
      float m_new = fmaxf(m_run[qslot], mx);
      float p = 0.f, corr = 1.f;
      if (m_new > -INFINITY) {
        p = __expf(sc - m_new);
        corr = __expf(m_run[qslot] - m_new);           // exp(-inf) = 0 on the first tile with keys
      }
      float ps = p;
      for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xFFFFFFFFu, ps, o);
      l_run[qslot] = l_run[qslot] * corr + ps;
      m_run[qslot] = m_new;
      shP[warp * KT + lane] = p;
      __syncwarp();
#pragma unroll
      for (int e = 0; e < DPL; ++e) o_run[qslot][e] *= corr;
      for (int kk = 0; kk < KT; ++kk) {
        float pk = shP[warp * KT + kk];
#pragma unroll
        for (int e = 0; e < DPL; ++e) o_run[qslot][e] = fmaf(pk, to_f32(shV[kk * HD + lane + 32 * e]), o_run[qslot][e]);
      }
      __syncwarp();
    }
  }
  // partial results: [row][head][split][HD + 2]
  int qslot = 0;
  for (int qi = warp; qi < nqv; qi += nwarps, ++qslot) {
    int r = row0 + qi / group, h = kvh * group + qi % group;
    float *dst = partials + (((size_t)r * nq + h) * n_splits + split) * (HD + 2);
#pragma unroll
    for (int e = 0; e < DPL; ++e) dst[lane + 32 * e] = o_run[qslot][e];
    if (lane == 0) { dst[HD] = m_run[qslot]; dst[HD + 1] = l_run[qslot]; }
  }
}

// grid (R * nq), block HD: merge the splits of one (row, head).
template <typename T, int HD>
__global__ void attn_combine_kernel(const float *__restrict__ partials, const int *__restrict__ row_pos, int nq,
                                    int keys_per_split, int n_splits, T *__restrict__ out) {
  int rh = blockIdx.x, r = rh / nq;
  int used = min(n_splits, row_pos[r] / keys_per_split + 1);     // splits that hold keys <= own position
  const float *src = partials + (size_t)rh * n_splits * (HD + 2);
  float m = -INFINITY;
  for (int s = 0; s < used; ++s) m = fmaxf(m, src[s * (HD + 2) + HD]);
  float l = 0.f, o = 0.f;
  for (int s = 0; s < used; ++s) {
    float ms = src[s * (HD + 2) + HD];
    float w = (ms > -INFINITY) ? __expf(ms - m) : 0.f;
    l += w * src[s * (HD + 2) + HD + 1];
    o += w * src[s * (HD + 2) + threadIdx.x];
  }
  out[(size_t)rh * HD + threadIdx.x] = from_f32<T>(o / l);
}

static size_t attn_smem_bytes(int group, int hd, size_t elem) {
  return (size_t)kAttnRows * group * hd * 4 + (size_t)kAttnKeyTile * (hd + 2) * elem + (size_t)kAttnKeyTile * hd * elem +
         (kAttnThreads / 32) * kAttnKeyTile * 4;
}

template <typename T, int HD>
static int attention_t(const ModelDims &md, const void *q, const RowBatch &rb, const int *page_table, const void *k_pool,
                       const void *v_pool, float *partials, int keys_per_split, int n_splits, void *att_out, cudaStream_t s) {
  int group = md.nq / md.nkv;
  size_t smem = attn_smem_bytes(group, HD, sizeof(T));
  static bool attr_set = false;
  if (!attr_set) {
    HSD_CUDA_OK(cudaFuncSetAttribute(attn_split_kernel<T, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    attr_set = true;
  }
  dim3 grid(n_splits, md.nkv, rb.n_attn);
  attn_split_kernel<T, HD><<<grid, kAttnThreads, smem, s>>>((const T *)q, rb.attn, page_table, (const T *)k_pool,
                                                           (const T *)v_pool, partials, md.nq, md.nkv, md.page,
                                                           md.pages_per_seq, md.n_pages, keys_per_split, n_splits, rsqrtf((float)HD));
  if (cudaGetLastError() != cudaSuccess) return HSD_E_CUDA;
  attn_combine_kernel<T, HD><<<rb.R * md.nq, HD, 0, s>>>(partials, rb.row_pos, md.nq, keys_per_split, n_splits, (T *)att_out);
  hsd_count_launches(2);
  return hsd_launch_status();
}

// ------------------------------------------------------------------------------ launchers
int launch_embed(const ModelDims &md, const void *embed, const int *tokens, const RowBatch &rb, float *x, cudaStream_t s) {
  if (rb.R == 0) return HSD_OK;
  if (md.dtype == HSD_BF16)
    embed_kernel<__nv_bfloat16><<<rb.R, 256, 0, s>>>((const __nv_bfloat16 *)embed, tokens, rb.row_seq, rb.row_pos, md.d, md.max_seq, md.V, x);
  else
    embed_kernel<float><<<rb.R, 256, 0, s>>>((const float *)embed, tokens, rb.row_seq, rb.row_pos, md.d, md.max_seq, md.V, x);
  hsd_count_launches(1);
  return hsd_launch_status();
}

int launch_rmsnorm(const ModelDims &md, const float *x, const void *gain, const int *src, int rows, void *out, cudaStream_t s) {
  if (rows == 0) return HSD_OK;
  if (md.dtype == HSD_BF16)
    rmsnorm_kernel<__nv_bfloat16><<<rows, 256, 0, s>>>(x, (const __nv_bfloat16 *)gain, src, md.d, md.eps, (__nv_bfloat16 *)out);
  else
    rmsnorm_kernel<float><<<rows, 256, 0, s>>>(x, (const float *)gain, src, md.d, md.eps, (float *)out);
  hsd_count_launches(1);
  return hsd_launch_status();
}

int launch_gemm_simt(const ModelDims &md, const void *A, int R, int K, const GemmSegs &segs, int mode, float *out_f32,
                     void *out_t, const long long *dst, cudaStream_t s) {
  if (R == 0) return HSD_OK;
  return md.dtype == HSD_BF16 ? gemm_simt_t<__nv_bfloat16>(A, R, K, segs, mode, out_f32, out_t, dst, s)
                              : gemm_simt_t<float>(A, R, K, segs, mode, out_f32, out_t, dst, s);
}

int launch_rope_kv(const ModelDims &md, const float *qkv, const RowBatch &rb, const float *cos_tab, const float *sin_tab,
                   const int *page_table, void *k_pool, void *v_pool, void *q_out, cudaStream_t s) {
  if (rb.R == 0) return HSD_OK;
  dim3 grid(rb.R, md.nq + 2 * md.nkv);
  int threads = md.hd >= 128 ? 64 : 32;
  if (md.dtype == HSD_BF16)
    rope_kv_kernel<__nv_bfloat16><<<grid, threads, 0, s>>>(qkv, rb.row_seq, rb.row_pos, cos_tab, sin_tab, page_table,
                                                          (__nv_bfloat16 *)k_pool, (__nv_bfloat16 *)v_pool,
                                                          (__nv_bfloat16 *)q_out, md.nq, md.nkv, md.hd, md.page, md.pages_per_seq, md.n_pages);
  else
    rope_kv_kernel<float><<<grid, threads, 0, s>>>(qkv, rb.row_seq, rb.row_pos, cos_tab, sin_tab, page_table, (float *)k_pool,
                                                  (float *)v_pool, (float *)q_out, md.nq, md.nkv, md.hd, md.page, md.pages_per_seq, md.n_pages);
  hsd_count_launches(1);
  return hsd_launch_status();
}

size_t attn_partial_floats(const ModelDims &md, int max_rows, int max_splits) {
  return (size_t)max_rows * md.nq * max_splits * (md.hd + 2);
}

int launch_attention(const ModelDims &md, const void *q, const RowBatch &rb, const int *page_table, const void *k_pool,
                     const void *v_pool, float *partials, int keys_per_split, int n_splits, void *att_out, cudaStream_t s) {
  if (rb.R == 0) return HSD_OK;
  if (md.nq % md.nkv != 0 || md.nq / md.nkv > 8) return HSD_E_UNSUPPORTED;
#define HSD_ATTN_CASE(TT, HDV) \
  return attention_t<TT, HDV>(md, q, rb, page_table, k_pool, v_pool, partials, keys_per_split, n_splits, att_out, s)
  if (md.dtype == HSD_BF16) {
    if (md.hd == 128) HSD_ATTN_CASE(__nv_bfloat16, 128);
    if (md.hd == 64) HSD_ATTN_CASE(__nv_bfloat16, 64);
    if (md.hd == 32) HSD_ATTN_CASE(__nv_bfloat16, 32);
  } else {
    if (md.hd == 128) HSD_ATTN_CASE(float, 128);
    if (md.hd == 64) HSD_ATTN_CASE(float, 64);
    if (md.hd == 32) HSD_ATTN_CASE(float, 32);
  }
#undef HSD_ATTN_CASE
  return HSD_E_UNSUPPORTED;
}

// Read-only streaming pass over a buffer: what the weight stream of a verification forward does to HBM, without the
// arithmetic.  The measured rate is the denominator a weight-streaming pass can be held against.
__global__ void __launch_bounds__(512) stream_read_kernel(const uint4 *__restrict__ src, size_t n_vec, unsigned *__restrict__ sink) {
  unsigned acc = 0u;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride * 4) {
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const size_t j = i + (size_t)u * stride;
      v[u] = j < n_vec ? __ldg(src + j) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) acc += v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  if (acc == 0x9E3779B9u && sink) *sink = acc;              // keeps the loads alive; practically never taken
}

}  // namespace hsd

extern "C" int hsd_stream_read(const void *buffer, size_t bytes, void *sink, void *stream) {
  if (!buffer || bytes < 16 || ((uintptr_t)buffer & 15) != 0) return HSD_E_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return HSD_E_CUDA;
  hsd::stream_read_kernel<<<sms * 8, 512, 0, (cudaStream_t)stream>>>((const uint4 *)buffer, bytes / 16, (unsigned *)sink);
  hsd_count_launches(1);
  return hsd_launch_status();
}
