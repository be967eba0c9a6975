// Host-side interface of the verifier-forward kernels (Algorithm 2: "run verifier M_idx in
// parallel on all prefixes"): embedding gather, RMSNorm, weight-streaming skinny GEMMs, rotary
// embedding + paged KV append, causal attention over the paged KV cache, SwiGLU.
#pragma once
#include "common.cuh"

namespace hsd {

// Geometry of the decoder (Llama-style; shared by every early-exit level).
struct ModelDims {
  int n_layers, d, nq, nkv, hd, ff, V;
  int dtype;            // HSD_F32 / HSD_BF16: storage type of weights, KV cache, logits, GEMM inputs
  float eps, theta;
  int max_seq, page, pages_per_seq;
  int n_pages;          // pages per KV pool: a pool is [kv head][page][token in page][head dim] (one head's pages are adjacent)
};

// One packed batch of rows for a forward pass; all arrays are device memory.
struct RowBatch {
  int R;                      // packed rows
  const int *row_seq;         // [R] sequence index of each row
  const int *row_pos;         // [R] position of each row in its sequence
  int n_attn;                 // attention work items (a run of <= kAttnRows rows of one sequence)
  const int4 *attn;           // [n_attn] (first packed row, rows, sequence, position of first row)
  int max_kv_len;             // largest pos0 + rows over the work items
  int L;                      // rows that produce logits
  const int *lrow_src;        // [L] packed row index
  const long long *lrow_dst;  // [L] destination row in the level's logits buffer
};

constexpr int kAttnRows = 8;         // rows of one sequence handled by one attention block
constexpr int kAttnKeyTile = 32;
constexpr int kGemmRowTile = 16;     // rows per weight stream in the SIMT GEMM

// Up to three weight matrices [N_i, K] whose outputs are concatenated along N.
struct GemmSegs {
  const void *w[3];
  int n[3];
  int count;
};
enum GemmMode { GEMM_STORE_F32 = 0, GEMM_ADD_F32 = 1, GEMM_STORE_T_SCATTER = 2, GEMM_SWIGLU_T = 3 };

int launch_embed(const ModelDims &md, const void *embed, const int *tokens, const RowBatch &rb, float *x, cudaStream_t s);
// out[i, :] = T(rmsnorm(x[src ? src[i] : i, :]) * gain)
int launch_rmsnorm(const ModelDims &md, const float *x, const void *gain, const int *src, int rows, void *out, cudaStream_t s);
// SIMT GEMM: A [R, K] (storage type) times the segments' W^T, epilogue by mode.
//   STORE_F32        out_f32[r, n] = acc                       (ldo = total N)
//   ADD_F32          out_f32[r, n] += acc                      (residual stream)
//   STORE_T_SCATTER  out_t[dst[r], n] = T(acc)                 (logits rows)
//   SWIGLU_T         segments = (gate, up): out_t[r, n] = T(silu(g) * u)
int launch_gemm_simt(const ModelDims &md, const void *A, int R, int K, const GemmSegs &segs, int mode, float *out_f32,
                     void *out_t, const long long *dst, cudaStream_t s);
// q_out[r] = T(rope(q)); K (after rope) and V rows written to their pages.
int launch_rope_kv(const ModelDims &md, const float *qkv, const RowBatch &rb, const float *cos_tab, const float *sin_tab,
                   const int *page_table, void *k_pool, void *v_pool, void *q_out, cudaStream_t s);
// Causal attention of the packed rows over the paged cache; att_out [R, nq*hd] in storage type.
size_t attn_partial_floats(const ModelDims &md, int max_rows, int max_splits);
int launch_attention(const ModelDims &md, const void *q, const RowBatch &rb, const int *page_table, const void *k_pool,
                     const void *v_pool, float *partials, int keys_per_split, int n_splits, void *att_out, cudaStream_t s);

}  // namespace hsd
