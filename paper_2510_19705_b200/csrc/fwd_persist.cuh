// Persistent single-launch verifier forward (bf16 models): one cooperative kernel, one CTA per SM,
// runs every layer of a level's forward pass.  The TMA weight stream never stops at a GEMM
// boundary: the producer keeps filling the shared-memory ring with the next projection's weight
// tiles while the other warps go through a grid barrier and the small phases (RMSNorm, attention).
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace hsd {

struct FwdLayerDev {
  const __nv_bfloat16 *attn_norm, *mlp_norm;
  __nv_bfloat16 *k_pool, *v_pool;
};

struct FwdArgs {
  // geometry
  int d, nq, nkv, hd, ff, V, n_run, lm_map, max_seq, page, page_shift, pages_per_seq, n_pages;   // page = 1 << page_shift; KV pools are [kv head][n_pages][page][hd]
  float eps;
  // immutable inputs
  const CUtensorMap *wmaps;        // global memory: 7 per layer (wq wk wv wo wg wu wd), then the output head
  const FwdLayerDev *layers;       // global memory [n_layers]
  const __nv_bfloat16 *embed, *final_norm;
  const float *cos_tab, *sin_tab;
  // this call
  int R, L, n_attn, attn_rows, n_splits, keys_per_split;
  int a_box_rows;                  // rows of one activation TMA box (<= the row padding)
  int fuse_qkv;                    // 1: every sequence is one attention item; the item's CTAs finish its q / k / v themselves
  int fuse_gu;                     // 1: at most 4 rows; the down projection's CTAs build their activation tiles from the gate / up pieces
  int gu_pieces_max;               // pieces per gate / up tile at most (its split geometry; filled in by the launcher)
  int early_norm;                  // 1: the RMSNorm after a residual projection runs on CTAs that have no part in that projection;
                                   //    they start as soon as its pieces are complete (a counter), one grid barrier less per norm
                                   //    (filled in by the launcher)
  int tc_attn;                     // 1: work items with long key ranges run on tcgen05 / tensor memory (head size 128; needs fuse_qkv = 0)
  float *pieces2;                  // split pieces of the down projection while `pieces` still holds gate / up (fuse_gu)
  const int *tokens, *page_table, *row_seq, *row_pos, *lrow_src;
  const int4 *attn_items;          // (first packed row, rows, sequence, position of first row)
  const long long *lrow_dst;
  // buffers
  float *x;
  __nv_bfloat16 *h, *q, *att, *act, *hf, *logits;
  float *attn_partials;
  int *attn_counters;              // zero on entry, zero on exit
  float *pieces;
  int *tile_counters;              // zero on entry, zero on exit
  unsigned *grid_counter;          // zero on entry; [16] (64 bytes on) counts the CTAs that have stored their pieces of the
                                   // residual projections so far (early_norm), zero on entry as well
  int *status;                     // set non-zero when a bounded wait gave up
  unsigned long long *prof;        // optional [gridDim][kFwdProfEvents]: barrier arrive / depart times (ns)
  CUtensorMap amap[4];             // activations h, att, act, hf; box rows = row padding of this launch
};

constexpr int kFwdThreads = 384;
constexpr int kFwdProfEvents = 1024;
// rows of one sequence per attention work item for a given GQA group and head size
inline int fwd_attn_rows(int group, int hd) {
  int r = 4096 / (group * hd);
  return r < 1 ? 1 : (r > 8 ? 8 : r);
}
bool fwd_persist_supported(int hd, int group);
int launch_forward_persistent(const FwdArgs &args, int npad, int sm_count, cudaStream_t s);
// The attention tiles phase alone, one key split per item (args: geometry, R, n_attn, attn_rows, n_splits = 1,
// keys_per_split, page table, attn_items, q, att; fuse_qkv = 0): the item's rows of `att` are written.
int launch_attention_tiles(const FwdArgs &args, __nv_bfloat16 *k_pool, __nv_bfloat16 *v_pool, int sm_count, cudaStream_t s);

}  // namespace hsd
