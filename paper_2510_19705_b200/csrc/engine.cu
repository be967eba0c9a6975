// Host control of the HSD hot path: Algorithm 1's recursion (level-synchronous over a batch of
// independent sequences), the per-level verification step (multi-row forward -> acceptance /
// resample -> KV rollback), KV paging, workspace carving, statistics and the decision log.
#include <stdio.h>
#include <stdlib.h>
#include <math.h>
#include <algorithm>
#include <new>
#include <vector>

#include "forward.cuh"
#include "fwd_persist.cuh"
#include "gemm_tc.cuh"
#include "sampling_api.cuh"

using namespace hsd;

namespace {

constexpr int kRingSlots = 48;
constexpr int kTimerPairs = 64;
constexpr int kAttnBlocksTarget = 512;
constexpr int kMaxSplits = 64;
constexpr int kTcAttnMinKeys = 2048;           // = the kernel's thresholds for the tensor-memory attention path:
constexpr int kTcAttnMinVectors = 8;          //   keys of a work item, query vectors of an attention item
constexpr int kPrefillRows = 128;              // rows of one prompt chunk: the largest pass the one-launch forward takes
constexpr uint32_t kTraceMagic = 0x48534454u;

constexpr size_t kTcCtrlBytes = 16384 + 256;    // status word (first 256 bytes) + per-tile counters
constexpr int kHeadMaps = 17;                   // output-head tensor maps: one per level (<= 16), then the shared head

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
int device_sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      sms < 1)
    return 148;
  return sms;
}
size_t elem_size(int dtype) { return dtype == HSD_BF16 ? 2 : 4; }

// Workspace layout, shared by the workspace-size calls and the create calls.  One part per model (its KV
// pools, activations, rotary tables, tensor-core scratch) and one part that all levels share (token buffer,
// page table, per-level logits rows, decision scratch, descriptor ring).
struct ModelLayout {
  size_t cos_tab, sin_tab, k_pool, v_pool, pool_layer_stride, x, h, qkv, q, att, act, partials, hf, tc_scratch,
      tc_pieces_bytes, tc_pieces2, wmaps_dev, layers_dev, attn_counters, prof;
  int partial_rows;
};
struct Layout {
  size_t tokens, page_table, vscratch, n_acc, ring, grid_counter, total;
  std::vector<size_t> logits;
  std::vector<int> slots;
  std::vector<ModelLayout> model;
  int max_rows, pages_per_seq, n_pages, max_logit_rows;
  size_t ring_slot;
};

bool valid_dims(const hsd_model_desc *m) {
  if (!m) return false;
  if (m->n_layers < 1 || m->d_model < 8 || m->n_q_heads < 1 || m->n_kv_heads < 1 || m->head_dim < 2 || m->d_ff < 8 ||
      m->vocab < 2)
    return false;
  if (m->dtype != HSD_F32 && m->dtype != HSD_BF16) return false;
  if (m->max_batch < 1 || m->max_seq < 4 || m->page_size < 0) return false;
  if (m->n_q_heads % m->n_kv_heads != 0 || (m->head_dim & 1)) return false;
  return true;
}
bool valid_T(int n_levels, const int32_t *T) {
  if (n_levels < 1 || n_levels > 16) return false;
  if (n_levels > 1 && !T) return false;
  for (int i = 0; i + 1 < n_levels; ++i)
    if (T[i] < 1 || T[i] > 64) return false;
  return true;
}
// One decoder, levels = early exits.
bool valid_model(const hsd_model_desc *m, const int32_t *exits, int n_levels, const int32_t *T) {
  if (!valid_dims(m) || !exits || !valid_T(n_levels, T)) return false;
  for (int i = 0; i < n_levels; ++i) {
    if (exits[i] < 1 || exits[i] > m->n_layers) return false;
    if (i > 0 && exits[i] <= exits[i - 1]) return false;
  }
  return exits[n_levels - 1] == m->n_layers;
}
// One model per level: what the levels must have in common (vocabulary, storage type, capacity, page size).
bool valid_models(const hsd_model_desc *ms, int n_levels, const int32_t *T) {
  if (!ms || !valid_T(n_levels, T)) return false;
  for (int i = 0; i < n_levels; ++i) {
    if (!valid_dims(&ms[i])) return false;
    if (ms[i].vocab != ms[0].vocab || ms[i].dtype != ms[0].dtype || ms[i].max_batch != ms[0].max_batch ||
        ms[i].max_seq != ms[0].max_seq || ms[i].page_size != ms[0].page_size)
      return false;
  }
  return true;
}

Layout make_layout(const hsd_model_desc *models, int n_models, int n_levels, const int32_t *T) {
  Layout L;
  const hsd_model_desc *m0 = &models[0];
  const size_t es = elem_size(m0->dtype);
  const int page = m0->page_size ? m0->page_size : 16;
  const int B = m0->max_batch;
  int sumT = 0;
  L.slots.resize(n_levels);
  for (int i = 0; i < n_levels; ++i) {
    if (i + 1 < n_levels) sumT += T[i];
    L.slots[i] = sumT + 1;                                  // level i keeps at most sum_{j<=i} T_j (+1) rows
  }
  if (n_levels == 1) L.slots[0] = 1;
  // rows of one forward: drafts of the level below + catch-up rows (<= n_levels), per sequence
  int decode_rows = B * (sumT + n_levels + 1);
  L.max_rows = std::max(kPrefillRows, decode_rows);
  L.pages_per_seq = (m0->max_seq + page - 1) / page;
  L.n_pages = B * L.pages_per_seq;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.tokens = take((size_t)B * m0->max_seq * 4);
  L.page_table = take((size_t)B * L.pages_per_seq * 4);
  L.max_logit_rows = 0;
  L.logits.resize(n_levels);
  for (int i = 0; i < n_levels; ++i) {
    L.logits[i] = take((size_t)B * L.slots[i] * m0->vocab * es);
    L.max_logit_rows = std::max(L.max_logit_rows, B * L.slots[i]);
  }
  L.vscratch = take(verify_scratch_bytes(B, sumT + 1));
  L.n_acc = take((size_t)B * 4);
  L.ring_slot = align_up((size_t)L.max_rows * 40 + (size_t)B * 96 + 1024, 256);
  L.ring = take(L.ring_slot * kRingSlots);
  L.grid_counter = take(256);
  L.model.resize(n_models);
  for (int mi = 0; mi < n_models; ++mi) {
    const hsd_model_desc *m = &models[mi];
    ModelLayout &M = L.model[mi];
    const int d = m->d_model, hd = m->head_dim, nq = m->n_q_heads, nkv = m->n_kv_heads;
    M.partial_rows = std::max(L.max_rows + kAttnRows * kAttnBlocksTarget / nkv + kAttnRows * kMaxSplits,
                              L.max_rows * 20);   // the persistent forward may cut every row's keys into up to 20 splits
    M.cos_tab = take((size_t)m->max_seq * (hd / 2) * 4);
    M.sin_tab = take((size_t)m->max_seq * (hd / 2) * 4);
    M.pool_layer_stride = align_up((size_t)L.n_pages * nkv * page * hd * es, 256);
    M.k_pool = take(M.pool_layer_stride * m->n_layers);
    M.v_pool = take(M.pool_layer_stride * m->n_layers);
    M.x = take((size_t)L.max_rows * d * 4);
    M.h = take((size_t)L.max_rows * d * es);
    M.qkv = take((size_t)L.max_rows * (nq + 2 * nkv) * hd * 4);
    M.q = take((size_t)L.max_rows * nq * hd * es);
    M.att = take((size_t)L.max_rows * nq * hd * es);
    M.act = take((size_t)L.max_rows * m->d_ff * es);
    M.partials = take((size_t)M.partial_rows * nq * (hd + 2) * 4);
    M.hf = take((size_t)L.max_logit_rows * d * es);
    // tensor-core GEMM scratch: [status word | per-tile counters (16 KiB)] + split pieces (largest plan)
    M.tc_pieces_bytes = 0;
    if (m->dtype == HSD_BF16) {
      const int sms = device_sm_count();
      const int npads[5] = {16, 32, 64, 128, 256};
      const int shapes[5][4] = {{nq * hd, nkv * hd, nkv * hd, d}, {d, 0, 0, nq * hd}, {m->d_ff, m->d_ff, 0, d},
                                {d, 0, 0, m->d_ff}, {m->vocab, 0, 0, d}};
      const int modes[5] = {GEMM_STORE_F32, GEMM_ADD_F32, GEMM_SWIGLU_T, GEMM_ADD_F32, GEMM_STORE_T_SCATTER};
      for (int g = 0; g < 5; ++g)
        for (int np : npads) {
          if (shapes[g][3] % kTcBlockK) continue;
          int nsegs = shapes[g][2] ? 3 : (shapes[g][1] ? 2 : 1);
          TcGemmPlan pl = tc_plan(shapes[g], nsegs, modes[g], shapes[g][3], np, sms);
          M.tc_pieces_bytes = std::max(M.tc_pieces_bytes, pl.scratch_bytes);
        }
    }
    M.tc_scratch = take(kTcCtrlBytes + M.tc_pieces_bytes);
    M.tc_pieces2 = take(M.tc_pieces_bytes);       // second piece buffer (down projection of passes with few rows)
    M.wmaps_dev = take(((size_t)m->n_layers * 7 + kHeadMaps) * sizeof(CUtensorMap));
    M.layers_dev = take((size_t)m->n_layers * sizeof(FwdLayerDev));
    M.attn_counters = take(16384);
    M.prof = take((size_t)device_sm_count() * kFwdProfEvents * 8);
  }
  L.total = off;
  return L;
}

struct SeqWork {
  int b, start, end;     // rows = positions [start, end)
  int logit_first;       // first position whose output row is wanted (-1: none); rows up to end - 1
  int slot0;             // destination slot of that first row in the level's logits buffer
};

struct TimerPair { cudaEvent_t a, b; int level; };

}  // namespace

// One decoder: its geometry, weights, part of the workspace and tensor-core state.  A hierarchy of early exits
// has one (every level runs its first exits[level] layers); a hierarchy of separate models has one per level.
struct Model {
  ModelDims md;
  ModelLayout lay;
  const void *embed, *final_norm, *lm_head;
  std::vector<const void *> lw;
  bool use_tc = false, use_persist = false;   // tensor-core GEMMs / the one-launch persistent forward (bf16 models)
  std::vector<CUtensorMap> wmaps;             // [n_layers * 7 + kHeadMaps]: wq wk wv wo wg wu wd per layer, then the levels' heads, the shared head
  CUtensorMap amaps[4][5];                    // activation buffers {h, att, act, hf} x row padding {16, 32, 64, 128, 256}
  CUtensorMap amaps_rows[4][16];              // the same buffers with a box of exactly 1..16 rows (persistent forward, few rows)
};

struct hsd_ctx {
  ModelDims md;                               // what all levels share is read from here: V, dtype, max_seq, page, pages_per_seq
  int n_levels, max_batch;
  std::vector<int> exits, T;                  // exits[level] = layers the level runs of its model
  std::vector<Model> models;
  std::vector<int> level_model;               // model of each level (all 0 for early exits of one decoder)
  bool shared_cache = true;                   // early exits: level i's pass also refreshes the KV of the levels below it
  Layout lay;
  char *ws;
  // pinned host mirrors
  char *ring_host;
  int *n_acc_host;
  int *page_table_host;
  int ring_next, ring_in_flight;
  // per-sequence state
  std::vector<int> buf_len;
  std::vector<std::vector<int>> len_g;        // [b][level]: leading positions whose KV in group `level` is valid
  std::vector<std::vector<uint32_t>> serial;  // [b][level]
  std::vector<int> n_pages_of;
  std::vector<int> free_pages;
  std::vector<char> pt_dirty;
  // statistics / timing
  std::vector<hsd_level_stats> stats;
  TimerPair timers[kTimerPairs];
  int timers_used;
  bool timers_ok;
  // decision log
  FILE *trace;
  int trace_logit_calls, trace_records;
  cudaStream_t stream;
  uint64_t seed;
  bool any_tc = false;                        // some model runs the tensor-core kernels (their status word is polled)
  bool no_fuse_qkv = false;                   // keep the QKV finish phase in every pass (hsd_set_phase_folding)
  bool no_fuse_gu = false;                    // keep the gate / up finish phase in every pass
  bool no_early_norm = false;                 // keep the grid barrier between a residual projection and its norm
  bool no_tc_attn = false;                    // long key ranges on the mma.sync path as well (hsd_set_tensor_attention)
  bool prefer_tc_attn = false;                // never cut the keys into splits shorter than that path takes (a test hook)
  int sm_count;
  std::vector<const void *> level_head, level_norm;   // output head and final norm gain of each level (the model's own unless set)
  std::vector<uint32_t> coin24;               // per level: kNoCoin, or the IID acceptance probability x 2^24 (ablation)
  int *status_host;
  size_t status_off;                          // the one status word every tensor-core kernel of the context raises

  Model &model_of(int level) { return models[level_model[level]]; }

  template <typename U> U *dev(size_t off) const { return reinterpret_cast<U *>(ws + off); }
};

namespace {

int sync_stream(hsd_ctx *c) {
  if (c->any_tc &&
      cudaMemcpyAsync(c->status_host, c->ws + c->status_off, 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess)
    return HSD_E_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return HSD_E_CUDA;
  if (c->any_tc && *c->status_host != 0) return HSD_E_DEVICE_TIMEOUT;
  c->ring_in_flight = 0;
  for (int i = 0; i < c->timers_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->timers[i].a, c->timers[i].b) == cudaSuccess) c->stats[c->timers[i].level].ms += ms;
  }
  c->timers_used = 0;
  return HSD_OK;
}

// A slot of the descriptor ring: host pointer to fill + matching device address.
int ring_acquire(hsd_ctx *c, char **host, char **devp) {
  if (c->ring_in_flight >= kRingSlots) {
    int st = sync_stream(c);
    if (st) return st;
  }
  int s = c->ring_next;
  c->ring_next = (c->ring_next + 1) % kRingSlots;
  c->ring_in_flight++;
  *host = c->ring_host + (size_t)s * c->lay.ring_slot;
  *devp = c->ws + c->lay.ring + (size_t)s * c->lay.ring_slot;
  return HSD_OK;
}

int ensure_pages(hsd_ctx *c, int b, int upto_len) {
  const int page = c->md.page;
  int need = (upto_len + page - 1) / page;
  if (need > c->md.pages_per_seq) return HSD_E_INVALID_ARG;
  while (c->n_pages_of[b] < need) {
    if (c->free_pages.empty()) return HSD_E_OUT_OF_PAGES;
    int pg = c->free_pages.back();
    c->free_pages.pop_back();
    c->page_table_host[(size_t)b * c->md.pages_per_seq + c->n_pages_of[b]] = pg;
    c->n_pages_of[b]++;
    c->pt_dirty[b] = 1;
  }
  return HSD_OK;
}

void trim_pages(hsd_ctx *c, int b, int keep_len) {
  const int page = c->md.page;
  int keep = (keep_len + page - 1) / page;
  while (c->n_pages_of[b] > keep) {
    c->n_pages_of[b]--;
    c->free_pages.push_back(c->page_table_host[(size_t)b * c->md.pages_per_seq + c->n_pages_of[b]]);
  }
}

int upload_page_tables(hsd_ctx *c) {
  for (int b = 0; b < c->max_batch; ++b) {
    if (!c->pt_dirty[b]) continue;
    size_t off = (size_t)b * c->md.pages_per_seq;
    HSD_CUDA_OK(cudaMemcpyAsync(c->dev<int>(c->lay.page_table) + off, c->page_table_host + off,
                                (size_t)c->n_pages_of[b] * 4, cudaMemcpyHostToDevice, c->stream));
    c->pt_dirty[b] = 0;
  }
  return HSD_OK;
}

// Matrix product of the forward pass: tensor cores for bf16 models, CUDA cores otherwise.
// abuf names the activation buffer A lives in (0 = h, 1 = att, 2 = act, 3 = hf); wmap0 the index of
// the first segment's tensor map.
int gemm(hsd_ctx *c, Model &M, int abuf, const void *A, int R, int K, const GemmSegs &segs, int wmap0, int mode, float *out_f32,
         void *out_t, const long long *dst) {
  if (!M.use_tc) return launch_gemm_simt(M.md, A, R, K, segs, mode, out_f32, out_t, dst, c->stream);
  TcGemmArgs a;
  int total = 0;
  for (int i = 0; i < 3; ++i) {
    a.seg_n[i] = i < segs.count ? segs.n[i] : 0;
    if (i < segs.count) a.w[i] = M.wmaps[wmap0 + i];
    total += a.seg_n[i];
  }
  a.n_segs = segs.count;
  a.K = K;
  a.mode = mode;
  a.out_f32 = out_f32;
  a.out_bf16 = (__nv_bfloat16 *)out_t;
  a.dst = dst;
  a.ldo = (mode == GEMM_SWIGLU_T) ? segs.n[0] : total;
  a.status = (int *)(c->ws + c->status_off);
  a.counters = (int *)(c->ws + M.lay.tc_scratch + 256);
  a.pieces = (float *)(c->ws + M.lay.tc_scratch + kTcCtrlBytes);
  for (int r0 = 0; r0 < R; r0 += 256) {
    a.R = std::min(256, R - r0);
    a.row0 = r0;
    int np = tc_npad(a.R);
    a.a = M.amaps[abuf][np == 16 ? 0 : np == 32 ? 1 : np == 64 ? 2 : np == 128 ? 3 : 4];
    int st = launch_gemm_tc(a, c->sm_count, c->stream);
    if (st) return st;
  }
  return HSD_OK;
}

// One forward pass of level `level` (layers 1..exit) over the given rows; logits of the wanted
// rows go to the level's logits buffer.  KV of every processed position is (re)written.
int forward(hsd_ctx *c, int level, const std::vector<SeqWork> &work) {
  Model &M = c->model_of(level);
  const ModelDims &md = M.md;
  const Layout &L = c->lay;
  const ModelLayout &ML = M.lay;
  int R = 0, n_attn = 0, n_logit = 0, max_kv = 0;
  bool one_item_per_seq = true;
  const int arows = M.use_persist ? fwd_attn_rows(md.nq / md.nkv, md.hd) : kAttnRows;   // rows per attention item
  for (const SeqWork &w : work) {
    int rows = w.end - w.start;
    if (rows <= 0 || w.start < 0 || w.end > md.max_seq) return HSD_E_INVALID_ARG;
    R += rows;
    n_attn += (rows + arows - 1) / arows;
    if (rows > arows) one_item_per_seq = false;
    if (w.logit_first >= 0) {
      if (w.logit_first < w.start || w.logit_first >= w.end) return HSD_E_INVALID_ARG;
      n_logit += w.end - w.logit_first;
    }
    max_kv = std::max(max_kv, w.end);
    int st = ensure_pages(c, w.b, w.end);
    if (st) return st;
  }
  if (R == 0) return HSD_OK;
  if (R > L.max_rows) return HSD_E_INVALID_ARG;
  char *host, *devp;
  int st = ring_acquire(c, &host, &devp);
  if (st) return st;
  // slot layout: row_seq[R] | row_pos[R] | attn int4[n_attn] | lrow_src[n_logit] | lrow_dst int64[n_logit]
  size_t o_seq = 0, o_pos = align_up(o_seq + (size_t)R * 4, 16), o_attn = align_up(o_pos + (size_t)R * 4, 16),
         o_src = align_up(o_attn + (size_t)n_attn * 16, 16), o_dst = align_up(o_src + (size_t)n_logit * 4, 16),
         bytes = o_dst + (size_t)n_logit * 8;
  if (bytes > L.ring_slot) return HSD_E_INVALID_ARG;
  int *row_seq = (int *)(host + o_seq), *row_pos = (int *)(host + o_pos), *lsrc = (int *)(host + o_src);
  int4 *attn = (int4 *)(host + o_attn);
  long long *ldst = (long long *)(host + o_dst);
  int r = 0, ia = 0, il = 0;
  for (const SeqWork &w : work) {
    for (int p0 = w.start; p0 < w.end; p0 += arows) {
      int rows = std::min(arows, w.end - p0);
      attn[ia++] = make_int4(r + (p0 - w.start), rows, w.b, p0);
    }
    for (int p = w.start; p < w.end; ++p, ++r) {
      row_seq[r] = w.b;
      row_pos[r] = p;
      if (w.logit_first >= 0 && p >= w.logit_first) {
        lsrc[il] = r;
        ldst[il] = (long long)w.b * L.slots[level] + w.slot0 + (p - w.logit_first);
        if (w.slot0 + (p - w.logit_first) >= L.slots[level]) return HSD_E_INVALID_ARG;
        ++il;
      }
    }
  }
  // Attention work items are dealt to the CTAs round-robin in this order: the most expensive first (keys x
  // 16-row query tiles), so that a CTA's items sample the whole cost range.
  const int qgroup = md.nq / md.nkv;
  auto item_cost = [&](const int4 &it) { return (long long)(it.w + it.y) * ((it.y * qgroup + 15) / 16); };
  if (M.use_persist && n_attn > 1)
    std::stable_sort(attn, attn + n_attn, [&](const int4 &x, const int4 &y) { return item_cost(x) > item_cost(y); });
  HSD_CUDA_OK(cudaMemcpyAsync(devp, host, bytes, cudaMemcpyHostToDevice, c->stream));
  st = upload_page_tables(c);
  if (st) return st;
  RowBatch rb;
  rb.R = R;
  rb.row_seq = (const int *)(devp + o_seq);
  rb.row_pos = (const int *)(devp + o_pos);
  rb.n_attn = n_attn;
  rb.attn = (const int4 *)(devp + o_attn);
  rb.max_kv_len = max_kv;
  rb.L = n_logit;
  rb.lrow_src = (const int *)(devp + o_src);
  rb.lrow_dst = (const long long *)(devp + o_dst);

  // attention split: enough blocks to fill the GPU, never more partial rows than the buffer holds
  const int blocks_target = M.use_persist ? c->sm_count : kAttnBlocksTarget;
  const int max_splits = M.use_persist ? 20 : kMaxSplits;      // the persistent merge phase takes <= 20 splits
  int n_splits = std::max(1, std::min(max_splits, blocks_target / std::max(1, n_attn * md.nkv)));
  // the tensor-memory attention path: head size 128, a pass of the one-launch forward in which at least half of the
  // attention items have enough query vectors for it to pay (the pass then has its QKV finish phase and holds the
  // O projection's weights back until the attention phase is over)
  int n_vec_items = 0;
  for (int i = 0; i < n_attn; ++i)
    if (attn[i].y * (md.nq / md.nkv) >= kTcAttnMinVectors) ++n_vec_items;
  const bool tc_capable = M.use_persist && md.hd == 128 && !c->no_tc_attn && R <= 128 && n_logit <= 128 && 2 * n_vec_items >= n_attn;
  if (M.use_persist && max_kv >= 2048) {
    // Long contexts: the key loop dominates and the items differ in cost, so the split count is chosen by a
    // small model of the tiles phase: a work unit (item, KV head, split) costs a fixed part plus its keys x
    // query tiles, units go to the CTAs round-robin in item order (as the kernel deals them), the phase lasts
    // as long as the most loaded CTA; more than one split adds the merge phase.
    const int G = c->sm_count;
    double best = 1e30;
    int best_s = 1;
    std::vector<double> diff(G + 1);
    for (int s_try : {1, 2, 3, 4, 6, 8, 10, 12, 16, 20}) {
      const int kps = (int)align_up((size_t)(max_kv + s_try - 1) / s_try, 16);
      if (s_try > 1 && kps < 256) break;
      std::fill(diff.begin(), diff.end(), 0.0);
      double everywhere = 0;
      long long off = 0;
      for (int i = 0; i < n_attn; ++i) {
        const int kv = attn[i].w + attn[i].y, mt = (attn[i].y * qgroup + 15) / 16, keys = std::min(kps, kv);
        // key ranges of kTcAttnMinKeys and more run on tensor memory: 64-key tiles, whatever the number of query vectors
        const bool tc_item = tc_capable && keys >= kTcAttnMinKeys;      // in such a pass every long key range takes that path
        const double unit = tc_item ? 6.0 + ((keys + 63) / 64) * 0.8 : 5.0 + mt * ((keys + 127) / 128) * 1.9;
        // all s_try x nkv slots of the item are dealt out; splits past its last key return at once
        const long long used = (long long)std::min(s_try, (kv + kps - 1) / kps) * md.nkv, slots = (long long)s_try * md.nkv;
        everywhere += unit * (double)(used / G);
        const int rem = (int)(used % G), at = (int)(off % G);
        if (rem) {
          diff[at] += unit;
          if (at + rem <= G) diff[at + rem] -= unit;
          else { diff[G] -= unit; diff[0] += unit; diff[at + rem - G] -= unit; }
        }
        off += slots;
      }
      double load = 0, worst = 0;
      for (int g = 0; g < G; ++g) { load += diff[g]; worst = std::max(worst, load); }
      // merge phase: a barrier and a load round trip, then one (row, head) per 128 threads
      const double merge = 6.0 + 1.5 * (((double)R * md.nq + 2 * G - 1) / (2 * G));
      const double t = everywhere + worst + (s_try > 1 ? merge : 0.0);
      if (t < best) { best = t; best_s = s_try; }
    }
    n_splits = best_s;
    if (tc_capable && c->prefer_tc_attn) n_splits = std::max(1, std::min(n_splits, max_kv / kTcAttnMinKeys));
  }
  // passes with more rows than the one-launch forward takes (prompt chunks): every attention item keeps one key split
  const bool big_pass = M.use_persist && !(R <= 128 && n_logit <= 128);
  if (big_pass) n_splits = 1;
  int keys_per_split = (int)align_up((size_t)(max_kv + n_splits - 1) / n_splits, M.use_persist ? 16 : kAttnKeyTile);
  n_splits = (max_kv + keys_per_split - 1) / keys_per_split;
  if ((size_t)R * n_splits > (size_t)ML.partial_rows) return HSD_E_INVALID_ARG;

  TimerPair *tp = nullptr;
  if (c->timers_ok && c->timers_used < kTimerPairs) {
    tp = &c->timers[c->timers_used++];
    tp->level = level;
    cudaEventRecord(tp->a, c->stream);
  }
  cudaStream_t s = c->stream;
  auto mark_valid = [&]() {
    // the pass (re)wrote the KV of its rows in every layer it ran: with early exits that covers the caches of
    // the levels below as well (they ARE the first layers); a separate model has a cache of its own
    for (const SeqWork &w : work)
      for (int g = c->shared_cache ? 0 : level; g <= level; ++g) c->len_g[w.b][g] = w.end;
  };
  if (M.use_persist && R <= 128 && n_logit <= 128) {
    // one cooperative launch runs the whole pass
    FwdArgs a;
    a.d = md.d; a.nq = md.nq; a.nkv = md.nkv; a.hd = md.hd; a.ff = md.ff; a.V = md.V;
    a.n_run = c->exits[level]; a.lm_map = md.n_layers * 7 + level; a.max_seq = md.max_seq; a.page = md.page;
    a.page_shift = 0;
    while ((1 << a.page_shift) < md.page) ++a.page_shift;
    a.pages_per_seq = md.pages_per_seq; a.n_pages = md.n_pages; a.eps = md.eps;
    a.wmaps = c->dev<CUtensorMap>(ML.wmaps_dev);
    a.layers = c->dev<FwdLayerDev>(ML.layers_dev);
    a.embed = (const __nv_bfloat16 *)M.embed; a.final_norm = (const __nv_bfloat16 *)c->level_norm[level];
    a.cos_tab = c->dev<float>(ML.cos_tab); a.sin_tab = c->dev<float>(ML.sin_tab);
    a.R = R; a.L = n_logit; a.n_attn = n_attn; a.attn_rows = arows; a.n_splits = n_splits; a.keys_per_split = keys_per_split;
    a.tokens = c->dev<int>(L.tokens); a.page_table = c->dev<int>(L.page_table);
    a.row_seq = rb.row_seq; a.row_pos = rb.row_pos; a.lrow_src = rb.lrow_src; a.attn_items = rb.attn; a.lrow_dst = rb.lrow_dst;
    a.x = c->dev<float>(ML.x);
    a.h = c->dev<__nv_bfloat16>(ML.h); a.q = c->dev<__nv_bfloat16>(ML.q); a.att = c->dev<__nv_bfloat16>(ML.att);
    a.act = c->dev<__nv_bfloat16>(ML.act); a.hf = c->dev<__nv_bfloat16>(ML.hf);
    a.logits = (__nv_bfloat16 *)(c->ws + L.logits[level]);
    a.attn_partials = c->dev<float>(ML.partials); a.attn_counters = c->dev<int>(ML.attn_counters);
    a.pieces = (float *)(c->ws + ML.tc_scratch + kTcCtrlBytes); a.tile_counters = (int *)(c->ws + ML.tc_scratch + 256);
    a.grid_counter = c->dev<unsigned>(L.grid_counter); a.status = (int *)(c->ws + c->status_off);
    const int np = tc_npad(std::max(R, n_logit));
    const int pi = np == 16 ? 0 : np == 32 ? 1 : np == 64 ? 2 : 3;
    // few rows: fetch exactly the rows that exist (the MMA still reads `np` rows of the stage; the rest is stale
    // shared memory that only feeds accumulator columns nobody reads): 148 CTAs x K / 64 boxes per GEMM add up
    const int box_rows = std::max(R, n_logit) <= 16 ? std::max(R, n_logit) : np;
    a.a_box_rows = box_rows;
    // the new keys of an attention item are then its own rows only: the QKV finish phase folds into attention
    a.fuse_qkv = (one_item_per_seq && !c->no_fuse_qkv) ? 1 : 0;
    // few rows: the SwiGLU finish folds into the down projection (its CTAs build their activation tiles)
    a.fuse_gu = (R <= 4 && !c->no_fuse_gu) ? 1 : 0;
    // the norms after the residual projections start on otherwise idle CTAs as soon as the pieces are there
    a.early_norm = c->no_early_norm ? 0 : 1;
    // long key ranges: attention work items on tcgen05 / tensor memory (they take their q / k / v from the finish phase)
    a.tc_attn = (tc_capable && keys_per_split >= kTcAttnMinKeys) ? 1 : 0;
    if (a.tc_attn) a.fuse_qkv = 0;
    a.pieces2 = (float *)(c->ws + ML.tc_pieces2);
    for (int b = 0; b < 4; ++b) a.amap[b] = box_rows <= 16 ? M.amaps_rows[b][box_rows - 1] : M.amaps[b][pi];
    a.prof = nullptr;
#ifdef HSD_PROFILE
    // profiling build (-DHSD_PROFILE): HSD_PROFILE=<file> dumps the barrier timeline of the latest top-level pass
    const char *prof_path = getenv("HSD_PROFILE");
    const char *prof_rows = getenv("HSD_PROFILE_MIN_ROWS");       // e.g. 100: the prompt's chunks instead of decode passes
    const bool prof = prof_path && level == c->n_levels - 1 && (prof_rows ? R >= atoi(prof_rows) : n_logit > 0);
    if (prof) {
      a.prof = c->dev<unsigned long long>(ML.prof);
      HSD_CUDA_OK(cudaMemsetAsync(a.prof, 0, (size_t)c->sm_count * kFwdProfEvents * 8, s));
    }
#endif
    HSD_CUDA_OK(cudaMemsetAsync(a.grid_counter, 0, 128, s));
    int stp = launch_forward_persistent(a, np, c->sm_count, s);
    if (stp) return stp;
#ifdef HSD_PROFILE
    if (prof) {
      std::vector<unsigned long long> ev((size_t)c->sm_count * kFwdProfEvents);
      if (cudaMemcpyAsync(ev.data(), a.prof, ev.size() * 8, cudaMemcpyDeviceToHost, s) == cudaSuccess &&
          cudaStreamSynchronize(s) == cudaSuccess) {
        FILE *f = fopen(prof_path, "w");
        if (f) {
          fprintf(f, "%d %d %d %d\n", c->sm_count, kFwdProfEvents, a.n_run, R);
          for (int b = 0; b < c->sm_count; ++b) {
            for (int e = 0; e < kFwdProfEvents; ++e)
              fprintf(f, "%llu ", ev[(size_t)b * kFwdProfEvents + e]);
            fprintf(f, "\n");
          }
          fclose(f);
        }
      }
    }
#endif
    if (tp) cudaEventRecord(tp->b, s);
    c->stats[level].forwards++;
    c->stats[level].rows += R;
    mark_valid();
    return HSD_OK;
  }
  float *x = c->dev<float>(ML.x);
  void *h = c->dev<void>(ML.h), *q = c->dev<void>(ML.q), *att = c->dev<void>(ML.att), *act = c->dev<void>(ML.act);
  float *qkv = c->dev<float>(ML.qkv);
  const int *pt = c->dev<int>(L.page_table);
#define HSD_TRY(e) do { int st__ = (e); if (st__) return st__; } while (0)
  HSD_TRY(launch_embed(md, M.embed, c->dev<int>(L.tokens), rb, x, s));
  for (int l = 0; l < c->exits[level]; ++l) {
    const void *const *w = &M.lw[(size_t)l * 9];
    void *kp = c->ws + ML.k_pool + ML.pool_layer_stride * l, *vp = c->ws + ML.v_pool + ML.pool_layer_stride * l;
    HSD_TRY(launch_rmsnorm(md, x, w[0], nullptr, R, h, s));
    GemmSegs qkv_segs = {{w[1], w[2], w[3]}, {md.nq * md.hd, md.nkv * md.hd, md.nkv * md.hd}, 3};
    HSD_TRY(gemm(c, M, 0, h, R, md.d, qkv_segs, l * 7 + 0, GEMM_STORE_F32, qkv, nullptr, nullptr));
    HSD_TRY(launch_rope_kv(md, qkv, rb, c->dev<float>(ML.cos_tab), c->dev<float>(ML.sin_tab), pt, kp, vp, q, s));
    if (big_pass) {                                       // tensor-core attention of the persistent forward, as a launch of its own
      FwdArgs fa = {};
      fa.d = md.d; fa.nq = md.nq; fa.nkv = md.nkv; fa.hd = md.hd; fa.ff = md.ff; fa.V = md.V; fa.max_seq = md.max_seq; fa.page = md.page;
      while ((1 << fa.page_shift) < md.page) ++fa.page_shift;
      fa.pages_per_seq = md.pages_per_seq; fa.n_pages = md.n_pages;
      fa.R = R; fa.n_attn = n_attn; fa.attn_rows = arows; fa.n_splits = 1; fa.keys_per_split = keys_per_split;
      fa.page_table = pt; fa.attn_items = rb.attn; fa.row_seq = rb.row_seq; fa.row_pos = rb.row_pos;
      fa.q = (__nv_bfloat16 *)q; fa.att = (__nv_bfloat16 *)att; fa.attn_partials = c->dev<float>(ML.partials);
      HSD_TRY(launch_attention_tiles(fa, (__nv_bfloat16 *)kp, (__nv_bfloat16 *)vp, c->sm_count, s));
    } else {
      HSD_TRY(launch_attention(md, q, rb, pt, kp, vp, c->dev<float>(ML.partials), keys_per_split, n_splits, att, s));
    }
    GemmSegs o_segs = {{w[4], nullptr, nullptr}, {md.d, 0, 0}, 1};
    HSD_TRY(gemm(c, M, 1, att, R, md.nq * md.hd, o_segs, l * 7 + 3, GEMM_ADD_F32, x, nullptr, nullptr));
    HSD_TRY(launch_rmsnorm(md, x, w[5], nullptr, R, h, s));
    GemmSegs gu_segs = {{w[6], w[7], nullptr}, {md.ff, md.ff, 0}, 2};
    HSD_TRY(gemm(c, M, 0, h, R, md.d, gu_segs, l * 7 + 4, GEMM_SWIGLU_T, nullptr, act, nullptr));
    GemmSegs d_segs = {{w[8], nullptr, nullptr}, {md.d, 0, 0}, 1};
    HSD_TRY(gemm(c, M, 2, act, R, md.ff, d_segs, l * 7 + 6, GEMM_ADD_F32, x, nullptr, nullptr));
  }
  if (n_logit > 0) {
    void *hf = c->dev<void>(ML.hf);
    HSD_TRY(launch_rmsnorm(md, x, c->level_norm[level], rb.lrow_src, n_logit, hf, s));
    GemmSegs lm_segs = {{c->level_head[level], nullptr, nullptr}, {md.V, 0, 0}, 1};
    HSD_TRY(gemm(c, M, 3, hf, n_logit, md.d, lm_segs, md.n_layers * 7 + level, GEMM_STORE_T_SCATTER, nullptr, c->ws + L.logits[level],
                 rb.lrow_dst));
  }
  if (tp) cudaEventRecord(tp->b, s);
  c->stats[level].forwards++;
  c->stats[level].rows += R;
  mark_valid();
  return HSD_OK;
}

// ---------------------------------------------------------------------------- decision log
int fetch_tokens(hsd_ctx *c, int b, int pos0, int n, std::vector<int32_t> &out) {
  size_t base = out.size();
  out.resize(base + n);
  if (n == 0) return HSD_OK;
  if (cudaMemcpyAsync(out.data() + base, c->dev<int>(c->lay.tokens) + (size_t)b * c->md.max_seq + pos0, (size_t)n * 4,
                      cudaMemcpyDeviceToHost, c->stream) != cudaSuccess)
    return HSD_E_CUDA;
  return cudaStreamSynchronize(c->stream) == cudaSuccess ? HSD_OK : HSD_E_CUDA;
}

int trace_write(hsd_ctx *c, int level, int b, uint32_t serial, int ctx_len, int t, int n, int fwd_rows, int logit_rows,
                long long logit_row0, const std::vector<int32_t> &toks) {
  if (!c->trace) return HSD_OK;
  const ModelDims &md = c->md;
  int has_logits = c->trace_records < c->trace_logit_calls;
  int32_t hdr[12] = {(int32_t)kTraceMagic, level, b, (int32_t)serial, ctx_len, t, n, fwd_rows, logit_rows, has_logits, md.V,
                     md.dtype};
  std::vector<char> rows;
  if (has_logits) {
    rows.resize((size_t)logit_rows * md.V * elem_size(md.dtype));
    if (cudaMemcpyAsync(rows.data(), c->ws + c->lay.logits[level] + (size_t)logit_row0 * md.V * elem_size(md.dtype),
                        rows.size(), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess)
      return HSD_E_CUDA;
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return HSD_E_CUDA;
  }
  if (fwrite(hdr, 4, 12, c->trace) != 12) return HSD_E_IO;
  if (!toks.empty() && fwrite(toks.data(), 4, toks.size(), c->trace) != toks.size()) return HSD_E_IO;
  if (has_logits && fwrite(rows.data(), 1, rows.size(), c->trace) != rows.size()) return HSD_E_IO;
  c->trace_records++;
  return HSD_OK;
}

// ---------------------------------------------------------------------------- Algorithm 1
// Level 0: T_0 single-step forwards, each followed by the draft sample written into the token
// buffer on the device (no host round trip inside the loop).
int run_level0(hsd_ctx *c, const std::vector<int> &act) {
  const Layout &L = c->lay;
  const int steps = c->n_levels > 1 ? c->T[0] : 1;
  std::vector<int> ctx0(act.size());
  std::vector<uint32_t> ser(act.size());
  for (size_t i = 0; i < act.size(); ++i) {
    ctx0[i] = c->buf_len[act[i]];
    ser[i] = c->serial[act[i]][0]++;
  }
  for (int j = 0; j < steps; ++j) {
    std::vector<SeqWork> work;
    for (int b : act) {
      int len = c->buf_len[b];
      int start = std::min(c->len_g[b][0], len - 1);
      work.push_back({b, start, len, len - 1, j});
    }
    HSD_TRY(forward(c, 0, work));
    char *host, *devp;
    HSD_TRY(ring_acquire(c, &host, &devp));
    SampleRow *rows = (SampleRow *)host;
    for (size_t i = 0; i < act.size(); ++i) {
      int b = act[i];
      rows[i].logit_row = (long long)b * L.slots[0] + j;
      rows[i].out_index = (long long)b * c->md.max_seq + c->buf_len[b];
      rows[i].j = j; rows[i].serial = ser[i]; rows[i].seq = b; rows[i].level = 0;
      c->buf_len[b]++;
    }
    HSD_CUDA_OK(cudaMemcpyAsync(devp, host, act.size() * sizeof(SampleRow), cudaMemcpyHostToDevice, c->stream));
    HSD_TRY(launch_draft_sample(c->ws + L.logits[0], c->md.dtype, c->md.V, (const SampleRow *)devp, (int)act.size(), 1, 0,
                                c->seed, c->dev<int>(L.tokens), c->stream));
  }
  for (size_t i = 0; i < act.size(); ++i) {
    hsd_level_stats &st = c->stats[0];
    st.calls++;
    st.emitted += steps;
    if (c->trace) {
      std::vector<int32_t> toks;
      HSD_TRY(fetch_tokens(c, act[i], ctx0[i], steps, toks));
      HSD_TRY(trace_write(c, 0, act[i], ser[i], ctx0[i], 0, steps, steps, steps, (long long)act[i] * L.slots[0], toks));
    }
  }
  return HSD_OK;
}

// Verify(level) for the active sequences: drafts are tokens [ctx[b], buf_len[b]) with draft rows in
// the lower level's slots 0..t-1; this level's rows go to its slots count[b]..count[b]+t.
int run_verify(hsd_ctx *c, int level, const std::vector<int> &act, const std::vector<int> &ctx, std::vector<int> &count) {
  const Layout &L = c->lay;
  std::vector<SeqWork> work;
  int t_max = 0;
  for (int b : act) {
    int t = c->buf_len[b] - ctx[b];
    if (t < 1 || ctx[b] < 1) return HSD_E_INVALID_ARG;
    int start = std::min(c->len_g[b][level], ctx[b] - 1);
    work.push_back({b, start, c->buf_len[b], ctx[b] - 1, count[b]});
    t_max = std::max(t_max, t);
  }
  HSD_TRY(forward(c, level, work));
  char *host, *devp;
  HSD_TRY(ring_acquire(c, &host, &devp));
  VerifySeq *vs = (VerifySeq *)host;
  std::vector<uint32_t> ser(act.size());
  for (size_t i = 0; i < act.size(); ++i) {
    int b = act[i];
    ser[i] = c->serial[b][level]++;
    vs[i].p_row0 = (long long)b * L.slots[level] + count[b];
    vs[i].q_row0 = (long long)b * L.slots[level - 1];
    vs[i].tok_off = (long long)b * c->md.max_seq + ctx[b];
    vs[i].t = c->buf_len[b] - ctx[b];
    vs[i].serial = ser[i]; vs[i].seq = b; vs[i].level = level;
  }
  HSD_CUDA_OK(cudaMemcpyAsync(devp, host, act.size() * sizeof(VerifySeq), cudaMemcpyHostToDevice, c->stream));
  std::vector<std::vector<int32_t>> drafts(c->trace ? act.size() : 0);
  for (size_t i = 0; i < drafts.size(); ++i) HSD_TRY(fetch_tokens(c, act[i], ctx[act[i]], c->buf_len[act[i]] - ctx[act[i]], drafts[i]));
  HSD_TRY(launch_verify(c->ws + L.logits[level], c->ws + L.logits[level - 1], c->dev<int>(L.tokens), c->md.dtype, c->md.V,
                        (int)act.size(), t_max, (const VerifySeq *)devp, 0, 0, 0, c->ws + L.vscratch, c->seed, nullptr,
                        c->dev<int>(L.n_acc), 1, c->stream, c->coin24[level]));
  HSD_CUDA_OK(cudaMemcpyAsync(c->n_acc_host, c->dev<int>(L.n_acc), act.size() * 4, cudaMemcpyDeviceToHost, c->stream));
  HSD_TRY(sync_stream(c));
  hsd_level_stats &st = c->stats[level];
  for (size_t i = 0; i < act.size(); ++i) {
    int b = act[i], t = c->buf_len[b] - ctx[b], n = c->n_acc_host[i];
    if (n < 0 || n > t) return HSD_E_CUDA;
    // rollback / commit: the buffer keeps x_1..x_n and m; the position of m (and everything the
    // rejected drafts wrote) is valid in no layer group
    c->buf_len[b] = ctx[b] + n + 1;
    for (int g = 0; g < c->n_levels; ++g) c->len_g[b][g] = std::min(c->len_g[b][g], ctx[b] + n);
    trim_pages(c, b, c->buf_len[b]);
    st.calls++;
    st.drafted += t;
    st.tested += std::min(n + 1, t);
    st.accepted += n;
    st.emitted += n + 1;
    if (c->trace) {
      HSD_TRY(fetch_tokens(c, b, ctx[b] + n, 1, drafts[i]));          // the final token m
      HSD_TRY(trace_write(c, level, b, ser[i], ctx[b], t, n, work[i].end - work[i].start, t + 1,
                          (long long)b * L.slots[level] + count[b], drafts[i]));
    }
    count[b] += n + 1;
  }
  return HSD_OK;
}

int run_level(hsd_ctx *c, int level, const std::vector<int> &act) {
  if (act.empty()) return HSD_OK;
  if (level == 0) return run_level0(c, act);
  const int K = c->n_levels - 1;
  std::vector<int> ctx(c->max_batch, 0), count(c->max_batch, 0);
  if (level == K) {
    for (int b : act) ctx[b] = c->buf_len[b];
    HSD_TRY(run_level(c, level - 1, act));
    return run_verify(c, level, act, ctx, count);
  }
  for (;;) {
    std::vector<int> need;
    for (int b : act)
      if (count[b] < c->T[level]) need.push_back(b);
    if (need.empty()) break;
    for (int b : need) ctx[b] = c->buf_len[b];
    HSD_TRY(run_level(c, level - 1, need));
    HSD_TRY(run_verify(c, level, need, ctx, count));
  }
  return HSD_OK;
}

int prefill(hsd_ctx *c, int batch, int prompt_len) {
  // the target runs over prompt positions [0, P-1); the last prompt token stays unprocessed and is
  // every level's first catch-up row
  const int K = c->n_levels - 1;
  int end = prompt_len - 1;
  std::vector<int> done(batch, 0);
  for (;;) {
    std::vector<SeqWork> work;
    int budget = kPrefillRows;
    for (int b = 0; b < batch && budget > 0; ++b) {
      if (done[b] >= end) continue;
      int rows = std::min(budget, end - done[b]);
      work.push_back({b, done[b], done[b] + rows, -1, 0});
      done[b] += rows;
      budget -= rows;
    }
    if (work.empty()) break;
    // early exits: the target's pass fills the one cache; separate models: each fills its own
    for (int lvl = c->shared_cache ? K : 0; lvl <= K; ++lvl) HSD_TRY(forward(c, lvl, work));
  }
  return HSD_OK;
}

// Sets up one model of a context: rotary tables, tensor maps, device-side tables.  `head_levels`: the levels whose
// output-head tensor map slots are (re)built for this model.
int init_model(hsd_ctx *c, Model &M, const hsd_model_desc *model, const ModelLayout &ml) {
  const Layout &lay = c->lay;
  M.md = ModelDims{model->n_layers, model->d_model, model->n_q_heads, model->n_kv_heads, model->head_dim, model->d_ff,
                   model->vocab, model->dtype, model->rms_eps, model->rope_theta, model->max_seq,
                   model->page_size ? model->page_size : 16, lay.pages_per_seq, lay.n_pages};
  M.lay = ml;
  M.embed = model->embed; M.final_norm = model->final_norm; M.lm_head = model->lm_head;
  M.lw.assign(model->layer_weights, model->layer_weights + (size_t)model->n_layers * 9);
  const ModelDims &md = M.md;
  {  // rotary tables: angles in double, rounded to fp32
    const int half = md.hd / 2;
    std::vector<float> cs((size_t)md.max_seq * half), sn((size_t)md.max_seq * half);
    for (int p = 0; p < md.max_seq; ++p)
      for (int k = 0; k < half; ++k) {
        double ang = (double)p * pow((double)md.theta, -2.0 * k / (double)md.hd);
        cs[(size_t)p * half + k] = (float)cos(ang);
        sn[(size_t)p * half + k] = (float)sin(ang);
      }
    if (cudaMemcpy(c->ws + ml.cos_tab, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(c->ws + ml.sin_tab, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess)
      return HSD_E_CUDA;
  }
  // tensor-core path: bf16 model whose contraction sizes are multiples of the 64-element k-block
  M.use_tc = model->dtype == HSD_BF16 && model->d_model % kTcBlockK == 0 && model->d_ff % kTcBlockK == 0 &&
             (model->n_q_heads * model->head_dim) % kTcBlockK == 0 && tc_init() == HSD_OK;
  if (!M.use_tc) return HSD_OK;
  int st = HSD_OK;
  M.wmaps.resize((size_t)md.n_layers * 7 + kHeadMaps);
  const long long rows7[7] = {(long long)md.nq * md.hd, (long long)md.nkv * md.hd, (long long)md.nkv * md.hd, md.d, md.ff, md.ff, md.d};
  const long long cols7[7] = {md.d, md.d, md.d, (long long)md.nq * md.hd, md.d, md.d, md.ff};
  const int widx[7] = {1, 2, 3, 4, 6, 7, 8};
  for (int l = 0; l < md.n_layers && !st; ++l)
    for (int k = 0; k < 7 && !st; ++k)
      st = tc_make_map(&M.wmaps[(size_t)l * 7 + k], M.lw[(size_t)l * 9 + widx[k]], rows7[k], cols7[k], kTcBoxRows);
  for (int i = 0; i < kHeadMaps && !st; ++i) st = tc_make_map(&M.wmaps[(size_t)md.n_layers * 7 + i], M.lm_head, md.V, md.d, kTcBoxRows);
  const size_t abuf_off[4] = {ml.h, ml.att, ml.act, ml.hf};
  const long long acols[4] = {md.d, (long long)md.nq * md.hd, md.ff, md.d};
  const long long arows[4] = {lay.max_rows, lay.max_rows, lay.max_rows, lay.max_logit_rows};
  const int npads[5] = {16, 32, 64, 128, 256};
  for (int b = 0; b < 4 && !st; ++b)
    for (int p = 0; p < 5 && !st; ++p) st = tc_make_map(&M.amaps[b][p], c->ws + abuf_off[b], arows[b], acols[b], npads[p]);
  for (int b = 0; b < 4 && !st; ++b)
    for (int r = 1; r <= 16 && !st; ++r) st = tc_make_map(&M.amaps_rows[b][r - 1], c->ws + abuf_off[b], arows[b], acols[b], r);
  if (!st && cudaMemset(c->ws + ml.tc_scratch, 0, kTcCtrlBytes) != cudaSuccess) st = HSD_E_CUDA;
  if (st) return st;
  // tables of the persistent forward: tensor maps and per-layer pointers in device memory
  std::vector<FwdLayerDev> ld(md.n_layers);
  for (int l = 0; l < md.n_layers; ++l) {
    ld[l].attn_norm = (const __nv_bfloat16 *)M.lw[(size_t)l * 9 + 0];
    ld[l].mlp_norm = (const __nv_bfloat16 *)M.lw[(size_t)l * 9 + 5];
    ld[l].k_pool = (__nv_bfloat16 *)(c->ws + ml.k_pool + ml.pool_layer_stride * l);
    ld[l].v_pool = (__nv_bfloat16 *)(c->ws + ml.v_pool + ml.pool_layer_stride * l);
  }
  if (cudaMemcpy(c->ws + ml.wmaps_dev, M.wmaps.data(), M.wmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(c->ws + ml.layers_dev, ld.data(), ld.size() * sizeof(FwdLayerDev), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemset(c->ws + ml.attn_counters, 0, 16384) != cudaSuccess)
    return HSD_E_CUDA;
  int coop = 0, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
  M.use_persist = coop != 0 && fwd_persist_supported(md.hd, md.nq / md.nkv) && md.d % 256 == 0 && md.d <= 4096 &&
                  (md.d / kTcBlockM) * 2 <= c->sm_count && md.n_layers <= 64 && (md.page & (md.page - 1)) == 0 && md.page >= 16;
  return HSD_OK;
}

bool supported_dims(const hsd_model_desc *model) {
  if (model->head_dim != 32 && model->head_dim != 64 && model->head_dim != 128) return false;
  if (model->n_q_heads / model->n_kv_heads > 8) return false;
  const int vec = model->dtype == HSD_BF16 ? 8 : 4;
  return !(model->d_model % vec || model->d_ff % vec || (model->n_q_heads * model->head_dim) % vec);
}

// Common part of the two create calls.  models[0 .. n_models): one decoder (early exits) or one per level.
int create_ctx(const hsd_model_desc *models, int n_models, const int32_t *exit_layers, int n_levels, const int32_t *T,
                      void *workspace, size_t workspace_bytes, hsd_ctx **out) {
  for (int mi = 0; mi < n_models; ++mi) {
    const hsd_model_desc *model = &models[mi];
    if (!model->embed || !model->final_norm || !model->lm_head || !model->layer_weights) return HSD_E_INVALID_ARG;
    for (int i = 0; i < model->n_layers * 9; ++i)
      if (!model->layer_weights[i]) return HSD_E_INVALID_ARG;
    if (!supported_dims(model)) return HSD_E_UNSUPPORTED;
  }
  if (!workspace || ((uintptr_t)workspace & 255) != 0) return HSD_E_INVALID_ARG;
  Layout lay = make_layout(models, n_models, n_levels, T);
  if (workspace_bytes < lay.total) return HSD_E_WORKSPACE_TOO_SMALL;
  hsd_ctx *c = new (std::nothrow) hsd_ctx();
  if (!c) return HSD_E_INVALID_ARG;
  c->n_levels = n_levels;
  c->max_batch = models[0].max_batch;
  c->shared_cache = exit_layers != nullptr;
  c->exits.resize(n_levels);
  c->level_model.resize(n_levels);
  for (int i = 0; i < n_levels; ++i) {
    c->level_model[i] = c->shared_cache ? 0 : i;
    c->exits[i] = c->shared_cache ? exit_layers[i] : models[i].n_layers;
  }
  if (n_levels > 1) c->T.assign(T, T + n_levels - 1);
  c->lay = lay;
  c->ws = (char *)workspace;
  c->coin24.assign(n_levels, kNoCoin);
  c->ring_host = nullptr; c->n_acc_host = nullptr; c->page_table_host = nullptr; c->status_host = nullptr;
  c->sm_count = device_sm_count();
  c->trace = nullptr; c->trace_logit_calls = 0; c->trace_records = 0;
  c->ring_next = 0; c->ring_in_flight = 0; c->timers_used = 0; c->timers_ok = true; c->stream = nullptr; c->seed = 0;
  c->status_off = lay.model[0].tc_scratch;
  bool ok = cudaMallocHost(&c->ring_host, lay.ring_slot * kRingSlots) == cudaSuccess &&
            cudaMallocHost(&c->n_acc_host, (size_t)c->max_batch * 4) == cudaSuccess &&
            cudaMallocHost(&c->page_table_host, (size_t)c->max_batch * lay.pages_per_seq * 4) == cudaSuccess &&
            cudaMallocHost(&c->status_host, 4) == cudaSuccess;
  for (int i = 0; i < kTimerPairs; ++i) { c->timers[i].a = nullptr; c->timers[i].b = nullptr; }
  for (int i = 0; ok && i < kTimerPairs; ++i)
    c->timers_ok = c->timers_ok && cudaEventCreate(&c->timers[i].a) == cudaSuccess && cudaEventCreate(&c->timers[i].b) == cudaSuccess;
  int st = ok ? HSD_OK : HSD_E_CUDA;
  if (!st && (cudaMemset(c->ws + c->status_off, 0, 256) != cudaSuccess || cudaMemset(c->ws + lay.grid_counter, 0, 256) != cudaSuccess))
    st = HSD_E_CUDA;
  c->models.resize(n_models);
  for (int mi = 0; mi < n_models && !st; ++mi) {
    st = init_model(c, c->models[mi], &models[mi], lay.model[mi]);
    c->any_tc = c->any_tc || c->models[mi].use_tc;
  }
  if (st) {
    hsd_destroy(c);
    return st;
  }
  c->md = c->models.back().md;
  c->level_head.resize(n_levels);
  c->level_norm.resize(n_levels);
  for (int i = 0; i < n_levels; ++i) {
    c->level_head[i] = c->model_of(i).lm_head;
    c->level_norm[i] = c->model_of(i).final_norm;
  }
  c->stats.assign(n_levels, hsd_level_stats{});
  *c->status_host = 0;
  *out = c;
  return HSD_OK;
}

}  // namespace

extern "C" {

size_t hsd_workspace_bytes(const hsd_model_desc *model, const int32_t *exit_layers, int n_levels, const int32_t *T) {
  if (!valid_model(model, exit_layers, n_levels, T)) return 0;
  return make_layout(model, 1, n_levels, T).total;
}

size_t hsd_models_workspace_bytes(const hsd_model_desc *models, int n_levels, const int32_t *T) {
  if (!valid_models(models, n_levels, T)) return 0;
  return make_layout(models, n_levels, n_levels, T).total;
}

int hsd_create(const hsd_model_desc *model, const int32_t *exit_layers, int n_levels, const int32_t *T, void *workspace,
               size_t workspace_bytes, hsd_ctx **out) {
  if (!out) return HSD_E_INVALID_ARG;
  *out = nullptr;
  if (!valid_model(model, exit_layers, n_levels, T)) return HSD_E_INVALID_ARG;
  return create_ctx(model, 1, exit_layers, n_levels, T, workspace, workspace_bytes, out);
}

int hsd_create_models(const hsd_model_desc *models, int n_levels, const int32_t *T, void *workspace, size_t workspace_bytes,
                      hsd_ctx **out) {
  if (!out) return HSD_E_INVALID_ARG;
  *out = nullptr;
  if (!valid_models(models, n_levels, T)) return HSD_E_INVALID_ARG;
  return create_ctx(models, n_levels, nullptr, n_levels, T, workspace, workspace_bytes, out);
}

int hsd_set_phase_folding(hsd_ctx *c, int fold_qkv, int fold_gate_up, int early_norm) {
  if (!c) return HSD_E_INVALID_ARG;
  c->no_fuse_qkv = fold_qkv == 0;
  c->no_fuse_gu = fold_gate_up == 0;
  c->no_early_norm = early_norm == 0;
  return HSD_OK;
}

int hsd_set_tensor_attention(hsd_ctx *c, int enabled) {
  if (!c) return HSD_E_INVALID_ARG;
  c->no_tc_attn = enabled == 0;
  c->prefer_tc_attn = enabled == 2;
  return HSD_OK;
}

int hsd_generate(hsd_ctx *c, const int32_t *prompt_ids, int batch, int prompt_len, int n_new, uint64_t seed, void *stream,
                 int32_t *out_tokens, hsd_level_stats *stats, double *timing_ms) {
  if (!c || !prompt_ids || !out_tokens || batch < 1 || batch > c->max_batch || prompt_len < 1 || n_new < 1)
    return HSD_E_INVALID_ARG;
  int sumT = 0;
  for (int t : c->T) sumT += t;
  if ((long long)prompt_len + n_new + sumT + c->n_levels + 1 > c->md.max_seq) return HSD_E_INVALID_ARG;
  c->stream = (cudaStream_t)stream;
  c->seed = seed;
  c->stats.assign(c->n_levels, hsd_level_stats{});
  c->buf_len.assign(c->max_batch, 0);
  c->len_g.assign(c->max_batch, std::vector<int>(c->n_levels, 0));
  c->serial.assign(c->max_batch, std::vector<uint32_t>(c->n_levels, 0));
  c->n_pages_of.assign(c->max_batch, 0);
  c->pt_dirty.assign(c->max_batch, 0);
  c->free_pages.clear();
  for (int p = c->lay.n_pages - 1; p >= 0; --p) c->free_pages.push_back(p);
  c->trace_records = 0;
  cudaEvent_t e0 = nullptr, e1 = nullptr, e2 = nullptr;
  bool ev = cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess && cudaEventCreate(&e2) == cudaSuccess;
  int st = HSD_OK;
  auto body = [&]() -> int {
    if (ev) cudaEventRecord(e0, c->stream);
    HSD_CUDA_OK(cudaMemcpy2DAsync(c->dev<int>(c->lay.tokens), (size_t)c->md.max_seq * 4, prompt_ids, (size_t)prompt_len * 4,
                                  (size_t)prompt_len * 4, batch, cudaMemcpyDeviceToDevice, c->stream));
    for (int b = 0; b < batch; ++b) c->buf_len[b] = prompt_len;
    HSD_TRY(prefill(c, batch, prompt_len));
    HSD_TRY(sync_stream(c));
    c->stats.assign(c->n_levels, hsd_level_stats{});      // level counters cover the generation loop only
    if (ev) cudaEventRecord(e1, c->stream);
    const int K = c->n_levels - 1;
    for (;;) {
      std::vector<int> act;
      for (int b = 0; b < batch; ++b)
        if (c->buf_len[b] - prompt_len < n_new) act.push_back(b);
      if (act.empty()) break;
      HSD_TRY(run_level(c, K, act));
    }
    HSD_CUDA_OK(cudaMemcpy2DAsync(out_tokens, (size_t)n_new * 4, c->dev<int>(c->lay.tokens) + prompt_len,
                                  (size_t)c->md.max_seq * 4, (size_t)n_new * 4, batch, cudaMemcpyDeviceToDevice, c->stream));
    if (ev) cudaEventRecord(e2, c->stream);
    return sync_stream(c);
  };
  st = body();
  if (st != HSD_OK) cudaStreamSynchronize(c->stream);
  if (st == HSD_OK && timing_ms) {
    float a = 0.f, b = 0.f;
    if (ev) { cudaEventElapsedTime(&a, e0, e1); cudaEventElapsedTime(&b, e1, e2); }
    timing_ms[0] = a; timing_ms[1] = b;
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (e2) cudaEventDestroy(e2);
  if (st == HSD_OK && stats)
    for (int i = 0; i < c->n_levels; ++i) stats[i] = c->stats[i];
  if (c->trace) fflush(c->trace);
  return st;
}

// Logits of chosen exit layers at every position of one token sequence: the input of the calibration of
// Section 4.2 (acceptance rates between all candidate drafters).  One pass over the layers with the
// one-kernel-per-op path; after each chosen layer the shared final norm and output head are applied to all rows.
int hsd_layer_logits(hsd_ctx *c, const int32_t *token_ids, int n_tokens, const int32_t *layers, int n_layers_sel,
                     void *out_logits, void *stream) {
  if (!c || !token_ids || !layers || !out_logits || n_tokens < 1 || n_layers_sel < 1) return HSD_E_INVALID_ARG;
  Model &M = c->models.back();                  // the target's decoder
  const ModelDims &md = M.md;
  const Layout &L = c->lay;
  const ModelLayout &ML = M.lay;
  if (n_tokens > L.max_rows || n_tokens > md.max_seq || n_tokens > 128) return HSD_E_INVALID_ARG;
  for (int i = 0; i < n_layers_sel; ++i)
    if (layers[i] < 1 || layers[i] > md.n_layers || (i > 0 && layers[i] <= layers[i - 1])) return HSD_E_INVALID_ARG;
  c->stream = (cudaStream_t)stream;
  cudaStream_t s = c->stream;
  // the call owns the context like a generation does: sequence 0 holds the tokens, its pages are (re)assigned
  c->buf_len.assign(c->max_batch, 0);
  c->len_g.assign(c->max_batch, std::vector<int>(c->n_levels, 0));
  c->n_pages_of.assign(c->max_batch, 0);
  c->pt_dirty.assign(c->max_batch, 0);
  c->free_pages.clear();
  for (int p = L.n_pages - 1; p >= 0; --p) c->free_pages.push_back(p);
  HSD_CUDA_OK(cudaMemcpyAsync(c->dev<int>(L.tokens), token_ids, (size_t)n_tokens * 4, cudaMemcpyDeviceToDevice, s));
  HSD_TRY(ensure_pages(c, 0, n_tokens));
  const int R = n_tokens, n_attn = (R + kAttnRows - 1) / kAttnRows;
  char *host, *devp;
  HSD_TRY(ring_acquire(c, &host, &devp));
  size_t o_seq = 0, o_pos = align_up(o_seq + (size_t)R * 4, 16), o_attn = align_up(o_pos + (size_t)R * 4, 16),
         o_src = align_up(o_attn + (size_t)n_attn * 16, 16), o_dst = align_up(o_src + (size_t)R * 4, 16),
         bytes = o_dst + (size_t)R * 8;
  if (bytes > L.ring_slot) return HSD_E_INVALID_ARG;
  int *row_seq = (int *)(host + o_seq), *row_pos = (int *)(host + o_pos), *lsrc = (int *)(host + o_src);
  int4 *attn = (int4 *)(host + o_attn);
  long long *ldst = (long long *)(host + o_dst);
  for (int r = 0; r < R; ++r) { row_seq[r] = 0; row_pos[r] = r; lsrc[r] = r; ldst[r] = r; }
  for (int i = 0; i < n_attn; ++i) attn[i] = make_int4(i * kAttnRows, std::min(kAttnRows, R - i * kAttnRows), 0, i * kAttnRows);
  HSD_CUDA_OK(cudaMemcpyAsync(devp, host, bytes, cudaMemcpyHostToDevice, s));
  HSD_TRY(upload_page_tables(c));
  RowBatch rb;
  rb.R = R; rb.row_seq = (const int *)(devp + o_seq); rb.row_pos = (const int *)(devp + o_pos);
  rb.n_attn = n_attn; rb.attn = (const int4 *)(devp + o_attn); rb.max_kv_len = R; rb.L = R;
  rb.lrow_src = (const int *)(devp + o_src); rb.lrow_dst = (const long long *)(devp + o_dst);
  int n_splits = std::max(1, std::min((int)kMaxSplits, kAttnBlocksTarget / std::max(1, n_attn * md.nkv)));
  int keys_per_split = (int)align_up((size_t)(R + n_splits - 1) / n_splits, kAttnKeyTile);
  n_splits = (R + keys_per_split - 1) / keys_per_split;
  float *x = c->dev<float>(ML.x);
  void *h = c->dev<void>(ML.h), *q = c->dev<void>(ML.q), *att = c->dev<void>(ML.att), *act = c->dev<void>(ML.act);
  float *qkv = c->dev<float>(ML.qkv);
  const int *pt = c->dev<int>(L.page_table);
  const size_t es = elem_size(md.dtype);
  HSD_TRY(launch_embed(md, M.embed, c->dev<int>(L.tokens), rb, x, s));
  int next = 0;
  for (int l = 0; l < md.n_layers && next < n_layers_sel; ++l) {
    const void *const *w = &M.lw[(size_t)l * 9];
    void *kp = c->ws + ML.k_pool + ML.pool_layer_stride * l, *vp = c->ws + ML.v_pool + ML.pool_layer_stride * l;
    HSD_TRY(launch_rmsnorm(md, x, w[0], nullptr, R, h, s));
    GemmSegs qkv_segs = {{w[1], w[2], w[3]}, {md.nq * md.hd, md.nkv * md.hd, md.nkv * md.hd}, 3};
    HSD_TRY(gemm(c, M, 0, h, R, md.d, qkv_segs, l * 7 + 0, GEMM_STORE_F32, qkv, nullptr, nullptr));
    HSD_TRY(launch_rope_kv(md, qkv, rb, c->dev<float>(ML.cos_tab), c->dev<float>(ML.sin_tab), pt, kp, vp, q, s));
    HSD_TRY(launch_attention(md, q, rb, pt, kp, vp, c->dev<float>(ML.partials), keys_per_split, n_splits, att, s));
    GemmSegs o_segs = {{w[4], nullptr, nullptr}, {md.d, 0, 0}, 1};
    HSD_TRY(gemm(c, M, 1, att, R, md.nq * md.hd, o_segs, l * 7 + 3, GEMM_ADD_F32, x, nullptr, nullptr));
    HSD_TRY(launch_rmsnorm(md, x, w[5], nullptr, R, h, s));
    GemmSegs gu_segs = {{w[6], w[7], nullptr}, {md.ff, md.ff, 0}, 2};
    HSD_TRY(gemm(c, M, 0, h, R, md.d, gu_segs, l * 7 + 4, GEMM_SWIGLU_T, nullptr, act, nullptr));
    GemmSegs d_segs = {{w[8], nullptr, nullptr}, {md.d, 0, 0}, 1};
    HSD_TRY(gemm(c, M, 2, act, R, md.ff, d_segs, l * 7 + 6, GEMM_ADD_F32, x, nullptr, nullptr));
    if (layers[next] == l + 1) {                         // exit after layer l + 1: shared final norm + head on every row
      // (the normalised rows go to the h buffer, free between two layers and large enough for every row; the
      // buffer of the generation path's final norm holds the few logit rows of a verification only)
      HSD_TRY(launch_rmsnorm(md, x, M.final_norm, rb.lrow_src, R, h, s));
      GemmSegs lm_segs = {{M.lm_head, nullptr, nullptr}, {md.V, 0, 0}, 1};
      HSD_TRY(gemm(c, M, 0, h, R, md.d, lm_segs, md.n_layers * 7 + kHeadMaps - 1, GEMM_STORE_T_SCATTER, nullptr,
                   (char *)out_logits + (size_t)next * R * md.V * es, rb.lrow_dst));
      ++next;
    }
  }
  return sync_stream(c);
}

int hsd_set_exit_heads(hsd_ctx *c, const void *const *final_norms, const void *const *lm_heads) {
  if (!c) return HSD_E_INVALID_ARG;
  int st = sync_stream(c);                      // no pass of this context may be in flight
  if (st) return st;
  for (int i = 0; i < c->n_levels; ++i) {
    Model &M = c->model_of(i);
    c->level_norm[i] = (final_norms && final_norms[i]) ? final_norms[i] : M.final_norm;
    c->level_head[i] = (lm_heads && lm_heads[i]) ? lm_heads[i] : M.lm_head;
    if (((uintptr_t)c->level_head[i] & 15) != 0) return HSD_E_INVALID_ARG;
  }
  for (int i = 0; i < c->n_levels && !st; ++i) {
    Model &M = c->model_of(i);
    if (!M.use_tc) continue;
    const size_t slot = (size_t)M.md.n_layers * 7 + i;
    st = tc_make_map(&M.wmaps[slot], c->level_head[i], M.md.V, M.md.d, kTcBoxRows);
    if (!st && cudaMemcpy(c->ws + M.lay.wmaps_dev + slot * sizeof(CUtensorMap), &M.wmaps[slot], sizeof(CUtensorMap),
                          cudaMemcpyHostToDevice) != cudaSuccess)
      st = HSD_E_CUDA;
  }
  return st;
}

int hsd_set_iid_acceptance(hsd_ctx *c, const double *alphas) {
  if (!c) return HSD_E_INVALID_ARG;
  if (alphas)
    for (int i = 0; i + 1 < c->n_levels; ++i)
      if (!(alphas[i] >= 0.0 && alphas[i] <= 1.0)) return HSD_E_INVALID_ARG;
  for (int i = 1; i < c->n_levels; ++i)
    c->coin24[i] = alphas ? (uint32_t)(alphas[i - 1] * 16777216.0 + 0.5) : kNoCoin;
  return HSD_OK;
}

int hsd_set_trace(hsd_ctx *c, const char *path, int logit_calls) {
  if (!c) return HSD_E_INVALID_ARG;
  if (c->trace) { fclose(c->trace); c->trace = nullptr; }
  if (!path) return HSD_OK;
  c->trace = fopen(path, "wb");
  if (!c->trace) return HSD_E_IO;
  c->trace_logit_calls = logit_calls < 0 ? 0 : logit_calls;
  c->trace_records = 0;
  return HSD_OK;
}

size_t hsd_gemm_workspace_bytes(int R, int N, int K) {
  if (R < 1 || R > 256 || N < 1 || K < kTcBlockK || K % kTcBlockK) return 0;
  int seg[3] = {N, 0, 0};
  return kTcCtrlBytes + tc_plan(seg, 1, GEMM_STORE_F32, K, tc_npad(R), device_sm_count()).scratch_bytes;
}

int hsd_gemm_bf16(const void *A, int R, int K, const void *W, int N, float *out, void *workspace, size_t workspace_bytes,
                  void *stream) {
  if (!A || !W || !out || !workspace || ((uintptr_t)workspace & 255)) return HSD_E_INVALID_ARG;
  size_t need = hsd_gemm_workspace_bytes(R, N, K);
  if (need == 0) return HSD_E_INVALID_ARG;
  if (workspace_bytes < need) return HSD_E_WORKSPACE_TOO_SMALL;
  int st = tc_init();
  if (st) return st;
  TcGemmArgs a;
  st = tc_make_map(&a.w[0], W, N, K, kTcBoxRows);
  if (!st) st = tc_make_map(&a.a, A, R, K, tc_npad(R));
  if (st) return st;
  a.seg_n[0] = N; a.seg_n[1] = a.seg_n[2] = 0; a.n_segs = 1;
  a.K = K; a.R = R; a.row0 = 0; a.mode = GEMM_STORE_F32;
  a.out_f32 = out; a.out_bf16 = nullptr; a.dst = nullptr; a.ldo = N;
  a.status = (int *)workspace;
  a.counters = (int *)((char *)workspace + 256);
  a.pieces = (float *)((char *)workspace + kTcCtrlBytes);
  HSD_CUDA_OK(cudaMemsetAsync(workspace, 0, kTcCtrlBytes, (cudaStream_t)stream));
  return launch_gemm_tc(a, device_sm_count(), (cudaStream_t)stream);
}

int hsd_gemm_status(void *workspace, void *stream) {
  if (!workspace) return HSD_E_INVALID_ARG;
  int flag = 0;
  if (cudaMemcpyAsync(&flag, workspace, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess) return HSD_E_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return HSD_E_CUDA;
  return flag ? HSD_E_DEVICE_TIMEOUT : HSD_OK;
}

void hsd_destroy(hsd_ctx *c) {
  if (!c) return;
  if (c->trace) fclose(c->trace);
  if (c->ring_host) cudaFreeHost(c->ring_host);
  if (c->n_acc_host) cudaFreeHost(c->n_acc_host);
  if (c->page_table_host) cudaFreeHost(c->page_table_host);
  if (c->status_host) cudaFreeHost(c->status_host);
  for (int i = 0; i < kTimerPairs; ++i) {
    if (c->timers[i].a) cudaEventDestroy(c->timers[i].a);
    if (c->timers[i].b) cudaEventDestroy(c->timers[i].b);
  }
  delete c;
}

}  // extern "C"
