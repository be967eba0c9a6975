// Persistent verifier forward (see fwd_persist.cuh).
//
// Warp roles (12 warps): 0 = weight-tile TMA producer, 1 = activation-tile TMA producer, 2 = TMEM
// owner + MMA issuer, 3 = spare, 4..7 = GEMM epilogue (each reads its own TMEM lane quarter) and
// phase workers, 8..11 = phase workers only.  The 256 worker threads walk the phase program
//   embed+norm | QKV(+rope, KV append) | attention | O(+residual) | norm | gate/up(+SwiGLU) |
//   down(+residual) | norm | ... | final norm | output head
// with a grid barrier between phases.  The weight producer is not tied to the barriers: weights are
// read-only, so it runs ahead into the next GEMM as far as the ring allows; the activation producer
// waits for the barrier that completes its operand.  GEMM work is split evenly over the CTAs in
// (tile, k-block) units; each segment's partial sums go to a piece buffer and the following phase
// (the next RMSNorm for the residual projections, a short finish phase otherwise) adds them up.
// In decode passes two finish phases fold into their consumer: the attention phase finishes the
// q / k / v of its own rows, and with at most four rows the down projection's CTAs build their
// activation tiles from the gate / up pieces in shared memory (warps 5, 7, 9, 11).
// Every wait (mbarrier, grid barrier) is bounded by wall time and raises a status word.
#include "fwd_persist.cuh"
#include "forward.cuh"
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace hsd {
namespace {

using namespace ptx;

constexpr int kWBytes = kTcBlockM * kTcBlockK * 2;     // 16 KiB weight tile
constexpr int kBoxBytes = kTcBoxRows * kTcBlockK * 2;  // 8 KiB TMA box
constexpr int kScratchBytes = 78 * 1024;               // union: epilogue staging / attention buffers, + rope cache
constexpr int kCtrlBytes = 4096;                       // barriers, flags, page-id cache, per-row info
constexpr int kSmemTotal = 232448;
constexpr int kMaxLayersSh = 64;                       // layers whose pointer table fits the control area

enum { MODE_QKV = 0, MODE_ADD = 1, MODE_SWIGLU = 2, MODE_LOGITS = 3 };

// Barrier-timeline stamps and cycle laps exist only in a profiling build (-DHSD_PROFILE).
#ifdef HSD_PROFILE
#define HSD_PROF(a) ((a).prof != nullptr)
#else
#define HSD_PROF(a) false
#endif

template <int NPAD> struct PCfg {
  static constexpr int kStageBytes = kWBytes + NPAD * kTcBlockK * 2;
  static constexpr int kStages = (kSmemTotal - 1024 - kCtrlBytes - kScratchBytes) / kStageBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + kScratchBytes + kCtrlBytes + 1024;
  static constexpr int kTmemCols = (2 * NPAD < 32) ? 32 : 2 * NPAD;
  static constexpr int kChunk = NPAD < 32 ? NPAD : 32;      // accumulator columns handled at a time
};

struct Gemm {
  const CUtensorMap *w[3];
  const CUtensorMap *amap;
  int seg_n[3];
  int n_segs, K, KB, n_tiles, mode, rows;
};

__device__ __forceinline__ Gemm make_gemm(const FwdArgs &a, int p) {
  Gemm g;
  const int l = p >> 2, j = p & 3;
  g.w[1] = g.w[2] = nullptr;
  g.seg_n[1] = g.seg_n[2] = 0;
  g.n_segs = 1;
  g.rows = a.R;
  if (l >= a.n_run) {                       // output head
    g.w[0] = a.wmaps + a.lm_map; g.seg_n[0] = a.V; g.amap = &a.amap[3]; g.K = a.d; g.mode = MODE_LOGITS; g.rows = a.L;
  } else if (j == 0) {
    const CUtensorMap *m = a.wmaps + l * 7;
    g.w[0] = m; g.w[1] = m + 1; g.w[2] = m + 2;
    g.seg_n[0] = a.nq * a.hd; g.seg_n[1] = g.seg_n[2] = a.nkv * a.hd;
    g.n_segs = 3; g.amap = &a.amap[0]; g.K = a.d; g.mode = MODE_QKV;
  } else if (j == 1) {
    g.w[0] = a.wmaps + l * 7 + 3; g.seg_n[0] = a.d; g.amap = &a.amap[1]; g.K = a.nq * a.hd; g.mode = MODE_ADD;
  } else if (j == 2) {
    g.w[0] = a.wmaps + l * 7 + 4; g.w[1] = a.wmaps + l * 7 + 5; g.seg_n[0] = g.seg_n[1] = a.ff;
    g.n_segs = 2; g.amap = &a.amap[0]; g.K = a.d; g.mode = MODE_SWIGLU;
  } else {
    g.w[0] = a.wmaps + l * 7 + 6; g.seg_n[0] = a.d; g.amap = &a.amap[2]; g.K = a.ff; g.mode = MODE_ADD;
  }
  g.KB = g.K / kTcBlockK;
  if (g.mode == MODE_SWIGLU) g.n_tiles = (g.seg_n[0] + kTcBoxRows - 1) / kTcBoxRows;
  else {
    g.n_tiles = 0;
    for (int s = 0; s < g.n_segs; ++s) g.n_tiles += (g.seg_n[s] + kTcBlockM - 1) / kTcBlockM;
  }
  return g;
}

struct Tile { int seg, row0, col0; };
__device__ __forceinline__ Tile tile_of(const Gemm &g, int tile) {
  Tile t;
  if (g.mode == MODE_SWIGLU) { t.seg = 0; t.row0 = tile * kTcBoxRows; t.col0 = 0; return t; }
  int tt = tile, col0 = 0;
  for (int s = 0; s < g.n_segs; ++s) {
    int nt = (g.seg_n[s] + kTcBlockM - 1) / kTcBlockM;
    if (tt < nt || s == g.n_segs - 1) { t.seg = s; t.row0 = tt * kTcBlockM; t.col0 = col0; return t; }
    tt -= nt;
    col0 += g.seg_n[s];
  }
  t.seg = 0; t.row0 = 0; t.col0 = 0;
  return t;
}
// Unit arithmetic in 32 bits (the launcher checks n_tiles * KB * grid < 2^31).
__device__ __forceinline__ int cta_begin(int U, int G, int c) { return (int)(((unsigned)U * (unsigned)c) / (unsigned)G); }
// CTA c owns units [floor(U c / G), floor(U (c + 1) / G)): the owner of unit u is the largest c with
// floor(U c / G) <= u, i.e. c < (u + 1) G / U, i.e. c = floor(((u + 1) G - 1) / U).
__device__ __forceinline__ int unit_owner(int U, int G, int u) {
  return (int)((((unsigned)u + 1u) * (unsigned)G - 1u) / (unsigned)U);
}
// Work of one CTA in one GEMM, a segment (tile, k-block range) at a time.  One SM can pull only its
// share of HBM bandwidth, so every GEMM is split evenly over all CTAs in (tile, k-block) units;
// each segment's partial sums go to a piece buffer and the next phase adds the pieces of a tile in
// fixed piece order (bit-reproducible; no CTA waits for another inside a GEMM).
struct Seg { int tile, kb0, kb1; };
struct SegIter { int tile, kb, left; };        // next k-block (tile, kb) and the k-blocks still to hand out
// regular: every tile is cut into `parts` equal k-ranges (GEMMs with few tiles: at most 4 pieces per
// tile, so the consumer can fetch all of them in one batch); otherwise the (tile, k-block) units are
// dealt out evenly (tiles >= CTAs / 2: a tile then spans at most 3 CTAs).
struct SplitGeom { int U, Gp, pieces_max, parts; };
__device__ __forceinline__ SplitGeom split_geom(const Gemm &g, int G) {
  SplitGeom sg;
  sg.U = g.n_tiles * g.KB;
  if (g.n_tiles * 2 <= G) {
    sg.parts = min(min(4, G / g.n_tiles), g.KB);
    sg.Gp = g.n_tiles * sg.parts;
    sg.pieces_max = sg.parts;
  } else {
    sg.parts = 0;
    sg.Gp = min(G, sg.U);
    const int per = sg.U / sg.Gp;
    sg.pieces_max = (g.KB + per - 1) / per + 1;
  }
  return sg;
}
// The divisions happen once, here; seg_next only counts (the pipeline roles call it on their critical path).
__device__ __forceinline__ SegIter seg_begin(const Gemm &g, int G, int c) {
  SegIter it;
  const SplitGeom sg = split_geom(g, G);
  it.tile = 0; it.kb = 0; it.left = 0;
  if (c < sg.Gp) {
    if (sg.parts) {
      const int tile = c / sg.parts, part = c - tile * sg.parts;
      it.tile = tile;
      it.kb = cta_begin(g.KB, sg.parts, part);
      it.left = cta_begin(g.KB, sg.parts, part + 1) - it.kb;
    } else {
      const int cur = cta_begin(sg.U, sg.Gp, c);
      it.left = cta_begin(sg.U, sg.Gp, c + 1) - cur;
      it.tile = cur / g.KB;
      it.kb = cur - it.tile * g.KB;
    }
  }
  return it;
}
__device__ __forceinline__ bool seg_next(const Gemm &g, SegIter &it, Seg &s) {
  if (it.left <= 0) return false;
  const int n = min(g.KB - it.kb, it.left);
  s.tile = it.tile; s.kb0 = it.kb; s.kb1 = it.kb + n;
  it.left -= n; it.kb = 0; ++it.tile;
  return true;
}
// Pieces of a tile: they belong to consecutive CTAs first_owner .. first_owner + n - 1.
__device__ __forceinline__ void tile_pieces(const Gemm &g, const SplitGeom &geo, int tile, int &first_owner, int &n) {
  if (geo.parts) { first_owner = tile * geo.parts; n = geo.parts; return; }
  first_owner = unit_owner(geo.U, geo.Gp, tile * g.KB);
  n = unit_owner(geo.U, geo.Gp, tile * g.KB + g.KB - 1) - first_owner + 1;
}
// Phase p is a down projection whose activation tiles are built in place from the gate / up pieces: its own
// pieces then go to the second buffer (the first is still being read by slower CTAs).
__device__ __forceinline__ bool built_down(const FwdArgs &a, int p) { return a.fuse_gu && (p & 3) == 3 && p < 4 * a.n_run; }
__device__ __forceinline__ float *pieces_of(const FwdArgs &a, int p) { return built_down(a, p) ? a.pieces2 : a.pieces; }
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 2, 256;" ::: "memory"); }
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// barrier of one 128-thread worker group (id 1 = warps 4..7, the epilogue group; id 3 = warps 8..11)
__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Grid-wide barrier of the worker threads.  `epoch` counts barriers; the counter only grows.
// If ready_bar != 0 the spinning thread then releases the activation producer for the next GEMM.
__device__ __forceinline__ bool grid_barrier(const FwdArgs &a, unsigned &epoch, volatile int *abort_flag, int wt,
                                             uint32_t ready_bar) {
  // The CTA's writes of this phase are ordered before the arrival by the CTA barrier plus ONE release at gpu
  // scope by the arriving thread (cumulative over what it has observed through the barrier), instead of a
  // fence in every thread.
  // The activations this phase wrote with plain stores are read by the next GEMM's TMA loads (async proxy):
  // every writer orders its generic-proxy writes before async-proxy accesses here, ahead of the release.
  if (ready_bar) asm volatile("fence.proxy.async.global;" ::: "memory");
  worker_sync();
  ++epoch;
  if (*abort_flag) return false;
  if (wt == 0) {
    const unsigned target = epoch * gridDim.x;
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.grid_counter) : "memory");
    if (HSD_PROF(a) && 2 * epoch + 1 < (unsigned)kFwdProfEvents) a.prof[(size_t)blockIdx.x * kFwdProfEvents + 2 * epoch] = globaltimer_ns();
    bool ok = true;
    unsigned long long t0 = 0;                       // the clock is read only once the wait has lasted a while
    for (uint32_t it = 0; (int)(ld_acquire_u32(a.grid_counter) - target) < 0; ++it) {
      if ((it & 31u) == 31u) {
        const unsigned long long now = globaltimer_ns();
        if (t0 == 0) t0 = now;
        if (*abort_flag || *reinterpret_cast<volatile int *>(a.status) != 0 || now - t0 > kWaitLimitNs) {
          ok = false;
          break;
        }
      }
    }
    if (!ok) {
      *abort_flag = 1;
      atomicExch(a.status, 1);
    } else {
      if (HSD_PROF(a) && 2 * epoch + 1 < (unsigned)kFwdProfEvents)
        a.prof[(size_t)blockIdx.x * kFwdProfEvents + 2 * epoch + 1] = globaltimer_ns();
      // the acquire load that left the spin orders everything after it; the CTA barrier below hands that on
      if (ready_bar) {
        mbar_arrive(ready_bar);
      }
    }
  }
  worker_sync();
  return *abort_flag == 0;
}

// ------------------------------------------------------------------------------ RMSNorm phase
// One row per CTA turn, held in registers (all loads issued before their first use).
//   src_embed: the row comes from the embedding table (and is copied to x).
//   pend:      the residual-add projection that ran just before; its split pieces are added to the
//              row in fixed piece order (x <- x + p_0 + p_1 + ...) and x is written back.
// Requires d % 4 == 0 and d <= 4096.
//   pieces_target != 0: the CTA was idle in that projection and has passed no grid barrier since; it waits until
//              the counter of CTAs that have stored their pieces reaches pieces_target.
template <int NPAD>
__device__ __forceinline__ bool norm_phase(const FwdArgs &a, int n_rows, const int *row_list, bool src_embed,
                                           const Gemm *pend, const float *pend_pieces, const __nv_bfloat16 *gain, __nv_bfloat16 *dst,
                                           float *red, int wt, unsigned pieces_target, volatile int *abort_flag) {
  constexpr int MAXV = 4;                                  // float4 slots per thread
  constexpr int PB = 4;                                    // pieces loaded at a time per slot
  const int d = a.d, nvec = d >> 2;
  SplitGeom geo;
  geo.U = 1; geo.Gp = 1; geo.pieces_max = 1;
  if (pend) geo = split_geom(*pend, gridDim.x);
  // rows go to the LAST CTAs of the grid when the norm may start early: those have no tile of the projection
  const int first = a.early_norm ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x;
  if (pieces_target != 0u && first < n_rows) {
    if (wt == 0) {
      const unsigned *cnt = a.grid_counter + 16;
      unsigned long long t0 = 0;
      for (uint32_t it = 0; (int)(ld_acquire_u32(cnt) - pieces_target) < 0; ++it) {
        if ((it & 31u) == 31u) {
          const unsigned long long now = globaltimer_ns();
          if (t0 == 0) t0 = now;
          if (*abort_flag || now - t0 > kWaitLimitNs) { *abort_flag = 1; break; }
        }
      }
    }
    worker_sync();
    if (*abort_flag) return false;
  }
  for (int i = first; i < n_rows; i += gridDim.x) {
    const int row = row_list ? row_list[i] : i;
    float *xrow = a.x + (size_t)row * d;
    float4 v[MAXV];
    if (src_embed) {
      // an id outside the vocabulary (only possible after non-finite logits) must not become an address
      const int tok = min(max(a.tokens[(size_t)a.row_seq[row] * a.max_seq + a.row_pos[row]], 0), a.V - 1);
      const __nv_bfloat16 *erow = a.embed + (size_t)tok * d;
      uint2 raw[MAXV];
#pragma unroll
      for (int j = 0; j < MAXV; ++j) {
        const int iv = wt + 256 * j;
        raw[j] = iv < nvec ? __ldg(reinterpret_cast<const uint2 *>(erow) + iv) : make_uint2(0u, 0u);
      }
#pragma unroll
      for (int j = 0; j < MAXV; ++j)
        v[j] = make_float4(__uint_as_float(raw[j].x << 16), __uint_as_float(raw[j].x & 0xFFFF0000u),
                           __uint_as_float(raw[j].y << 16), __uint_as_float(raw[j].y & 0xFFFF0000u));
    } else {
#pragma unroll
      for (int j = 0; j < MAXV; ++j) {
        const int iv = wt + 256 * j;
        v[j] = iv < nvec ? __ldcg(reinterpret_cast<const float4 *>(xrow) + iv) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    uint2 graw[MAXV];
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
      const int iv = wt + 256 * j;
      graw[j] = iv < nvec ? __ldg(reinterpret_cast<const uint2 *>(gain) + iv) : make_uint2(0u, 0u);
    }
    if (pend) {
      // every piece of every slot in one batch of loads: the residual projections have at most d / 128
      // = 32 tiles, so they are always cut the regular way (the launcher checks it), `parts` <= 4
      // pieces per tile at a fixed stride
      const int np = geo.parts;
      float4 t[MAXV][PB];
#pragma unroll
      for (int j = 0; j < MAXV; ++j) {
        const int iv = wt + 256 * j, k = iv << 2, tile = k >> 7, mm = k & 127;
        const float *base = pend_pieces + ((size_t)tile * np * NPAD + row) * kTcBlockM + mm;
#pragma unroll
        for (int pp = 0; pp < PB; ++pp)
          t[j][pp] = (iv < nvec && pp < np) ? __ldcg(reinterpret_cast<const float4 *>(base + (size_t)pp * NPAD * kTcBlockM))
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int j = 0; j < MAXV; ++j)
#pragma unroll
        for (int pp = 0; pp < PB; ++pp) {
          v[j].x += t[j][pp].x; v[j].y += t[j][pp].y; v[j].z += t[j][pp].z; v[j].w += t[j][pp].w;
        }
    }
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < MAXV; ++j) ss += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    worker_sync();
    if ((wt & 31) == 0) red[wt >> 5] = ss;
    worker_sync();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)d + a.eps);
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
      const int iv = wt + 256 * j;
      if (iv < nvec) {
        if (src_embed || pend) reinterpret_cast<float4 *>(xrow)[iv] = v[j];
        const float g0 = __uint_as_float(graw[j].x << 16), g1 = __uint_as_float(graw[j].x & 0xFFFF0000u);
        const float g2 = __uint_as_float(graw[j].y << 16), g3 = __uint_as_float(graw[j].y & 0xFFFF0000u);
        __nv_bfloat162 lo = __floats2bfloat162_rn(v[j].x * inv * g0, v[j].y * inv * g1);
        __nv_bfloat162 hi = __floats2bfloat162_rn(v[j].z * inv * g2, v[j].w * inv * g3);
        uint2 out;
        out.x = *reinterpret_cast<unsigned *>(&lo);
        out.y = *reinterpret_cast<unsigned *>(&hi);
        reinterpret_cast<uint2 *>(dst + (size_t)i * d)[iv] = out;
      }
    }
  }
  return true;
}

// ------------------------------------------------------------------------------ attention phases
// Under the weight stream every dependent global round trip costs microseconds, so the attention is
// two phases.  Phase A: work item = (attention item, KV head, key split), partial (o, m, l) to global
// memory.  Phase B (after a grid barrier): one (row, head) per 128 threads merges the partials of its
// splits.
constexpr int kRopeCacheRows = 12;                     // rows whose cos / sin values are kept in shared memory
constexpr int kAttnMaxSplits = 20;

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}

struct PageCache { int tag_item, tag_tile; int pg[128]; };   // pg[warp * 16 + j]: page of the warp's j-th sub-tile

__device__ __forceinline__ void mma_bf16_16x8x16(float *c, const unsigned *a, unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Four 8x8 b16 matrices; lane l gives the address of row l % 8 of matrix l / 8; register i of lane (g, t) holds
// matrix i's elements [g][2t .. 2t + 1] (.trans: [2t .. 2t + 1][g]).
__device__ __forceinline__ void ldmatrix_x4(unsigned *r, const void *row_ptr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row_ptr)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned *r, const void *row_ptr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row_ptr)));
}

// ------------------------------------------------------------------------------ long key ranges on tcgen05
// One work item (attention item, KV head, key split) with a long key range, head size 128, at most 32 query
// vectors.  Keys go through in tiles of 64, dealt to two independent streams (tile j to stream j & 1), each with
// its own running reference maximum, row sums and output accumulator; per tile
//   S[128 x 64]   = Q[128 (<= 32 real rows) x 128] K_tile[64 x 128]^T       tcgen05.mma, both operands K-major
//   P             = exp2((S - m_ref) scale log2 e)  as bf16, row per thread  (m_ref moves only when a row maximum
//                                                                             passes it by a factor 256: then O is rescaled)
//   O[128 x 128] += P[128 x 64] V_tile[64 keys x 128]                        V as the MN-major B operand, as it lies in the cache
// S and O live in tensor memory (S double-buffered per stream: 2 x 2 x 64 columns, O 2 x 128: all 512 columns,
// the GEMM accumulators are idle during this phase).  Rows 32..127 of the A operands are whatever shared memory
// follows the real rows: their results are never read.  The eight worker warps: per stream (warps 0-3 / 4-7) warp
// 0 = softmax (the only one whose TMEM lane quarter holds real rows), warp 1 = K tiles (three buffers: a K buffer
// is free as soon as S is complete), warp 2 = V tiles (two buffers), warp 3 = MMA issue (one lane).  Shared memory:
// the weight ring and the attention scratch together (the weight producer does not run ahead over this phase).
constexpr int kTcaTile = 64, kTcaKBufs = 3, kTcaVBufs = 2;
constexpr int kTcaTileBytes = 2 * kTcaTile * 128;                 // two 64-column blocks of [64 keys][128 B]
constexpr int kTcaOffK = 8192, kTcaOffV = kTcaOffK + 2 * kTcaKBufs * kTcaTileBytes, kTcaOffP = kTcaOffV + 2 * kTcaVBufs * kTcaTileBytes;
constexpr int kTcaOffBar = kTcaOffP + 4 * 4096 + 12288, kTcaBytes = kTcaOffBar + 256;
constexpr int kTcaMinKeys = 1920;                                 // shorter key ranges stay on the mma.sync path (the host plans splits of
                                                                  // 2048 keys and more; the last split of a range may fall a little short)
static_assert(kTcaBytes <= 4 * (kWBytes + 128 * kTcBlockK * 2) + kScratchBytes - 2 * 12 * 64 * 4, "tcgen05 attention buffers exceed the ring + scratch");

__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr, uint32_t lbo_bytes) {   // MN-major, 128-byte swizzle
  uint64_t d = (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(lbo_bytes >> 4) << 16;                          // between the 64-element blocks along N
  d |= (uint64_t)(1024 >> 4) << 32;                               // between the 8-row groups along K
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float *o) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
               ::"r"(taddr), "r"(__float_as_uint(o[0])), "r"(__float_as_uint(o[1])), "r"(__float_as_uint(o[2])),
               "r"(__float_as_uint(o[3])), "r"(__float_as_uint(o[4])), "r"(__float_as_uint(o[5])), "r"(__float_as_uint(o[6])),
               "r"(__float_as_uint(o[7])), "r"(__float_as_uint(o[8])), "r"(__float_as_uint(o[9])), "r"(__float_as_uint(o[10])),
               "r"(__float_as_uint(o[11])), "r"(__float_as_uint(o[12])), "r"(__float_as_uint(o[13])), "r"(__float_as_uint(o[14])),
               "r"(__float_as_uint(o[15])) : "memory");
}

struct TcaItem { int row0, nrows, seq, pos0, kvh, split, key_lo, key_hi, nqv, group; };

__device__ __noinline__ void attn_item_tc(const FwdArgs &a, const __nv_bfloat16 *kpool, const __nv_bfloat16 *vpool, uint8_t *smem,
                                          uint32_t tmem, const TcaItem it, int wt, volatile int *abort_flag, long long *dbg) {
  constexpr int HD = 128, TK = kTcaTile, NKB = kTcaKBufs, NVB = kTcaVBufs;
  const uint32_t s0 = smem_u32(smem), b0 = s0 + kTcaOffBar;
  // per stream s: k_free[3] (= S complete) k_full[3] v_full[2] v_free[2] p_ready[2]
  auto k_full = [&](int s, int b) { return b0 + 8u * (s * 12 + b); };
  auto k_free = [&](int s, int b) { return b0 + 8u * (s * 12 + 3 + b); };
  auto v_full = [&](int s, int b) { return b0 + 8u * (s * 12 + 6 + b); };
  auto v_free = [&](int s, int b) { return b0 + 8u * (s * 12 + 8 + b); };
  auto p_ready = [&](int s, int b) { return b0 + 8u * (s * 12 + 10 + b); };
  const int warp = wt >> 5, lane = wt & 31, s = warp >> 2, role = warp & 3;
#ifdef HSD_PROFILE
  // profiling build: CTA 0's first softmax warp laps its set-up [5], waits for S [6], softmax up to P ready [7] and the
  // item's end [8]; [9] counts the items
  long long cyc = clock64();
  auto lap = [&](int k) { if (a.prof && wt == 0 && blockIdx.x == 0) { const long long n_ = clock64(); dbg[k] += n_ - cyc; cyc = n_; } };
  if (a.prof && wt == 0 && blockIdx.x == 0) dbg[9] += 1;
#else
  auto lap = [](int) {};
#endif
  if (wt == 0) {
    for (int ss = 0; ss < 2; ++ss) {
      for (int b = 0; b < NKB; ++b) { mbar_init(k_full(ss, b), 32); mbar_init(k_free(ss, b), 1); }
      for (int b = 0; b < NVB; ++b) { mbar_init(v_full(ss, b), 32); mbar_init(v_free(ss, b), 1); mbar_init(p_ready(ss, b), 1); }
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Q: K-major, 128-byte swizzle, k-block kb (64 columns) at kb * 4096, rows 0..31 (rows past the item's vectors zero)
  for (int i = wt; i < 32 * 16; i += 256) {
    const int qi = i >> 4, c = i & 15, kb = c >> 3, cc = c & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (qi < it.nqv) {
      const int r = qi / it.group, gq = qi - r * it.group;
      v = __ldcg(reinterpret_cast<const uint4 *>(a.q + ((size_t)(it.row0 + r) * a.nq + it.kvh * it.group + gq) * HD + c * 8));
    }
    *reinterpret_cast<uint4 *>(smem + kb * 4096 + (qi >> 3) * 1024 + (qi & 7) * 128 + ((cc ^ (qi & 7)) << 4)) = v;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  worker_sync();
  tc_fence_after();
  lap(5);
  const int n_tiles = (it.key_hi - it.key_lo + TK - 1) / TK;
  const int n_mine = (n_tiles - s + 1) / 2;                      // tiles s, s + 2, ...
  const float sc = rsqrtf((float)HD) * 1.4426950408889634f;      // raw scores -> log2 units
  float m_ref = -INFINITY, l = 0.f;                              // the softmax warps' state (raw score units)
  bool ok = true;
  const uint32_t tS = tmem + (uint32_t)(s * 128), tO = tmem + 256u + (uint32_t)(s * 128);
  if (role == 1 || role == 2) {
    // ---------------- loader warp of one operand: LAG tiles in flight behind the one being issued
    const bool isk = role == 1;
    const int NB = isk ? NKB : NVB, LAG = isk ? 2 : 1;
    const __nv_bfloat16 *pool = isk ? kpool : vpool;
    const uint32_t base = isk ? kTcaOffK + s * NKB * kTcaTileBytes : kTcaOffV + s * NVB * kTcaTileBytes;
    const int *pt = a.page_table + (size_t)it.seq * a.pages_per_seq;
    for (int t = 0; t < n_mine + LAG; ++t) {
      if (t >= LAG) {                                            // tile t - LAG has landed: hand it over before anything can block
        if (isk) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const int tt = t - LAG;
        mbar_arrive(isk ? k_full(s, tt % NKB) : v_full(s, tt % NVB));
      }
      if (t < n_mine) {
        const int b = t % NB;
        if (t >= NB) {
          const int use = t / NB - 1;                            // completion number of the buffer's previous use
          if (lane == 0) mbar_wait(isk ? k_free(s, b) : v_free(s, b), (uint32_t)(use & 1), abort_flag);
          __syncwarp();
        }
        if (*abort_flag) break;
        const int key0 = it.key_lo + (2 * t + s) * TK;
        // the tile's four 16-key groups lie in one page each (pages hold >= 16 tokens, key ranges start on multiples of 16)
        int pg = 0;
        if (lane < 4 && key0 + lane * 16 < it.key_hi) pg = pt[(key0 + lane * 16) >> a.page_shift];
        const uint32_t tb = base + b * kTcaTileBytes;
        const int c = lane & 15, blk = c >> 3, cc = c & 7, h = lane >> 4;
        if (key0 + TK <= it.key_hi) {
          // a whole tile: per 16-key group one source base (its page) and eight copies per lane, rows 2 i + h; the
          // swizzled destination differs from row to row by compile-time constants only
          const uint32_t dst0 = s0 + tb + blk * (TK * 128) + h * 128;
          const int cch = cc ^ h;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int pgr = __shfl_sync(0xFFFFFFFFu, pg, g);
            const __nv_bfloat16 *src = pool + ((((size_t)it.kvh * a.n_pages + pgr) << a.page_shift) + ((key0 + 16 * g) & (a.page - 1)) + h) * HD + c * 8;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r7 = (2 * i) & 7;                         // (row & 7) without h; row = 16 g + 2 i + h
              const uint32_t dst = dst0 + (uint32_t)((2 * g + (i >> 2)) * 1024 + r7 * 128) + (uint32_t)((cch ^ r7) << 4);
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src + (size_t)(2 * i) * HD) : "memory");
            }
          }
        } else {
#pragma unroll 4
          for (int i = 0; i < TK / 2; ++i) {
            const int r = 2 * i + h, key = key0 + r;
            const int pgr = __shfl_sync(0xFFFFFFFFu, pg, r >> 4);
            const uint32_t off = tb + blk * (TK * 128) + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
            if (key < it.key_hi)
              cp_async16(smem + off, pool + ((((size_t)it.kvh * a.n_pages + pgr) << a.page_shift) + (key & (a.page - 1))) * HD + c * 8);
            else
              *reinterpret_cast<uint4 *>(smem + off) = make_uint4(0u, 0u, 0u, 0u);    // P is 0 there, V must be finite
          }
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else if (role == 3) {
    // ---------------- MMA issue for stream s (one lane)
    if (lane == 0) {
      const uint32_t id1 = umma_idesc_bf16(TK), id2 = umma_idesc_bf16(HD) | (1u << 16);     // bit 16: B is MN-major
      auto issue_s = [&](int t) {                                 // S[t & 1] = Q K_t^T
        const int b = t % NKB;
        ok = mbar_wait(k_full(s, b), (uint32_t)((t / NKB) & 1), abort_flag);
        if (!ok) return;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const uint64_t da = umma_desc(s0 + (ks >> 2) * 4096 + (ks & 3) * 32);
          const uint64_t db = umma_desc(s0 + kTcaOffK + (s * NKB + b) * kTcaTileBytes + (ks >> 2) * (TK * 128) + (ks & 3) * 32);
          umma_bf16(tS + (uint32_t)((t & 1) * 64), da, db, id1, ks > 0 ? 1u : 0u);
        }
        umma_commit(k_free(s, b));                                // S(t) complete = the K buffer is free
      };
      if (n_mine > 0) issue_s(0);
      if (n_mine > 1 && ok) issue_s(1);
      for (int t = 0; t < n_mine && ok; ++t) {
        // P(t) is written (so S(t) has been read as well) and V(t) has landed
        ok = mbar_wait(p_ready(s, t & 1), (uint32_t)((t >> 1) & 1), abort_flag);
        if (!ok) break;
        const int vb = t % NVB;
        ok = mbar_wait(v_full(s, vb), (uint32_t)((t / NVB) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t p_off = kTcaOffP + (s * 2 + (t & 1)) * 4096;
#pragma unroll
        for (int ks = 0; ks < TK / 16; ++ks) {
          const uint64_t da = umma_desc(s0 + p_off + ks * 32);
          const uint64_t db = umma_desc_mn(s0 + kTcaOffV + (s * NVB + vb) * kTcaTileBytes + ks * 2048, TK * 128);
          umma_bf16(tO, da, db, id2, (t > 0 || ks > 0) ? 1u : 0u);
        }
        umma_commit(v_free(s, vb));
        if (t + 2 < n_mine) issue_s(t + 2);                       // its S buffer (t & 1) was read before P(t) was written
      }
    }
  } else {
    // ---------------- stream s: softmax (thread = query vector `lane`)
    auto sync_ok = [&]() { ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0; };
    const int qpos = it.pos0 + lane / it.group;                   // causal limit of this thread's query vector
    const bool real = lane < it.nqv;
    for (int t = 0; t < n_mine && ok; ++t) {
      if (lane == 0) ok = mbar_wait(k_free(s, t % NKB), (uint32_t)((t / NKB) & 1), abort_flag);
      sync_ok();
      if (!ok) break;
      lap(6);
      tc_fence_after();
      float sv[TK];
#pragma unroll
      for (int c = 0; c < TK; c += 16) tmem_ld16(tS + (uint32_t)((t & 1) * 64 + c), sv + c);
      tmem_ld_wait();
      const int key0 = it.key_lo + (2 * t + s) * TK;
      if (!real) {
#pragma unroll
        for (int c = 0; c < TK; ++c) sv[c] = 0.f;
      } else if (key0 + TK > it.key_hi || key0 + TK - 1 > qpos) {
#pragma unroll
        for (int c = 0; c < TK; ++c)
          if (key0 + c >= it.key_hi || key0 + c > qpos) sv[c] = -INFINITY;
      }
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < TK; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], sv[c]);
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      // the reference maximum moves only when a row's maximum has passed it by more than 8 in log2 units
      const bool grow = (mx - m_ref) * sc > 8.f;                  // false while both are -inf (no key of the row so far)
      if (t == 0) m_ref = mx;
      else if (__any_sync(0xFFFFFFFFu, grow)) {
        // O of this stream is rescaled: its previous P V must be complete
        if (lane == 0) ok = mbar_wait(v_free(s, (t - 1) % NVB), (uint32_t)(((t - 1) / NVB) & 1), abort_flag);
        sync_ok();
        if (!ok) break;
        tc_fence_after();
        const float m_new = grow ? mx : m_ref;
        const float f = (m_new > -INFINITY && m_ref > -INFINITY) ? ex2_approx((m_ref - m_new) * sc) : (m_new > -INFINITY ? 0.f : 1.f);
#pragma unroll 1
        for (int c = 0; c < HD; c += 16) {
          float o[16];
          tmem_ld16(tO + (uint32_t)c, o);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) o[e] *= f;
          tmem_st16(tO + (uint32_t)c, o);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        l *= f;
        m_ref = m_new;
      }
      // P buffer t & 1 was read by the P V of tile t - 2
      if (t >= 2) {
        if (lane == 0) ok = mbar_wait(v_free(s, (t - 2) % NVB), (uint32_t)(((t - 2) / NVB) & 1), abort_flag);
        sync_ok();
        if (!ok) break;
      }
      uint8_t *prow = smem + kTcaOffP + (s * 2 + (t & 1)) * 4096 + (lane >> 3) * 1024 + (lane & 7) * 128;
      const float mneg = m_ref > -INFINITY ? -m_ref * sc : 0.f;   // a row without keys so far: exp2(-inf) = 0 everywhere
      float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c8 = 0; c8 < TK / 8; ++c8) {
        unsigned w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p0 = ex2_approx(fmaf(sv[c8 * 8 + 2 * e], sc, mneg)), p1 = ex2_approx(fmaf(sv[c8 * 8 + 2 * e + 1], sc, mneg));
          l4[e] += p0 + p1;
          const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
          w[e] = *reinterpret_cast<const unsigned *>(&pb);
        }
        *reinterpret_cast<uint4 *>(prow + ((c8 ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      l += (l4[0] + l4[1]) + (l4[2] + l4[3]);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_ready(s, t & 1));
      lap(7);
    }
    if (ok && n_mine > 0) {                                       // the stream's last P V
      const int tl = n_mine - 1;
      if (lane == 0) ok = mbar_wait(v_free(s, tl % NVB), (uint32_t)((tl / NVB) & 1), abort_flag);
      sync_ok();
    }
    tc_fence_after();
  }
  // ---- all MMAs of the item are complete once both softmax warps are here; stream 1 hands (O, m, l) to stream 0
  //      through shared memory (over the K buffers), stream 0 writes the item's result
  tc_fence_before();
  worker_sync();
  tc_fence_after();
  if (*abort_flag) return;
  if (wt == 0)                                                    // nobody waits on the item's barriers any more: their memory
    for (int i = 0; i < 24; ++i)                                  // goes back to the weight ring / the next item
      asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(b0 + 8u * i) : "memory");
  float *xch = reinterpret_cast<float *>(smem + kTcaOffK);       // [32][HD + 2]
  if (role == 0 && s == 1) {
    if (n_mine > 0)
      for (int c = 0; c < HD; c += 16) {
        float o[16];
        tmem_ld16(tO + (uint32_t)c, o);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 16; ++e) xch[lane * (HD + 2) + c + e] = o[e];
      }
    xch[lane * (HD + 2) + HD] = n_mine > 0 ? m_ref : -INFINITY;
    xch[lane * (HD + 2) + HD + 1] = n_mine > 0 ? l : 0.f;
  }
  tc_fence_before();
  worker_sync();
  if (role == 0 && s == 0) {
    const float m1 = xch[lane * (HD + 2) + HD], l1 = xch[lane * (HD + 2) + HD + 1];
    const float mm = fmaxf(m_ref, m1);
    const float f0 = m_ref > -INFINITY ? ex2_approx((m_ref - mm) * sc) : 0.f, f1 = m1 > -INFINITY ? ex2_approx((m1 - mm) * sc) : 0.f;
    const float lt = l * f0 + l1 * f1;
    const bool real = lane < it.nqv;
    const int r = it.row0 + lane / it.group, hq = it.kvh * it.group + lane % it.group;
    float *dst = a.attn_partials + (((size_t)r * a.nq + hq) * a.n_splits + it.split) * (HD + 2);
    __nv_bfloat16 *adst = a.att + ((size_t)r * a.nq + hq) * HD;
    const float inv = lt > 0.f ? 1.f / lt : 0.f;
    for (int c = 0; c < HD; c += 16) {
      float o[16];
      tmem_ld16(tO + (uint32_t)c, o);
      tmem_ld_wait();
      if (real) {
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float o1 = m1 > -INFINITY ? xch[lane * (HD + 2) + c + e] : 0.f;
          o[e] = (f0 > 0.f ? o[e] * f0 : 0.f) + o1 * f1;
        }
        if (a.n_splits == 1) {
#pragma unroll
          for (int e = 0; e < 16; e += 2)
            *reinterpret_cast<__nv_bfloat162 *>(adst + c + e) = __floats2bfloat162_rn(o[e] * inv, o[e + 1] * inv);
        } else {
#pragma unroll
          for (int e = 0; e < 16; e += 2) *reinterpret_cast<float2 *>(dst + c + e) = make_float2(o[e], o[e + 1]);
        }
      }
    }
    if (real && a.n_splits > 1) { dst[HD] = mm * rsqrtf((float)HD); dst[HD + 1] = lt; }   // m in natural-log units, as the merge phase expects
    tc_fence_before();
  }
  lap(8);
}

// Phase A: warp-level online softmax.  A work item is (attention item, KV head, key split); its keys
// are cut into 16-key sub-tiles (one KV page or part of one: the launcher requires pages of >= 16
// tokens) that the warps take in turn, each warp with its own running (m, l, O) in registers and its
// own K and V sub-tile buffers, so nothing synchronises the CTA inside the key loop.  S = Q K^T and
// O += P V run on mma.sync m16n8k16 (the S accumulators are re-packed as the A operand of P V; P is
// split into bf16 hi + lo halves, so P V keeps ~16 bits of P); K of the warp's next sub-tile is fetched
// under the softmax and P V of this one, the next V under the next Q K^T.  With up to 16 query vectors
// (rows x group) every warp works on its own sub-tiles; with 17..32 the warps pair up on a sub-tile,
// one 16-row m-tile each.  At the end the warps' states are merged through shared memory and the
// split's partial (o, m, l) goes to global memory.
template <int NPAD, int HD, bool TC>
__device__ __forceinline__ void attn_tiles_phase(const FwdArgs &a, const FwdLayerDev &lay, uint8_t *scratch, PageCache *pc, int wt, long long *dbg,
                                                 const int *first_item, const int *qkv_geom, const int *row_pg_sh, const float *rope_cos_sh,
                                                 const float *rope_sin_sh, uint8_t *tc_smem, uint32_t tmem, volatile int *abort_flag) {
  constexpr int CPR = HD / 8;                      // 16-byte chunks per row
  // Rows of Q, K, V in shared memory: HD >= 64: unpadded, the 16-byte chunk index XORed with the row's low
  // three bits; HD = 32: padded by 16 bytes.  Either way the fragment loads (eight rows, same chunk) and
  // ldmatrix (eight rows of one 8x8 block) touch all banks once.
  constexpr bool SWZ = HD >= 64;
  constexpr int RS = SWZ ? HD : HD + 8;            // row stride (bf16 elements)
  auto swz = [](int row, int chunk) { return SWZ ? (chunk ^ (row & 7)) : chunk; };
  constexpr int KST = HD / 16;                     // k-steps of Q K^T
  constexpr int NT = HD / 8;                       // 8-wide output n-tiles
  constexpr int MS = HD + 8;                       // merge row: o[HD], m, l; stride = 8 mod 32 words: conflict-free float2 stores
  const int group = a.nq / a.nkv;
  const int warp = wt >> 5, lane = wt & 31, g = lane >> 2, t = lane & 3;
  __nv_bfloat16 *shQ = reinterpret_cast<__nv_bfloat16 *>(scratch);                              // [32][RS]
  __nv_bfloat16 *shK = shQ + 32 * RS + warp * (32 * RS);                                        // this warp's [16][RS]
  __nv_bfloat16 *shV = shK + 16 * RS;                                                           // this warp's [16][RS]
  float *shMerge = reinterpret_cast<float *>(scratch);                                          // [8 warps][16][MS], over Q and the K/V buffers
  static_assert(8 * 16 * MS * 4 <= 9 * 32 * RS * 2, "merge area must fit the Q and K/V buffers");
  static_assert(9 * 32 * RS * 2 <= kScratchBytes - 2 * kRopeCacheRows * (HD / 2) * 4, "attention buffers overlap the rope cache");
  const __nv_bfloat16 *kpool = lay.k_pool, *vpool = lay.v_pool;
  const float scale = rsqrtf((float)HD), inv_group = 1.f / (float)group;
  const int n_work = a.n_attn * a.nkv * a.n_splits;
#pragma unroll 1
  for (int wi = blockIdx.x; wi < n_work; wi += gridDim.x) {
#ifdef HSD_PROFILE
    long long cyc = clock64();
    auto lap = [&](int k) { if (a.prof && wt == 0 && blockIdx.x == 0) { const long long n_ = clock64(); dbg[k] += n_ - cyc; cyc = n_; } };
#else
    auto lap = [](int) {};
#endif
    const int split = wi % a.n_splits, kvh = (wi / a.n_splits) % a.nkv, ai = wi / (a.n_splits * a.nkv);
    const int4 it = wi == (int)blockIdx.x ? make_int4(first_item[0], first_item[1], first_item[2], first_item[3])
                                          : a.attn_items[ai];   // the CTA's first item was fetched at kernel start
    const int row0 = it.x, nrows = it.y, seq = it.z, pos0 = it.w;
    const int kv_len = pos0 + nrows;
    const int key_lo = split * a.keys_per_split, key_hi = min(kv_len, key_lo + a.keys_per_split);
    if (key_lo >= kv_len) continue;                              // uniform over the CTA
    const int nqv = nrows * group, n_mt = (nqv + 15) >> 4;
    if (TC && HD == 128 && key_hi - key_lo >= kTcaMinKeys) {     // tensor memory path (uniform over the CTA)
      worker_sync();                                             // the previous item is done with the shared memory
      if (wt == 0) pc->tag_item = -1;
      TcaItem ti;
      ti.row0 = row0; ti.nrows = nrows; ti.seq = seq; ti.pos0 = pos0; ti.kvh = kvh; ti.split = split;
      ti.key_lo = key_lo; ti.key_hi = key_hi; ti.nqv = nqv; ti.group = group;
      attn_item_tc(a, kpool, vpool, tc_smem, tmem, ti, wt, abort_flag, dbg);
      if (*abort_flag) return;
      continue;
    }
    const int n_sub = (key_hi - key_lo + 15) >> 4;
    const int first = n_mt == 2 ? (warp >> 1) : warp, step = n_mt == 2 ? 4 : 8, mt = n_mt == 2 ? (warp & 1) : 0;
    const int n_mine = first < n_sub ? (n_sub - first + step - 1) / step : 0;       // sub-tiles of this warp
    worker_sync();                                               // previous item's merge area fully read
    // ---- q rows of the item (whole CTA) and this warp's page ids: lane j holds the page of the warp's j-th
    //      sub-tile (re-read every 32 sub-tiles); kept in shared memory across layers when the CTA has one item
    if (!a.fuse_qkv) {
      for (int i = wt; i < nqv * CPR; i += 256) {
        const int qi = i / CPR, ch = i % CPR;
        const int r = qi / group, gq = qi % group;
        cp_async16(shQ + qi * RS + swz(qi, ch) * 8, a.q + ((size_t)(row0 + r) * a.nq + kvh * group + gq) * HD + ch * 8);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    const bool pages_cached = (pc->tag_item == wi) && n_mine <= 16;
    int pg_reg = 0, pg_base = 0;
    auto load_pages = [&](int j0) {                              // pages of sub-tiles j0 .. j0 + 31 of this warp
      pg_base = j0;
      const int j = j0 + lane;
      if (j < n_mine) {
        if (pages_cached) pg_reg = pc->pg[warp * 16 + j];
        else {
          const int key = key_lo + (first + j * step) * 16;
          pg_reg = a.page_table[(size_t)seq * a.pages_per_seq + (key >> a.page_shift)];
          if (n_mine <= 16) pc->pg[warp * 16 + j] = pg_reg;
        }
      }
    };
    load_pages(0);
    // `key_stop`: keys from there on are not fetched (fused QKV finish: the item's own new keys are written
    // straight into the buffers of a warp's first sub-tile by the threads that compute them)
    auto issue = [&](const __nv_bfloat16 *pool, __nv_bfloat16 *sh, int j, bool zero_pad, int key_stop) {    // one sub-tile, one operand
      const int kt = key_lo + (first + j * step) * 16, nk = min(16, key_hi - kt), nload = min(nk, key_stop - kt);
      const int pg = __shfl_sync(0xFFFFFFFFu, pg_reg, j - pg_base);
      const size_t base = ((((size_t)kvh * a.n_pages + pg) << a.page_shift) + (kt & (a.page - 1))) * HD;
#pragma unroll
      for (int i = 0; i < 16 * CPR / 32; ++i) {
        const int idx = i * 32 + lane, kk = idx / CPR, ch = idx % CPR;
        if (kk < nload) cp_async16(sh + kk * RS + swz(kk, ch) * 8, pool + base + (size_t)kk * HD + ch * 8);
        else if (zero_pad && kk >= nk) *reinterpret_cast<uint4 *>(sh + kk * RS + ch * 8) = make_uint4(0u, 0u, 0u, 0u);   // P is 0 there, V must be finite
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    constexpr int kAllKeys = 0x7FFFFFFF;
    const int first_stop = a.fuse_qkv ? pos0 : kAllKeys;
    if (n_mine > 0) { issue(kpool, shK, 0, false, first_stop); issue(vpool, shV, 0, true, first_stop); }
    else { asm volatile("cp.async.commit_group;\n\tcp.async.commit_group;" ::: "memory"); }
    if (a.fuse_qkv) {
      // ---- QKV finish of the item's own rows: pieces of the projection summed in piece order, rotary embedding,
      //      q -> the Q buffer, k / v of the rows whose position falls into this key split -> their cache page
      //      (and the first sub-tile's buffers, when that is where they belong).  A unit = 8 columns of one
      //      vector plus the 8 columns half a head further on (rotation partners): two 16-byte chunks.
      // geometry of the QKV projection's pieces (the same in every layer; worked out once at kernel start):
      // qg[0..6] = first tile of k, first tile of v, parts, pieces_max, U, Gp, KB
      constexpr int UPV = HD / 16, HALF = HD / 2;
      const int tile_k = qkv_geom[0], tile_v = qkv_geom[1], g_parts = qkv_geom[2], g_pmax = qkv_geom[3];
      const int nr_lo = max(0, key_lo - pos0), n_new = max(0, min(nrows, key_hi - pos0) - nr_lo);
      const int n_units = (nqv + 2 * n_new) * UPV;
      const bool rope_cached = a.R <= kRopeCacheRows;
      const size_t pstride = (size_t)NPAD * kTcBlockM;
#pragma unroll 1
      for (int u = wt; u < n_units; u += 256) {
        const int vec = u / UPV, c8 = u % UPV;
        int kind, rr, n, tile0;
        if (vec < nqv) { kind = 0; rr = (int)(((float)vec + 0.5f) * inv_group); n = (kvh * group + vec - rr * group) * HD; tile0 = 0; }
        else {
          const int v2 = vec - nqv, isv = v2 >= n_new ? 1 : 0;
          kind = 1 + isv; rr = nr_lo + v2 - isv * n_new; n = kvh * HD; tile0 = isv ? tile_v : tile_k;
        }
        n += c8 * 8;
        const int tile = tile0 + n / kTcBlockM, m = n % kTcBlockM;
        int n_pieces = g_parts;
        if (g_parts == 0) {                                      // dealt units: the owners of the tile's first and last k-block
          const int U = qkv_geom[4], Gp = qkv_geom[5], KB = qkv_geom[6];
          n_pieces = unit_owner(U, Gp, tile * KB + KB - 1) - unit_owner(U, Gp, tile * KB) + 1;
        }
        const float *base = a.pieces + ((size_t)(tile * g_pmax) * NPAD + (row0 + rr)) * kTcBlockM + m;
        float4 pc4[4][4];                                        // [piece][low 0-3, low 4-7, high 0-3, high 4-7]
#pragma unroll
        for (int pp = 0; pp < 4; ++pp) {
          const float4 *src = reinterpret_cast<const float4 *>(base + pp * pstride);
          const bool on = pp < n_pieces;
          pc4[pp][0] = on ? __ldcg(src) : make_float4(0.f, 0.f, 0.f, 0.f);
          pc4[pp][1] = on ? __ldcg(src + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
          pc4[pp][2] = on ? __ldcg(src + HALF / 4) : make_float4(0.f, 0.f, 0.f, 0.f);
          pc4[pp][3] = on ? __ldcg(src + HALF / 4 + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float cs[8], sn[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { cs[e] = 1.f; sn[e] = 0.f; }
        if (kind < 2) {
          const float *ct = rope_cached ? rope_cos_sh + (row0 + rr) * HALF + c8 * 8 : a.cos_tab + (size_t)(pos0 + rr) * HALF + c8 * 8;
          const float *st = rope_cached ? rope_sin_sh + (row0 + rr) * HALF + c8 * 8 : a.sin_tab + (size_t)(pos0 + rr) * HALF + c8 * 8;
#pragma unroll
          for (int e = 0; e < 8; e += 4) {
            const float4 cv = *reinterpret_cast<const float4 *>(ct + e), sv = *reinterpret_cast<const float4 *>(st + e);
            cs[e] = cv.x; cs[e + 1] = cv.y; cs[e + 2] = cv.z; cs[e + 3] = cv.w;
            sn[e] = sv.x; sn[e + 1] = sv.y; sn[e + 2] = sv.z; sn[e + 3] = sv.w;
          }
        }
        float lo[8], hi[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { lo[e] = 0.f; hi[e] = 0.f; }
#pragma unroll
        for (int pp = 0; pp < 4; ++pp) {
          lo[0] += pc4[pp][0].x; lo[1] += pc4[pp][0].y; lo[2] += pc4[pp][0].z; lo[3] += pc4[pp][0].w;
          lo[4] += pc4[pp][1].x; lo[5] += pc4[pp][1].y; lo[6] += pc4[pp][1].z; lo[7] += pc4[pp][1].w;
          hi[0] += pc4[pp][2].x; hi[1] += pc4[pp][2].y; hi[2] += pc4[pp][2].z; hi[3] += pc4[pp][2].w;
          hi[4] += pc4[pp][3].x; hi[5] += pc4[pp][3].y; hi[6] += pc4[pp][3].z; hi[7] += pc4[pp][3].w;
        }
        unsigned wl[4], wh[4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          const __nv_bfloat162 l2 = __floats2bfloat162_rn(lo[e] * cs[e] - hi[e] * sn[e], lo[e + 1] * cs[e + 1] - hi[e + 1] * sn[e + 1]);
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(hi[e] * cs[e] + lo[e] * sn[e], hi[e + 1] * cs[e + 1] + lo[e + 1] * sn[e + 1]);
          wl[e >> 1] = *reinterpret_cast<const unsigned *>(&l2);
          wh[e >> 1] = *reinterpret_cast<const unsigned *>(&h2);
        }
        const uint4 vl = make_uint4(wl[0], wl[1], wl[2], wl[3]), vh = make_uint4(wh[0], wh[1], wh[2], wh[3]);
        if (kind == 0) {
          *reinterpret_cast<uint4 *>(shQ + vec * RS + swz(vec, c8) * 8) = vl;
          *reinterpret_cast<uint4 *>(shQ + vec * RS + swz(vec, c8 + CPR / 2) * 8) = vh;
        } else {
          const int pos = pos0 + rr;
          __nv_bfloat16 *pool = kind == 1 ? lay.k_pool : lay.v_pool;
          const size_t off = (((size_t)kvh * a.n_pages + row_pg_sh[row0 + rr]) * a.page + (pos & (a.page - 1))) * HD + c8 * 8;
          *reinterpret_cast<uint4 *>(pool + off) = vl;
          *reinterpret_cast<uint4 *>(pool + off + HALF) = vh;
          const int st = (pos - key_lo) >> 4, kk = (pos - key_lo) & 15;
          if (st < step) {                                       // a first sub-tile: its warp (pair) is waiting for these rows
            const int w0 = n_mt == 2 ? 2 * st : st;
            for (int ww = w0; ww < w0 + (n_mt == 2 ? 2 : 1); ++ww) {
              __nv_bfloat16 *sh = shQ + 32 * RS + ww * (32 * RS) + (kind == 2 ? 16 * RS : 0);
              *reinterpret_cast<uint4 *>(sh + kk * RS + swz(kk, c8) * 8) = vl;
              *reinterpret_cast<uint4 *>(sh + kk * RS + swz(kk, c8 + CPR / 2) * 8) = vh;
            }
          }
        }
      }
    }
    float o[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[n][e] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int qrow[2] = {mt * 16 + g, mt * 16 + g + 8};          // query vectors of this thread's accumulator rows
    const int qpos[2] = {pos0 + qrow[0] / group, pos0 + qrow[1] / group};
    asm volatile("cp.async.wait_group 2;" ::: "memory");         // q rows landed (this thread's copies)
    worker_sync();                                               // ... and everybody's; page ids of the item stored
    if (wt == 0) pc->tag_item = (wi == (int)blockIdx.x && n_work <= (int)gridDim.x) ? wi : -1;
    lap(0);
#pragma unroll 1
    for (int j = 0; j < n_mine; ++j) {
      const int kt = key_lo + (first + j * step) * 16;
      if (j + 1 < n_mine && j + 1 - pg_base >= 32) load_pages(j + 1);
      lap(14);
      asm volatile("cp.async.wait_group 1;" ::: "memory");       // K of this sub-tile landed; V may be in flight
      __syncwarp();
      lap(10);
      // ---- S = Q K^T for 16 query vectors x 16 keys
      float sacc[2][4];
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) sacc[n][e] = 0.f;
      // fragments by ldmatrix: Q as the A operand (matrices: rows 0-7 / 8-15 x k 0-7 / 8-15), K as the B operand
      // of both 8-key n-tiles (keys 0-7 / 8-15 x k 0-7 / 8-15)
      {
        const int mi = lane >> 3, r8 = lane & 7;
        const int qrow_l = (mi & 1) * 8 + r8, krow_l = (mi >> 1) * 8 + r8;
        const __nv_bfloat16 *qbase = shQ + (mt * 16 + qrow_l) * RS, *kbase = shK + krow_l * RS;
#pragma unroll
        for (int ks = 0; ks < KST; ++ks) {
          unsigned af[4], bf4[4];
          ldmatrix_x4(af, qbase + swz(qrow_l, 2 * ks + (mi >> 1)) * 8);
          ldmatrix_x4(bf4, kbase + swz(krow_l, 2 * ks + (mi & 1)) * 8);
          mma_bf16_16x8x16(sacc[0], af, bf4[0], bf4[1]);
          mma_bf16_16x8x16(sacc[1], af, bf4[2], bf4[3]);
        }
      }
      __syncwarp();                                              // every lane is done with the K buffer
      lap(11);
      if (j + 1 < n_mine) issue(kpool, shK, j + 1, false, kAllKeys);
      else asm volatile("cp.async.commit_group;" ::: "memory");  // keep the group count uniform
      // ---- online softmax on the accumulator rows (g and g + 8); P re-packed as the A operand of P V
      unsigned ph[4], pl[4];
      float corr_h[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float sv[4];
        float mx = -INFINITY;
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int key = kt + n * 8 + 2 * t + e;
            float v = sacc[n][h * 2 + e] * scale;
            if (key >= key_hi || key > qpos[h] || qrow[h] >= nqv) v = -INFINITY;
            sv[n * 2 + e] = v;
            mx = fmaxf(mx, v);
          }
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
        const float m_new = fmaxf(m_run[h], mx);
        const float corr = (m_new > -INFINITY) ? __expf(m_run[h] - m_new) : 1.f;
        float ps = 0.f, pv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          pv[i] = (sv[i] > -INFINITY) ? __expf(sv[i] - m_new) : 0.f;
          ps += pv[i];
        }
        m_run[h] = m_new;
        l_run[h] = l_run[h] * corr + ps;                         // this thread's columns only; summed over t at the end
        corr_h[h] = corr;
#pragma unroll
        for (int n = 0; n < 2; ++n) {                            // A fragment: a[h] <- keys 2t.. of n-tile 0, a[2 + h] <- n-tile 1
          const __nv_bfloat162 hi = __floats2bfloat162_rn(pv[n * 2], pv[n * 2 + 1]);
          const float2 hf = __bfloat1622float2(hi);
          const __nv_bfloat162 lo = __floats2bfloat162_rn(pv[n * 2] - hf.x, pv[n * 2 + 1] - hf.y);
          ph[n * 2 + h] = *reinterpret_cast<const unsigned *>(&hi);
          pl[n * 2 + h] = *reinterpret_cast<const unsigned *>(&lo);
        }
      }
      lap(12);
      asm volatile("cp.async.wait_group 1;" ::: "memory");       // V of this sub-tile landed; the next K may be in flight
      __syncwarp();
      lap(13);
      // ---- O = O * corr + P V (the rescale is skipped while no row of the warp has a new maximum)
      if (__any_sync(0xFFFFFFFFu, corr_h[0] != 1.f || corr_h[1] != 1.f)) {
#pragma unroll
        for (int n = 0; n < NT; ++n) { o[n][0] *= corr_h[0]; o[n][1] *= corr_h[0]; o[n][2] *= corr_h[1]; o[n][3] *= corr_h[1]; }
      }
      {
        const int mi = lane >> 3, key_l = (mi & 1) * 8 + (lane & 7);
        const __nv_bfloat16 *vbase = shV + key_l * RS;
#pragma unroll
        for (int n = 0; n < NT; n += 2) {          // two 8-wide slices of the head dimension per ldmatrix
          unsigned bv[4];
          ldmatrix_x4_trans(bv, vbase + swz(key_l, n + (mi >> 1)) * 8);
          mma_bf16_16x8x16(o[n], ph, bv[0], bv[1]);
          mma_bf16_16x8x16(o[n], pl, bv[0], bv[1]);
          mma_bf16_16x8x16(o[n + 1], ph, bv[2], bv[3]);
          mma_bf16_16x8x16(o[n + 1], pl, bv[2], bv[3]);
        }
      }
      __syncwarp();                                              // every lane is done with the V buffer
      if (j + 1 < n_mine) issue(vpool, shV, j + 1, true, kAllKeys);
      else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    lap(1);
    // ---- merge the warps' states: each warp writes (o, m, l) of its 16 query vectors over the K/V buffers
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      l_run[h] += __shfl_xor_sync(0xFFFFFFFFu, l_run[h], 1);
      l_run[h] += __shfl_xor_sync(0xFFFFFFFFu, l_run[h], 2);
    }
    worker_sync();                                               // all warps are done with their K/V buffers
    lap(2);
    {
      float *mine = shMerge + (size_t)warp * 16 * MS;
      if (n_mine > 0) {
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          if (qrow[0] < nqv) *reinterpret_cast<float2 *>(mine + g * MS + n * 8 + 2 * t) = make_float2(o[n][0], o[n][1]);
          if (qrow[1] < nqv) *reinterpret_cast<float2 *>(mine + (g + 8) * MS + n * 8 + 2 * t) = make_float2(o[n][2], o[n][3]);
        }
      }
      if (t == 0) {                                              // a warp without keys contributes m = -inf only
        mine[g * MS + HD] = m_run[0]; mine[g * MS + HD + 1] = l_run[0];
        mine[(g + 8) * MS + HD] = m_run[1]; mine[(g + 8) * MS + HD + 1] = l_run[1];
      }
    }
    worker_sync();
    lap(3);
#pragma unroll 1
    for (int idx = wt; idx < nqv * (HD / 2); idx += 256) {       // two output dims per thread
      const int qi = idx / (HD / 2), dd = (idx % (HD / 2)) * 2;
      const int w0 = n_mt == 2 ? (qi >> 4) : 0, wstep = n_mt == 2 ? 2 : 1, rr = qi & 15;
      const float *src0 = shMerge + ((size_t)w0 * 16 + rr) * MS;
      const int wstride = wstep * 16 * MS, nw = min(n_mt == 2 ? 4 : 8, n_sub);     // warps (pairs) that had keys
      // one pass, all loads of four warps' states in flight together
      float mm = -INFINITY, l = 0.f, ox = 0.f, oy = 0.f;
#pragma unroll 1
      for (int k0 = 0; k0 < nw; k0 += 4) {
        float mw[4], lw[4];
        float2 ov[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float *src = src0 + (k0 + i) * wstride;
          const bool on = k0 + i < nw;
          mw[i] = on ? src[HD] : -INFINITY;
          lw[i] = on ? src[HD + 1] : 0.f;
          ov[i] = on ? *reinterpret_cast<const float2 *>(src + dd) : make_float2(0.f, 0.f);
        }
        float mn = mm;
#pragma unroll
        for (int i = 0; i < 4; ++i) mn = fmaxf(mn, mw[i]);
        const float c0 = (mn > -INFINITY) ? __expf(mm - mn) : 1.f;
        l *= c0; ox *= c0; oy *= c0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float sc = (mw[i] > -INFINITY) ? __expf(mw[i] - mn) : 0.f;
          l += sc * lw[i]; ox += sc * ov[i].x; oy += sc * ov[i].y;
        }
        mm = mn;
      }
      const int r = row0 + qi / group, hq = kvh * group + qi % group;
      if (a.n_splits == 1) {                                     // the only split: this is the attention output
        *reinterpret_cast<__nv_bfloat162 *>(a.att + ((size_t)r * a.nq + hq) * HD + dd) = __floats2bfloat162_rn(ox / l, oy / l);
      } else {
        float *dst = a.attn_partials + (((size_t)r * a.nq + hq) * a.n_splits + split) * (HD + 2);
        *reinterpret_cast<float2 *>(dst + dd) = make_float2(ox, oy);
        if (dd == 0) { dst[HD] = mm; dst[HD + 1] = l; }
      }
    }
    lap(4);
  }
}

// Phase B: merge the split partials of one (row, head) per HD / 2 threads (two output dimensions each); a single
// batch of loads.
template <int HD>
__device__ __forceinline__ void attn_merge_phase(const FwdArgs &a, const int *row_pos_sh, int wt) {
  constexpr int TPI = HD / 2, PER = 256 / TPI;                    // threads per item, items per CTA turn
  const int g = wt / TPI, dd = (wt % TPI) * 2;
  const int n_items = a.R * a.nq;
  for (int it = blockIdx.x * PER + g; it < n_items; it += PER * gridDim.x) {
    const int r = it / a.nq;
    const int used = min(a.n_splits, row_pos_sh[r] / a.keys_per_split + 1);   // splits holding keys <= own position
    const float *src = a.attn_partials + (size_t)it * a.n_splits * (HD + 2);
    float ms[kAttnMaxSplits], ls[kAttnMaxSplits];
    float2 os[kAttnMaxSplits];
#pragma unroll
    for (int s = 0; s < kAttnMaxSplits; ++s) {
      const bool on = s < used;
      const float2 ml = on ? __ldcg(reinterpret_cast<const float2 *>(src + s * (HD + 2) + HD)) : make_float2(-INFINITY, 0.f);
      ms[s] = ml.x; ls[s] = ml.y;
      os[s] = on ? __ldcg(reinterpret_cast<const float2 *>(src + s * (HD + 2) + dd)) : make_float2(0.f, 0.f);
    }
    float m = -INFINITY;
#pragma unroll
    for (int s = 0; s < kAttnMaxSplits; ++s) m = fmaxf(m, ms[s]);
    float l = 0.f, ox = 0.f, oy = 0.f;
#pragma unroll
    for (int s = 0; s < kAttnMaxSplits; ++s) {
      const float w = (ms[s] > -INFINITY) ? __expf(ms[s] - m) : 0.f;
      l += w * ls[s];
      ox += w * os[s].x;
      oy += w * os[s].y;
    }
    *reinterpret_cast<__nv_bfloat162 *>(a.att + (size_t)it * HD + dd) = __floats2bfloat162_rn(ox / l, oy / l);
  }
}

// ------------------------------------------------------------------------------ epilogue stores
// v[i] = final value of output feature (tile row m) for token row c0 + i.
template <int CH>
__device__ __forceinline__ void final_store(const FwdArgs &a, const Gemm &g, const Tile &ti, const FwdLayerDev &lay, int m, int et,
                                            int c0, const float *v, float *staging, const int *rpos, const int *rpg,
                                            const float *cs, const float *sn, int bar_id) {
  const int rows = g.rows;
  if (g.mode == MODE_ADD) {
    // residual-add projections never get here: their pieces are summed by the next norm phase
  } else if (g.mode == MODE_LOGITS) {
    const int n = ti.row0 + m;
    if (n < g.seg_n[0]) {
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const int r = c0 + i;
        if (r < rows) a.logits[(size_t)a.lrow_dst[r] * a.V + n] = __float2bfloat16_rn(v[i]);
      }
    }
  } else if (g.mode == MODE_SWIGLU) {
#pragma unroll
    for (int i = 0; i < CH; ++i) staging[m * (CH + 1) + i] = v[i];
    group_sync(bar_id);
    for (int idx = et; idx < kTcBoxRows * CH; idx += 128) {
      const int cc = idx % kTcBoxRows, i = idx / kTcBoxRows;
      const int r = c0 + i, col = ti.row0 + cc;
      if (r < rows && col < g.seg_n[0]) {
        const float gt = staging[cc * (CH + 1) + i], up = staging[(cc + kTcBoxRows) * (CH + 1) + i];
        a.act[(size_t)r * a.ff + col] = __float2bfloat16_rn(silu_mul(gt, up));
      }
    }
    group_sync(bar_id);
  } else {   // MODE_QKV: rotary embedding on q and k (cos / sin preloaded by the caller), then q -> buffer,
             // k / v -> their cache pages (row position and page id come from the per-launch row table)
#pragma unroll
    for (int i = 0; i < CH; ++i) staging[m * (CH + 1) + i] = v[i];
    group_sync(bar_id);
    const int n = ti.row0 + m;
    if (n < g.seg_n[ti.seg]) {
      const int hd = a.hd, half = hd >> 1;
      const int dd = n % hd, head = n / hd;
      const int mp = dd < half ? m + half : m - half;
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const int r = c0 + i;
        if (r < rows) {
          float out = v[i];
          if (ti.seg < 2) {
            const float pv = staging[mp * (CH + 1) + i];
            out = dd < half ? v[i] * cs[i] - pv * sn[i] : v[i] * cs[i] + pv * sn[i];
          }
          if (ti.seg == 0) {
            a.q[(size_t)r * g.seg_n[0] + n] = __float2bfloat16_rn(out);
          } else {
            const size_t off = (((size_t)head * a.n_pages + rpg[r]) * a.page + (rpos[r] & (a.page - 1))) * hd + dd;
            (ti.seg == 1 ? lay.k_pool : lay.v_pool)[off] = __float2bfloat16_rn(out);
          }
        }
      }
    }
    group_sync(bar_id);
  }
}

struct WorkerCtx {
  uint32_t tmem_base, accf_bar0, acce_bar0;      // accumulator-full / -empty barrier b = base + 8 b
  volatile int *abort_flag, *wait_ok;
  float *staging;
  const int *row_pos_sh, *row_pg_sh;
  const FwdLayerDev *layers_sh;
  const float *rope_cos_sh, *rope_sin_sh;
  int wt, lane, q, G, c;
  int seg_idx;
};

// GEMM phase p, epilogue side (warps 4..7): accumulator -> this CTA's piece of the tile.  Group-uniform:
// a give-up is decided by one thread and shared. 

template <int NPAD>
__device__ __forceinline__ void gemm_epilogue(const FwdArgs &a, WorkerCtx &w, int p) {
  constexpr int CH = PCfg<NPAD>::kChunk;
  const int m = w.q * 32 + w.lane;

    const Gemm g = make_gemm(a, p);
    const SplitGeom geo = split_geom(g, w.G);
    SegIter it = seg_begin(g, w.G, w.c);
    Seg sg;
    for (; seg_next(g, it, sg); ++w.seg_idx) {
      const int ab = w.seg_idx & 1;
      // this CTA's piece of the tile (the next phase sums the pieces): worked out while the MMAs run
      int fo, np_tile;
      tile_pieces(g, geo, sg.tile, fo, np_tile);
      const int piece = w.c - fo;
      float *mine = pieces_of(a, p) + ((size_t)sg.tile * geo.pieces_max + piece) * NPAD * kTcBlockM;
      if (w.wt == 0) w.wait_ok[w.seg_idx & 1] = mbar_wait((w.accf_bar0 + 8u * ab), (uint32_t)((w.seg_idx >> 1) & 1), w.abort_flag) ? 1 : 0;
      epi_sync();
      if (!w.wait_ok[w.seg_idx & 1]) return;
      tc_fence_after();
      const uint32_t tbase = w.tmem_base + ((uint32_t)(w.q * 32) << 16) + (uint32_t)(ab * NPAD);
#pragma unroll 1
      for (int c0 = 0; c0 < NPAD; c0 += CH) {
        float v[CH];
#pragma unroll
        for (int j = 0; j < CH / 16; ++j) tmem_ld16(tbase + c0 + j * 16, v + j * 16);
        tmem_ld_wait();
        if (c0 + CH >= NPAD) {                   // accumulator fully read: hand it back to the MMA warp
          tc_fence_before();
          __syncwarp();
          if (w.lane == 0) mbar_arrive((w.acce_bar0 + 8u * ab));
        }
        if (c0 < g.rows) {
#pragma unroll
          for (int i = 0; i < CH; ++i)
            if (c0 + i < g.rows) mine[(c0 + i) * kTcBlockM + m] = v[i];
        }
      }
    }
    // residual projection whose norm starts early: tell the norm's CTAs that this CTA's pieces are in place (the
    // stores of the 128 epilogue threads are ordered before the release by the group barrier, as in the grid barrier)
    if (a.early_norm && g.mode == MODE_ADD && w.c < geo.Gp) {
      epi_sync();
      if (w.wt == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.grid_counter + 16) : "memory");
    }
  }

// Down projection p of a pass with at most four rows: the worker warps build its activation tiles straight into
// the ring slots (SwiGLU of the gate / up pieces, summed in piece order; k-block kb of the down projection is tile
// kb of gate / up), in the layout the activation TMA box would have had (128-byte rows, 16-byte chunk index XOR
// row & 7).  Builder warp i of four takes the CTA's stages i, i + 4, ...; a lane covers one row x 8 columns.  Under the weight
// stream a load from L2 takes longer than a ring slot's turn-around, so with at most two pieces per tile (PB = 2)
// a warp keeps the loads of its next two stages in flight (DEPTH = 2).
template <int NPAD, int PB, int DEPTH>
__device__ __forceinline__ void build_act_stages(const FwdArgs &a, WorkerCtx &w, int p, uint8_t *ring, uint32_t full_bar0,
                                                 uint32_t empty_bar0, volatile unsigned *ring_pos, const int *bgeom) {
  constexpr int STAGES = PCfg<NPAD>::kStages;
  // geometry worked out once at kernel start (the same in every layer): this CTA's k-blocks of the down projection
  // (residual projections: one segment per CTA) and how the gate / up tiles are cut into pieces
  SegIter it;
  it.tile = 0; it.kb = bgeom[0]; it.left = bgeom[1];
  const int g_parts = bgeom[2], g_pmax = bgeom[3];
  const int KBg = a.d / kTcBlockK, Ug = ((a.ff + kTcBoxRows - 1) / kTcBoxRows) * KBg, Gpg = min(w.G, Ug);
  const float inv_U = 1.f / (float)Ug;
  // unit_owner without an integer division (all quantities < 2^24, so the float quotient is off by one at most)
  auto owner = [&](int u) {
    const int x = (u + 1) * Gpg - 1;
    int q = (int)((float)x * inv_U);
    const int rem = x - q * Ug;
    return rem < 0 ? q - 1 : (rem >= Ug ? q + 1 : q);
  };
  // builders: the four worker warps that share no scheduler with the weight producer or the MMA issuer (single
  // threads whose issue rate bounds the phase)
  if (it.left <= 0 || ((w.wt >> 5) & 1) == 0) return;
  // ring position (slot, parity of its empty barrier) of the phase's first stage, published by the weight producer
  ring_pos += (p >> 2) & 15;
  unsigned rp = *ring_pos;
  if ((int)(rp >> 16) != p) {
    const unsigned long long t0 = globaltimer_ns();
    while ((int)((rp = *ring_pos) >> 16) != p)
      if (*w.abort_flag || globaltimer_ns() - t0 > kWaitLimitNs) { *w.abort_flag = 1; return; }
  }
  const int s0 = (int)(rp & 0xFFu), warp4 = w.wt >> 6, r = w.lane >> 3, c8 = w.lane & 7;
  const uint32_t par0 = (rp >> 8) & 1u;
  const bool on = r < a.R;
  const size_t pstride = (size_t)NPAD * kTcBlockM;
  const float *lane_base = a.pieces + (size_t)r * kTcBlockM + c8 * 8;
  float4 t[DEPTH][PB][4];                                      // [stage in flight][piece][gate 0-3, gate 4-7, up 0-3, up 4-7]
  auto load = [&](float4 (&dst)[PB][4], int i) {               // pieces of the CTA's stage i (this lane's row and columns)
    const int kb = it.kb + i;
    int n_pieces = 0;
    if (i < it.left) n_pieces = g_parts ? g_parts : owner(kb * KBg + KBg - 1) - owner(kb * KBg) + 1;
    const float *tbase = lane_base + (size_t)kb * g_pmax * pstride;
#pragma unroll
    for (int pp = 0; pp < PB; ++pp) {
      const float4 *src = reinterpret_cast<const float4 *>(tbase + pp * pstride);
      const bool ld = on && pp < n_pieces;
      dst[pp][0] = ld ? __ldcg(src) : make_float4(0.f, 0.f, 0.f, 0.f);
      dst[pp][1] = ld ? __ldcg(src + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
      dst[pp][2] = ld ? __ldcg(src + kTcBoxRows / 4) : make_float4(0.f, 0.f, 0.f, 0.f);
      dst[pp][3] = ld ? __ldcg(src + kTcBoxRows / 4 + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
#pragma unroll
  for (int dpt = 0; dpt < DEPTH; ++dpt) load(t[dpt], warp4 + 4 * dpt);
#pragma unroll 1
  for (int i0 = warp4; i0 < it.left; i0 += 4 * DEPTH) {
#pragma unroll
    for (int dpt = 0; dpt < DEPTH; ++dpt) {
      const int i = i0 + 4 * dpt;
      if (i >= it.left) break;
      const int pos = s0 + i, s = pos % STAGES;
      const uint32_t par = par0 ^ (uint32_t)((pos / STAGES) & 1);
      bool ok = true;                                          // the slot is free once its previous MMAs have retired
      if (w.lane == 0) ok = mbar_wait(empty_bar0 + 8u * s, par, w.abort_flag);
      if (!__shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0)) return;
      float gt[8], up[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) { gt[e] = 0.f; up[e] = 0.f; }
#pragma unroll
      for (int pp = 0; pp < PB; ++pp) {
        gt[0] += t[dpt][pp][0].x; gt[1] += t[dpt][pp][0].y; gt[2] += t[dpt][pp][0].z; gt[3] += t[dpt][pp][0].w;
        gt[4] += t[dpt][pp][1].x; gt[5] += t[dpt][pp][1].y; gt[6] += t[dpt][pp][1].z; gt[7] += t[dpt][pp][1].w;
        up[0] += t[dpt][pp][2].x; up[1] += t[dpt][pp][2].y; up[2] += t[dpt][pp][2].z; up[3] += t[dpt][pp][2].w;
        up[4] += t[dpt][pp][3].x; up[5] += t[dpt][pp][3].y; up[6] += t[dpt][pp][3].z; up[7] += t[dpt][pp][3].w;
      }
      if (on) {
        unsigned o[4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          const __nv_bfloat162 v2 = __floats2bfloat162_rn(silu_mul(gt[e], up[e]), silu_mul(gt[e + 1], up[e + 1]));
          o[e >> 1] = *reinterpret_cast<const unsigned *>(&v2);
        }
        uint8_t *slot = ring + (size_t)s * PCfg<NPAD>::kStageBytes + kWBytes;
        *reinterpret_cast<uint4 *>(slot + r * 128 + ((c8 ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads the tile through the async proxy
      __syncwarp();
      if (w.lane == 0) mbar_arrive(full_bar0 + 8u * s);
      load(t[dpt], i + 4 * DEPTH);                               // this buffer's next stage
    }
  }
}

// Finish phase of GEMM p (QKV, gate/up, output head): units of (tile, block of up to 8 token rows)
// round-robin over the CTAs, two at a time (one per 128-thread group); the pieces of a tile (at most
// four) are added in piece order and the result goes through the projection's own epilogue.  The
// loads of the next four rows (pieces, rope values) are in flight while the current four are stored.
template <int NPAD>
__device__ __forceinline__ void gemm_finish(const FwdArgs &a, WorkerCtx &w, int p) {
  constexpr int RG = 4;                          // token rows per load batch (decode passes have few rows)
  constexpr int PBF = 4;                         // pieces per tile at most (regular: <= 4 parts; dealt units: <= 3)
  constexpr int RB = 8;                          // token rows per unit (two load batches; more units than 2 x CTAs at 24+ rows)
  const Gemm g = make_gemm(a, p);
  const SplitGeom geo = split_geom(g, w.G);
  const int layer = p >> 2;
  const int gidx = w.wt >> 7, gm = w.wt & 127;   // two groups of 128 threads, one unit each at a time
  float *gstage = w.staging + gidx * (kTcBlockM * (RG + 1));
  const int n_rb = (g.rows + RB - 1) / RB, n_units = g.n_tiles * n_rb;
  const bool rope_cached = a.R <= kRopeCacheRows;
  if (g.mode == MODE_SWIGLU) {
    // gate / up: a thread owns one of the tile's 64 columns (gate in tile row c, up in tile row c + 64) and four of
    // the unit's eight token rows; all its loads are in flight at once, no staging and no barrier
    const int cc = gm & (kTcBoxRows - 1), rh = (gm >> 6) * (RB / 2);
#pragma unroll 1
    for (int u = w.c + gidx * w.G; u < n_units; u += 2 * w.G) {
      const int tile = u / n_rb, r0 = (u - tile * n_rb) * RB + rh, col = tile * kTcBoxRows + cc;
      int fo, n_pieces;
      tile_pieces(g, geo, tile, fo, n_pieces);
      const float *base = a.pieces + (size_t)tile * geo.pieces_max * NPAD * kTcBlockM + cc;
      float tg[PBF][RB / 2], tu[PBF][RB / 2];
#pragma unroll
      for (int pp = 0; pp < PBF; ++pp)
#pragma unroll
        for (int i = 0; i < RB / 2; ++i) {
          const bool on = pp < n_pieces && r0 + i < g.rows;
          const float *src = base + ((size_t)pp * NPAD + r0 + i) * kTcBlockM;
          tg[pp][i] = on ? __ldcg(src) : 0.f;
          tu[pp][i] = on ? __ldcg(src + kTcBoxRows) : 0.f;
        }
      if (col < g.seg_n[0]) {
#pragma unroll
        for (int i = 0; i < RB / 2; ++i) {
          float gt = 0.f, up = 0.f;
#pragma unroll
          for (int pp = 0; pp < PBF; ++pp) { gt += tg[pp][i]; up += tu[pp][i]; }
          if (r0 + i < g.rows) a.act[(size_t)(r0 + i) * a.ff + col] = __float2bfloat16_rn(silu_mul(gt, up));
        }
      }
    }
    return;
  }
#pragma unroll 1
  for (int u = w.c + gidx * w.G; u < n_units; u += 2 * w.G) {
    const int tile = u / n_rb, r_lo = (u - tile * n_rb) * RB, r_hi = min(g.rows, r_lo + RB);
    const Tile ti = tile_of(g, tile);
    int fo, n_pieces;
    tile_pieces(g, geo, tile, fo, n_pieces);
    const float *base = a.pieces + (size_t)tile * geo.pieces_max * NPAD * kTcBlockM + gm;
    const int half = a.hd >> 1, dh = ((ti.row0 + gm) % a.hd) % half;
    const bool rope = (g.mode == MODE_QKV && ti.seg < 2);
    float tn[PBF][RG], csn[RG], snn[RG];
    auto fetch = [&](int c0) {                   // pieces and rope values of rows c0 .. c0 + RG - 1
#pragma unroll
      for (int pp = 0; pp < PBF; ++pp)
#pragma unroll
        for (int i = 0; i < RG; ++i)
          tn[pp][i] = (pp < n_pieces && c0 + i < r_hi) ? __ldcg(base + ((size_t)pp * NPAD + c0 + i) * kTcBlockM) : 0.f;
#pragma unroll
      for (int i = 0; i < RG; ++i) {
        csn[i] = 1.f; snn[i] = 0.f;
        if (rope && c0 + i < r_hi) {
          if (rope_cached) {
            csn[i] = w.rope_cos_sh[(c0 + i) * half + dh];
            snn[i] = w.rope_sin_sh[(c0 + i) * half + dh];
          } else {
            csn[i] = __ldg(a.cos_tab + (size_t)w.row_pos_sh[c0 + i] * half + dh);
            snn[i] = __ldg(a.sin_tab + (size_t)w.row_pos_sh[c0 + i] * half + dh);
          }
        }
      }
    };
    fetch(r_lo);
#pragma unroll 1
    for (int c0 = r_lo; c0 < r_hi; c0 += RG) {
      float v[RG], cs[RG], sn[RG];
#pragma unroll
      for (int i = 0; i < RG; ++i) {
        v[i] = 0.f;
#pragma unroll
        for (int pp = 0; pp < PBF; ++pp) v[i] += tn[pp][i];
        cs[i] = csn[i]; sn[i] = snn[i];
      }
      if (c0 + RG < r_hi) fetch(c0 + RG);
      final_store<RG>(a, g, ti, w.layers_sh[layer < a.n_run ? layer : 0], gm, gm, c0, v, gstage, w.row_pos_sh,
                      w.row_pg_sh, cs, sn, 1 + 2 * gidx);
    }
  }
}

// TC: the launch's long attention work items run on tensor memory (a.tc_attn; head size 128 only).  A kernel of its
// own, so that the other launches keep their code (and its place in the instruction cache) unchanged.
template <int NPAD, int HD, bool TC>
__global__ void __launch_bounds__(kFwdThreads, 1) fwd_persistent_kernel(const __grid_constant__ FwdArgs a) {
  using Cfg = PCfg<NPAD>;
  constexpr int STAGES = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t *ring = smem;
  uint8_t *scratch = smem + STAGES * Cfg::kStageBytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(scratch + kScratchBytes);
  // bars: full[STAGES] | empty[STAGES] | acc_full[2] | acc_empty[2] | ready[2]
  uint32_t *ctl = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 6);
  uint32_t *tmem_slot = ctl;
  volatile int *abort_flag = reinterpret_cast<volatile int *>(ctl + 1);
  int *first_item_sh = reinterpret_cast<int *>(ctl + 148);               // [4] this CTA's first attention item
  int *qkv_geom_sh = reinterpret_cast<int *>(ctl + 152);                 // [7] piece geometry of the QKV projection
  // [16] phase << 16 | parity << 8 | slot of the first stage of built down projection number (layer & 15): the
  // weight producer is at most one ring (8 stages) ahead, so never 16 such phases
  volatile unsigned *ring_pos_sh = reinterpret_cast<volatile unsigned *>(ctl + 928);
  int *bgeom_sh = reinterpret_cast<int *>(ctl + 944);                    // [4] geometry of the built down projection
  static_assert((2 * Cfg::kStages + 6) * 8 + (944 + 4) * 4 <= kCtrlBytes - 128, "control area overflow");
  volatile int *wait_ok = reinterpret_cast<volatile int *>(ctl + 4);   // [2]
  float *red = reinterpret_cast<float *>(ctl + 8);                      // [8]
  PageCache *pcache = reinterpret_cast<PageCache *>(ctl + 16);          // 130 words
  int *row_pos_sh = reinterpret_cast<int *>(ctl + 160);                 // [128] position of each packed row
  int *row_pg_sh = reinterpret_cast<int *>(ctl + 288);                  // [128] KV page holding that position
  FwdLayerDev *layers_sh = reinterpret_cast<FwdLayerDev *>(ctl + 416);  // [<= kMaxLayersSh] pointer table
  long long *dbg_cy = reinterpret_cast<long long *>(reinterpret_cast<uint8_t *>(bars) + kCtrlBytes - 128);   // debug cycle counters [16]
  // cos / sin of the launch's rows (the tables are touched once per layer, so the weight stream would
  // evict them from L2 between uses): [kRopeCacheRows][hd / 2] each, after the attention / staging area
  float *rope_cos_sh = reinterpret_cast<float *>(scratch + kScratchBytes - 2 * kRopeCacheRows * (HD / 2) * 4);
  float *rope_sin_sh = rope_cos_sh + kRopeCacheRows * (HD / 2);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
  auto ready_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 4 + b); };
  const uint32_t attn_done_bar = smem_u32(dbg_cy + 15);         // the last counter slot (laps use 0..14)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, c = blockIdx.x;
  const int n_phases = 4 * a.n_run + (a.L > 0 ? 1 : 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4); mbar_init(ready_bar(b), 1); }
    *abort_flag = 0;
    for (int i = 0; i < 15; ++i) dbg_cy[i] = 0;
    mbar_init(attn_done_bar, 1);
    for (int i = 0; i < 16; ++i) ring_pos_sh[i] = 0xFFFFFFFFu;
    pcache->tag_item = -1;
    pcache->tag_tile = -1;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  constexpr uint32_t tmem_cols = TC ? 512u : (uint32_t)Cfg::kTmemCols;      // the attention phase takes all of tensor memory
  if (warp == 2) tmem_alloc(smem_u32(tmem_slot), tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The three pipeline roles below are single threads: a lone thread runs ~5 cycles per dependent
  // instruction, and with whole-tile GEMMs one SM has to sustain up to twice its fair share of the
  // weight stream (~90 GB/s = one 16 KiB stage per 180 ns).  So they keep wrapped slot counters and
  // parities in registers instead of dividing a stage count, ring slots are handed back in pairs (a
  // tcgen05.commit costs the tensor pipe as much as three MMAs of this shape), and
  // tcgen05.fence::after_thread_sync (~0.1 us while MMAs are in flight) is issued only where another
  // thread's tcgen05 operations must come first (accumulator reuse), not after the wait on TMA data.
  constexpr int WGS = 1;                                          // landing slots handed back together
  if (warp == 0) {
    // ------------------------------------------------------------ weight-tile producer (runs ahead)
    if (lane == 0) {
      int s = 0, n_issued = 0;
      uint32_t par = 1;                                  // parity to wait for on the slot group's empty barrier
      const uint64_t w_policy = l2_policy_evict_first();  // weights are read once per pass: first out of L2
      bool ok = true;
      for (int p = 0; p < n_phases && ok; ++p) {
        const Gemm g = make_gemm(a, p);
        SegIter it = seg_begin(g, G, c);
        Seg sg;
        // the tensor-memory attention phase uses the ring's memory: the O projection's tiles wait until it is over
        // (one completion per layer, waited for in every layer, so the parity never is ambiguous)
        if (TC && (p & 3) == 1 && p < 4 * a.n_run && !mbar_wait(attn_done_bar, (uint32_t)((p >> 2) & 1), abort_flag)) { ok = false; break; }
        if (built_down(a, p)) ring_pos_sh[(p >> 2) & 15] = (unsigned)s | (par << 8) | ((unsigned)p << 16);   // where the builders' tiles go
        while (ok && seg_next(g, it, sg)) {
          const Tile ti = tile_of(g, sg.tile);
          const bool second = (g.mode == MODE_SWIGLU) || (ti.row0 + kTcBoxRows < g.seg_n[ti.seg]);
          const CUtensorMap *m0 = g.mode == MODE_SWIGLU ? g.w[0] : g.w[ti.seg];
          const CUtensorMap *m1 = g.mode == MODE_SWIGLU ? g.w[1] : m0;
          const int row1 = g.mode == MODE_SWIGLU ? ti.row0 : ti.row0 + kTcBoxRows;
          const uint32_t tx = (second ? 2 : 1) * kBoxBytes;
          for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
            if (s % WGS == 0 && !mbar_wait(empty_bar(s / WGS), par, abort_flag)) { ok = false; break; }
            const uint32_t dst = smem_u32(ring) + (uint32_t)(s * Cfg::kStageBytes);
            mbar_expect_tx(full_bar(s), tx);
            tma_load_2d_hint(dst, m0, kb * kTcBlockK, ti.row0, full_bar(s), w_policy);
            if (second) tma_load_2d_hint(dst + kBoxBytes, m1, kb * kTcBlockK, row1, full_bar(s), w_policy);
            ++n_issued;
            if (++s == STAGES) { s = 0; par ^= 1u; }
          }
        }
      }
      if (!ok) {
        atomicExch(a.status, 1);
        // let copies in flight land (bounded): the last min(n_issued, STAGES) slots, newest first
        uint32_t fpar = par ^ 1u;                        // full-barrier parity of the current round
        for (int i = 0, sl = s; i < STAGES && i < n_issued; ++i) {
          if (--sl < 0) { sl = STAGES - 1; fpar ^= 1u; }
          unsigned long long t0 = globaltimer_ns();
          while (!mbar_try_wait(full_bar(sl), fpar))
            if (globaltimer_ns() - t0 > kWaitLimitNs / 4) break;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ activation-tile producer
    if (lane == 0) {
      int s = 0;
      uint32_t par = 1;
      bool ok = true;
      const uint32_t a_bytes = (uint32_t)a.a_box_rows * kTcBlockK * 2;
      for (int p = 0; p < n_phases && ok; ++p) {
        const Gemm g = make_gemm(a, p);
        SegIter it = seg_begin(g, G, c);
        Seg sg;
        bool have = seg_next(g, it, sg);
        // the operand of phase p is complete once the workers have passed the barrier before it
        if (!mbar_wait(ready_bar(p & 1), (uint32_t)((p >> 1) & 1), abort_flag)) { ok = false; break; }
        const bool built = built_down(a, p);
        while (ok && have) {
          for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
            if (s % WGS == 0 && !mbar_wait(empty_bar(s / WGS), par, abort_flag)) { ok = false; break; }
            const uint32_t dst = smem_u32(ring) + (uint32_t)(s * Cfg::kStageBytes) + kWBytes;
            if (!built) {                                // built down projection: the workers fill the tile and arrive
              mbar_expect_tx(full_bar(s), a_bytes);
              tma_load_2d(dst, g.amap, kb * kTcBlockK, 0, full_bar(s));
            }
            if (++s == STAGES) { s = 0; par ^= 1u; }
          }
          have = seg_next(g, it, sg);
        }
      }
      if (!ok) atomicExch(a.status, 1);
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(NPAD);
      const uint64_t da0 = umma_desc(smem_u32(ring));
      int s = 0, seg_idx = 0;
      uint32_t par = 0;
      bool ok = true;
      for (int p = 0; p < n_phases && ok; ++p) {
        const Gemm g = make_gemm(a, p);
        SegIter it = seg_begin(g, G, c);
        Seg sg;
        for (; ok && seg_next(g, it, sg); ++seg_idx) {
          const int ab = seg_idx & 1;
          if (!mbar_wait(acce_bar(ab), (uint32_t)(((seg_idx >> 1) & 1) ^ 1), abort_flag)) { ok = false; break; }
          tc_fence_after();                              // the epilogue's tcgen05.ld of this accumulator come first
          const uint32_t d_tmem = tmem_base + (uint32_t)(ab * NPAD);
          uint32_t acc = 0u;
          for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
            if (!mbar_wait(full_bar(s), par, abort_flag)) { ok = false; break; }
            const uint64_t da = da0 + (uint64_t)(s * (Cfg::kStageBytes >> 4)), db = da + (uint64_t)(kWBytes >> 4);
            umma_bf16(d_tmem, da, db, idesc, acc);
#pragma unroll
            for (int k = 1; k < kTcBlockK / 16; ++k) umma_bf16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, 1u);
            acc = 1u;
            if (s % WGS == WGS - 1) umma_commit(empty_bar(s / WGS));
            if (++s == STAGES) { s = 0; par ^= 1u; }
          }
          if (ok) umma_commit(accf_bar(ab));
        }
      }
      if (!ok) atomicExch(a.status, 1);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------ workers (+ epilogue: warps 4..7)
    const int wt = threadIdx.x - 128;              // 0..255
    const bool is_epi = warp < 8;
    const int q = warp & 3;
    float *staging = reinterpret_cast<float *>(scratch);
    unsigned epoch = 0;
    bool alive = true;

    WorkerCtx w;
    w.tmem_base = tmem_base; w.accf_bar0 = accf_bar(0); w.acce_bar0 = acce_bar(0);
    w.abort_flag = abort_flag; w.wait_ok = wait_ok; w.staging = staging;
    w.row_pos_sh = row_pos_sh; w.row_pg_sh = row_pg_sh; w.layers_sh = layers_sh;
    w.rope_cos_sh = rope_cos_sh; w.rope_sin_sh = rope_sin_sh;
    w.wt = wt; w.lane = lane; w.q = q; w.G = G; w.c = c; w.seg_idx = 0;

    // ---- phase program
    if (HSD_PROF(a) && wt == 0) a.prof[(size_t)blockIdx.x * kFwdProfEvents] = globaltimer_ns();
    for (int l = wt; l < a.n_run; l += 256) layers_sh[l] = a.layers[l];
    if (a.R <= kRopeCacheRows)
      for (int i = wt; i < a.R * (HD / 2); i += 256) {
        const int r = i / (HD / 2), k = i % (HD / 2);
        rope_cos_sh[i] = a.cos_tab[(size_t)a.row_pos[r] * (HD / 2) + k];
        rope_sin_sh[i] = a.sin_tab[(size_t)a.row_pos[r] * (HD / 2) + k];
      }
    for (int r = wt; r < a.R; r += 256) {             // per-row facts every layer needs, fetched once
      const int pos = a.row_pos[r];
      row_pos_sh[r] = pos;
      row_pg_sh[r] = a.page_table[(size_t)a.row_seq[r] * a.pages_per_seq + pos / a.page];
    }
    // descriptor of this CTA's first attention work item, kept in shared memory (the same in every layer; a
    // dependent global load at the start of every attention phase otherwise)
    if (wt == 0) {
      const int n_work = a.n_attn * a.nkv * a.n_splits;
      int4 fi = make_int4(0, 0, 0, 0);
      if ((int)blockIdx.x < n_work) fi = a.attn_items[blockIdx.x / (a.n_splits * a.nkv)];
      first_item_sh[0] = fi.x; first_item_sh[1] = fi.y; first_item_sh[2] = fi.z; first_item_sh[3] = fi.w;
      const Gemm gq = make_gemm(a, 0);
      const SplitGeom geo = split_geom(gq, G);
      qkv_geom_sh[0] = (gq.seg_n[0] + kTcBlockM - 1) / kTcBlockM;
      qkv_geom_sh[1] = qkv_geom_sh[0] + (gq.seg_n[1] + kTcBlockM - 1) / kTcBlockM;
      qkv_geom_sh[2] = geo.parts; qkv_geom_sh[3] = geo.pieces_max; qkv_geom_sh[4] = geo.U; qkv_geom_sh[5] = geo.Gp; qkv_geom_sh[6] = gq.KB;
      const Gemm gdn = make_gemm(a, 3);
      const SplitGeom geo_gu = split_geom(make_gemm(a, 2), G);
      const SegIter itd = seg_begin(gdn, G, c);
      bgeom_sh[0] = itd.kb; bgeom_sh[1] = itd.left; bgeom_sh[2] = geo_gu.parts; bgeom_sh[3] = geo_gu.pieces_max;
    }
    // One step loop, one call site per phase body: the whole per-layer program has to stay resident in
    // the instruction cache (every phase runs once per layer, so code that does not fit is fetched
    // cold through the saturated memory system every single time).
    //   t = 0                embed + norm                                  -> ready(QKV 0)
    //   t = 1 + 10 l + s     s: 0 QKV pieces | 1 QKV finish | 2 attention tiles | 3 attention merge -> ready(O)
    //                           4 O pieces | 5 norm (+O pieces) -> ready(gate/up) | 6 gate/up pieces
    //                           7 gate/up finish -> ready(down) | 8 down pieces | 9 norm (+down pieces) -> ready(next)
    //   t = 1 + 10 n, + 1    output-head pieces | output-head finish
    // Steps 1 and 7 are empty (no barrier) when the finish is folded into the phase after it.
    const int n_steps = 1 + 10 * a.n_run + (a.L > 0 ? 2 : 0);
    enum { K_EPI, K_FIN, K_ATTN_A, K_ATTN_B, K_NORM, K_NONE };
    // CTAs with pieces of the two residual projections; pieces stored so far (what the early norm waits for)
    const unsigned add_ctas_o = (unsigned)min(G, split_geom(make_gemm(a, 1), G).Gp), add_ctas_d = (unsigned)min(G, split_geom(make_gemm(a, 3), G).Gp);
    unsigned pieces_target = 0u;
#pragma unroll 1
    for (int t = 0; t < n_steps && alive; ++t) {
      int kind, gp = 0, ready = -1, l = 0;
      bool barrier = true;
      if (t == 0) { kind = K_NORM; ready = 0; }
      else if (t > 10 * a.n_run) { gp = 4 * a.n_run; kind = (t == 1 + 10 * a.n_run) ? K_EPI : K_FIN; barrier = (kind == K_EPI); }
      else {
        l = (t - 1) / 10;
        const int sstep = (t - 1) % 10, p = 4 * l;
        switch (sstep) {
          case 0: kind = K_EPI; gp = p; break;
          case 1:                                            // folded into the attention phase when every item stands alone
            if (a.fuse_qkv) { kind = K_NONE; barrier = false; }
            else { kind = K_FIN; gp = p; }
            break;
          case 2: kind = K_ATTN_A; if (a.n_splits == 1) ready = p + 1; break;       // a single key split needs no merge phase
          case 3:
            if (a.n_splits == 1) { kind = K_NONE; barrier = false; }
            else { kind = K_ATTN_B; ready = p + 1; }
            break;
          case 4: kind = K_EPI; gp = p + 1; barrier = !a.early_norm; break;
          case 5: kind = K_NORM; gp = p + 1; ready = p + 2; break;
          case 6: kind = K_EPI; gp = p + 2; if (a.fuse_gu) ready = p + 3; break;
          case 7:                                            // folded into the down projection in passes with few rows
            if (a.fuse_gu) { kind = K_NONE; barrier = false; }
            else { kind = K_FIN; gp = p + 2; ready = p + 3; }
            break;
          case 8: kind = K_EPI; gp = p + 3; barrier = (l + 1 < a.n_run || a.L > 0) && !a.early_norm; break;
          default:
            kind = (l + 1 < a.n_run || a.L > 0) ? K_NORM : K_NONE; gp = p + 3; ready = p + 4;
            barrier = (kind == K_NORM);
            break;
        }
      }
      switch (kind) {
        case K_EPI:
          if (built_down(a, gp)) {
            if (a.gu_pieces_max <= 2) build_act_stages<NPAD, 2, 2>(a, w, gp, ring, full_bar(0), empty_bar(0), ring_pos_sh, bgeom_sh);
            else build_act_stages<NPAD, 4, 1>(a, w, gp, ring, full_bar(0), empty_bar(0), ring_pos_sh, bgeom_sh);
          }
          if (is_epi) gemm_epilogue<NPAD>(a, w, gp);
          break;
        case K_FIN: gemm_finish<NPAD>(a, w, gp); break;
        case K_ATTN_A:
          attn_tiles_phase<NPAD, HD, TC>(a, layers_sh[l], scratch, pcache, wt, dbg_cy, first_item_sh, qkv_geom_sh, row_pg_sh, rope_cos_sh, rope_sin_sh,
                                     ring, tmem_base, abort_flag);
          if (TC) {                                               // the ring's memory is the weight producer's again
            worker_sync();
            if (wt == 0) mbar_arrive(attn_done_bar);
          }
          break;
        case K_ATTN_B: attn_merge_phase<HD>(a, row_pos_sh, wt); break;
        case K_NORM: {
          const bool first = (t == 0);
          const bool last = !first && (((t - 1) % 10) == 9) && (l + 1 >= a.n_run);      // final norm over the logit rows
          const bool mid = !first && (((t - 1) % 10) == 5);
          const Gemm pend = make_gemm(a, first ? 0 : gp);
          const __nv_bfloat16 *gain = first ? a.layers[0].attn_norm
                                            : (last ? a.final_norm : (mid ? layers_sh[l].mlp_norm : layers_sh[l + 1].attn_norm));
          if (!first && a.early_norm) pieces_target += mid ? add_ctas_o : add_ctas_d;
          alive = norm_phase<NPAD>(a, last ? a.L : a.R, last ? a.lrow_src : nullptr, first, first ? nullptr : &pend, pieces_of(a, gp), gain,
                                   last ? a.hf : a.h, red, wt, (!first && a.early_norm) ? pieces_target : 0u, abort_flag);
          break;
        }
        default: break;
      }
      if (barrier && alive) alive = grid_barrier(a, epoch, abort_flag, wt, ready >= 0 ? ready_bar(ready & 1) : 0u);
    }
  }
  if (HSD_PROF(a) && blockIdx.x == 0 && threadIdx.x == 128) for (int i = 0; i < 15; ++i) a.prof[940 + i] = (unsigned long long)dbg_cy[i];
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 2) tmem_dealloc(tmem_base, tmem_cols);
  if (threadIdx.x == 0 && *abort_flag) atomicExch(a.status, 1);
}

// The attention tiles phase as a launch of its own (prompt passes with more rows than the persistent forward takes):
// one key split per item, so every work item writes its rows of the attention output itself.  256 threads = the
// phase's eight worker warps; q / k / v of the pass are in place (separate finish kernels).
template <int HD>
__global__ void __launch_bounds__(256, 2) attn_tiles_kernel(const __grid_constant__ FwdArgs a, __nv_bfloat16 *k_pool, __nv_bfloat16 *v_pool) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *scratch = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ PageCache pcache;
  __shared__ int first_item_sh[4];
  __shared__ int qkv_geom_sh[8];
  __shared__ long long dbg_cy[16];
  if (threadIdx.x == 0) {
    pcache.tag_item = -1;
    pcache.tag_tile = -1;
    const int n_work = a.n_attn * a.nkv * a.n_splits;
    int4 fi = make_int4(0, 0, 0, 0);
    if ((int)blockIdx.x < n_work) fi = a.attn_items[blockIdx.x / (a.n_splits * a.nkv)];
    first_item_sh[0] = fi.x; first_item_sh[1] = fi.y; first_item_sh[2] = fi.z; first_item_sh[3] = fi.w;
  }
  __syncthreads();
  FwdLayerDev lay;
  lay.attn_norm = nullptr; lay.mlp_norm = nullptr; lay.k_pool = k_pool; lay.v_pool = v_pool;
  attn_tiles_phase<128, HD, false>(a, lay, scratch, &pcache, (int)threadIdx.x, dbg_cy, first_item_sh, qkv_geom_sh, nullptr, nullptr, nullptr,
                            nullptr, 0u, nullptr);
}

template <int HD>
int launch_attn_tiles_t(const FwdArgs &a, __nv_bfloat16 *k_pool, __nv_bfloat16 *v_pool, int sm_count, cudaStream_t s) {
  static bool attr_set = false;
  const int smem = kScratchBytes + 1024;
  if (!attr_set) {
    HSD_CUDA_OK(cudaFuncSetAttribute(attn_tiles_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_set = true;
  }
  const int n_work = a.n_attn * a.nkv * a.n_splits;
  attn_tiles_kernel<HD><<<std::min(n_work, 2 * sm_count), 256, smem, s>>>(a, k_pool, v_pool);
  hsd_count_launches(1);
  return hsd_launch_status();
}

template <int NPAD, int HD, bool TC>
int launch_t(const FwdArgs &args, int sm_count, cudaStream_t s) {
  using Cfg = PCfg<NPAD>;
  static bool attr_set = false;
  if (!attr_set) {
    HSD_CUDA_OK(cudaFuncSetAttribute(fwd_persistent_kernel<NPAD, HD, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    attr_set = true;
  }
  void *params[1] = {const_cast<FwdArgs *>(&args)};
  HSD_CUDA_OK(cudaLaunchCooperativeKernel((const void *)fwd_persistent_kernel<NPAD, HD, TC>, dim3(sm_count), dim3(kFwdThreads), params,
                                          (size_t)Cfg::kSmemBytes, s));
  hsd_count_launches(1);
  return HSD_OK;
}

template <int HD, bool TC>
int launch_hd(const FwdArgs &args, int npad, int sm_count, cudaStream_t s) {
  switch (npad) {
    case 16: return launch_t<16, HD, TC>(args, sm_count, s);
    case 32: return launch_t<32, HD, TC>(args, sm_count, s);
    case 64: return launch_t<64, HD, TC>(args, sm_count, s);
    case 128: return launch_t<128, HD, TC>(args, sm_count, s);
    default: return HSD_E_INVALID_ARG;
  }
}

}  // namespace

int launch_attention_tiles(const FwdArgs &args, __nv_bfloat16 *k_pool, __nv_bfloat16 *v_pool, int sm_count, cudaStream_t s) {
  if (args.fuse_qkv || args.n_splits != 1 || args.n_attn < 1) return HSD_E_INVALID_ARG;
  switch (args.hd) {
    case 128: return launch_attn_tiles_t<128>(args, k_pool, v_pool, sm_count, s);
    case 64: return launch_attn_tiles_t<64>(args, k_pool, v_pool, sm_count, s);
    case 32: return launch_attn_tiles_t<32>(args, k_pool, v_pool, sm_count, s);
    default: return HSD_E_UNSUPPORTED;
  }
}

bool fwd_persist_supported(int hd, int group) {
  return (hd == 32 || hd == 64 || hd == 128) && group >= 1 && group <= 8 && fwd_attn_rows(group, hd) * group <= 32;
}

int launch_forward_persistent(const FwdArgs &args, int npad, int sm_count, cudaStream_t s) {
  if (args.R < 1 || args.R > npad || args.L > npad) return HSD_E_INVALID_ARG;
  if (args.n_run > kMaxLayersSh) return HSD_E_UNSUPPORTED;
  if (((args.d + kTcBlockM - 1) / kTcBlockM) * 2 > sm_count) return HSD_E_UNSUPPORTED;   // norm phase: regular split only
  {  // unit arithmetic on the device is 32-bit
    long long tiles = std::max<long long>((args.V + 127) / 128, (args.ff + 63) / 64);
    long long kb = std::max(args.ff, std::max(args.d, args.nq * args.hd)) / kTcBlockK;
    if (tiles * kb * sm_count >= (1ll << 31)) return HSD_E_UNSUPPORTED;
  }
  if (args.tc_attn && (args.hd != 128 || args.fuse_qkv)) return HSD_E_INVALID_ARG;
  FwdArgs a = args;
  {  // pieces per gate / up tile (the device's split_geom, for a grid of sm_count CTAs)
    const int n_tiles = (a.ff + kTcBoxRows - 1) / kTcBoxRows, KB = a.d / kTcBlockK;
    if (n_tiles * 2 <= sm_count) a.gu_pieces_max = std::min(std::min(4, sm_count / n_tiles), KB);
    else {
      const int U = n_tiles * KB, Gp = std::min(sm_count, U), per = U / Gp;
      a.gu_pieces_max = (KB + per - 1) / per + 1;
    }
    if (a.gu_pieces_max > 4) a.fuse_gu = 0;
  }
  {  // CTAs without a tile of the residual projections (the device's split_geom): enough of them for every row?
    const int n_tiles = (a.d + kTcBlockM - 1) / kTcBlockM;
    int idle = 0;
    if (n_tiles * 2 <= sm_count) idle = sm_count - n_tiles * std::min(4, sm_count / n_tiles);   // >= the device's count of idle CTAs
    a.early_norm = (a.early_norm && a.R <= idle && a.L <= idle) ? 1 : 0;
  }
  switch (a.hd) {
    case 128: return a.tc_attn ? launch_hd<128, true>(a, npad, sm_count, s) : launch_hd<128, false>(a, npad, sm_count, s);
    case 64: return launch_hd<64, false>(a, npad, sm_count, s);
    case 32: return launch_hd<32, false>(a, npad, sm_count, s);
    default: return HSD_E_UNSUPPORTED;
  }
}

}  // namespace hsd
