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
constexpr int kScratchBytes = 34 * 1024;               // union: epilogue staging / attention tiles
constexpr int kCtrlBytes = 1024;
constexpr int kSmemTotal = 232448;
constexpr int kKeyTile = 32;

enum { MODE_QKV = 0, MODE_ADD = 1, MODE_SWIGLU = 2, MODE_LOGITS = 3 };

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
__device__ __forceinline__ int unit_owner(int U, int G, int u) {
  int c = (int)(((unsigned)u * (unsigned)G) / (unsigned)U);
  while (c + 1 < G && cta_begin(U, G, c + 1) <= u) ++c;
  while (c > 0 && cta_begin(U, G, c) > u) --c;
  return c;
}
// Work of one CTA in one GEMM, a segment (tile, k-block range) at a time.  One SM can pull only its
// share of HBM bandwidth, so every GEMM is split evenly over all CTAs in (tile, k-block) units;
// each segment's partial sums go to a piece buffer and the next phase adds the pieces of a tile in
// fixed piece order (bit-reproducible; no CTA waits for another inside a GEMM).
struct Seg { int tile, kb0, kb1; };
struct SegIter { int cur, end; };
struct SplitGeom { int U, Gp, pieces_max; };
__device__ __forceinline__ SplitGeom split_geom(const Gemm &g, int G) {
  SplitGeom sg;
  sg.U = g.n_tiles * g.KB;
  sg.Gp = min(G, sg.U);
  const int per = sg.U / sg.Gp;
  sg.pieces_max = (g.KB + per - 1) / per + 1;
  return sg;
}
__device__ __forceinline__ SegIter seg_begin(const Gemm &g, int G, int c) {
  SegIter it;
  const SplitGeom sg = split_geom(g, G);
  it.cur = c < sg.Gp ? cta_begin(sg.U, sg.Gp, c) : 0;
  it.end = c < sg.Gp ? cta_begin(sg.U, sg.Gp, c + 1) : 0;
  return it;
}
__device__ __forceinline__ bool seg_next(const Gemm &g, SegIter &it, Seg &s) {
  if (it.cur >= it.end) return false;
  s.tile = it.cur / g.KB; s.kb0 = it.cur % g.KB;
  s.kb1 = min(g.KB, s.kb0 + (it.end - it.cur));
  it.cur += s.kb1 - s.kb0;
  return true;
}
// Pieces of a tile: they belong to consecutive CTAs first_owner .. first_owner + n - 1.
__device__ __forceinline__ void tile_pieces(const Gemm &g, const SplitGeom &geo, int tile, int &first_owner, int &n) {
  first_owner = unit_owner(geo.U, geo.Gp, tile * g.KB);
  n = unit_owner(geo.U, geo.Gp, tile * g.KB + g.KB - 1) - first_owner + 1;
}
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 2, 256;" ::: "memory"); }
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float bf(const __nv_bfloat16 v) { return __bfloat162float(v); }

// Grid-wide barrier of the worker threads.  `epoch` counts barriers; the counter only grows.
// If ready_bar != 0 the spinning thread then releases the activation producer for the next GEMM.
__device__ __forceinline__ bool grid_barrier(const FwdArgs &a, unsigned &epoch, volatile int *abort_flag, int wt,
                                             uint32_t ready_bar) {
  __threadfence();
  worker_sync();
  ++epoch;
  if (*abort_flag) return false;
  if (wt == 0) {
    const unsigned target = epoch * gridDim.x;
    atomicAdd(a.grid_counter, 1u);
    unsigned long long t0 = globaltimer_ns();
    if (a.prof && 2 * epoch + 1 < (unsigned)kFwdProfEvents) a.prof[(size_t)blockIdx.x * kFwdProfEvents + 2 * epoch] = t0;
    bool ok = true;
    for (uint32_t it = 0; (int)(ld_acquire_u32(a.grid_counter) - target) < 0; ++it) {
      if ((it & 31u) == 31u) {
        if (*abort_flag || *reinterpret_cast<volatile int *>(a.status) != 0 || globaltimer_ns() - t0 > kWaitLimitNs) {
          ok = false;
          break;
        }
      }
    }
    if (!ok) {
      *abort_flag = 1;
      atomicExch(a.status, 1);
    } else {
      if (a.prof && 2 * epoch + 1 < (unsigned)kFwdProfEvents)
        a.prof[(size_t)blockIdx.x * kFwdProfEvents + 2 * epoch + 1] = globaltimer_ns();
      __threadfence();
      if (ready_bar) {
        asm volatile("fence.proxy.async;" ::: "memory");   // generic-proxy writes -> visible to TMA reads
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
template <int NPAD>
__device__ __forceinline__ void norm_phase(const FwdArgs &a, int n_rows, const int *row_list, bool src_embed,
                                           const Gemm *pend, const __nv_bfloat16 *gain, __nv_bfloat16 *dst, float *red,
                                           int wt) {
  constexpr int MAXV = 4;                                  // float4 slots per thread
  constexpr int PB = 8;                                    // pieces loaded at a time per slot
  const int d = a.d, nvec = d >> 2;
  SplitGeom geo;
  geo.U = 1; geo.Gp = 1; geo.pieces_max = 1;
  if (pend) geo = split_geom(*pend, gridDim.x);
  for (int i = blockIdx.x; i < n_rows; i += gridDim.x) {
    const int row = row_list ? row_list[i] : i;
    float *xrow = a.x + (size_t)row * d;
    float4 v[MAXV];
    if (src_embed) {
      const __nv_bfloat16 *erow = a.embed + (size_t)a.tokens[(size_t)a.row_seq[row] * a.max_seq + a.row_pos[row]] * d;
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
#pragma unroll
      for (int j0 = 0; j0 < MAXV; j0 += 2) {               // two slots at a time: all their loads in flight together
        int np[2];
        const float *base[2];
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
          const int iv = wt + 256 * (j0 + jj);
          np[jj] = 0;
          base[jj] = a.pieces;
          if (iv < nvec) {
            const int k = iv << 2, tile = k >> 7, mm = k & 127;
            int fo;
            tile_pieces(*pend, geo, tile, fo, np[jj]);
            base[jj] = a.pieces + ((size_t)tile * geo.pieces_max * NPAD + row) * kTcBlockM + mm;
          }
        }
        for (int p0 = 0; p0 < max(np[0], np[1]); p0 += PB) {
          float4 t[2][PB];
#pragma unroll
          for (int jj = 0; jj < 2; ++jj)
#pragma unroll
            for (int pp = 0; pp < PB; ++pp)
              t[jj][pp] = (p0 + pp < np[jj])
                              ? __ldcg(reinterpret_cast<const float4 *>(base[jj] + (size_t)(p0 + pp) * NPAD * kTcBlockM))
                              : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int jj = 0; jj < 2; ++jj)
#pragma unroll
            for (int pp = 0; pp < PB; ++pp) {
              v[j0 + jj].x += t[jj][pp].x; v[j0 + jj].y += t[jj][pp].y;
              v[j0 + jj].z += t[jj][pp].z; v[j0 + jj].w += t[jj][pp].w;
            }
        }
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
}

// ------------------------------------------------------------------------------ attention phase
// Work item = (attention item, KV head, key split); online softmax per query; the last split of an
// (item, head) to finish merges the partials and writes the attention output.
template <int HD>
__device__ __forceinline__ void attn_phase(const FwdArgs &a, int layer, uint8_t *scratch, volatile int *flag, int wt) {
  constexpr int DPL = HD / 32;
  const int group = a.nq / a.nkv;
  const int warp = wt >> 5, lane = wt & 31;
  float *shQ = reinterpret_cast<float *>(scratch);                                        // [attn_rows*group][HD]
  __nv_bfloat16 *shK = reinterpret_cast<__nv_bfloat16 *>(scratch + 16384);                // [32][HD+2]
  __nv_bfloat16 *shV = shK + kKeyTile * (HD + 2);                                         // [32][HD]
  float *shP = reinterpret_cast<float *>(shV + kKeyTile * HD);                            // [8][32]
  const __nv_bfloat16 *kpool = a.layers[layer].k_pool, *vpool = a.layers[layer].v_pool;
  const float scale = rsqrtf((float)HD);
  const int n_work = a.n_attn * a.nkv * a.n_splits;
  for (int wi = blockIdx.x; wi < n_work; wi += gridDim.x) {
    const int split = wi % a.n_splits, kvh = (wi / a.n_splits) % a.nkv, ai = wi / (a.n_splits * a.nkv);
    const int4 it = a.attn_items[ai];
    const int row0 = it.x, nrows = it.y, seq = it.z, pos0 = it.w;
    const int kv_len = pos0 + nrows;
    const int key_lo = split * a.keys_per_split, key_hi = min(kv_len, key_lo + a.keys_per_split);
    if (key_lo >= kv_len) continue;                              // uniform over the CTA
    const int ns_item = (kv_len + a.keys_per_split - 1) / a.keys_per_split;
    const int nqv = nrows * group;
    worker_sync();
    // (bf16 has no __ldcg overload: read the 16-bit pattern through L2 and widen)
    for (int i = wt; i < nqv * HD; i += 256) {
      int qi = i / HD, dd = i % HD;
      int r = qi / group, g = qi % group;
      unsigned short bits = __ldcg(reinterpret_cast<const unsigned short *>(a.q) + ((size_t)(row0 + r) * a.nq + kvh * group + g) * HD + dd);
      shQ[i] = __uint_as_float((unsigned)bits << 16);
    }
    float m_run[4], l_run[4], o_run[4][DPL];                     // <= 32 queries over 8 warps
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      m_run[i] = -INFINITY; l_run[i] = 0.f;
#pragma unroll
      for (int e = 0; e < DPL; ++e) o_run[i][e] = 0.f;
    }
    for (int kt = key_lo; kt < key_hi; kt += kKeyTile) {
      worker_sync();
      for (int i = wt; i < kKeyTile * (HD / 2); i += 256) {
        int kk = i / (HD / 2), w2 = i % (HD / 2);
        int key = kt + kk;
        unsigned kb2 = 0u, vb2 = 0u;
        if (key < key_hi) {
          int pg = a.page_table[(size_t)seq * a.pages_per_seq + key / a.page];
          size_t off = (((size_t)pg * a.nkv + kvh) * a.page + (key % a.page)) * HD + 2 * w2;
          kb2 = __ldcg(reinterpret_cast<const unsigned *>(kpool + off));
          vb2 = __ldcg(reinterpret_cast<const unsigned *>(vpool + off));
        }
        *reinterpret_cast<unsigned *>(shK + kk * (HD + 2) + 2 * w2) = kb2;
        *reinterpret_cast<unsigned *>(shV + kk * HD + 2 * w2) = vb2;
      }
      worker_sync();
      int qslot = 0;
      for (int qi = warp; qi < nqv; qi += 8, ++qslot) {
        const int qpos = pos0 + qi / group;
        const int key = kt + lane;
        const float *qv = shQ + qi * HD;
        const __nv_bfloat16 *kr = shK + lane * (HD + 2);
        float sc = 0.f;
#pragma unroll 8
        for (int dd = 0; dd < HD; dd += 2) {
          unsigned kk2 = *reinterpret_cast<const unsigned *>(kr + dd);
          sc = fmaf(qv[dd], __uint_as_float(kk2 << 16), sc);
          sc = fmaf(qv[dd + 1], __uint_as_float(kk2 & 0xFFFF0000u), sc);
        }
        sc *= scale;
        if (key >= key_hi || key > qpos) sc = -INFINITY;
        float mx = sc;
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        const float m_new = fmaxf(m_run[qslot], mx);
        float p = 0.f, corr = 1.f;
        if (m_new > -INFINITY) {
          p = __expf(sc - m_new);
          corr = __expf(m_run[qslot] - m_new);
        }
        float ps = p;
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xFFFFFFFFu, ps, o);
        l_run[qslot] = l_run[qslot] * corr + ps;
        m_run[qslot] = m_new;
        shP[warp * kKeyTile + lane] = p;
        __syncwarp();
#pragma unroll
        for (int e = 0; e < DPL; ++e) o_run[qslot][e] *= corr;
        for (int kk = 0; kk < kKeyTile; ++kk) {
          const float pk = shP[warp * kKeyTile + kk];
#pragma unroll
          for (int e = 0; e < DPL; ++e) o_run[qslot][e] = fmaf(pk, bf(shV[kk * HD + lane + 32 * e]), o_run[qslot][e]);
        }
        __syncwarp();
      }
    }
    {
      int qslot = 0;
      for (int qi = warp; qi < nqv; qi += 8, ++qslot) {
        int r = row0 + qi / group, h = kvh * group + qi % group;
        float *dst = a.attn_partials + (((size_t)r * a.nq + h) * a.n_splits + split) * (HD + 2);
#pragma unroll
        for (int e = 0; e < DPL; ++e) dst[lane + 32 * e] = o_run[qslot][e];
        if (lane == 0) { dst[HD] = m_run[qslot]; dst[HD + 1] = l_run[qslot]; }
      }
    }
    __threadfence();
    worker_sync();
    if (wt == 0) {
      int prev = atomicAdd(&a.attn_counters[ai * a.nkv + kvh], 1);
      int last = (prev == ns_item - 1);
      if (last) a.attn_counters[ai * a.nkv + kvh] = 0;
      *flag = last;
      __threadfence();
    }
    worker_sync();
    if (*flag) {
      for (int i = wt; i < nqv * HD; i += 256) {
        int qi = i / HD, dd = i % HD;
        int r = row0 + qi / group, h = kvh * group + qi % group;
        int used = min(ns_item, (pos0 + qi / group) / a.keys_per_split + 1);
        const float *src = a.attn_partials + ((size_t)r * a.nq + h) * a.n_splits * (HD + 2);
        float m = -INFINITY;
        for (int s = 0; s < used; ++s) m = fmaxf(m, __ldcg(src + s * (HD + 2) + HD));
        float l = 0.f, o = 0.f;
        for (int s = 0; s < used; ++s) {
          float ms = __ldcg(src + s * (HD + 2) + HD);
          float w = (ms > -INFINITY) ? __expf(ms - m) : 0.f;
          l += w * __ldcg(src + s * (HD + 2) + HD + 1);
          o += w * __ldcg(src + s * (HD + 2) + dd);
        }
        a.att[((size_t)r * a.nq + h) * HD + dd] = __float2bfloat16_rn(o / l);
      }
    }
  }
}

// ------------------------------------------------------------------------------ epilogue stores
// v[i] = final value of output feature (tile row m) for token row c0 + i.
template <int CH>
__device__ __forceinline__ void final_store(const FwdArgs &a, const Gemm &g, const Tile &ti, int layer, int m, int et,
                                            int c0, const float *v, float *staging) {
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
    epi_sync();
    for (int idx = et; idx < kTcBoxRows * CH; idx += 128) {
      const int cc = idx % kTcBoxRows, i = idx / kTcBoxRows;
      const int r = c0 + i, col = ti.row0 + cc;
      if (r < rows && col < g.seg_n[0]) {
        const float gt = staging[cc * (CH + 1) + i], up = staging[(cc + kTcBoxRows) * (CH + 1) + i];
        a.act[(size_t)r * a.ff + col] = __float2bfloat16_rn(gt / (1.f + __expf(-gt)) * up);
      }
    }
    epi_sync();
  } else {   // MODE_QKV: rotary embedding on q and k, then q -> buffer, k / v -> their cache pages
#pragma unroll
    for (int i = 0; i < CH; ++i) staging[m * (CH + 1) + i] = v[i];
    epi_sync();
    const int n = ti.row0 + m;
    if (n < g.seg_n[ti.seg]) {
      const int hd = a.hd, half = hd >> 1;
      const int dd = n % hd, head = n / hd;
      const int mp = dd < half ? m + half : m - half;
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const int r = c0 + i;
        if (r < rows) {
          const int pos = a.row_pos[r];
          float out = v[i];
          if (ti.seg < 2) {
            const float pv = staging[mp * (CH + 1) + i];
            const float cs = a.cos_tab[(size_t)pos * half + (dd % half)], sn = a.sin_tab[(size_t)pos * half + (dd % half)];
            out = dd < half ? v[i] * cs - pv * sn : v[i] * cs + pv * sn;
          }
          if (ti.seg == 0) {
            a.q[(size_t)r * g.seg_n[0] + n] = __float2bfloat16_rn(out);
          } else {
            const int pg = a.page_table[(size_t)a.row_seq[r] * a.pages_per_seq + pos / a.page];
            const size_t off = (((size_t)pg * a.nkv + head) * a.page + (pos % a.page)) * hd + dd;
            (ti.seg == 1 ? a.layers[layer].k_pool : a.layers[layer].v_pool)[off] = __float2bfloat16_rn(out);
          }
        }
      }
    }
    epi_sync();
  }
}

template <int NPAD, int HD>
__global__ void __launch_bounds__(kFwdThreads, 1) fwd_persistent_kernel(const __grid_constant__ FwdArgs a) {
  using Cfg = PCfg<NPAD>;
  constexpr int STAGES = Cfg::kStages;
  constexpr int CH = Cfg::kChunk;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t *ring = smem;
  uint8_t *scratch = smem + STAGES * Cfg::kStageBytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(scratch + kScratchBytes);
  // bars: full[STAGES] | empty[STAGES] | acc_full[2] | acc_empty[2] | ready[2]
  uint32_t *ctl = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 6);
  uint32_t *tmem_slot = ctl;
  volatile int *abort_flag = reinterpret_cast<volatile int *>(ctl + 1);
  volatile int *last_flag = reinterpret_cast<volatile int *>(ctl + 2);
  volatile int *wait_ok = reinterpret_cast<volatile int *>(ctl + 4);   // [2]
  float *red = reinterpret_cast<float *>(ctl + 8);                      // [8]
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
  auto ready_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 4 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, c = blockIdx.x;
  const int n_phases = 4 * a.n_run + (a.L > 0 ? 1 : 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4); mbar_init(ready_bar(b), 1); }
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) tmem_alloc(smem_u32(tmem_slot), Cfg::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ weight-tile producer (runs ahead)
    if (lane == 0) {
      long long issued = 0;
      bool ok = true;
      for (int p = 0; p < n_phases && ok; ++p) {
        const Gemm g = make_gemm(a, p);
        SegIter it = seg_begin(g, G, c);
        Seg sg;
        while (ok && seg_next(g, it, sg)) {
          const Tile ti = tile_of(g, sg.tile);
          const bool second = (g.mode == MODE_SWIGLU) || (ti.row0 + kTcBoxRows < g.seg_n[ti.seg]);
          for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++issued) {
            const int s = (int)(issued % STAGES);
            const uint32_t ph = (uint32_t)((issued / STAGES) & 1);
            if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t dst = smem_u32(ring + (size_t)s * Cfg::kStageBytes);
            mbar_expect_tx(full_bar(s), (second ? 2 : 1) * kBoxBytes);
            if (g.mode == MODE_SWIGLU) {
              tma_load_2d(dst, g.w[0], kb * kTcBlockK, ti.row0, full_bar(s));
              tma_load_2d(dst + kBoxBytes, g.w[1], kb * kTcBlockK, ti.row0, full_bar(s));
            } else {
              tma_load_2d(dst, g.w[ti.seg], kb * kTcBlockK, ti.row0, full_bar(s));
              if (second) tma_load_2d(dst + kBoxBytes, g.w[ti.seg], kb * kTcBlockK, ti.row0 + kTcBoxRows, full_bar(s));
            }
          }
        }
      }
      if (!ok) {
        atomicExch(a.status, 1);
        long long first = issued > STAGES ? issued - STAGES : 0;     // let copies in flight land (bounded)
        for (long long i = first; i < issued; ++i) {
          unsigned long long t0 = globaltimer_ns();
          while (!mbar_try_wait(full_bar((int)(i % STAGES)), (uint32_t)((i / STAGES) & 1)))
            if (globaltimer_ns() - t0 > kWaitLimitNs / 4) break;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ activation-tile producer
    if (lane == 0) {
      long long issued = 0;
      bool ok = true;
      for (int p = 0; p < n_phases && ok; ++p) {
        const Gemm g = make_gemm(a, p);
        // the operand of phase p is complete once the workers have passed the barrier before it
        if (!mbar_wait(ready_bar(p & 1), (uint32_t)((p >> 1) & 1), abort_flag)) { ok = false; break; }
        SegIter it = seg_begin(g, G, c);
        Seg sg;
        while (ok && seg_next(g, it, sg)) {
          for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++issued) {
            const int s = (int)(issued % STAGES);
            const uint32_t ph = (uint32_t)((issued / STAGES) & 1);
            if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t dst = smem_u32(ring + (size_t)s * Cfg::kStageBytes) + kWBytes;
            mbar_expect_tx(full_bar(s), NPAD * kTcBlockK * 2);
            tma_load_2d(dst, g.amap, kb * kTcBlockK, 0, full_bar(s));
          }
        }
      }
      if (!ok) atomicExch(a.status, 1);
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(NPAD);
      long long consumed = 0;
      int seg_idx = 0;
      bool ok = true;
      for (int p = 0; p < n_phases && ok; ++p) {
        const Gemm g = make_gemm(a, p);
        SegIter it = seg_begin(g, G, c);
        Seg sg;
        for (; ok && seg_next(g, it, sg); ++seg_idx) {
          const int kb0 = sg.kb0, kb1 = sg.kb1;
          const int ab = seg_idx & 1;
          if (!mbar_wait(acce_bar(ab), (uint32_t)(((seg_idx >> 1) & 1) ^ 1), abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(ab * NPAD);
          for (int kb = kb0; kb < kb1; ++kb, ++consumed) {
            const int s = (int)(consumed % STAGES);
            if (!mbar_wait(full_bar(s), (uint32_t)((consumed / STAGES) & 1), abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t wa = smem_u32(ring + (size_t)s * Cfg::kStageBytes);
            const uint64_t da = umma_desc(wa), db = umma_desc(wa + kWBytes);
#pragma unroll
            for (int k = 0; k < kTcBlockK / 16; ++k)
              umma_bf16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
            umma_commit(empty_bar(s));
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
    const int et = wt;                             // 0..127 for the epilogue warps
    const int q = warp & 3, m = q * 32 + lane;
    float *staging = reinterpret_cast<float *>(scratch);
    unsigned epoch = 0;
    int seg_idx = 0;
    bool alive = true;

    // GEMM phase p, epilogue side.  Group-uniform: a give-up is decided by one thread and shared.
    auto epilogue = [&](int p) {
      const Gemm g = make_gemm(a, p);
      const SplitGeom geo = split_geom(g, G);
      SegIter it = seg_begin(g, G, c);
      Seg sg;
      for (; seg_next(g, it, sg); ++seg_idx) {
        const int ab = seg_idx & 1;
        if (et == 0) wait_ok[seg_idx & 1] = mbar_wait(accf_bar(ab), (uint32_t)((seg_idx >> 1) & 1), abort_flag) ? 1 : 0;
        epi_sync();
        if (!wait_ok[seg_idx & 1]) return;
        tc_fence_after();
        const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * NPAD);
        // this CTA's piece of the tile; the next phase sums the pieces
        const int piece = c - unit_owner(geo.U, geo.Gp, sg.tile * g.KB);
        float *mine = a.pieces + ((size_t)sg.tile * geo.pieces_max + piece) * NPAD * kTcBlockM;
#pragma unroll 1
        for (int c0 = 0; c0 < NPAD; c0 += CH) {
          float v[CH];
#pragma unroll
          for (int j = 0; j < CH / 16; ++j) tmem_ld16(tbase + c0 + j * 16, v + j * 16);
          tmem_ld_wait();
          if (c0 + CH >= NPAD) {                   // accumulator fully read: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(ab));
          }
          if (c0 < g.rows) {
#pragma unroll
            for (int i = 0; i < CH; ++i)
              if (c0 + i < g.rows) mine[(c0 + i) * kTcBlockM + m] = v[i];
          }
        }
      }
    };

    // Finish phase of GEMM p (QKV, gate/up, output head): tiles round-robin over the CTAs; the pieces of
    // a tile are added in piece order and the result goes through the projection's own epilogue.
    auto finish = [&](int p) {
      const Gemm g = make_gemm(a, p);
      const SplitGeom geo = split_geom(g, G);
      const int layer = p >> 2;
      for (int tile = c; tile < g.n_tiles; tile += G) {
        const Tile ti = tile_of(g, tile);
        int fo, n_pieces;
        tile_pieces(g, geo, tile, fo, n_pieces);
        const float *base = a.pieces + (size_t)tile * geo.pieces_max * NPAD * kTcBlockM + m;
#pragma unroll 1
        for (int c0 = 0; c0 < NPAD && c0 < g.rows; c0 += CH) {
          float v[CH];
#pragma unroll
          for (int i = 0; i < CH; ++i) v[i] = 0.f;
          for (int pc = 0; pc < n_pieces; ++pc) {
            float t[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i)
              t[i] = (c0 + i < g.rows) ? __ldcg(base + ((size_t)pc * NPAD + c0 + i) * kTcBlockM) : 0.f;
#pragma unroll
            for (int i = 0; i < CH; ++i) v[i] += t[i];
          }
          final_store<CH>(a, g, ti, layer, m, et, c0, v, staging);
        }
      }
    };

    // ---- phase program
    if (a.prof && wt == 0) a.prof[(size_t)blockIdx.x * kFwdProfEvents] = globaltimer_ns();
    norm_phase<NPAD>(a, a.R, nullptr, true, nullptr, a.layers[0].attn_norm, a.h, red, wt);
    alive = grid_barrier(a, epoch, abort_flag, wt, ready_bar(0));
    for (int l = 0; l < a.n_run && alive; ++l) {
      const int p = 4 * l;
      if (is_epi) epilogue(p);                                            // QKV pieces
      alive = grid_barrier(a, epoch, abort_flag, wt, 0);
      if (!alive) break;
      if (is_epi) finish(p);                                              // sum, rope, q / KV append
      alive = grid_barrier(a, epoch, abort_flag, wt, 0);
      if (!alive) break;
      attn_phase<HD>(a, l, scratch, last_flag, wt);
      alive = grid_barrier(a, epoch, abort_flag, wt, ready_bar((p + 1) & 1));
      if (!alive) break;
      if (is_epi) epilogue(p + 1);                                        // O projection into the residual
      alive = grid_barrier(a, epoch, abort_flag, wt, 0);
      if (!alive) break;
      {
        const Gemm pend = make_gemm(a, p + 1);
        norm_phase<NPAD>(a, a.R, nullptr, false, &pend, a.layers[l].mlp_norm, a.h, red, wt);
      }
      alive = grid_barrier(a, epoch, abort_flag, wt, ready_bar((p + 2) & 1));
      if (!alive) break;
      if (is_epi) epilogue(p + 2);                                        // gate / up pieces
      alive = grid_barrier(a, epoch, abort_flag, wt, 0);
      if (!alive) break;
      if (is_epi) finish(p + 2);                                          // sum, SwiGLU
      alive = grid_barrier(a, epoch, abort_flag, wt, ready_bar((p + 3) & 1));
      if (!alive) break;
      if (is_epi) epilogue(p + 3);                                        // down projection into the residual
      if (l + 1 < a.n_run || a.L > 0) {
        alive = grid_barrier(a, epoch, abort_flag, wt, 0);
        if (!alive) break;
        const Gemm pend = make_gemm(a, p + 3);
        if (l + 1 < a.n_run) norm_phase<NPAD>(a, a.R, nullptr, false, &pend, a.layers[l + 1].attn_norm, a.h, red, wt);
        else norm_phase<NPAD>(a, a.L, a.lrow_src, false, &pend, a.final_norm, a.hf, red, wt);
        alive = grid_barrier(a, epoch, abort_flag, wt, ready_bar((p + 4) & 1));
      }
    }
    if (alive && a.L > 0) {                                               // output head
      if (is_epi) epilogue(4 * a.n_run);
      alive = grid_barrier(a, epoch, abort_flag, wt, 0);
      if (alive && is_epi) finish(4 * a.n_run);
    }
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 2) tmem_dealloc(tmem_base, Cfg::kTmemCols);
  if (threadIdx.x == 0 && *abort_flag) atomicExch(a.status, 1);
}

template <int NPAD, int HD>
int launch_t(const FwdArgs &args, int sm_count, cudaStream_t s) {
  using Cfg = PCfg<NPAD>;
  static bool attr_set = false;
  if (!attr_set) {
    HSD_CUDA_OK(cudaFuncSetAttribute(fwd_persistent_kernel<NPAD, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    attr_set = true;
  }
  void *params[1] = {const_cast<FwdArgs *>(&args)};
  HSD_CUDA_OK(cudaLaunchCooperativeKernel((const void *)fwd_persistent_kernel<NPAD, HD>, dim3(sm_count), dim3(kFwdThreads), params,
                                          (size_t)Cfg::kSmemBytes, s));
  hsd_count_launches(1);
  return HSD_OK;
}

template <int HD>
int launch_hd(const FwdArgs &args, int npad, int sm_count, cudaStream_t s) {
  switch (npad) {
    case 16: return launch_t<16, HD>(args, sm_count, s);
    case 32: return launch_t<32, HD>(args, sm_count, s);
    case 64: return launch_t<64, HD>(args, sm_count, s);
    case 128: return launch_t<128, HD>(args, sm_count, s);
    default: return HSD_E_INVALID_ARG;
  }
}

}  // namespace

bool fwd_persist_supported(int hd, int group) {
  return (hd == 32 || hd == 64 || hd == 128) && group >= 1 && group <= 8 && fwd_attn_rows(group, hd) * group <= 32;
}

int launch_forward_persistent(const FwdArgs &args, int npad, int sm_count, cudaStream_t s) {
  if (args.R < 1 || args.R > npad || args.L > npad) return HSD_E_INVALID_ARG;
  {  // unit arithmetic on the device is 32-bit
    long long tiles = std::max<long long>((args.V + 127) / 128, (args.ff + 63) / 64);
    long long kb = std::max(args.ff, std::max(args.d, args.nq * args.hd)) / kTcBlockK;
    if (tiles * kb * sm_count >= (1ll << 31)) return HSD_E_UNSUPPORTED;
  }
  switch (args.hd) {
    case 128: return launch_hd<128>(args, npad, sm_count, s);
    case 64: return launch_hd<64>(args, npad, sm_count, s);
    case 32: return launch_hd<32>(args, npad, sm_count, s);
    default: return HSD_E_UNSUPPORTED;
  }
}

}  // namespace hsd
