// tcgen05 / TMEM / TMA weight-streaming GEMM (see gemm_tc.cuh).
//
// One CTA per SM, 192 threads: warp 0 = TMA producer (one lane), warp 1 = TMEM owner + MMA issuer
// (one lane), warps 2..5 = epilogue (each reads its own 32-lane quarter of TMEM).  Shared-memory
// ring of STAGES x (128x64 weight tile + NPADx64 activation tile), both K-major with the 128-byte
// swizzle TMA writes and the UMMA descriptors read.  Two TMEM accumulators so the epilogue of one
// tile overlaps the MMAs of the next.  Every wait is bounded by wall time; a wait that gives up
// raises a flag, every role leaves its loop, TMEM is freed and a status word tells the host.
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace hsd {
namespace {

using namespace ptx;

constexpr int kThreads = 192;
constexpr int kStageWBytes = kTcBlockM * kTcBlockK * 2;       // 16 KiB
constexpr int kBoxBytes = kTcBoxRows * kTcBlockK * 2;         // 8 KiB
constexpr int kSmemBudget = 232448 - 1024;                    // 227 KiB minus alignment slack

template <int NPAD> struct TcCfg {
  static constexpr int kStageBytes = kStageWBytes + NPAD * kTcBlockK * 2;
  static constexpr int kChunk = NPAD < 32 ? NPAD : 32;        // accumulator columns (token rows) the epilogue handles at a time
  static constexpr int kStagingBytes = kTcBlockM * (kChunk + 1) * 4;
  static constexpr int kCtrlBytes = 1024;
  static constexpr int kStages = (kSmemBudget - kCtrlBytes - kStagingBytes) / kStageBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + kCtrlBytes + 1024;
  static constexpr int kTmemCols = (2 * NPAD < 32) ? 32 : 2 * NPAD;
};

struct TileInfo { int seg, row0, col0; };
__device__ __forceinline__ TileInfo tile_info(const TcGemmArgs &a, int tile) {
  TileInfo ti;
  if (a.mode == GEMM_SWIGLU_T) { ti.seg = 0; ti.row0 = tile * kTcBoxRows; ti.col0 = 0; return ti; }
  int t = tile, col0 = 0;
  for (int s = 0; s < a.n_segs; ++s) {
    int nt = (a.seg_n[s] + kTcBlockM - 1) / kTcBlockM;
    if (t < nt || s == a.n_segs - 1) { ti.seg = s; ti.row0 = t * kTcBlockM; ti.col0 = col0; return ti; }
    t -= nt;
    col0 += a.seg_n[s];
  }
  ti.seg = 0; ti.row0 = 0; ti.col0 = 0;
  return ti;
}
__device__ __forceinline__ long long cta_begin(long long U, int G, int c) { return (U * c) / G; }
__device__ __forceinline__ int unit_owner(long long U, int G, long long u) {
  int c = (int)((u * G) / U);
  while (c + 1 < G && cta_begin(U, G, c + 1) <= u) ++c;
  while (c > 0 && cta_begin(U, G, c) > u) --c;
  return c;
}

template <int NPAD, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ TcGemmArgs args, int n_tiles, int KB, int pieces_max) {
  using Cfg = TcCfg<NPAD>;
  constexpr int STAGES = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t *ring = smem;
  float *staging = reinterpret_cast<float *>(smem + STAGES * Cfg::kStageBytes);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * Cfg::kStageBytes + Cfg::kStagingBytes);
  // bars: full[STAGES] | empty[STAGES] | acc_full[2] | acc_empty[2]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  volatile int *last_flag = reinterpret_cast<volatile int *>(tmem_slot + 2);
  volatile int *wait_ok = reinterpret_cast<volatile int *>(tmem_slot + 4);      // [2], alternating per tile
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x, c = blockIdx.x;
  const long long U = (long long)n_tiles * KB;
  const long long u0 = cta_begin(U, G, c), u1 = cta_begin(U, G, c + 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), 4); }
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(Cfg::kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      long long issued = 0;
      bool ok = true;
      for (long long u = u0; u < u1 && ok;) {
        const int tile = (int)(u / KB), kb0 = (int)(u % KB);
        const int kb1 = (int)min((long long)KB, kb0 + (u1 - u));
        const TileInfo ti = tile_info(args, tile);
        const bool second = (MODE == GEMM_SWIGLU_T) || (ti.row0 + kTcBoxRows < args.seg_n[ti.seg]);
        const uint32_t bytes = (second ? 2 : 1) * kBoxBytes + NPAD * kTcBlockK * 2;
        for (int kb = kb0; kb < kb1; ++kb, ++issued) {
          const int s = (int)(issued % STAGES);
          const uint32_t ph = (uint32_t)((issued / STAGES) & 1);
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = smem_u32(ring + (size_t)s * Cfg::kStageBytes);
          mbar_expect_tx(full_bar(s), bytes);
          if (MODE == GEMM_SWIGLU_T) {
            tma_load_2d(dst, &args.w[0], kb * kTcBlockK, ti.row0, full_bar(s));
            tma_load_2d(dst + kBoxBytes, &args.w[1], kb * kTcBlockK, ti.row0, full_bar(s));
          } else {
            tma_load_2d(dst, &args.w[ti.seg], kb * kTcBlockK, ti.row0, full_bar(s));
            if (second) tma_load_2d(dst + kBoxBytes, &args.w[ti.seg], kb * kTcBlockK, ti.row0 + kTcBoxRows, full_bar(s));
          }
          tma_load_2d(dst + kStageWBytes, &args.a, kb * kTcBlockK, args.row0, full_bar(s));
        }
        u += kb1 - kb0;
      }
      if (!ok) {
        // wait (bounded) for the copies still in flight before the CTA's shared memory goes away
        long long first = issued > STAGES ? issued - STAGES : 0;
        for (long long i = first; i < issued; ++i) {
          unsigned long long t0 = globaltimer_ns();
          while (!mbar_try_wait(full_bar((int)(i % STAGES)), (uint32_t)((i / STAGES) & 1)))
            if (globaltimer_ns() - t0 > kWaitLimitNs) break;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NPAD >> 3) << 17) | ((uint32_t)(kTcBlockM >> 4) << 24);
      long long consumed = 0;
      int seg_idx = 0;
      bool ok = true;
      for (long long u = u0; u < u1 && ok; ++seg_idx) {
        const int kb0 = (int)(u % KB);
        const int kb1 = (int)min((long long)KB, kb0 + (u1 - u));
        const int ab = seg_idx & 1;
        const uint32_t aph = (uint32_t)((seg_idx >> 1) & 1);
        if (!mbar_wait(acce_bar(ab), aph ^ 1u, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)(ab * NPAD);
        for (int kb = kb0; kb < kb1; ++kb, ++consumed) {
          const int s = (int)(consumed % STAGES);
          const uint32_t ph = (uint32_t)((consumed / STAGES) & 1);
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t wa = smem_u32(ring + (size_t)s * Cfg::kStageBytes);
          const uint64_t da = umma_desc(wa), db = umma_desc(wa + kStageWBytes);
#pragma unroll
          for (int k = 0; k < kTcBlockK / 16; ++k)
            umma_bf16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          umma_commit(empty_bar(s));            // the stage is free once these MMAs have read it
        }
        if (ok) umma_commit(accf_bar(ab));      // accumulator complete
        u += kb1 - kb0;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                     // TMEM lane quarter this warp may read
    const int m = q * 32 + lane;                // row of the tile held by this thread
    const int et = threadIdx.x - 64;            // 0..127 among the epilogue threads
    int seg_idx = 0;
    bool ok = true;
    for (long long u = u0; u < u1 && ok; ++seg_idx) {
      const int tile = (int)(u / KB), kb0 = (int)(u % KB);
      const int kb1 = (int)min((long long)KB, kb0 + (u1 - u));
      const int ab = seg_idx & 1;
      const uint32_t aph = (uint32_t)((seg_idx >> 1) & 1);
      // one thread waits, all 128 take the same decision (a bail-out must not split the group)
      if (et == 0) wait_ok[seg_idx & 1] = mbar_wait(accf_bar(ab), aph, abort_flag) ? 1 : 0;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (!wait_ok[seg_idx & 1]) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      constexpr int CH = Cfg::kChunk;
      const TileInfo ti = tile_info(args, tile);
      const bool whole = (kb0 == 0 && kb1 == KB);
      const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * NPAD);
      int n_pieces = 1, piece = 0;
      if (!whole) {
        const int first_owner = unit_owner(U, G, (long long)tile * KB);
        const int last_owner = unit_owner(U, G, (long long)tile * KB + KB - 1);
        n_pieces = last_owner - first_owner + 1;
        piece = c - first_owner;
      }
      // values of the tile's row m for token rows c0 .. c0 + CH - 1 -> the projection's output
      auto finish_chunk = [&](int c0, float *v) {
        if (MODE == GEMM_SWIGLU_T) {
#pragma unroll
          for (int r = 0; r < CH; ++r) staging[m * (CH + 1) + r] = v[r];
          asm volatile("bar.sync 1, 128;" ::: "memory");
          for (int i = et; i < kTcBoxRows * CH; i += 128) {
            const int cc = i % kTcBoxRows, r = c0 + i / kTcBoxRows;
            const int col = ti.row0 + cc;
            if (r < args.R && col < args.seg_n[0]) {
              const float g = staging[cc * (CH + 1) + (r - c0)], up = staging[(cc + kTcBoxRows) * (CH + 1) + (r - c0)];
              args.out_bf16[(size_t)(args.row0 + r) * args.ldo + col] = __float2bfloat16_rn(ptx::silu_mul(g, up));
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
        } else {
          const int n = ti.row0 + m;
          if (n < args.seg_n[ti.seg]) {
            const int col = ti.col0 + n;
            if (MODE == GEMM_ADD_F32) {
              // residual add: all of the chunk's old values are fetched before the first store (a read-modify-write
              // per row would be one dependent round trip per row)
              float old[CH];
#pragma unroll
              for (int i = 0; i < CH; ++i)
                old[i] = c0 + i < args.R ? __ldcg(args.out_f32 + (size_t)(args.row0 + c0 + i) * args.ldo + col) : 0.f;
#pragma unroll
              for (int i = 0; i < CH; ++i)
                if (c0 + i < args.R) args.out_f32[(size_t)(args.row0 + c0 + i) * args.ldo + col] = old[i] + v[i];
            } else {
#pragma unroll
              for (int i = 0; i < CH; ++i) {
                const int r = c0 + i;
                if (r < args.R) {
                  if (MODE == GEMM_STORE_F32) args.out_f32[(size_t)(args.row0 + r) * args.ldo + col] = v[i];
                  else args.out_bf16[(size_t)args.dst[args.row0 + r] * args.ldo + col] = __float2bfloat16_rn(v[i]);
                }
              }
            }
          }
        }
      };
      float *mine = args.pieces + ((size_t)tile * pieces_max + piece) * NPAD * kTcBlockM;
#pragma unroll 1
      for (int c0 = 0; c0 < NPAD; c0 += CH) {
        float v[CH];
#pragma unroll
        for (int j = 0; j < CH / 16; ++j) tmem_ld16(tbase + (uint32_t)(c0 + j * 16), v + j * 16);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (c0 + CH >= NPAD) {                     // accumulator fully read: hand it back to the MMA warp
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(acce_bar(ab));
        }
        if (c0 >= args.R) continue;                // padding rows: nothing to write
        if (whole) finish_chunk(c0, v);
        else {
#pragma unroll
          for (int i = 0; i < CH; ++i) mine[(c0 + i) * kTcBlockM + m] = v[i];
        }
      }
      if (!whole) {
        // split tile: this piece is published; the last arriver sums all pieces in piece order
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0) {
          int prev = atomicAdd(&args.counters[tile], 1);
          int last = (prev == n_pieces - 1);
          if (last) args.counters[tile] = 0;
          *last_flag = last;
          __threadfence();
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const bool finish = (*last_flag != 0);
        asm volatile("bar.sync 1, 128;" ::: "memory");   // last_flag may be rewritten by the next tile
        if (finish) {
#pragma unroll 1
          for (int c0 = 0; c0 < NPAD && c0 < args.R; c0 += CH) {
            float v[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i) v[i] = 0.f;
            for (int p = 0; p < n_pieces; ++p) {
              const float *src = args.pieces + ((size_t)tile * pieces_max + p) * NPAD * kTcBlockM;
#pragma unroll
              for (int i = 0; i < CH; ++i) v[i] += __ldcg(src + (c0 + i) * kTcBlockM + m);
            }
            finish_chunk(c0, v);
          }
        }
      }
      u += kb1 - kb0;
    }
  }
  // ------------------------------------------------------------------ teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::kTmemCols));
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(args.status, 1);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

template <int NPAD, int MODE>
int launch_t(const TcGemmArgs &args, const TcGemmPlan &plan, cudaStream_t s) {
  using Cfg = TcCfg<NPAD>;
  static bool attr_set = false;
  if (!attr_set) {
    HSD_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<NPAD, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    attr_set = true;
  }
  gemm_tc_kernel<NPAD, MODE><<<plan.grid, kThreads, Cfg::kSmemBytes, s>>>(args, plan.n_tiles, plan.kb, plan.pieces_max);
  hsd_count_launches(1);
  return hsd_launch_status();
}

template <int NPAD>
int launch_mode(const TcGemmArgs &args, const TcGemmPlan &plan, cudaStream_t s) {
  switch (args.mode) {
    case GEMM_STORE_F32: return launch_t<NPAD, GEMM_STORE_F32>(args, plan, s);
    case GEMM_ADD_F32: return launch_t<NPAD, GEMM_ADD_F32>(args, plan, s);
    case GEMM_STORE_T_SCATTER: return launch_t<NPAD, GEMM_STORE_T_SCATTER>(args, plan, s);
    case GEMM_SWIGLU_T: return launch_t<NPAD, GEMM_SWIGLU_T>(args, plan, s);
    default: return HSD_E_INVALID_ARG;
  }
}

}  // namespace

int tc_init() {
  if (g_encode) return HSD_OK;
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return HSD_E_UNSUPPORTED;
  g_encode = (EncodeTiledFn)fn;
  return HSD_OK;
}

int tc_make_map(CUtensorMap *map, const void *base, long long rows, long long cols, int box_rows) {
  if (!g_encode) return HSD_E_UNSUPPORTED;
  if (((uintptr_t)base & 15) != 0 || (cols * 2) % 16 != 0 || box_rows < 1 || box_rows > 256) return HSD_E_INVALID_ARG;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kTcBlockK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? HSD_OK : HSD_E_CUDA;
}

int tc_npad(int rows) { return rows <= 16 ? 16 : rows <= 32 ? 32 : rows <= 64 ? 64 : rows <= 128 ? 128 : 256; }

TcGemmPlan tc_plan(const int *seg_n, int n_segs, int mode, int K, int npad, int sm_count) {
  TcGemmPlan p;
  p.kb = K / kTcBlockK;
  p.n_tiles = 0;
  if (mode == GEMM_SWIGLU_T) p.n_tiles = (seg_n[0] + kTcBoxRows - 1) / kTcBoxRows;
  else
    for (int s = 0; s < n_segs; ++s) p.n_tiles += (seg_n[s] + kTcBlockM - 1) / kTcBlockM;
  long long U = (long long)p.n_tiles * p.kb;
  p.grid = (int)std::min<long long>(sm_count, U);
  long long per = U / p.grid;                     // every CTA gets at least this many k-blocks
  p.pieces_max = (int)((p.kb + per - 1) / per) + 1;
  p.scratch_bytes = (size_t)p.n_tiles * p.pieces_max * npad * kTcBlockM * 4 + (size_t)p.n_tiles * 4 + 256;
  return p;
}

int launch_gemm_tc(const TcGemmArgs &args, int sm_count, cudaStream_t s) {
  if (args.R < 1 || args.R > 256 || args.K % kTcBlockK != 0) return HSD_E_UNSUPPORTED;
  const int npad = tc_npad(args.R);
  TcGemmPlan plan = tc_plan(args.seg_n, args.n_segs, args.mode, args.K, npad, sm_count);
  switch (npad) {
    case 16: return launch_mode<16>(args, plan, s);
    case 32: return launch_mode<32>(args, plan, s);
    case 64: return launch_mode<64>(args, plan, s);
    case 128: return launch_mode<128>(args, plan, s);
    default: return launch_mode<256>(args, plan, s);
  }
}

}  // namespace hsd
