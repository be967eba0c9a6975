// Weight-streaming skinny GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), operands fed
// by TMA.  out[r, n] = sum_k A[r, k] * W[n, k]: the weight rows sit on the MMA's M side (128 per
// tile), the token rows on its N side (padded to 16..128), so every weight byte is read from HBM
// exactly once per pass whatever the row count.  The k-blocks of all tiles are split evenly over a
// persistent grid (stream-K); tiles cut by a split are finished by whichever CTA arrives last,
// summing the pieces in a fixed order (bit-reproducible, no CTA ever waits for another).
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "forward.cuh"

namespace hsd {

constexpr int kTcBlockM = 128;     // weight rows per tile
constexpr int kTcBlockK = 64;      // bf16 per k-block (one 128-byte swizzle row)
constexpr int kTcBoxRows = 64;     // weight rows per TMA box

// Encoders obtained from the driver at run time (no link-time dependency on libcuda).
int tc_init();                     // HSD_OK when the tensor-map encoder is available
// 2-D bf16 tensor map over a row-major [rows, cols] matrix, box = [box_rows, 64], 128-byte swizzle.
int tc_make_map(CUtensorMap *map, const void *base, long long rows, long long cols, int box_rows);

struct TcGemmPlan {
  int n_tiles, kb, grid, pieces_max;
  size_t scratch_bytes;            // split pieces + per-tile counters
};
// Decomposition for a GEMM with the given segment sizes (mode as in GemmMode), K, row padding.
TcGemmPlan tc_plan(const int *seg_n, int n_segs, int mode, int K, int npad, int sm_count);
int tc_npad(int rows);             // 16, 32, 64 or 128 (rows <= 128)

struct TcGemmArgs {
  CUtensorMap w[3];                // weight maps (box rows 64)
  CUtensorMap a;                   // activation map (box rows = npad), covers the whole buffer
  int seg_n[3], n_segs;
  int K, R, row0;                  // R rows of A starting at buffer row row0
  int mode;                        // GemmMode
  float *out_f32;                  // STORE_F32 / ADD_F32: [.., ldo], written at rows row0..row0+R-1
  __nv_bfloat16 *out_bf16;         // STORE_T_SCATTER: [dst[row], ldo];  SWIGLU_T: [row, ldo]
  const long long *dst;
  int ldo;
  float *pieces;                   // scratch: split pieces
  int *counters;                   // scratch: per-tile arrival counters (zero on entry, zero on exit)
  int *status;                     // device word: set non-zero if a bounded wait gave up
};
int launch_gemm_tc(const TcGemmArgs &args, int sm_count, cudaStream_t s);

}  // namespace hsd
