// Shared host/device helpers of the HSD library: status handling, integer types, launch checks.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/hsd.h"

typedef unsigned long long u64;
typedef unsigned int u32;

#define HSD_CUDA_OK(expr)                         \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return HSD_E_CUDA;    \
  } while (0)

// Kernel launches issued by this library (reported by hsd_kernel_launches()).
extern unsigned long long g_hsd_launches;
static inline void hsd_count_launches(int n) { g_hsd_launches += (unsigned long long)n; }

static inline int hsd_launch_status() {
  return cudaGetLastError() == cudaSuccess ? HSD_OK : HSD_E_CUDA;
}

__host__ __device__ static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Stored value -> fp32 (bf16 widens exactly).
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
