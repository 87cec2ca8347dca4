// Shared host/device helpers of the GRASS B200 library (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "grass.h"

namespace grass {

// Status word layout on the device: [0] first error code, [1] detail.
// Kernels record with record_status(); the first error wins.
__device__ __forceinline__ void record_status(int* status, int code, int detail) {
  if (atomicCAS(&status[0], 0, code) == 0) status[1] = detail;
}

// Device address of the current device's status word (host function, common.cu).
int* status_word(cudaError_t* err);

// Brackets one kernel launch with events while a profile is active (common.cu).
void profile_mark_begin(int kernel_id, cudaStream_t s);
void profile_mark_end(cudaStream_t s);
struct ProfileScope {
  cudaStream_t s;
  ProfileScope(int kernel_id, cudaStream_t stream) : s(stream) { profile_mark_begin(kernel_id, s); }
  ~ProfileScope() { profile_mark_end(s); }
};

#define GRASS_CUDA_TRY(expr)                                                             \
  do {                                                                                   \
    cudaError_t e__ = (expr);                                                            \
    if (e__ != cudaSuccess) {                                                            \
      fprintf(stderr, "grass: %s failed: %s (%s:%d)\n", #expr, cudaGetErrorString(e__),  \
              __FILE__, __LINE__);                                                       \
      return GRASS_ERR_CUDA;                                                             \
    }                                                                                    \
  } while (0)

#define GRASS_LAUNCH_CHECK() GRASS_CUDA_TRY(cudaGetLastError())

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace grass
