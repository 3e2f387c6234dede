// Shared host/device helpers of the sp24 library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sp24.h"

namespace sp24 {

__host__ __device__ inline int elem_bytes(sp24_dtype t) {
  switch (t) {
    case SP24_F16:
    case SP24_BF16: return 2;
    case SP24_I8:
    case SP24_E4M3:
    case SP24_E5M2: return 1;
    case SP24_F32:
    case SP24_I32: return 4;
  }
  return 0;
}

inline bool is_fp8(sp24_dtype t) { return t == SP24_E4M3 || t == SP24_E5M2; }
// types of the 2:4 pattern (SP24_F32, the 1:2 pattern, is handled apart)
inline bool is_ab_type(sp24_dtype t) { return t == SP24_F16 || t == SP24_BF16 || t == SP24_I8 || is_fp8(t); }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The current device must be a compute-capability 10.x part; the answer is cached per device.
sp24_status check_arch();

inline sp24_status cuda_status(cudaError_t e) { return e == cudaSuccess ? SP24_OK : SP24_ERR_CUDA; }

#define SP24_RETURN_IF(cond, code) \
  do {                             \
    if (cond) return (code);       \
  } while (0)

#define SP24_CUDA_CHECK(expr)                    \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) return SP24_ERR_CUDA; \
  } while (0)

}  // namespace sp24
