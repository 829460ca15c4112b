// Host-side helpers shared by the C-ABI entry points: status codes, argument checks,
// last-error bookkeeping.  No device code.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/mpfa.h"

namespace mpfa {

constexpr int HEAD_DIM = 128;
constexpr int TILE = 128;        // tokens per quantization / attention tile
constexpr int PAGE = 64;         // tokens per KV-cache page
constexpr int DECODE_SPLIT = 1024;  // tokens per decode partition (8 x 128, Section 5.3)

extern thread_local int g_last_cuda_error;

inline int pad128(int n) { return (n + TILE - 1) / TILE * TILE; }
inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline mpfa_status cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return MPFA_ERR_CUDA;
}

#define MPFA_CUDA_OK(expr)                                    \
  do {                                                        \
    cudaError_t _e = (expr);                                  \
    if (_e != cudaSuccess) return ::mpfa::cuda_fail(_e);      \
  } while (0)

#define MPFA_LAUNCH_OK()                                      \
  do {                                                        \
    cudaError_t _e = cudaGetLastError();                      \
    if (_e != cudaSuccess) return ::mpfa::cuda_fail(_e);      \
  } while (0)

// The kernels use sm_100a-only instructions; refuse other devices up front.
mpfa_status check_arch();

}  // namespace mpfa
