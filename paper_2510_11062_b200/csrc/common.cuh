// Shared host/device helpers of libatgrpo (status word, workspace carving, launch checks).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "atgrpo.h"

namespace atgrpo {

// First error wins; the word stays set until the caller clears it.
__device__ __forceinline__ void raise_status(int32_t* status, int32_t code) {
  if (status != nullptr) atomicCAS(status, 0, code);
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Sequential carving of one caller-provided workspace into 256-byte aligned pieces.
struct Carver {
  char* base;
  size_t off = 0;
  explicit Carver(void* p) : base(static_cast<char*>(p)) {}
  template <class T> T* take(size_t n) {
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += align_up(n * sizeof(T), 256);
    return p;
  }
};

#define ATGRPO_CUDA_OK(expr)                          \
  do {                                                \
    cudaError_t e__ = (expr);                         \
    if (e__ != cudaSuccess) return ATGRPO_ERR_CUDA;   \
  } while (0)

inline int launch_ok() { return cudaGetLastError() == cudaSuccess ? ATGRPO_OK : ATGRPO_ERR_CUDA; }

}  // namespace atgrpo
