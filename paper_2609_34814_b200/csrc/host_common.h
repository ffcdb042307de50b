// Host-side helpers shared by the entry points: thread-local error text and launch counter.
#pragma once
#include <cstdarg>
#include <cstdio>
#include <cuda_runtime.h>
#include "waveal.h"

namespace waveal {

char* last_error_buffer();          // thread-local, 512 bytes
int32_t& launch_counter();          // thread-local

inline waveal_status fail(waveal_status s, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(last_error_buffer(), 512, fmt, ap);
  va_end(ap);
  return s;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

#define WAVEAL_CUDA_OK(expr)                                                                 \
  do {                                                                                       \
    cudaError_t e__ = (expr);                                                                \
    if (e__ != cudaSuccess)                                                                  \
      return ::waveal::fail(WAVEAL_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

}  // namespace waveal
