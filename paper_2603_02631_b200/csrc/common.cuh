// Shared host/device helpers of the library: error reporting, small device utilities.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdarg>
#include <cstdio>

#include "spf.h"

namespace spf {

// Records the calling thread's failure text and returns `code` (so call sites can `return fail(...)`).
int32_t fail(int32_t code, const char* fmt, ...);
void clear_error();

#define SPF_CUDA_CHECK(expr)                                                                      \
  do {                                                                                            \
    cudaError_t err__ = (expr);                                                                   \
    if (err__ != cudaSuccess)                                                                     \
      return ::spf::fail(SPF_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(err__));       \
  } while (0)

constexpr int kMaxLayers = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Device pointers of the per-layer key caches, passed to kernels by value.
struct LayerPtrs {
  const __nv_bfloat16* p[kMaxLayers];
};

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float fast_log2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace spf
