// Shared host-side helpers of the treeverify library (error text, argument checks).
#pragma once
#include <cuda_runtime.h>
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "treeverify.h"

namespace tv {

// Per-thread message buffer behind tv_last_error().
char* error_buffer();
int fail(int code, const char* fmt, ...);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#define TV_REQUIRE(cond, ...)                                        \
  do {                                                               \
    if (!(cond)) return ::tv::fail(TV_ERR_INVALID_ARG, __VA_ARGS__); \
  } while (0)

#define TV_CUDA_OK(expr)                                                                   \
  do {                                                                                     \
    cudaError_t e__ = (expr);                                                              \
    if (e__ != cudaSuccess)                                                                \
      return ::tv::fail(TV_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__));            \
  } while (0)

// Process-wide count of kernels this library has launched (diagnostics only).
void count_launches(int n);

constexpr int kFatalStatus = TV_ST_BAD_TREE | TV_ST_BAD_INDEX | TV_ST_CAPACITY | TV_ST_TIMEOUT;

}  // namespace tv
