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

#ifdef __CUDACC__
// Programmatic dependent launch for the small kernels of a step.  Launched with programmatic stream
// serialisation, such a kernel first waits for everything in front of it in the stream and only then lets the
// next kernel be scheduled: the next launch overlaps this kernel's body, and no kernel ever runs ahead of data
// it reads (a kernel that reads inputs before its own wait, as tree_verify_attn does with the committed
// prefix, can therefore only overtake the body of the kernel directly in front of it).
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
// For a kernel that writes something a later kernel reads BEFORE that kernel's own wait (prefix_len, which
// tree_verify_attn reads at once): wait for everything in front, and never release the next launch early - it is
// released when this grid has completed and its writes are visible.
__device__ __forceinline__ void pdl_wait_only() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Process-wide count of kernels this library has launched (diagnostics only).
void count_launches(int n);

constexpr int kFatalStatus = TV_ST_BAD_TREE | TV_ST_BAD_INDEX | TV_ST_CAPACITY | TV_ST_TIMEOUT;

}  // namespace tv
