// Shared host/device helpers of the TurboBoA CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "turboboa.h"

// A failed runtime call leaves its code in the runtime's last-error slot; it is cleared here so
// that the next, unrelated launch check does not report it again.
#define TB_CUDA_CHECK(expr)                      \
  do {                                           \
    cudaError_t tb_e_ = (expr);                  \
    if (tb_e_ != cudaSuccess) {                  \
      (void)cudaGetLastError();                  \
      return TB_ERR_CUDA;                        \
    }                                            \
  } while (0)

// Follows every kernel launch of the library (one check per launch); also counts them.
#define TB_LAUNCH_CHECK()                                   \
  do {                                                      \
    ++tb::g_launch_count;                                   \
    if (cudaGetLastError() != cudaSuccess) return TB_ERR_CUDA; \
  } while (0)

#define TB_TRY(expr)                   \
  do {                                 \
    tb_status tb_s_ = (expr);          \
    if (tb_s_ != TB_OK) return tb_s_;  \
  } while (0)

namespace tb {

extern unsigned long long g_launch_count;  // kernels launched by the library in this process (tb_api.cu)

// Bump allocator over a caller-provided workspace.  With base == nullptr it
// only measures (used by the *_workspace queries), so sizes and carving can
// never disagree.
struct Bump {
  char* base;
  size_t off;
  explicit Bump(void* b) : base(static_cast<char*>(b)), off(0) {}
  template <typename T>
  T* take(size_t n) {
    off = (off + 255) & ~static_cast<size_t>(255);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
  size_t total() const { return (off + 255) & ~static_cast<size_t>(255); }
};

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

template <typename TO, typename TI>
__device__ __forceinline__ TO cvt(TI v) {
  return static_cast<TO>(v);
}
template <>
__device__ __forceinline__ float cvt<float, __nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}
template <>
__device__ __forceinline__ double cvt<double, __nv_bfloat16>(__nv_bfloat16 v) {
  return static_cast<double>(__bfloat162float(v));
}

template <typename T>
__device__ __forceinline__ T zero_of() {
  return T(0);
}
template <>
__device__ __forceinline__ __nv_bfloat16 zero_of<__nv_bfloat16>() {
  return __float2bfloat16(0.0f);
}

__device__ __forceinline__ double shfl_d(double v, int src) {
  return __shfl_sync(0xffffffffu, v, src);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Round to nearest integer, ties to even, for |x| < 2^51 (two full-rate adds).
__device__ __forceinline__ double rne(double x) {
  const double magic = 6755399441055744.0;  // 1.5 * 2^52
  return __dadd_rn(__dadd_rn(x, magic), -magic);
}

}  // namespace tb
