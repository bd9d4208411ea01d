// Shared device helpers for the BSR kernels (storage-type packs, warp reductions, status word).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bsr {

typedef __nv_bfloat16 bf16;

// Device status word bits (read and cleared by bsr_sync_status).
enum : int { STATUS_TIMEOUT = 1, STATUS_NONFINITE = 2, STATUS_GUARD = 4, STATUS_CHECK = 8 };

// Index checks of the checked build (-DBSR_DEBUG): a failed check raises STATUS_CHECK in the status word (never a trap:
// the context stays usable) and the caller of the macro skips the access.  In the normal build the condition is not
// evaluated.
#ifdef BSR_DEBUG
#define BSR_CHECK(cond, status) ((cond) ? true : (((status) != nullptr ? (void)atomicOr((status), bsr::STATUS_CHECK) : (void)0), false))
#else
#define BSR_CHECK(cond, status) (true)
#endif

template <typename T> struct Pack;          // 16-byte vector of storage elements
template <> struct Pack<float> { static constexpr int N = 4; };
template <> struct Pack<bf16> { static constexpr int N = 8; };

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// 16-byte aligned load/store of Pack<T>::N consecutive elements, widened to float.
__device__ __forceinline__ void load16(const float* p, float* f) {
  float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
__device__ __forceinline__ void load16(const bf16* p, float* f) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x; f[2 * i + 1] = t.y;
  }
}
__device__ __forceinline__ void store16(float* p, const float* f) {
  *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
__device__ __forceinline__ void store16(bf16* p, const float* f) {
  uint4 v;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  *reinterpret_cast<uint4*>(p) = v;
}

// four consecutive elements (16 bytes of float, 8 bytes of bf16)
__device__ __forceinline__ void load4(const float* p, float* f) { load16(p, f); }
__device__ __forceinline__ void load4(const bf16* p, float* f) {
  uint2 v = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
  float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
  f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}
__device__ __forceinline__ void store4(float* p, const float* f) { store16(p, f); }
__device__ __forceinline__ void store4(bf16* p, const float* f) {
  uint2 v;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
  h[0] = __floats2bfloat162_rn(f[0], f[1]);
  h[1] = __floats2bfloat162_rn(f[2], f[3]);
  *reinterpret_cast<uint2*>(p) = v;
}

// N consecutive elements (N = 4 or 8) through 16-byte accesses, whatever the element type.
template <int N> __device__ __forceinline__ void load_n(const float* p, float* f) {
#pragma unroll
  for (int j = 0; j < N; j += 4) load16(p + j, f + j);
}
template <int N> __device__ __forceinline__ void load_n(const bf16* p, float* f) {
  static_assert(N == 8, "bf16 packs hold 8 elements");
  load16(p, f);
}
template <int N> __device__ __forceinline__ void store_n(float* p, const float* f) {
#pragma unroll
  for (int j = 0; j < N; j += 4) store16(p + j, f + j);
}
template <int N> __device__ __forceinline__ void store_n(bf16* p, const float* f) {
  static_assert(N == 8, "bf16 packs hold 8 elements");
  store16(p, f);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Exact GELU x * Phi(x) and its derivative Phi(x) + x * phi(x).
__device__ __forceinline__ float gelu_f(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_grad_f(float x) {
  return 0.5f * (1.0f + erff(x * 0.70710678118654752f)) + x * 0.39894228040143268f * expf(-0.5f * x * x);
}

// Host-side count of kernel launches made by this library (read through bsr_profile_read).
extern long g_kernel_launches;
static inline void note_launch(int n = 1) { g_kernel_launches += n; }

// The dynamic shared-memory limit of a kernel is an attribute of the (kernel, device) pair, so the largest value set so
// far is remembered per device ordinal.  It only grows: launches captured earlier in a graph keep working.
struct SmemLimit {
  size_t set[64] = {};
};
template <typename Kernel>
static inline bool ensure_smem(SmemLimit& lim, Kernel kern, size_t bytes) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  if (bytes > lim.set[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
    lim.set[dev] = bytes;
  }
  return true;
}

static inline int ceil_div(long a, long b) { return (int)((a + b - 1) / b); }

}  // namespace bsr
