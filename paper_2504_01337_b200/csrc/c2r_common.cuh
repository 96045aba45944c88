// Shared host/device helpers of the C2R library (internal; the public surface is include/c2r.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "c2r.h"

namespace c2r {

extern thread_local int g_last_cuda_error;
extern unsigned long long g_launch_count;  // kernels launched by this library in this process

inline int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return C2R_ERR_CUDA;
}

#define C2R_CUDA(expr)                                  \
  do {                                                  \
    cudaError_t _e = (expr);                            \
    if (_e != cudaSuccess) return ::c2r::cuda_fail(_e); \
  } while (0)

#define C2R_LAUNCH_CHECK()                                        \
  do {                                                            \
    __atomic_fetch_add(&::c2r::g_launch_count, 1ull, __ATOMIC_RELAXED); \
    C2R_CUDA(cudaGetLastError());                                 \
  } while (0)

#define C2R_REQUIRE(cond, code) \
  do {                          \
    if (!(cond)) return (code); \
  } while (0)

inline int check_config(const c2r_config* c) {
  if (!c) return C2R_ERR_INVALID_ARG;
  if (c->dtype != C2R_F32 && c->dtype != C2R_BF16) return C2R_ERR_INVALID_ARG;
  if (c->N < 0 || c->d <= 0 || c->E <= 0 || c->K <= 0 || c->row_align < 1) return C2R_ERR_INVALID_ARG;
  if (c->K > 8 || c->K > c->E) return C2R_ERR_UNSUPPORTED_SHAPE;
  if (c->E > 64 || (c->I_s > 0 && c->E > 63)) return C2R_ERR_UNSUPPORTED_SHAPE;
  if (c->d % 8 != 0) return C2R_ERR_UNSUPPORTED_SHAPE;
  if (c->I < 0 || c->I % 16 != 0 || c->I_s < 0 || c->I_s % 16 != 0) return C2R_ERR_UNSUPPORTED_SHAPE;
  if ((int64_t)c->N * c->K >= (1ll << 30)) return C2R_ERR_UNSUPPORTED_SHAPE;
  return C2R_OK;
}

inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

inline int64_t permuted_rows(const c2r_config* c) {
  return round_up((int64_t)c->N * c->K + (int64_t)c->E * (c->row_align - 1), c->row_align);
}

// Tokens owned by one block of the dispatch's counting sort: the largest count that keeps a block at no
// more than 512 slots and a whole number of 32-slot groups (K = 1, 2, 4, 8: exactly 512 slots).
__host__ __device__ inline int perm_tokens_per_block(int K) {
  const int m = 32 / (K & -K);  // tokens per whole number of 32-slot groups (K <= 8)
  return (512 / K) / m * m;
}

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// ---- device helpers -------------------------------------------------------------------------

template <typename T>
struct Vec16;  // 16-byte vector of T
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  float4 v;
  __device__ void load(const float* p) { v = *reinterpret_cast<const float4*>(p); }
  __device__ void store(float* p) const { *reinterpret_cast<float4*>(p) = v; }
  __device__ void to_float(float* f) const { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
  __device__ void from_float(const float* f) { v = make_float4(f[0], f[1], f[2], f[3]); }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  uint4 v;
  __device__ void load(const __nv_bfloat16* p) { v = *reinterpret_cast<const uint4*>(p); }
  __device__ void store(__nv_bfloat16* p) const { *reinterpret_cast<uint4*>(p) = v; }
  __device__ void to_float(float* f) const {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(u[i] << 16);
      f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
    }
  }
  __device__ void from_float(const float* f) {
    uint32_t u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      u[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    v = make_uint4(u[0], u[1], u[2], u[3]);
  }
};

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }


}  // namespace c2r
