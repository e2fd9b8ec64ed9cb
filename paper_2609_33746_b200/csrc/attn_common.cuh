// Helpers shared by the attention kernels: fp16/bf16 unpacking and online-softmax state.
#pragma once

#include "common.cuh"

namespace pqhsa {
namespace {

template <typename T> struct Unpack;
template <> struct Unpack<__nv_bfloat16> {
  static __device__ __forceinline__ void run(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ float one(const __nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ __forceinline__ __nv_bfloat16 pack(float v) { return __float2bfloat16_rn(v); }
};
template <> struct Unpack<__half> {
  static __device__ __forceinline__ void run(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      f[2 * i] = p.x;
      f[2 * i + 1] = p.y;
    }
  }
  static __device__ __forceinline__ float one(const __half v) { return __half2float(v); }
  static __device__ __forceinline__ __half pack(float v) { return __float2half_rn(v); }
};

// Online-softmax state of a lane group: running max m (log2 units), normaliser Z and the 16
// output dims the lane owns.
struct GroupState {
  float m, Z;
  float acc[16];
};

__device__ __forceinline__ float safe_scale(float m_from, float m_to, float Z) {
  return Z > 0.f ? fast_exp2(m_from - m_to) : 0.f;
}

}  // namespace
}  // namespace pqhsa
