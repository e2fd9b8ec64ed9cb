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

// Split-K partial of one score row: m (log2 units), Z, the smallest exact logit the partial
// saw among the selected tokens (log2 units; +inf if none), a kind word, N[128] (16-byte
// aligned).  Kinds:
//   0  ordinary: contributes Z and N scaled by exp2(m - m_row);
//   1  raw N: a correction to the numerator alone (variant Bx), Z is zero by construction;
//   2  shared logit: Z and N are counts-weighted sums that all carry the logit
//      min over the row's ordinary partials of their word [2] (variant C2b).
constexpr int kPartStride = 4 + kHeadDim;
constexpr int kMaxParts = 128;       // partials per row a 128-thread merge can take
constexpr float kKindRaw = 1.f, kKindSharedMin = 2.f;

// Merges the n_part <= 128 partials of one row and writes y = N / Z (Eq. 5) and, if asked,
// the log-sum-exp and the output before it is rounded.  Called by all 128 threads of the CTA
// that finished last for the row, after a fence.  Every load of a phase is independent (one L2
// round trip per phase): thread t fetches the header of partial t; then warp w sums N of
// partials w, w + 4, ..., a lane owning 4 dims; shared memory joins the four warps.  s_red:
// 4 x 128 floats, s_aux: 128 + 8 floats.
template <typename T>
__device__ __forceinline__ void merge_row(const float* __restrict__ pr, int n_part, int row,
                                          int tid, float (*s_red)[kHeadDim], float* s_aux,
                                          T* __restrict__ out, float* __restrict__ lse,
                                          float* __restrict__ out_f32) {
  const int lane = tid & 31, warp = tid >> 5;
  float m_t = -CUDART_INF_F, Z_t = 0.f, lmin_t = CUDART_INF_F, kind_t = 0.f;
  if (tid < n_part) {
    const float4 hd = __ldcg(reinterpret_cast<const float4*>(pr + (size_t)tid * kPartStride));
    m_t = hd.x; Z_t = hd.y; lmin_t = hd.z; kind_t = hd.w;
  }
  __syncthreads();                      // callers may still be reading s_red / s_aux
  // shared-logit partials take the smallest exact logit of the row's selected tokens
  float lmin_w = kind_t == 0.f ? lmin_t : CUDART_INF_F;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) lmin_w = fminf(lmin_w, __shfl_xor_sync(0xffffffffu, lmin_w, o));
  if (lane == 0) s_aux[kMaxParts + warp] = lmin_w;
  __syncthreads();
  if (kind_t == kKindSharedMin) {
    m_t = fminf(fminf(s_aux[kMaxParts], s_aux[kMaxParts + 1]),
                fminf(s_aux[kMaxParts + 2], s_aux[kMaxParts + 3]));
    if (!(m_t < CUDART_INF_F)) Z_t = 0.f;            // no selected token: no shared logit
  }
  __syncthreads();
  float m_w = Z_t > 0.f ? m_t : -CUDART_INF_F;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m_w = fmaxf(m_w, __shfl_xor_sync(0xffffffffu, m_w, o));
  if (lane == 0) s_aux[kMaxParts + warp] = m_w;
  __syncthreads();
  const float m_r = fmaxf(fmaxf(s_aux[kMaxParts], s_aux[kMaxParts + 1]),
                          fmaxf(s_aux[kMaxParts + 2], s_aux[kMaxParts + 3]));
  float a_t = safe_scale(m_t, m_r, Z_t);
  if (kind_t == kKindRaw && m_r > -CUDART_INF_F && m_t > -CUDART_INF_F) a_t = fast_exp2(m_t - m_r);
  s_aux[tid] = a_t;
  float Z_w = Z_t * a_t;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) Z_w += __shfl_xor_sync(0xffffffffu, Z_w, o);
  if (lane == 0) s_aux[kMaxParts + 4 + warp] = Z_w;
  __syncthreads();
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = warp; s0 < n_part; s0 += 32) {
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int s = s0 + 4 * u;
      v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (s < n_part)
        v[u] = __ldcg(reinterpret_cast<const float4*>(pr + (size_t)s * kPartStride + 4) + lane);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int s = s0 + 4 * u;
      const float a = s < n_part ? s_aux[s] : 0.f;
      acc.x = fmaf(v[u].x, a, acc.x); acc.y = fmaf(v[u].y, a, acc.y);
      acc.z = fmaf(v[u].z, a, acc.z); acc.w = fmaf(v[u].w, a, acc.w);
    }
  }
  *reinterpret_cast<float4*>(&s_red[warp][4 * lane]) = acc;
  __syncthreads();
  const float Z_r = s_aux[kMaxParts + 4] + s_aux[kMaxParts + 5] + s_aux[kMaxParts + 6] +
                    s_aux[kMaxParts + 7];
  const float N_r = s_red[0][tid] + s_red[1][tid] + s_red[2][tid] + s_red[3][tid];
  const float y = Z_r > 0.f ? N_r / Z_r : 0.f;
  out[(size_t)row * kHeadDim + tid] = Unpack<T>::pack(y);
  if (out_f32 != nullptr) out_f32[(size_t)row * kHeadDim + tid] = y;
  if (lse != nullptr && tid == 0)
    lse[row] = Z_r > 0.f ? (m_r + log2f(Z_r)) / kLog2e : -CUDART_INF_F;
}

}  // namespace
}  // namespace pqhsa
