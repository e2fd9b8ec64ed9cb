// Step 1 of the decode operator: lookup-table construction (Sec. 3.1, text after Eq. 2).
//
// For every query head h of a (sequence, KV head):  coarse[j] = sm_scale * q_h . c_j  and
// LUT[z][m] = sm_scale * q_h^(m) . p_{m,z}.  Since q = r_q u_q, these are the paper's
// r_q/sqrt(d) * (u_q . c_j) and r_q/sqrt(d) * (u_q^(m) . p_{m,z}).  The tables are written in
// the layout the scan wants to find in shared memory: [z][m][g] with g the head inside its
// head group, so one 16-byte read serves the four heads of a GQA group.
#include "common.cuh"

namespace pqhsa {

constexpr int kLutThreads = 256;
constexpr int kLutChunks = 32;       // CTAs per (sequence, KV head)
constexpr int kMaxGroup = 16;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}

template <typename T>
__global__ void __launch_bounds__(kLutThreads)
build_lut_kernel(Plan pl, const T* __restrict__ q, const float* __restrict__ centroids,
                 const float* __restrict__ codebooks, float* __restrict__ lut,
                 float* __restrict__ coarse) {
  __shared__ __align__(16) float sq[kMaxGroup][kHeadDim];   // sm_scale * q of the G heads
  const int kv = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = pl.G, Gc = pl.Gc, n_hg = pl.n_hg;
  const size_t ukv = (size_t)b * pl.Hkv + kv;

  for (int i = tid; i < G * kHeadDim; i += kLutThreads) {
    int h = i / kHeadDim, t = i % kHeadDim;
    sq[h][t] = pl.sm_scale * to_f32(q[((size_t)b * pl.Hq + kv * G + h) * kHeadDim + t]);
  }
  __syncthreads();

  // ---- coarse term: one warp per centroid row, a lane holds 4 of the 128 dims
  const int rows_per_cta = (pl.n_list + kLutChunks - 1) / kLutChunks;
  const int r0 = blockIdx.x * rows_per_cta;
  const int r1 = min(pl.n_list, r0 + rows_per_cta);
  for (int j = r0 + warp; j < r1; j += kLutThreads / 32) {
    const float4 c = __ldg(reinterpret_cast<const float4*>(
                               centroids + (ukv * pl.n_list + j) * kHeadDim) + lane);
    for (int slot = 0; slot < n_hg * Gc; ++slot) {
      float v = 0.f;
      if (slot < G) {
        const float4 qq = *reinterpret_cast<const float4*>(&sq[slot][4 * lane]);
        v = warp_sum(c.x * qq.x + c.y * qq.y + c.z * qq.z + c.w * qq.w);
      }
      if (lane == 0) {
        int hg = slot / Gc, g = slot % Gc;
        coarse[(((ukv * n_hg + hg) * pl.n_list) + j) * Gc + g] = v;
      }
    }
  }

  // ---- PQ table: one thread per (m, z); consecutive threads take consecutive z
  const int n_ent = pl.M * kNCode;
  const int ent_per_cta = (n_ent + kLutChunks - 1) / kLutChunks;
  const int e0 = blockIdx.x * ent_per_cta;
  const int e1 = min(n_ent, e0 + ent_per_cta);
  for (int e = e0 + tid; e < e1; e += kLutThreads) {
    const int m = e / kNCode, z = e % kNCode;
    const float* p = codebooks + ((ukv * pl.M + m) * kNCode + z) * pl.dsub;
    float cw[16];
#pragma unroll
    for (int t = 0; t < 16; ++t) cw[t] = (t < pl.dsub) ? __ldg(p + t) : 0.f;
    for (int hg = 0; hg < n_hg; ++hg) {
      float* dst = lut + (((ukv * n_hg + hg) * kNCode + z) * pl.M + m) * Gc;
      for (int g = 0; g < Gc; ++g) {
        const int h = hg * Gc + g;
        float v = 0.f;
        if (h < G) {
#pragma unroll
          for (int t = 0; t < 16; ++t)
            if (t < pl.dsub) v = fmaf(cw[t], sq[h][m * pl.dsub + t], v);
        }
        dst[g] = v;
      }
    }
  }
}

cudaError_t launch_build_lut(const Plan& pl, const void* q, const pqhsa_index& ix, float* lut,
                             float* coarse, cudaStream_t st) {
  dim3 grid(kLutChunks, pl.Hkv, pl.B);
  if (pl.dtype == PQHSA_F16)
    build_lut_kernel<__half><<<grid, kLutThreads, 0, st>>>(
        pl, static_cast<const __half*>(q), ix.centroids, ix.codebooks, lut, coarse);
  else
    build_lut_kernel<__nv_bfloat16><<<grid, kLutThreads, 0, st>>>(
        pl, static_cast<const __nv_bfloat16*>(q), ix.centroids, ix.codebooks, lut, coarse);
  return cudaGetLastError();
}

}  // namespace pqhsa
