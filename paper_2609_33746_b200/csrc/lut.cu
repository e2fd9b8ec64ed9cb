// Step 1 of the decode operator: lookup-table construction (Sec. 3.1, text after Eq. 2).
//
// For every query head h of a (sequence, KV head):  coarse[j] = sm_scale * q_h . c_j  and
// LUT[z][m] = sm_scale * q_h^(m) . p_{m,z}.  Since q = r_q u_q, these are the paper's
// r_q/sqrt(d) * (u_q . c_j) and r_q/sqrt(d) * (u_q^(m) . p_{m,z}).  The tables are written in
// the layout the scan wants to find in shared memory: [z][m][g] with g the head inside its
// head group, so one 16-byte read serves the four heads of a GQA group.
//
// The kernel is latency bound (a few MB of reads spread over the whole GPU), so every thread
// issues all of its global loads (centroid rows, codewords) before the first use.  In the
// fused decode call it also clears the counters and histograms that the top-k needs.
#include "common.cuh"

namespace pqhsa {

constexpr int kLutThreads = 256;
constexpr int kLutWarps = kLutThreads / 32;
constexpr int kLutChunks = 32;       // CTAs per (sequence, KV head)
constexpr int kMaxGroup = 16;
constexpr int kRowsPerWarp = 4;      // centroid rows a warp holds in flight

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}

template <typename T>
__global__ void __launch_bounds__(kLutThreads)
build_lut_kernel(Plan pl, const T* __restrict__ q, const float* __restrict__ centroids,
                 const float* __restrict__ codebooks, float* __restrict__ lut,
                 float* __restrict__ coarse, uint4* __restrict__ zero_ptr, size_t zero_n16) {
  __shared__ __align__(16) float sq[kMaxGroup][kHeadDim];   // sm_scale * q of the G heads
  const int kv = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = pl.G, Gc = pl.Gc, n_hg = pl.n_hg;
  const size_t ukv = (size_t)b * pl.Hkv + kv;

  // query -> shared (first dependent load of the kernel)
  float qreg[(kMaxGroup * kHeadDim) / kLutThreads];
#pragma unroll
  for (int u = 0; u < (kMaxGroup * kHeadDim) / kLutThreads; ++u) {
    const int i = u * kLutThreads + tid;
    qreg[u] = (i < G * kHeadDim)
                  ? to_f32(q[((size_t)b * pl.Hq + kv * G) * kHeadDim + i]) : 0.f;
  }

  // ---- prefetch: centroid rows of this warp and the codeword of this thread
  const int rows_per_cta = (pl.n_list + kLutChunks - 1) / kLutChunks;
  const int r0 = blockIdx.x * rows_per_cta;
  const int r1 = min(pl.n_list, r0 + rows_per_cta);
  const int n_ent = pl.M * kNCode;
  const int ent_per_cta = (n_ent + kLutChunks - 1) / kLutChunks;
  const int e0 = blockIdx.x * ent_per_cta;
  const int e1 = min(n_ent, e0 + ent_per_cta);

  float4 crow[kRowsPerWarp];
#pragma unroll
  for (int u = 0; u < kRowsPerWarp; ++u) {
    const int j = r0 + warp + u * kLutWarps;
    crow[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j < r1)
      crow[u] = __ldg(reinterpret_cast<const float4*>(centroids + (ukv * pl.n_list + j) * kHeadDim) + lane);
  }
  float cw[16];
  {
    const int e = e0 + tid;
    const float* p = codebooks + (ukv * (size_t)n_ent + min(e, n_ent - 1)) * pl.dsub;
#pragma unroll
    for (int t = 0; t < 16; ++t) cw[t] = (t < pl.dsub && e < e1) ? __ldg(p + t) : 0.f;
  }

  // ---- side job: clear a slice of the caller's zero region
  if (zero_ptr != nullptr) {
    const size_t nthreads = (size_t)gridDim.x * gridDim.y * gridDim.z * kLutThreads;
    const size_t gtid = ((size_t)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) *
                            kLutThreads + tid;
    for (size_t i = gtid; i < zero_n16; i += nthreads) zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
  }

#pragma unroll
  for (int u = 0; u < (kMaxGroup * kHeadDim) / kLutThreads; ++u) {
    const int i = u * kLutThreads + tid;
    if (i < G * kHeadDim) sq[i / kHeadDim][i % kHeadDim] = pl.sm_scale * qreg[u];
  }
  __syncthreads();

  // ---- coarse term: one warp per centroid row, a lane holds 4 of the 128 dims
  for (int jb = r0; jb < r1; jb += kLutWarps * kRowsPerWarp) {
    if (jb != r0) {
#pragma unroll
      for (int u = 0; u < kRowsPerWarp; ++u) {
        const int j = jb + warp + u * kLutWarps;
        crow[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < r1)
          crow[u] = __ldg(reinterpret_cast<const float4*>(centroids + (ukv * pl.n_list + j) * kHeadDim) + lane);
      }
    }
#pragma unroll
    for (int u = 0; u < kRowsPerWarp; ++u) {
      const int j = jb + warp + u * kLutWarps;
      if (j >= r1) continue;                       // warp-uniform
      const float4 c = crow[u];
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
  }

  // ---- PQ table: one thread per (m, z); consecutive threads take consecutive z
  for (int eb = e0; eb < e1; eb += kLutThreads) {
    const int e = eb + tid;
    if (eb != e0 && e < e1) {
      const float* p = codebooks + (ukv * (size_t)n_ent + e) * pl.dsub;
#pragma unroll
      for (int t = 0; t < 16; ++t) cw[t] = (t < pl.dsub) ? __ldg(p + t) : 0.f;
    }
    if (e >= e1) continue;
    const int m = e / kNCode, z = e % kNCode;
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
                             float* coarse, void* zero_ptr, size_t zero_bytes, cudaStream_t st) {
  dim3 grid(kLutChunks, pl.Hkv, pl.B);
  uint4* zp = static_cast<uint4*>(zero_ptr);
  const size_t zn = zero_bytes / 16;
  if (pl.dtype == PQHSA_F16)
    build_lut_kernel<__half><<<grid, kLutThreads, 0, st>>>(
        pl, static_cast<const __half*>(q), ix.centroids, ix.codebooks, lut, coarse, zp, zn);
  else
    build_lut_kernel<__nv_bfloat16><<<grid, kLutThreads, 0, st>>>(
        pl, static_cast<const __nv_bfloat16*>(q), ix.centroids, ix.codebooks, lut, coarse, zp, zn);
  return cudaGetLastError();
}

}  // namespace pqhsa
