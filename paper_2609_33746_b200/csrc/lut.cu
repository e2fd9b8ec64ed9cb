// Step 1 of the decode operator: lookup-table construction (Sec. 3.1, text after Eq. 2).
//
// For every query head h of a (sequence, KV head):  coarse[j] = sm_scale * q_h . c_j  and
// LUT[z][m] = sm_scale * q_h^(m) . p_{m,z}.  Since q = r_q u_q, these are the paper's
// r_q/sqrt(d) * (u_q . c_j) and r_q/sqrt(d) * (u_q^(m) . p_{m,z}).  The tables are written in
// the layout the scan wants to find in shared memory: [z][m][g] with g the head inside its
// head group, so one 16-byte read serves the four heads of a GQA group.
//
// The kernel moves a few MB and is bound by latency and instruction issue, so every thread
// issues its global loads (centroid rows, codeword) before the first use, the subspace
// width is a template parameter, and four heads are reduced across a warp together.  In
// the fused decode call it also clears the counters and histograms that the top-k needs.
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

// Sums four per-lane values over the warp with 6 shuffles; afterwards every lane of the
// 8-lane group g = lane >> 3 holds the total of value g.
__device__ __forceinline__ float warp_sum4(float p0, float p1, float p2, float p3, int lane) {
  const bool up16 = (lane & 16) != 0;
  float keep0 = up16 ? p2 : p0, keep1 = up16 ? p3 : p1;
  float send0 = up16 ? p0 : p2, send1 = up16 ? p1 : p3;
  keep0 += __shfl_xor_sync(0xffffffffu, send0, 16);
  keep1 += __shfl_xor_sync(0xffffffffu, send1, 16);
  const bool up8 = (lane & 8) != 0;
  float keep = up8 ? keep1 : keep0, send = up8 ? keep0 : keep1;
  keep += __shfl_xor_sync(0xffffffffu, send, 8);
  keep += __shfl_xor_sync(0xffffffffu, keep, 4);
  keep += __shfl_xor_sync(0xffffffffu, keep, 2);
  keep += __shfl_xor_sync(0xffffffffu, keep, 1);
  return keep;
}

template <typename T, int DSUB>
__global__ void __launch_bounds__(kLutThreads)
build_lut_kernel(Plan pl, const T* __restrict__ q, const float* __restrict__ centroids,
                 const float* __restrict__ codebooks, float* __restrict__ lut,
                 float* __restrict__ coarse, uint4* __restrict__ zero_ptr, size_t zero_n16) {
  __shared__ __align__(16) float sq[kMaxGroup][kHeadDim];   // sm_scale * q of the heads, 0-padded
  const int kv = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = pl.G, Gc = pl.Gc, n_hg = pl.n_hg;
  const int n_slots = n_hg * Gc;                            // head slots, >= G
  const int gc_shift = Gc == 4 ? 2 : (Gc == 2 ? 1 : 0);     // Gc is 1, 2 or 4
  const int code_shift = 31 - __clz(pl.n_code);             // n_code is 16 or 256
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  pdl_wait();
  pdl_launch_dependents();

  // query (first dependent load of the kernel)
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
  const int kEntPerM = pl.n_code;
  const int n_ent = pl.M * kEntPerM;
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
  float cw[DSUB];
  auto load_codeword = [&](int e) {
    const float* p = codebooks + (ukv * (size_t)n_ent + e) * DSUB;
    if constexpr (DSUB == 2) {
      const float2 v = __ldg(reinterpret_cast<const float2*>(p));
      cw[0] = v.x; cw[1] = v.y;
    } else {
#pragma unroll
      for (int c = 0; c < DSUB / 4; ++c) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p) + c);
        cw[4 * c] = v.x; cw[4 * c + 1] = v.y; cw[4 * c + 2] = v.z; cw[4 * c + 3] = v.w;
      }
    }
  };
  if (e0 + tid < e1) load_codeword(e0 + tid);

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
    sq[i / kHeadDim][i % kHeadDim] = pl.sm_scale * qreg[u];      // rows >= G are zero
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
    // the lane's slice of the four query heads is the same for every row: one set of reads per
    // batch of rows
    for (int hb = 0; hb < n_slots; hb += 4) {
      float4 qq[4];
#pragma unroll
      for (int t = 0; t < 4; ++t)
        qq[t] = *reinterpret_cast<const float4*>(&sq[(hb + t) & (kMaxGroup - 1)][4 * lane]);
      const int slot = hb + (lane >> 3);
      const int hg = slot >> gc_shift, g = slot & (Gc - 1);
      float* dst = coarse + ((ukv * n_hg + hg) * (size_t)pl.n_list) * Gc + g;
#pragma unroll
      for (int u = 0; u < kRowsPerWarp; ++u) {
        const int j = jb + warp + u * kLutWarps;
        if (j >= r1) continue;                       // warp-uniform
        const float4 c = crow[u];
        float p[4];
#pragma unroll
        for (int t = 0; t < 4; ++t)
          p[t] = c.x * qq[t].x + c.y * qq[t].y + c.z * qq[t].z + c.w * qq[t].w;
        const float tot = warp_sum4(p[0], p[1], p[2], p[3], lane);
        if ((lane & 7) == 0 && slot < n_slots) dst[(size_t)j * Gc] = tot;
      }
    }
  }

  // ---- PQ table: one thread per (m, z); consecutive threads take consecutive z, so the
  //      subspace m (and with it the query sub-vector) is uniform over a warp
  float* const lut_u = lut + ukv * n_hg * (size_t)pl.n_code * pl.M * Gc;
  for (int eb = e0; eb < e1; eb += kLutThreads) {
    const int e = eb + tid;
    if (eb != e0 && e < e1) load_codeword(e);
    if (e >= e1) continue;
    const int m = e >> code_shift, z = e & (kEntPerM - 1);
    for (int hg = 0; hg < n_hg; ++hg) {
      float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (g < Gc) {
          // (same products in the same order as a scalar loop; the reads are 8 or 16 bytes wide)
          const float* qs = &sq[(hg * Gc + g) & (kMaxGroup - 1)][m * DSUB];
          float qv[DSUB];
          if constexpr (DSUB == 2) {
            const float2 t2 = *reinterpret_cast<const float2*>(qs);
            qv[0] = t2.x; qv[1] = t2.y;
          } else {
#pragma unroll
            for (int c = 0; c < DSUB / 4; ++c) {
              const float4 t4 = *reinterpret_cast<const float4*>(qs + 4 * c);
              qv[4 * c] = t4.x; qv[4 * c + 1] = t4.y; qv[4 * c + 2] = t4.z; qv[4 * c + 3] = t4.w;
            }
          }
#pragma unroll
          for (int t = 0; t < DSUB; ++t) v[g] = fmaf(cw[t], qv[t], v[g]);
        }
      }
      float* dst = lut_u + (((size_t)hg * pl.n_code + z) * pl.M + m) * Gc;
      if (Gc == 4) *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
      else if (Gc == 2) *reinterpret_cast<float2*>(dst) = make_float2(v[0], v[1]);
      else dst[0] = v[0];
    }
  }
}

template <typename T>
static cudaError_t launch_lut_t(const Plan& pl, const T* q, const pqhsa_index& ix, float* lut,
                                float* coarse, uint4* zp, size_t zn, cudaStream_t st) {
  dim3 grid(kLutChunks, pl.Hkv, pl.B);
  switch (pl.dsub) {
    case 2: return launch_pdl(build_lut_kernel<T, 2>, grid, dim3(kLutThreads), 0, st, pl, q, ix.centroids, ix.codebooks, lut, coarse, zp, zn);
    case 4: return launch_pdl(build_lut_kernel<T, 4>, grid, dim3(kLutThreads), 0, st, pl, q, ix.centroids, ix.codebooks, lut, coarse, zp, zn);
    case 8: return launch_pdl(build_lut_kernel<T, 8>, grid, dim3(kLutThreads), 0, st, pl, q, ix.centroids, ix.codebooks, lut, coarse, zp, zn);
    case 16: return launch_pdl(build_lut_kernel<T, 16>, grid, dim3(kLutThreads), 0, st, pl, q, ix.centroids, ix.codebooks, lut, coarse, zp, zn);
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_build_lut(const Plan& pl, const void* q, const pqhsa_index& ix, float* lut,
                             float* coarse, void* zero_ptr, size_t zero_bytes, cudaStream_t st) {
  uint4* zp = static_cast<uint4*>(zero_ptr);
  const size_t zn = zero_bytes / 16;
  if (pl.dtype == PQHSA_F16)
    return launch_lut_t(pl, static_cast<const __half*>(q), ix, lut, coarse, zp, zn, st);
  return launch_lut_t(pl, static_cast<const __nv_bfloat16*>(q), ix, lut, coarse, zp, zn, st);
}

}  // namespace pqhsa
