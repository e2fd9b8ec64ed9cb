// Batched index build (Sec. 3.3, first paragraph; App. C, "Index build"): the k-means problems
// of ALL (sequence, KV head) units are trained together, one launch per step for all of them --
// one coarse problem per unit over its key directions, then one product-quantisation problem
// per (unit, subspace) over the residuals -- instead of thousands of small per-head launches.
// Direction-norm residual IVF-PQ of Sec. 3.1: r_i = |k_i| in fp32 from the cached key,
// u_i = k_i / r_i (0 for a zero key), Lloyd iterations with squared Euclidean distance, a
// centroid is the arithmetic mean of its members (not re-normalised: Eq. 2 uses c_j as is), an
// empty cluster is re-seeded with the point farthest from its centre, ties go to the lower index.
// The random draws of the method (which points seed the centroids and the codewords) are inputs.
//
//   build_prepare_kernel     norms and unit directions U (fp32, workspace) from the paged cache
//   build_seed_kernel        centroids <- U rows at the given positions
//   build_assign_kernel      nearest centroid of every token: a register-tiled fp32 product
//                            U (128 tokens) x C^T (64 centroids at a time) with the argmin fused
//                            into its epilogue; distance = (|u|^2 - 2 u.c) + |c|^2, the form the
//                            reference builder uses.  No tensor cores: the argmin flips under
//                            tf32 / bf16 rounding, and a split-precision tensor-core product
//                            with an exact re-check of near-ties is future work.  This kernel
//                            is bound by the fp32 FMA pipe (2 * 128 * n_list flops per token
//                            against 512 bytes), not by memory.
//   build_accumulate_kernel  per-list sums of the member directions (64-bit fixed point, so the
//                            result does not depend on the order of the atomics) and member
//                            counts; build_update_centroids_kernel takes the mean
//   build_reseed_kernel      empty lists take the farthest points (rare)
//   build_pq_* kernels       the same three steps for the residual sub-vectors
//   build_value_* kernels    list value means and member counts from the paged values
#include "attn_common.cuh"
#include "common.cuh"

namespace pqhsa {

namespace {

constexpr int kD = kHeadDim;            // 128
constexpr int kPrepThreads = 256;

// Sums of member vectors are taken in 64-bit fixed point with integer atomics: integer
// addition is associative, so the centroids (and with them the whole index) do not depend on
// the order in which the atomics land -- two builds of the same input are bit-identical.
// Directions and residuals are below 2 in magnitude (scale 2^40, 131,072 members stay below
// 2^58); values are cache-dtype numbers (scale 2^24, exact for bf16 / fp16 inputs up to 2^15).
constexpr float kFixDir = 1099511627776.0f;      // 2^40
constexpr float kFixVal = 16777216.0f;           // 2^24
__device__ __forceinline__ void fix_add(long long* dst, float v, float scale) {
  atomicAdd(reinterpret_cast<unsigned long long*>(dst), (unsigned long long)__float2ll_rn(v * scale));
}
__device__ __forceinline__ float fix_mean(long long s, int count, float scale) {
  return (float)(((double)s / (double)scale) / (double)count);
}

__device__ __forceinline__ long long kv_row(const Plan& pl, const int32_t* __restrict__ bt, int pos,
                                            int kv, long long sp, long long st, long long sh) {
  const int page = __ldg(bt + pos / pl.page_size);
  return (long long)page * sp + (long long)(pos % pl.page_size) * st + (long long)kv * sh;
}

// ---- norms and directions: a warp per token, a lane holds 4 of the 128 dims
template <typename T>
__global__ void __launch_bounds__(kPrepThreads)
build_prepare_kernel(Plan pl, const T* __restrict__ kc, long long sp, long long st, long long sh,
                     const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                     float* __restrict__ U, float* __restrict__ key_norms) {
  const int kv = blockIdx.y, b = blockIdx.z;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;
  for (int i = blockIdx.x * (kPrepThreads / 32) + warp; i < n; i += gridDim.x * (kPrepThreads / 32)) {
    const T* row = kc + kv_row(pl, bt, i, kv, sp, st, sh);
    float x[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) x[t] = Unpack<T>::one(row[4 * lane + t]);
    const float ss = warp_sum(x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3]);
    const float r = sqrtf(ss);
    const float inv = r > 0.f ? 1.f / r : 0.f;
    *reinterpret_cast<float4*>(U + (ukv * pl.N_max + i) * kD + 4 * lane) =
        make_float4(x[0] * inv, x[1] * inv, x[2] * inv, x[3] * inv);
    if (lane == 0) key_norms[ukv * pl.N_max + i] = r;
  }
}

// ---- seeds: row j of `dst` [units][n_rows][kD] <- U row at seed_pos[unit][j] (zero if < 0)
__global__ void build_seed_kernel(Plan pl, const float* __restrict__ U,
                                  const int32_t* __restrict__ seed_pos, int n_rows,
                                  float* __restrict__ dst) {
  const size_t unit = blockIdx.y;
  const int j = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (j >= n_rows) return;
  const int pos = seed_pos[unit * n_rows + j];
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (pos >= 0 && pos < pl.N_max) v = *reinterpret_cast<const float4*>(U + (unit * pl.N_max + pos) * kD + 4 * lane);
  *reinterpret_cast<float4*>(dst + (unit * n_rows + j) * kD + 4 * lane) = v;
}

// ---- nearest centroid.  CTA: 128 tokens of one unit; 256 threads as 16 x 16; thread (ty, tx)
// owns tokens ty + 16 i (i < 8) and, of every 64-centroid tile, centroids tx + 16 j (j < 4).
// Both tiles sit in shared memory row-major with a stride of 132 floats, so that the float4
// reads along the dims are conflict free (the rows a quarter warp reads start 4 banks apart).
constexpr int kAsgTok = 128, kAsgCen = 64, kAsgThreads = 256, kAsgStride = kD + 4;
constexpr int kAsgSmemBytes = (kAsgTok + kAsgCen) * kAsgStride * 4 + kAsgCen * 4;

__global__ void __launch_bounds__(kAsgThreads, 2)
build_assign_kernel(Plan pl, const float* __restrict__ U, const float* __restrict__ centroids,
                    const int32_t* __restrict__ seq_lens, uint16_t* __restrict__ list_ids,
                    float* __restrict__ dmin) {
  extern __shared__ __align__(16) float s_asg[];
  float* s_u = s_asg;                                   // [128][132]
  float* s_c = s_u + kAsgTok * kAsgStride;              // [64][132]
  float* s_cn = s_c + kAsgCen * kAsgStride;             // [64] |c|^2
  const int kv = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const int t0 = blockIdx.x * kAsgTok;
  if (t0 >= n) return;
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  const float* Ub = U + (ukv * pl.N_max + t0) * kD;
  const float* Cb = centroids + ukv * (size_t)pl.n_list * kD;
  const int n_tok = min(kAsgTok, n - t0);
  for (int i = tid; i < kAsgTok * (kD / 4); i += kAsgThreads) {
    const int r = i / (kD / 4), c4 = i % (kD / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < n_tok) v = __ldg(reinterpret_cast<const float4*>(Ub + (size_t)r * kD) + c4);
    *reinterpret_cast<float4*>(s_u + r * kAsgStride + 4 * c4) = v;
  }
  __syncthreads();
  float xs2[8];                                         // |u|^2 of my tokens
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float* ur = s_u + (ty + 16 * i) * kAsgStride;
    float a = 0.f;
    for (int k = 0; k < kD; ++k) a = fmaf(ur[k], ur[k], a);
    xs2[i] = a;
  }
  float best_d[8];
  int best_j[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { best_d[i] = CUDART_INF_F; best_j[i] = 0; }

  for (int c0 = 0; c0 < pl.n_list; c0 += kAsgCen) {
    __syncthreads();                                    // previous tile consumed
    for (int i = tid; i < kAsgCen * (kD / 4); i += kAsgThreads) {
      const int r = i / (kD / 4), c4 = i % (kD / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c0 + r < pl.n_list) v = __ldg(reinterpret_cast<const float4*>(Cb + (size_t)(c0 + r) * kD) + c4);
      *reinterpret_cast<float4*>(s_c + r * kAsgStride + 4 * c4) = v;
    }
    __syncthreads();
    if (tid < kAsgCen) {
      const float* cr = s_c + tid * kAsgStride;
      float a = 0.f;
      for (int k = 0; k < kD; ++k) a = fmaf(cr[k], cr[k], a);
      s_cn[tid] = a;
    }
    float acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 2
    for (int k = 0; k < kD; k += 4) {
      float4 uv[8], cv[4];
#pragma unroll
      for (int i = 0; i < 8; ++i) uv[i] = *reinterpret_cast<const float4*>(s_u + (ty + 16 * i) * kAsgStride + k);
#pragma unroll
      for (int j = 0; j < 4; ++j) cv[j] = *reinterpret_cast<const float4*>(s_c + (tx + 16 * j) * kAsgStride + k);
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(uv[i].x, cv[j].x, acc[i][j]);
          acc[i][j] = fmaf(uv[i].y, cv[j].y, acc[i][j]);
          acc[i][j] = fmaf(uv[i].z, cv[j].z, acc[i][j]);
          acc[i][j] = fmaf(uv[i].w, cv[j].w, acc[i][j]);
        }
    }
    __syncthreads();                                    // s_cn written
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int cj = c0 + tx + 16 * j;
      if (cj < pl.n_list) {
        const float cn = s_cn[tx + 16 * j];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float d = (xs2[i] - 2.0f * acc[i][j]) + cn;
          if (d < best_d[i] || (d == best_d[i] && cj < best_j[i])) { best_d[i] = d; best_j[i] = cj; }
        }
      }
    }
  }
  // the 16 threads of a row (same ty: consecutive lanes of a half warp) join their minima
#pragma unroll
  for (int i = 0; i < 8; ++i) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      const float od = __shfl_xor_sync(0xffffffffu, best_d[i], o);
      const int oj = __shfl_xor_sync(0xffffffffu, best_j[i], o);
      if (od < best_d[i] || (od == best_d[i] && oj < best_j[i])) { best_d[i] = od; best_j[i] = oj; }
    }
    const int r = ty + 16 * i;
    if (tx == 0 && r < n_tok) {
      list_ids[ukv * pl.N_max + t0 + r] = (uint16_t)best_j[i];
      dmin[ukv * pl.N_max + t0 + r] = best_d[i];
    }
  }
}

// ---- per-list sums of member directions: a warp per token, one 16-byte reduction per lane
__global__ void __launch_bounds__(kPrepThreads)
build_accumulate_kernel(Plan pl, const float* __restrict__ U, const uint16_t* __restrict__ list_ids,
                        const int32_t* __restrict__ seq_lens,
                        long long* __restrict__ sums, int32_t* __restrict__ counts) {
  const int kv = blockIdx.y, b = blockIdx.z;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  for (int i = blockIdx.x * (kPrepThreads / 32) + warp; i < n; i += gridDim.x * (kPrepThreads / 32)) {
    const uint32_t j = min((uint32_t)list_ids[ukv * pl.N_max + i], (uint32_t)(pl.n_list - 1));
    const float4 u = *reinterpret_cast<const float4*>(U + (ukv * pl.N_max + i) * kD + 4 * lane);
    long long* dst = sums + (ukv * pl.n_list + j) * kD + 4 * lane;
    fix_add(dst, u.x, kFixDir); fix_add(dst + 1, u.y, kFixDir);
    fix_add(dst + 2, u.z, kFixDir); fix_add(dst + 3, u.w, kFixDir);
    if (lane == 0) atomicAdd(&counts[ukv * pl.n_list + j], 1);
  }
}

// c_j <- mean of its members; an empty list keeps its centre and is counted; sums are cleared
__global__ void build_update_centroids_kernel(Plan pl, long long* __restrict__ sums,
                                              const int32_t* __restrict__ counts,
                                              float* __restrict__ centroids,
                                              int32_t* __restrict__ n_empty) {
  const size_t unit = blockIdx.y;
  const int j = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (j >= pl.n_list) return;
  const size_t at = (unit * pl.n_list + j) * kD + 4 * lane;
  const int c = counts[unit * pl.n_list + j];
  if (c > 0) {
    *reinterpret_cast<float4*>(centroids + at) =
        make_float4(fix_mean(sums[at], c, kFixDir), fix_mean(sums[at + 1], c, kFixDir),
                    fix_mean(sums[at + 2], c, kFixDir), fix_mean(sums[at + 3], c, kFixDir));
  } else if (lane == 0) {
    atomicAdd(&n_empty[unit], 1);
  }
#pragma unroll
  for (int t = 0; t < 4; ++t) sums[at + t] = 0;
}

// Empty lists take the farthest points: the e-th empty list (in index order) gets the point
// with the e-th largest distance to its centre (ties: lower position).  One CTA per unit;
// rare, so a plain repeated arg-max over the unit's distances; at most kMaxReseed lists per call.
constexpr int kMaxReseed = 64;
__global__ void __launch_bounds__(1024)
build_reseed_kernel(Plan pl, const float* __restrict__ U, float* __restrict__ dmin,
                    const int32_t* __restrict__ counts, const int32_t* __restrict__ seq_lens,
                    int32_t* __restrict__ n_empty, float* __restrict__ centroids) {
  __shared__ float s_d[32];
  __shared__ int s_i[32];
  __shared__ int s_pick;
  const int unit = blockIdx.x, b = unit / pl.Hkv, tid = threadIdx.x;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const int ne = n_empty[unit];
  if (ne == 0 || n <= pl.n_list) { if (tid == 0) n_empty[unit] = 0; return; }
  float* d = dmin + (size_t)unit * pl.N_max;
  int j = 0;
  for (int e = 0; e < min(ne, kMaxReseed); ++e) {
    while (j < pl.n_list && counts[(size_t)unit * pl.n_list + j] > 0) ++j;       // uniform
    if (j >= pl.n_list) break;
    float bd = -CUDART_INF_F;
    int bi = 0x7fffffff;
    for (int i = tid; i < n; i += blockDim.x) {
      const float v = d[i];
      if (v > bd || (v == bd && i < bi)) { bd = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float od = __shfl_xor_sync(0xffffffffu, bd, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (od > bd || (od == bd && oi < bi)) { bd = od; bi = oi; }
    }
    if ((tid & 31) == 0) { s_d[tid >> 5] = bd; s_i[tid >> 5] = bi; }
    __syncthreads();
    if (tid < 32) {
      bd = tid < (int)(blockDim.x >> 5) ? s_d[tid] : -CUDART_INF_F;
      bi = tid < (int)(blockDim.x >> 5) ? s_i[tid] : 0x7fffffff;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float od = __shfl_xor_sync(0xffffffffu, bd, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (od > bd || (od == bd && oi < bi)) { bd = od; bi = oi; }
      }
      if (tid == 0) { s_pick = bi; d[bi] = -CUDART_INF_F; }      // taken: not picked again
    }
    __syncthreads();
    const int pick = s_pick;
    if (tid < kD) centroids[((size_t)unit * pl.n_list + j) * kD + tid] = U[((size_t)unit * pl.N_max + pick) * kD + tid];
    ++j;
    __syncthreads();
  }
  if (tid == 0) n_empty[unit] = 0;
}

// ---- product quantisation of the residuals e_i = u_i - c_{a_i}.  Codebooks [unit][M][n_code][dsub].
// Seeds: codeword z of subspace m <- residual sub-vector m of the token at seed_pos[unit][z].
template <int DSUB>
__global__ void build_pq_seed_kernel(Plan pl, const float* __restrict__ U,
                                     const float* __restrict__ centroids,
                                     const uint16_t* __restrict__ list_ids,
                                     const int32_t* __restrict__ seed_pos,
                                     float* __restrict__ codebooks) {
  const size_t unit = blockIdx.y;
  const int z = blockIdx.x, d = threadIdx.x;                 // 128 threads: one per dim
  const int pos = seed_pos[unit * pl.n_code + z];
  float e = 0.f;
  if (pos >= 0 && pos < pl.N_max) {
    const uint32_t a = min((uint32_t)list_ids[unit * pl.N_max + pos], (uint32_t)(pl.n_list - 1));
    e = U[(unit * pl.N_max + pos) * kD + d] - centroids[(unit * pl.n_list + a) * kD + d];
  }
  const int m = d / DSUB, t = d % DSUB;
  codebooks[((unit * pl.M + m) * pl.n_code + z) * DSUB + t] = e;
}

// Nearest codeword of every (token, subspace): CTA = 128 tokens x one group of subspaces whose
// codebooks fit shared memory; a thread owns a token, walks the codewords (broadcast reads).
// distance = (|e|^2 - 2 e.p) + |p|^2.  Optionally accumulates the per-codeword sums for the
// next Lloyd step (training) or writes the final codes (encode).
template <int DSUB>
__global__ void __launch_bounds__(128)
build_pq_assign_kernel(Plan pl, const float* __restrict__ U, const float* __restrict__ centroids,
                       const uint16_t* __restrict__ list_ids, const float* __restrict__ codebooks,
                       const int32_t* __restrict__ seq_lens, int m_per_cta,
                       long long* __restrict__ pq_sums, int32_t* __restrict__ pq_counts,
                       uint8_t* __restrict__ codes_out) {
  extern __shared__ __align__(16) float s_cb[];             // [m_per_cta][n_code][DSUB + 1 (|p|^2)]
  const int kv = blockIdx.y % pl.Hkv, b = blockIdx.y / pl.Hkv;
  const int mg = blockIdx.z, tid = threadIdx.x;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const int i = blockIdx.x * 128 + tid;
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  const int m0 = mg * m_per_cta, m1 = min(pl.M, m0 + m_per_cta);
  if (blockIdx.x * 128 >= n) return;
  constexpr int kW = DSUB + 1;
  for (int idx = tid; idx < (m1 - m0) * pl.n_code; idx += 128) {
    const float* p = codebooks + ((ukv * pl.M + m0) * pl.n_code + idx) * DSUB;
    float pn = 0.f;
#pragma unroll
    for (int t = 0; t < DSUB; ++t) { const float v = p[t]; s_cb[idx * kW + t] = v; pn = fmaf(v, v, pn); }
    s_cb[idx * kW + DSUB] = pn;
  }
  __syncthreads();
  if (i >= n) return;
  const uint32_t a = min((uint32_t)list_ids[ukv * pl.N_max + i], (uint32_t)(pl.n_list - 1));
  const float* ur = U + (ukv * pl.N_max + i) * kD;
  const float* cr = centroids + (ukv * pl.n_list + a) * kD;
  for (int m = m0; m < m1; ++m) {
    float e[DSUB], en = 0.f;
#pragma unroll
    for (int t = 0; t < DSUB; ++t) { e[t] = ur[m * DSUB + t] - cr[m * DSUB + t]; en = fmaf(e[t], e[t], en); }
    const float* cb = s_cb + (size_t)(m - m0) * pl.n_code * kW;
    float bd = CUDART_INF_F;
    int bz = 0;
    for (int z = 0; z < pl.n_code; ++z) {
      float dot = 0.f;
#pragma unroll
      for (int t = 0; t < DSUB; ++t) dot = fmaf(e[t], cb[z * kW + t], dot);
      const float dist = (en - 2.0f * dot) + cb[z * kW + DSUB];
      if (dist < bd) { bd = dist; bz = z; }                  // z ascends: the first minimum stays
    }
    if (pq_sums != nullptr) {
      long long* dst = pq_sums + ((ukv * pl.M + m) * pl.n_code + bz) * DSUB;
#pragma unroll
      for (int t = 0; t < DSUB; ++t) fix_add(dst + t, e[t], kFixDir);
      atomicAdd(&pq_counts[(ukv * pl.M + m) * pl.n_code + bz], 1);
    }
    if (codes_out != nullptr) {
      if (pl.n_code == 16) {
        // two 4-bit codes per byte, subspace 2j in the low nibble: the thread owns the token,
        // so consecutive subspaces of one byte are written by the same thread in order
        uint8_t* dst = codes_out + (ukv * pl.N_max + i) * pl.code_bytes + (m >> 1);
        *dst = (m & 1) ? (uint8_t)(*dst | (bz << 4)) : (uint8_t)bz;
      } else {
        codes_out[(ukv * pl.N_max + i) * pl.code_bytes + m] = (uint8_t)bz;
      }
    }
  }
}

// codeword <- mean of its members (kept if it has none); sums and counts cleared
__global__ void build_pq_update_kernel(size_t n_entries, int dsub, long long* __restrict__ pq_sums,
                                       int32_t* __restrict__ pq_counts, float* __restrict__ codebooks) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n_entries) return;
  const int c = pq_counts[e];
  for (int t = 0; t < dsub; ++t) {
    if (c > 0) codebooks[e * dsub + t] = fix_mean(pq_sums[e * dsub + t], c, kFixDir);
    pq_sums[e * dsub + t] = 0;
  }
  pq_counts[e] = 0;
}

// ---- list value means over the members inside R and member counts (Eq. 4's vbar_j)
template <typename T>
__global__ void __launch_bounds__(kPrepThreads)
build_value_sums_kernel(Plan pl, const T* __restrict__ vc, long long sp, long long st, long long sh,
                        const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                        const uint16_t* __restrict__ list_ids, long long* __restrict__ sums,
                        int32_t* __restrict__ counts) {
  const int kv = blockIdx.y, b = blockIdx.z;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const Region rg = region_of(pl, n, b);
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;
  for (int i = rg.r_begin + blockIdx.x * (kPrepThreads / 32) + warp; i < rg.r_end;
       i += gridDim.x * (kPrepThreads / 32)) {
    const uint32_t j = min((uint32_t)list_ids[ukv * pl.N_max + i], (uint32_t)(pl.n_list - 1));
    const T* row = vc + kv_row(pl, bt, i, kv, sp, st, sh);
    long long* dst = sums + (ukv * pl.n_list + j) * kD + 4 * lane;
#pragma unroll
    for (int t = 0; t < 4; ++t) fix_add(dst + t, Unpack<T>::one(row[4 * lane + t]), kFixVal);
    if (lane == 0) atomicAdd(&counts[ukv * pl.n_list + j], 1);
  }
}

__global__ void build_value_means_kernel(Plan pl, long long* __restrict__ sums, const int32_t* __restrict__ counts,
                                         float* __restrict__ vmeans, int32_t* __restrict__ list_counts) {
  const size_t unit = blockIdx.y;
  const int j = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (j >= pl.n_list) return;
  const size_t at = (unit * pl.n_list + j) * kD + 4 * lane;
  const int c = counts[unit * pl.n_list + j];
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c > 0)
    s = make_float4(fix_mean(sums[at], c, kFixVal), fix_mean(sums[at + 1], c, kFixVal),
                    fix_mean(sums[at + 2], c, kFixVal), fix_mean(sums[at + 3], c, kFixVal));
  *reinterpret_cast<float4*>(vmeans + at) = s;
#pragma unroll
  for (int t = 0; t < 4; ++t) sums[at + t] = 0;
  if (lane == 0) list_counts[unit * pl.n_list + j] = c;
}

struct BuildWs {
  size_t U, dmin, sums, counts, n_empty, pq_sums, pq_counts, total;
};
size_t up256(size_t x) { return (x + 255) / 256 * 256; }
BuildWs build_layout(const Plan& pl) {
  BuildWs w;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up256(o + bytes); return at; };
  const size_t units = (size_t)pl.B * pl.Hkv;
  w.U = take(units * pl.N_max * kD * 4);
  w.dmin = take(units * pl.N_max * 4);
  w.sums = take(units * pl.n_list * kD * 8);
  w.counts = take(units * pl.n_list * 4);
  w.n_empty = take(units * 4);
  w.pq_sums = take(units * pl.M * pl.n_code * pl.dsub * 8);
  w.pq_counts = take(units * pl.M * pl.n_code * 4);
  w.total = o;
  return w;
}

template <typename T, int DSUB>
cudaError_t run_build(const Plan& pl, const pqhsa_paged_kv& kv, const int32_t* seq_lens,
                      const int32_t* seed_lists, const int32_t* seed_codes, int coarse_iters,
                      int pq_iters, const pqhsa_index_out& ix, char* ws, cudaStream_t st) {
  const BuildWs w = build_layout(pl);
  float* U = reinterpret_cast<float*>(ws + w.U);
  float* dmin = reinterpret_cast<float*>(ws + w.dmin);
  long long* sums = reinterpret_cast<long long*>(ws + w.sums);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + w.counts);
  int32_t* n_empty = reinterpret_cast<int32_t*>(ws + w.n_empty);
  long long* pq_sums = reinterpret_cast<long long*>(ws + w.pq_sums);
  int32_t* pq_counts = reinterpret_cast<int32_t*>(ws + w.pq_counts);
  const int units = pl.B * pl.Hkv;
  const T* kc = static_cast<const T*>(kv.k_cache);
  const T* vc = static_cast<const T*>(kv.v_cache);
  const long long sp = kv.stride_page, stt = kv.stride_token, sh = kv.stride_head;
  cudaError_t e;
#define PQHSA_TRY(x) do { e = (x); if (e != cudaSuccess) return e; } while (0)
  PQHSA_TRY(cudaMemsetAsync(ws + w.sums, 0, w.total - w.sums, st));
  const int tok_ctas = min(1024, (pl.N_max + 7) / 8);
  build_prepare_kernel<T><<<dim3(tok_ctas, pl.Hkv, pl.B), kPrepThreads, 0, st>>>(
      pl, kc, sp, stt, sh, kv.block_table, seq_lens, U, ix.key_norms);
  build_seed_kernel<<<dim3((pl.n_list + 7) / 8, units), 256, 0, st>>>(pl, U, seed_lists, pl.n_list, ix.centroids);
  PQHSA_TRY(cudaFuncSetAttribute(build_assign_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAsgSmemBytes));
  const dim3 asg_grid((pl.N_max + kAsgTok - 1) / kAsgTok, pl.Hkv, pl.B);
  const dim3 list_grid((pl.n_list + 7) / 8, units);
  for (int it = 0; it < coarse_iters; ++it) {
    build_assign_kernel<<<asg_grid, kAsgThreads, kAsgSmemBytes, st>>>(pl, U, ix.centroids, seq_lens, ix.list_ids, dmin);
    PQHSA_TRY(cudaMemsetAsync(counts, 0, (size_t)units * pl.n_list * 4, st));
    build_accumulate_kernel<<<dim3(tok_ctas, pl.Hkv, pl.B), kPrepThreads, 0, st>>>(pl, U, ix.list_ids, seq_lens, sums, counts);
    build_update_centroids_kernel<<<list_grid, 256, 0, st>>>(pl, sums, counts, ix.centroids, n_empty);
    build_reseed_kernel<<<units, 1024, 0, st>>>(pl, U, dmin, counts, seq_lens, n_empty, ix.centroids);
  }
  build_assign_kernel<<<asg_grid, kAsgThreads, kAsgSmemBytes, st>>>(pl, U, ix.centroids, seq_lens, ix.list_ids, dmin);
  // product quantisation of the residuals: as many subspaces per CTA as fit 96 KB of codebooks
  int m_per_cta = (96 * 1024) / (pl.n_code * (DSUB + 1) * 4);
  if (m_per_cta > pl.M) m_per_cta = pl.M;
  if (m_per_cta < 1) return cudaErrorInvalidValue;
  const int pq_smem = m_per_cta * pl.n_code * (DSUB + 1) * 4;
  PQHSA_TRY(cudaFuncSetAttribute(build_pq_assign_kernel<DSUB>, cudaFuncAttributeMaxDynamicSharedMemorySize, pq_smem));
  const dim3 pq_grid((pl.N_max + 127) / 128, units, (pl.M + m_per_cta - 1) / m_per_cta);
  const size_t n_entries = (size_t)units * pl.M * pl.n_code;
  build_pq_seed_kernel<DSUB><<<dim3(pl.n_code, units), kD, 0, st>>>(pl, U, ix.centroids, ix.list_ids, seed_codes, ix.codebooks);
  for (int it = 0; it < pq_iters; ++it) {
    build_pq_assign_kernel<DSUB><<<pq_grid, 128, pq_smem, st>>>(pl, U, ix.centroids, ix.list_ids, ix.codebooks,
                                                               seq_lens, m_per_cta, pq_sums, pq_counts, nullptr);
    build_pq_update_kernel<<<(unsigned)((n_entries + 255) / 256), 256, 0, st>>>(n_entries, DSUB, pq_sums, pq_counts, ix.codebooks);
  }
  build_pq_assign_kernel<DSUB><<<pq_grid, 128, pq_smem, st>>>(pl, U, ix.centroids, ix.list_ids, ix.codebooks,
                                                             seq_lens, m_per_cta, nullptr, nullptr, ix.codes);
  // list value means and member counts
  PQHSA_TRY(cudaMemsetAsync(counts, 0, (size_t)units * pl.n_list * 4, st));
  build_value_sums_kernel<T><<<dim3(tok_ctas, pl.Hkv, pl.B), kPrepThreads, 0, st>>>(
      pl, vc, sp, stt, sh, kv.block_table, seq_lens, ix.list_ids, sums, counts);
  build_value_means_kernel<<<list_grid, 256, 0, st>>>(pl, sums, counts, ix.list_vmeans, ix.list_counts);
#undef PQHSA_TRY
  return cudaGetLastError();
}

}  // namespace
}  // namespace pqhsa

using namespace pqhsa;

extern "C" {

size_t pqhsa_index_build_workspace_bytes(const pqhsa_params* params) {
  Plan pl;
  if (make_plan(params, &pl) != PQHSA_OK) return 0;
  return build_layout(pl).total;
}

int pqhsa_index_build(const pqhsa_params* params, const pqhsa_paged_kv* kv, const int32_t* seq_lens,
                      const int32_t* seed_lists, const int32_t* seed_codes, int32_t coarse_iters,
                      int32_t pq_iters, const pqhsa_index_out* index, void* ws, size_t ws_bytes,
                      void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (kv == nullptr || kv->k_cache == nullptr || kv->v_cache == nullptr || kv->block_table == nullptr ||
      seq_lens == nullptr || seed_lists == nullptr || seed_codes == nullptr || index == nullptr ||
      index->centroids == nullptr || index->codebooks == nullptr || index->codes == nullptr ||
      index->list_ids == nullptr || index->key_norms == nullptr || index->list_vmeans == nullptr ||
      index->list_counts == nullptr || coarse_iters < 0 || pq_iters < 0 || ws == nullptr ||
      (reinterpret_cast<uintptr_t>(ws) & 255u) != 0)
    return PQHSA_ERR_INVALID_ARG;
  if (kv->stride_page % 8 || kv->stride_token % 8 || kv->stride_head % 8) return PQHSA_ERR_UNSUPPORTED;
  if (ws_bytes < build_layout(pl).total) return PQHSA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  cudaError_t e = cudaErrorInvalidValue;
#define PQHSA_BUILD_CASE(DS)                                                                        \
  if (pl.dsub == DS)                                                                                \
    e = pl.dtype == PQHSA_F16                                                                       \
            ? run_build<__half, DS>(pl, *kv, seq_lens, seed_lists, seed_codes, coarse_iters,        \
                                    pq_iters, *index, w, st)                                        \
            : run_build<__nv_bfloat16, DS>(pl, *kv, seq_lens, seed_lists, seed_codes, coarse_iters, \
                                           pq_iters, *index, w, st);
  PQHSA_BUILD_CASE(2) PQHSA_BUILD_CASE(4) PQHSA_BUILD_CASE(8) PQHSA_BUILD_CASE(16)
#undef PQHSA_BUILD_CASE
  return e == cudaSuccess ? PQHSA_OK : PQHSA_ERR_CUDA;
}

}  // extern "C"
