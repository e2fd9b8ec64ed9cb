// Index maintenance between decode steps (Sec. 3.3, first paragraph): tokens that leave the
// local window are encoded into the existing lists, without re-clustering, and the list value
// means are refreshed.  Encoding follows Sec. 3.1: r_i = |k_i| (fp32), u_i = k_i / r_i,
// a_i = the list whose centroid is nearest to u_i (squared Euclidean distance, lower index on
// ties), z_im = the codeword nearest to the m-th sub-vector of the residual u_i - c_{a_i}.
//
//   index_encode_kernel         8 new tokens per CTA.  Centroids pass through shared memory
//       in tiles of 32 rows (a lane owns a centroid, a warp a token); for the codes a warp owns
//       a subspace and a lane a codeword, so a codebook row is read once, coalesced, for all 8
//       tokens.  Writes codes, list ids and norms at the tokens' positions.
//   index_refresh_means_kernel  one CTA per (sequence, KV head).  Groups the new tokens by list
//       (first occurrence = leader), sums each group's value rows in token order and sets
//       vbar_j = (n_j vbar_j + sum) / (n_j + new_j), n_j += new_j.
#include "attn_common.cuh"
#include "common.cuh"

namespace pqhsa {

namespace {

constexpr int kUpdTok = 8;              // tokens per CTA = warps per CTA
constexpr int kUpdThreads = 32 * kUpdTok;
constexpr int kCTile = 32;              // centroid rows per shared-memory tile
constexpr int kCStride = kHeadDim + 1;  // padded row: lane j reads row j without conflicts
constexpr int kMaxNew = 1024;           // new tokens per sequence and call

// cache row of token `pos` of (sequence b, KV head kv), in elements
__device__ __forceinline__ long long row_offset(const Plan& pl, const int32_t* __restrict__ bt,
                                                int pos, int kv, long long stride_page,
                                                long long stride_token, long long stride_head) {
  const int page = __ldg(bt + pos / pl.page_size);
  return (long long)page * stride_page + (long long)(pos % pl.page_size) * stride_token +
         (long long)kv * stride_head;
}

template <typename T, int DSUB>
__global__ void __launch_bounds__(kUpdThreads)
index_encode_kernel(Plan pl, const T* __restrict__ kc, long long stride_page, long long stride_token,
                    long long stride_head, const int32_t* __restrict__ block_table,
                    const int32_t* __restrict__ first_pos, const int32_t* __restrict__ n_new,
                    int max_new, const float* __restrict__ centroids,
                    const float* __restrict__ codebooks, uint8_t* __restrict__ codes,
                    uint16_t* __restrict__ list_ids, float* __restrict__ key_norms) {
  __shared__ float s_u[kUpdTok][kHeadDim];          // direction, later the residual
  __shared__ float s_c[kCTile][kCStride];
  __shared__ int s_a[kUpdTok];
  __shared__ uint8_t s_code[kUpdTok][64];
  const int kv = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  pdl_wait();
  pdl_launch_dependents();
  const int nb = min(max(n_new[b], 0), max_new);
  const int t0 = blockIdx.x * kUpdTok;
  if (t0 >= nb) return;
  const int ntok = min(kUpdTok, nb - t0);
  const int p0 = first_pos[b] + t0;                 // position of this CTA's first token
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;
  // tokens whose position falls outside the index rows are left alone
  const bool mine_ok = warp < ntok && p0 + warp >= 0 && p0 + warp < pl.N_max;

  // ---- norm and direction: warp w <-> token w, a lane holds 4 of the 128 dims
  {
    float x[4] = {0.f, 0.f, 0.f, 0.f};
    if (mine_ok) {
      const T* row = kc + row_offset(pl, bt, p0 + warp, kv, stride_page, stride_token, stride_head);
#pragma unroll
      for (int i = 0; i < 4; ++i) x[i] = Unpack<T>::one(row[4 * lane + i]);
    }
    const float ss = warp_sum(x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3]);
    const float r = sqrtf(ss);
    const float inv = r > 0.f ? 1.f / r : 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) s_u[warp][4 * lane + i] = x[i] * inv;
    if (mine_ok && lane == 0) key_norms[ukv * pl.N_max + p0 + warp] = r;
  }

  // ---- nearest centroid: |u - c|^2 = |u|^2 - 2 u.c + |c|^2, the first term is common
  float best_d = CUDART_INF_F;
  int best_j = 0;
  const float* cbase = centroids + ukv * (size_t)pl.n_list * kHeadDim;
  for (int c0 = 0; c0 < pl.n_list; c0 += kCTile) {
    __syncthreads();                                // previous tile consumed, s_u complete
    for (int i = tid; i < kCTile * (kHeadDim / 4); i += kUpdThreads) {
      const int rr = i / (kHeadDim / 4), c4 = i % (kHeadDim / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c0 + rr < pl.n_list)
        v = __ldg(reinterpret_cast<const float4*>(cbase + (size_t)(c0 + rr) * kHeadDim) + c4);
      s_c[rr][4 * c4] = v.x; s_c[rr][4 * c4 + 1] = v.y;
      s_c[rr][4 * c4 + 2] = v.z; s_c[rr][4 * c4 + 3] = v.w;
    }
    __syncthreads();
    float dot = 0.f, cn = 0.f;
#pragma unroll 8
    for (int d = 0; d < kHeadDim; ++d) {
      const float c = s_c[lane][d];
      dot = fmaf(s_u[warp][d], c, dot);
      cn = fmaf(c, c, cn);
    }
    const float dist = fmaf(-2.f, dot, cn);
    if (c0 + lane < pl.n_list && dist < best_d) { best_d = dist; best_j = c0 + lane; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float od = __shfl_xor_sync(0xffffffffu, best_d, o);
    const int oj = __shfl_xor_sync(0xffffffffu, best_j, o);
    if (od < best_d || (od == best_d && oj < best_j)) { best_d = od; best_j = oj; }
  }
  if (lane == 0) {
    s_a[warp] = best_j;
    if (mine_ok) list_ids[ukv * pl.N_max + p0 + warp] = (uint16_t)best_j;
  }
  // ---- residual, in place
  {
    const float4 c = __ldg(reinterpret_cast<const float4*>(cbase + (size_t)best_j * kHeadDim) + lane);
    s_u[warp][4 * lane] -= c.x; s_u[warp][4 * lane + 1] -= c.y;
    s_u[warp][4 * lane + 2] -= c.z; s_u[warp][4 * lane + 3] -= c.w;
  }
  __syncthreads();

  // ---- codes: warp <-> subspaces m = warp, warp + 8, ...; lane <-> codewords lane + 32 i
  for (int m = warp; m < pl.M; m += kUpdTok) {
    float bd[kUpdTok];
    int bz[kUpdTok];
#pragma unroll
    for (int t = 0; t < kUpdTok; ++t) { bd[t] = CUDART_INF_F; bz[t] = 0; }
    const float* cb = codebooks + (ukv * pl.M + m) * (size_t)pl.n_code * DSUB;
    for (int z0 = 0; z0 < pl.n_code; z0 += 32) {
      const int z = min(z0 + lane, pl.n_code - 1);      // lanes past the codebook repeat its last word
      float p[DSUB];
      if constexpr (DSUB == 2) {
        const float2 v = __ldg(reinterpret_cast<const float2*>(cb + (size_t)z * DSUB));
        p[0] = v.x; p[1] = v.y;
      } else {
#pragma unroll
        for (int c4 = 0; c4 < DSUB / 4; ++c4) {
          const float4 v = __ldg(reinterpret_cast<const float4*>(cb + (size_t)z * DSUB) + c4);
          p[4 * c4] = v.x; p[4 * c4 + 1] = v.y; p[4 * c4 + 2] = v.z; p[4 * c4 + 3] = v.w;
        }
      }
#pragma unroll
      for (int t = 0; t < kUpdTok; ++t) {
        float dist = 0.f;
#pragma unroll
        for (int dd = 0; dd < DSUB; ++dd) {
          const float e = s_u[t][m * DSUB + dd] - p[dd];
          dist = fmaf(e, e, dist);
        }
        if (dist < bd[t]) { bd[t] = dist; bz[t] = z; }      // z ascends: first minimum stays
      }
    }
#pragma unroll
    for (int t = 0; t < kUpdTok; ++t) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float od = __shfl_xor_sync(0xffffffffu, bd[t], o);
        const int oz = __shfl_xor_sync(0xffffffffu, bz[t], o);
        if (od < bd[t] || (od == bd[t] && oz < bz[t])) { bd[t] = od; bz[t] = oz; }
      }
      if (lane == 0) s_code[t][m] = (uint8_t)bz[t];
    }
  }
  __syncthreads();
  // one byte per code, or two 4-bit codes per byte (subspace 2j in the low nibble of byte j)
  for (int i = tid; i < ntok * pl.code_bytes; i += kUpdThreads) {
    const int t = i / pl.code_bytes, j = i - t * pl.code_bytes;
    const int pos = p0 + t;
    const uint8_t byte = pl.n_code == 16 ? (uint8_t)(s_code[t][2 * j] | (s_code[t][2 * j + 1] << 4))
                                         : s_code[t][j];
    if (pos >= 0 && pos < pl.N_max) codes[(ukv * pl.N_max + pos) * pl.code_bytes + j] = byte;
  }
}

template <typename T>
__global__ void __launch_bounds__(kUpdThreads)
index_refresh_means_kernel(Plan pl, const T* __restrict__ vc, long long stride_page,
                           long long stride_token, long long stride_head,
                           const int32_t* __restrict__ block_table,
                           const int32_t* __restrict__ first_pos, const int32_t* __restrict__ n_new,
                           int max_new, const uint16_t* __restrict__ list_ids,
                           float* __restrict__ list_vmeans, int32_t* __restrict__ list_counts) {
  __shared__ uint16_t s_lid[kMaxNew];
  __shared__ int s_lead[kMaxNew];
  __shared__ uint32_t s_nlead;
  const int kv = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  pdl_wait();                                        // the list ids come from the encode kernel
  pdl_launch_dependents();
  const int p0 = first_pos[b];
  int nb = min(max(n_new[b], 0), max_new);
  if (p0 < 0) nb = 0;
  nb = min(nb, pl.N_max - p0);                       // same positions as the encode kernel
  if (nb <= 0) return;
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;
  for (int t = tid; t < nb; t += kUpdThreads) s_lid[t] = list_ids[ukv * pl.N_max + p0 + t];
  if (tid == 0) s_nlead = 0u;
  __syncthreads();
  // leaders: the first new token of every list that received one
  for (int t = tid; t < nb; t += kUpdThreads) {
    const uint16_t j = s_lid[t];
    bool first = true;
    for (int e = 0; e < t; ++e) first = first && (s_lid[e] != j);
    if (first) s_lead[atomicAdd(&s_nlead, 1u)] = t;
  }
  __syncthreads();
  const int n_lead = (int)s_nlead;
  for (int l = warp; l < n_lead; l += kUpdTok) {
    const int t_first = s_lead[l];
    const int j = s_lid[t_first];
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    int cnt = 0;
    for (int t = t_first; t < nb; ++t) {             // token order: the sum is deterministic
      if (s_lid[t] != j) continue;                   // warp-uniform
      const T* row = vc + row_offset(pl, bt, p0 + t, kv, stride_page, stride_token, stride_head);
      sum.x += Unpack<T>::one(row[4 * lane]);     sum.y += Unpack<T>::one(row[4 * lane + 1]);
      sum.z += Unpack<T>::one(row[4 * lane + 2]); sum.w += Unpack<T>::one(row[4 * lane + 3]);
      ++cnt;
    }
    float4* mean = reinterpret_cast<float4*>(list_vmeans + (ukv * pl.n_list + j) * kHeadDim) + lane;
    const int n_old = list_counts[ukv * pl.n_list + j];
    const float w_old = (float)n_old, inv = 1.f / (float)(n_old + cnt);
    float4 v = *mean;
    v.x = (w_old * v.x + sum.x) * inv; v.y = (w_old * v.y + sum.y) * inv;
    v.z = (w_old * v.z + sum.z) * inv; v.w = (w_old * v.w + sum.w) * inv;
    *mean = v;
    __syncwarp();
    if (lane == 0) list_counts[ukv * pl.n_list + j] = n_old + cnt;
  }
}

template <typename T>
cudaError_t launch_update_t(const Plan& pl, const pqhsa_index_rw& ix, const pqhsa_paged_kv& kv,
                            const int32_t* first_pos, const int32_t* n_new, int max_new,
                            cudaStream_t st) {
  const dim3 grid((max_new + kUpdTok - 1) / kUpdTok, pl.Hkv, pl.B), block(kUpdThreads);
  const T* kc = static_cast<const T*>(kv.k_cache);
  const T* vc = static_cast<const T*>(kv.v_cache);
  cudaError_t e;
#define PQHSA_UPD_CASE(D)                                                                       \
  case D:                                                                                       \
    e = launch_pdl(index_encode_kernel<T, D>, grid, block, 0, st, pl, kc,                       \
                   (long long)kv.stride_page, (long long)kv.stride_token,                       \
                   (long long)kv.stride_head, kv.block_table, first_pos, n_new, max_new,        \
                   ix.centroids, ix.codebooks, ix.codes, ix.list_ids, ix.key_norms);            \
    break;
  switch (pl.dsub) {
    PQHSA_UPD_CASE(2) PQHSA_UPD_CASE(4) PQHSA_UPD_CASE(8) PQHSA_UPD_CASE(16)
    default: return cudaErrorInvalidValue;
  }
#undef PQHSA_UPD_CASE
  if (e != cudaSuccess) return e;
  return launch_pdl(index_refresh_means_kernel<T>, dim3(pl.Hkv, pl.B), block, 0, st, pl, vc,
                    (long long)kv.stride_page, (long long)kv.stride_token,
                    (long long)kv.stride_head, kv.block_table, first_pos, n_new, max_new,
                    static_cast<const uint16_t*>(ix.list_ids), ix.list_vmeans, ix.list_counts);
}

}  // namespace
}  // namespace pqhsa

using namespace pqhsa;

extern "C" int pqhsa_index_update(const pqhsa_params* params, const pqhsa_index_rw* index,
                                  const pqhsa_paged_kv* kv, const int32_t* first_pos,
                                  const int32_t* n_new, int32_t max_new, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (index == nullptr || kv == nullptr || first_pos == nullptr || n_new == nullptr ||
      index->centroids == nullptr || index->codebooks == nullptr || index->codes == nullptr ||
      index->list_ids == nullptr || index->key_norms == nullptr || index->list_vmeans == nullptr ||
      index->list_counts == nullptr || kv->k_cache == nullptr || kv->v_cache == nullptr ||
      kv->block_table == nullptr || max_new < 0 || max_new > kMaxNew)
    return PQHSA_ERR_INVALID_ARG;
  if (kv->stride_page % 8 || kv->stride_token % 8 || kv->stride_head % 8) return PQHSA_ERR_UNSUPPORTED;
  if (max_new == 0) return PQHSA_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const cudaError_t e =
      pl.dtype == PQHSA_F16
          ? launch_update_t<__half>(pl, *index, *kv, first_pos, n_new, max_new, st)
          : launch_update_t<__nv_bfloat16>(pl, *index, *kv, first_pos, n_new, max_new, st);
  return e == cudaSuccess ? PQHSA_OK : PQHSA_ERR_CUDA;
}
