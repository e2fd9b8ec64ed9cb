// Step 2 of the decode operator: the ADC scan (Eq. 2) with the fused per-list reduction
// (Sec. 3.3, "code scan with a fused per-list reduction").
//
// One pass over the uint8 codes of a KV head produces the score rows of all Gc query heads
// of a head group.  A persistent CTA keeps the head group's lookup table in shared memory in
// the layout [z][m][g]; a lane owns one token and, at step s, looks up subspace
// m = s ^ (lane & 7).  The shared-memory bank of an entry then depends on m only, so the
// eight lanes of a quarter warp always hit eight different 16-byte bank groups whatever the
// codes are: every 16-byte table read is conflict free.  To keep the byte positions static
// each lane permutes its own code bytes once per token (byte p <- byte p ^ (lane & 7)).
//
// The per-list exp-sums need a reference logit.  A CTA scans its token range twice: pass A
// computes and stores the scores and the range's maximum per head, pass B re-reads the scores
// it has just written (L2 hits), and adds exp(l~ - max) into a [Gc][n_list] table in shared
// memory, which is flushed as one partial (reference + sums) per (score row, CTA segment).
#include "common.cuh"

namespace pqhsa {

template <int GC> struct VecT;
template <> struct VecT<1> { using type = float; };
template <> struct VecT<2> { using type = float2; };
template <> struct VecT<4> { using type = float4; };

template <int GC> __device__ __forceinline__ void vec_add(float (&acc)[GC],
                                                          const typename VecT<GC>::type& v);
template <> __device__ __forceinline__ void vec_add<1>(float (&a)[1], const float& v) { a[0] += v; }
template <> __device__ __forceinline__ void vec_add<2>(float (&a)[2], const float2& v) {
  a[0] += v.x; a[1] += v.y;
}
template <> __device__ __forceinline__ void vec_add<4>(float (&a)[4], const float4& v) {
  a[0] += v.x; a[1] += v.y; a[2] += v.z; a[3] += v.w;
}

template <int M> struct TokenRec {
  uint32_t w[M / 4];   // code bytes
  float norm;          // r_i
  uint32_t lid;        // a_i
};

template <int M>
__device__ __forceinline__ void load_token(TokenRec<M>& r, const uint8_t* __restrict__ codes,
                                           const uint16_t* __restrict__ lids,
                                           const float* __restrict__ norms, size_t row_base,
                                           int i, bool valid) {
  if (valid) {
    const uint8_t* p = codes + (row_base + i) * M;
    if constexpr (M == 8) {
      uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
      r.w[0] = v.x; r.w[1] = v.y;
    } else {
#pragma unroll
      for (int c = 0; c < M / 16; ++c) {
        uint4 v = __ldg(reinterpret_cast<const uint4*>(p) + c);
        r.w[4 * c + 0] = v.x; r.w[4 * c + 1] = v.y; r.w[4 * c + 2] = v.z; r.w[4 * c + 3] = v.w;
      }
    }
    r.lid = __ldg(lids + row_base + i);
    r.norm = norms ? __ldg(norms + row_base + i) : 1.0f;
  } else {
#pragma unroll
    for (int c = 0; c < M / 4; ++c) r.w[c] = 0u;
    r.lid = 0u;
    r.norm = 0.f;
  }
}

template <int M, int GC>
__global__ void __launch_bounds__(kScanThreads, 1)
scan_kernel(Plan pl, const uint8_t* __restrict__ codes, const uint16_t* __restrict__ lids,
            const float* __restrict__ norms, const float* __restrict__ lut,
            const float* __restrict__ coarse, const int32_t* __restrict__ seq_lens,
            float* __restrict__ scores, float* __restrict__ partials, int* __restrict__ status) {
  using Vec = typename VecT<GC>::type;
  constexpr int kLutFloats = kNCode * M * GC;
  constexpr int kEntryBytes = GC * 4;
  constexpr int kRowBytes = M * kEntryBytes;       // stride between consecutive z
  constexpr int kWarps = kScanThreads / 32;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_lut = reinterpret_cast<float*>(smem_raw);
  float* s_sums = s_lut + kLutFloats;                       // [GC][n_list]
  float* s_coarse = s_sums + GC * pl.n_list;                // [n_list][GC] when it fits
  __shared__ float s_red[kWarps][GC];
  __shared__ float s_ref[GC];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = blockIdx.x;
  const int n_list = pl.n_list, N_max = pl.N_max, upb = pl.upb;

  const ScanSplit sp = scan_split(seq_lens, pl.B, N_max, upb, pl.scan_ctas);
  if (c == 0 && tid == 0) {
    for (int b = 0; b < pl.B; ++b)
      if (seq_lens[b] < 0 || seq_lens[b] > N_max) atomicOr(status, 2);
  }
  if (c >= sp.P_eff || sp.T == 0) return;
  long long lo = split_start(sp, c);
  const long long hi = split_start(sp, c + 1);

  // per-lane constants of the skewed lookup
  const int lx = lane & 7;
  const uint32_t byte_sel = 0x3210u ^ (uint32_t(lane & 3) * 0x1111u);
  const bool swap_words = (lane & 4) != 0;
  const unsigned char* lut_bytes = reinterpret_cast<const unsigned char*>(s_lut);
  uint32_t lane_off[8];   // byte offset of entry (z = 0, m = t ^ lx) for t = s & 7
#pragma unroll
  for (int t = 0; t < 8; ++t) lane_off[t] = uint32_t((t ^ lx) * kEntryBytes);

  // locate the sequence that holds tile `lo`
  int b = 0;
  long long base = 0;
  while (b < pl.B) {
    long long sz = (long long)seq_tiles(seq_lens, b, N_max) * upb;
    if (lo < base + sz) break;
    base += sz;
    ++b;
  }

  while (lo < hi && b < pl.B) {
    const int tb = seq_tiles(seq_lens, b, N_max);
    const int w = (int)((lo - base) / tb);
    const int t0 = (int)((lo - base) - (long long)w * tb);
    const int cnt = (int)min((long long)(tb - t0), hi - lo);
    const int slot = c - split_cta_of(sp, base + (long long)w * tb);
    const int Nb = clamp_len(seq_lens[b], N_max);
    const int kv = w / pl.n_hg, hg = w % pl.n_hg;
    const size_t ukv = (size_t)b * pl.Hkv + kv;
    const size_t unit = ukv * pl.n_hg + hg;
    const size_t row_base = ukv * (size_t)N_max;             // token row of codes / ids / norms
    const int row0 = b * pl.Hq + kv * pl.G + hg * GC;        // first score row of the group
    const int n_heads = min(GC, pl.G - hg * GC);             // real heads in this head group
    const float* g_coarse = coarse + unit * (size_t)n_list * GC;

    __syncthreads();   // previous segment's tables are no longer in use
    {
      const float4* src = reinterpret_cast<const float4*>(lut + unit * (size_t)kLutFloats);
      float4* dst = reinterpret_cast<float4*>(s_lut);
      for (int i = tid; i < kLutFloats / 4; i += kScanThreads) dst[i] = __ldg(src + i);
      for (int i = tid; i < GC * n_list; i += kScanThreads) s_sums[i] = 0.f;
      if (pl.coarse_in_smem)
        for (int i = tid; i < GC * n_list; i += kScanThreads) s_coarse[i] = __ldg(g_coarse + i);
    }
    __syncthreads();

    // ------------------------------------------------------------------ pass A: scores
    float mx[GC];
#pragma unroll
    for (int g = 0; g < GC; ++g) mx[g] = -CUDART_INF_F;
    const int tend = t0 + cnt;
    int t = t0 + warp;
    TokenRec<M> cur;
    if (t < tend) load_token<M>(cur, codes, lids, norms, row_base, t * kTile + lane,
                                t * kTile + lane < Nb);
    while (t < tend) {
      const int tn = t + kWarps;
      TokenRec<M> nxt = cur;
      if (tn < tend) load_token<M>(nxt, codes, lids, norms, row_base, tn * kTile + lane,
                                   tn * kTile + lane < Nb);
      const int i = t * kTile + lane;
      const bool valid = i < Nb;

      // position p of the lane's code array <- original byte p ^ (lane & 7)
      uint32_t cw[M / 4];
#pragma unroll
      for (int j = 0; j < M / 8; ++j) {
        const uint32_t a = cur.w[2 * j], bb = cur.w[2 * j + 1];
        cw[2 * j] = __byte_perm(swap_words ? bb : a, 0u, byte_sel);
        cw[2 * j + 1] = __byte_perm(swap_words ? a : bb, 0u, byte_sel);
      }
      float acc[GC];
#pragma unroll
      for (int g = 0; g < GC; ++g) acc[g] = 0.f;
#pragma unroll
      for (int s = 0; s < M; ++s) {
        const uint32_t z = __byte_perm(cw[s >> 2], 0u, 0x4440u | uint32_t(s & 3));
        const uint32_t off = lane_off[s & 7] + z * uint32_t(kRowBytes) +
                             uint32_t((s & ~7) * kEntryBytes);
        vec_add<GC>(acc, *reinterpret_cast<const Vec*>(lut_bytes + off));
      }
      float co[GC];
#pragma unroll
      for (int g = 0; g < GC; ++g) co[g] = 0.f;
      if (pl.coarse_in_smem)
        vec_add<GC>(co, *reinterpret_cast<const Vec*>(s_coarse + cur.lid * GC));
      else
        vec_add<GC>(co, __ldg(reinterpret_cast<const Vec*>(g_coarse + cur.lid * GC)));
      if (valid) {
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          if (g < n_heads) {
            const float sc = cur.norm * (co[g] + acc[g]);
            scores[(size_t)(row0 + g) * N_max + i] = sc;
            mx[g] = fmaxf(mx[g], sc);
          }
        }
      }
      cur = nxt;
      t = tn;
    }

    // segment maximum per head -> reference of the exp-sums
#pragma unroll
    for (int g = 0; g < GC; ++g) {
      const float v = warp_max(mx[g]);
      if (lane == 0) s_red[warp][g] = v;
    }
    __syncthreads();
    if (tid < GC) {
      float v = -CUDART_INF_F;
      for (int ww = 0; ww < kWarps; ++ww) v = fmaxf(v, s_red[ww][tid]);
      s_ref[tid] = v;
    }
    __syncthreads();   // also orders pass A's score stores before pass B's loads

    // ------------------------------------------------------------------ pass B: list sums
    float ref2[GC];
#pragma unroll
    for (int g = 0; g < GC; ++g) ref2[g] = s_ref[g] * kLog2e;
    const int i_begin = t0 * kTile;
    const int i_end = min(Nb, tend * kTile);
    for (int i = i_begin + tid; i < i_end; i += kScanThreads) {
      const uint32_t lid = __ldg(lids + row_base + i);
#pragma unroll
      for (int g = 0; g < GC; ++g) {
        if (g < n_heads) {
          const float s = __ldcg(scores + (size_t)(row0 + g) * N_max + i);
          const float x = fmaf(s, kLog2e, -ref2[g]);
          if (x > kNegligibleLog2) atomicAdd(&s_sums[g * n_list + lid], fast_exp2(x));
        }
      }
    }
    __syncthreads();
    for (int idx = tid; idx < n_heads * (n_list + 1); idx += kScanThreads) {
      const int g = idx / (n_list + 1), j = idx - g * (n_list + 1);
      const float v = (j == 0) ? s_ref[g] : s_sums[g * n_list + j - 1];
      partials[((size_t)(row0 + g) * pl.n_part + slot) * (n_list + 1) + j] = v;
    }

    lo += cnt;
    if (lo >= base + (long long)tb * upb) {
      base += (long long)tb * upb;
      ++b;
      while (b < pl.B && seq_tiles(seq_lens, b, N_max) == 0) ++b;
    }
  }
}

size_t scan_smem_bytes(const Plan& pl, bool coarse_in_smem) {
  size_t f = (size_t)kNCode * pl.M * pl.Gc + (size_t)pl.Gc * pl.n_list;
  if (coarse_in_smem) f += (size_t)pl.Gc * pl.n_list;
  return f * sizeof(float);
}

template <int M, int GC>
static cudaError_t launch_scan_t(const Plan& pl, const pqhsa_index& ix, const float* lut,
                                 const float* coarse, const int32_t* seq_lens, float* scores,
                                 float* partials, int* status, cudaStream_t st) {
  const size_t smem = scan_smem_bytes(pl, pl.coarse_in_smem != 0);
  cudaError_t e = cudaFuncSetAttribute(scan_kernel<M, GC>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  scan_kernel<M, GC><<<pl.scan_ctas, kScanThreads, smem, st>>>(
      pl, ix.codes, ix.list_ids, ix.key_norms, lut, coarse, seq_lens, scores, partials, status);
  return cudaGetLastError();
}

cudaError_t launch_scan(const Plan& pl, const pqhsa_index& ix, const float* lut,
                        const float* coarse, const int32_t* seq_lens, float* scores,
                        float* list_partials, int* status, cudaStream_t st) {
#define PQHSA_SCAN_CASE(MM, GG)                                                              \
  if (pl.M == MM && pl.Gc == GG)                                                             \
    return launch_scan_t<MM, GG>(pl, ix, lut, coarse, seq_lens, scores, list_partials, status, st);
  PQHSA_SCAN_CASE(8, 1) PQHSA_SCAN_CASE(8, 2) PQHSA_SCAN_CASE(8, 4)
  PQHSA_SCAN_CASE(16, 1) PQHSA_SCAN_CASE(16, 2) PQHSA_SCAN_CASE(16, 4)
  PQHSA_SCAN_CASE(32, 1) PQHSA_SCAN_CASE(32, 2) PQHSA_SCAN_CASE(32, 4)
  PQHSA_SCAN_CASE(64, 1) PQHSA_SCAN_CASE(64, 2)
#undef PQHSA_SCAN_CASE
  return cudaErrorInvalidValue;
}

}  // namespace pqhsa
