// Step 2 of the decode operator: the ADC scan (Eq. 2) with the fused per-list reduction
// (Sec. 3.3, "code scan with a fused per-list reduction").
//
// One pass over the uint8 codes of a KV head produces the score rows of all Gc query heads
// of a head group.  A persistent CTA keeps the head group's lookup table in shared memory in
// the layout [z][m][g] (fetched with one bulk async copy); a lane owns one token and, at step
// s, looks up subspace m = s ^ (lane & 7).  The shared-memory bank of an entry then depends
// on m only, so the eight lanes of a quarter warp always hit eight different 16-byte bank
// groups whatever the codes are: every 16-byte table read is conflict free.  To keep the byte
// positions static each lane permutes its own code bytes once per token
// (byte p <- byte p ^ (lane & 7)).
//
// Per-list exp-sums: the CTA takes the maximum logit of its first round of tiles (one tile
// per warp) as reference and adds exp(l~ - ref) into a [Gc][n_list] table in shared memory
// while it scans.  When the segment is done the sums are re-based to the segment's true
// maximum and flushed as one partial (maximum + sums) per (score row, CTA segment).  If some
// logit exceeds the reference by so much that exp could overflow, the CTA discards the table
// and rebuilds it in a second pass over the scores it has just written (L2 hits).
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

constexpr float kOverflowGuardLog2 = 96.0f;   // exp2 arguments above this trigger the rebuild
constexpr int kMbarSpinLimit = 1 << 22;

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

// ---- bulk async copy global -> shared, completion on an mbarrier (TMA, no tensor map)
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Bounded wait: returns false if the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (int it = 0; it < kMbarSpinLimit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
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
  constexpr int kBlk = 8;                          // table reads issued back to back

  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* s_lut = reinterpret_cast<float*>(smem_raw);
  float* s_sums = s_lut + kLutFloats;                       // [GC][n_list]
  float* s_coarse = s_sums + GC * pl.n_list;                // [n_list][GC] when it fits
  __shared__ float s_red[kWarps][GC];
  __shared__ float s_ref[GC], s_max[GC];
  __shared__ int s_overflow;
  __shared__ __align__(8) uint64_t s_bar;

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

  if (tid == 0) {
    mbar_init(&s_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  uint32_t bar_parity = 0;

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
    const int tend = t0 + cnt;

    __syncthreads();   // previous segment's tables are no longer in use
    if (tid == 0) {
      const uint32_t lut_bytes_n = kLutFloats * 4;
      const uint32_t co_bytes = pl.coarse_in_smem ? uint32_t(GC * n_list * 4) : 0u;
      mbar_expect_tx(&s_bar, lut_bytes_n + co_bytes);
      bulk_g2s(s_lut, lut + unit * (size_t)kLutFloats, lut_bytes_n, &s_bar);
      if (co_bytes) bulk_g2s(s_coarse, g_coarse, co_bytes, &s_bar);
      s_overflow = 0;
    }
    for (int i = tid; i < GC * n_list; i += kScanThreads) s_sums[i] = 0.f;

    // first tile of this warp: its global loads overlap the table copy
    int t = t0 + warp;
    TokenRec<M> cur;
    load_token<M>(cur, codes, lids, norms, row_base, t * kTile + lane,
                  t < tend && t * kTile + lane < Nb);
    if (!mbar_wait(&s_bar, bar_parity)) atomicOr(status, 4);
    bar_parity ^= 1u;
    __syncthreads();   // s_sums zeroed, tables landed

    float mx[GC], ref2[GC];
#pragma unroll
    for (int g = 0; g < GC; ++g) { mx[g] = -CUDART_INF_F; ref2[g] = 0.f; }
    bool first = true;
    bool more = true;
    while (more) {
      const bool have = t < tend;
      const int tn = t + kWarps;
      TokenRec<M> nxt = cur;
      if (have && tn < tend)
        load_token<M>(nxt, codes, lids, norms, row_base, tn * kTile + lane,
                      tn * kTile + lane < Nb);
      const int i = t * kTile + lane;
      const bool valid = have && i < Nb;
      float sc[GC];
#pragma unroll
      for (int g = 0; g < GC; ++g) sc[g] = -CUDART_INF_F;

      if (have) {
        // position p of the lane's code array <- original byte p ^ (lane & 7)
        uint32_t cw[M / 4];
#pragma unroll
        for (int j = 0; j < M / 8; ++j) {
          const uint32_t a = cur.w[2 * j], bb = cur.w[2 * j + 1];
          cw[2 * j] = __byte_perm(swap_words ? bb : a, 0u, byte_sel);
          cw[2 * j + 1] = __byte_perm(swap_words ? a : bb, 0u, byte_sel);
        }
        float acc0[GC], acc1[GC];
#pragma unroll
        for (int g = 0; g < GC; ++g) { acc0[g] = 0.f; acc1[g] = 0.f; }
#pragma unroll
        for (int sb = 0; sb < M; sb += kBlk) {
          Vec v[kBlk];
#pragma unroll
          for (int u = 0; u < kBlk; ++u) {
            const int s = sb + u;
            const uint32_t z = __byte_perm(cw[s >> 2], 0u, 0x4440u | uint32_t(s & 3));
            const uint32_t off = lane_off[s & 7] + z * uint32_t(kRowBytes) +
                                 uint32_t((s & ~7) * kEntryBytes);
            v[u] = *reinterpret_cast<const Vec*>(lut_bytes + off);
          }
#pragma unroll
          for (int u = 0; u < kBlk; u += 2) {
            vec_add<GC>(acc0, v[u]);
            vec_add<GC>(acc1, v[u + 1]);
          }
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
              sc[g] = cur.norm * (co[g] + (acc0[g] + acc1[g]));
              scores[(size_t)(row0 + g) * N_max + i] = sc[g];
              mx[g] = fmaxf(mx[g], sc[g]);
            }
          }
        }
      }

      if (first) {
        // reference of the exp-sums: maximum over the first round of tiles of the CTA
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          const float v = warp_max(mx[g]);
          if (lane == 0) s_red[warp][g] = v;
        }
        __syncthreads();
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          float v = -CUDART_INF_F;
#pragma unroll
          for (int ww = 0; ww < kWarps; ++ww) v = fmaxf(v, s_red[ww][g]);
          ref2[g] = v * kLog2e;
        }
        if (tid < GC) s_ref[tid] = ref2[tid];
        first = false;
      }
      if (valid) {
        bool over = false;
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          if (g < n_heads) {
            const float x = fmaf(sc[g], kLog2e, -ref2[g]);
            if (x > kOverflowGuardLog2) over = true;
            else if (x > kNegligibleLog2) atomicAdd(&s_sums[g * n_list + cur.lid], fast_exp2(x));
          }
        }
        if (over) s_overflow = 1;
      }
      cur = nxt;
      t = tn;
      more = t < tend;
    }

    // segment maximum per head
    __syncthreads();   // s_red free again, all table updates done
#pragma unroll
    for (int g = 0; g < GC; ++g) {
      const float v = warp_max(mx[g]);
      if (lane == 0) s_red[warp][g] = v;
    }
    __syncthreads();
    if (tid < GC) {
      float v = -CUDART_INF_F;
      for (int ww = 0; ww < kWarps; ++ww) v = fmaxf(v, s_red[ww][tid]);
      s_max[tid] = v;
    }
    __syncthreads();   // also orders this CTA's score stores before the rebuild's loads

    if (s_overflow) {
      // rare: rebuild the table against the true maximum from the scores just written
      for (int i = tid; i < GC * n_list; i += kScanThreads) s_sums[i] = 0.f;
      __syncthreads();
      if (tid < GC) s_ref[tid] = s_max[tid] * kLog2e;
      __syncthreads();
      const int i_begin = t0 * kTile;
      const int i_end = min(Nb, tend * kTile);
      for (int i = i_begin + tid; i < i_end; i += kScanThreads) {
        const uint32_t lid = __ldg(lids + row_base + i);
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          if (g < n_heads) {
            const float s = __ldcg(scores + (size_t)(row0 + g) * N_max + i);
            const float x = fmaf(s, kLog2e, -s_ref[g]);
            if (x > kNegligibleLog2) atomicAdd(&s_sums[g * n_list + lid], fast_exp2(x));
          }
        }
      }
      __syncthreads();
    }
    // flush: header = segment maximum, sums re-based from the reference to that maximum
    for (int idx = tid; idx < n_heads * (n_list + 1); idx += kScanThreads) {
      const int g = idx / (n_list + 1), j = idx - g * (n_list + 1);
      const float rescale = fast_exp2(s_ref[g] - s_max[g] * kLog2e);
      const float v = (j == 0) ? s_max[g] : s_sums[g * n_list + j - 1] * rescale;
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
