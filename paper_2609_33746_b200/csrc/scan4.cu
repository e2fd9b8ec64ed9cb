// Step 2 of the decode operator for 4-bit codes: the ADC scan (Eq. 2) with the fused per-list
// reduction (Sec. 3.3), in the paper's own index setting (App. A: eight 16-dim subspaces of
// four bits, 4 bytes of codes per token and KV head).
//
// A token is then 4 (M = 8) or 8 (M = 16) bytes of codes, a norm and a list id: 10 bytes read
// and 4 * G bytes of scores written, against 8 table reads.  The kernel is laid out around that
// record size, not around the 8-bit kernel's:
//   * a lane owns FOUR consecutive tokens per iteration, so every global access is one 16-byte
//     (codes, norms, one score row) or 8-byte (list ids) vector per lane, fully coalesced over
//     the warp, and the next iteration's three loads are in flight while this one computes.
//     No shared-memory staging of the codes at all;
//   * the lookup table of a head group is 16 * M entries of 16 bytes (2 KB at M = 8) in the
//     layout [z][m][g]; at step s a lane looks up subspace m = s ^ (lane & 7), so the bank group
//     depends on m only and every 16-byte read is conflict free, as in the 8-bit kernel.  The
//     address is formed with two instructions: a rotate that brings nibble m to the row-index
//     bits, and one and-or with the lane's entry offset (the table is aligned to its size);
//   * the coarse table has one 128-byte row per list holding the entry once per lane of a
//     quarter warp (half warp, warp for Gc = 2, 1), so the random per-token read never has a
//     bank conflict; lists beyond what shared memory holds fall back to one entry per list;
//   * per-list exp-sums: one vector reduction per token into the CTA's partial in global memory
//     (L2), exactly as in the 8-bit kernel, with the same reference / rebuild rule.
// What bounds it: the load/store data pipe again (table reads 32 wavefronts per 32 tokens, the
// scattered reduction about 17, stores, coarse reads and loads about 14), at roughly a third
// of the 8-bit kernel's time.
#include "scan_common.cuh"

namespace pqhsa {

namespace {

constexpr int kTok4 = 4;                         // consecutive tokens per lane and iteration
constexpr int kWarpTok = 32 * kTok4;             // 128 tokens per warp and iteration
constexpr int kStepTok4 = (kScanThreads / 32) * kWarpTok;

template <int GC> struct Packed {               // the Gc values of a token, two per 64-bit word
  static constexpr int kW = GC == 4 ? 2 : 1;
  unsigned long long v[kW];
};
__device__ __forceinline__ unsigned long long pk2(float a, float b) {
  return (unsigned long long)__float_as_uint(a) | ((unsigned long long)__float_as_uint(b) << 32);
}
__device__ __forceinline__ float lo32(unsigned long long v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float hi32(unsigned long long v) { return __uint_as_float((uint32_t)(v >> 32)); }
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b,
                                                   unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
template <int GC> __device__ __forceinline__ void lds_entry(Packed<GC>& p, uint32_t saddr) {
  if constexpr (GC == 4)
    asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(p.v[0]), "=l"(p.v[1]) : "r"(saddr));
  else if constexpr (GC == 2)
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(p.v[0]) : "r"(saddr));
  else {
    uint32_t w;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(saddr));
    p.v[0] = w;
  }
}
template <int GC> __device__ __forceinline__ void ldg_entry(Packed<GC>& p, const float* q) {
  if constexpr (GC == 4) {
    const float4 f = __ldg(reinterpret_cast<const float4*>(q));
    p.v[0] = pk2(f.x, f.y); p.v[1] = pk2(f.z, f.w);
  } else if constexpr (GC == 2) {
    const float2 f = __ldg(reinterpret_cast<const float2*>(q));
    p.v[0] = pk2(f.x, f.y);
  } else {
    p.v[0] = pk2(__ldg(q), 0.f);
  }
}

// One iteration's inputs of a lane: the records of its four tokens.
template <int CW> struct Records {
  uint32_t code[kTok4 * CW];     // CW words of codes per token
  float norm[kTok4];
  uint32_t lid2[2];              // four 16-bit list ids
};

template <int CW>
__device__ __forceinline__ void load_records(Records<CW>& r, const uint8_t* __restrict__ code_row,
                                             const float* __restrict__ norm_row,
                                             const uint16_t* __restrict__ lid_row, int i4, bool ok) {
#pragma unroll
  for (int j = 0; j < kTok4 * CW; ++j) r.code[j] = 0u;
#pragma unroll
  for (int k = 0; k < kTok4; ++k) r.norm[k] = 0.f;
  r.lid2[0] = r.lid2[1] = 0u;
  if (ok) {
#pragma unroll
    for (int c = 0; c < CW; ++c) {
      const uint4 w = __ldg(reinterpret_cast<const uint4*>(code_row + (size_t)i4 * (4 * CW)) + c);
      r.code[4 * c] = w.x; r.code[4 * c + 1] = w.y; r.code[4 * c + 2] = w.z; r.code[4 * c + 3] = w.w;
    }
    if (norm_row) {
      const float4 f = __ldg(reinterpret_cast<const float4*>(norm_row + i4));
      r.norm[0] = f.x; r.norm[1] = f.y; r.norm[2] = f.z; r.norm[3] = f.w;
    } else {
#pragma unroll
      for (int k = 0; k < kTok4; ++k) r.norm[k] = 1.0f;
    }
    const uint2 l = __ldg(reinterpret_cast<const uint2*>(lid_row + i4));
    r.lid2[0] = l.x; r.lid2[1] = l.y;
  }
}

// coarse_mode: 0 = read from global memory, 1 = one entry per list in shared memory,
// 2 = one 128-byte row per list in shared memory (the entry once per lane of the access group).
template <int M, int GC>
__global__ void __launch_bounds__(kScanThreads, 1)
scan4_kernel(Plan pl, const uint8_t* __restrict__ codes, const uint16_t* __restrict__ lids,
             const float* __restrict__ norms, const float* __restrict__ lut,
             const float* __restrict__ coarse, const int32_t* __restrict__ seq_lens,
             float* __restrict__ scores, float* __restrict__ partials, int* __restrict__ status) {
  constexpr int kCW = M / 8;                          // 32-bit words of codes per token
  constexpr int kLutFloats = 16 * M * GC;
  constexpr int kEntryBytes = GC * 4;
  constexpr int kRowBytes = M * kEntryBytes;          // stride between consecutive z
  constexpr int kRowShift = (M == 8 ? 3 : 4) + (GC == 4 ? 4 : GC == 2 ? 3 : 2);   // log2(kRowBytes)
  static_assert((1 << kRowShift) == kRowBytes, "row stride");
  constexpr uint32_t kRowMask = 15u << kRowShift;
  constexpr int kRep = 128 / kEntryBytes;             // lanes of one shared-memory access group
  constexpr int kW = Packed<GC>::kW;
  constexpr int kWarps = kScanThreads / 32;

  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ float s_red[kWarps][GC];
  __shared__ float s_ref[GC], s_max[GC];
  __shared__ int s_overflow;
  __shared__ __align__(8) uint64_t s_bar;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = blockIdx.x;
  const int n_list = pl.n_list, N_max = pl.N_max, upb = pl.upb;
  const int coarse_mode = pl.coarse_in_smem;
  // the table is addressed by or-ing the row index into the entry offset: align it to its size
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t lut_u32 = (raw_u32 + (kLutFloats * 4 - 1)) & ~uint32_t(kLutFloats * 4 - 1);
  const uint32_t coarse_u32 = lut_u32 + kLutFloats * 4;
  unsigned char* lut_ptr = smem_raw + (lut_u32 - raw_u32);
  unsigned char* coarse_ptr = lut_ptr + kLutFloats * 4;

  pdl_wait();
  pdl_launch_dependents();
  const ScanSplit sp = scan_split(seq_lens, pl.B, N_max, upb, pl.scan_ctas);
  if (c == 0 && tid == 0) {
    for (int b = 0; b < pl.B; ++b)
      if (seq_lens[b] < 0 || seq_lens[b] > N_max) atomicOr(status, kStatusSeqLen);
  }
  if (c >= sp.P_eff || sp.T == 0) return;
  long long lo = split_start(sp, c);
  const long long hi = split_start(sp, c + 1);

  if (tid == 0) {
    mbar_init(&s_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  uint32_t bar_parity = 0;

  // per-lane constants of the skewed lookup: at step s the lane reads subspace m = s ^ (lane & 7)
  const int lx = lane & 7;
  uint32_t rot[8], ent[8];
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    const int m = s ^ lx;
    rot[s] = uint32_t(4 * m - kRowShift) & 31u;          // rotate right: nibble m -> row-index bits
    ent[s] = lut_u32 + uint32_t(m * kEntryBytes);
  }
  const uint32_t rep_off = uint32_t(lane & (kRep - 1)) * kEntryBytes;
  const unsigned long long l2e2 = pk2(kLog2e, kLog2e);

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
    const Region rg = region_of(pl, Nb, b);   // only R enters top-k and sums
    const int kv = w / pl.n_hg, hg = w % pl.n_hg;
    const size_t ukv = (size_t)b * pl.Hkv + kv;
    const size_t unit = ukv * pl.n_hg + hg;
    const size_t row_base = ukv * (size_t)N_max;             // token row of codes / ids / norms
    const int row0 = b * pl.Hq + kv * pl.G + hg * GC;        // first score row of the group
    const int n_heads = min(GC, pl.G - hg * GC);             // real heads in this head group
    const float* g_coarse = coarse + unit * (size_t)n_list * GC;
    const int seg_begin = t0 * kTile, seg_end = min(Nb, (t0 + cnt) * kTile);
    const int r_lo = max(rg.r_begin, seg_begin);             // tokens of R: [r_lo, r_lo + r_span)
    const unsigned r_span = (unsigned)max(0, min(rg.r_end, seg_end) - r_lo);
    float* part = partials + (unit * pl.n_part + slot) * (size_t)(GC * (n_list + 2));
    float* part_sums = part + 2 * GC;
    const uint8_t* code_row = codes + row_base * (4 * kCW);
    const float* norm_row = norms ? norms + row_base : nullptr;
    const uint16_t* lid_row = lids + row_base;
    float* sc_row[GC];
#pragma unroll
    for (int g = 0; g < GC; ++g) sc_row[g] = scores + (size_t)(row0 + (g < n_heads ? g : 0)) * N_max;

    __syncthreads();   // previous segment's tables are no longer in use
    if (tid == 0) {
      const uint32_t co_bytes = coarse_mode == 1 ? uint32_t(GC * n_list * 4) : 0u;
      mbar_expect_tx(&s_bar, kLutFloats * 4 + co_bytes);
      bulk_g2s(lut_ptr, lut + unit * (size_t)kLutFloats, kLutFloats * 4, &s_bar);
      if (co_bytes) bulk_g2s(coarse_ptr, g_coarse, co_bytes, &s_bar);
      s_overflow = 0;
    }
    if (coarse_mode == 2) {
      // row j: the entry of list j once per lane of the access group
      for (int idx = tid; idx < n_list * kRep; idx += kScanThreads) {
        const int j = idx / kRep;
        Packed<GC> e;
        ldg_entry<GC>(e, g_coarse + (size_t)j * GC);
        if constexpr (GC == 4)
          *reinterpret_cast<ulonglong2*>(coarse_ptr + (size_t)idx * kEntryBytes) = make_ulonglong2(e.v[0], e.v[1]);
        else if constexpr (GC == 2)
          *reinterpret_cast<unsigned long long*>(coarse_ptr + (size_t)idx * kEntryBytes) = e.v[0];
        else
          *reinterpret_cast<uint32_t*>(coarse_ptr + (size_t)idx * kEntryBytes) = (uint32_t)e.v[0];
      }
    }
    for (int i = tid; i < GC * n_list; i += kScanThreads) part_sums[i] = 0.f;

    int i4 = seg_begin + warp * kWarpTok + lane * kTok4;     // this lane's first token
    Records<kCW> cur, nxt;
    load_records<kCW>(cur, code_row, norm_row, lid_row, i4, i4 < seg_end);
    if (!mbar_wait(&s_bar, bar_parity)) atomicOr(status, kStatusCopyTimeout);
    bar_parity ^= 1u;
    __syncthreads();   // partial zeroed, tables landed

    float mx[GC];
    unsigned long long nref2[kW];           // -(reference * log2 e) per head, packed
#pragma unroll
    for (int g = 0; g < GC; ++g) mx[g] = -CUDART_INF_F;
#pragma unroll
    for (int j = 0; j < kW; ++j) nref2[j] = 0ull;
    bool first = true;
    bool more = true;
    while (more) {
      const bool have = i4 < seg_end;                        // per lane
      load_records<kCW>(nxt, code_row, norm_row, lid_row, i4 + kStepTok4, i4 + kStepTok4 < seg_end);
      unsigned long long sc2[kTok4][kW];
#pragma unroll
      for (int k = 0; k < kTok4; ++k) {
        Packed<GC> acc0, acc1;
#pragma unroll
        for (int j = 0; j < kW; ++j) { acc0.v[j] = 0ull; acc1.v[j] = 0ull; }
#pragma unroll
        for (int cw = 0; cw < kCW; ++cw) {
          const uint32_t word = cur.code[k * kCW + cw];     // nibble m = code of subspace 8 cw + m
          Packed<GC> v[8];
#pragma unroll
          for (int s = 0; s < 8; ++s) {
            const uint32_t row = __funnelshift_r(word, word, rot[s]) & kRowMask;
            lds_entry<GC>(v[s], (row | ent[s]) + uint32_t(cw * 8 * kEntryBytes));
          }
#pragma unroll
          for (int s = 0; s < 8; s += 2) {
#pragma unroll
            for (int j = 0; j < kW; ++j) {
              acc0.v[j] = add2(acc0.v[j], v[s].v[j]);
              acc1.v[j] = add2(acc1.v[j], v[s + 1].v[j]);
            }
          }
        }
        // (a list id outside [0, n_list) is an index error, not a reason to read out of bounds)
        PQHSA_DEBUG_CHECK(i4 + k >= seg_end || list_id_ok((cur.lid2[k >> 1] >> (16 * (k & 1))) & 0xffffu, n_list),
                          kStatusListId, status);
        const uint32_t lid = min((cur.lid2[k >> 1] >> (16 * (k & 1))) & 0xffffu, (uint32_t)(n_list - 1));
        Packed<GC> co;
        if (coarse_mode == 2) lds_entry<GC>(co, coarse_u32 + lid * 128u + rep_off);
        else if (coarse_mode == 1) lds_entry<GC>(co, coarse_u32 + lid * uint32_t(kEntryBytes));
        else ldg_entry<GC>(co, g_coarse + (size_t)lid * GC);
        // l~ = r_i * (coarse + sum of table entries); sink and window tokens are attended
        // exactly and tokens past the segment end are not ours: their score is -inf (their
        // norm was read as 0, so the product is finite), the top-k never picks them and they
        // add nothing to the list sums
        const bool in_r = (unsigned)(i4 + k - r_lo) < r_span;
        const float bias = in_r ? 0.f : -CUDART_INF_F;
        // (what the arrays hold past the sequence end is unspecified: no NaN norm may leak in)
        const float nrm = (i4 + k < seg_end) ? cur.norm[k] : 0.f;
        const unsigned long long nn = pk2(nrm, nrm), bb = pk2(bias, bias);
#pragma unroll
        for (int j = 0; j < kW; ++j)
          sc2[k][j] = fma2(add2(add2(acc0.v[j], acc1.v[j]), co.v[j]), nn, bb);
#pragma unroll
        for (int g = 0; g < GC; ++g)
          mx[g] = fmaxf(mx[g], (g & 1) ? hi32(sc2[k][g >> 1]) : lo32(sc2[k][g >> 1]));
      }
      if (have) {
        // one 16-byte store per head: the scores of the lane's four tokens
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          if (g < n_heads) {
            float4 o;
            o.x = (g & 1) ? hi32(sc2[0][g >> 1]) : lo32(sc2[0][g >> 1]);
            o.y = (g & 1) ? hi32(sc2[1][g >> 1]) : lo32(sc2[1][g >> 1]);
            o.z = (g & 1) ? hi32(sc2[2][g >> 1]) : lo32(sc2[2][g >> 1]);
            o.w = (g & 1) ? hi32(sc2[3][g >> 1]) : lo32(sc2[3][g >> 1]);
            *reinterpret_cast<float4*>(sc_row[g] + i4) = o;
          }
        }
      }

      if (first) {
        // reference of the exp-sums: maximum over the first round of the CTA, plus headroom
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          const float v = warp_max(mx[g]);
          if (lane == 0) s_red[warp][g] = v;
        }
        __syncthreads();
        float r[GC];
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          float v = -CUDART_INF_F;
#pragma unroll
          for (int ww = 0; ww < kWarps; ++ww) v = fmaxf(v, s_red[ww][g]);
          const float vr = v + kRefHeadroom;            // (-inf stays -inf)
          r[g] = -(vr * kLog2e);
          if (tid == g) s_ref[g] = vr;                   // header value: same units as the scores
        }
#pragma unroll
        for (int j = 0; j < kW; ++j) nref2[j] = pk2(r[2 * j], GC > 1 ? r[(2 * j + 1) % GC] : 0.f);
        first = false;
      }
      // exp-sums: a token outside R has score -inf and adds exp2(-inf) = 0 (or, against a
      // reference of -inf, a NaN that no comparison below accepts)
#pragma unroll
      for (int k = 0; k < kTok4; ++k) {
        float x[GC];
#pragma unroll
        for (int j = 0; j < kW; ++j) {
          const unsigned long long x2 = fma2(sc2[k][j], l2e2, nref2[j]);
          x[2 * j] = lo32(x2);
          if (2 * j + 1 < GC) x[2 * j + 1] = hi32(x2);
        }
        float xm = x[0];
#pragma unroll
        for (int g = 1; g < GC; ++g) xm = fmaxf(xm, x[g]);
        if (xm > kOverflowGuardLog2) s_overflow = 1;
        if (xm > kScanNegligibleLog2) {
          float e[GC];
#pragma unroll
          for (int g = 0; g < GC; ++g) e[g] = fast_exp2(x[g]);
          const uint32_t lid = min((cur.lid2[k >> 1] >> (16 * (k & 1))) & 0xffffu, (uint32_t)(n_list - 1));
          red_add<GC>(part_sums + lid * GC, e);
        }
      }
      cur = nxt;
      i4 += kStepTok4;
      more = __any_sync(0xffffffffu, i4 < seg_end);
    }

    // segment maximum per head
    __syncthreads();   // s_red free again
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
      // rare: rebuild the partial against the true maximum from the scores just written.
      // The reductions in flight target the same addresses as the clearing stores, so they
      // are fenced first.
      __threadfence();
      __syncthreads();
      for (int i = tid; i < GC * n_list; i += kScanThreads) part_sums[i] = 0.f;
      if (tid < GC) s_ref[tid] = s_max[tid];
      __threadfence();
      __syncthreads();
      // (eight tokens per thread in flight: the pass is a chain of L2 round trips otherwise)
      constexpr int kRb = 8;
      for (int i0 = seg_begin + tid; i0 < seg_end; i0 += kRb * kScanThreads) {
        uint32_t lid[kRb];
        float sv[kRb][GC];
#pragma unroll
        for (int u = 0; u < kRb; ++u) {
          const int i = i0 + u * kScanThreads;
          lid[u] = i < seg_end ? (uint32_t)__ldg(lid_row + i) : 0u;
#pragma unroll
          for (int g = 0; g < GC; ++g)
            sv[u][g] = (g < n_heads && i < seg_end) ? __ldcg(sc_row[g] + i) : -CUDART_INF_F;
        }
#pragma unroll
        for (int u = 0; u < kRb; ++u) {
          float e[GC];
          bool any = false;
#pragma unroll
          for (int g = 0; g < GC; ++g) {
            const float x = fmaf(sv[u][g], kLog2e, -(s_ref[g] * kLog2e));     // -inf outside R
            e[g] = 0.f;
            if (x > kNegligibleLog2) { e[g] = fast_exp2(x); any = true; }
          }
          if (any) red_add<GC>(part_sums + (size_t)min(lid[u], (uint32_t)(n_list - 1)) * GC, e);
        }
      }
    }
    // header: the reference the sums are relative to (same units as the scores) and the
    // segment's maximum; a segment without any token of R has both at -inf
    if (tid < GC) {
      part[tid] = s_max[tid] > -CUDART_INF_F ? s_ref[tid] : -CUDART_INF_F;
      part[GC + tid] = s_max[tid];
    }

    lo += cnt;
    if (lo >= base + (long long)tb * upb) {
      base += (long long)tb * upb;
      ++b;
      while (b < pl.B && seq_tiles(seq_lens, b, N_max) == 0) ++b;
    }
  }
}

template <int M, int GC>
cudaError_t launch_scan4_t(const Plan& pl, const pqhsa_index& ix, const float* lut,
                           const float* coarse, const int32_t* seq_lens, float* scores,
                           float* partials, int* status, cudaStream_t st) {
  const size_t smem = scan4_smem_bytes(pl, pl.coarse_in_smem);
  cudaError_t e = cudaFuncSetAttribute(scan4_kernel<M, GC>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(scan4_kernel<M, GC>, dim3(pl.scan_ctas), dim3(kScanThreads), smem, st, pl,
                    ix.codes, ix.list_ids, ix.key_norms, lut, coarse, seq_lens, scores, partials,
                    status);
}

}  // namespace

// Dynamic shared memory of the 4-bit scan: the table (aligned to its size inside the buffer)
// and the coarse table in the given mode (0: none, 1: one entry per list, 2: a 128-byte row).
size_t scan4_smem_bytes(const Plan& pl, int coarse_mode) {
  const size_t lut = (size_t)16 * pl.M * pl.Gc * 4;
  size_t co = 0;
  if (coarse_mode == 1) co = (size_t)pl.n_list * pl.Gc * 4;
  if (coarse_mode == 2) co = (size_t)pl.n_list * 128;
  return 2 * lut + co;
}

cudaError_t launch_scan4(const Plan& pl, const pqhsa_index& ix, const float* lut,
                         const float* coarse, const int32_t* seq_lens, float* scores,
                         float* list_partials, int* status, cudaStream_t st) {
#define PQHSA_SCAN4_CASE(MM, GG)                                                              \
  if (pl.M == MM && pl.Gc == GG)                                                              \
    return launch_scan4_t<MM, GG>(pl, ix, lut, coarse, seq_lens, scores, list_partials, status, st);
  PQHSA_SCAN4_CASE(8, 1) PQHSA_SCAN4_CASE(8, 2) PQHSA_SCAN4_CASE(8, 4)
  PQHSA_SCAN4_CASE(16, 1) PQHSA_SCAN4_CASE(16, 2) PQHSA_SCAN4_CASE(16, 4)
#undef PQHSA_SCAN4_CASE
  return cudaErrorInvalidValue;
}

}  // namespace pqhsa
