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
// The table reads bound the kernel: 16 bytes of shared memory per token, subspace and head
// group against 128 bytes per SM and clock, and the same load/store data pipe also carries
// every other shared or global access of the SM (measured: the kernel runs at one wavefront
// of that pipe per clock).  So everything else is kept as light on that pipe as it can be:
//   * the codes stream from HBM through a per-warp ring of cp.async stages in shared memory
//     (kStages tiles of 32 tokens in flight per warp), so the bytes in flight do not depend on
//     registers; 16-byte chunks are placed with an XOR swizzle that makes the lane-per-token
//     16-byte reads conflict free as well.  Norms and list ids (6 bytes per token) are
//     prefetched one tile ahead in registers;
//   * the per-list exp-sums are not kept in shared memory, where a float atomic is a
//     compare-and-swap loop: the CTA's partial for its segment lives in global memory
//     ([list][head], L2 resident) and every token adds its Gc terms with ONE fire-and-forget
//     vector reduction (red.global.add.v4.f32), resolved in L2.
//
// Per-list exp-sums: the CTA takes the maximum logit of its first round of tiles (one tile
// per warp) as reference ref_s and adds exp(l~ - ref_s) for every token of R.  The partial's
// header keeps ref_s and the segment's true maximum; the consumer (background preparation)
// re-bases the segments of a unit to the row's maximum.  If some logit exceeds the reference
// by so much that exp could overflow, the CTA clears its partial and rebuilds it against the
// true maximum in a second pass over the scores it has just written (L2 hits).
#include "scan_common.cuh"

namespace pqhsa {

struct TokenMeta {
  float norm;          // r_i
  uint32_t lid;        // a_i
};

__device__ __forceinline__ void load_meta(TokenMeta& r, const uint16_t* __restrict__ lids,
                                          const float* __restrict__ norms, size_t row_base, int i,
                                          bool valid) {
  r.lid = 0u;
  r.norm = 0.f;
  if (valid) {
    r.lid = __ldg(lids + row_base + i);
    r.norm = norms ? __ldg(norms + row_base + i) : 1.0f;
  }
}

// ---- per-warp cp.async ring for the code tiles; M here = bytes of codes per token
template <int M> struct CodeTile {
  static constexpr int kChunkBytes = M < 16 ? M : 16;       // one cp.async
  static constexpr int kChunksPerToken = M / kChunkBytes;   // C
  static constexpr int kChunks = kTile * kChunksPerToken;
  static constexpr int kBytes = kTile * M;
  // chunk c of token tok sits at chunk slot c ^ swz(tok): lanes of a quarter warp then read
  // eight different 16-byte bank groups
  static __device__ __forceinline__ int swz(int tok) {
    return (tok * kChunksPerToken >> 3) & (kChunksPerToken - 1);
  }
};

template <int kBytes> __device__ __forceinline__ void cp_async(uint32_t dst, const void* src) {
  if constexpr (kBytes == 16)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
  else if constexpr (kBytes == 8)
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
  else
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() {
  asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Issues the copies of tile t (tokens t*32 .. t*32+31 of the row) into a ring slot.
template <int M>
__device__ __forceinline__ void issue_tile(uint32_t slot, const uint8_t* __restrict__ codes,
                                           size_t row_base, int t, int tend, int Nb, int lane) {
  using CT = CodeTile<M>;
  if (t < tend) {
#pragma unroll
    for (int q0 = 0; q0 < CT::kChunks; q0 += 32) {
      const int q = q0 + lane;
      const int tok = q / CT::kChunksPerToken, c = q % CT::kChunksPerToken;
      const int i = t * kTile + tok;
      if (i < Nb)
        cp_async<CT::kChunkBytes>(slot + tok * M + ((c ^ CT::swz(tok)) * CT::kChunkBytes),
                                  codes + (row_base + i) * M + c * CT::kChunkBytes);
    }
  }
  cp_async_commit();
}

// This lane's token: its code bytes from the ring slot, 4 per register, in original order.
template <int M>
__device__ __forceinline__ void read_codes(uint32_t slot, int lane, uint32_t (&w)[M / 4]) {
  using CT = CodeTile<M>;
  const uint32_t tok_addr = slot + lane * M;
  if constexpr (M == 4) {
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w[0]) : "r"(tok_addr));
  } else if constexpr (M == 8) {
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "r"(tok_addr));
  } else {
#pragma unroll
    for (int c = 0; c < CT::kChunksPerToken; ++c) {
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(w[4 * c]), "=r"(w[4 * c + 1]), "=r"(w[4 * c + 2]), "=r"(w[4 * c + 3])
                   : "r"(tok_addr + ((c ^ CT::swz(lane)) * 16)));
    }
  }
}

// One byte per code, 256-entry tables (4-bit codes: scan4.cu).
// kHalf (M = 32, GC = 4 only): the tables are held in shared memory as fp16 (8 bytes per entry
// of four heads), which halves the table reads that bound the kernel.  The scores are then
// approximate (about 1e-3 relative per table entry instead of 6e-8): an opt-in mode, not the one
// the parity tolerances of the scan stage are stated for.
template <int M, int GC, int kStages, bool kHalf>
__global__ void __launch_bounds__(kScanThreads, 1)
scan_kernel(Plan pl, const uint8_t* __restrict__ codes, const uint16_t* __restrict__ lids,
            const float* __restrict__ norms, const float* __restrict__ lut,
            const float* __restrict__ coarse, const int32_t* __restrict__ seq_lens,
            float* __restrict__ scores, float* __restrict__ partials, int* __restrict__ status) {
  constexpr int kCodes = 256;                         // codewords per subspace
  constexpr int kCB = M;                              // bytes of codes per token
  constexpr int kLutFloats = kCodes * M * GC;
  constexpr int kEntryBytes = GC * 4;
  constexpr int kRowBytes = M * kEntryBytes;       // stride between consecutive z
  constexpr int kWarps = kScanThreads / 32;
  constexpr int kBlk = 8;             // table reads issued back to back

  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* s_lut = reinterpret_cast<float*>(smem_raw);
  float* s_coarse = s_lut + kLutFloats;                     // [n_list][GC] when it fits
  // the code ring sits behind the tables: kStages tiles per warp
  const uint32_t table_bytes =
      uint32_t(kLutFloats + (pl.coarse_in_smem ? GC * pl.n_list : 0)) * 4u;
  const uint32_t ring0 = smem_u32(smem_raw) + ((table_bytes + 127u) & ~127u) +
                         uint32_t((threadIdx.x >> 5) * kStages * CodeTile<kCB>::kBytes);
  __shared__ float s_red[kWarps][GC];
  __shared__ float s_ref[GC], s_max[GC];
  __shared__ int s_overflow;
  __shared__ __align__(8) uint64_t s_bar;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = blockIdx.x;
  const int n_list = pl.n_list, N_max = pl.N_max, upb = pl.upb;

  // The tables come from the kernel right before this one (the table build); everything else
  // this kernel reads is an input of the call, and what it writes (scores, list partials) is
  // read only by later kernels.  Every CTA of the table build waits for ITS predecessors before
  // it releases this grid, so a CTA of this kernel may run ahead of its own dependency wait
  // until it needs the tables: the split, the first code copies, the first token metadata and
  // the clearing of its partial overlap the tail of the table build.
  pdl_launch_dependents();
  bool waited = false;
  const ScanSplit sp = scan_split(seq_lens, pl.B, N_max, upb, pl.scan_ctas);
  if (c >= sp.P_eff || sp.T == 0) {
    pdl_wait();        // (the status word is cleared by the kernel before this one)
    if (c == 0 && tid == 0)
      for (int b = 0; b < pl.B; ++b)
        if (seq_lens[b] < 0 || seq_lens[b] > N_max) atomicOr(status, kStatusSeqLen);
    return;
  }
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
  const uint32_t byte_sel2 = byte_sel + (swap_words ? 0x4444u : 0u);
  uint32_t lane_off[8];   // shared-window address of entry (z = 0, m = t ^ lx) for t = s & 7
#pragma unroll
  for (int t = 0; t < 8; ++t) lane_off[t] = smem_u32(s_lut) + uint32_t((t ^ lx) * kEntryBytes);
  // fp16 tables: 8-byte entries, a half warp per wavefront, so the skew runs over 16 subspaces:
  // at step s the lane reads subspace (s & 16) + ((s & 15) ^ (lane & 15))
  const uint32_t lxs = uint32_t(lane & 15) << 3;
  const uint32_t hsel = 0x3210u ^ (uint32_t(lane & 3) * 0x1111u);      // byte order inside a word
  const bool hswap1 = (lane & 4) != 0, hswap2 = (lane & 8) != 0;        // word order inside 16 bytes
  // the fp16 table (64 KB: 256 rows of 256 bytes) starts at the first 64 KB boundary inside the
  // 128 KB fp32 landing zone, so the lookup address is one xor of the table address, the row
  // index shifted into place and the offsets below 256
  const uint32_t lut_h = (smem_u32(s_lut) + 0xffffu) & ~0xffffu;
  uint2* const s_lut_h = reinterpret_cast<uint2*>(smem_raw + (lut_h - smem_u32(s_lut)));
  const uint32_t lane_h = lut_h ^ lxs;
  static_assert(!kHalf || (M == 32 && GC == 4), "fp16 tables: M = 32, four heads per group");

  // locate the sequence that holds tile `lo`
  int b = 0;
  long long base = 0;
  while (b < pl.B) {
    long long sz = (long long)seq_tiles(seq_lens, b, N_max) * upb;
    if (lo < base + sz) break;
    base += sz;
    ++b;
  }

  [[maybe_unused]] float nmax = 0.f;     // fp16 tables: largest key norm seen in the segment
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
    const int tend = t0 + cnt;
    // this CTA's partial of the unit: header [2 GC] (reference, maximum), sums [n_list][GC]
    float* part = partials + (unit * pl.n_part + slot) * (size_t)(GC * (n_list + 2));
    float* part_sums = part + 2 * GC;

    for (int i = tid; i < GC * n_list; i += kScanThreads) part_sums[i] = 0.f;

    // prologue of the ring: the first kStages-1 tiles of this warp (overlaps the table copy)
    int t = t0 + warp;
#pragma unroll
    for (int st = 0; st < kStages - 1; ++st)
      issue_tile<kCB>(ring0 + st * CodeTile<kCB>::kBytes, codes, row_base, t + st * kWarps, tend,
                      Nb, lane);
    TokenMeta cur;
    load_meta(cur, lids, norms, row_base, t * kTile + lane, t < tend && t * kTile + lane < Nb);
    if (!waited) {                                  // the tables exist from here on
      pdl_wait();
      waited = true;
      if (c == 0 && tid == 0)
        for (int bb = 0; bb < pl.B; ++bb)
          if (seq_lens[bb] < 0 || seq_lens[bb] > N_max) atomicOr(status, kStatusSeqLen);
    }
    __syncthreads();   // previous segment's tables are no longer in use
    if (tid == 0) {
      const uint32_t lut_bytes_n = kLutFloats * 4;
      const uint32_t co_bytes = pl.coarse_in_smem ? uint32_t(GC * n_list * 4) : 0u;
      mbar_expect_tx(&s_bar, lut_bytes_n + co_bytes);
      bulk_g2s(s_lut, lut + unit * (size_t)kLutFloats, lut_bytes_n, &s_bar);
      if (co_bytes) bulk_g2s(s_coarse, g_coarse, co_bytes, &s_bar);
      s_overflow = 0;
    }
    if (!mbar_wait(&s_bar, bar_parity)) atomicOr(status, kStatusCopyTimeout);
    bar_parity ^= 1u;
    __syncthreads();   // partial zeroed, tables landed
    if constexpr (kHalf) {
      // in place: every thread takes its 16 entries into registers, and only when all are read
      // does anybody write the 8-byte versions over the first half of the same memory
      constexpr int kPer = kCodes * M / kScanThreads;
      float4 e[kPer];
#pragma unroll
      for (int u = 0; u < kPer; ++u) e[u] = reinterpret_cast<const float4*>(s_lut)[u * kScanThreads + tid];
      __syncthreads();
#pragma unroll
      for (int u = 0; u < kPer; ++u) {
        const __half2 a = __floats2half2_rn(e[u].x, e[u].y), bq = __floats2half2_rn(e[u].z, e[u].w);
        uint2 w;
        w.x = *reinterpret_cast<const uint32_t*>(&a);
        w.y = *reinterpret_cast<const uint32_t*>(&bq);
        s_lut_h[u * kScanThreads + tid] = w;
      }
      __syncthreads();
    }

    float mx[GC], ref2[GC];
#pragma unroll
    for (int g = 0; g < GC; ++g) { mx[g] = -CUDART_INF_F; ref2[g] = 0.f; }
    bool first = true;
    bool more = true;
    int it = 0;
    while (more) {
      const bool have = t < tend;
      const int tn = t + kWarps;
      __syncwarp();      // every lane is done reading the slot that is refilled next
      issue_tile<kCB>(ring0 + ((it + kStages - 1) % kStages) * CodeTile<kCB>::kBytes, codes, row_base,
                    t + (kStages - 1) * kWarps, tend, Nb, lane);
      TokenMeta nxt;
      load_meta(nxt, lids, norms, row_base, tn * kTile + lane, tn < tend && tn * kTile + lane < Nb);
      cp_async_wait<kStages - 1>();
      __syncwarp();      // the copies of all lanes for tile t have landed
      const int i = t * kTile + lane;
      const bool valid = have && i < Nb;
      const bool in_r = valid && i >= rg.r_begin && i < rg.r_end;
      if constexpr (kHalf) nmax = fmaxf(nmax, cur.norm);
      float sc[GC];
#pragma unroll
      for (int g = 0; g < GC; ++g) sc[g] = -CUDART_INF_F;

      if (have) {
        Acc<GC> acc0, acc1;
        acc0.zero();
        acc1.zero();
        uint32_t raw[M / 4], cw[M / 4];
        read_codes<M>(ring0 + (it % kStages) * CodeTile<M>::kBytes, lane, raw);
        if constexpr (kHalf) {
          // position p of every 16-byte group <- original byte p ^ (lane & 15)
#pragma unroll
          for (int q4 = 0; q4 < M / 16; ++q4) {
            uint32_t r0 = raw[4 * q4], r1 = raw[4 * q4 + 1], r2 = raw[4 * q4 + 2], r3 = raw[4 * q4 + 3];
            if (hswap1) { uint32_t t_ = r0; r0 = r1; r1 = t_; t_ = r2; r2 = r3; r3 = t_; }
            if (hswap2) { uint32_t t_ = r0; r0 = r2; r2 = t_; t_ = r1; r1 = r3; r3 = t_; }
            cw[4 * q4] = __byte_perm(r0, 0u, hsel); cw[4 * q4 + 1] = __byte_perm(r1, 0u, hsel);
            cw[4 * q4 + 2] = __byte_perm(r2, 0u, hsel); cw[4 * q4 + 3] = __byte_perm(r3, 0u, hsel);
          }
          // four lookups are summed in fp16 (two levels), then widened and added in fp32
#pragma unroll
          for (int sb = 0; sb < M; sb += 4) {
            unsigned long long v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int s = sb + u;
              const uint32_t zrow = __byte_perm(cw[s >> 2], 0u, 0x4404u | (uint32_t(s & 3) << 4));   // z << 8
              asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v[u])
                           : "r"(zrow ^ lane_h ^ uint32_t(((s & 15) << 3) | ((s >> 4) << 7))));
            }
            uint32_t lo[4], hi[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { lo[u] = (uint32_t)v[u]; hi[u] = (uint32_t)(v[u] >> 32); }
            uint32_t l01, l23, h01, h23, l4, h4;
            asm("add.rn.f16x2 %0, %1, %2;" : "=r"(l01) : "r"(lo[0]), "r"(lo[1]));
            asm("add.rn.f16x2 %0, %1, %2;" : "=r"(l23) : "r"(lo[2]), "r"(lo[3]));
            asm("add.rn.f16x2 %0, %1, %2;" : "=r"(h01) : "r"(hi[0]), "r"(hi[1]));
            asm("add.rn.f16x2 %0, %1, %2;" : "=r"(h23) : "r"(hi[2]), "r"(hi[3]));
            asm("add.rn.f16x2 %0, %1, %2;" : "=r"(l4) : "r"(l01), "r"(l23));
            asm("add.rn.f16x2 %0, %1, %2;" : "=r"(h4) : "r"(h01), "r"(h23));
            const float2 fl = __half22float2(*reinterpret_cast<const __half2*>(&l4));
            const float2 fh = __half22float2(*reinterpret_cast<const __half2*>(&h4));
            Acc<GC> w;
            w.lo = (unsigned long long)__float_as_uint(fl.x) | ((unsigned long long)__float_as_uint(fl.y) << 32);
            w.hi = (unsigned long long)__float_as_uint(fh.x) | ((unsigned long long)__float_as_uint(fh.y) << 32);
            if (sb & 4) acc1.merge(w); else acc0.merge(w);
          }
        } else {
        // position p of the lane's code array <- original byte p ^ (lane & 7)
#pragma unroll
        for (int j = 0; j < M / 8; ++j) {
          const uint32_t a = raw[2 * j], bb = raw[2 * j + 1];
          cw[2 * j] = __byte_perm(a, bb, byte_sel2);
          cw[2 * j + 1] = __byte_perm(a, bb, byte_sel2 ^ 0x4444u);
        }
#pragma unroll
        for (int sb = 0; sb < M; sb += kBlk) {
          Acc<GC> v[kBlk];
#pragma unroll
          for (int u = 0; u < kBlk; ++u) {
            const int s = sb + u;
            const uint32_t z = __byte_perm(cw[s >> 2], 0u, 0x4440u | uint32_t(s & 3));
            v[u].load(lane_off[s & 7] + z * uint32_t(kRowBytes) + uint32_t((s & ~7) * kEntryBytes));
          }
#pragma unroll
          for (int u = 0; u < kBlk; u += 2) {
            acc0.merge(v[u]);
            acc1.merge(v[u + 1]);
          }
        }
        }
        acc0.merge(acc1);
        float accf[GC], co[GC];
        acc0.get(accf);
        // (a list id outside [0, n_list) is an index error, not a reason to read out of bounds)
        PQHSA_DEBUG_CHECK(!valid || list_id_ok(cur.lid, n_list), kStatusListId, status);
        if (pl.coarse_in_smem) load_vec<GC>(co, s_coarse + min(cur.lid, (uint32_t)(n_list - 1)) * GC);
        else load_vec<GC>(co, g_coarse + min(cur.lid, (uint32_t)(n_list - 1)) * GC);
        if (valid) {
          // sink and window tokens are attended exactly: their score is -inf, so that the
          // top-k never picks them and they add nothing to the list sums
          float* srow = scores + (size_t)row0 * N_max + i;      // row of head 0; heads N_max apart
#pragma unroll
          for (int g = 0; g < GC; ++g) {
            if (g < n_heads) {
              if (in_r) sc[g] = cur.norm * (co[g] + accf[g]);
              srow[g * N_max] = sc[g];
              mx[g] = fmaxf(mx[g], sc[g]);
            }
          }
        }
      }

      if (first) {
        // reference of the exp-sums: maximum over the first round of tiles of the CTA, plus headroom
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
          const float vr = v + kRefHeadroom;            // (-inf stays -inf)
          ref2[g] = vr * kLog2e;
          if (tid == g) s_ref[g] = vr;                   // header value: same units as the scores
        }
        first = false;
      }
      {
        // a token outside R has score -inf and adds exp2(-inf) = 0 (or, against a reference of
        // -inf, a NaN that no comparison below accepts)
        float x[GC], xm = -CUDART_INF_F;
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          x[g] = fmaf(sc[g], kLog2e, -ref2[g]);
          xm = fmaxf(xm, x[g]);
        }
        if (xm > kOverflowGuardLog2) s_overflow = 1;
        if (xm > kScanNegligibleLog2) {
          float e[GC];
#pragma unroll
          for (int g = 0; g < GC; ++g) e[g] = fast_exp2(x[g]);
          red_add<GC>(part_sums + min(cur.lid, (uint32_t)(n_list - 1)) * GC, e);
        }
      }
      cur = nxt;
      t = tn;
      ++it;
      more = t < tend;
    }

    cp_async_wait<0>();
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
      // rare: rebuild the partial against the true maximum from the scores just written.
      // The reductions in flight target the same addresses as the clearing stores, so they
      // are fenced first.
      __threadfence();
      __syncthreads();
      for (int i = tid; i < GC * n_list; i += kScanThreads) part_sums[i] = 0.f;
      if (tid < GC) s_ref[tid] = s_max[tid];
      __threadfence();
      __syncthreads();
      const int i_begin = t0 * kTile;
      const int i_end = min(Nb, tend * kTile);
      // (eight tokens per thread in flight: the pass is a chain of L2 round trips otherwise)
      constexpr int kRb = 8;
      for (int i0 = i_begin + tid; i0 < i_end; i0 += kRb * kScanThreads) {
        uint32_t lid[kRb];
        float sv[kRb][GC];
#pragma unroll
        for (int u = 0; u < kRb; ++u) {
          const int i = i0 + u * kScanThreads;
          lid[u] = i < i_end ? (uint32_t)__ldg(lids + row_base + i) : 0u;
#pragma unroll
          for (int g = 0; g < GC; ++g)
            sv[u][g] = (g < n_heads && i < i_end) ? __ldcg(scores + (size_t)(row0 + g) * N_max + i)
                                                  : -CUDART_INF_F;
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
    if constexpr (kHalf) {
      // largest key norm of the segment: with it the re-score pass bounds the error that the
      // fp16 tables put on any score of the row
      const float v = warp_max(nmax);
      __syncthreads();
      if (lane == 0) s_red[warp][0] = v;
      __syncthreads();
      if (tid == 0 && pl.norm_seg != nullptr) {
        float m = 0.f;
        for (int ww = 0; ww < kWarps; ++ww) m = fmaxf(m, s_red[ww][0]);
        pl.norm_seg[unit * pl.n_part + slot] = m;
      }
      nmax = 0.f;
    }
    // header: the reference the sums are relative to (same units as the scores; the exponent
    // was formed as fma(l~, log2 e, -(ref * log2 e)) in base 2) and the segment's maximum; a
    // segment without any token of R has both at -inf
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

size_t scan_smem_bytes(const Plan& pl, bool coarse_in_smem, int stages) {
  size_t f = (size_t)pl.n_code * pl.M * pl.Gc;
  if (coarse_in_smem) f += (size_t)pl.Gc * pl.n_list;
  const size_t tables = (f * sizeof(float) + 127) / 128 * 128;    // the ring is 128-byte aligned
  return tables + (size_t)(kScanThreads / 32) * stages * kTile * pl.code_bytes;
}

template <int M, int GC, int S, bool kHalf = false>
static cudaError_t launch_scan_t(const Plan& pl, const pqhsa_index& ix, const float* lut,
                                 const float* coarse, const int32_t* seq_lens, float* scores,
                                 float* partials, int* status, cudaStream_t st) {
  const size_t smem = scan_smem_bytes(pl, pl.coarse_in_smem != 0, S);
  cudaError_t e = cudaFuncSetAttribute(scan_kernel<M, GC, S, kHalf>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(scan_kernel<M, GC, S, kHalf>, dim3(pl.scan_ctas), dim3(kScanThreads), smem, st, pl,
                    ix.codes, ix.list_ids, ix.key_norms, lut, coarse, seq_lens, scores, partials,
                    status);
}

cudaError_t launch_scan(const Plan& pl, const pqhsa_index& ix, const float* lut,
                        const float* coarse, const int32_t* seq_lens, float* scores,
                        float* list_partials, int* status, cudaStream_t st) {
  if (pl.n_code == 16)
    return launch_scan4(pl, ix, lut, coarse, seq_lens, scores, list_partials, status, st);
  if (pl.half_tables) {
    if (pl.M != 32 || pl.Gc != 4) return cudaErrorInvalidValue;          // (rejected by make_plan)
    if (pl.scan_stages >= 3)
      return launch_scan_t<32, 4, 3, true>(pl, ix, lut, coarse, seq_lens, scores, list_partials, status, st);
    return launch_scan_t<32, 4, 2, true>(pl, ix, lut, coarse, seq_lens, scores, list_partials, status, st);
  }
#define PQHSA_SCAN_CASE(MM, GG)                                                               \
  if (pl.M == MM && pl.Gc == GG) {                                                            \
    if (pl.scan_stages >= 3)                                                                  \
      return launch_scan_t<MM, GG, 3>(pl, ix, lut, coarse, seq_lens, scores, list_partials,   \
                                      status, st);                                            \
    return launch_scan_t<MM, GG, 2>(pl, ix, lut, coarse, seq_lens, scores, list_partials,     \
                                    status, st);                                              \
  }
  PQHSA_SCAN_CASE(8, 1) PQHSA_SCAN_CASE(8, 2) PQHSA_SCAN_CASE(8, 4)
  PQHSA_SCAN_CASE(16, 1) PQHSA_SCAN_CASE(16, 2) PQHSA_SCAN_CASE(16, 4)
  PQHSA_SCAN_CASE(32, 1) PQHSA_SCAN_CASE(32, 2) PQHSA_SCAN_CASE(32, 4)
  PQHSA_SCAN_CASE(64, 1) PQHSA_SCAN_CASE(64, 2)
#undef PQHSA_SCAN_CASE
  return cudaErrorInvalidValue;
}

}  // namespace pqhsa
