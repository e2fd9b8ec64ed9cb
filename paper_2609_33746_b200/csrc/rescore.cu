// fp16 lookup tables with an fp32 re-score of the near-threshold tokens (an IVF-PQ fast-scan
// refinement carried over to the scan of Sec. 3.1; the selection rule is still Eq. 3).
//
// With fp16 tables every approximate score s~_i carries an error of at most
//     eps = r_max * (E * 2^-9 + M * 2^-24),   E = sum_m max_z |LUT[z][m]|,
// (entry rounding 2^-11 and two levels of fp16 additions per group of four entries, all
// relative to the entries' magnitudes; r_max the largest key norm of the row's tokens, which
// the scan records per segment; the second term covers entries below the fp16 normal range).
// Let t~ be the k-th largest approximate score.  Then every token with s~ > t~ + 2 eps is in
// the top-k of the fp32-table scores and no token with s~ < t~ - 2 eps is, so the fp32
// selection is: those certain tokens plus the best of the POOL { |s~ - t~| <= 2 eps } by their
// fp32-table score (ties: lower position), as many as the approximate selection took from the
// pool.  The pool is a few dozen tokens per row; the kernel finds it in the top-k's candidate
// list (or, when that list does not reach down to t~ - 2 eps, in the score row itself),
// re-scores it from the fp32 tables in global memory, and swaps losers for gainers in sel_idx.
// kth_score becomes the exact k-th largest fp32-table score.  The score rows keep the
// approximate values: the list sums were formed from them, and the background preparation
// takes out of a list exactly what the scan put in.
#include "common.cuh"

namespace pqhsa {

namespace {

constexpr int kRsThreads = 512;
constexpr int kRsWarps = kRsThreads / 32;
constexpr int kPoolCap = 1024;
constexpr int kRsCodes = 256;      // codewords per subspace in this mode
constexpr int kRsM = 32;           // subspaces in this mode (one lane each)
constexpr int kTieCap = 64;        // pool tokens AT the approximate threshold looked up in sel_idx

__global__ void __launch_bounds__(kRsThreads)
rescore_kernel(Plan pl, const float* __restrict__ lut, const float* __restrict__ coarse,
               const uint8_t* __restrict__ codes, const uint16_t* __restrict__ lids,
               const float* __restrict__ norms, const float* __restrict__ scores,
               const int32_t* __restrict__ seq_lens, const uint32_t* __restrict__ counters,
               const int32_t* __restrict__ rowstate, const uint2* __restrict__ cand,
               int32_t* __restrict__ sel_idx, float* __restrict__ kth, int* __restrict__ status) {
  __shared__ float s_wmax[kRsWarps][kRsM];
  __shared__ int s_pos[kPoolCap + 8], s_lose[kPoolCap], s_gain[kPoolCap], s_tie[kTieCap];
  __shared__ float s_apx[kPoolCap], s_ex[kPoolCap + 8];
  __shared__ unsigned char s_had[kPoolCap];
  __shared__ uint32_t s_np, s_nt, s_nsel, s_nl, s_ng, s_kmin;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = row / pl.Hq, h = row % pl.Hq;
  const int kv = h / pl.G, hg = (h % pl.G) / pl.Gc, g = (h % pl.G) % pl.Gc;
  const int Gc = pl.Gc, n_list = pl.n_list;
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  const size_t unit = ukv * pl.n_hg + hg;
  const float* lut_u = lut + unit * (size_t)kRsCodes * kRsM * Gc;  // [z][m][g]
  const float* co_u = coarse + unit * (size_t)n_list * Gc;
  const size_t row_base = ukv * (size_t)pl.N_max;

  // ---- before the wait for the top-k: the error bound of this row.  The tables and the
  // segment norms come from kernels that are complete when any CTA of this one runs (every CTA
  // of every kernel in between waits for its predecessor before it lets its dependents go).
  // lane = subspace: a warp reads the 512 contiguous bytes of one codeword row [m][g] per load,
  // 32 rows per lane in flight; then the maxima of the eight warps are combined per subspace
  {
    float v[kRsCodes / kRsWarps];
#pragma unroll
    for (int zz = 0; zz < kRsCodes / kRsWarps; ++zz)
      v[zz] = __ldg(lut_u + ((size_t)(zz * kRsWarps + warp) * kRsM + lane) * Gc + g);
    float x = 0.f;
#pragma unroll
    for (int zz = 0; zz < kRsCodes / kRsWarps; ++zz) x = fmaxf(x, fabsf(v[zz]));
    s_wmax[warp][lane] = x;
  }
  if (tid == 0) { s_np = 0u; s_nt = 0u; s_nsel = 0u; s_nl = 0u; s_ng = 0u; s_kmin = 0xffffffffu; }
  float r_max = 0.f;
  {
    const ScanSplit sp = scan_split(seq_lens, pl.B, pl.N_max, pl.upb, pl.scan_ctas);
    const int tb = seq_tiles(seq_lens, b, pl.N_max);
    if (tb > 0 && sp.T > 0) {
      long long base = 0;
      for (int bb = 0; bb < b; ++bb) base += (long long)seq_tiles(seq_lens, bb, pl.N_max) * pl.upb;
      const long long s_u = base + (long long)(kv * pl.n_hg + hg) * tb;
      const int c_first = split_cta_of(sp, s_u);
      const int nseg = min(kMaxSeg, split_cta_of(sp, s_u + tb - 1) - c_first + 1);
      for (int sgm = lane; sgm < nseg; sgm += 32)
        r_max = fmaxf(r_max, __ldcg(pl.norm_seg + unit * pl.n_part + sgm));
      r_max = warp_max(r_max);
    }
  }
  __syncthreads();
  float E = 0.f;                                                  // every warp forms the same sum
  {
    float x = 0.f;
#pragma unroll
    for (int w = 0; w < kRsWarps; ++w) x = fmaxf(x, s_wmax[w][lane]);
    E = warp_sum(x);
  }
  const float eps = r_max * (E * 0.001953125f + (float)kRsM * 5.9604645e-8f) * 1.001f;

  pdl_wait();               // (nothing above this line may return)
  pdl_launch_dependents();
  const int4 st = __ldcg(reinterpret_cast<const int4*>(rowstate) + row);
  const uint4 cn = __ldcg(reinterpret_cast<const uint4*>(counters) + row);   // fallbacks, ticket, W, C
  const float kt = __ldcg(kth + row);
  const float lo_f = __int_as_float(st.x), hi_f = __int_as_float(st.y);
  const int k = st.z, n = st.w;
  if (k == 0) return;
  const Region rg = region_of(pl, n, b);
  if (k >= rg.r_end - rg.r_begin) return;                        // all of R is selected anyway
  const float e2 = 2.f * eps + fabsf(kt) * 2e-6f;                // + the rounding of two fp32 evaluations
  const float win_lo = kt - e2, win_hi = kt + e2;
  const float* rs = scores + (size_t)row * pl.N_max;
  int32_t* sel = sel_idx + (size_t)row * pl.k_max;
  const int W = (int)cn.z, C = (int)cn.w;
  const bool covered = cn.x == 0u && W <= k && W + C >= k && C <= pl.cand_cap && lo_f <= win_lo;

  // ---- the pool: position and approximate score of every token in the threshold zone
  // (all 32 lanes call; one shared-memory atomic per warp)
  auto append = [&](bool in_zone, int pos, float s) {
    const unsigned m = __ballot_sync(0xffffffffu, in_zone);
    if (m == 0u) return;
    uint32_t base = 0u;
    if (lane == 0) base = atomicAdd(&s_np, (uint32_t)__popc(m));
    base = __shfl_sync(0xffffffffu, base, 0);
    const uint32_t j = base + __popc(m & ((1u << lane) - 1u));
    if (in_zone && j < (uint32_t)kPoolCap) { s_pos[j] = pos; s_apx[j] = s; }
  };
  if (covered) {
    const uint2* rc = cand + (size_t)row * pl.cand_cap;
    for (int i0 = 0; i0 < C; i0 += 4 * kRsThreads) {
      uint2 it[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kRsThreads + tid;
        it[u] = i < C ? __ldcg(rc + i) : make_uint2(0u, 0u);     // key 0: NaN, never in the zone
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float s = key_score(it[u].x);
        append(s >= win_lo && s <= win_hi, (int)it[u].y, s);
      }
    }
    if (!(hi_f >= win_hi)) {
      // winners (above the bracket, so not in the candidate list) that are not certain
      for (int t0 = 0; t0 < k; t0 += kRsThreads) {
        const int t = t0 + tid;
        const int pos = t < k ? __ldcg(sel + t) : -1;
        const float s = (unsigned)pos < (unsigned)n ? __ldcg(rs + pos) : CUDART_NAN_F;
        append(s > hi_f && s <= win_hi, pos, s);
      }
    }
  } else {
    // the candidate list does not reach down to the zone's lower edge (or the top-k took its
    // fallback path): read the zone off the score row
    for (int i0 = rg.r_begin; i0 < rg.r_end; i0 += 8 * kRsThreads) {
      float sv[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kRsThreads + tid;
        sv[u] = i < rg.r_end ? __ldcg(rs + i) : CUDART_NAN_F;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        append(sv[u] >= win_lo && sv[u] <= win_hi, i0 + u * kRsThreads + tid, sv[u]);
    }
  }
  __syncthreads();
  const int P = (int)s_np;
  if (P > kPoolCap) {
    if (tid == 0) atomicOr(status, kStatusRescoreSkipped);
    return;
  }
  if (P == 0) return;

  // ---- which pool tokens the approximate top-k holds: those above its threshold kt do, those
  // below do not, and the few AT kt (equal scores are taken by position) are looked up in sel_idx
  for (int j0 = 0; j0 < P; j0 += kRsThreads) {
    const int j = j0 + tid;
    const float s = j < P ? s_apx[j] : -CUDART_INF_F;
    if (j < P) s_had[j] = s > kt ? 1 : 0;
    const unsigned above = __ballot_sync(0xffffffffu, s > kt);
    if (lane == 0 && above) atomicAdd(&s_nsel, (uint32_t)__popc(above));
    if (s == kt) {                                   // rare: usually the k-th token alone
      const uint32_t t = atomicAdd(&s_nt, 1u);
      if (t < (uint32_t)kTieCap) s_tie[t] = j;
    }
  }
  __syncthreads();
  const int T = (int)s_nt;
  if (T > kTieCap) {
    if (tid == 0) atomicOr(status, kStatusRescoreSkipped);
    return;
  }
  for (int t = tid; t < k; t += kRsThreads) {
    const int pos = __ldcg(sel + t);
    for (int i = 0; i < T; ++i)
      if (s_pos[s_tie[i]] == pos) { s_had[s_tie[i]] = 1; atomicAdd(&s_nsel, 1u); }
  }

  if (tid < 8) { s_ex[P + tid] = -CUDART_INF_F; s_pos[P + tid] = 0x7fffffff; }   // padding for the ranking
  // ---- fp32-table scores of the pool: a warp takes sixteen tokens at a time, lane = subspace
  constexpr int kPer = 16;
  for (int j0 = warp * kPer; j0 < P; j0 += kRsWarps * kPer) {
    uint32_t z[kPer];
    float v[kPer];
    // lane u < 16 also fetches token u's list id and norm, then its coarse term
    const int my = j0 + lane < P && lane < kPer ? s_pos[j0 + lane] : -1;
    uint32_t lid = 0u;
    float nr = 0.f;
    if (my >= 0) {
      lid = min((uint32_t)__ldg(lids + row_base + my), (uint32_t)(n_list - 1));
      nr = norms ? __ldg(norms + row_base + my) : 1.0f;
    }
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const int pos = j0 + u < P ? s_pos[j0 + u] : -1;
      z[u] = pos >= 0 ? (uint32_t)__ldg(codes + (row_base + pos) * kRsM + lane) : 0xffffffffu;
    }
    const float co = my >= 0 ? __ldg(co_u + (size_t)lid * Gc + g) : 0.f;
#pragma unroll
    for (int u = 0; u < kPer; ++u)
      v[u] = z[u] != 0xffffffffu ? __ldg(lut_u + ((size_t)z[u] * kRsM + lane) * Gc + g) : 0.f;
    float mine = 0.f;
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const float sum = warp_sum(v[u]);                            // same tree for every token
      if (lane == u) mine = sum;
    }
    if (my >= 0) s_ex[j0 + lane] = nr * (co + mine);
  }
  __syncthreads();
  const int p_sel = (int)s_nsel;                                  // >= 1: the k-th token itself is in the pool

  // ---- rank the pool by fp32 score (ties: lower position); the best p_sel are selected.
  // One thread per token; all threads walk the pool together (broadcast reads).
  for (int j0 = 0; j0 < P; j0 += kRsThreads) {
    const int j = min(j0 + tid, P - 1);
    const bool live = j0 + tid < P;
    const float e = s_ex[j];
    const int pos = s_pos[j];
    int rank = 0;
    for (int i = 0; i < P; i += 8) {               // (entries past P hold -inf: they never count)
      float ei[8];
      int pi[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { ei[u] = s_ex[i + u]; pi[u] = s_pos[i + u]; }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        rank += ((ei[u] > e) | ((ei[u] == e) & (pi[u] < pos))) ? 1 : 0;
    }
    const bool take = live && rank < p_sel, had = s_had[j] != 0;
    uint32_t kmin = take ? score_key(e) : 0xffffffffu;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    if (lane == 0 && kmin != 0xffffffffu) atomicMin(&s_kmin, kmin);
    if (live && had && !take) s_lose[atomicAdd(&s_nl, 1u)] = pos;      // a handful per row
    if (live && !had && take) s_gain[atomicAdd(&s_ng, 1u)] = pos;
  }
  __syncthreads();
  const int n_swap = (int)s_nl;
  if (n_swap != (int)s_ng) {                                       // cannot happen: as many in as out
    if (tid == 0) atomicOr(status, kStatusCountMismatch);
    return;
  }
  if (n_swap > 0)
    for (int t = tid; t < k; t += kRsThreads) {
      const int pos = __ldcg(sel + t);
      for (int i = 0; i < n_swap; ++i)
        if (s_lose[i] == pos) sel[t] = s_gain[i];
    }
  if (tid == 0) kth[row] = key_score(s_kmin);
}

}  // namespace

cudaError_t launch_rescore(const Plan& pl, const WsLayout& L, char* ws, const pqhsa_index& ix,
                           const float* lut, const float* coarse, const float* scores,
                           const int32_t* seq_lens, int32_t* sel_idx, const int32_t* sel_count,
                           float* kth, cudaStream_t st) {
  (void)sel_count;
  Plan plan = pl;
  plan.norm_seg = reinterpret_cast<float*>(ws + L.norm_seg);
  return launch_pdl(rescore_kernel, dim3(pl.rows), dim3(kRsThreads), 0, st, plan, lut, coarse,
                    ix.codes, ix.list_ids, ix.key_norms, scores, seq_lens,
                    reinterpret_cast<const uint32_t*>(ws + L.counters),
                    reinterpret_cast<const int32_t*>(ws + L.rowstate),
                    reinterpret_cast<const uint2*>(ws + L.cand), sel_idx, kth,
                    reinterpret_cast<int*>(ws + L.status));
}

}  // namespace pqhsa
