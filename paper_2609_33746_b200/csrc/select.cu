// Step 3 of the decode operator: exact top-k over every score row (Eq. 3),
// T(q) = TopK_{k, i in R} l~_i with k = ceil(rho |R|).
//
// Radix threshold select on order-preserving 32-bit keys, digits of 12 / 12 / 8 bits:
//   hist kernel    every CTA histograms the top digit of its 8192-score chunk of a row; the
//                  last CTA of the row to finish finds the digit b1 that holds the k-th key;
//   filter kernel  keys above b1 are winners and are written out at once; keys inside b1
//                  are appended to a candidate list and histogrammed on the second digit;
//                  the last CTA of the row resolves the remaining two digits on the
//                  candidates.
// A CTA keeps its 16 scores per thread in registers, counts, takes its output slots with one
// atomic per list, and writes.  Equal keys at the threshold are taken in order of position
// (lowest first), the stable rule of a full sort.  No CTA ever waits for another: "last CTA"
// is decided by an atomic ticket.
#include "common.cuh"

namespace pqhsa {

namespace {

constexpr int kElems = kSelChunk / kSelThreads;   // scores per thread (16)
constexpr int kStashCap = 2048;

// Largest digit D with  count(digits > D) < k <= count(digits >= D).  `hist` may be global
// (read through L2) or shared.  All kSelThreads threads must call; k >= 1 and the histogram
// must hold at least k items.  Returns D and count(digits > D).
template <bool kGlobal>
__device__ void find_digit(const uint32_t* hist, int nbins, int k, int* s_scan, int& digit,
                           int& above) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (nbins + kSelThreads - 1) / kSelThreads;
  // thread t owns digits [hi - per, hi) with hi = nbins - t*per, walked from the top down
  const int hi = nbins - tid * per;
  uint32_t mine[8];
  uint32_t local = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int d = hi - 1 - j;
    mine[j] = (j < per && d >= 0) ? (kGlobal ? __ldcg(hist + d) : hist[d]) : 0u;
    local += mine[j];
  }
  if (tid == 0) { s_scan[32] = 0; s_scan[33] = 0; }
  uint32_t inc = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) s_scan[warp] = (int)inc;
  __syncthreads();
  if (warp == 0) {
    int v = (lane < kSelThreads / 32) ? s_scan[lane] : 0;
    int w = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int u = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += u;
    }
    if (lane < kSelThreads / 32) s_scan[lane] = w - v;   // exclusive warp offsets
  }
  __syncthreads();
  const uint32_t before = (uint32_t)s_scan[warp] + inc - local;   // items in digits above mine
  if (before < (uint32_t)k && (uint32_t)k <= before + local) {
    uint32_t run = before;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (run < (uint32_t)k && run + mine[j] >= (uint32_t)k) {
        s_scan[32] = hi - 1 - j;
        s_scan[33] = (int)run;
      }
      run += mine[j];
    }
  }
  __syncthreads();
  digit = s_scan[32];
  above = s_scan[33];
  __syncthreads();
}

// Slot for each `flag`ged lane through one atomic per warp (counter in shared or global
// memory); -1 for the others.  All 32 lanes must call.
__device__ __forceinline__ int warp_append(bool flag, uint32_t* counter) {
  const unsigned m = __ballot_sync(0xffffffffu, flag);
  if (m == 0) return -1;
  const int lane = threadIdx.x & 31;
  const int leader = __ffs(m) - 1;
  uint32_t base = 0;
  if (lane == leader) base = atomicAdd(counter, (uint32_t)__popc(m));
  base = __shfl_sync(0xffffffffu, base, leader);
  return flag ? (int)(base + __popc(m & ((1u << lane) - 1u))) : -1;
}

// The 16 scores of this thread: 4 float4 at float4-index chunk*2048 + j*512 + tid.
__device__ __forceinline__ void load_chunk(const float* __restrict__ rs, int chunk, int n,
                                           float (&v)[kElems], int (&pos0)[4]) {
  const int tid = threadIdx.x;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int i = chunk * kSelChunk + (j * kSelThreads + tid) * 4;
    pos0[j] = i;
    if (i + 3 < n) {
      const float4 f = __ldcg(reinterpret_cast<const float4*>(rs + i));
      v[4 * j] = f.x; v[4 * j + 1] = f.y; v[4 * j + 2] = f.z; v[4 * j + 3] = f.w;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) v[4 * j + e] = (i + e < n) ? __ldcg(rs + i + e) : 0.f;
    }
  }
}

// ------------------------------------------------------------------------- hist kernel
__global__ void __launch_bounds__(kSelThreads)
sel_hist_kernel(Plan pl, const float* __restrict__ scores, const int32_t* __restrict__ seq_lens,
                uint32_t* __restrict__ hist1, uint32_t* __restrict__ counters,
                int32_t* __restrict__ rowstate, int32_t* __restrict__ sel_count,
                float* __restrict__ kth) {
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ int s_scan[34];
  __shared__ int s_last;
  const int row = blockIdx.y, tid = threadIdx.x, chunk = blockIdx.x;
  const int b = row / pl.Hq;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const int k = budget_k(n, pl.ppm);
  if (k == 0) {
    if (chunk == 0 && tid == 0) {
      rowstate[row * 4 + 0] = -1; rowstate[row * 4 + 1] = 0;
      rowstate[row * 4 + 2] = 0;  rowstate[row * 4 + 3] = n;
      sel_count[row] = 0;
      kth[row] = CUDART_NAN_F;
    }
    return;
  }
  uint32_t* gh = hist1 + (size_t)row * kHistBins;
  const int n_chunks = (n + kSelChunk - 1) / kSelChunk;
  if (chunk < n_chunks) {
    const float* rs = scores + (size_t)row * pl.N_max;
    float v[kElems], nv[kElems];
    int pos0[4], npos0[4];
    load_chunk(rs, chunk, n, v, pos0);
    for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
    __syncthreads();
    for (int ch = chunk; ch < n_chunks; ch += gridDim.x) {
      const bool more = ch + (int)gridDim.x < n_chunks;
      if (more) load_chunk(rs, ch + gridDim.x, n, nv, npos0);     // in flight during the atomics
      if ((ch + 1) * kSelChunk <= n) {               // full chunk: no bounds checks
#pragma unroll
        for (int e = 0; e < kElems; ++e) atomicAdd(&s_hist[score_key(v[e]) >> 20], 1u);
      } else {
#pragma unroll
        for (int e = 0; e < kElems; ++e)
          if (pos0[e >> 2] + (e & 3) < n) atomicAdd(&s_hist[score_key(v[e]) >> 20], 1u);
      }
      if (more) {
#pragma unroll
        for (int e = 0; e < kElems; ++e) v[e] = nv[e];
#pragma unroll
        for (int j = 0; j < 4; ++j) pos0[j] = npos0[j];
      }
    }
    __syncthreads();
    for (int i = tid; i < kHistBins; i += kSelThreads)
      if (s_hist[i]) atomicAdd(gh + i, s_hist[i]);
    __threadfence();
  }
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&counters[row * 4 + 0], 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  int b1, above;
  find_digit<true>(gh, kHistBins, k, s_scan, b1, above);
  if (tid == 0) {
    rowstate[row * 4 + 0] = b1;
    rowstate[row * 4 + 1] = k - above;
    rowstate[row * 4 + 2] = k;
    rowstate[row * 4 + 3] = n;
  }
}

// ------------------------------------------------------------------------- filter kernel
// Calls f(valid, key, position) for every candidate of the row, from the candidate list or,
// if that overflowed, from the score row itself.  Uniform trip count: f may use warp votes.
template <class F>
__device__ __forceinline__ void for_each_candidate(bool overflow, const uint2* cand, int n_stored,
                                                   const float* rs, int n, uint32_t b1, F f) {
  const int tid = threadIdx.x;
  constexpr int U = 4;
  if (!overflow) {
    for (int base = 0; base < n_stored; base += kSelThreads * U) {
      uint2 c[U];
      bool v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = base + u * kSelThreads + tid;
        v[u] = i < n_stored;
        c[u] = make_uint2(0u, 0u);
        if (v[u]) c[u] = __ldcg(cand + i);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) f(v[u], c[u].x, (int)c[u].y);
    }
  } else {
    for (int base = 0; base < n; base += kSelThreads * U) {
      float s[U];
      bool v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = base + u * kSelThreads + tid;
        v[u] = i < n;
        s[u] = v[u] ? __ldcg(rs + i) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint32_t key = score_key(s[u]);
        f(v[u] && (key >> 20) == b1, key, base + u * kSelThreads + tid);
      }
    }
  }
}

__device__ int block_count(int local, int* s_scan) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int v = local;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) s_scan[warp] = v;
  __syncthreads();
  int tot = 0;
  for (int w = 0; w < kSelThreads / 32; ++w) tot += s_scan[w];
  __syncthreads();
  return tot;
}

__global__ void __launch_bounds__(kSelThreads, 2)
sel_filter_kernel(Plan pl, const float* __restrict__ scores, const uint32_t* __restrict__ hist1,
                  uint32_t* __restrict__ hist2, uint32_t* __restrict__ counters,
                  const int32_t* __restrict__ rowstate, uint2* __restrict__ cand,
                  int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_count,
                  float* __restrict__ kth, int* __restrict__ status) {
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ uint2 s_stash[kStashCap];
  __shared__ int s_scan[34];
  __shared__ int s_last;
  __shared__ uint32_t s_cnt[2];
  __shared__ int s_scan2[2][32];
  __shared__ uint32_t s_base2[2][2];
  const int row = blockIdx.y, tid = threadIdx.x, chunk = blockIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int b1 = rowstate[row * 4 + 0], k1 = rowstate[row * 4 + 1];
  const int k = rowstate[row * 4 + 2], n = rowstate[row * 4 + 3];
  if (k == 0) return;
  const float* rs = scores + (size_t)row * pl.N_max;
  int32_t* out = sel_idx + (size_t)row * pl.k_max;
  uint2* rc = cand + (size_t)row * pl.cand_cap;
  uint32_t* n_out = &counters[row * 4 + 2];
  uint32_t* n_cand = &counters[row * 4 + 3];
  uint32_t* gh = hist2 + (size_t)row * kHistBins;

  const int n_chunks = (n + kSelChunk - 1) / kSelChunk;
  if (chunk < n_chunks) {
    float v[kElems], nv[kElems];
    int pos0[4], npos0[4];
    load_chunk(rs, chunk, n, v, pos0);
    for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
    // The key is monotone in the score, so "digit above / equal to b1" are two float
    // compares: scores in [lo_f, hi_f] have top digit b1, scores above hi_f a larger one.
    float lo_f = key_score((uint32_t)b1 << 20), hi_f = key_score(((uint32_t)b1 << 20) | 0xfffffu);
    if (lo_f != lo_f) lo_f = -CUDART_INF_F;        // digit that starts inside the NaN patterns
    __syncthreads();
    for (int ch = chunk; ch < n_chunks; ch += gridDim.x) {
      const bool more = ch + (int)gridDim.x < n_chunks;
      if (more) load_chunk(rs, ch + gridDim.x, n, nv, npos0);     // in flight during this chunk
      uint32_t win_mask = 0, cand_mask = 0;
      const bool full = (ch + 1) * kSelChunk <= n;
#pragma unroll
      for (int e = 0; e < kElems; ++e) {
        const bool valid = full || pos0[e >> 2] + (e & 3) < n;
        const bool win = v[e] > hi_f;
        const bool cnd = !win && v[e] >= lo_f;
        if (valid && win) win_mask |= 1u << e;
        if (valid && cnd) {
          cand_mask |= 1u << e;
          atomicAdd(&s_hist[(score_key(v[e]) >> 8) & 0xfffu], 1u);
        }
      }
      // exclusive scan of (winners << 16 | candidates) over the CTA
      const uint32_t mine = ((uint32_t)__popc(win_mask) << 16) | (uint32_t)__popc(cand_mask);
      uint32_t inc = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += u;
      }
      int* scan_buf = s_scan2[(ch / gridDim.x) & 1];     // two sets: no barrier to reuse them
      uint32_t* base_buf = s_base2[(ch / gridDim.x) & 1];
      if (lane == 31) scan_buf[warp] = (int)inc;
      __syncthreads();
      if (warp == 0) {
        uint32_t wv = (lane < kSelThreads / 32) ? (uint32_t)scan_buf[lane] : 0u;
        uint32_t ws = wv;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t u = __shfl_up_sync(0xffffffffu, ws, o);
          if (lane >= o) ws += u;
        }
        if (lane < kSelThreads / 32) scan_buf[16 + lane] = (int)(ws - wv);
        if (lane == kSelThreads / 32 - 1) {        // CTA totals: take the output slots
          const uint32_t tw = ws >> 16, tc = ws & 0xffffu;
          base_buf[0] = tw ? atomicAdd(n_out, tw) : 0u;
          base_buf[1] = tc ? atomicAdd(n_cand, tc) : 0u;
        }
      }
      __syncthreads();
      const uint32_t excl = (uint32_t)scan_buf[16 + warp] + inc - mine;
      uint32_t pw = base_buf[0] + (excl >> 16), pc = base_buf[1] + (excl & 0xffffu);
#pragma unroll
      for (int e = 0; e < kElems; ++e) {
        const int pos = pos0[e >> 2] + (e & 3);
        if (win_mask & (1u << e)) {
          if (pw < (uint32_t)pl.k_max) out[pw] = pos;
          ++pw;
        }
        if (cand_mask & (1u << e)) {
          if (pc < (uint32_t)pl.cand_cap) rc[pc] = make_uint2(score_key(v[e]), (uint32_t)pos);
          ++pc;
        }
      }
      if (more) {
#pragma unroll
        for (int e = 0; e < kElems; ++e) v[e] = nv[e];
#pragma unroll
        for (int j = 0; j < 4; ++j) pos0[j] = npos0[j];
      }
    }
    __syncthreads();
    for (int i = tid; i < kHistBins; i += kSelThreads)
      if (s_hist[i]) atomicAdd(gh + i, s_hist[i]);
    __threadfence();
  }
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&counters[row * 4 + 1], 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- last CTA of the row: resolve digits 2 and 3 on the candidates of digit b1
  const int n_in_bin = (int)__ldcg(hist1 + (size_t)row * kHistBins + b1);
  const bool overflow = n_in_bin > pl.cand_cap;
  const int n_stored = overflow ? 0 : n_in_bin;
  const uint32_t base_out = __ldcg(n_out);          // winners written by the main phase
  int b2, above2;
  find_digit<true>(gh, kHistBins, k1, s_scan, b2, above2);
  const int k2 = k1 - above2;
  for (int i = tid; i < 256; i += kSelThreads) s_hist[i] = 0u;
  if (tid == 0) { s_cnt[0] = 0u; s_cnt[1] = 0u; }
  __syncthreads();
  // one pass: second digit above b2 -> winner; equal -> third-digit histogram + stash
  for_each_candidate(overflow, rc, n_stored, rs, n, (uint32_t)b1,
                     [&](bool v, uint32_t key, int pos) {
                       const int d2 = (int)((key >> 8) & 0xfffu);
                       const int p = warp_append(v && d2 > b2, &s_cnt[0]);
                       if (p >= 0 && base_out + p < (uint32_t)pl.k_max) out[base_out + p] = pos;
                       const bool tie = v && d2 == b2;
                       if (tie) atomicAdd(&s_hist[key & 0xffu], 1u);
                       const int ps = warp_append(tie, &s_cnt[1]);
                       if (ps >= 0 && ps < kStashCap) s_stash[ps] = make_uint2(key, (uint32_t)pos);
                     });
  __syncthreads();
  int b3, above3;
  find_digit<false>(s_hist, 256, k2, s_scan, b3, above3);
  const int k3 = k2 - above3;                      // how many keys equal to the k-th are taken
  const int ties = (int)s_hist[b3];
  const int n_stash = (int)s_cnt[1];
  const bool stash_ok = n_stash <= kStashCap;
  const uint32_t kstar = ((uint32_t)b1 << 20) | ((uint32_t)b2 << 8) | (uint32_t)b3;
  int max_tie_pos = n;                             // take ties at positions <= this
  if (ties != k3) {
    // k3-th smallest position among the keys equal to the k-th, by bisection on the position
    int plo = 0, phi = n - 1;
    while (plo < phi) {
      const int mid = plo + (phi - plo) / 2;
      int local = 0;
      if (stash_ok) {
        for (int i = tid; i < n_stash; i += kSelThreads)
          if (s_stash[i].x == kstar && (int)s_stash[i].y <= mid) ++local;
      } else {
        for_each_candidate(overflow, rc, n_stored, rs, n, (uint32_t)b1,
                           [&](bool v, uint32_t key, int pos) {
                             if (v && key == kstar && pos <= mid) ++local;
                           });
      }
      const int cnt = block_count(local, s_scan);
      if (cnt >= k3) phi = mid; else plo = mid + 1;
    }
    max_tie_pos = plo;
  }
  if (stash_ok) {
    for (int base = 0; base < n_stash; base += kSelThreads) {
      const int i = base + tid;
      bool take = false;
      int pos = 0;
      if (i < n_stash) {
        const int low = (int)(s_stash[i].x & 0xffu);
        pos = (int)s_stash[i].y;
        take = low > b3 || (low == b3 && pos <= max_tie_pos);
      }
      const int p = warp_append(take, &s_cnt[0]);
      if (p >= 0 && base_out + p < (uint32_t)pl.k_max) out[base_out + p] = pos;
    }
  } else {
    for_each_candidate(overflow, rc, n_stored, rs, n, (uint32_t)b1,
                       [&](bool v, uint32_t key, int pos) {
                         const bool pre = v && (int)((key >> 8) & 0xfffu) == b2;
                         const int low = (int)(key & 0xffu);
                         const bool take = pre && (low > b3 || (low == b3 && pos <= max_tie_pos));
                         const int p = warp_append(take, &s_cnt[0]);
                         if (p >= 0 && base_out + p < (uint32_t)pl.k_max) out[base_out + p] = pos;
                       });
  }
  __syncthreads();
  if (tid == 0) {
    sel_count[row] = k;
    kth[row] = key_score(kstar);
    if ((int)(base_out + s_cnt[0]) != k) atomicOr(status, 1);
  }
}

}  // namespace

cudaError_t launch_select(const Plan& pl, const WsLayout& L, char* ws, const float* scores,
                          const int32_t* seq_lens, int32_t* sel_idx, int32_t* sel_count,
                          float* kth, cudaStream_t st) {
  uint32_t* hist1 = reinterpret_cast<uint32_t*>(ws + L.hist1);
  uint32_t* hist2 = reinterpret_cast<uint32_t*>(ws + L.hist2);
  uint32_t* counters = reinterpret_cast<uint32_t*>(ws + L.counters);
  int32_t* rowstate = reinterpret_cast<int32_t*>(ws + L.rowstate);
  uint2* cand = reinterpret_cast<uint2*>(ws + L.cand);
  int* status = reinterpret_cast<int*>(ws + L.status);
  dim3 grid(pl.hist_chunks, pl.rows);
  sel_hist_kernel<<<grid, kSelThreads, 0, st>>>(pl, scores, seq_lens, hist1, counters, rowstate,
                                                sel_count, kth);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  sel_filter_kernel<<<grid, kSelThreads, 0, st>>>(pl, scores, hist1, hist2, counters, rowstate,
                                                  cand, sel_idx, sel_count, kth, status);
  return cudaGetLastError();
}

}  // namespace pqhsa
