// Step 3 of the decode operator: exact top-k over every score row (Eq. 3),
// T(q) = TopK_{k, i in R} l~_i with k = ceil(rho |R|).
//
// Radix threshold select on order-preserving 32-bit keys, digits of 12 / 12 / 8 bits:
//   hist kernel    every CTA histograms the top digit of its chunk of a row; the last CTA of
//                  the row to finish finds the digit b1 that holds the k-th largest key;
//   filter kernel  keys above b1 are winners and are emitted at once; keys inside b1 are
//                  appended to a candidate list and histogrammed on the second digit; the
//                  last CTA of the row resolves the remaining two digits on the candidates.
// Equal keys at the threshold are taken in order of position (lowest first), which is the
// stable rule of a full sort.  No CTA ever waits for another: "last CTA" is decided by an
// atomic ticket.
#include "common.cuh"

namespace pqhsa {

namespace {

struct RowState { int b1, k1, k, n; };

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
  uint32_t local = 0;
  for (int j = 0; j < per; ++j) {
    const int d = hi - 1 - j;
    if (d >= 0) local += kGlobal ? __ldcg(hist + d) : hist[d];
  }
  // inclusive scan over threads (thread 0 = top digits)
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
  __syncthreads();
  if (before < (uint32_t)k && (uint32_t)k <= before + local) {
    uint32_t run = before;
    for (int j = 0; j < per; ++j) {
      const int d = hi - 1 - j;
      if (d < 0) break;
      const uint32_t c = kGlobal ? __ldcg(hist + d) : hist[d];
      if (run + c >= (uint32_t)k) {
        s_scan[32] = d;
        s_scan[33] = (int)run;
        break;
      }
      run += c;
    }
  }
  __syncthreads();
  digit = s_scan[32];
  above = s_scan[33];
  __syncthreads();
}

// Appends `flag`ged lanes' values through one atomic per warp; returns the slot or -1.
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

__device__ __forceinline__ void row_chunk(int n, int chunks, int c, int& lo, int& hi) {
  int per = (n + chunks - 1) / chunks;
  per = (per + 3) & ~3;                      // keep float4 loads aligned
  lo = min(n, c * per);
  hi = min(n, lo + per);
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
  const int row = blockIdx.y, tid = threadIdx.x;
  const int b = row / pl.Hq;
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const int k = budget_k(n, pl.ppm);
  if (k == 0) {
    if (blockIdx.x == 0 && tid == 0) {
      rowstate[row * 4 + 0] = -1; rowstate[row * 4 + 1] = 0;
      rowstate[row * 4 + 2] = 0;  rowstate[row * 4 + 3] = n;
      sel_count[row] = 0;
      kth[row] = CUDART_NAN_F;
    }
    return;
  }
  for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
  __syncthreads();
  int lo, hi;
  row_chunk(n, gridDim.x, blockIdx.x, lo, hi);
  const float* rs = scores + (size_t)row * pl.N_max;
  for (int i = lo + tid * 4; i < hi; i += kSelThreads * 4) {
    if (i + 3 < hi) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(rs + i));
      atomicAdd(&s_hist[score_key(v.x) >> 20], 1u);
      atomicAdd(&s_hist[score_key(v.y) >> 20], 1u);
      atomicAdd(&s_hist[score_key(v.z) >> 20], 1u);
      atomicAdd(&s_hist[score_key(v.w) >> 20], 1u);
    } else {
      for (int j = i; j < hi; ++j) atomicAdd(&s_hist[score_key(__ldcg(rs + j)) >> 20], 1u);
    }
  }
  __syncthreads();
  uint32_t* gh = hist1 + (size_t)row * kHistBins;
  for (int i = tid; i < kHistBins; i += kSelThreads)
    if (s_hist[i]) atomicAdd(gh + i, s_hist[i]);
  __threadfence();
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
  if (!overflow) {
    for (int base = 0; base < n_stored; base += kSelThreads) {
      const int i = base + tid;
      const bool v = i < n_stored;
      uint2 c = make_uint2(0u, 0u);
      if (v) c = __ldcg(cand + i);
      f(v, c.x, (int)c.y);
    }
  } else {
    for (int base = 0; base < n; base += kSelThreads) {
      const int i = base + tid;
      bool v = i < n;
      uint32_t key = 0u;
      if (v) key = score_key(__ldcg(rs + i));
      v = v && (key >> 20) == b1;
      f(v, key, i);
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

__global__ void __launch_bounds__(kSelThreads)
sel_filter_kernel(Plan pl, const float* __restrict__ scores, const uint32_t* __restrict__ hist1,
                  uint32_t* __restrict__ hist2, uint32_t* __restrict__ counters,
                  const int32_t* __restrict__ rowstate, uint2* __restrict__ cand,
                  int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_count,
                  float* __restrict__ kth, int* __restrict__ status) {
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ int s_scan[34];
  __shared__ int s_last;
  const int row = blockIdx.y, tid = threadIdx.x;
  const int b1 = rowstate[row * 4 + 0], k1 = rowstate[row * 4 + 1];
  const int k = rowstate[row * 4 + 2], n = rowstate[row * 4 + 3];
  if (k == 0) return;
  for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
  __syncthreads();
  int lo, hi;
  row_chunk(n, gridDim.x, blockIdx.x, lo, hi);
  const float* rs = scores + (size_t)row * pl.N_max;
  int32_t* out = sel_idx + (size_t)row * pl.k_max;
  uint2* rc = cand + (size_t)row * pl.cand_cap;
  uint32_t* n_out = &counters[row * 4 + 2];
  uint32_t* n_cand = &counters[row * 4 + 3];

  for (int base = lo; base < hi; base += kSelThreads * 4) {
    const int i = base + tid * 4;
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (i + 3 < hi) {
      const float4 f4 = __ldcg(reinterpret_cast<const float4*>(rs + i));
      v[0] = f4.x; v[1] = f4.y; v[2] = f4.z; v[3] = f4.w;
    } else {
      for (int j = 0; j < 4; ++j) if (i + j < hi) v[j] = __ldcg(rs + i + j);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bool valid = i + j < hi;
      const uint32_t key = score_key(v[j]);
      const int bin = (int)(key >> 20);
      const int p = warp_append(valid && bin > b1, n_out);
      if (p >= 0 && p < pl.k_max) out[p] = i + j;
      const bool is_c = valid && bin == b1;
      if (is_c) atomicAdd(&s_hist[(key >> 8) & 0xfffu], 1u);
      const int pc = warp_append(is_c, n_cand);
      if (pc >= 0 && pc < pl.cand_cap) rc[pc] = make_uint2(key, (uint32_t)(i + j));
    }
  }
  __syncthreads();
  uint32_t* gh = hist2 + (size_t)row * kHistBins;
  for (int i = tid; i < kHistBins; i += kSelThreads)
    if (s_hist[i]) atomicAdd(gh + i, s_hist[i]);
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&counters[row * 4 + 1], 1u) == gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- last CTA of the row: resolve digits 2 and 3 on the candidates of digit b1
  const int n_in_bin = (int)__ldcg(hist1 + (size_t)row * kHistBins + b1);
  const bool overflow = n_in_bin > pl.cand_cap;
  const int n_stored = overflow ? 0 : n_in_bin;
  int b2, above2;
  find_digit<true>(gh, kHistBins, k1, s_scan, b2, above2);
  const int k2 = k1 - above2;
  for (int i = tid; i < 256; i += kSelThreads) s_hist[i] = 0u;
  __syncthreads();
  for_each_candidate(overflow, rc, n_stored, rs, n, (uint32_t)b1,
                     [&](bool v, uint32_t key, int pos) {
                       const int d2 = (int)((key >> 8) & 0xfffu);
                       const int p = warp_append(v && d2 > b2, n_out);
                       if (p >= 0 && p < pl.k_max) out[p] = pos;
                       if (v && d2 == b2) atomicAdd(&s_hist[key & 0xffu], 1u);
                     });
  __syncthreads();
  int b3, above3;
  find_digit<false>(s_hist, 256, k2, s_scan, b3, above3);
  const int k3 = k2 - above3;                      // how many keys equal to the k-th are taken
  const int ties = (int)s_hist[b3];
  const uint32_t kstar = ((uint32_t)b1 << 20) | ((uint32_t)b2 << 8) | (uint32_t)b3;
  int max_tie_pos = n;                             // take ties at positions <= this
  if (ties != k3) {
    // k3-th smallest position among the ties, by bisection on the position
    int plo = 0, phi = n - 1;
    while (plo < phi) {
      const int mid = plo + (phi - plo) / 2;
      int local = 0;
      for_each_candidate(overflow, rc, n_stored, rs, n, (uint32_t)b1,
                         [&](bool v, uint32_t key, int pos) {
                           if (v && key == kstar && pos <= mid) ++local;
                         });
      const int cnt = block_count(local, s_scan);
      if (cnt >= k3) phi = mid; else plo = mid + 1;
    }
    max_tie_pos = plo;
  }
  for_each_candidate(overflow, rc, n_stored, rs, n, (uint32_t)b1,
                     [&](bool v, uint32_t key, int pos) {
                       const bool pre = v && (int)((key >> 8) & 0xfffu) == b2;
                       const int low = (int)(key & 0xffu);
                       const bool take = pre && (low > b3 || (low == b3 && pos <= max_tie_pos));
                       const int p = warp_append(take, n_out);
                       if (p >= 0 && p < pl.k_max) out[p] = pos;
                     });
  __syncthreads();
  if (tid == 0) {
    sel_count[row] = k;
    kth[row] = key_score(kstar);
    __threadfence();
    if ((int)atomicAdd(n_out, 0u) != k) atomicOr(status, 1);
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
