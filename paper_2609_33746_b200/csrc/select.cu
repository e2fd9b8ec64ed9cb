// Step 3 of the decode operator: exact top-k over every score row (Eq. 3),
// T(q) = TopK_{k, i in R} l~_i with k = ceil(rho |R|).
//
// One pass over the scores instead of a multi-pass radix sort of the whole row:
//   sample kernel  one CTA per row reads up to 16384 scores (1024 groups of 16 at a jittered
//                  stride; never more than a quarter of the row) and takes two order
//                  statistics of the sample that bracket the k-th largest score of the row
//                  with a 6-sigma margin: lo <= s_k <= hi (one histogram of the sample over
//                  4096 equal buckets of its range; the bracket's edges are bucket edges).  At
//                  a 1 % budget and 128K tokens about half of the k winners lie above hi;
//   filter kernel  scores above hi are certain winners and are written out at once; scores in
//                  [lo, hi] are appended, as (key, position) pairs, to a candidate list; the
//                  last CTA of the row (atomic ticket, nobody waits) checks the bracket by
//                  counting (#winners <= k <= #winners + #candidates) and finishes exactly:
//                  one histogram of the candidates over 4096 equal buckets of their range,
//                  everything above the bucket of the k-th largest is taken, the few items
//                  inside it are ranked against each other (a 12/12/8-bit radix select remains
//                  for candidate sets that do not fit shared memory or pile up in one bucket).
// If the bracket misses (a row whose order defeats the sample), that last CTA redoes the
// row from the scores themselves with the same radix select, so the result is always the
// exact top-k; equal scores at the threshold are taken in order of position (lowest first),
// the stable rule of a full sort.
#include "common.cuh"

namespace pqhsa {

namespace {

constexpr int kElems = kSelChunk / kSelThreads;   // scores per thread per chunk (16)
constexpr int kStashCap = 5120;                   // candidates resolved from shared memory
constexpr int kFilterSmemBytes = kHistBins * 4 + kStashCap * 8;   // dynamic: above the 48 KB static limit
constexpr int kSample = 16384;                    // sampled scores per row (at most a quarter of it)
constexpr int kSamplePer = kSample / kSelThreads; // per thread (32)
constexpr int kSampleGroups = kSample / 16;       // groups of 16 consecutive scores (64 bytes)
constexpr float kBracketSigmas = 6.0f;

// rowstate: [0] lo, [1] hi (float bits), [2] k, [3] n

// Largest digit D with  count(digits > D) < k <= count(digits >= D) in a shared-memory
// histogram.  All kSelThreads threads must call; 1 <= k <= number of items.  Returns D and
// count(digits > D).
__device__ void find_digit(const uint32_t* hist, int nbins, int k, int* s_scan, int& digit,
                           int& above) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (nbins + kSelThreads - 1) / kSelThreads;
  // thread t owns digits [hi - per, hi) with hi = nbins - t*per, walked from the top down
  const int hi = nbins - tid * per;
  uint32_t mine[8];
  uint32_t local = 0;
  if (per == 8 && hi >= 8) {
    // two 16-byte reads instead of eight 4-byte reads 32 bytes apart (8-way bank conflicts)
    const uint4 v0 = *reinterpret_cast<const uint4*>(hist + hi - 8);
    const uint4 v1 = *reinterpret_cast<const uint4*>(hist + hi - 4);
    mine[0] = v1.w; mine[1] = v1.z; mine[2] = v1.y; mine[3] = v1.x;
    mine[4] = v0.w; mine[5] = v0.z; mine[6] = v0.y; mine[7] = v0.x;
#pragma unroll
    for (int j = 0; j < 8; ++j) local += mine[j];
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int d = hi - 1 - j;
      mine[j] = (j < per && d >= 0) ? hist[d] : 0u;
      local += mine[j];
    }
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

// ------------------------------------------------------------------------- sample kernel
// Bucket of a score in a linear partition of [lo, lo + kHistBins / scale) into kHistBins
// buckets; a larger score never gets a smaller bucket (the product is monotone and clamped).
__device__ __forceinline__ int linear_bucket(float s, float lo, float scale) {
  const float t = (s - lo) * scale;
  return t >= (float)(kHistBins - 1) ? kHistBins - 1 : (t > 0.f ? (int)t : 0);   // NaN -> 0
}

// Buckets (from the top) that hold the rank_a-th and rank_b-th largest (0-based) of the items
// counted in `hist`, and the number of items in the buckets above the first of them; one pass
// over the histogram serves both ranks.
__device__ void find_two_buckets(const uint32_t* hist, int rank_a, int rank_b, int* s_scan,
                                 int& bucket_a, int& bucket_b, int& above_a) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int per = kHistBins / kSelThreads;                 // 8 bins per thread, top down
  const int hi = kHistBins - tid * per;
  const uint4 v0 = *reinterpret_cast<const uint4*>(hist + hi - 8);
  const uint4 v1 = *reinterpret_cast<const uint4*>(hist + hi - 4);
  const uint32_t mine[8] = {v1.w, v1.z, v1.y, v1.x, v0.w, v0.z, v0.y, v0.x};
  uint32_t local = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) local += mine[j];
  if (tid == 0) { s_scan[32] = 0; s_scan[33] = 0; s_scan[34] = 0; }
  uint32_t inc = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) s_scan[warp] = (int)inc;
  __syncthreads();
  if (warp == 0) {
    const int v = (lane < kSelThreads / 32) ? s_scan[lane] : 0;
    int w = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += u;
    }
    if (lane < kSelThreads / 32) s_scan[lane] = w - v;       // exclusive warp offsets
  }
  __syncthreads();
  uint32_t run = (uint32_t)s_scan[warp] + inc - local;       // items in buckets above mine
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (run <= (uint32_t)rank_a && (uint32_t)rank_a < run + mine[j]) { s_scan[32] = hi - 1 - j; s_scan[34] = (int)run; }
    if (run <= (uint32_t)rank_b && (uint32_t)rank_b < run + mine[j]) s_scan[33] = hi - 1 - j;
    run += mine[j];
  }
  __syncthreads();
  bucket_a = s_scan[32];
  bucket_b = s_scan[33];
  above_a = s_scan[34];
  __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads, 2)     // two rows per SM: 64 registers
sel_sample_kernel(Plan pl, const float* __restrict__ scores, const int32_t* __restrict__ seq_lens,
                  int32_t* __restrict__ rowstate, int32_t* __restrict__ sel_count,
                  float* __restrict__ kth) {
  __shared__ __align__(16) uint32_t s_hist[kHistBins];
  __shared__ int s_scan[36];
  __shared__ float s_mm[2][kSelThreads / 32];
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = row / pl.Hq;
  // what depends on the call's inputs only (row length, budget, sample offsets, the cleared
  // histogram) is done before the wait for the scan's scores
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const int k = region_budget(pl, n, b);
  const Region rg = region_of(pl, n, b);
  // n_groups aligned groups of 16 consecutive scores (1024 of them on a long row, never more
  // than a quarter of the row); group g sits in the g-th of n_groups equal strides of the
  // row at a hashed offset, and four neighbouring threads read its 64 bytes
  const int n_groups = min(kSampleGroups, n / 64);
  const uint32_t stride = n_groups > 0 ? (uint32_t)n / (uint32_t)n_groups : 0u;     // >= 64
  int off[kSamplePer / 4];
#pragma unroll
  for (int u = 0; u < kSamplePer / 4; ++u) {
    const int g = (u * kSelThreads + tid) >> 2;
    const uint32_t h = (uint32_t)g * 2654435761u;
    off[u] = g < n_groups ? (int)min(((uint32_t)g * stride + __umulhi(h, stride)) & ~15u, (uint32_t)(n - 16) & ~15u) + 4 * (tid & 3) : -1;
  }
  for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
  pdl_wait();
  pdl_launch_dependents();
  float lo = -CUDART_INF_F, hi = CUDART_INF_F;     // default: every score is a candidate
  if (k == 0) {
    if (tid == 0) { sel_count[row] = 0; kth[row] = CUDART_NAN_F; }
  } else if (k == rg.r_end - rg.r_begin) {
    hi = -CUDART_INF_F;                            // all of R: every score above -inf is a winner
  } else if (n > kSelChunk) {
    const float* rs = scores + (size_t)row * pl.N_max;
    float s[kSamplePer];
#pragma unroll
    for (int u = 0; u < kSamplePer / 4; ++u) {
      float4 f = make_float4(CUDART_NAN_F, CUDART_NAN_F, CUDART_NAN_F, CUDART_NAN_F);   // not sampled
      if (off[u] >= 0) f = __ldcg(reinterpret_cast<const float4*>(rs + off[u]));
      s[4 * u] = f.x; s[4 * u + 1] = f.y; s[4 * u + 2] = f.z; s[4 * u + 3] = f.w;
    }
    // range of the finite samples (sink and window positions hold -inf)
    float mn = CUDART_INF_F, mx = -CUDART_INF_F;
#pragma unroll
    for (int e = 0; e < kSamplePer; ++e) {
      const bool fin = fabsf(s[e]) < CUDART_INF_F;
      mn = fin ? fminf(mn, s[e]) : mn;
      mx = fin ? fmaxf(mx, s[e]) : mx;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if (lane == 0) { s_mm[0][warp] = mn; s_mm[1][warp] = mx; }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kSelThreads / 32; ++w) { mn = fminf(mn, s_mm[0][w]); mx = fmaxf(mx, s_mm[1][w]); }
    // the k-th largest of the row sits near rank p * n_sample of the sample; the bracket is
    // +- 6 sigma of that count (binomial bound on the hypergeometric spread), + 2
    const int n_sample = 16 * n_groups;
    const float p = (float)k / (float)n;
    const float r = p * n_sample;
    const int mgn = (int)ceilf(kBracketSigmas * sqrtf(n_sample * p * (1.f - p))) + 2;
    const int r_hi = (int)floorf(r) - mgn, r_lo = (int)ceilf(r) + mgn;
    if (mx > mn) {
      // one histogram of the samples over 4096 equal buckets of [mn, mx] (non-finite samples
      // fall into the bottom bucket); the bracket is the outer edges of the two buckets that
      // hold the order statistics, one bucket wider on each side for the rounding of the edges.
      // Whatever the bracket is, the filter kernel checks it by counting.
      // If both order statistics land within a few buckets of each other, the range was
      // stretched by outliers (one score at -1e6 puts every other score into one bucket): the
      // histogram is then repeated over the span of those buckets, with the samples above it
      // counted as ranked higher, up to twice (4096-fold zoom each time).
      const int rk_hi = max(r_hi, 0), rk_lo = min(r_lo, n_sample - 1);
      float lo_r = mn, hi_r = mx;
      uint32_t alive = 0u;                         // samples inside the current range
#pragma unroll
      for (int e = 0; e < kSamplePer; ++e) alive |= (s[e] == s[e] ? 1u : 0u) << e;
      int above = 0;                               // samples ranked above the current range
      for (int pass = 0;; ++pass) {
        const float scale = (float)kHistBins / (hi_r - lo_r);
        const float width = (hi_r - lo_r) / (float)kHistBins;
#pragma unroll
        for (int e = 0; e < kSamplePer; ++e)
          if ((alive >> e) & 1u) atomicAdd(&s_hist[linear_bucket(s[e], lo_r, scale)], 1u);
        __syncthreads();
        int b_hi, b_lo, above_hi;
        find_two_buckets(s_hist, rk_hi - above, rk_lo - above, s_scan, b_hi, b_lo, above_hi);
        if (b_hi - b_lo >= 8 || pass == 2 || !(width > 0.f)) {
          if (r_hi >= 0) hi = lo_r + (float)(b_hi + 2) * width;
          if (r_lo < n_sample && (b_lo >= 2 || pass > 0)) lo = lo_r + (float)(b_lo - 1) * width;
          break;
        }
        // zoom into buckets b_lo .. b_hi
#pragma unroll
        for (int e = 0; e < kSamplePer; ++e) {
          const int bk = linear_bucket(s[e], lo_r, scale);
          if (bk < b_lo || bk > b_hi) alive &= ~(1u << e);
        }
        above += above_hi;
        const float nlo = lo_r + (float)b_lo * width, nhi = lo_r + (float)(b_hi + 1) * width;
        if (!(nhi > nlo)) {                        // the floats between the edges ran out
          if (r_hi >= 0) hi = lo_r + (float)(b_hi + 2) * width;
          if (r_lo < n_sample) lo = lo_r + (float)(b_lo - 1) * width;
          break;
        }
        lo_r = nlo;
        hi_r = nhi;
        for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
        __syncthreads();
      }
    } else if (mx == mn) {
      hi = mx;                                     // all finite samples equal: take that value
      lo = mn;                                     // as the whole bracket
    }
    if (hi != hi) hi = CUDART_INF_F;
    if (lo != lo) lo = -CUDART_INF_F;
  }
  if (tid == 0) {
    rowstate[row * 4 + 0] = __float_as_int(lo);
    rowstate[row * 4 + 1] = __float_as_int(hi);
    rowstate[row * 4 + 2] = k;
    rowstate[row * 4 + 3] = n;
  }
}

// ------------------------------------------------------------------------- filter kernel
enum Source { kFromStash = 0, kFromList = 1, kFromRow = 2 };

// Calls f(valid, key, position) for every item of the source: the candidates staged in
// shared memory as (key, position), the candidate list in global memory (the same pairs),
// or the whole score row.  Uniform trip
// count: f may use warp votes.
template <class F>
__device__ __forceinline__ void for_each_item(int src, const uint2* s_stash, const uint2* cand,
                                              int n_items, const float* rs, F f) {
  const int tid = threadIdx.x;
  constexpr int U = 4;
  if (src == kFromStash) {
    for (int base = 0; base < n_items; base += kSelThreads) {
      const int i = base + tid;
      const bool v = i < n_items;
      const uint2 c = v ? s_stash[i] : make_uint2(0u, 0u);
      f(v, c.x, (int)c.y);
    }
  } else if (src == kFromList) {
    for (int base = 0; base < n_items; base += kSelThreads * U) {
      uint2 it[U];
      bool v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = base + u * kSelThreads + tid;
        v[u] = i < n_items;
        it[u] = v[u] ? __ldcg(cand + i) : make_uint2(0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) f(v[u], it[u].x, (int)it[u].y);
    }
  } else {
    for (int base = 0; base < n_items; base += kSelThreads * U) {
      float s[U];
      bool v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = base + u * kSelThreads + tid;
        v[u] = i < n_items;
        s[u] = v[u] ? __ldcg(rs + i) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < U; ++u) f(v[u], score_key(s[u]), base + u * kSelThreads + tid);
    }
  }
}

// Exact selection of the `r` largest of the source's items (ties: lowest position), appended
// to out[base_out ...].  Radix digits 12 / 12 / 8.  Returns the key of the r-th largest.
// Runs in one CTA; 1 <= r <= n_items.
__device__ uint32_t resolve_top_r(int src, const uint2* s_stash, const uint2* cand, int n_items,
                                  const float* rs, int n, int r, int32_t* out, uint32_t base_out,
                                  int k_max, uint32_t* s_hist, int* s_scan, uint32_t* s_emit) {
  const int tid = threadIdx.x;
  auto emit = [&](bool take, int pos) {
    const int p = warp_append(take, s_emit);
    if (p >= 0 && base_out + p < (uint32_t)k_max) out[base_out + p] = pos;
  };
  int d, above;
  // digit 1
  for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
  __syncthreads();
  for_each_item(src, s_stash, cand, n_items, rs, [&](bool v, uint32_t key, int) {
    if (v) atomicAdd(&s_hist[key >> 20], 1u);
  });
  __syncthreads();
  find_digit(s_hist, kHistBins, r, s_scan, d, above);
  const uint32_t d1 = (uint32_t)d;
  const int r1 = r - above;
  // digit 2 (and emit everything above digit 1)
  for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
  __syncthreads();
  for_each_item(src, s_stash, cand, n_items, rs, [&](bool v, uint32_t key, int pos) {
    const uint32_t t = key >> 20;
    emit(v && t > d1, pos);
    if (v && t == d1) atomicAdd(&s_hist[(key >> 8) & 0xfffu], 1u);
  });
  __syncthreads();
  find_digit(s_hist, kHistBins, r1, s_scan, d, above);
  const uint32_t p2 = (d1 << 12) | (uint32_t)d;    // 24-bit prefix of the r-th largest
  const int r2 = r1 - above;
  // digit 3 (and emit everything above digit 2 inside digit 1)
  for (int i = tid; i < 256; i += kSelThreads) s_hist[i] = 0u;
  __syncthreads();
  for_each_item(src, s_stash, cand, n_items, rs, [&](bool v, uint32_t key, int pos) {
    const uint32_t t = key >> 8;
    emit(v && (t >> 12) == d1 && t > p2, pos);
    if (v && t == p2) atomicAdd(&s_hist[key & 0xffu], 1u);
  });
  __syncthreads();
  find_digit(s_hist, 256, r2, s_scan, d, above);
  const uint32_t kstar = (p2 << 8) | (uint32_t)d;
  const int r3 = r2 - above;                       // how many items equal to the r-th are taken
  const int ties = (int)s_hist[d];
  int max_tie_pos = n;                             // take equal keys at positions <= this
  if (ties != r3) {
    // r3-th smallest position among the items equal to the r-th largest: bisection
    int plo = 0, phi = n - 1;
    while (plo < phi) {
      const int mid = plo + (phi - plo) / 2;
      int local = 0;
      for_each_item(src, s_stash, cand, n_items, rs, [&](bool v, uint32_t key, int pos) {
        if (v && key == kstar && pos <= mid) ++local;
      });
      const int cnt = block_count(local, s_scan);
      if (cnt >= r3) phi = mid; else plo = mid + 1;
    }
    max_tie_pos = plo;
  }
  for_each_item(src, s_stash, cand, n_items, rs, [&](bool v, uint32_t key, int pos) {
    emit(v && (key >> 8) == p2 && (key > kstar || (key == kstar && pos <= max_tie_pos)), pos);
  });
  __syncthreads();
  return kstar;
}

__global__ void __launch_bounds__(kSelThreads, 3)
sel_filter_kernel(Plan pl, const float* __restrict__ scores, uint32_t* __restrict__ counters,
                  const int32_t* __restrict__ rowstate, uint2* __restrict__ cand,
                  int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_count,
                  float* __restrict__ kth, int* __restrict__ status) {
  // main pass: a 512-entry hit buffer per warp; last CTA: histogram + candidate stash.
  // The two uses never overlap in time, so they share the same shared memory.
  extern __shared__ __align__(16) unsigned char s_raw[];          // kFilterSmemBytes
  uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_raw);
  uint2* s_stash = reinterpret_cast<uint2*>(s_raw + kHistBins * 4);
  uint32_t* s_hits = reinterpret_cast<uint32_t*>(s_raw);          // [16 warps][512]
  __shared__ int s_scan[34];
  __shared__ int s_last;
  __shared__ uint32_t s_emit, s_tie, s_kstar;
  const int row = blockIdx.y, tid = threadIdx.x, chunk = blockIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  pdl_launch_dependents();
  const float lo_f = __int_as_float(rowstate[row * 4 + 0]);
  const float hi_f = __int_as_float(rowstate[row * 4 + 1]);
  const int k = rowstate[row * 4 + 2], n = rowstate[row * 4 + 3];
  if (k == 0) return;
  const float* rs = scores + (size_t)row * pl.N_max;
  int32_t* out = sel_idx + (size_t)row * pl.k_max;
  uint2* rc = cand + (size_t)row * pl.cand_cap;          // (key, position) pairs
  uint32_t* n_out = &counters[row * 4 + 2];
  uint32_t* n_cand = &counters[row * 4 + 3];

  // Main pass.  Warps work independently: a lane marks which of its 16 scores reach the
  // bracket and the warp packs the positions of the hits (bit 31 = certain winner) into its
  // shared-memory buffer.  The buffer is written out when it would overflow and at the end,
  // with one atomic per destination list, so the round trip of that atomic is paid once per
  // warp and not once per chunk.
  const int n_chunks = (n + kSelChunk - 1) / kSelChunk;
  const bool no_winners = !(hi_f < CUDART_INF_F);   // bracket open at the top: candidates only
  constexpr int kBuf = kSelChunk / 16;              // entries per warp: one chunk's worst case
  uint32_t* my_hits = s_hits + warp * kBuf;
  int buf_n = 0;                                    // warp-uniform
  auto flush = [&]() {
    if (buf_n == 0) return;
    int nw = 0, nc = 0;
    for (int i0 = 0; i0 < buf_n; i0 += 32) {
      const bool v_ok = i0 + lane < buf_n;
      const uint32_t ent = v_ok ? my_hits[i0 + lane] : 0u;
      nw += __popc(__ballot_sync(0xffffffffu, v_ok && (ent >> 31)));
      nc += __popc(__ballot_sync(0xffffffffu, v_ok && !(ent >> 31)));
    }
    uint32_t bw = 0, bc = 0;
    if (lane == 0) {
      if (nw) bw = atomicAdd(n_out, (uint32_t)nw);
      if (nc) bc = atomicAdd(n_cand, (uint32_t)nc);
    }
    bw = __shfl_sync(0xffffffffu, bw, 0);
    bc = __shfl_sync(0xffffffffu, bc, 0);
    const unsigned lt = (1u << lane) - 1u;
    for (int i0 = 0; i0 < buf_n; i0 += 32) {
      const bool v_ok = i0 + lane < buf_n;
      const uint32_t ent = v_ok ? my_hits[i0 + lane] : 0u;
      const bool is_win = v_ok && (ent >> 31);
      const bool is_cnd = v_ok && !(ent >> 31);
      const unsigned mw = __ballot_sync(0xffffffffu, is_win);
      const unsigned mc = __ballot_sync(0xffffffffu, is_cnd);
      if (is_win) {
        const uint32_t p = bw + __popc(mw & lt);
        if (p < (uint32_t)pl.k_max) out[p] = (int)(ent & 0x7fffffffu);
      }
      if (is_cnd) {
        // the score comes back from L2 (this warp read it a moment ago), so that the row's
        // last CTA finds key and position together and has no dependent gather to wait for
        const uint32_t p = bc + __popc(mc & lt);
        if (p < (uint32_t)pl.cand_cap) rc[p] = make_uint2(score_key(__ldcg(rs + ent)), ent);
      }
      bw += __popc(mw);
      bc += __popc(mc);
    }
    __syncwarp();
    buf_n = 0;
  };
  for (int ch = chunk; ch < n_chunks; ch += gridDim.x) {
    float v[kElems];
    int pos0[4];
    load_chunk(rs, ch, n, v, pos0);
    const bool full = (ch + 1) * kSelChunk <= n;
    uint32_t hit = 0, win = 0;
    if (full && no_winners) {
#pragma unroll
      for (int e = 0; e < kElems; ++e) hit |= (v[e] >= lo_f ? 1u : 0u) << e;
    } else {
#pragma unroll
      for (int e = 0; e < kElems; ++e) {
        const bool valid = full || pos0[e >> 2] + (e & 3) < n;
        hit |= (valid && v[e] >= lo_f ? 1u : 0u) << e;
        win |= (valid && v[e] > hi_f ? 1u : 0u) << e;
      }
    }
    // exclusive scan of the per-lane hit counts over the warp
    const int mine = __popc(hit);
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += u;
    }
    const int total = __shfl_sync(0xffffffffu, inc, 31);
    if (total == 0) continue;                        // warp-uniform
    if (buf_n + total > kBuf) flush();
    int slot = buf_n + inc - mine;
    const int pos_base = ch * kSelChunk + tid * 4;   // position of element e: + (e>>2)*2048 + (e&3)
    while (hit) {
      const int e = __ffs(hit) - 1;
      hit &= hit - 1;
      my_hits[slot++] = (uint32_t)(pos_base + (e >> 2) * (kSelThreads * 4) + (e & 3)) |
                        (((win >> e) & 1u) << 31);
    }
    __syncwarp();
    buf_n += total;
  }
  flush();
  if (!cta_arrived_last(&counters[row * 4 + 1], gridDim.x, &s_last)) return;

  // ---- last CTA of the row: check the bracket by counting, then select among the candidates
  const int W = (int)__ldcg(n_out), C = (int)__ldcg(n_cand);
  if (tid == 0) s_emit = 0u;
  __syncthreads();
  uint32_t kstar;
  int emitted_before = W;
  if (W <= k && W + C >= k && C <= pl.cand_cap) {
    const int r = k - W;
    if (r == 0) {
      // no candidate is taken: the k-th largest is the smallest winner
      uint32_t mn = 0xffffffffu;
      for (int i = tid; i < W; i += kSelThreads)
        mn = min(mn, score_key(__ldcg(rs + __ldcg(out + i))));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      if (lane == 0) s_scan[warp] = (int)mn;
      __syncthreads();
      kstar = 0xffffffffu;
      for (int w = 0; w < kSelThreads / 32; ++w) kstar = min(kstar, (uint32_t)s_scan[w]);
      __syncthreads();
    } else {
      int src = kFromList;
      uint32_t kmin = 0xffffffffu, kmax = 0u;                  // range of the finite staged keys
      if (C <= kStashCap) {
        constexpr int kPer = kStashCap / kSelThreads;          // 10: all loads issued together
        uint2 it[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
          const int i = u * kSelThreads + tid;
          it[u] = i < C ? __ldcg(rc + i) : make_uint2(0x80000000u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
          const int i = u * kSelThreads + tid;
          if (i < C) {
            s_stash[i] = it[u];
            if (fabsf(key_score(it[u].x)) < CUDART_INF_F) {
              kmin = min(kmin, it[u].x);
              kmax = max(kmax, it[u].x);
            }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
          kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
        }
        if (lane == 0) { s_scan[warp] = (int)kmin; s_scan[16 + warp] = (int)kmax; }
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kSelThreads / 32; ++w) {
          kmin = min(kmin, (uint32_t)s_scan[w]);
          kmax = max(kmax, (uint32_t)s_scan[16 + w]);
        }
        __syncthreads();                                       // s_scan is reused below
        src = kFromStash;
      }
      bool done = false;
      if (src == kFromStash && kmax > kmin) {
        // Fast finish.  ONE histogram of the staged candidates over 4096 equal buckets of the
        // range of their finite scores (candidates at -inf, the sink and window positions of a
        // row that was not bracketed from below, fall into the bottom bucket) finds the bucket of
        // the r-th largest; everything in a higher bucket is taken at once, and the few items of
        // that bucket are ranked against each other (larger score first, then lower position:
        // the stable rule).
        const float lo_h = key_score(kmin);
        const float scale = (float)kHistBins / (key_score(kmax) - lo_h);
        for (int i = tid; i < kHistBins; i += kSelThreads) s_hist[i] = 0u;
        __syncthreads();
        for (int i = tid; i < C; i += kSelThreads)
          atomicAdd(&s_hist[linear_bucket(key_score(s_stash[i].x), lo_h, scale)], 1u);
        __syncthreads();
        int d, above;
        find_digit(s_hist, kHistBins, r, s_scan, d, above);
        const int m = (int)s_hist[d], need = r - above;        // 1 <= need <= m
        __syncthreads();                                         // everybody has read s_hist[d]
        constexpr int kTieCap = kHistBins / 2;                   // (key, position) pairs in s_hist's place
        if (m <= kTieCap) {
          uint2* tie = reinterpret_cast<uint2*>(s_hist);
          if (tid == 0) s_tie = 0u;
          __syncthreads();
          for (int base = 0; base < C; base += kSelThreads) {
            const int i = base + tid;
            const bool v = i < C;
            const uint2 it = v ? s_stash[i] : make_uint2(0u, 0u);
            const int bk = v ? linear_bucket(key_score(it.x), lo_h, scale) : -1;
            const int p = warp_append(v && bk > d, &s_emit);
            if (p >= 0 && (uint32_t)W + p < (uint32_t)pl.k_max) out[W + p] = (int)it.y;
            if (v && bk == d) tie[atomicAdd(&s_tie, 1u)] = it;
          }
          __syncthreads();
          for (int base = 0; base < m; base += kSelThreads) {
            const int i = base + tid;
            const bool v = i < m;
            const uint2 me = v ? tie[i] : make_uint2(0u, 0u);
            int rank = 0;
            for (int j = 0; j < m; ++j) {
              const uint2 o = tie[j];
              rank += (o.x > me.x || (o.x == me.x && o.y < me.y)) ? 1 : 0;
            }
            const int p = warp_append(v && rank < need, &s_emit);
            if (p >= 0 && (uint32_t)W + p < (uint32_t)pl.k_max) out[W + p] = (int)me.y;
            if (v && rank == need - 1) s_kstar = me.x;
          }
          __syncthreads();
          kstar = s_kstar;
          done = true;
        }
      }
      if (!done)
        kstar = resolve_top_r(src, s_stash, rc, C, rs, n, r, out, (uint32_t)W, pl.k_max, s_hist,
                              s_scan, &s_emit);
    }
  } else {
    // the sample's bracket missed: redo the row from the scores (slow, exact)
    emitted_before = 0;
    kstar = resolve_top_r(kFromRow, s_stash, rc, n, rs, n, k, out, 0u, pl.k_max, s_hist, s_scan,
                          &s_emit);
    if (tid == 0) atomicAdd(&counters[row * 4 + 0], 1u);   // fallback counter (diagnostic)
  }
  if (tid == 0) {
    sel_count[row] = k;
    kth[row] = key_score(kstar);
    if (emitted_before + (int)s_emit != k) atomicOr(status, kStatusCountMismatch);
  }
}

}  // namespace

cudaError_t launch_select(const Plan& pl, const WsLayout& L, char* ws, const float* scores,
                          const int32_t* seq_lens, int32_t* sel_idx, int32_t* sel_count,
                          float* kth, cudaStream_t st) {
  uint32_t* counters = reinterpret_cast<uint32_t*>(ws + L.counters);
  int32_t* rowstate = reinterpret_cast<int32_t*>(ws + L.rowstate);
  uint2* cand = reinterpret_cast<uint2*>(ws + L.cand);
  int* status = reinterpret_cast<int*>(ws + L.status);
  cudaError_t e = launch_pdl(sel_sample_kernel, dim3(pl.rows), dim3(kSelThreads), 0, st, pl, scores,
                             seq_lens, rowstate, sel_count, kth);
  if (e != cudaSuccess) return e;
  // more than 48 KB of dynamic shared memory needs an opt-in (per device, so set every time)
  e = cudaFuncSetAttribute(sel_filter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kFilterSmemBytes);
  if (e != cudaSuccess) return e;
  return launch_pdl(sel_filter_kernel, dim3(pl.hist_chunks, pl.rows), dim3(kSelThreads),
                    kFilterSmemBytes, st, pl,
                    scores, counters, rowstate, cand, sel_idx, sel_count, kth, status);
}

}  // namespace pqhsa
