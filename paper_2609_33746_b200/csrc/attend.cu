// Step 4 of the decode operator: hybrid exact + background attention (Eq. 4-5).
//
//   background preparation (one CTA per score row)
//       merges the scan's per-segment list sums by log-sum-exp, takes the selected tokens'
//       approximate mass exp(l~_i - m) out of their lists (M_j = sum over B n R_j, Eq. 4) and
//       leaves M_j (clamped at 0) relative to m = max_i l~_i;
//   attend (split-K, several CTAs per score row)
//       each CTA gathers a slice of the selected K/V rows from the paged cache in place,
//       computes exact logits q.k_i/sqrt(d) with an online softmax, and adds a slice of the
//       background terms M_j * vbar_j; the last CTA of the row to finish merges the partial
//       (m, Z, N) triples and writes y^ = (N_E + N^_B) / (Z_E + Z^_B)  (Eq. 5).
// All exponentials are taken in base 2 on logits pre-multiplied by log2(e).
//
// The mechanism variants of the paper's ablation (Table 2; App. B) change the background term
// only: T drops it, C / C2 / C2b replace the list means by one global mean (and C2 / C2b the
// logits by one shared logit), Bx replaces each list mean by the mean of the list's unselected
// members, which costs one more pass over the selected value rows (bx_corr_kernel).
//
// Launch order and dependencies: bg_prep_kernel -> [bx_corr_kernel] -> attend_kernel, each
// launched with programmatic stream serialisation.  EVERY CTA of bg_prep_kernel and of
// bx_corr_kernel executes griddepcontrol.wait before it lets its dependents go and before it
// can return; so when a CTA of attend_kernel starts, the kernels before bg_prep_kernel (scan,
// top-k) are complete.  That is what allows the exact CTAs of attend_kernel, which read only
// what the top-k wrote, to skip their own griddepcontrol.wait and run beside the background
// preparation.  Nothing may be added above those waits that returns early.
#include "attn_common.cuh"
#include "common.cuh"
#include "scan_common.cuh"

namespace pqhsa {

namespace {

constexpr int kBgThreads = 128;

__device__ __forceinline__ int attend_parts_dev(const Plan& pl) {
  return pl.splits + pl.bg_splits + (pl.variant == PQHSA_VARIANT_BX ? pl.splits : 0);
}

// grid (bg_ctas, rows).  CTA c merges a slice of the lists and subtracts a slice of the
// selected tokens; both go into bg_mass (zeroed by the caller) with float atomics, so the
// CTAs of a row need no ordering.  A list's mass can come out slightly negative when its
// members are all selected (rounding); the consumer clamps at 0.
__global__ void __launch_bounds__(kBgThreads)
bg_prep_kernel(Plan pl, const float* __restrict__ scores, const float* __restrict__ partials,
               const int32_t* __restrict__ sel_idx, const int32_t* __restrict__ sel_count,
               const uint16_t* __restrict__ lids, const int32_t* __restrict__ seq_lens,
               float* __restrict__ bg_mass, float* __restrict__ bg_max,
               float* __restrict__ bg_aux, int32_t* __restrict__ bg_tcount) {
  __shared__ float s_scale[kMaxSeg], s_ref2[kMaxSeg];
  __shared__ int s_segend[kMaxSeg];      // first tile of the row (32-token units) past segment sg
  const int row = blockIdx.y, c = blockIdx.x, C = gridDim.x, tid = threadIdx.x;
  const int b = row / pl.Hq, h = row % pl.Hq;
  const int kv = h / pl.G, hg = (h % pl.G) / pl.Gc;
  const int n_list = pl.n_list;
  pdl_wait();               // (nothing above this line may return: see the file header)
  pdl_launch_dependents();
  const int n = clamp_len(seq_lens[b], pl.N_max);
  float* mass = bg_mass + (size_t)row * n_list;
  if (n == 0 || pl.variant == PQHSA_VARIANT_T) {          // T: no background term at all
    if (c == 0 && tid == 0) bg_max[row] = -CUDART_INF_F;
    return;
  }
  // the selected tokens of this CTA's slice: start their gathers first
  const int cnt = min(max(sel_count[row], 0), pl.k_max);   // (a count outside [0, k_max] is not followed)
  const int tl = (int)((long long)c * cnt / C), th = (int)((long long)(c + 1) * cnt / C);
  const int32_t* sel = sel_idx + (size_t)row * pl.k_max;
  const float* rs = scores + (size_t)row * pl.N_max;
  const uint16_t* rl = lids + ((size_t)b * pl.Hkv + kv) * pl.N_max;
  constexpr int kSelPer = 6;
  int idx[kSelPer];
  float sc[kSelPer];
  uint32_t li[kSelPer];
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) {
    const int t = tl + u * kBgThreads + tid;
    const int v = t < th ? sel[t] : -1;
    idx[u] = (unsigned)v < (unsigned)n ? v : -1;          // a position outside the sequence is skipped
#ifdef PQHSA_DEBUG
    {
      const Region rg_dbg = region_of(pl, n, b);
      PQHSA_DEBUG_CHECK(t >= th || position_ok(v, rg_dbg.r_begin, rg_dbg.r_end), kStatusPosition, pl.status);
    }
#endif
  }
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) {
    sc[u] = idx[u] >= 0 ? rs[idx[u]] : 0.f;
    li[u] = idx[u] >= 0 ? min((uint32_t)rl[idx[u]], (uint32_t)(n_list - 1)) : 0u;
  }
  if (pl.variant == PQHSA_VARIANT_C2 || pl.variant == PQHSA_VARIANT_C2B) {
    // one shared logit for every background token: C2 needs the mean approximate logit of the
    // selected tokens (summed here), C2b the smallest exact logit (found by the attend kernel)
    if (pl.variant == PQHSA_VARIANT_C2) {
      float part = 0.f;
#pragma unroll
      for (int u = 0; u < kSelPer; ++u) part += sc[u];
      for (int t = tl + kSelPer * kBgThreads + tid; t < th; t += kBgThreads) {
        const int i = sel[t];
        if ((unsigned)i < (unsigned)n) part += rs[i];
      }
      part = warp_sum(part);
      if ((tid & 31) == 0 && part != 0.f) atomicAdd(&bg_aux[row * 4], part);
    }
    if (c == 0 && tid == 0) bg_max[row] = 0.f;            // marks "has a background"
    return;
  }

  // which scan segments cover this row's unit
  const ScanSplit sp = scan_split(seq_lens, pl.B, pl.N_max, pl.upb, pl.scan_ctas);
  long long base = 0;
  for (int bb = 0; bb < b; ++bb) base += (long long)seq_tiles(seq_lens, bb, pl.N_max) * pl.upb;
  const int tb = seq_tiles(seq_lens, b, pl.N_max);
  const long long s_u = base + (long long)(kv * pl.n_hg + hg) * tb;
  const int c_first = split_cta_of(sp, s_u);
  const int nseg = min(kMaxSeg, split_cta_of(sp, s_u + tb - 1) - c_first + 1);
  // the unit's partials: per segment a header [2 Gc] (reference, maximum per head) and the sums
  // [n_list][Gc] relative to the reference
  const int Gc = pl.Gc, g = (h % pl.G) % Gc;
  const size_t seg_stride = (size_t)Gc * (n_list + 2);
  const float* pr = partials + (((size_t)b * pl.Hkv + kv) * pl.n_hg + hg) * pl.n_part * seg_stride;

  float m = -CUDART_INF_F;
  for (int sg = tid; sg < nseg; sg += kBgThreads) {                    // segment maxima
    const float v = pr[(size_t)sg * seg_stride + Gc + g];
    s_scale[sg] = v;
  }
  __syncthreads();
  for (int s = 0; s < nseg; ++s) m = fmaxf(m, s_scale[s]);
  if (!(m > -CUDART_INF_F)) {            // no token of R in this row: no background at all
    if (c == 0 && tid == 0) bg_max[row] = -CUDART_INF_F;
    return;
  }
  const float m2 = m * kLog2e;
  __syncthreads();
  for (int sg = tid; sg < nseg; sg += kBgThreads) {
    // a segment's sums are relative to its reference: exp2(l~ log2 e - ref log2 e)
    const float ref = pr[(size_t)sg * seg_stride + g];
    s_scale[sg] = s_scale[sg] > -CUDART_INF_F ? fast_exp2(ref * kLog2e - m2) : 0.f;
    s_ref2[sg] = __fmul_rn(ref, kLog2e);           // the scan's own product, rounded as there
    s_segend[sg] = sg + 1 < nseg ? (int)(split_start(sp, c_first + sg + 1) - s_u) : 0x7fffffff;
  }
  __syncthreads();
  const int jl = (int)((long long)c * n_list / C), jh = (int)((long long)(c + 1) * n_list / C);
  const float* sums = pr + 2 * Gc + g;
  for (int j = jl + tid; j < jh; j += kBgThreads) {
    float acc = 0.f;
    for (int s0 = 0; s0 < nseg; s0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        v[u] = (s0 + u < nseg) ? sums[(size_t)(s0 + u) * seg_stride + (size_t)j * Gc] : 0.f;
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (s0 + u < nseg) acc = fmaf(v[u], s_scale[s0 + u], acc);
    }
    if (acc != 0.f) atomicAdd(&mass[j], acc);
  }
  // Take the selected tokens out of their lists' sums.  A selected token can hold nearly all of
  // its list's mass, and what is left after the subtraction is multiplied by the list's mean
  // value, so the term taken out is formed exactly as the scan formed the term it put in (the
  // exponent against the reference of the token's own segment, the same instructions) and
  // scaled like that segment's sums: what remains is the rounding of the additions alone.
  const float inv_seg_tiles = (float)sp.P_eff / (float)sp.T;          // segments per tile
  const float tile_off = (float)(s_u - split_start(sp, c_first));     // tiles of segment 0 before this unit
  auto take_out = [&](int i, float s, uint32_t lid) {
    // segments are equally long up to one tile: estimate, then settle against the boundaries
    const int tile = i / kTile;
    int sg = min(nseg - 1, max(0, (int)(((float)tile + tile_off) * inv_seg_tiles)));
    while (sg > 0 && tile < s_segend[sg - 1]) --sg;
    while (tile >= s_segend[sg]) ++sg;             // (the last entry is INT_MAX)
    const float x = fmaf(s, kLog2e, -s_ref2[sg]);
    if (x > kScanNegligibleLog2) atomicAdd(&mass[lid], -(fast_exp2(x) * s_scale[sg]));
    if (bg_tcount != nullptr) atomicAdd(&bg_tcount[(size_t)row * n_list + lid], 1);
  };
#pragma unroll
  for (int u = 0; u < kSelPer; ++u)
    if (idx[u] >= 0) take_out(idx[u], sc[u], li[u]);
  for (int t = tl + kSelPer * kBgThreads + tid; t < th; t += kBgThreads) {
    const int i = sel[t];
    if ((unsigned)i >= (unsigned)n) continue;
    take_out(i, rs[i], min((uint32_t)rl[i], (uint32_t)(n_list - 1)));
  }
  if (c == 0 && tid == 0) bg_max[row] = m;
}

// One grid, two kinds of CTA.
//   CTAs [0, rows * S): split s of score row r gathers its share of the selected K/V rows
//     (8 lanes per 256-byte row, 16 rows in flight per warp, positions and page ids fetched
//     one 32-token window ahead) and keeps an online softmax in base 2.  These CTAs read
//     only what the top-k wrote, so they do not wait for the background preparation, which
//     runs while they gather.
//   CTAs [rows * S, rows * S + units * BS): slice c of the lists of one (sequence, KV head,
//     head group): Z += M_j, N += M_j * vbar_j for the up to 4 heads of the group from one
//     read of the vbar rows.  These wait for the background preparation.
// Every CTA leaves one partial per row it worked for and takes a ticket of that row; the
// CTA that draws the last ticket merges the row (nobody waits).
template <typename T, int U>
__global__ void __launch_bounds__(kAttendThreads, 4)
attend_kernel(Plan pl, const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
              long long stride_page, long long stride_token, long long stride_head,
              const int32_t* __restrict__ block_table, const int32_t* __restrict__ sel_idx,
              const int32_t* __restrict__ sel_count, const int32_t* __restrict__ seq_lens,
              const float* __restrict__ bg_mass, const float* __restrict__ bg_max,
              const float* __restrict__ bg_aux, const int32_t* __restrict__ bg_tcount,
              const float* __restrict__ vmeans, const int32_t* __restrict__ list_counts,
              float* __restrict__ split_part, uint32_t* __restrict__ tickets,
              T* __restrict__ out, float* __restrict__ lse, float* __restrict__ out_f32) {
  constexpr int kWarps = kAttendThreads / 32;
  __shared__ float s_m[kWarps], s_Z[4 * kWarps], s_m4[4 * kWarps];
  __shared__ __align__(16) float s_N[4 * kWarps][kHeadDim];
  __shared__ int s_last[4];
  __shared__ float s_aux[kMaxParts + 8];

  const int S = pl.splits, BS = pl.bg_splits, n_part = attend_parts_dev(pl);
  const int n_tickets = S + BS;            // CTAs of this kernel that work for a row
  const int variant = pl.variant;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_list = pl.n_list;

  if ((int)blockIdx.x >= pl.rows * S) {
    // ================= background CTA =================
    const int id = (int)blockIdx.x - pl.rows * S;
    const int unit = id / BS, c = id % BS;                  // unit = (b, kv, head group)
    const int hg = unit % pl.n_hg, kv = (unit / pl.n_hg) % pl.Hkv, b = unit / (pl.n_hg * pl.Hkv);
    const int h0 = kv * pl.G + hg * pl.Gc;                  // first head of the group
    const int n_heads = min(pl.Gc, pl.G - hg * pl.Gc);
    const int row0 = b * pl.Hq + h0;
    pdl_wait();
    pdl_launch_dependents();
    const int jl = (int)((long long)c * n_list / BS), jh = (int)((long long)(c + 1) * n_list / BS);
    const int per = (jh - jl + kWarps - 1) / kWarps;
    const int a = min(jh, jl + warp * per), e = min(jh, a + per);
    const float4* vm = reinterpret_cast<const float4*>(
        vmeans + ((size_t)b * pl.Hkv + kv) * n_list * kHeadDim);
    const int32_t* cnt_j = list_counts ? list_counts + ((size_t)b * pl.Hkv + kv) * n_list : nullptr;
    // lane (g, i) = (lane >> 3, lane & 7) fetches the mass of head g for list j0 + i
    const int mg = lane >> 3, mi = lane & 7;
    const size_t mrow = (size_t)(row0 + (mg < n_heads ? mg : 0)) * n_list;
    const bool global_mean = variant >= PQHSA_VARIANT_C;   // C, C2, C2b: one mean for all lists
    const bool shared_logit = variant >= PQHSA_VARIANT_C2;
    float4 acc[4];
    float z = 0.f;                                          // lane (g, *) sums head g's masses
    float4 cw = make_float4(0.f, 0.f, 0.f, 0.f);            // sum_j |R_j| vbar_j (this lane's 4 dims)
    float ctot = 0.f;                                       // sum_j |R_j|
#pragma unroll
    for (int g = 0; g < 4; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j0 = a; j0 < e; j0 += 8) {
      const bool in = mg < n_heads && j0 + mi < e;
      float mine = (in && !shared_logit) ? fmaxf(bg_mass[mrow + j0 + mi], 0.f) : 0.f;   // M_j
      float wgt = mine;                                     // what multiplies vbar_j
      float nj = 0.f;
      if (cnt_j != nullptr && j0 + mi < e) nj = (float)cnt_j[j0 + mi];
      if (variant == PQHSA_VARIANT_BX) {
        // mean of the list's unselected members: (|R_j| vbar_j - sum_{T n R_j} v_i) / |B n R_j|;
        // the sum over the selected members is taken out by bx_corr_kernel
        const float left = in ? nj - (float)bg_tcount[mrow + j0 + mi] : 0.f;
        mine = left > 0.f ? mine : 0.f;
        wgt = left > 0.f ? mine * nj / left : 0.f;
      }
      const unsigned nz = __ballot_sync(0xffffffffu, global_mean ? nj > 0.f : wgt > 0.f);
      const unsigned live = (nz | (nz >> 8) | (nz >> 16) | (nz >> 24)) & 0xffu;   // any head
      float4 v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if ((live >> i) & 1u) v[i] = __ldg(vm + (size_t)(j0 + i) * (kHeadDim / 4) + lane);
      }
      z += mine;
      if (global_mean) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float n_i = __shfl_sync(0xffffffffu, nj, i);   // lane (0, i) holds list j0 + i
          cw.x = fmaf(n_i, v[i].x, cw.x); cw.y = fmaf(n_i, v[i].y, cw.y);
          cw.z = fmaf(n_i, v[i].z, cw.z); cw.w = fmaf(n_i, v[i].w, cw.w);
          ctot += n_i;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const float mj = __shfl_sync(0xffffffffu, wgt, 8 * g + i);
            acc[g].x = fmaf(mj, v[i].x, acc[g].x); acc[g].y = fmaf(mj, v[i].y, acc[g].y);
            acc[g].z = fmaf(mj, v[i].z, acc[g].z); acc[g].w = fmaf(mj, v[i].w, acc[g].w);
          }
        }
      }
    }
    z += __shfl_xor_sync(0xffffffffu, z, 1);
    z += __shfl_xor_sync(0xffffffffu, z, 2);
    z += __shfl_xor_sync(0xffffffffu, z, 4);
    if (global_mean) {
      // every lane has added the same counts, and the warps hold disjoint lists: the CTA (the
      // only background CTA of the unit for these variants) sums both over its warps below
      *reinterpret_cast<float4*>(&s_N[4 * warp][4 * lane]) = cw;
      if (lane == 0) s_Z[4 * warp] = ctot;
      if (mi == 0) s_m4[4 * warp + mg] = z;
    } else {
#pragma unroll
      for (int g = 0; g < 4; ++g) *reinterpret_cast<float4*>(&s_N[4 * warp + g][4 * lane]) = acc[g];
      if (mi == 0) s_Z[4 * warp + mg] = z;
    }
    __syncthreads();
    for (int g = 0; g < n_heads; ++g) {
      float Z_c = 0.f, N_c = 0.f, m_c = bg_max[row0 + g] * kLog2e, kind = 0.f;
      if (!global_mean) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { Z_c += s_Z[4 * w + g]; N_c += s_N[4 * w + g][tid]; }
      } else {
        float tot = 0.f, wsum = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { tot += s_Z[4 * w]; wsum += s_N[4 * w][tid]; Z_c += s_m4[4 * w + g]; }
        const float vg = tot > 0.f ? wsum / tot : 0.f;      // global mean value, this thread's dim
        if (shared_logit) {
          // every background token carries the same logit: Z = |B|, N = |B| vbar_global
          const int row = row0 + g;
          const int n_seq = clamp_len(seq_lens[b], pl.N_max);
          const Region rg = region_of(pl, n_seq, b);
          const int k_sel = min(max(sel_count[row], 0), pl.k_max);
          Z_c = (float)max(0, rg.r_end - rg.r_begin - k_sel);
          if (k_sel <= 0 || !(bg_max[row] > -CUDART_INF_F)) Z_c = 0.f;   // no T: no shared logit
          if (variant == PQHSA_VARIANT_C2) m_c = (k_sel > 0 ? bg_aux[row * 4] / (float)k_sel : 0.f) * kLog2e;
          else { m_c = 0.f; kind = kKindSharedMin; }                      // logit set at the merge
        }
        N_c = Z_c * vg;
      }
      float* part = split_part + ((size_t)(row0 + g) * n_part + S + c) * kPartStride;
      part[4 + tid] = N_c;
      if (tid == 0) { part[0] = m_c; part[1] = Z_c; part[2] = CUDART_INF_F; part[3] = kind; }
    }
    // one ticket per row of the group (see cta_arrived_last for the fences)
    __syncthreads();
    if (tid < n_heads) {
      __threadfence();
      const bool last = atomicAdd(&tickets[row0 + tid], 1u) == (uint32_t)(n_tickets - 1);
      if (last) __threadfence();
      s_last[tid] = last ? 1 : 0;
    }
    __syncthreads();
    for (int g = 0; g < n_heads; ++g) {
      if (!s_last[g]) continue;
      merge_row(split_part + (size_t)(row0 + g) * n_part * kPartStride, n_part, row0 + g, tid,
                s_N, s_aux, out, lse, out_f32);
    }
    return;
  }

  // ================= exact (selected-token) CTA =================
  const int row = (int)blockIdx.x / S, split = (int)blockIdx.x % S;
  const int b = row / pl.Hq, h = row % pl.Hq, kv = h / pl.G;
  // (variant Bx: the CTA that merges a row also reads the correction partials of the kernel
  // right before this one, so it cannot skip the wait)
  if (variant == PQHSA_VARIANT_BX) pdl_wait();
  pdl_launch_dependents();
  // the exact set E = T u S u L (Sec. 3.2), as one index space: the selected tokens first,
  // then the sink prefix, then the local window
  const int cnt = min(max(sel_count[row], 0), pl.k_max);   // (a count outside [0, k_max] is not followed)
  const int n_seq = clamp_len(seq_lens[b], pl.N_max);
  const Region rg = region_of(pl, n_seq, b);
  const int n_s = rg.r_begin, n_exact = cnt + n_s + (n_seq - rg.r_end);
  const int tl = (int)((long long)split * n_exact / S);
  const int th = (int)((long long)(split + 1) * n_exact / S);
  const int per_warp = (th - tl + kWarps - 1) / kWarps;
  const int wl = min(th, tl + warp * per_warp), wh = min(th, wl + per_warp);
  const int32_t* sel = sel_idx + (size_t)row * pl.k_max;
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;
  auto pos_of = [&](int t) -> int {        // position of item t of E, -1 past the warp's slice
    if (t >= wh) return -1;
    if (t < cnt) {                          // (a position outside the sequence is skipped)
      const int v = sel[t];
      return (unsigned)v < (unsigned)n_seq ? v : -1;
    }
    const int u = t - cnt;
    return u < n_s ? u : rg.r_end + (u - n_s);
  };
  int my_pos = pos_of(wl + lane);

  const int gi = lane >> 3, gl = lane & 7;      // lane group (4 per warp) and lane in group
  float qf[16];
  {
    const T* qr = q + (size_t)row * kHeadDim;
    const float sc = pl.sm_scale * kLog2e;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      qf[t] = sc * Unpack<T>::one(qr[8 * gl + t]);
      qf[8 + t] = sc * Unpack<T>::one(qr[64 + 8 * gl + t]);
    }
  }
  GroupState st;
  st.m = -CUDART_INF_F;
  st.Z = 0.f;
  float lmin = CUDART_INF_F;               // smallest exact logit among the selected tokens seen
#pragma unroll
  for (int t = 0; t < 16; ++t) st.acc[t] = 0.f;

  // page id of this lane's first token (second dependent load); later windows prefetch
  // position and page one window ahead, while the current window's rows are in flight
  int my_page = my_pos >= 0 ? __ldg(bt + my_pos / pl.page_size) : 0;
  PQHSA_DEBUG_CHECK(page_ok(my_page), kStatusPage, pl.status);
  for (int base = wl; base < wh; base += 32) {
    long long off = -1;                      // -1: nothing to read (past the slice or skipped)
    if (my_pos >= 0)
      off = (long long)my_page * stride_page + (long long)(my_pos % pl.page_size) * stride_token +
            (long long)kv * stride_head;
    const int nxt_pos = pos_of(base + 32 + lane);
    int nxt_page = 0;
    const int nb = min(32, wh - base);
    for (int j0 = 0; j0 < nb; j0 += 4 * U) {
      uint4 kr[U][2], vr[U][2];
      bool ok[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int tok = j0 + 4 * u + gi;
        const long long o = __shfl_sync(0xffffffffu, off, tok & 31);
        ok[u] = tok < nb && o >= 0;
        if (ok[u]) {
          const uint4* kp = reinterpret_cast<const uint4*>(kc + o);
          const uint4* vp = reinterpret_cast<const uint4*>(vc + o);
          kr[u][0] = __ldg(kp + gl); kr[u][1] = __ldg(kp + 8 + gl);
          vr[u][0] = __ldg(vp + gl); vr[u][1] = __ldg(vp + 8 + gl);
        } else {
          kr[u][0] = kr[u][1] = vr[u][0] = vr[u][1] = make_uint4(0u, 0u, 0u, 0u);
        }
      }
      if (j0 == 0 && nxt_pos >= 0) nxt_page = __ldg(bt + nxt_pos / pl.page_size);
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float kf[8];
        float s = 0.f;
        Unpack<T>::run(kr[u][0], kf);
#pragma unroll
        for (int t = 0; t < 8; ++t) s = fmaf(qf[t], kf[t], s);
        Unpack<T>::run(kr[u][1], kf);
#pragma unroll
        for (int t = 0; t < 8; ++t) s = fmaf(qf[8 + t], kf[t], s);
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        s += __shfl_xor_sync(0xffffffffu, s, 4);
        if (ok[u]) {                                  // uniform within the lane group
          if (base + j0 + 4 * u + gi < cnt) lmin = fminf(lmin, s);
          if (s > st.m) {
            const float a = st.Z > 0.f ? fast_exp2(st.m - s) : 0.f;
            st.Z *= a;
#pragma unroll
            for (int t = 0; t < 16; ++t) st.acc[t] *= a;
            st.m = s;
          }
          const float p = fast_exp2(s - st.m);
          st.Z += p;
          float vf[8];
          Unpack<T>::run(vr[u][0], vf);
#pragma unroll
          for (int t = 0; t < 8; ++t) st.acc[t] = fmaf(p, vf[t], st.acc[t]);
          Unpack<T>::run(vr[u][1], vf);
#pragma unroll
          for (int t = 0; t < 8; ++t) st.acc[8 + t] = fmaf(p, vf[t], st.acc[8 + t]);
        }
      }
    }
    my_pos = nxt_pos;
    my_page = nxt_page;
  }
  // merge the 4 lane groups of the warp (lanes with equal gl own the same dims)
#pragma unroll
  for (int o = 8; o <= 16; o <<= 1) {
    const float m_o = __shfl_xor_sync(0xffffffffu, st.m, o);
    const float Z_o = __shfl_xor_sync(0xffffffffu, st.Z, o);
    const float m_n = fmaxf(st.m, m_o);
    const float a = safe_scale(st.m, m_n, st.Z), bsc = safe_scale(m_o, m_n, Z_o);
    st.Z = st.Z * a + Z_o * bsc;
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      const float acc_o = __shfl_xor_sync(0xffffffffu, st.acc[t], o);
      st.acc[t] = st.acc[t] * a + acc_o * bsc;
    }
    st.m = m_n;
  }
  lmin = fminf(lmin, __shfl_xor_sync(0xffffffffu, lmin, 8));
  lmin = fminf(lmin, __shfl_xor_sync(0xffffffffu, lmin, 16));
  if (gi == 0) {
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      s_N[warp][8 * gl + t] = st.acc[t];
      s_N[warp][64 + 8 * gl + t] = st.acc[8 + t];
    }
    if (gl == 0) { s_m[warp] = st.m; s_Z[warp] = st.Z; s_m4[warp] = lmin; }
  }
  __syncthreads();

  // ---- CTA partial: thread d owns output dim d
  float m_c = -CUDART_INF_F;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) if (s_Z[w] > 0.f) m_c = fmaxf(m_c, s_m[w]);
  float Z_c = 0.f, N_c = 0.f;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const float a = safe_scale(s_m[w], m_c, s_Z[w]);
    Z_c = fmaf(s_Z[w], a, Z_c);
    N_c = fmaf(s_N[w][tid], a, N_c);
  }
  float* part = split_part + ((size_t)row * n_part + split) * kPartStride;
  part[4 + tid] = N_c;
  if (tid == 0) {
    part[0] = m_c; part[1] = Z_c;
    part[2] = fminf(fminf(s_m4[0], s_m4[1]), fminf(s_m4[2], s_m4[3]));
    part[3] = 0.f;
  }
  if (!cta_arrived_last(&tickets[row], (uint32_t)n_tickets, &s_last[0])) return;
  merge_row(split_part + (size_t)row * n_part * kPartStride, n_part, row, tid, s_N, s_aux, out, lse,
            out_f32);
}

// Variant Bx (App. B): the background value of list j is the mean of its UNSELECTED members,
// (|R_j| vbar_j - sum_{i in T n R_j} v_i) / |B n R_j|.  The background CTAs of attend_kernel
// add M_j |R_j| / |B n R_j| * vbar_j; this kernel takes out sum_i w_i v_i over the selected
// tokens, w_i = M_j / |B n R_j| with j = a_i, as one more partial per exact split ("raw N":
// it changes the numerator only; the normaliser stays B's).  grid (splits, rows), 128 threads:
// thread d owns output dim d and walks the split's selected tokens; the 256-byte value row is
// read by the whole CTA at once.
template <typename T>
__global__ void __launch_bounds__(kAttendThreads)
bx_corr_kernel(Plan pl, const T* __restrict__ vc, long long stride_page, long long stride_token,
               long long stride_head, const int32_t* __restrict__ block_table,
               const int32_t* __restrict__ sel_idx, const int32_t* __restrict__ sel_count,
               const int32_t* __restrict__ seq_lens, const uint16_t* __restrict__ lids,
               const int32_t* __restrict__ list_counts, const float* __restrict__ bg_mass,
               const float* __restrict__ bg_max, const int32_t* __restrict__ bg_tcount,
               float* __restrict__ split_part) {
  const int split = blockIdx.x, row = blockIdx.y, tid = threadIdx.x;
  const int b = row / pl.Hq, h = row % pl.Hq, kv = h / pl.G;
  const int S = pl.splits, n_part = attend_parts_dev(pl), n_list = pl.n_list;
  pdl_wait();               // (nothing above this line may return: see the file header)
  pdl_launch_dependents();
  const int n_seq = clamp_len(seq_lens[b], pl.N_max);
  const int cnt = min(max(sel_count[row], 0), pl.k_max);   // (a count outside [0, k_max] is not followed)
  const int tl = (int)((long long)split * cnt / S), th = (int)((long long)(split + 1) * cnt / S);
  const int32_t* sel = sel_idx + (size_t)row * pl.k_max;
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  const uint16_t* rl = lids + ukv * pl.N_max;
  const int32_t* cj = list_counts + ukv * n_list;
  const float* mass = bg_mass + (size_t)row * n_list;
  const int32_t* tc = bg_tcount + (size_t)row * n_list;
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;
  float acc = 0.f;
  for (int t = tl; t < th; ++t) {
    const int pos = sel[t];
    if ((unsigned)pos >= (unsigned)n_seq) continue;                    // uniform over the CTA
    const uint32_t j = min((uint32_t)rl[pos], (uint32_t)(n_list - 1));
    const float left = (float)(cj[j] - tc[j]);
    const float w = left > 0.f ? fmaxf(mass[j], 0.f) / left : 0.f;
    if (w == 0.f) continue;
    const long long off = (long long)bt[pos / pl.page_size] * stride_page +
                          (long long)(pos % pl.page_size) * stride_token + (long long)kv * stride_head;
    acc = fmaf(w, Unpack<T>::one(vc[off + tid]), acc);
  }
  float* part = split_part + ((size_t)row * n_part + S + pl.bg_splits + split) * kPartStride;
  part[4 + tid] = -acc;
  if (tid == 0) {
    part[0] = bg_max[row] * kLog2e; part[1] = 0.f; part[2] = CUDART_INF_F; part[3] = kKindRaw;
  }
}

}  // namespace

cudaError_t launch_attend(const Plan& pl_in, const WsLayout& L, char* ws, const void* q,
                          const pqhsa_paged_kv& kv, const pqhsa_index& ix, const float* scores,
                          const float* list_partials, const int32_t* sel_idx,
                          const int32_t* sel_count, const int32_t* seq_lens, void* out,
                          float* lse, float* out_f32, cudaStream_t st) {
  Plan plan = pl_in;
  plan.status = reinterpret_cast<int*>(ws + L.status);
  const Plan& pl = plan;
  float* bg_mass = reinterpret_cast<float*>(ws + L.bg_mass);
  float* bg_max = reinterpret_cast<float*>(ws + L.bg_max);
  float* bg_aux = reinterpret_cast<float*>(ws + L.bg_aux);
  int32_t* bg_tcount = pl.variant == PQHSA_VARIANT_BX ? reinterpret_cast<int32_t*>(ws + L.bg_tcount)
                                                      : nullptr;
  float* split_part = reinterpret_cast<float*>(ws + L.split_part);
  uint32_t* tickets = reinterpret_cast<uint32_t*>(ws + L.attend_tickets);
  if (attend_parts(pl) > kMaxParts) return cudaErrorInvalidValue;
  cudaError_t e = launch_pdl(bg_prep_kernel, dim3(pl.bg_ctas, pl.rows), dim3(kBgThreads), 0, st, pl,
                             scores, list_partials, sel_idx, sel_count, ix.list_ids, seq_lens,
                             bg_mass, bg_max, bg_aux, bg_tcount);
  if (e != cudaSuccess) return e;
  const bool f16 = pl.dtype == PQHSA_F16;
  if (pl.variant == PQHSA_VARIANT_BX) {
    const dim3 g2(pl.splits, pl.rows);
    if (f16)
      e = launch_pdl(bx_corr_kernel<__half>, g2, dim3(kAttendThreads), 0, st, pl,
                     static_cast<const __half*>(kv.v_cache), (long long)kv.stride_page,
                     (long long)kv.stride_token, (long long)kv.stride_head, kv.block_table, sel_idx,
                     sel_count, seq_lens, ix.list_ids, ix.list_counts, bg_mass, bg_max, bg_tcount,
                     split_part);
    else
      e = launch_pdl(bx_corr_kernel<__nv_bfloat16>, g2, dim3(kAttendThreads), 0, st, pl,
                     static_cast<const __nv_bfloat16*>(kv.v_cache), (long long)kv.stride_page,
                     (long long)kv.stride_token, (long long)kv.stride_head, kv.block_table, sel_idx,
                     sel_count, seq_lens, ix.list_ids, ix.list_counts, bg_mass, bg_max, bg_tcount,
                     split_part);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(pl.rows * pl.splits + pl.B * pl.Hkv * pl.n_hg * pl.bg_splits);
  if (f16)
    return launch_pdl(attend_kernel<__half, 4>, grid, dim3(kAttendThreads), 0, st, pl,
                      static_cast<const __half*>(q), static_cast<const __half*>(kv.k_cache),
                      static_cast<const __half*>(kv.v_cache), (long long)kv.stride_page,
                      (long long)kv.stride_token, (long long)kv.stride_head, kv.block_table,
                      sel_idx, sel_count, seq_lens, bg_mass, bg_max, bg_aux, bg_tcount,
                      ix.list_vmeans, ix.list_counts, split_part, tickets,
                      static_cast<__half*>(out), lse, out_f32);
  return launch_pdl(attend_kernel<__nv_bfloat16, 4>, grid, dim3(kAttendThreads), 0, st, pl,
                    static_cast<const __nv_bfloat16*>(q),
                    static_cast<const __nv_bfloat16*>(kv.k_cache),
                    static_cast<const __nv_bfloat16*>(kv.v_cache), (long long)kv.stride_page,
                    (long long)kv.stride_token, (long long)kv.stride_head, kv.block_table, sel_idx,
                    sel_count, seq_lens, bg_mass, bg_max, bg_aux, bg_tcount, ix.list_vmeans,
                    ix.list_counts, split_part, tickets, static_cast<__nv_bfloat16*>(out), lse,
                    out_f32);
}

}  // namespace pqhsa
