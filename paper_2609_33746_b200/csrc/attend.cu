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
#include "attn_common.cuh"
#include "common.cuh"

namespace pqhsa {

namespace {

constexpr int kBgThreads = 256;
constexpr int kPartStride = 2 + kHeadDim;     // m, Z, N[128]
constexpr int kMaxSeg = 160;                  // >= n_part for any plan (148 SMs / 1 unit + 2)

// grid (bg_ctas, rows).  CTA c merges a slice of the lists and subtracts a slice of the
// selected tokens; both go into bg_mass (zeroed by the caller) with float atomics, so the
// CTAs of a row need no ordering.  A list's mass can come out slightly negative when its
// members are all selected (rounding); the consumer clamps at 0.
__global__ void __launch_bounds__(kBgThreads)
bg_prep_kernel(Plan pl, const float* __restrict__ scores, const float* __restrict__ partials,
               const int32_t* __restrict__ sel_idx, const int32_t* __restrict__ sel_count,
               const uint16_t* __restrict__ lids, const int32_t* __restrict__ seq_lens,
               float* __restrict__ bg_mass, float* __restrict__ bg_max) {
  __shared__ float s_scale[kMaxSeg];
  const int row = blockIdx.y, c = blockIdx.x, C = gridDim.x, tid = threadIdx.x;
  const int b = row / pl.Hq, h = row % pl.Hq;
  const int kv = h / pl.G, hg = (h % pl.G) / pl.Gc;
  const int n_list = pl.n_list;
  pdl_wait();
  pdl_launch_dependents();
  const int n = clamp_len(seq_lens[b], pl.N_max);
  float* mass = bg_mass + (size_t)row * n_list;
  if (n == 0) {
    if (c == 0 && tid == 0) bg_max[row] = -CUDART_INF_F;
    return;
  }
  // the selected tokens of this CTA's slice: start their gathers first
  const int cnt = sel_count[row];
  const int tl = (int)((long long)c * cnt / C), th = (int)((long long)(c + 1) * cnt / C);
  const int32_t* sel = sel_idx + (size_t)row * pl.k_max;
  const float* rs = scores + (size_t)row * pl.N_max;
  const uint16_t* rl = lids + ((size_t)b * pl.Hkv + kv) * pl.N_max;
  constexpr int kSelPer = 4;
  int idx[kSelPer];
  float sc[kSelPer];
  uint32_t li[kSelPer];
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) {
    const int t = tl + u * kBgThreads + tid;
    idx[u] = t < th ? sel[t] : -1;
  }
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) {
    sc[u] = idx[u] >= 0 ? rs[idx[u]] : 0.f;
    li[u] = idx[u] >= 0 ? rl[idx[u]] : 0u;
  }

  // which scan segments cover this row's unit
  const ScanSplit sp = scan_split(seq_lens, pl.B, pl.N_max, pl.upb, pl.scan_ctas);
  long long base = 0;
  for (int bb = 0; bb < b; ++bb) base += (long long)seq_tiles(seq_lens, bb, pl.N_max) * pl.upb;
  const int tb = seq_tiles(seq_lens, b, pl.N_max);
  const long long s_u = base + (long long)(kv * pl.n_hg + hg) * tb;
  const int c_first = split_cta_of(sp, s_u);
  const int nseg = min(kMaxSeg, split_cta_of(sp, s_u + tb - 1) - c_first + 1);
  const float* pr = partials + (size_t)row * pl.n_part * (n_list + 1);

  if (tid < nseg) s_scale[tid] = pr[(size_t)tid * (n_list + 1)];     // segment maxima
  __syncthreads();
  float m = -CUDART_INF_F;
  for (int s = 0; s < nseg; ++s) m = fmaxf(m, s_scale[s]);
  const float m2 = m * kLog2e;
  __syncthreads();
  if (tid < nseg) s_scale[tid] = fast_exp2(fmaf(s_scale[tid], kLog2e, -m2));
  __syncthreads();
  const int jl = (int)((long long)c * n_list / C), jh = (int)((long long)(c + 1) * n_list / C);
  for (int j = jl + tid; j < jh; j += kBgThreads) {
    float acc = 0.f;
    for (int s0 = 0; s0 < nseg; s0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        v[u] = (s0 + u < nseg) ? pr[(size_t)(s0 + u) * (n_list + 1) + 1 + j] : 0.f;
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (s0 + u < nseg) acc = fmaf(v[u], s_scale[s0 + u], acc);
    }
    if (acc != 0.f) atomicAdd(&mass[j], acc);
  }
  // take the selected tokens out of their lists' sums
#pragma unroll
  for (int u = 0; u < kSelPer; ++u) {
    if (idx[u] >= 0) {
      const float x = fmaf(sc[u], kLog2e, -m2);
      if (x > kNegligibleLog2) atomicAdd(&mass[li[u]], -fast_exp2(x));
    }
  }
  for (int t = tl + kSelPer * kBgThreads + tid; t < th; t += kBgThreads) {
    const int i = sel[t];
    const float x = fmaf(rs[i], kLog2e, -m2);
    if (x > kNegligibleLog2) atomicAdd(&mass[rl[i]], -fast_exp2(x));
  }
  if (c == 0 && tid == 0) bg_max[row] = m;
}

template <typename T, int U>
__global__ void __launch_bounds__(kAttendThreads, 4)
attend_kernel(Plan pl, const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
              long long stride_page, long long stride_token, long long stride_head,
              const int32_t* __restrict__ block_table, const int32_t* __restrict__ sel_idx,
              const int32_t* __restrict__ sel_count, const float* __restrict__ bg_mass,
              const float* __restrict__ bg_max, const float* __restrict__ vmeans,
              float* __restrict__ split_part, uint32_t* __restrict__ tickets,
              T* __restrict__ out, float* __restrict__ lse) {
  constexpr int kWarps = kAttendThreads / 32;
  __shared__ float s_m[2 * kWarps], s_Z[2 * kWarps];
  __shared__ __align__(16) float s_N[2 * kWarps][kHeadDim];
  __shared__ int s_last;

  const int split = blockIdx.x, S = gridDim.x, row = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = row / pl.Hq, h = row % pl.Hq, kv = h / pl.G;
  const size_t ukv = (size_t)b * pl.Hkv + kv;
  const int n_list = pl.n_list;
  pdl_wait();
  pdl_launch_dependents();
  const int cnt = sel_count[row];

  // ---- this warp's slice of the selected tokens: resolve cache offsets first (two
  //      dependent loads: position, then page id), so they overlap the background part
  const int tl = (int)((long long)split * cnt / S);
  const int th = (int)((long long)(split + 1) * cnt / S);
  const int per_warp = (th - tl + kWarps - 1) / kWarps;
  const int wl = min(th, tl + warp * per_warp), wh = min(th, wl + per_warp);
  const int32_t* sel = sel_idx + (size_t)row * pl.k_max;
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;
  int my_pos = (wl + lane < wh) ? sel[wl + lane] : -1;

  const float m_bg = bg_max[row] * kLog2e;    // reference of the background masses (log2 units)

  // ---- background slice: Z += M_j, N += M_j * vbar_j  (all relative to m_bg)
  {
    const int jl = (int)((long long)split * n_list / S);
    const int jh = (int)((long long)(split + 1) * n_list / S);
    const int per = (jh - jl + kWarps - 1) / kWarps;
    const int a = min(jh, jl + warp * per), e = min(jh, a + per);
    const float* mass = bg_mass + (size_t)row * n_list;
    const float4* vm = reinterpret_cast<const float4*>(vmeans + ukv * n_list * kHeadDim);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float z = 0.f;
    for (int j0 = a; j0 < e; j0 += 32) {
      const float mine = (j0 + lane < e) ? fmaxf(mass[j0 + lane], 0.f) : 0.f;
      unsigned live = __ballot_sync(0xffffffffu, mine > 0.f);
      while (live) {
        int jj[4];
        float mj[4];
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          jj[u] = live ? __ffs(live) - 1 : -1;
          if (live) live &= live - 1;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          mj[u] = __shfl_sync(0xffffffffu, mine, jj[u] < 0 ? 0 : jj[u]);
          v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (jj[u] >= 0) v[u] = __ldg(vm + (size_t)(j0 + jj[u]) * (kHeadDim / 4) + lane);
          else mj[u] = 0.f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          acc.x = fmaf(mj[u], v[u].x, acc.x); acc.y = fmaf(mj[u], v[u].y, acc.y);
          acc.z = fmaf(mj[u], v[u].z, acc.z); acc.w = fmaf(mj[u], v[u].w, acc.w);
          z += mj[u];
        }
      }
    }
    *reinterpret_cast<float4*>(&s_N[kWarps + warp][4 * lane]) = acc;
    if (lane == 0) { s_m[kWarps + warp] = m_bg; s_Z[kWarps + warp] = z; }
  }

  // ---- exact slice
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
  st.m = m_bg;
  st.Z = 0.f;
#pragma unroll
  for (int t = 0; t < 16; ++t) st.acc[t] = 0.f;

  // page id of this lane's first token (second dependent load); later batches prefetch
  // position and page one batch ahead, while the current batch's rows are in flight
  int my_page = my_pos >= 0 ? __ldg(bt + my_pos / pl.page_size) : 0;
  for (int base = wl; base < wh; base += 32) {
    long long off = 0;
    if (my_pos >= 0)
      off = (long long)my_page * stride_page + (long long)(my_pos % pl.page_size) * stride_token +
            (long long)kv * stride_head;
    const int nxt_pos = (base + 32 + lane < wh) ? sel[base + 32 + lane] : -1;
    int nxt_page = 0;
    const int nb = min(32, wh - base);
    for (int j0 = 0; j0 < nb; j0 += 4 * U) {
      uint4 kr[U][2], vr[U][2];
      bool ok[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int tok = j0 + 4 * u + gi;
        const long long o = __shfl_sync(0xffffffffu, off, tok & 31);
        ok[u] = tok < nb;
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
          if (s > st.m) {
            const float a = fast_exp2(st.m - s);
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
  if (gi == 0) {
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      s_N[warp][8 * gl + t] = st.acc[t];
      s_N[warp][64 + 8 * gl + t] = st.acc[8 + t];
    }
    if (gl == 0) { s_m[warp] = st.m; s_Z[warp] = st.Z; }
  }
  __syncthreads();

  // ---- CTA partial: thread d owns output dim d
  float m_c = -CUDART_INF_F;
#pragma unroll
  for (int w = 0; w < 2 * kWarps; ++w) if (s_Z[w] > 0.f) m_c = fmaxf(m_c, s_m[w]);
  float Z_c = 0.f, N_c = 0.f;
#pragma unroll
  for (int w = 0; w < 2 * kWarps; ++w) {
    const float a = safe_scale(s_m[w], m_c, s_Z[w]);
    Z_c = fmaf(s_Z[w], a, Z_c);
    N_c = fmaf(s_N[w][tid], a, N_c);
  }
  float* part = split_part + ((size_t)row * S + split) * kPartStride;
  part[2 + tid] = N_c;
  if (tid == 0) { part[0] = m_c; part[1] = Z_c; }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&tickets[row], 1u) == (uint32_t)(S - 1));
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- last CTA of the row: merge the S partials and normalise (Eq. 5)
  const float* pr = split_part + (size_t)row * S * kPartStride;
  float m_r = -CUDART_INF_F;
  for (int s = 0; s < S; ++s)
    if (__ldcg(pr + s * kPartStride + 1) > 0.f) m_r = fmaxf(m_r, __ldcg(pr + s * kPartStride));
  float Z_r = 0.f, N_r = 0.f;
  for (int s0 = 0; s0 < S; s0 += 4) {
    float Zs[4], ms[4], Ns[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = s0 + u;
      Zs[u] = s < S ? __ldcg(pr + s * kPartStride + 1) : 0.f;
      ms[u] = s < S ? __ldcg(pr + s * kPartStride) : 0.f;
      Ns[u] = s < S ? __ldcg(pr + s * kPartStride + 2 + tid) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float a = safe_scale(ms[u], m_r, Zs[u]);
      Z_r = fmaf(Zs[u], a, Z_r);
      N_r = fmaf(Ns[u], a, N_r);
    }
  }
  out[(size_t)row * kHeadDim + tid] = Unpack<T>::pack(Z_r > 0.f ? N_r / Z_r : 0.f);
  if (lse != nullptr && tid == 0)
    lse[row] = Z_r > 0.f ? (m_r + log2f(Z_r)) / kLog2e : -CUDART_INF_F;
}

}  // namespace

cudaError_t launch_attend(const Plan& pl, const WsLayout& L, char* ws, const void* q,
                          const pqhsa_paged_kv& kv, const pqhsa_index& ix, const float* scores,
                          const float* list_partials, const int32_t* sel_idx,
                          const int32_t* sel_count, const int32_t* seq_lens, void* out,
                          float* lse, cudaStream_t st) {
  float* bg_mass = reinterpret_cast<float*>(ws + L.bg_mass);
  float* bg_max = reinterpret_cast<float*>(ws + L.bg_max);
  float* split_part = reinterpret_cast<float*>(ws + L.split_part);
  uint32_t* tickets = reinterpret_cast<uint32_t*>(ws + L.attend_tickets);
  cudaError_t e = launch_pdl(bg_prep_kernel, dim3(pl.bg_ctas, pl.rows), dim3(kBgThreads), 0, st, pl,
                             scores, list_partials, sel_idx, sel_count, ix.list_ids, seq_lens,
                             bg_mass, bg_max);
  if (e != cudaSuccess) return e;
  dim3 grid(pl.splits, pl.rows);
  if (pl.dtype == PQHSA_F16)
    return launch_pdl(attend_kernel<__half, 4>, grid, dim3(kAttendThreads), 0, st, pl,
                      static_cast<const __half*>(q), static_cast<const __half*>(kv.k_cache),
                      static_cast<const __half*>(kv.v_cache), (long long)kv.stride_page,
                      (long long)kv.stride_token, (long long)kv.stride_head, kv.block_table,
                      sel_idx, sel_count, bg_mass, bg_max, ix.list_vmeans, split_part, tickets,
                      static_cast<__half*>(out), lse);
  return launch_pdl(attend_kernel<__nv_bfloat16, 4>, grid, dim3(kAttendThreads), 0, st, pl,
                    static_cast<const __nv_bfloat16*>(q),
                    static_cast<const __nv_bfloat16*>(kv.k_cache),
                    static_cast<const __nv_bfloat16*>(kv.v_cache), (long long)kv.stride_page,
                    (long long)kv.stride_token, (long long)kv.stride_head, kv.block_table, sel_idx,
                    sel_count, bg_mass, bg_max, ix.list_vmeans, split_part, tickets,
                    static_cast<__nv_bfloat16*>(out), lse);
}

}  // namespace pqhsa
