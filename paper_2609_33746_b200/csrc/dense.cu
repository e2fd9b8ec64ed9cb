// Dense decode attention over the whole paged KV cache: the comparator of the context-length
// sweep (Eq. 1 with E = every cached token).  Not part of the PQ-HSA path; it exists so that
// the operator's time can be set against a full-KV read on the same GPU and the same cache.
//
// Split-K flash decoding.  grid (splits, KV heads, sequences); the CTA has one warp per query
// head of the GQA group, and all warps walk the same slice of tokens, so a K/V row comes from
// HBM once and from L1 for the other heads.  Inside a warp: 8 lanes per 256-byte row, 16 rows
// in flight, online softmax in base 2.  The last CTA of a (sequence, KV head) merges the
// partial (m, Z, N) triples of its G rows (atomic ticket; nobody waits).
#include "attn_common.cuh"
#include "common.cuh"

namespace pqhsa {

namespace {

constexpr int kDensePart = kPartStride;
constexpr int kMaxDenseWarps = 16;

template <typename T, int U>
__global__ void __launch_bounds__(32 * kMaxDenseWarps)
dense_decode_kernel(Plan pl, const T* __restrict__ q, const T* __restrict__ kc,
                    const T* __restrict__ vc, long long stride_page, long long stride_token,
                    long long stride_head, const int32_t* __restrict__ block_table,
                    const int32_t* __restrict__ seq_lens, float* __restrict__ part,
                    uint32_t* __restrict__ tickets, T* __restrict__ out) {
  __shared__ int s_last;
  const int split = blockIdx.x, S = gridDim.x, kv = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = b * pl.Hq + kv * pl.G + warp;         // one query head per warp
  pdl_wait();
  pdl_launch_dependents();
  const int n = clamp_len(seq_lens[b], pl.N_max);
  const int tl = (int)((long long)split * n / S), th = (int)((long long)(split + 1) * n / S);
  const int32_t* bt = block_table + (size_t)b * pl.max_pages;

  const int gi = lane >> 3, gl = lane & 7;
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
#pragma unroll
  for (int t = 0; t < 16; ++t) st.acc[t] = 0.f;

  int my_page = (tl + lane < th) ? __ldg(bt + (tl + lane) / pl.page_size) : 0;
  for (int base = tl; base < th; base += 32) {
    const int pos = base + lane;
    long long off = 0;
    if (pos < th)
      off = (long long)my_page * stride_page + (long long)(pos % pl.page_size) * stride_token +
            (long long)kv * stride_head;
    const int nb = min(32, th - base);
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
      if (j0 == 0 && base + 32 + lane < th) my_page = __ldg(bt + (base + 32 + lane) / pl.page_size);
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
        if (ok[u]) {
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
  }
  // merge the 4 lane groups of the warp
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
  float* pr = part + ((size_t)row * S + split) * kDensePart;
  if (gi == 0) {
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      pr[4 + 8 * gl + t] = st.acc[t];
      pr[4 + 64 + 8 * gl + t] = st.acc[8 + t];
    }
    if (gl == 0) { pr[0] = st.m; pr[1] = st.Z; }
  }
  if (!cta_arrived_last(&tickets[b * pl.Hkv + kv], (uint32_t)S, &s_last)) return;
  // last CTA of this (sequence, KV head): each warp merges its row (lane t fetches (m, Z) of
  // partials t, t + 32, ...; then every lane sums its 4 dims over the partials, 8 in flight)
  const float* rp = part + (size_t)row * S * kDensePart;
  float m_r = -CUDART_INF_F;
  for (int s = lane; s < S; s += 32) {
    const float2 mz = __ldcg(reinterpret_cast<const float2*>(rp + (size_t)s * kDensePart));
    if (mz.y > 0.f) m_r = fmaxf(m_r, mz.x);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m_r = fmaxf(m_r, __shfl_xor_sync(0xffffffffu, m_r, o));
  float Z_r = 0.f;
  float4 N_r = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < S; s0 += 8) {
    float2 mz[8];
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      mz[u] = make_float2(0.f, 0.f);
      v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (s0 + u < S) {
        mz[u] = __ldcg(reinterpret_cast<const float2*>(rp + (size_t)(s0 + u) * kDensePart));
        v[u] = __ldcg(reinterpret_cast<const float4*>(rp + (size_t)(s0 + u) * kDensePart + 4) + lane);
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const float a = safe_scale(mz[u].x, m_r, mz[u].y);
      Z_r = fmaf(mz[u].y, a, Z_r);
      N_r.x = fmaf(v[u].x, a, N_r.x); N_r.y = fmaf(v[u].y, a, N_r.y);
      N_r.z = fmaf(v[u].z, a, N_r.z); N_r.w = fmaf(v[u].w, a, N_r.w);
    }
  }
  const float inv = Z_r > 0.f ? 1.f / Z_r : 0.f;
  T* o = out + (size_t)row * kHeadDim + 4 * lane;
  o[0] = Unpack<T>::pack(N_r.x * inv); o[1] = Unpack<T>::pack(N_r.y * inv);
  o[2] = Unpack<T>::pack(N_r.z * inv); o[3] = Unpack<T>::pack(N_r.w * inv);
}

int dense_splits(const Plan& pl) {
  int s = (4 * pl.num_sms) / (pl.B * pl.Hkv);
  const int max_s = pl.N_max / 256 > 0 ? pl.N_max / 256 : 1;
  if (s > max_s) s = max_s;
  if (s > 256) s = 256;
  return s < 1 ? 1 : s;
}

size_t align256d(size_t x) { return (x + 255) / 256 * 256; }

// Read-only probe of the gather that the exact part of the attend step performs: the K and V
// rows of the selected tokens, through the block table and the strides, nothing computed (the
// words are xor-ed into a sink that is never written).  A warp takes 32 selected tokens of a
// row at a time: every lane resolves one token's address (position, page) one round ahead,
// then half-warps fetch the K and the V rows, sixteen tokens in flight.  Its time is what the
// memory system charges for these bytes at these addresses: the ceiling the attend kernel is
// measured against.
constexpr int kProbeRows = 16;      // selected tokens per warp in flight (K and V row each)

__global__ void __launch_bounds__(256)
gather_probe_kernel(Plan pl, const unsigned char* __restrict__ kc, const unsigned char* __restrict__ vc,
                    long long stride_page, long long stride_token, long long stride_head,
                    const int32_t* __restrict__ block_table, const int32_t* __restrict__ sel_idx,
                    const int32_t* __restrict__ sel_count, const int32_t* __restrict__ seq_lens,
                    uint4* __restrict__ sink) {
  const int lane = threadIdx.x & 31, half = lane >> 4, l16 = lane & 15;
  const int warp = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  const int n_warps = (int)((gridDim.x * blockDim.x) >> 5);
  const int cpr = (pl.k_max + 31) / 32;                  // rounds of 32 tokens per row
  const int rounds = pl.rows * cpr;
  const unsigned char* base = half ? vc : kc;            // lanes 0-15: the K row, 16-31: the V row
  uint4 acc = make_uint4(0u, 0u, 0u, 0u);
  // byte offset of the row of this lane's token in round r, -1 if there is none
  auto resolve = [&](int r) -> long long {
    if (r >= rounds) return -1;
    const int row = r / cpr, t = (r - row * cpr) * 32 + lane;
    const int b = row / pl.Hq, kv = (row % pl.Hq) / pl.G;
    const int cnt = min(max(__ldg(sel_count + row), 0), pl.k_max);
    if (t >= cnt) return -1;
    const int pos = __ldg(sel_idx + (size_t)row * pl.k_max + t);
    if ((unsigned)pos >= (unsigned)clamp_len(seq_lens[b], pl.N_max)) return -1;
    const int page = __ldg(block_table + (size_t)b * pl.max_pages + pos / pl.page_size);
    return 2 * ((long long)page * stride_page + (long long)(pos % pl.page_size) * stride_token +
                (long long)kv * stride_head);             // strides are in 2-byte elements
  };
  long long off = resolve(warp);
  for (int r = warp; r < rounds; r += n_warps) {
    const long long nxt = resolve(r + n_warps);
#pragma unroll
    for (int j0 = 0; j0 < 32; j0 += kProbeRows) {
      uint4 v[kProbeRows];
#pragma unroll
      for (int u = 0; u < kProbeRows; ++u) {
        const long long o = __shfl_sync(0xffffffffu, off, j0 + u);
        v[u] = o >= 0 ? __ldg(reinterpret_cast<const uint4*>(base + o) + l16) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < kProbeRows; ++u) { acc.x ^= v[u].x; acc.y ^= v[u].y; acc.z ^= v[u].z; acc.w ^= v[u].w; }
    }
    off = nxt;
  }
  // (the store keeps the loads alive; the pattern does not occur)
  if (acc.x == 0x9e3779b9u && acc.y == 0x7f4a7c15u && acc.z == 0xf39cc060u && acc.w == 0x5cedc834u)
    sink[0] = acc;
}

}  // namespace
}  // namespace pqhsa

using namespace pqhsa;

extern "C" {

size_t pqhsa_dense_workspace_bytes(const pqhsa_params* params) {
  Plan pl;
  if (make_plan(params, &pl) != PQHSA_OK) return 0;
  return align256d((size_t)pl.B * pl.Hkv * 4) +
         align256d((size_t)pl.rows * dense_splits(pl) * kDensePart * 4);
}

int pqhsa_dense_decode(const pqhsa_params* params, const void* q, const pqhsa_paged_kv* kv,
                       const int32_t* seq_lens, void* out, void* ws, size_t ws_bytes, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (q == nullptr || kv == nullptr || kv->k_cache == nullptr || kv->v_cache == nullptr ||
      kv->block_table == nullptr || seq_lens == nullptr || out == nullptr || ws == nullptr ||
      (reinterpret_cast<uintptr_t>(ws) & 255u) != 0)
    return PQHSA_ERR_INVALID_ARG;
  if (kv->stride_page % 8 || kv->stride_token % 8 || kv->stride_head % 8) return PQHSA_ERR_UNSUPPORTED;
  if (pl.G > kMaxDenseWarps) return PQHSA_ERR_UNSUPPORTED;
  if (ws_bytes < pqhsa_dense_workspace_bytes(params)) return PQHSA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  const size_t tick_bytes = align256d((size_t)pl.B * pl.Hkv * 4);
  if (cudaMemsetAsync(w, 0, tick_bytes, st) != cudaSuccess) return PQHSA_ERR_CUDA;
  uint32_t* tickets = reinterpret_cast<uint32_t*>(w);
  float* part = reinterpret_cast<float*>(w + tick_bytes);
  const dim3 grid(dense_splits(pl), pl.Hkv, pl.B), block(32 * pl.G);
  cudaError_t e;
  if (pl.dtype == PQHSA_F16)
    e = launch_pdl(dense_decode_kernel<__half, 4>, grid, block, 0, st, pl,
                   static_cast<const __half*>(q), static_cast<const __half*>(kv->k_cache),
                   static_cast<const __half*>(kv->v_cache), (long long)kv->stride_page,
                   (long long)kv->stride_token, (long long)kv->stride_head, kv->block_table,
                   seq_lens, part, tickets, static_cast<__half*>(out));
  else
    e = launch_pdl(dense_decode_kernel<__nv_bfloat16, 4>, grid, block, 0, st, pl,
                   static_cast<const __nv_bfloat16*>(q),
                   static_cast<const __nv_bfloat16*>(kv->k_cache),
                   static_cast<const __nv_bfloat16*>(kv->v_cache), (long long)kv->stride_page,
                   (long long)kv->stride_token, (long long)kv->stride_head, kv->block_table,
                   seq_lens, part, tickets, static_cast<__nv_bfloat16*>(out));
  return e == cudaSuccess ? PQHSA_OK : PQHSA_ERR_CUDA;
}

int pqhsa_gather_probe(const pqhsa_params* params, const pqhsa_paged_kv* kv, const int32_t* sel_idx,
                       const int32_t* sel_count, const int32_t* seq_lens, void* sink16, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (kv == nullptr || kv->k_cache == nullptr || kv->v_cache == nullptr || kv->block_table == nullptr ||
      sel_idx == nullptr || sel_count == nullptr || seq_lens == nullptr || sink16 == nullptr ||
      (reinterpret_cast<uintptr_t>(sink16) & 15u) != 0)
    return PQHSA_ERR_INVALID_ARG;
  if (kv->stride_page % 8 || kv->stride_token % 8 || kv->stride_head % 8) return PQHSA_ERR_UNSUPPORTED;
  const cudaError_t e = launch_pdl(
      gather_probe_kernel, dim3(8 * pl.num_sms), dim3(256), 0, static_cast<cudaStream_t>(stream), pl,
      static_cast<const unsigned char*>(kv->k_cache), static_cast<const unsigned char*>(kv->v_cache),
      (long long)kv->stride_page, (long long)kv->stride_token, (long long)kv->stride_head,
      kv->block_table, sel_idx, sel_count, seq_lens, static_cast<uint4*>(sink16));
  return e == cudaSuccess ? PQHSA_OK : PQHSA_ERR_CUDA;
}

}  // extern "C"
