// Shared declarations of the PQ-HSA decode library (host + device).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "pqhsa.h"

namespace pqhsa {

constexpr int kHeadDim = 128;
constexpr int kNCode = 256;
constexpr int kTile = 32;            // tokens per scan tile: one token per lane
constexpr int kScanThreads = 512;
constexpr int kScanMinTiles = kScanThreads / 32;   // a scan CTA gets at least one tile per warp
constexpr int kMaxSeg = 320;                       // scan segments one unit may be cut into (n_part)
constexpr int kHistBins = 4096;      // 12-bit radix digits of the select's shared-memory histograms
constexpr int kSelThreads = 512;
constexpr int kSelChunk = 8192;      // scores per select CTA: 16 per thread, kept in registers
constexpr int kAttendThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegligibleLog2 = -40.0f;   // exp2 arguments below this are left out of a sum

// Host-derived launch plan; passed by value to kernels.
struct Plan {
  int B, Hq, Hkv, G, Gc, n_hg;       // Gc heads per scan pass, n_hg = ceil(G / Gc)
  int n_list, M, dsub;
  int n_code;                        // codewords per subspace: 256 (one byte per code) or 16 (two codes per byte)
  int code_bytes;                    // bytes of codes per token: M or M / 2
  int N_max, page_size, max_pages;
  int k_max;
  int n_sink, n_local;               // |S| and |L| of Sec. 3.2 (upper bounds: clipped per sequence)
  int exact_multiple;                // > 1: |S| + |L| + k is rounded up to this multiple (App. A)
  int variant;                       // pqhsa_variant: how the background term is formed
  int half_tables;                   // scan keeps its lookup tables in fp16 (approximate scores)
  int rescore;                       // ... and the top-k is re-decided from fp32 tables near its threshold
  float* norm_seg;                   // device [units][n_part]: largest key norm per scan segment (fp16 tables), or null
  const int32_t* indexed_lens;       // device [B] or null: positions covered by the index
  int* status;                       // device status word, or null (set by the launchers)
  uint32_t ppm;
  float sm_scale;
  int dtype;
  int scan_ctas;                     // P: persistent scan CTAs (= number of SMs)
  int n_part;                        // list-partial slots per score row
  int upb;                           // scan units per sequence = Hkv * n_hg
  int rows;                          // B * Hq score rows
  int hist_chunks;                   // CTAs per row in the select kernels
  int cand_cap;                      // candidate slots per row
  int splits;                        // exact (split-K) CTAs per row in the attend kernel
  int bg_splits;                     // background CTAs per (sequence, KV head, head group) there
  int bg_ctas;                       // CTAs per row in the background preparation
  int coarse_in_smem;                // scan keeps the coarse table in shared memory (4-bit scan: 2 =
                                     // one conflict-free 128-byte row per list)
  int scan_stages;                   // stages per warp in the scan's code ring (3 or 2)
  int num_sms;
};

// Workspace carve-up (byte offsets from a 256-byte aligned base).
struct WsLayout {
  size_t status;                     // int32[4]: device status word (+ padding)
  size_t zero_begin, zero_bytes;     // region cleared by one memset before select
  size_t counters;                   // uint32 [rows][4]: fallbacks, ticket, n_out, n_cand
  size_t attend_tickets;             // uint32 [rows]
  size_t attend_zero_bytes;          // tickets + bg_mass: what the attend stage needs cleared
  size_t rowstate;                   // int32  [rows][4]: lo, hi (float bits), k, n
  size_t cand;                       // uint2  [rows][cand_cap]: candidates as (score key, position)
  size_t bg_mass;                    // float  [rows][n_list]: M_j relative to bg_max (accumulated)
  size_t bg_aux;                     // float  [rows][4]: [0] sum of the selected tokens' approximate logits
  size_t bg_tcount;                  // int32  [rows][n_list]: selected tokens per list (variant Bx only)
  size_t bg_max;                     // float  [rows]
  size_t split_part;                 // float  [rows][splits + bg_splits][4 + 128]: m, Z, pad, N[128]
  size_t norm_seg;                   // float  [units][n_part]: largest key norm per scan segment (fp16 tables)
  size_t stage_end;                  // end of what a single stage call needs
  // intermediates of the fused entry point
  size_t lut, coarse, scores, list_partials, sel_idx, sel_count, kth, out_f32;
  size_t total;
};

int make_plan(const pqhsa_params* p, Plan* plan);          // returns pqhsa_status
void make_layout(const Plan& plan, WsLayout* L);
int attend_parts(const Plan& plan);                        // partials per score row in the attend stage

// ------------------------------------------------------------------ index checks
// The release build never trusts an index it reads from memory: a list id is clamped to
// [0, n_list), a selected position outside its sequence is skipped.  A build with
// -DPQHSA_DEBUG also RECORDS such an index: the access is still made safe the same way, and a
// bit is or-ed into the status word that pqhsa_last_device_status reads (no trap, no assert:
// the context stays usable).  The predicates are host + device so that they can be unit
// tested without a GPU (pqhsa_debug_predicate).
constexpr int kStatusCountMismatch = 1;    // top-k emitted a number of positions other than k
constexpr int kStatusSeqLen = 2;           // seq_lens[b] outside [0, max_seq_len]
constexpr int kStatusCopyTimeout = 4;      // a bounded wait on a bulk copy ran out
constexpr int kStatusRescoreSkipped = 64;  // fp16 tables: a row's near-threshold pool did not fit; its top-k is the approximate one
constexpr int kStatusListId = 8;           // debug: list id >= n_list
constexpr int kStatusPosition = 16;        // debug: selected position outside the indexed region
constexpr int kStatusPage = 32;            // debug: negative page id in the block table
__host__ __device__ inline bool list_id_ok(long long lid, long long n_list) {
  return lid >= 0 && lid < n_list;
}
__host__ __device__ inline bool position_ok(long long pos, long long lo, long long hi) {
  return pos >= lo && pos < hi;
}
__host__ __device__ inline bool page_ok(long long page) { return page >= 0; }
#ifdef PQHSA_DEBUG
#define PQHSA_DEBUG_CHECK(ok, bit, status_ptr)                                    \
  do {                                                                            \
    if (!(ok) && (status_ptr) != nullptr) atomicOr((status_ptr), (bit));          \
  } while (0)
#else
#define PQHSA_DEBUG_CHECK(ok, bit, status_ptr) \
  do {                                         \
  } while (0)
#endif

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint32_t score_key(float s) {
  // Order-preserving map float -> uint32 (larger score <-> larger key); -0 and +0 coincide.
  const uint32_t u = __float_as_uint(s + 0.0f);
  return u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t k) {
  uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(u);
}

// k_b = ceil(n * ppm / 1e6) in 64-bit integers, clipped to n (Eq. 3).
__device__ __forceinline__ int budget_k(int n, uint32_t ppm) {
  if (n <= 0) return 0;
  long long k = ((long long)n * (long long)ppm + 999999LL) / 1000000LL;
  return (int)(k < (long long)n ? k : (long long)n);
}

__device__ __forceinline__ int clamp_len(int n, int n_max) {
  return n < 0 ? 0 : (n > n_max ? n_max : n);
}

// Position partition of sequence b with n tokens (Sec. 3.2): sink prefix S = [0, r_begin),
// indexed region R = [r_begin, r_end), window L = [r_end, n).  The window holds what the index
// does not cover (Sec. 3.3): with indexed_lens given, everything from indexed_lens[b] on;
// otherwise the last n_local tokens.
struct Region {
  int r_begin, r_end;
};
__device__ __forceinline__ Region region_of(const Plan& pl, int n, int b) {
  Region r;
  r.r_begin = pl.n_sink < n ? pl.n_sink : n;
  int end = n - pl.n_local;
  if (pl.indexed_lens != nullptr) {
    const int covered = __ldg(pl.indexed_lens + b);
    end = covered < n ? covered : n;
  }
  r.r_end = end > r.r_begin ? end : r.r_begin;
  return r;
}
// k of Eq. 3 for sequence b with n tokens: ceil(rho |R|); with exact_multiple > 1 the size of
// the exact set |S| + |L| + k is rounded up to that multiple first (never beyond |R|).
__device__ __forceinline__ int region_budget(const Plan& pl, int n, int b) {
  const Region r = region_of(pl, n, b);
  const int n_r = r.r_end - r.r_begin;
  int k = budget_k(n_r, pl.ppm);
  if (pl.exact_multiple > 1) {
    const long long fixed = n - n_r;
    const long long total = (fixed + k + pl.exact_multiple - 1) / pl.exact_multiple * pl.exact_multiple;
    k = (int)(total - fixed < n_r ? total - fixed : n_r);
  }
  return k;
}

// The scan walks one global sequence of 32-token tiles: sequence-major, then the
// H_kv * n_hg units (KV head, head group) of the sequence, then the tiles of the unit.
// CTA c of P_eff owns tiles [c*T/P_eff, (c+1)*T/P_eff).  Producer (scan) and consumer
// (background preparation) both derive the same split from seq_lens alone.
struct ScanSplit {
  long long T;       // total tiles
  int P_eff;         // CTAs that take part
};
__device__ __forceinline__ int seq_tiles(const int32_t* seq_lens, int b, int n_max) {
  return (clamp_len(seq_lens[b], n_max) + kTile - 1) / kTile;
}
__device__ __forceinline__ ScanSplit scan_split(const int32_t* seq_lens, int B, int n_max,
                                                int upb, int P) {
  long long T = 0;
  for (int b = 0; b < B; ++b) T += (long long)seq_tiles(seq_lens, b, n_max) * upb;
  long long pe = T / kScanMinTiles;
  if (pe < 1) pe = 1;
  if (pe > P) pe = P;
  return ScanSplit{T, (int)pe};
}
__device__ __forceinline__ long long split_start(const ScanSplit& s, int c) {
  return (long long)c * s.T / s.P_eff;
}
__device__ __forceinline__ int split_cta_of(const ScanSplit& s, long long tile) {
  int c = (int)(tile * s.P_eff / s.T);
  if (c + 1 < s.P_eff && split_start(s, c + 1) <= tile) ++c;
  return c;
}

// 2^x by the SFU (ex2.approx): about 2 ulp, flushes results below 2^-126 to zero.
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Programmatic dependent launch: every kernel of the library starts with pdl_wait() (blocks
// until the preceding kernel of the stream has completed and its writes are visible; a no-op
// for a normal launch) followed by pdl_launch_dependents() (lets the next kernel's launch
// overlap this one's execution; it still waits for this grid at its own pdl_wait()).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Last-arrival ticket among the CTAs that share `counter`.  Every thread of the CTA calls it
// after the CTA's global writes; it returns true, to all threads, in the CTA that arrived
// last, which may then read what the others wrote.  One thread fences for the whole CTA
// (fences are cumulative): the first barrier orders the CTA's writes before that thread's
// fence and draw, the second orders its draw and fence before the CTA's reads.  Nobody waits.
__device__ __forceinline__ bool cta_arrived_last(uint32_t* counter, uint32_t n_arrivals,
                                                 int* s_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const bool last = atomicAdd(counter, 1u) == n_arrivals - 1u;
    if (last) __threadfence();
    *s_flag = last ? 1 : 0;
  }
  __syncthreads();
  return *s_flag != 0;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Launch with programmatic stream serialization allowed (see pdl_wait above).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ------------------------------------------------------------------ stage launchers
// Each returns a cudaError_t from the launch (cudaSuccess if nothing had to run).
// zero_ptr / zero_bytes: optional region (16-byte granules) the kernel clears on the side.
cudaError_t launch_build_lut(const Plan& pl, const void* q, const pqhsa_index& ix, float* lut,
                             float* coarse, void* zero_ptr, size_t zero_bytes, cudaStream_t st);
cudaError_t launch_scan(const Plan& pl, const pqhsa_index& ix, const float* lut,
                        const float* coarse, const int32_t* seq_lens, float* scores,
                        float* list_partials, int* status, cudaStream_t st);
// fp16 tables with re-score: re-decides every row's top-k among the tokens whose approximate
// score is within the table-rounding bound of the k-th one, from the fp32 tables.
cudaError_t launch_rescore(const Plan& pl, const WsLayout& L, char* ws, const pqhsa_index& ix,
                           const float* lut, const float* coarse, const float* scores,
                           const int32_t* seq_lens, int32_t* sel_idx, const int32_t* sel_count,
                           float* kth, cudaStream_t st);
cudaError_t launch_select(const Plan& pl, const WsLayout& L, char* ws, const float* scores,
                          const int32_t* seq_lens, int32_t* sel_idx, int32_t* sel_count,
                          float* kth, cudaStream_t st);
cudaError_t launch_attend(const Plan& pl, const WsLayout& L, char* ws, const void* q,
                          const pqhsa_paged_kv& kv, const pqhsa_index& ix, const float* scores,
                          const float* list_partials, const int32_t* sel_idx,
                          const int32_t* sel_count, const int32_t* seq_lens, void* out,
                          float* lse, float* out_f32, cudaStream_t st);
cudaError_t launch_scan4(const Plan& pl, const pqhsa_index& ix, const float* lut,
                         const float* coarse, const int32_t* seq_lens, float* scores,
                         float* list_partials, int* status, cudaStream_t st);
size_t scan_smem_bytes(const Plan& pl, bool coarse_in_smem, int stages);
size_t scan4_smem_bytes(const Plan& pl, int coarse_mode);

}  // namespace pqhsa
