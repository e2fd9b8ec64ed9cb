// Host side of the C ABI: argument validation, launch plan, workspace carve-up and the
// entry points declared in pqhsa.h.  Nothing here allocates device memory or synchronises,
// except pqhsa_last_device_status and pqhsa_decode_host, which say so.
#include <mutex>

#include "common.cuh"

namespace pqhsa {

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kMaxSmemPerCta = 227 * 1024 - 1024;   // opt-in limit minus static shared memory
constexpr int kDefaultSms = 148;                        // B200

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

int sm_count() {
  static int cached[64];
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return kDefaultSms; }
  std::lock_guard<std::mutex> lock(mu);
  if (dev < 0 || dev >= 64) return kDefaultSms;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = kDefaultSms;
    }
    cached[dev] = n;
  }
  return cached[dev];
}

int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }

}  // namespace

int make_plan(const pqhsa_params* p, Plan* pl) {
  if (p == nullptr || pl == nullptr) return PQHSA_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->head_dim <= 0 ||
      p->n_list <= 0 || p->pq_m <= 0 || p->pq_dsub <= 0 || p->pq_ncode <= 0 ||
      p->max_seq_len <= 0 || p->page_size <= 0 || p->max_pages_per_seq <= 0 || p->k_max <= 0 ||
      p->n_sink < 0 || p->n_local < 0 || p->exact_set_multiple < 0)
    return PQHSA_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return PQHSA_ERR_INVALID_ARG;
  if (p->pq_m * p->pq_dsub != p->head_dim) return PQHSA_ERR_INVALID_ARG;
  if (p->budget_ppm > 1000000u) return PQHSA_ERR_INVALID_ARG;
  if (p->dtype != PQHSA_F16 && p->dtype != PQHSA_BF16) return PQHSA_ERR_INVALID_ARG;
  if (!(p->sm_scale > 0.f)) return PQHSA_ERR_INVALID_ARG;
  if (p->variant < PQHSA_VARIANT_B || p->variant > PQHSA_VARIANT_C2B) return PQHSA_ERR_INVALID_ARG;
  if (p->table_precision != PQHSA_TABLES_FP32 && p->table_precision != PQHSA_TABLES_FP16 &&
      p->table_precision != PQHSA_TABLES_FP16_RESCORE)
    return PQHSA_ERR_INVALID_ARG;
  if ((long long)p->max_pages_per_seq * p->page_size < p->max_seq_len) return PQHSA_ERR_INVALID_ARG;
  long long k_need = ((long long)p->max_seq_len * p->budget_ppm + 999999LL) / 1000000LL;
  if (p->exact_set_multiple > 1) k_need += p->exact_set_multiple - 1;     // rounding slack
  if (k_need > p->max_seq_len) k_need = p->max_seq_len;
  if (p->k_max < k_need) return PQHSA_ERR_INVALID_ARG;

  if (p->head_dim != kHeadDim) return PQHSA_ERR_UNSUPPORTED;
  if (p->pq_ncode == 256) {
    if (p->pq_m != 8 && p->pq_m != 16 && p->pq_m != 32 && p->pq_m != 64) return PQHSA_ERR_UNSUPPORTED;
  } else if (p->pq_ncode == 16) {      // 4-bit codes, two per byte (the paper's own index setting)
    if (p->pq_m != 8 && p->pq_m != 16) return PQHSA_ERR_UNSUPPORTED;
  } else {
    return PQHSA_ERR_UNSUPPORTED;
  }
  if (p->n_list > 4096 || p->max_seq_len % 4 != 0) return PQHSA_ERR_UNSUPPORTED;
  const int G = p->n_q_heads / p->n_kv_heads;
  if (G > 16) return PQHSA_ERR_UNSUPPORTED;
  // fp16 tables: the layer shape of the benchmark only (32 one-byte subspaces, groups of 4 heads)
  if (p->table_precision != PQHSA_TABLES_FP32 && (p->pq_ncode != 256 || p->pq_m != 32 || G < 3))
    return PQHSA_ERR_UNSUPPORTED;

  Plan& o = *pl;
  o.B = p->batch; o.Hq = p->n_q_heads; o.Hkv = p->n_kv_heads; o.G = G;
  o.Gc = G <= 2 ? G : 4;
  o.n_hg = (G + o.Gc - 1) / o.Gc;
  o.n_list = p->n_list; o.M = p->pq_m; o.dsub = p->pq_dsub;
  o.n_code = p->pq_ncode; o.code_bytes = p->pq_ncode == 16 ? p->pq_m / 2 : p->pq_m;
  o.N_max = p->max_seq_len; o.page_size = p->page_size; o.max_pages = p->max_pages_per_seq;
  o.k_max = p->k_max; o.n_sink = p->n_sink; o.n_local = p->n_local;
  o.exact_multiple = p->exact_set_multiple; o.ppm = p->budget_ppm; o.sm_scale = p->sm_scale; o.dtype = p->dtype;
  o.variant = p->variant; o.indexed_lens = p->indexed_lens; o.status = nullptr;
  o.half_tables = p->table_precision != PQHSA_TABLES_FP32 ? 1 : 0;
  o.rescore = p->table_precision == PQHSA_TABLES_FP16_RESCORE ? 1 : 0;
  o.norm_seg = nullptr;
  o.num_sms = sm_count();
  o.scan_ctas = o.num_sms;                                  // persistent scan CTAs: one per SM
  o.upb = o.Hkv * o.n_hg;
  o.n_part = o.scan_ctas / o.upb + 2;
  if (o.n_part > kMaxSeg) return PQHSA_ERR_UNSUPPORTED;     // more SMs than this build plans for
  o.rows = o.B * o.Hq;
  // the coarse table is bulk-copied: its byte size and unit stride must be multiples of 16.
  // Prefer the coarse table in shared memory (a random 16-byte read per token either way, but
  // without a tag lookup), then a third stage of the code ring.
  const bool co_ok = (o.Gc * o.n_list) % 4 == 0;
  if (o.n_code == 16) {
    // 4-bit scan: the table is tiny, so the coarse table gets a conflict-free 128-byte row per
    // list when that fits, else one entry per list, else it stays in global memory
    o.scan_stages = 0;
    if (scan4_smem_bytes(o, 2) <= kMaxSmemPerCta) o.coarse_in_smem = 2;
    else if (co_ok && scan4_smem_bytes(o, 1) <= kMaxSmemPerCta) o.coarse_in_smem = 1;
    else o.coarse_in_smem = 0;
  } else
  if (co_ok && scan_smem_bytes(o, true, 3) <= kMaxSmemPerCta) { o.coarse_in_smem = 1; o.scan_stages = 3; }
  else if (co_ok && scan_smem_bytes(o, true, 2) <= kMaxSmemPerCta) { o.coarse_in_smem = 1; o.scan_stages = 2; }
  else if (scan_smem_bytes(o, false, 3) <= kMaxSmemPerCta) { o.coarse_in_smem = 0; o.scan_stages = 3; }
  else if (scan_smem_bytes(o, false, 2) <= kMaxSmemPerCta) { o.coarse_in_smem = 0; o.scan_stages = 2; }
  else return PQHSA_ERR_UNSUPPORTED;

  // select CTAs per row, each looping over 8192-score chunks of its row: with few rows
  // exactly one wave of resident CTAs (3 per SM; a straggling second wave would double the
  // kernel), with many rows short CTAs in at least two waves
  const int sel_slots = 3 * o.num_sms;
  o.hist_chunks = 2 * o.rows <= sel_slots ? sel_slots / o.rows : ceil_div(2LL * sel_slots, o.rows);
  if (o.hist_chunks > ceil_div(o.N_max, kSelChunk)) o.hist_chunks = ceil_div(o.N_max, kSelChunk);
  if (o.hist_chunks < 1) o.hist_chunks = 1;
  o.cand_cap = o.N_max / 8 > kSelChunk ? o.N_max / 8 : kSelChunk;
  if (o.cand_cap > o.N_max) o.cand_cap = o.N_max;
  // attend kernel, background CTAs per (sequence, KV head, head group): about two per SM in
  // total, at least 32 lists each
  o.bg_splits = ceil_div(2LL * o.num_sms, (long long)o.B * o.upb);
  if (o.bg_splits > o.n_list / 32) o.bg_splits = o.n_list / 32;
  if (o.bg_splits > 16) o.bg_splits = 16;
  if (o.bg_splits < 1) o.bg_splits = 1;
  // the variants with a global mean value need all lists of a unit in one CTA
  if (o.variant >= PQHSA_VARIANT_C) o.bg_splits = 1;
  // attend kernel, split-K CTAs per row: about 512 selected tokens each, but enough CTAs to
  // fill the GPU when there are few rows (one wave of 4 resident CTAs per SM, background
  // CTAs included), as long as every CTA keeps at least 32 tokens
  const long long n_exact = (long long)o.k_max + (o.n_sink < o.N_max ? o.n_sink : o.N_max) +
                            (o.n_local < o.N_max ? o.n_local : o.N_max);
  o.splits = ceil_div(n_exact, 512);
  int fill = (4 * o.num_sms - o.B * o.upb * o.bg_splits) / o.rows;
  const int max_fill = n_exact / 32 > 0 ? (int)(n_exact / 32) : 1;
  if (fill > max_fill) fill = max_fill;
  if (o.splits < fill) o.splits = fill;
  if (o.splits > 64) o.splits = 64;
  // variant Bx adds one correction partial per exact split; a row's merge takes 128 partials
  if (o.variant == PQHSA_VARIANT_BX && 2 * o.splits + o.bg_splits > 128) o.splits = (128 - o.bg_splits) / 2;
  if (o.splits < 1) o.splits = 1;
  // background preparation: CTAs per row
  o.bg_ctas = ceil_div(2LL * o.num_sms, o.rows);
  if (o.bg_ctas > 8) o.bg_ctas = 8;
  if (o.bg_ctas < ceil_div(o.k_max, 768)) o.bg_ctas = ceil_div(o.k_max, 768);   // 6 tokens per thread
  if (o.bg_ctas < 1) o.bg_ctas = 1;
  return PQHSA_OK;
}

static size_t buffer_elems(const Plan& pl, int which) {
  const size_t units = (size_t)pl.B * pl.Hkv * pl.n_hg;
  switch (which) {
    case PQHSA_BUF_LUT: return units * pl.n_code * pl.M * pl.Gc;
    case PQHSA_BUF_COARSE: return units * pl.n_list * pl.Gc;
    case PQHSA_BUF_SCORES: return (size_t)pl.rows * pl.N_max;
    case PQHSA_BUF_LIST_PARTIALS: return units * pl.n_part * pl.Gc * (pl.n_list + 2);
    case PQHSA_BUF_SEL_IDX: return (size_t)pl.rows * pl.k_max;
    case PQHSA_BUF_SEL_COUNT: return (size_t)pl.rows;
    case PQHSA_BUF_KTH: return (size_t)pl.rows;
    case PQHSA_BUF_BG_MASS: return (size_t)pl.rows * pl.n_list;
    case PQHSA_BUF_BG_MAX: return (size_t)pl.rows;
    case PQHSA_BUF_OUT_F32: return (size_t)pl.rows * kHeadDim;
    default: return 0;
  }
}

// Partials per score row in the attend stage: the exact splits, the background slices and,
// for variant Bx, one correction partial per exact split.
int attend_parts(const Plan& pl) {
  return pl.splits + pl.bg_splits + (pl.variant == PQHSA_VARIANT_BX ? pl.splits : 0);
}

void make_layout(const Plan& pl, WsLayout* L) {
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
  L->zero_begin = o;
  L->status = take(16);
  L->counters = take((size_t)pl.rows * 16);
  L->attend_tickets = take((size_t)pl.rows * 4);
  L->bg_mass = take((size_t)pl.rows * pl.n_list * 4);
  L->bg_aux = take((size_t)pl.rows * 16);
  L->bg_tcount = take(pl.variant == PQHSA_VARIANT_BX ? (size_t)pl.rows * pl.n_list * 4 : 0);
  L->attend_zero_bytes = o - L->attend_tickets;
  L->zero_bytes = o - L->zero_begin;
  L->rowstate = take((size_t)pl.rows * 16);
  L->cand = take((size_t)pl.rows * pl.cand_cap * 8);
  L->bg_max = take((size_t)pl.rows * 4);
  L->split_part = take((size_t)pl.rows * attend_parts(pl) * (4 + kHeadDim) * 4);
  L->norm_seg = take(pl.half_tables ? (size_t)pl.B * pl.upb * pl.n_part * 4 : 0);
  L->stage_end = o;
  L->lut = take(buffer_elems(pl, PQHSA_BUF_LUT) * 4);
  L->coarse = take(buffer_elems(pl, PQHSA_BUF_COARSE) * 4);
  L->scores = take(buffer_elems(pl, PQHSA_BUF_SCORES) * 4);
  L->list_partials = take(buffer_elems(pl, PQHSA_BUF_LIST_PARTIALS) * 4);
  L->sel_idx = take(buffer_elems(pl, PQHSA_BUF_SEL_IDX) * 4);
  L->sel_count = take(buffer_elems(pl, PQHSA_BUF_SEL_COUNT) * 4);
  L->kth = take(buffer_elems(pl, PQHSA_BUF_KTH) * 4);
  L->out_f32 = take(buffer_elems(pl, PQHSA_BUF_OUT_F32) * 4);
  L->total = o;
}

}  // namespace pqhsa

using namespace pqhsa;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_index(const pqhsa_index* ix) {
  if (ix == nullptr || ix->centroids == nullptr || ix->codebooks == nullptr ||
      ix->codes == nullptr || ix->list_ids == nullptr || ix->list_vmeans == nullptr)
    return PQHSA_ERR_INVALID_ARG;
  if (!aligned16(ix->centroids) || !aligned16(ix->codes) || !aligned16(ix->list_vmeans))
    return PQHSA_ERR_INVALID_ARG;
  return PQHSA_OK;
}

int check_variant(const Plan& pl, const pqhsa_index* ix) {
  if (pl.variant >= PQHSA_VARIANT_BX && ix->list_counts == nullptr) return PQHSA_ERR_INVALID_ARG;
  return PQHSA_OK;
}

int check_kv(const pqhsa_paged_kv* kv) {
  if (kv == nullptr || kv->k_cache == nullptr || kv->v_cache == nullptr ||
      kv->block_table == nullptr)
    return PQHSA_ERR_INVALID_ARG;
  if (!aligned16(kv->k_cache) || !aligned16(kv->v_cache)) return PQHSA_ERR_INVALID_ARG;
  if (kv->stride_page < 0 || kv->stride_token < 0 || kv->stride_head < 0)
    return PQHSA_ERR_INVALID_ARG;
  if (kv->stride_page % 8 || kv->stride_token % 8 || kv->stride_head % 8)
    return PQHSA_ERR_UNSUPPORTED;
  return PQHSA_OK;
}

int check_ws(const void* ws, size_t ws_bytes, size_t need) {
  if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PQHSA_ERR_INVALID_ARG;
  return ws_bytes < need ? PQHSA_ERR_WORKSPACE : PQHSA_OK;
}

int cuda_status(cudaError_t e) { return e == cudaSuccess ? PQHSA_OK : PQHSA_ERR_CUDA; }

}  // namespace

extern "C" {

int pqhsa_heads_per_group(const pqhsa_params* params) {
  Plan pl;
  int rc = make_plan(params, &pl);
  return rc != PQHSA_OK ? rc : pl.Gc;
}

int pqhsa_num_partials(const pqhsa_params* params) {
  Plan pl;
  int rc = make_plan(params, &pl);
  return rc != PQHSA_OK ? rc : pl.n_part;
}

size_t pqhsa_buffer_elems(const pqhsa_params* params, int which) {
  Plan pl;
  if (make_plan(params, &pl) != PQHSA_OK) return 0;
  return buffer_elems(pl, which);
}

size_t pqhsa_workspace_bytes(const pqhsa_params* params) {
  Plan pl;
  if (make_plan(params, &pl) != PQHSA_OK) return 0;
  WsLayout L;
  make_layout(pl, &L);
  return L.total;
}

size_t pqhsa_decode_buffer_offset(const pqhsa_params* params, int which) {
  Plan pl;
  if (make_plan(params, &pl) != PQHSA_OK) return (size_t)-1;
  WsLayout L;
  make_layout(pl, &L);
  switch (which) {
    case PQHSA_BUF_LUT: return L.lut;
    case PQHSA_BUF_COARSE: return L.coarse;
    case PQHSA_BUF_SCORES: return L.scores;
    case PQHSA_BUF_LIST_PARTIALS: return L.list_partials;
    case PQHSA_BUF_SEL_IDX: return L.sel_idx;
    case PQHSA_BUF_SEL_COUNT: return L.sel_count;
    case PQHSA_BUF_KTH: return L.kth;
    case PQHSA_BUF_BG_MASS: return L.bg_mass;
    case PQHSA_BUF_BG_MAX: return L.bg_max;
    case PQHSA_BUF_OUT_F32: return L.out_f32;
    default: return (size_t)-1;
  }
}

int pqhsa_decode_launch_count(const pqhsa_params* params) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  // LUT build, scan, select sample, select filter, background preparation, attend (+ the
  // correction pass of variant Bx, + the re-score pass of the fp16 tables)
  return 6 + (pl.variant == PQHSA_VARIANT_BX ? 1 : 0) + (pl.rescore ? 1 : 0);
}

int pqhsa_build_lut(const pqhsa_params* params, const void* q, const pqhsa_index* index,
                    float* lut, float* coarse, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if ((rc = check_index(index)) != PQHSA_OK) return rc;
  if (q == nullptr || lut == nullptr || coarse == nullptr || !aligned16(lut) || !aligned16(coarse))
    return PQHSA_ERR_INVALID_ARG;
  return cuda_status(launch_build_lut(pl, q, *index, lut, coarse, nullptr, 0,
                                      static_cast<cudaStream_t>(stream)));
}

int pqhsa_scan(const pqhsa_params* params, const pqhsa_index* index, const float* lut,
               const float* coarse, const int32_t* seq_lens, float* scores, float* list_partials,
               void* ws, size_t ws_bytes, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if ((rc = check_index(index)) != PQHSA_OK) return rc;
  if (lut == nullptr || coarse == nullptr || seq_lens == nullptr || scores == nullptr ||
      list_partials == nullptr || !aligned16(lut) || !aligned16(coarse) || !aligned16(scores))
    return PQHSA_ERR_INVALID_ARG;
  WsLayout L;
  make_layout(pl, &L);
  if ((rc = check_ws(ws, ws_bytes, L.stage_end)) != PQHSA_OK) return rc;
  char* w = static_cast<char*>(ws);
  if (pl.half_tables) pl.norm_seg = reinterpret_cast<float*>(w + L.norm_seg);
  return cuda_status(launch_scan(pl, *index, lut, coarse, seq_lens, scores, list_partials,
                                 reinterpret_cast<int*>(w + L.status),
                                 static_cast<cudaStream_t>(stream)));
}

int pqhsa_select(const pqhsa_params* params, const float* scores, const int32_t* seq_lens,
                 int32_t* sel_idx, int32_t* sel_count, float* kth_score, void* ws,
                 size_t ws_bytes, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (scores == nullptr || seq_lens == nullptr || sel_idx == nullptr || sel_count == nullptr ||
      kth_score == nullptr || !aligned16(scores))
    return PQHSA_ERR_INVALID_ARG;
  WsLayout L;
  make_layout(pl, &L);
  if ((rc = check_ws(ws, ws_bytes, L.stage_end)) != PQHSA_OK) return rc;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(w + L.zero_begin, 0, L.zero_bytes, st) != cudaSuccess) return PQHSA_ERR_CUDA;
  return cuda_status(launch_select(pl, L, w, scores, seq_lens, sel_idx, sel_count, kth_score, st));
}

int pqhsa_rescore(const pqhsa_params* params, const pqhsa_index* index, const float* lut,
                  const float* coarse, const float* scores, const int32_t* seq_lens,
                  int32_t* sel_idx, const int32_t* sel_count, float* kth_score, void* ws,
                  size_t ws_bytes, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (!pl.rescore) return PQHSA_ERR_INVALID_ARG;
  if ((rc = check_index(index)) != PQHSA_OK) return rc;
  if (lut == nullptr || coarse == nullptr || scores == nullptr || seq_lens == nullptr ||
      sel_idx == nullptr || sel_count == nullptr || kth_score == nullptr)
    return PQHSA_ERR_INVALID_ARG;
  WsLayout L;
  make_layout(pl, &L);
  if ((rc = check_ws(ws, ws_bytes, L.stage_end)) != PQHSA_OK) return rc;
  return cuda_status(launch_rescore(pl, L, static_cast<char*>(ws), *index, lut, coarse, scores,
                                    seq_lens, sel_idx, sel_count, kth_score,
                                    static_cast<cudaStream_t>(stream)));
}

int pqhsa_hybrid_attend(const pqhsa_params* params, const void* q, const pqhsa_paged_kv* kv,
                        const pqhsa_index* index, const float* scores, const float* list_partials,
                        const int32_t* sel_idx, const int32_t* sel_count, const int32_t* seq_lens,
                        void* out, float* lse_or_null, float* out_f32_or_null, void* ws,
                        size_t ws_bytes, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if ((rc = check_index(index)) != PQHSA_OK) return rc;
  if ((rc = check_variant(pl, index)) != PQHSA_OK) return rc;
  if ((rc = check_kv(kv)) != PQHSA_OK) return rc;
  if (q == nullptr || scores == nullptr || list_partials == nullptr || sel_idx == nullptr ||
      sel_count == nullptr || seq_lens == nullptr || out == nullptr)
    return PQHSA_ERR_INVALID_ARG;
  WsLayout L;
  make_layout(pl, &L);
  if ((rc = check_ws(ws, ws_bytes, L.stage_end)) != PQHSA_OK) return rc;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(w + L.attend_tickets, 0, L.attend_zero_bytes, st) != cudaSuccess)
    return PQHSA_ERR_CUDA;
  return cuda_status(launch_attend(pl, L, w, q, *kv, *index, scores, list_partials, sel_idx,
                                   sel_count, seq_lens, out, lse_or_null, out_f32_or_null, st));
}

static int decode_impl(const pqhsa_params* params, const void* q, const pqhsa_index* index,
                       const pqhsa_paged_kv* kv, const int32_t* seq_lens, void* out, void* ws,
                       size_t ws_bytes, void* stream, void* const* ev) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if ((rc = check_index(index)) != PQHSA_OK) return rc;
  if ((rc = check_variant(pl, index)) != PQHSA_OK) return rc;
  if ((rc = check_kv(kv)) != PQHSA_OK) return rc;
  if (q == nullptr || seq_lens == nullptr || out == nullptr) return PQHSA_ERR_INVALID_ARG;
  WsLayout L;
  make_layout(pl, &L);
  if ((rc = check_ws(ws, ws_bytes, L.total)) != PQHSA_OK) return rc;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* lut = reinterpret_cast<float*>(w + L.lut);
  float* coarse = reinterpret_cast<float*>(w + L.coarse);
  float* scores = reinterpret_cast<float*>(w + L.scores);
  float* partials = reinterpret_cast<float*>(w + L.list_partials);
  int32_t* sel_idx = reinterpret_cast<int32_t*>(w + L.sel_idx);
  int32_t* sel_count = reinterpret_cast<int32_t*>(w + L.sel_count);
  float* kth = reinterpret_cast<float*>(w + L.kth);
  auto mark = [&](int i) {
    return ev == nullptr ? cudaSuccess : cudaEventRecord(static_cast<cudaEvent_t>(ev[i]), st);
  };
  cudaError_t e = mark(0);
  // the LUT kernel also clears the status word, histograms, counters and tickets
  if (e == cudaSuccess)
    e = launch_build_lut(pl, q, *index, lut, coarse, w + L.zero_begin, L.zero_bytes, st);
  if (e == cudaSuccess) e = mark(1);
  if (pl.half_tables) pl.norm_seg = reinterpret_cast<float*>(w + L.norm_seg);
  if (e == cudaSuccess)
    e = launch_scan(pl, *index, lut, coarse, seq_lens, scores, partials,
                    reinterpret_cast<int*>(w + L.status), st);
  if (e == cudaSuccess) e = mark(2);
  if (e == cudaSuccess) e = launch_select(pl, L, w, scores, seq_lens, sel_idx, sel_count, kth, st);
  if (e == cudaSuccess && pl.rescore)
    e = launch_rescore(pl, L, w, *index, lut, coarse, scores, seq_lens, sel_idx, sel_count, kth, st);
  if (e == cudaSuccess) e = mark(3);
  if (e == cudaSuccess)
    e = launch_attend(pl, L, w, q, *kv, *index, scores, partials, sel_idx, sel_count, seq_lens,
                      out, nullptr, reinterpret_cast<float*>(w + L.out_f32), st);
  if (e == cudaSuccess) e = mark(4);
  return cuda_status(e);
}

int pqhsa_decode(const pqhsa_params* params, const void* q, const pqhsa_index* index,
                 const pqhsa_paged_kv* kv, const int32_t* seq_lens, void* out, void* ws,
                 size_t ws_bytes, void* stream) {
  return decode_impl(params, q, index, kv, seq_lens, out, ws, ws_bytes, stream, nullptr);
}

int pqhsa_decode_events(const pqhsa_params* params, const void* q, const pqhsa_index* index,
                        const pqhsa_paged_kv* kv, const int32_t* seq_lens, void* out, void* ws,
                        size_t ws_bytes, void* stream, void* const* stage_events) {
  if (stage_events == nullptr) return PQHSA_ERR_INVALID_ARG;
  for (int i = 0; i < PQHSA_N_STAGE_EVENTS; ++i)
    if (stage_events[i] == nullptr) return PQHSA_ERR_INVALID_ARG;
  return decode_impl(params, q, index, kv, seq_lens, out, ws, ws_bytes, stream, stage_events);
}

int pqhsa_decode_host(const pqhsa_params* params, const void* q_host, void* q_dev_staging,
                      const pqhsa_index* index, const pqhsa_paged_kv* kv, const int32_t* seq_lens,
                      void* out_dev_staging, void* out_host, void* ws, size_t ws_bytes,
                      void* stream) {
  if (params == nullptr || q_host == nullptr || q_dev_staging == nullptr ||
      out_dev_staging == nullptr || out_host == nullptr)
    return PQHSA_ERR_INVALID_ARG;
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)pl.rows * kHeadDim * 2;
  if (cudaMemcpyAsync(q_dev_staging, q_host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return PQHSA_ERR_CUDA;
  rc = pqhsa_decode(params, q_dev_staging, index, kv, seq_lens, out_dev_staging, ws, ws_bytes,
                    stream);
  if (rc != PQHSA_OK) return rc;
  if (cudaMemcpyAsync(out_host, out_dev_staging, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return PQHSA_ERR_CUDA;
  return cuda_status(cudaStreamSynchronize(st));
}

int pqhsa_last_device_status(const pqhsa_params* params, void* ws, void* stream) {
  Plan pl;
  int rc = make_plan(params, &pl);
  if (rc != PQHSA_OK) return rc;
  if (ws == nullptr) return PQHSA_ERR_INVALID_ARG;
  WsLayout L;
  make_layout(pl, &L);
  int host = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&host, static_cast<char*>(ws) + L.status, sizeof(int),
                      cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return PQHSA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return PQHSA_ERR_CUDA;
  return host == 0 ? PQHSA_OK : PQHSA_ERR_DEVICE_CHECK;
}

int pqhsa_debug_build(void) {
#ifdef PQHSA_DEBUG
  return 1;
#else
  return 0;
#endif
}

int pqhsa_debug_predicate(int which, long long value, long long lo, long long hi) {
  switch (which) {
    case 0: return list_id_ok(value, hi) ? 1 : 0;
    case 1: return position_ok(value, lo, hi) ? 1 : 0;
    case 2: return page_ok(value) ? 1 : 0;
    default: return -1;
  }
}

const char* pqhsa_status_string(int status) {
  switch (status) {
    case PQHSA_OK: return "ok";
    case PQHSA_ERR_INVALID_ARG: return "invalid argument";
    case PQHSA_ERR_UNSUPPORTED: return "unsupported configuration";
    case PQHSA_ERR_WORKSPACE: return "workspace too small";
    case PQHSA_ERR_CUDA: return "CUDA runtime error";
    case PQHSA_ERR_DEVICE_CHECK: return "device-side consistency check failed";
    default: return "unknown status";
  }
}

}  // extern "C"
