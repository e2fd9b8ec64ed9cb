/*
 * pqhsa.h -- C ABI of the PQ-HSA decode-step attention operator for NVIDIA B200 (sm_100a).
 *
 * The operator (paper Section 3, Eq. 2-5), per sequence b and query head h whose KV head is
 * g = h / G (G = n_q_heads / n_kv_heads):
 *
 *   1. LUT build   coarse[j] = q.c_j and LUT[m][z] = q^(m).p_{m,z}                    (Sec. 3.1)
 *   2. ADC scan    l~_i = r_i/sqrt(d) * (coarse[a_i] + sum_m LUT[m][z_im]) for every
 *                  indexed token i, one score row per query head from one pass over the
 *                  codes of the KV head, plus per-list sums of exp(l~_i - ref)        (Eq. 2, Sec. 3.3)
 *   3. top-k       T = the k = ceil(rho |R|) tokens with the largest l~_i             (Eq. 3)
 *   4. hybrid attention: exact logits from the original K rows of T, the approximate
 *                  logits of all other tokens summed per inverted list and multiplied
 *                  by the list's stored mean value, one softmax normaliser            (Eq. 4-5)
 *
 * (q = r_q u_q, so r_q * (u_q.x) = q.x: the library works with q directly; this is Eq. 2
 *  with the factor r_q multiplied in.)
 *
 * Conventions for every entry point
 *   - `params` is a HOST pointer.  Every other pointer is a DEVICE pointer owned by the
 *     caller unless a comment says "host".  The library never allocates, frees or
 *     synchronises (pqhsa_last_device_status and pqhsa_decode_host excepted), so calls may
 *     be captured in a CUDA graph.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Arguments are validated on the host first; on error nothing is launched and a
 *     negative pqhsa_status is returned.  PQHSA_OK (0) means "launched", not "finished".
 *   - Input arrays are read-only.  Rows past seq_lens[b] are never read.
 *   - v1 limits: head_dim == 128; pq_ncode == 256 (one byte per code, pq_m in {8,16,32,64}) or
 *     pq_ncode == 16 (two 4-bit codes per byte, pq_m in {8,16}: the paper's own index setting) with
 *     pq_m * pq_dsub == 128; n_list <= 4096 (and the per-CTA tables must fit shared memory,
 *     see PQHSA_ERR_UNSUPPORTED); max_seq_len % 4 == 0; page rows 16-byte aligned
 *     (strides multiples of 8 elements).
 */
#ifndef PQHSA_H_
#define PQHSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PQHSA_OK = 0,
  PQHSA_ERR_INVALID_ARG = -1,   /* null pointer, non-positive size, inconsistent shape      */
  PQHSA_ERR_UNSUPPORTED = -2,   /* valid request outside the v1 limits above                */
  PQHSA_ERR_WORKSPACE = -3,     /* ws_bytes smaller than pqhsa_workspace_bytes()            */
  PQHSA_ERR_CUDA = -4,          /* a CUDA runtime call (launch, memset, copy) failed        */
  PQHSA_ERR_DEVICE_CHECK = -5   /* a kernel recorded an inconsistency in the status word    */
} pqhsa_status;

typedef enum { PQHSA_F16 = 0, PQHSA_BF16 = 1 } pqhsa_dtype;

/* Shape of one decode step (host struct).  Notation follows the paper. */
typedef struct {
  int32_t batch;              /* B   sequences                                              */
  int32_t n_q_heads;          /* H_q query heads                                            */
  int32_t n_kv_heads;         /* H_kv KV heads; G = H_q / H_kv                              */
  int32_t head_dim;           /* d  (128)                                                   */
  int32_t n_list;             /* inverted lists per (sequence, KV head)                     */
  int32_t pq_m;               /* M  PQ subspaces                                            */
  int32_t pq_dsub;            /* dims per subspace, M * dsub == d                           */
  int32_t pq_ncode;           /* 2^b codewords per subspace: 256 or 16                       */
  int32_t max_seq_len;        /* N_max: row stride of codes / list_ids / key_norms / scores */
  int32_t page_size;          /* tokens per KV page                                         */
  int32_t max_pages_per_seq;  /* row stride of block_table                                  */
  int32_t n_sink;             /* sink prefix: S_b = first min(n_sink, N_b) tokens (Sec. 3.2) */
  int32_t n_local;            /* local window: L_b = last min(n_local, N_b - |S_b|) tokens   */
                              /* (see indexed_lens for a per-sequence window);               */
                              /* R_b = the tokens between; S_b and L_b are attended exactly  */
                              /* and take no part in the top-k or the background             */
  uint32_t budget_ppm;        /* rho in parts per million; k_b = ceil(|R_b| * ppm / 1e6),   */
                              /* computed in 64-bit integers on the device from seq_lens    */
  int32_t k_max;              /* row stride of sel_idx; >= ceil(max_seq_len * ppm / 1e6)    */
  float sm_scale;             /* 1/sqrt(d) (Eq. 1)                                          */
  int32_t dtype;              /* pqhsa_dtype of q, K, V and out                             */
  int32_t exact_set_multiple; /* 0 or 1: off.  m > 1: |S_b| + |L_b| + k_b is rounded up to a  */
                              /* multiple of m (App. A, budgets in whole pages), k_b <= |R_b|; */
                              /* k_max must then cover the extra m - 1                        */
  int32_t variant;            /* pqhsa_variant: how the background term is formed (Table 2);  */
                              /* 0 = PQ-HSA itself                                            */
  int32_t table_precision;    /* pqhsa_table_precision: 0 = fp32 lookup tables (the mode every  */
                              /* stated tolerance refers to), 1 = fp16 tables in the scan, 2 =   */
                              /* fp16 tables and an fp32 re-score of the top-k's threshold zone  */
  const int32_t* indexed_lens;/* DEVICE pointer [B] or NULL.  Number of leading positions of  */
                              /* each sequence that the index covers: R_b = [|S_b|,           */
                              /* indexed_lens[b]) and L_b = everything after (Sec. 3.3: a new */
                              /* token is attended exactly until the next index update        */
                              /* encodes it).  NULL: L_b is the last n_local tokens.  Values  */
                              /* are clipped to [|S_b|, seq_lens[b]]; n_local is then unused  */
} pqhsa_params;

/* Precision of the scan's lookup tables.  PQHSA_TABLES_FP16 is an opt-in fast mode (in the spirit of
 * Sec. 1 / Sec. 6: the scan is an IVF-PQ scan and takes that literature's reduced-precision tables):
 * the table build is unchanged, the scan holds the tables as fp16 and sums four entries in fp16
 * before it widens them, so an approximate logit carries an error of about 1e-3 of the table
 * entries' magnitude instead of fp32 rounding.  Everything downstream is unchanged: the top-k is
 * exact on those scores, the selected tokens are attended with exact logits, and the list sums use
 * the same approximate logits that are later taken out of them.  v1: pq_ncode == 256, pq_m == 32,
 * G >= 3 (groups of four heads).
 * PQHSA_TABLES_FP16_RESCORE adds the usual second stage of such scans: the tokens whose approximate
 * score lies within the table-rounding bound of the k-th one are scored again from the fp32 tables and
 * the top-k is re-decided among them (pqhsa_rescore), so that the selected set is the one the fp32
 * tables give (equal fp32 scores: lower position first) and kth_score is the exact k-th fp32 score.
 * The score rows and the list sums keep the fp16-table values. */
typedef enum {
  PQHSA_TABLES_FP32 = 0, PQHSA_TABLES_FP16 = 1, PQHSA_TABLES_FP16_RESCORE = 2
} pqhsa_table_precision;

/* Mechanism variants of the paper's ablation (Table 2; App. B, "Variant definitions").  All of
 * them keep the selector, the budget and the exact part; they differ in the background term.
 * Every variant but B and T needs pqhsa_index.list_counts. */
typedef enum {
  PQHSA_VARIANT_B = 0,    /* PQ-HSA: logit l~_i, value vbar_j (Eq. 4)                            */
  PQHSA_VARIANT_T = 1,    /* no background term                                                  */
  PQHSA_VARIANT_BX = 2,   /* B with vbar_j replaced by the mean over the list's unselected       */
                          /* members, (|R_j| vbar_j - sum_{T n R_j} v_i) / |B n R_j|             */
  PQHSA_VARIANT_C = 3,    /* logit l~_i, value = token-count-weighted global mean of the vbar_j  */
  PQHSA_VARIANT_C2 = 4,   /* one shared logit mean_{i in T} l~_i, global mean value              */
  PQHSA_VARIANT_C2B = 5   /* one shared logit min_{i in T} l_i (exact logits), global mean value */
} pqhsa_variant;

/* IVF-PQ index, one per (sequence, KV head) (Sec. 3.1).  Device pointers, read-only. */
typedef struct {
  const float* centroids;     /* [B][H_kv][n_list][d]      c_j                              */
  const float* codebooks;     /* [B][H_kv][M][256][dsub]   p_{m,z}; subspace m = dims       */
                              /*                           [m*dsub, (m+1)*dsub)             */
  const uint8_t* codes;       /* [B][H_kv][N_max][M]       z_im; with pq_ncode == 16         */
                              /* [B][H_kv][N_max][M/2]: byte j = z_{i,2j} | z_{i,2j+1} << 4   */
  const uint16_t* list_ids;   /* [B][H_kv][N_max]          a_i < n_list                     */
  const float* key_norms;     /* [B][H_kv][N_max]          r_i, or NULL for all ones        */
  const float* list_vmeans;   /* [B][H_kv][n_list][d]      stored mean value of ALL members */
                              /*                           of each list (Eq. 4); 0 if empty */
  const int32_t* list_counts; /* [B][H_kv][n_list]         |R_j|, members behind each stored */
                              /*                           mean; NULL unless a variant needs */
                              /*                           it (pqhsa_variant)                */
} pqhsa_index;

/* The same arrays as pqhsa_index, writable, plus the member count of every list: what
 * pqhsa_index_update maintains.  Centroids and codebooks stay fixed (no re-clustering). */
typedef struct {
  const float* centroids;     /* [B][H_kv][n_list][d]                                        */
  const float* codebooks;     /* [B][H_kv][M][256][dsub]                                     */
  uint8_t* codes;             /* [B][H_kv][N_max][M]                                         */
  uint16_t* list_ids;         /* [B][H_kv][N_max]                                            */
  float* key_norms;           /* [B][H_kv][N_max]     (required here)                        */
  float* list_vmeans;         /* [B][H_kv][n_list][d]                                        */
  int32_t* list_counts;       /* [B][H_kv][n_list]    members behind each stored mean        */
} pqhsa_index_rw;

/* Engine-owned paged KV cache, read in place through element strides (Sec. 3.3, App. E):
 * row of (page p, slot t, KV head g) starts at  base + p*stride_page + t*stride_token +
 * g*stride_head  elements and holds d contiguous elements.  Covers both a split layout
 * ([page][slot][head][d], K and V separate) and an interleaved one ([page][head][slot][2d],
 * v_cache = k_cache + d). */
typedef struct {
  const void* k_cache;
  const void* v_cache;
  int64_t stride_page, stride_token, stride_head;
  const int32_t* block_table; /* [B][max_pages_per_seq]: page id of the i-th page of b      */
} pqhsa_paged_kv;

/* Which intermediate buffer pqhsa_buffer_elems() sizes. */
typedef enum {
  PQHSA_BUF_LUT = 0,            /* float   [B][H_kv][n_hg][256][M][Gc]                        */
  PQHSA_BUF_COARSE = 1,         /* float   [B][H_kv][n_hg][n_list][Gc]                        */
  PQHSA_BUF_SCORES = 2,         /* float   [B][H_q][N_max]                                    */
  PQHSA_BUF_LIST_PARTIALS = 3,  /* float   [B][H_kv][n_hg][n_part][Gc * (2 + n_list)]         */
  PQHSA_BUF_SEL_IDX = 4,        /* int32   [B][H_q][k_max]                                    */
  PQHSA_BUF_SEL_COUNT = 5,      /* int32   [B][H_q]                                           */
  PQHSA_BUF_KTH = 6,            /* float   [B][H_q]                                           */
  /* scratch of the hybrid attention, for inspection through pqhsa_decode_buffer_offset (the   */
  /* offsets also hold for the `ws` of a pqhsa_hybrid_attend call):                             */
  PQHSA_BUF_BG_MASS = 7,        /* float   [B][H_q][n_list]  background mass M_j of Eq. 4,      */
                                /*         relative to exp(BG_MAX); may be slightly negative    */
                                /*         where every member of a list was selected (read as 0) */
  PQHSA_BUF_BG_MAX = 8,         /* float   [B][H_q]  max approximate logit of the row (-inf:    */
                                /*         no background)                                       */
  PQHSA_BUF_OUT_F32 = 9         /* float   [B][H_q][128]  what pqhsa_decode computed before it   */
                                /*         rounded it to the output dtype (fused call only)     */
} pqhsa_buffer;

/* Query heads of a group are processed Gc at a time (Gc = G for G <= 2, else 4); a group
 * has n_hg = ceil(G / Gc) such head groups.  In LUT / COARSE the last index is the head
 * within its head group; slots past G are zero. */
int pqhsa_heads_per_group(const pqhsa_params* params);        /* Gc, or <0 on error          */
int pqhsa_num_partials(const pqhsa_params* params);           /* n_part, or <0 on error      */
/* Number of ELEMENTS of an intermediate buffer (0 on error). Host-only arithmetic. */
size_t pqhsa_buffer_elems(const pqhsa_params* params, int which);
/* Bytes of scratch that any single entry point below needs (pqhsa_decode needs the most:
 * it also carves every intermediate buffer from it).  256-byte aligned base required. */
size_t pqhsa_workspace_bytes(const pqhsa_params* params);

/* Step 1 (Sec. 3.1, text after Eq. 2).  q [B][H_q][d] in params->dtype.
 * Writes lut[..][z][m][g] = sm_scale * q_h^(m).p_{m,z} and
 * coarse[..][j][g] = sm_scale * q_h.c_j with h = kv*G + hg*Gc + g. */
int pqhsa_build_lut(const pqhsa_params* params, const void* q, const pqhsa_index* index,
                    float* lut, float* coarse, void* stream);

/* Step 2 (Eq. 2 and the fused per-list reduction of Sec. 3.3).  seq_lens [B] int32.
 * Writes scores[b][h][i] = l~_i for the tokens i of the indexed region R_b and -inf for the
 * sink and window tokens (i < seq_lens[b]; they never compete in the top-k), and the list
 * partials: every (sequence, KV head, head group) is scanned in segments (contiguous token
 * ranges, one per CTA; at most n_part, the count is a function of seq_lens only), and segment s
 * leaves list_partials[b][kv][hg][s] = { ref[Gc], max[Gc], sum[n_list][Gc] } with, for head g of
 * the group, max[g] = max l~_i over the segment's tokens of R_b (-inf if it has none), ref[g] =
 * the reference of the sums (any value the segment chose; -inf if it has no token of R_b) and
 * sum[j][g] = sum over the segment's members of list j inside R_b of exp(l~_i - ref[g]). */
int pqhsa_scan(const pqhsa_params* params, const pqhsa_index* index, const float* lut,
               const float* coarse, const int32_t* seq_lens, float* scores,
               float* list_partials, void* ws, size_t ws_bytes, void* stream);

/* Step 3 (Eq. 3).  Exact top-k of every score row: sel_idx[b][h][0..k_b) = positions of the
 * k_b largest scores among positions [0, seq_lens[b]) (order unspecified; equal scores:
 * lower position first), sel_count[b][h] = k_b, kth_score[b][h] = the k_b-th largest score
 * (NaN if k_b == 0).  k_b comes from |R_b| (see pqhsa_params); positions outside R_b are
 * expected to hold -inf, as pqhsa_scan writes them, so that they rank last. */
int pqhsa_select(const pqhsa_params* params, const float* scores, const int32_t* seq_lens,
                 int32_t* sel_idx, int32_t* sel_count, float* kth_score,
                 void* ws, size_t ws_bytes, void* stream);

/* Step 3b, table_precision == PQHSA_TABLES_FP16_RESCORE only (PQHSA_ERR_INVALID_ARG otherwise): the
 * fp32 re-score of the threshold zone.  Call after pqhsa_select with the SAME `ws` that pqhsa_scan and
 * pqhsa_select were given (it holds the segment norms of the scan and the candidate lists of the
 * top-k) and with their lut / coarse / scores / sel_idx / sel_count / kth_score.  Replaces in sel_idx
 * the positions that the fp32 tables rank out of the top-k by those they rank in, and sets kth_score
 * to the k-th largest fp32-table score.  A row whose threshold zone holds more than 1024 tokens keeps
 * its approximate top-k and sets bit 64 of the device status word.  One launch on `stream`. */
int pqhsa_rescore(const pqhsa_params* params, const pqhsa_index* index, const float* lut,
                  const float* coarse, const float* scores, const int32_t* seq_lens,
                  int32_t* sel_idx, const int32_t* sel_count, float* kth_score, void* ws,
                  size_t ws_bytes, void* stream);

/* Step 4 (Eq. 4-5).  Gathers the K/V rows of the exact set E_b = S_b u L_b u T (sinks, window,
 * selected tokens) from the paged cache and attends them with exact logits, takes the
 * selected tokens' approximate mass out of their lists' sums, folds in the n_list
 * mean-value terms and normalises once.
 * out [B][H_q][d] in params->dtype; lse_or_null [B][H_q] = log of the normaliser;
 * out_f32_or_null [B][H_q][d] = the same output before it is rounded to params->dtype. */
int pqhsa_hybrid_attend(const pqhsa_params* params, const void* q, const pqhsa_paged_kv* kv,
                        const pqhsa_index* index, const float* scores,
                        const float* list_partials, const int32_t* sel_idx,
                        const int32_t* sel_count, const int32_t* seq_lens, void* out,
                        float* lse_or_null, float* out_f32_or_null, void* ws, size_t ws_bytes,
                        void* stream);

/* pqhsa_select without a workspace argument.  (No counterpart in the paper: this entry point
 * exists for integration, not for the method.)
 *
 * For callers that cannot allocate device memory where they need the top-k: code running
 * inside an engine's pre-planned memory pool, plugins that receive tensors but no allocator,
 * and paths where a driver allocation -- which may stall the whole device -- is not
 * acceptable.  The scratch that pqhsa_select takes from `ws` (counters and
 * candidate lists) lives instead in one fixed 16 MiB array inside the library image; every
 * GPU that loads the library holds that array until the process exits.
 *
 *   - Same inputs, outputs and results as pqhsa_select.  Neither this call nor anything it
 *     uses calls cudaMalloc, cudaFree or any allocating routine.
 *   - Shapes whose scratch exceeds the array (pqhsa_select_static_bytes(params) >
 *     pqhsa_select_static_capacity()) are rejected with PQHSA_ERR_WORKSPACE before anything
 *     is launched; use pqhsa_select with your own workspace for those.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current).  Make that first call outside any
 *     stream capture.  The address is kept per device for the life of the process: after a
 *     cudaDeviceReset the library has to be loaded again before this entry point is used.
 *   - All calls on a device share the one array and it keeps the last call's contents; each
 *     call clears the part that must start at zero on `stream` first.  Two calls that can
 *     overlap on the GPU (different streams, no dependency) race on it: serialise them.
 *   - pqhsa_last_device_status does not apply; a count mismatch is not reported here. */
size_t pqhsa_select_static_capacity(void);
size_t pqhsa_select_static_bytes(const pqhsa_params* params);   /* 0 on invalid params */
int pqhsa_select_static(const pqhsa_params* params, const float* scores, const int32_t* seq_lens,
                        int32_t* sel_idx, int32_t* sel_count, float* kth_score, void* stream);

/* Steps 1-4 back to back on one stream (Sec. 3.3: the decode step of one layer); all
 * intermediates live in `ws`. */
int pqhsa_decode(const pqhsa_params* params, const void* q, const pqhsa_index* index,
                 const pqhsa_paged_kv* kv, const int32_t* seq_lens, void* out,
                 void* ws, size_t ws_bytes, void* stream);

/* pqhsa_decode that also records five caller-created CUDA events (cudaEvent_t passed as
 * void*, in a HOST array) on `stream`: [0] before the first launch, [1] before the scan,
 * [2] before the top-k, [3] before the hybrid attention, [4] after the last kernel.  For
 * per-stage timing; the kernels and their launch configuration are those of pqhsa_decode. */
#define PQHSA_N_STAGE_EVENTS 5
int pqhsa_decode_events(const pqhsa_params* params, const void* q, const pqhsa_index* index,
                        const pqhsa_paged_kv* kv, const int32_t* seq_lens, void* out,
                        void* ws, size_t ws_bytes, void* stream, void* const* stage_events);

/* Index maintenance between decode steps (Sec. 3.3, first paragraph; encoding of Sec. 3.1).
 * For every sequence b the n_new[b] (<= max_new <= 1024) tokens at positions first_pos[b],
 * first_pos[b] + 1, ... are read from the paged cache and encoded into the EXISTING lists:
 * r_i = |k_i| in fp32, u_i = k_i / r_i (0 for a zero key), a_i = list of the nearest centroid
 * to u_i (squared Euclidean distance, lower index on ties), z_im = nearest codeword to the
 * m-th sub-vector of u_i - c_{a_i}; codes, list_ids and key_norms are written at those
 * positions, and every list that received tokens gets vbar_j = (n_j vbar_j + sum of the new
 * members' values) / (n_j + new_j), n_j += new_j.  first_pos / n_new: device int32 [B];
 * positions outside [0, max_seq_len) are skipped.  Two launches on `stream`, no workspace, no
 * synchronisation; must not overlap a decode call that reads the same index. */
int pqhsa_index_update(const pqhsa_params* params, const pqhsa_index_rw* index,
                       const pqhsa_paged_kv* kv, const int32_t* first_pos, const int32_t* n_new,
                       int32_t max_new, void* stream);

/* Batched index build (Sec. 3.3, first paragraph; App. C, "Index build"): trains the IVF-PQ
 * index of EVERY (sequence, KV head) in one call, one launch per step for all of them, from the
 * keys and values in the paged cache.  Per unit: r_i = |k_i| (fp32), u_i = k_i / r_i (0 for a
 * zero key); `coarse_iters` Lloyd iterations on the directions from the centroids seeded with the
 * tokens at seed_lists[b][kv][j] (squared Euclidean distance, lower index on ties, centroid =
 * arithmetic mean of its members, an empty list is re-seeded with the farthest point; a negative
 * seed position gives a zero row), then the final assignment a_i; `pq_iters` Lloyd iterations per
 * subspace on the residuals u_i - c_{a_i} from the codewords seeded with the residuals of the
 * tokens at seed_codes[b][kv][z], then the final codes; the list value means over the members
 * inside R_b and the member counts.  The two seed arrays are the method's random draws: device
 * int32 [B][H_kv][n_list] and [B][H_kv][pq_ncode].  All arrays of `index` are outputs.
 * ws: pqhsa_index_build_workspace_bytes(params) bytes (it holds the fp32 directions: 512 bytes
 * per token and KV head), 256-byte aligned.  Launches only; no synchronisation. */
typedef struct {
  float* centroids;           /* [B][H_kv][n_list][d]                                        */
  float* codebooks;           /* [B][H_kv][M][pq_ncode][dsub]                                */
  uint8_t* codes;             /* [B][H_kv][N_max][M] (or [M/2] with pq_ncode == 16)          */
  uint16_t* list_ids;         /* [B][H_kv][N_max]                                            */
  float* key_norms;           /* [B][H_kv][N_max]                                            */
  float* list_vmeans;         /* [B][H_kv][n_list][d]                                        */
  int32_t* list_counts;       /* [B][H_kv][n_list]                                           */
} pqhsa_index_out;
size_t pqhsa_index_build_workspace_bytes(const pqhsa_params* params);
int pqhsa_index_build(const pqhsa_params* params, const pqhsa_paged_kv* kv, const int32_t* seq_lens,
                      const int32_t* seed_lists, const int32_t* seed_codes, int32_t coarse_iters,
                      int32_t pq_iters, const pqhsa_index_out* index, void* ws, size_t ws_bytes,
                      void* stream);

/* Dense decode attention over the WHOLE paged KV cache (Eq. 1 with E = every cached token):
 * softmax(q K^T / sqrt d) V per query head, split-K with a log-sum-exp merge.  Not a step of
 * PQ-HSA: it is the comparator of the context-length sweep (the full-KV read the paper's
 * Sec. 4.4 measures against), run on the same cache through the same strides.  Uses batch,
 * heads, head_dim, max_seq_len, page fields, sm_scale and dtype of `params`.  `ws`: device
 * scratch of pqhsa_dense_workspace_bytes(params) bytes, 256-byte aligned. */
size_t pqhsa_dense_workspace_bytes(const pqhsa_params* params);
int pqhsa_dense_decode(const pqhsa_params* params, const void* q, const pqhsa_paged_kv* kv,
                       const int32_t* seq_lens, void* out, void* ws, size_t ws_bytes, void* stream);

/* Measurement aid, not a step of the method: reads the K and V rows of the selected tokens (the
 * addresses the exact part of pqhsa_hybrid_attend gathers, through the same block table and
 * strides) with many rows in flight and computes nothing.  Its duration is the memory system's
 * price for that gather, the ceiling the attend stage is set against in the benchmark.
 * sel_idx / sel_count as pqhsa_select leaves them; sink16: 16 device bytes, 16-byte aligned,
 * never written in practice.  One launch on `stream`. */
int pqhsa_gather_probe(const pqhsa_params* params, const pqhsa_paged_kv* kv, const int32_t* sel_idx,
                       const int32_t* sel_count, const int32_t* seq_lens, void* sink16, void* stream);

/* pqhsa_decode for a caller whose query and output live in HOST memory (pinned for the
 * copies to be asynchronous): copies q_host -> q_dev_staging, runs the step, copies
 * out_dev_staging -> out_host and waits for the stream.  The index, the KV cache and
 * seq_lens stay resident on the device, as they do in a serving engine. */
int pqhsa_decode_host(const pqhsa_params* params, const void* q_host, void* q_dev_staging,
                      const pqhsa_index* index, const pqhsa_paged_kv* kv,
                      const int32_t* seq_lens, void* out_dev_staging, void* out_host,
                      void* ws, size_t ws_bytes, void* stream);

/* Reads the status word kernels set when they meet an inconsistency: copies it to the host and
 * waits for `stream`.  Returns PQHSA_OK or PQHSA_ERR_DEVICE_CHECK.  Valid after pqhsa_scan /
 * pqhsa_select / pqhsa_hybrid_attend / pqhsa_decode on the same ws.  Bits: 1 selected count != k,
 * 2 seq_len outside [0, max_seq_len], 4 a bounded wait on a bulk copy ran out, 64 a row kept its
 * approximate top-k in the re-score pass (see pqhsa_rescore); a library built
 * with -DPQHSA_DEBUG (pqhsa_debug_build() == 1) also records the indices that the release
 * build silently clamps or skips: 8 list id >= n_list, 16 selected position outside the indexed
 * region, 32 negative page id.  No check traps: the CUDA context stays usable. */
int pqhsa_last_device_status(const pqhsa_params* params, void* ws, void* stream);
int pqhsa_debug_build(void);
/* The predicate behind a debug check, for host-side unit tests: which = 0 list id (value < hi),
 * 1 position (lo <= value < hi), 2 page id (value >= 0).  Returns 1 / 0, -1 for an unknown check. */
int pqhsa_debug_predicate(int which, long long value, long long lo, long long hi);

/* Byte offset inside `ws` of an intermediate buffer after pqhsa_decode (for inspection by
 * tests and tools); (size_t)-1 on error. */
size_t pqhsa_decode_buffer_offset(const pqhsa_params* params, int which);

/* Number of kernels (memsets included) pqhsa_decode enqueues for these params. */
int pqhsa_decode_launch_count(const pqhsa_params* params);

const char* pqhsa_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* PQHSA_H_ */
