"""Float64 CPU oracle of the PQ-HSA decode-step attention operator.

TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA library is checked
against; it is deliberately plain and slow, shares no code with the library, and is
imported only by the tests, the smoke check and the benchmark's CPU-baseline leg.
The product path never calls it.

Every function restates one passage of the paper (Section 3, Eq. 1-5) in numpy
float64, in the paper's order and notation, without blocking, fusion or
re-ordering:

    O1  position partition S / L / R and the budget k = ceil(rho |R|)   (Sec. 3.2, Eq. 3; App. A "Budgets")
    O2  q = r_q u_q                                                      (Sec. 3.1)
    O3  coarse_j = u_q . c_j ,  LUT[m][z] = u_q^(m) . p_{m,z}            (Sec. 3.1, text after Eq. 2)
    O4  approximate logit of every indexed token                         (Eq. 2)
    O5  T = the k positions of R with the largest approximate logit     (Eq. 3)
    O6  exact logits on E = S u L u T from the original keys             (Sec. 3.2)
    O7  common shift m_0, e_i on E, e~_i on B = R \\ T                    (Sec. 3.2)
    O8  per-list background mass M_j, Z^_B, N^_B with the stored means   (Eq. 4)
    O9  y^ = (N_E + N^_B) / (Z_E + Z^_B)                                 (Eq. 5)
    O10 index maintenance: new tokens encoded into the existing lists,  (Sec. 3.3, first paragraph;
        list means refreshed, no re-clustering                           Sec. 3.1 for the encoding)
    V   the mechanism variants T, Bx, C, C2, C2b: other ways to form     (Table 2; App. B, "Variant
        the background term, same selector, budget and exact part        definitions")

Readings where the paper is silent (the repository's design notes list them too):
  * top-k ties: stable, the lower position wins;
  * rho is given in parts per million and k is computed in integers;
  * u_q = 0 when r_q = 0;
  * the list mean that multiplies M_j is the stored mean over all members of the
    list, selected ones included (Sec. 3.2, last paragraph);
  * an empty list contributes zero (text after Eq. 4);
  * the window L holds whatever the index does not cover yet: with `indexed_len` given,
    R = [|S|, indexed_len) and L = [indexed_len, N) (Sec. 3.3: new tokens stay exact until
    the next periodic update), otherwise L is the last n_local tokens;
  * variants: |R_j| is counted from the list ids of R; with an empty T the shared logit of
    C2 / C2b does not exist and the background is dropped; a list with no unselected member
    has no Bx mean and no mass;
  * index maintenance: a new key goes to the list whose centroid is nearest to its direction
    in squared Euclidean distance (the assignment rule of k-means, the lower index on ties),
    each sub-vector of the residual to its nearest codeword likewise, a zero key has
    direction 0, and the refreshed list mean is the mean over old and new members.

Pins (tests/test_oracle_pins.py): brute-force loops on tiny inputs, the ADC sum
against a dense dot product with the reconstructed key, rho = 1 against textbook
softmax attention, the exact-reconstruction / constant-value-per-list case against
textbook attention at any budget, a hand-computed closed form, mass conservation,
shift and permutation invariance, the budgets the paper prints (1,456 and 2,752
tokens at 131,072, also as the k that decode_head selects there), and top-k against a full
sort; decode() (query head -> KV head map, paged reads through two stride layouts) against
scalar loops on dense per-head arrays; for O10 scalar-loop brute force, the from-scratch mean
of all members, a key on a centroid, and one update against two; for the variants scalar loops,
hand-computed closed forms (2.125 / 2.5 / 1) and the cases where two variants must coincide.
No function here is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np


# --------------------------------------------------------------------------- O1
def budget_k(n_indexed: int, budget_ppm: int) -> int:
    """k = ceil(rho * |R|) with rho = budget_ppm / 10^6, in integers (Eq. 3)."""
    if n_indexed <= 0:
        return 0
    k = (n_indexed * budget_ppm + 999_999) // 1_000_000
    return min(k, n_indexed)


def partition(seq_len: int, n_sink: int = 0, n_local: int = 0, indexed_len=None):
    """Sink prefix S, local window L (most recent tokens) and indexed region R
    (Sec. 3.2).  Returned as position arrays; they are disjoint and cover [0, N).

    The window holds the tokens that are not in the index yet (Sec. 3.3: a new token is
    attended exactly until the next periodic update encodes it).  `indexed_len` is the
    number of leading positions the index covers, so R = [|S|, indexed_len) and L is
    everything after; without it the window is the last n_local tokens."""
    n_s = min(n_sink, seq_len)
    if indexed_len is None:
        l_start = max(n_s, seq_len - n_local)
    else:
        l_start = min(seq_len, max(n_s, int(indexed_len)))
    S = np.arange(0, n_s, dtype=np.int64)
    R = np.arange(n_s, l_start, dtype=np.int64)
    L = np.arange(l_start, seq_len, dtype=np.int64)
    return S, L, R


def exact_set_tokens(seq_len: int, n_sink: int, n_local: int, budget_ppm: int,
                     round_to_page: int = 0, indexed_len=None) -> int:
    """Number of tokens attended exactly: |S| + |L| + ceil(rho |R|), optionally
    rounded up to whole pages (App. A, "Budgets")."""
    S, L, R = partition(seq_len, n_sink, n_local, indexed_len)
    total = len(S) + len(L) + budget_k(len(R), budget_ppm)
    if round_to_page:
        total = round_to_page * ((total + round_to_page - 1) // round_to_page)
    return total


# --------------------------------------------------------------------------- O2, O3
def split_query(q: np.ndarray):
    """q = r_q u_q (Sec. 3.1)."""
    q = np.asarray(q, dtype=np.float64)
    r_q = float(np.sqrt(np.sum(q * q)))
    u_q = q / r_q if r_q > 0.0 else np.zeros_like(q)
    return r_q, u_q


def build_lut(u_q: np.ndarray, centroids: np.ndarray, codebooks: np.ndarray):
    """coarse[j] = u_q . c_j and LUT[m][z] = u_q^(m) . p_{m,z} (Sec. 3.1).

    centroids [n_list, d]; codebooks [M, n_code, dsub]; subspace m covers the
    contiguous dims [m*dsub, (m+1)*dsub)."""
    centroids = np.asarray(centroids, dtype=np.float64)
    codebooks = np.asarray(codebooks, dtype=np.float64)
    M, n_code, dsub = codebooks.shape
    coarse = centroids @ u_q
    lut = np.empty((M, n_code), dtype=np.float64)
    for m in range(M):
        lut[m] = codebooks[m] @ u_q[m * dsub:(m + 1) * dsub]
    return coarse, lut


# --------------------------------------------------------------------------- O4
def adc_logits(r_q: float, coarse: np.ndarray, lut: np.ndarray, codes: np.ndarray,
               list_ids: np.ndarray, key_norms: np.ndarray, sm_scale: float) -> np.ndarray:
    """Eq. 2: l~_i = (r_q r_i / sqrt d) (u_q.c_{a_i} + sum_m LUT[m][z_im]).

    codes [n, M] uint8, list_ids [n], key_norms [n] (None = all ones).
    sm_scale is 1/sqrt(d)."""
    codes = np.asarray(codes).astype(np.int64)
    list_ids = np.asarray(list_ids).astype(np.int64)
    n, M = codes.shape
    s = coarse[list_ids].astype(np.float64)
    for m in range(M):
        s = s + lut[m][codes[:, m]]
    r = np.ones(n) if key_norms is None else np.asarray(key_norms, dtype=np.float64)
    return (r_q * r * sm_scale) * s


# --------------------------------------------------------------------------- O5
def select_topk(scores: np.ndarray, k: int) -> np.ndarray:
    """Indices (into `scores`) of the k largest entries; among equal scores the
    lower index is taken first (Eq. 3 with a stable tie rule)."""
    if k <= 0:
        return np.zeros(0, dtype=np.int64)
    order = np.argsort(-np.asarray(scores, dtype=np.float64), kind="stable")
    return np.sort(order[:k])


# --------------------------------------------------------------------------- paged KV
def gather_rows(cache_flat: np.ndarray, block_table_row: np.ndarray, positions: np.ndarray,
                kv_head: int, head_dim: int, page_size: int,
                stride_page: int, stride_token: int, stride_head: int) -> np.ndarray:
    """Rows of one KV head at the given sequence positions, read in place from a
    paged cache described by element strides (Sec. 3.3: the gather reads the
    engine's pages in place)."""
    positions = np.asarray(positions, dtype=np.int64)
    page = np.asarray(block_table_row, dtype=np.int64)[positions // page_size]
    off = page * stride_page + (positions % page_size) * stride_token + kv_head * stride_head
    idx = off[:, None] + np.arange(head_dim, dtype=np.int64)[None, :]
    return np.asarray(cache_flat)[idx].astype(np.float64)


# --------------------------------------------------------------------------- O6-O9
VARIANTS = ("B", "T", "Bx", "C", "C2", "C2b")


def hybrid_output(q: np.ndarray, keys_E: np.ndarray, vals_E: np.ndarray,
                  logits_B: np.ndarray, lists_B: np.ndarray, list_vmeans: np.ndarray,
                  sm_scale: float, variant: str = "B", list_counts=None, is_T=None,
                  lists_T=None, approx_T=None):
    """Eq. 4-5 for one query head.

    keys_E, vals_E: original rows of the exact set E.  logits_B, lists_B: the
    approximate logit and list id of every background token (B = R \\ T).
    list_vmeans [n_list, d]: stored per-list value means.
    Returns y^ and a dict with the intermediate sums (all relative to m_0).

    `variant` switches how the background term is formed (Table 2 and App. B, "Variant
    definitions"); selector, budget and exact part are the same in all of them:
      B    PQ-HSA itself: logit l~_i, value vbar_j                               (Eq. 4)
      T    no background term (its logits are -inf)
      Bx   B with vbar_j replaced by the mean over the list's UNSELECTED members,
           (|R_j| vbar_j - sum_{i in T n R_j} v_i) / |B n R_j|
      C    logit l~_i, value = the token-count-weighted global mean
           vbar_global = sum_j |R_j| vbar_j / sum_j |R_j|
      C2   one shared logit mean_{i in T} l~_i for every background token, vbar_global
      C2b  one shared logit min_{i in T} l_i (exact logits), vbar_global
    The variants other than B and T need list_counts [n_list] = |R_j|; Bx also needs
    is_T (bool over the rows of E) and lists_T (list id of each selected row, in the
    order they appear in E); C2 needs approx_T (l~_i of the selected rows).
    Reading: with an empty T the shared logit of C2 / C2b is undefined and the background
    is dropped; a list whose members are all selected has no unselected mean and no mass."""
    if variant not in VARIANTS:
        raise ValueError(variant)
    q = np.asarray(q, dtype=np.float64)
    d = q.shape[0]
    list_vmeans = np.asarray(list_vmeans, dtype=np.float64)
    n_list = list_vmeans.shape[0]
    logits_E = (np.asarray(keys_E, dtype=np.float64).reshape(-1, d) @ q) * sm_scale
    vals_E = np.asarray(vals_E, dtype=np.float64).reshape(-1, d)
    logits_B = np.asarray(logits_B, dtype=np.float64)
    lists_B = np.asarray(lists_B).astype(np.int64)

    # background logits of the variant
    if variant == "T":
        logits_B = np.full(logits_B.shape, -math.inf)
    elif variant in ("C2", "C2b"):
        n_T = 0 if is_T is None else int(np.count_nonzero(is_T))
        if n_T == 0:
            shared = -math.inf
        elif variant == "C2":
            shared = float(np.mean(np.asarray(approx_T, dtype=np.float64)))
        else:
            shared = float(np.min(logits_E[np.asarray(is_T, dtype=bool)]))
        logits_B = np.full(logits_B.shape, shared)

    cands = [x.max() for x in (logits_E, logits_B) if x.size]
    cands = [c for c in cands if c > -math.inf]
    if not cands:                                   # empty sequence
        return np.zeros(d), dict(m0=-math.inf, Z_E=0.0, Z_B=0.0, M=np.zeros(n_list),
                                 logits_E=logits_E)
    m0 = max(cands)
    e_E = np.exp(logits_E - m0)
    e_B = np.exp(logits_B - m0)
    Z_E = e_E.sum()
    N_E = e_E @ vals_E
    # M_j = sum of e~_i over the background members of list j (empty list -> 0)
    M_j = np.bincount(lists_B, weights=e_B, minlength=n_list).astype(np.float64)
    Z_B = M_j.sum()

    # background values of the variant
    if variant in ("B", "T"):
        N_B = M_j @ list_vmeans
    elif variant == "Bx":
        counts = np.asarray(list_counts, dtype=np.float64)
        sel_rows = vals_E[np.asarray(is_T, dtype=bool)]
        sel_lists = np.asarray(lists_T).astype(np.int64)
        sum_T = np.zeros((n_list, d))
        np.add.at(sum_T, sel_lists, sel_rows)
        n_unsel = counts - np.bincount(sel_lists, minlength=n_list)
        vbar_B = np.zeros((n_list, d))
        has = n_unsel > 0
        vbar_B[has] = (counts[has, None] * list_vmeans[has] - sum_T[has]) / n_unsel[has, None]
        N_B = M_j @ vbar_B
    else:                                            # C, C2, C2b
        counts = np.asarray(list_counts, dtype=np.float64)
        total = counts.sum()
        v_global = (counts @ list_vmeans) / total if total > 0 else np.zeros(d)
        N_B = Z_B * v_global
    y = (N_E + N_B) / (Z_E + Z_B)
    return y, dict(m0=m0, Z_E=Z_E, Z_B=Z_B, M=M_j, logits_E=logits_E,
                   lse=m0 + math.log(Z_E + Z_B))


def decode_head(q, centroids, codebooks, codes, list_ids, key_norms, list_vmeans,
                keys, vals, seq_len, budget_ppm, sm_scale, n_sink=0, n_local=0,
                round_exact_set_to_page=0, indexed_len=None, variant="B"):
    """One (sequence, query head): O1-O9.

    keys / vals are callables position-array -> rows [len, d] (original K, V of the
    query head's KV head); the index arrays belong to the same KV head and are
    indexed by sequence position.  Returns a dict with y^ and every intermediate."""
    q = np.asarray(q, dtype=np.float64)
    S, L, R = partition(seq_len, n_sink, n_local, indexed_len)
    k = budget_k(len(R), budget_ppm)
    if round_exact_set_to_page:
        total = exact_set_tokens(seq_len, n_sink, n_local, budget_ppm, round_exact_set_to_page,
                                 indexed_len)
        k = min(len(R), total - len(S) - len(L))
    r_q, u_q = split_query(q)
    coarse, lut = build_lut(u_q, centroids, codebooks)
    norms_R = None if key_norms is None else np.asarray(key_norms)[R]
    lists_R = np.asarray(list_ids)[R].astype(np.int64)
    approx = adc_logits(r_q, coarse, lut, np.asarray(codes)[R], lists_R, norms_R, sm_scale)
    sel_local = select_topk(approx, k)
    T = R[sel_local]
    mask_B = np.ones(len(R), dtype=bool)
    mask_B[sel_local] = False
    E = np.concatenate([S, L, T])
    is_T = np.concatenate([np.zeros(len(S) + len(L), dtype=bool), np.ones(len(T), dtype=bool)])
    n_list = np.asarray(list_vmeans).shape[0]
    y, aux = hybrid_output(q, keys(E), vals(E), approx[mask_B], lists_R[mask_B], list_vmeans,
                           sm_scale, variant=variant,
                           list_counts=np.bincount(lists_R, minlength=n_list), is_T=is_T,
                           lists_T=lists_R[sel_local], approx_T=approx[sel_local])
    kth = float(np.sort(approx)[::-1][k - 1]) if k > 0 else math.nan
    aux.update(y=y, r_q=r_q, u_q=u_q, coarse=coarse, lut=lut, approx=approx, R=R, T=T,
               E=E, k=k, kth_score=kth)
    return aux


def decode(q, centroids, codebooks, codes, list_ids, key_norms, list_vmeans,
           k_cache_flat, v_cache_flat, block_table, seq_lens, *, n_kv_heads, page_size,
           stride_page, stride_token, stride_head, budget_ppm, sm_scale,
           n_sink=0, n_local=0, heads=None, batch_items=None, round_exact_set_to_page=0,
           indexed_lens=None, variant="B"):
    """The whole operator: every (sequence, query head), reading the paged cache in
    place.  Array layouts are those of the C ABI (q [B,Hq,d]; centroids
    [B,Hkv,n_list,d]; codebooks [B,Hkv,M,n_code,dsub]; codes [B,Hkv,N_max,M];
    list_ids / key_norms [B,Hkv,N_max]; list_vmeans [B,Hkv,n_list,d]).  Query head h reads
    the index and the cache rows of KV head h // G, G = Hq / n_kv_heads (Sec. 3.3: the heads
    of a group share their KV head's codes).  indexed_lens [B] (optional): see partition().
    Returns {(b, h): decode_head result}; `heads` / `batch_items` restrict the work."""
    q = np.asarray(q, dtype=np.float64)
    B, Hq, d = q.shape
    G = Hq // n_kv_heads
    out = {}
    for b in (range(B) if batch_items is None else batch_items):
        n = int(seq_lens[b])
        for h in (range(Hq) if heads is None else heads):
            g = h // G
            keys = lambda pos, g=g, b=b: gather_rows(k_cache_flat, block_table[b], pos, g, d,
                                                     page_size, stride_page, stride_token,
                                                     stride_head)
            vals = lambda pos, g=g, b=b: gather_rows(v_cache_flat, block_table[b], pos, g, d,
                                                     page_size, stride_page, stride_token,
                                                     stride_head)
            out[(b, h)] = decode_head(
                q[b, h], centroids[b, g], codebooks[b, g], codes[b, g], list_ids[b, g],
                None if key_norms is None else key_norms[b, g], list_vmeans[b, g],
                keys, vals, n, budget_ppm, sm_scale, n_sink, n_local, round_exact_set_to_page,
                None if indexed_lens is None else int(indexed_lens[b]), variant)
    return out


# --------------------------------------------------------------------------- O10
def encode_keys(keys: np.ndarray, centroids: np.ndarray, codebooks: np.ndarray):
    """Direction-norm residual IVF-PQ encoding of keys [n, d] against fixed centroids
    [n_list, d] and codebooks [M, n_code, dsub] (Sec. 3.1): r_i = |k_i|, u_i = k_i / r_i,
    a_i = argmin_j |u_i - c_j|^2, z_im = argmin_z |(u_i - c_{a_i})^(m) - p_{m,z}|^2.
    Returns (norms [n], list_ids [n], codes [n, M], d_coarse [n, n_list], d_pq [n, M, n_code]);
    the two distance arrays let a test see how close a decision was."""
    keys = np.asarray(keys, dtype=np.float64)
    c = np.asarray(centroids, dtype=np.float64)
    cb = np.asarray(codebooks, dtype=np.float64)
    n, d = keys.shape
    M, n_code, dsub = cb.shape
    r = np.sqrt((keys * keys).sum(axis=1))
    u = np.zeros_like(keys)
    nz = r > 0
    u[nz] = keys[nz] / r[nz, None]
    d_coarse = ((u[:, None, :] - c[None, :, :]) ** 2).sum(axis=2)            # [n, n_list]
    a = d_coarse.argmin(axis=1)                                              # first minimum
    e = (u - c[a]).reshape(n, M, dsub)
    d_pq = ((e[:, :, None, :] - cb[None, :, :, :]) ** 2).sum(axis=3)         # [n, M, n_code]
    z = d_pq.argmin(axis=2)
    return r, a, z, d_coarse, d_pq


def index_update(centroids, codebooks, codes, list_ids, key_norms, list_vmeans, list_counts,
                 new_keys, new_vals, first_pos: int):
    """Index maintenance for one (sequence, KV head) (Sec. 3.3): the tokens at positions
    first_pos, first_pos + 1, ... are encoded into the existing lists (no re-clustering),
    and every list's value mean becomes the mean over its old and new members:
    vbar_j <- (n_j vbar_j + sum of the new members' values) / (n_j + new_j).
    Returns updated copies (codes, list_ids, key_norms, list_vmeans, list_counts) and the
    distance arrays of encode_keys."""
    new_vals = np.asarray(new_vals, dtype=np.float64)
    r, a, z, d_coarse, d_pq = encode_keys(new_keys, centroids, codebooks)
    n_new = len(r)
    codes = np.array(codes, copy=True)
    list_ids = np.array(list_ids, copy=True)
    key_norms = np.array(key_norms, dtype=np.float64, copy=True)
    vmeans = np.array(list_vmeans, dtype=np.float64, copy=True)
    counts = np.array(list_counts, dtype=np.int64, copy=True)
    pos = first_pos + np.arange(n_new)
    codes[pos] = z.astype(codes.dtype)
    list_ids[pos] = a.astype(list_ids.dtype)
    key_norms[pos] = r
    n_list = vmeans.shape[0]
    added = np.bincount(a, minlength=n_list)
    vsum = np.zeros_like(vmeans)
    np.add.at(vsum, a, new_vals)
    touched = added > 0
    vmeans[touched] = (counts[touched, None] * vmeans[touched] + vsum[touched]) / \
                      (counts[touched] + added[touched])[:, None]
    counts = counts + added
    return dict(codes=codes, list_ids=list_ids, key_norms=key_norms, list_vmeans=vmeans,
                list_counts=counts, d_coarse=d_coarse, d_pq=d_pq)

