"""Pins of the float64 oracle to things other than itself (CPU only).

Each test fixes part of oracle/pqhsa_oracle.py to a value or property that comes
from the paper or from plain mathematics: brute-force loops on tiny inputs, a dense
dot product with the reconstructed key, textbook softmax attention, a hand-computed
closed form, conservation laws, and the token budgets printed in the paper.
"""
import math
import os

import numpy as np
import pytest
from scipy.special import softmax

from oracle import pqhsa_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers
def dense_attention(q, K, V, sm_scale):
    """Textbook softmax attention (Eq. 1 with E = everything), via scipy's softmax."""
    w = softmax((K @ q) * sm_scale)
    return w @ V


def random_index(rng, n, d, n_list, M, n_code, exact=False):
    """A random IVF-PQ index over n tokens.  With exact=True the keys are built FROM
    the index (k_i = r_i (c_{a_i} + concat_m p_{m,z_im})) out of dyadic rationals, so
    the PQ reconstruction is exact in floating point."""
    dsub = d // M
    if exact:
        centroids = rng.integers(-4, 5, (n_list, d)) / 8.0
        codebooks = rng.integers(-4, 5, (M, n_code, dsub)) / 16.0
        norms = 2.0 ** rng.integers(-1, 2, n)
    else:
        centroids = rng.normal(size=(n_list, d)) * 0.3
        codebooks = rng.normal(size=(M, n_code, dsub)) * 0.1
        norms = rng.uniform(0.5, 2.0, n)
    list_ids = rng.integers(0, n_list, n)
    codes = rng.integers(0, n_code, (n, M)).astype(np.uint8)
    recon = centroids[list_ids] + np.concatenate(
        [codebooks[m][codes[:, m]] for m in range(M)], axis=1)
    return centroids, codebooks, codes, list_ids, norms, recon * norms[:, None]


def list_means(V, list_ids, n_list):
    out = np.zeros((n_list, V.shape[1]))
    for j in range(n_list):
        if np.any(list_ids == j):
            out[j] = V[list_ids == j].mean(axis=0)
    return out


def run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, ppm, n_sink=0, n_local=0, **kw):
    n, d = K.shape
    return O.decode_head(q, cen, cb, codes, ids, norms, vmeans,
                         lambda pos: K[pos], lambda pos: V[pos], n, ppm,
                         1.0 / math.sqrt(d), n_sink, n_local, **kw)


# ----------------------------------------------------------------------------- P1
def brute_force(q, cen, cb, codes, ids, norms, vmeans, K, V, ppm, n_sink, n_local):
    """Eq. 2-5 written as scalar loops, straight from the definitions."""
    n, d = K.shape
    M, n_code, dsub = cb.shape
    rq = math.sqrt(sum(float(x) ** 2 for x in q))
    uq = [float(x) / rq for x in q]
    n_s = min(n_sink, n)
    l0 = max(n_s, n - n_local)
    R = list(range(n_s, l0))
    approx = {}
    for i in R:
        acc = sum(uq[t] * cen[ids[i]][t] for t in range(d))
        for m in range(M):
            for t in range(dsub):
                acc += uq[m * dsub + t] * cb[m][codes[i][m]][t]
        approx[i] = rq * norms[i] / math.sqrt(d) * acc
    k = min(len(R), -(-len(R) * ppm // 1_000_000))
    T = sorted(R, key=lambda i: (-approx[i], i))[:k]
    E = list(range(n_s)) + list(range(l0, n)) + T
    Bset = [i for i in R if i not in set(T)]
    exact = {i: sum(float(q[t]) * K[i][t] for t in range(d)) / math.sqrt(d) for i in E}
    m0 = max(list(exact.values()) + [approx[i] for i in Bset])
    num = [0.0] * d
    den = 0.0
    for i in E:
        e = math.exp(exact[i] - m0)
        den += e
        for t in range(d):
            num[t] += e * V[i][t]
    Mj = [0.0] * len(vmeans)
    for i in Bset:
        Mj[ids[i]] += math.exp(approx[i] - m0)
    for j, mass in enumerate(Mj):
        den += mass
        for t in range(d):
            num[t] += mass * vmeans[j][t]
    return np.array(num) / den, sorted(T), approx


@pytest.mark.parametrize("seed,n,ppm,n_sink,n_local", [
    (0, 48, 125000, 0, 0), (1, 64, 62500, 2, 5), (2, 17, 300000, 0, 3), (3, 9, 1000000, 1, 1),
    (4, 33, 0, 2, 2)])
def test_p1_brute_force_tiny(seed, n, ppm, n_sink, n_local):
    rng = np.random.default_rng(seed)
    d, n_list, M, n_code = 4, 4, 2, 4
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    K = rng.normal(size=(n, d))
    V = rng.normal(size=(n, d))
    q = rng.normal(size=d)
    vmeans = rng.normal(size=(n_list, d))          # arbitrary stored means
    res = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, ppm, n_sink, n_local)
    y_bf, T_bf, approx_bf = brute_force(q, cen, cb, codes, ids, norms, vmeans, K, V, ppm,
                                        n_sink, n_local)
    assert sorted(res["T"].tolist()) == T_bf
    np.testing.assert_allclose(res["approx"], [approx_bf[i] for i in res["R"]], rtol=1e-12,
                               atol=1e-14)
    np.testing.assert_allclose(res["y"], y_bf, rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------------- P2
@pytest.mark.parametrize("d,M,n_code", [(128, 32, 256), (128, 16, 256), (16, 4, 8)])
def test_p2_adc_equals_dot_with_reconstructed_key(d, M, n_code):
    rng = np.random.default_rng(5)
    n, n_list = 300, 7
    cen, cb, codes, ids, norms, Khat = random_index(rng, n, d, n_list, M, n_code)
    q = rng.normal(size=d)
    r_q, u_q = O.split_query(q)
    coarse, lut = O.build_lut(u_q, cen, cb)
    got = O.adc_logits(r_q, coarse, lut, codes, ids, norms, 1 / math.sqrt(d))
    np.testing.assert_allclose(got, Khat @ q / math.sqrt(d), rtol=1e-11, atol=1e-12)
    assert lut.shape == (M, n_code) and coarse.shape == (n_list,)
    # without norms the keys are taken as unit-norm reconstructions
    got1 = O.adc_logits(r_q, coarse, lut, codes, ids, None, 1 / math.sqrt(d))
    np.testing.assert_allclose(got1, (Khat / norms[:, None]) @ q / math.sqrt(d), rtol=1e-11,
                               atol=1e-12)


def test_p2_norm_explicit_scaling():
    """Scaling a key and its stored norm by alpha leaves direction, list and codes
    unchanged, so the approximate logit scales by alpha (Sec. 3.1)."""
    rng = np.random.default_rng(6)
    d, M, n_code, n, n_list = 32, 8, 16, 50, 5
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    q = rng.normal(size=d)
    r_q, u_q = O.split_query(q)
    coarse, lut = O.build_lut(u_q, cen, cb)
    a = O.adc_logits(r_q, coarse, lut, codes, ids, norms, 0.25)
    b = O.adc_logits(r_q, coarse, lut, codes, ids, norms * 3.0, 0.25)
    np.testing.assert_allclose(b, 3.0 * a, rtol=1e-13)
    assert abs(np.linalg.norm(u_q) - 1.0) < 1e-14 and abs(r_q - np.linalg.norm(q)) < 1e-14


# ----------------------------------------------------------------------------- P3
@pytest.mark.parametrize("n_sink,n_local", [(0, 0), (4, 16)])
def test_p3_full_budget_is_dense_attention(n_sink, n_local):
    rng = np.random.default_rng(7)
    d, M, n_code, n, n_list = 32, 8, 16, 200, 6
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    K, V, q = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=d)
    vmeans = rng.normal(size=(n_list, d))          # must not matter: B is empty
    res = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 1_000_000, n_sink, n_local)
    np.testing.assert_allclose(res["y"], dense_attention(q, K, V, 1 / math.sqrt(d)),
                               rtol=1e-11, atol=1e-13)
    assert res["k"] == n - min(n_sink, n) - n_local and res["Z_B"] == 0.0


# ----------------------------------------------------------------------------- P4
@pytest.mark.parametrize("ppm", [0, 10000, 100000, 500000])
def test_p4_exact_reconstruction_constant_values_is_dense(ppm):
    """If PQ reconstructs every key exactly and all values of a list are equal (so
    they equal the list mean), Eq. 5 is full attention at ANY budget."""
    rng = np.random.default_rng(8)
    d, M, n_code, n, n_list = 16, 4, 8, 257, 5
    cen, cb, codes, ids, norms, K = random_index(rng, n, d, n_list, M, n_code, exact=True)
    per_list_value = rng.integers(-8, 9, (n_list, d)) / 4.0
    V = per_list_value[ids]
    q = rng.integers(-8, 9, d) / 4.0
    vmeans = list_means(V, ids, n_list)
    res = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, ppm)
    np.testing.assert_allclose(res["y"], dense_attention(q, K, V, 1 / math.sqrt(d)),
                               rtol=1e-10, atol=1e-12)
    # and the approximate logits ARE the exact logits here
    np.testing.assert_allclose(res["approx"], K @ q / math.sqrt(d), rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------------------- P5
def test_p5_closed_form_list_mean_counts_selected_members():
    """One list, identical keys with exact codes: every logit is equal, so with N=4,
    k=1 and scalar-like values 1,2,3,4 the stable rule selects position 0 and
    y = (v_0 + (N-k) * vbar) / N = (1 + 3*2.5)/4 = 2.125, because vbar is the mean
    over ALL members (Sec. 3.2, last paragraph).  Dense attention would give 2.5."""
    d, M, n_code = 4, 2, 2
    cen = np.array([[0.5, 0.5, 0.5, 0.5]])
    cb = np.zeros((M, n_code, d // M))
    codes = np.zeros((4, M), dtype=np.uint8)
    ids = np.zeros(4, dtype=np.int64)
    norms = np.ones(4)
    K = np.tile(cen, (4, 1))
    V = np.array([[1.0] * d, [2.0] * d, [3.0] * d, [4.0] * d])
    vmeans = V.mean(axis=0, keepdims=True)
    q = np.array([1.0, -2.0, 0.5, 3.0])
    res = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 250000)
    assert res["k"] == 1 and res["T"].tolist() == [0]
    np.testing.assert_allclose(res["y"], np.full(d, 2.125), rtol=1e-14)


# ----------------------------------------------------------------------------- P6
def test_p6_mass_conservation_hull_and_empty_lists():
    rng = np.random.default_rng(9)
    d, M, n_code, n, n_list = 32, 8, 16, 400, 12
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    ids[ids == 3] = 2                               # list 3 is empty
    K, V, q = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=d)
    vmeans = list_means(V, ids, n_list)
    res = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 50000)
    approx, T, m0 = res["approx"], res["T"], res["m0"]
    # Z^_B + sum over T of e~_i = sum over R of e~_i
    np.testing.assert_allclose(res["Z_B"] + np.exp(approx[T] - m0).sum(),
                               np.exp(approx - m0).sum(), rtol=1e-12)
    assert res["M"][3] == 0.0 and np.all(res["M"] >= 0)
    # y^ is a convex combination of exact values and list means
    pts = np.concatenate([V[res["E"]], vmeans])
    assert np.all(res["y"] <= pts.max(axis=0) + 1e-12)
    assert np.all(res["y"] >= pts.min(axis=0) - 1e-12)
    # m_0 is the maximum over exact and approximate logits that enter the softmax
    maskB = np.ones(n, bool)
    maskB[T] = False
    assert m0 == max((K[res["E"]] @ q / math.sqrt(d)).max(), approx[maskB].max())


def test_p6_permutation_invariance():
    rng = np.random.default_rng(10)
    d, M, n_code, n, n_list = 32, 8, 16, 300, 9
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    K, V, q = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=d)
    vmeans = list_means(V, ids, n_list)
    a = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 30000)
    p = rng.permutation(n)
    b = run_head(q, cen, cb, codes[p], ids[p], norms[p], vmeans, K[p], V[p], 30000)
    np.testing.assert_allclose(a["y"], b["y"], rtol=1e-11, atol=1e-13)
    assert sorted(p[b["T"]].tolist()) == sorted(a["T"].tolist())


# ----------------------------------------------------------------------------- P7
def test_p7_budgets_printed_in_the_paper():
    """tests/golden/paper_budgets.txt: exact-set sizes printed in App. A."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "paper_budgets.txt"))
            if l.strip() and not l.startswith("#")]
    assert rows
    for seq_len, n_sink, n_local, ppm, page, tokens in (map(int, r) for r in rows):
        assert O.exact_set_tokens(seq_len, n_sink, n_local, ppm, page) == tokens
    assert O.budget_k(4096, 20000) == 82            # ceil(0.02 * 4096)
    assert O.budget_k(131072, 10000) == 1311 and O.budget_k(131072, 20000) == 2622
    assert O.budget_k(0, 10000) == 0 and O.budget_k(5, 1_000_000) == 5
    assert O.budget_k(100, 10000) == 1 and O.budget_k(101, 10000) == 2
    S, L, R = O.partition(131072, 4, 128)
    assert (len(S), len(L), len(R)) == (4, 128, 130940) and R[0] == 4 and L[0] == 130944


# ----------------------------------------------------------------------------- P8
def test_p8_topk_against_full_sort_and_ties():
    rng = np.random.default_rng(11)
    x = rng.normal(size=1000)
    for k in (0, 1, 7, 999, 1000):
        got = O.select_topk(x, k)
        ref = np.sort(np.argsort(x)[::-1][:k])
        assert got.tolist() == ref.tolist()
    y = np.array([1.0, 3.0, 3.0, 2.0, 3.0, 0.0])
    assert O.select_topk(y, 2).tolist() == [1, 2]   # equal scores: lower position first
    assert O.select_topk(y, 4).tolist() == [1, 2, 3, 4]


# ----------------------------------------------------------------------------- paged gather
def test_gather_rows_two_layouts_and_flat_are_identical():
    """Rows gathered through a split layout, an interleaved layout and a flat buffer
    are the same bits (App. E: the gather reads either engine layout in place)."""
    rng = np.random.default_rng(12)
    n, H, d, P = 75, 3, 8, 16
    n_pages = (n + P - 1) // P
    K = rng.normal(size=(n, H, d)).astype(np.float32)
    V = rng.normal(size=(n, H, d)).astype(np.float32)
    table = rng.permutation(n_pages + 3)[:n_pages]
    split_k = np.zeros((n_pages + 3, P, H, d), np.float32)
    split_v = np.zeros_like(split_k)
    inter = np.zeros((n_pages + 3, H, P, 2 * d), np.float32)
    for i in range(n):
        split_k[table[i // P], i % P] = K[i]
        split_v[table[i // P], i % P] = V[i]
        inter[table[i // P], :, i % P, :d] = K[i]
        inter[table[i // P], :, i % P, d:] = V[i]
    pos = rng.permutation(n)[:40]
    for h in range(H):
        a = O.gather_rows(split_k.ravel(), table, pos, h, d, P, P * H * d, H * d, d)
        b = O.gather_rows(inter.ravel(), table, pos, h, d, P, H * P * 2 * d, 2 * d, P * 2 * d)
        assert np.array_equal(a, K[pos, h].astype(np.float64)) and np.array_equal(a, b)
        va = O.gather_rows(split_v.ravel(), table, pos, h, d, P, P * H * d, H * d, d)
        vb = O.gather_rows(inter.ravel()[d:], table, pos, h, d, P, H * P * 2 * d, 2 * d,
                           P * 2 * d)
        assert np.array_equal(va, V[pos, h].astype(np.float64)) and np.array_equal(va, vb)


# ----------------------------------------------------------------------------- O10 index maintenance
def _tiny_index(rng, n_list=3, d=4, M=2, n_code=4, n_old=7):
    centroids = rng.normal(size=(n_list, d))
    codebooks = rng.normal(size=(M, n_code, d // M)) * 0.3
    old_ids = rng.integers(0, n_list, size=n_old)
    old_vals = rng.normal(size=(n_old, d))
    vmeans = np.zeros((n_list, d))
    counts = np.bincount(old_ids, minlength=n_list)
    for j in range(n_list):
        if counts[j]:
            vmeans[j] = old_vals[old_ids == j].mean(axis=0)
    N = n_old + 8
    codes = np.zeros((N, M), dtype=np.uint8)
    ids = np.zeros(N, dtype=np.uint16)
    ids[:n_old] = old_ids
    norms = np.zeros(N)
    return centroids, codebooks, codes, ids, norms, vmeans, counts, old_ids, old_vals


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_index_update_brute_force_and_from_scratch_means(seed):
    """Scalar loops for the assignment and the codes; the refreshed means against the mean of
    all members computed from scratch."""
    rng = np.random.default_rng(seed)
    c, cb, codes, ids, norms, vmeans, counts, old_ids, old_vals = _tiny_index(rng)
    n_old, n_new = len(old_ids), 5
    keys = rng.normal(size=(n_new, 4)) * 2.0
    vals = rng.normal(size=(n_new, 4))
    out = O.index_update(c, cb, codes, ids, norms, vmeans, counts, keys, vals, first_pos=n_old)
    M, n_code, dsub = cb.shape
    for t in range(n_new):
        r = math.sqrt(sum(x * x for x in keys[t]))
        u = [x / r for x in keys[t]]
        best, best_j = None, None
        for j in range(len(c)):
            dist = sum((u[i] - c[j][i]) ** 2 for i in range(4))
            if best is None or dist < best:
                best, best_j = dist, j
        assert out["list_ids"][n_old + t] == best_j
        assert abs(out["key_norms"][n_old + t] - r) < 1e-12
        for m in range(M):
            e = [u[m * dsub + i] - c[best_j][m * dsub + i] for i in range(dsub)]
            bz, bd = None, None
            for z in range(n_code):
                dist = sum((e[i] - cb[m][z][i]) ** 2 for i in range(dsub))
                if bd is None or dist < bd:
                    bd, bz = dist, z
            assert out["codes"][n_old + t, m] == bz
    all_ids = np.concatenate([old_ids, out["list_ids"][n_old:n_old + n_new].astype(np.int64)])
    all_vals = np.concatenate([old_vals, vals])
    for j in range(len(c)):
        members = all_vals[all_ids == j]
        assert out["list_counts"][j] == len(members)
        if len(members):
            np.testing.assert_allclose(out["list_vmeans"][j], members.mean(axis=0), atol=1e-12)
    # nothing outside the new positions moved
    assert np.array_equal(out["codes"][:n_old], codes[:n_old])
    assert np.array_equal(out["list_ids"][:n_old], ids[:n_old])


def test_index_update_key_on_a_centroid_has_zero_residual():
    """Orthonormal centroids: a key 3 e_j has norm 3, lands in list j, and its residual is 0,
    so every sub-vector takes the zero codeword."""
    c = np.eye(4)
    cb = np.random.default_rng(3).normal(size=(2, 6, 2))
    cb[:, 5, :] = 0.0
    codes = np.zeros((4, 2), dtype=np.uint8)
    out = O.index_update(c, cb, codes, np.zeros(4, dtype=np.uint16), np.zeros(4),
                         np.zeros((4, 4)), np.zeros(4, dtype=np.int64),
                         new_keys=3.0 * np.eye(4)[[2, 0]], new_vals=np.ones((2, 4)), first_pos=1)
    assert out["list_ids"][1:3].tolist() == [2, 0]
    assert out["key_norms"][1:3].tolist() == [3.0, 3.0]
    assert out["codes"][1:3].tolist() == [[5, 5], [5, 5]]
    assert out["list_counts"].tolist() == [1, 0, 1, 0]
    np.testing.assert_array_equal(out["list_vmeans"][[0, 2]], np.ones((2, 4)))
    # a zero key: direction 0, norm 0, nearest centroid by the same rule (all at distance 1: list 0)
    out0 = O.index_update(c, cb, codes, np.zeros(4, dtype=np.uint16), np.zeros(4),
                          np.zeros((4, 4)), np.zeros(4, dtype=np.int64),
                          new_keys=np.zeros((1, 4)), new_vals=np.ones((1, 4)), first_pos=0)
    assert out0["key_norms"][0] == 0.0 and out0["list_ids"][0] == 0


def test_index_update_in_two_steps_equals_one_step():
    rng = np.random.default_rng(9)
    c, cb, codes, ids, norms, vmeans, counts, old_ids, old_vals = _tiny_index(rng, n_list=4)
    n_old = len(old_ids)
    keys = rng.normal(size=(8, 4))
    vals = rng.normal(size=(8, 4))
    one = O.index_update(c, cb, codes, ids, norms, vmeans, counts, keys, vals, first_pos=n_old)
    a = O.index_update(c, cb, codes, ids, norms, vmeans, counts, keys[:3], vals[:3], first_pos=n_old)
    b = O.index_update(c, cb, a["codes"], a["list_ids"], a["key_norms"], a["list_vmeans"],
                       a["list_counts"], keys[3:], vals[3:], first_pos=n_old + 3)
    assert np.array_equal(one["codes"], b["codes"]) and np.array_equal(one["list_ids"], b["list_ids"])
    assert np.array_equal(one["list_counts"], b["list_counts"])
    np.testing.assert_allclose(one["list_vmeans"], b["list_vmeans"], atol=1e-12)
    np.testing.assert_allclose(one["key_norms"], b["key_norms"], atol=0)


# ----------------------------------------------------------------------------- decode(): GQA map and paged glue
def _paged_case(rng, layout, B=2, Hkv=2, G=2, d=4, P=4, n_list=3, M=2, n_code=4,
                seq_lens=(21, 10)):
    """A tiny batch in the C ABI's layouts with a shuffled block table.  Returns the arrays
    decode() takes plus dense per-(sequence, KV head) copies K[b][g], V[b][g] for brute force."""
    Hq, dsub = Hkv * G, d // M
    N_max = max(seq_lens)
    pages = [(n + P - 1) // P for n in seq_lens]
    total = sum(pages) + 2                                   # two pages nobody owns
    perm = rng.permutation(total)
    table = np.zeros((B, max(pages)), dtype=np.int32)
    o = 0
    for b in range(B):
        table[b, :pages[b]] = perm[o:o + pages[b]]
        o += pages[b]
    K = rng.normal(size=(B, Hkv, N_max, d))
    V = rng.normal(size=(B, Hkv, N_max, d))
    if layout == "split":
        kc = np.full((total, P, Hkv, d), 99.0)
        vc = np.full((total, P, Hkv, d), -99.0)
        strides = (P * Hkv * d, Hkv * d, d)
        for b in range(B):
            for i in range(seq_lens[b]):
                kc[table[b, i // P], i % P] = K[b, :, i]
                vc[table[b, i // P], i % P] = V[b, :, i]
        k_flat, v_flat = kc.ravel(), vc.ravel()
    else:
        buf = np.full((total, Hkv, P, 2 * d), 99.0)
        strides = (Hkv * P * 2 * d, 2 * d, P * 2 * d)
        for b in range(B):
            for i in range(seq_lens[b]):
                buf[table[b, i // P], :, i % P, :d] = K[b, :, i]
                buf[table[b, i // P], :, i % P, d:] = V[b, :, i]
        k_flat, v_flat = buf.ravel(), buf.ravel()[d:]
    arrays = dict(
        q=rng.normal(size=(B, Hq, d)),
        centroids=rng.normal(size=(B, Hkv, n_list, d)) * 0.3,
        codebooks=rng.normal(size=(B, Hkv, M, n_code, dsub)) * 0.1,
        codes=rng.integers(0, n_code, (B, Hkv, N_max, M)).astype(np.uint8),
        list_ids=rng.integers(0, n_list, (B, Hkv, N_max)).astype(np.uint16),
        key_norms=rng.uniform(0.5, 2.0, (B, Hkv, N_max)),
        list_vmeans=rng.normal(size=(B, Hkv, n_list, d)),
        k_cache_flat=k_flat, v_cache_flat=v_flat, block_table=table,
        seq_lens=np.array(seq_lens, dtype=np.int32))
    return arrays, strides, K, V, dict(B=B, Hkv=Hkv, G=G, Hq=Hq, d=d, P=P)


@pytest.mark.parametrize("layout", ["split", "interleaved"])
def test_decode_maps_query_heads_to_kv_heads_and_reads_pages_in_place(layout):
    """decode() against scalar loops that choose the KV head floor(h / G) themselves and are
    handed dense K, V (Sec. 3.3: the query heads of a group share their KV head's codes; App. E:
    rows are read from the engine's pages through strides).  Every (sequence, KV head) has its
    own index and its own keys, so a wrong head map (h % H_kv, a swapped b/g) or a wrong page
    lookup changes the result."""
    rng = np.random.default_rng(21)
    a, strides, K, V, sh = _paged_case(rng, layout)
    ppm, n_sink, n_local = 200000, 1, 3
    res = O.decode(a["q"], a["centroids"], a["codebooks"], a["codes"], a["list_ids"],
                   a["key_norms"], a["list_vmeans"], a["k_cache_flat"], a["v_cache_flat"],
                   a["block_table"], a["seq_lens"], n_kv_heads=sh["Hkv"], page_size=sh["P"],
                   stride_page=strides[0], stride_token=strides[1], stride_head=strides[2],
                   budget_ppm=ppm, sm_scale=1.0 / math.sqrt(sh["d"]), n_sink=n_sink,
                   n_local=n_local)
    assert set(res) == {(b, h) for b in range(sh["B"]) for h in range(sh["Hq"])}
    for b in range(sh["B"]):
        n = int(a["seq_lens"][b])
        for h in range(sh["Hq"]):
            g = h // sh["G"]
            y_bf, T_bf, _ = brute_force(a["q"][b, h], a["centroids"][b, g], a["codebooks"][b, g],
                                        a["codes"][b, g, :n], a["list_ids"][b, g, :n],
                                        a["key_norms"][b, g, :n], a["list_vmeans"][b, g],
                                        K[b, g, :n], V[b, g, :n], ppm, n_sink, n_local)
            assert sorted(res[(b, h)]["T"].tolist()) == T_bf
            np.testing.assert_allclose(res[(b, h)]["y"], y_bf, rtol=1e-11, atol=1e-13)
    # the two query heads of a group see the same keys but are different rows
    assert not np.allclose(res[(0, 0)]["y"], res[(0, 1)]["y"])


def test_decode_head_restriction_keeps_absolute_head_numbers():
    rng = np.random.default_rng(22)
    a, strides, K, V, sh = _paged_case(rng, "split")
    kw = dict(n_kv_heads=sh["Hkv"], page_size=sh["P"], stride_page=strides[0],
              stride_token=strides[1], stride_head=strides[2], budget_ppm=250000,
              sm_scale=0.5)
    args = (a["q"], a["centroids"], a["codebooks"], a["codes"], a["list_ids"], a["key_norms"],
            a["list_vmeans"], a["k_cache_flat"], a["v_cache_flat"], a["block_table"], a["seq_lens"])
    full = O.decode(*args, **kw)
    part = O.decode(*args, heads=[3], batch_items=[1], **kw)
    assert list(part) == [(1, 3)]
    np.testing.assert_array_equal(part[(1, 3)]["y"], full[(1, 3)]["y"])


# ----------------------------------------------------------------------------- page-rounded budget inside decode_head
@pytest.mark.parametrize("ppm,k_want,tokens", [(10000, 1324, 1456), (20000, 2620, 2752)])
def test_decode_head_selects_the_page_rounded_budget_at_128k(ppm, k_want, tokens):
    """App. A, "Budgets": 4 sinks + 128 window tokens + ceil(rho |R|) retrieved tokens, rounded up
    to pages of 16, are 1,456 / 2,752 tokens at 131,072; decode_head must select exactly the
    difference (1,324 / 2,620) and report the k-th largest approximate logit."""
    rng = np.random.default_rng(31)
    n, d = 131072, 2
    cen = np.zeros((1, d))
    cb = rng.normal(size=(1, 256, d))                         # one subspace: the score is LUT[z_i]
    codes = rng.integers(0, 256, (n, 1)).astype(np.uint8)
    ids = np.zeros(n, dtype=np.uint16)
    norms = rng.uniform(0.5, 2.0, n)
    q = np.array([0.7, -1.1])
    zeros = lambda pos: np.zeros((len(pos), d))
    r = O.decode_head(q, cen, cb, codes, ids, norms, np.zeros((1, d)), zeros, zeros, n, ppm,
                      1.0, n_sink=4, n_local=128, round_exact_set_to_page=16)
    assert r["k"] == k_want and len(r["T"]) == k_want and len(r["E"]) == tokens
    assert len(r["R"]) == 130940 and r["T"].min() >= 4 and r["T"].max() < 131072 - 128
    want = norms[4:n - 128] * (cb[0][codes[4:n - 128, 0]] @ q)       # Eq. 2 with one subspace, c = 0
    np.testing.assert_allclose(r["approx"], want, rtol=1e-12, atol=1e-14)
    assert r["kth_score"] == np.sort(r["approx"])[-k_want]
    assert np.all(r["approx"][r["T"] - 4] >= r["kth_score"])
    # without rounding the same call takes ceil(rho |R|)
    r0 = O.decode_head(q, cen, cb, codes, ids, norms, np.zeros((1, d)), zeros, zeros, n, ppm,
                       1.0, n_sink=4, n_local=128)
    assert r0["k"] == -(-130940 * ppm // 1_000_000)


# ----------------------------------------------------------------------------- window = not yet indexed
def test_indexed_len_sets_the_window():
    """Sec. 3.3: tokens written since the last index update stay in the exactly-attended window.
    partition(indexed_len=r) is the partition with a window of seq_len - r tokens."""
    for n, n_sink, r_end in [(100, 4, 60), (100, 4, 100), (100, 4, 2), (5, 8, 3), (50, 0, 0)]:
        S, L, R = O.partition(n, n_sink, 0, indexed_len=r_end)
        S2, L2, R2 = O.partition(n, n_sink, max(0, n - max(r_end, min(n_sink, n))))
        assert S.tolist() == S2.tolist() and L.tolist() == L2.tolist() and R.tolist() == R2.tolist()
        assert sorted(S.tolist() + L.tolist() + R.tolist()) == list(range(n))
    rng = np.random.default_rng(41)
    n, d, n_list, M, n_code = 40, 4, 3, 2, 4
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    K, V, q = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=d)
    vmeans = rng.normal(size=(n_list, d))
    a = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 200000, n_sink=2, indexed_len=29)
    y_bf, T_bf, _ = brute_force(q, cen, cb, codes, ids, norms, vmeans, K, V, 200000, 2, n - 29)
    assert sorted(a["T"].tolist()) == T_bf and a["E"].tolist()[:13] == [0, 1] + list(range(29, 40))
    np.testing.assert_allclose(a["y"], y_bf, rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------------- mechanism variants (Table 2, App. B)
def brute_force_variant(variant, q, cen, cb, codes, ids, norms, vmeans, K, V, ppm):
    """Scalar loops for the variants of Table 2 (no sinks, no window), from their definitions."""
    n, d = K.shape
    M, n_code, dsub = cb.shape
    n_list = len(vmeans)
    rq = math.sqrt(sum(float(x) ** 2 for x in q))
    approx = []
    for i in range(n):
        acc = sum(float(q[t]) / rq * cen[ids[i]][t] for t in range(d))
        for m in range(M):
            acc += sum(float(q[m * dsub + t]) / rq * cb[m][codes[i][m]][t] for t in range(dsub))
        approx.append(rq * norms[i] / math.sqrt(d) * acc)
    k = min(n, -(-n * ppm // 1_000_000))
    T = sorted(range(n), key=lambda i: (-approx[i], i))[:k]
    Bset = [i for i in range(n) if i not in set(T)]
    exact = {i: sum(float(q[t]) * K[i][t] for t in range(d)) / math.sqrt(d) for i in T}
    count = [sum(1 for i in range(n) if ids[i] == j) for j in range(n_list)]
    v_global = [sum(count[j] * vmeans[j][t] for j in range(n_list)) / n for t in range(d)]
    if variant == "T" or (variant in ("C2", "C2b") and not T):
        bg_logit = {i: -math.inf for i in Bset}
    elif variant == "C2":
        bg_logit = {i: sum(approx[t] for t in T) / len(T) for i in Bset}
    elif variant == "C2b":
        bg_logit = {i: min(exact.values()) for i in Bset}
    else:
        bg_logit = {i: approx[i] for i in Bset}
    m0 = max(list(exact.values()) + list(bg_logit.values()))
    if m0 == -math.inf:           # nothing attended (k = 0 and no background): defined as zero
        return np.zeros(d)
    num, den = [0.0] * d, 0.0
    for i in T:
        e = math.exp(exact[i] - m0)
        den += e
        for t in range(d):
            num[t] += e * V[i][t]
    for i in Bset:
        e = math.exp(bg_logit[i] - m0)
        if e == 0.0:
            continue
        j = ids[i]
        if variant == "B":
            val = vmeans[j]
        elif variant == "Bx":     # mean of the list's unselected members, from the stored mean
            t_in = [s for s in T if ids[s] == j]
            val = [(count[j] * vmeans[j][t] - sum(V[s][t] for s in t_in)) / (count[j] - len(t_in))
                   for t in range(d)]
        else:
            val = v_global
        den += e
        for t in range(d):
            num[t] += e * val[t]
    return np.array(num) / den


@pytest.mark.parametrize("variant", ["B", "T", "Bx", "C", "C2", "C2b"])
@pytest.mark.parametrize("seed,n,ppm", [(0, 40, 150000), (1, 23, 50000), (2, 12, 0)])
def test_variants_against_scalar_loops(variant, seed, n, ppm):
    rng = np.random.default_rng(100 + seed)
    d, n_list, M, n_code = 4, 3, 2, 4
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    K, V, q = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=d)
    vmeans = list_means(V, ids, n_list) + rng.normal(size=(n_list, d)) * 0.05   # stored, not exact
    got = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, ppm, variant=variant)
    want = brute_force_variant(variant, q, cen, cb, codes, ids, norms, vmeans, K, V, ppm)
    np.testing.assert_allclose(got["y"], want, rtol=1e-10, atol=1e-12)


def test_variant_closed_forms():
    """Hand-checkable instances.  One list, four identical keys (all logits equal, exact codes),
    scalar values 1, 2, 3, 4 in every dim, k = 1 (the stable rule selects position 0):
      B   (1 + 3 * 2.5) / 4 = 2.125      the stored mean counts the selected member
      Bx  (1 + 3 * 3.0) / 4 = 2.5        mean of the unselected members (2 + 3 + 4) / 3
      C   one list, so the global mean is the list mean: 2.125
      C2, C2b  shared logit = the common logit, global mean 2.5: 2.125
      T   the selected token alone: 1"""
    d, n = 4, 4
    cen = np.array([[0.5, 0.0, 0.0, 0.0]])
    cb = np.zeros((2, 4, 2))
    codes = np.zeros((n, 2), dtype=np.uint8)
    ids = np.zeros(n, dtype=np.int64)
    norms = np.full(n, 2.0)
    K = np.tile(2.0 * cen, (n, 1))
    V = np.arange(1.0, 5.0)[:, None] * np.ones((1, d))
    q = np.array([1.0, 0.0, 0.0, 0.0])
    vmeans = V.mean(axis=0, keepdims=True)
    want = dict(B=2.125, Bx=2.5, C=2.125, C2=2.125, C2b=2.125, T=1.0)
    for variant, y in want.items():
        r = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 250000, variant=variant)
        assert r["T"].tolist() == [0]
        np.testing.assert_allclose(r["y"], np.full(d, y), rtol=1e-13)


def test_variant_relations():
    """T equals textbook attention over the exact set alone; Bx equals B when the values are
    constant inside every list; C equals B when every list stores the same mean; C2b with
    rho = 1 has no background left and is dense attention."""
    rng = np.random.default_rng(7)
    n, d, n_list, M, n_code = 60, 8, 4, 2, 8
    cen, cb, codes, ids, norms, _ = random_index(rng, n, d, n_list, M, n_code)
    K, V, q = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=d)
    vmeans = list_means(V, ids, n_list)
    t = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 100000, n_sink=2, n_local=3, variant="T")
    np.testing.assert_allclose(t["y"], dense_attention(q, K[t["E"]], V[t["E"]], 1 / math.sqrt(d)),
                               rtol=1e-12)
    assert t["Z_B"] == 0.0
    Vc = vmeans[ids]                                          # constant inside each list
    b = run_head(q, cen, cb, codes, ids, norms, vmeans, K, Vc, 100000, variant="B")
    bx = run_head(q, cen, cb, codes, ids, norms, vmeans, K, Vc, 100000, variant="Bx")
    np.testing.assert_allclose(bx["y"], b["y"], rtol=1e-10)
    same = np.tile(rng.normal(size=(1, d)), (n_list, 1))
    b = run_head(q, cen, cb, codes, ids, norms, same, K, V, 100000, variant="B")
    c = run_head(q, cen, cb, codes, ids, norms, same, K, V, 100000, variant="C")
    np.testing.assert_allclose(c["y"], b["y"], rtol=1e-12)
    full = run_head(q, cen, cb, codes, ids, norms, vmeans, K, V, 1000000, variant="C2b")
    np.testing.assert_allclose(full["y"], dense_attention(q, K, V, 1 / math.sqrt(d)), rtol=1e-12)
