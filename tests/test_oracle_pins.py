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
