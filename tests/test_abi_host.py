"""CPU-only checks of the C-ABI boundary: the shared library loads, exports every function
that include/pqhsa.h declares, and its host-side argument validation and size arithmetic
work without a GPU (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

from paper_2609_33746_b200 import pqhsa
from paper_2609_33746_b200.build import LIB, build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build_library()
    assert os.path.exists(LIB)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pqhsa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pqhsa_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 14 and "pqhsa_decode" in names
    handle = ctypes.CDLL(LIB)
    for n in names:
        assert hasattr(handle, n), f"{n} declared in pqhsa.h but not exported"
    assert sorted(pqhsa.EXPORTS) == sorted(n for n in names)


def params(**kw):
    base = dict(batch=1, n_q_heads=32, n_kv_heads=8, n_list=1024, pq_m=32, max_seq_len=131072,
                max_pages_per_seq=8192, budget_ppm=10000, dtype="bf16")
    base.update(kw)
    return pqhsa.make_params(**base)


def test_size_arithmetic_for_the_128k_workload():
    p = params()
    assert p.k_max == 1311 and p.pq_dsub == 4
    assert pqhsa.heads_per_group(p) == 4
    n_part = pqhsa.num_partials(p)
    assert n_part >= 3
    assert pqhsa.buffer_elems(p, pqhsa.BUF_LUT) == 8 * 256 * 32 * 4
    assert pqhsa.buffer_elems(p, pqhsa.BUF_COARSE) == 8 * 1024 * 4
    assert pqhsa.buffer_elems(p, pqhsa.BUF_SCORES) == 32 * 131072
    assert pqhsa.buffer_elems(p, pqhsa.BUF_LIST_PARTIALS) == 8 * n_part * 4 * (1024 + 2)
    assert pqhsa.buffer_elems(p, pqhsa.BUF_SEL_IDX) == 32 * 1311
    ws = pqhsa.workspace_bytes(p)
    assert ws > 4 * 32 * 131072 and ws % 256 == 0
    offs = [pqhsa.decode_buffer_offset(p, w) for w in range(7)]
    assert offs == sorted(offs) and all(o % 256 == 0 for o in offs) and offs[-1] < ws
    assert pqhsa.decode_launch_count(p) > 0


def test_group_of_eight_is_two_head_groups_and_padded_groups():
    assert pqhsa.heads_per_group(params(n_kv_heads=4)) == 4          # G = 8 -> 2 groups of 4
    p = params(n_q_heads=40, n_kv_heads=8)                           # G = 5 -> padded to 8 slots
    assert pqhsa.heads_per_group(p) == 4
    assert pqhsa.buffer_elems(p, pqhsa.BUF_LUT) == 8 * 2 * 256 * 32 * 4
    assert pqhsa.heads_per_group(params(n_q_heads=8, n_kv_heads=8)) == 1


@pytest.mark.parametrize("kw,status", [
    (dict(n_sink=-1), pqhsa.ERR_INVALID_ARG),
    (dict(n_local=-5), pqhsa.ERR_INVALID_ARG),
    (dict(exact_set_multiple=16, k_max=1311), pqhsa.ERR_INVALID_ARG),   # no room for the rounding
    (dict(head_dim=64, pq_m=16), pqhsa.ERR_UNSUPPORTED),
    (dict(pq_m=4), pqhsa.ERR_UNSUPPORTED),
    (dict(pq_ncode=16, pq_m=32), pqhsa.ERR_UNSUPPORTED),  # 4-bit codes: 8 or 16 subspaces
    (dict(pq_ncode=64), pqhsa.ERR_UNSUPPORTED),
    (dict(n_list=8192), pqhsa.ERR_UNSUPPORTED),
    (dict(max_seq_len=131070), pqhsa.ERR_UNSUPPORTED),
    (dict(n_q_heads=30), pqhsa.ERR_INVALID_ARG),          # not a multiple of n_kv_heads
    (dict(budget_ppm=2_000_000, k_max=10), pqhsa.ERR_INVALID_ARG),
    (dict(k_max=5), pqhsa.ERR_INVALID_ARG),               # smaller than ceil(N_max * rho)
    (dict(max_pages_per_seq=10), pqhsa.ERR_INVALID_ARG),
    (dict(batch=0), pqhsa.ERR_INVALID_ARG),
])
def test_invalid_shapes_are_rejected_on_the_host(kw, status):
    p = params(**kw)
    with pytest.raises(pqhsa.PqhsaError) as e:
        pqhsa.heads_per_group(p)
    assert e.value.status == status
    assert pqhsa.workspace_bytes(p) == 0


def test_status_strings():
    assert pqhsa.status_string(0) == "ok"
    assert "workspace" in pqhsa.status_string(pqhsa.ERR_WORKSPACE)
    assert pqhsa.status_string(-99) == "unknown status"


def test_debug_check_predicates_on_the_host():
    """The predicates behind the -DPQHSA_DEBUG index checks (list id, selected position, page id),
    exercised on the host: the GPU is never fed a bad index on purpose."""
    P = pqhsa.debug_predicate
    assert [P(0, v, 0, 64) for v in (0, 63, 64, 65535, -1)] == [1, 1, 0, 0, 0]          # list id < n_list
    assert [P(1, v, 4, 100) for v in (3, 4, 99, 100, -7)] == [0, 1, 1, 0, 0]            # r_begin <= pos < r_end
    assert [P(2, v, 0, 0) for v in (0, 12345, -1)] == [1, 1, 0]                         # page id >= 0
    assert P(9, 0, 0, 0) == -1
    assert pqhsa.debug_build() in (False, True)
