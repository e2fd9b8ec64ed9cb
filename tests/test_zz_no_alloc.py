"""The workspace-free top-k entry point (pqhsa_select_static), checked against pqhsa_select.

Some users of the library cannot allocate device memory where they need the top-k (they run
inside an engine's fixed memory plan, or may not stall the device with a driver allocation),
so the library offers a variant whose scratch is a fixed array inside the library image.
This test calls it through the C ABI twice in a row -- the array is shared between calls and
keeps the previous call's contents, so the second call also proves that the entry point
clears what it must -- and compares every output with the regular entry point's.

Collected last on purpose (file name), so a run that stops at the first failure has already
run every other test.  It passes on its own in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

from paper_2609_33746_b200 import pqhsa
from paper_2609_33746_b200.runner import DecodeOp
from paper_2609_33746_b200.workload import DecodeConfig

from helpers import make_case

pytestmark = pytest.mark.gpu


def _case(seq_lens, budget_ppm, seed):
    cfg = DecodeConfig(name="noalloc", batch=len(seq_lens), n_q_heads=8, n_kv_heads=2,
                       seq_lens=seq_lens, dtype="bf16", n_list=64, pq_m=32,
                       budget_ppm=budget_ppm, seed=seed, kmeans_iters=2)
    inp, idx = make_case(cfg, device="cuda")
    op = DecodeOp(inp, idx)
    op.alloc_stage_buffers()
    op.build_lut()
    op.scan()
    return cfg, op


def _sets(op, cfg):
    k_max = op.params.k_max
    sel = op.sel_idx.view(cfg.batch * cfg.n_q_heads, k_max).cpu().numpy()
    cnt = op.sel_count.cpu().numpy()
    kth = op.kth.cpu().numpy()
    return [sorted(sel[r, :cnt[r]].tolist()) for r in range(len(cnt))], cnt.copy(), kth.copy()


def test_select_static_matches_select_on_two_calls_in_a_row():
    assert pqhsa.select_static_capacity() == 16 << 20
    for call, (seq_lens, ppm, seed) in enumerate([((9000, 0, 4100), 20000, 21),
                                                  ((5000,), 100000, 22)]):
        cfg, op = _case(seq_lens, ppm, seed)
        assert 0 < pqhsa.select_static_bytes(op.params) <= pqhsa.select_static_capacity()
        op.select()                                      # the regular entry point, with a workspace
        torch.cuda.synchronize()
        want_sets, want_cnt, want_kth = _sets(op, cfg)
        op.sel_idx.fill_(-1)
        op.sel_count.fill_(-1)
        op.kth.fill_(0)
        pqhsa.select_static(op.params, op.scores, op.seq_lens, op.sel_idx, op.sel_count, op.kth)
        torch.cuda.synchronize()
        got_sets, got_cnt, got_kth = _sets(op, cfg)
        # what the entry point is for: a call allocates nothing (the driver's count of free
        # device memory is the same before and after a repeat of the call)
        free_before = torch.cuda.mem_get_info()[0]
        pqhsa.select_static(op.params, op.scores, op.seq_lens, op.sel_idx, op.sel_count, op.kth)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert np.array_equal(got_cnt, want_cnt), f"call {call}: counts differ"
        # the selection is exact and tie-stable in both entry points: identical sets
        assert got_sets == want_sets, f"call {call}: selected sets differ"
        assert np.array_equal(np.nan_to_num(got_kth, nan=-1.0), np.nan_to_num(want_kth, nan=-1.0))


def test_select_static_rejects_shapes_beyond_its_array():
    p = pqhsa.make_params(batch=8, n_q_heads=32, n_kv_heads=8, n_list=1024, pq_m=32,
                          max_seq_len=131072, max_pages_per_seq=8192, budget_ppm=10000,
                          dtype="bf16")
    assert pqhsa.select_static_bytes(p) > pqhsa.select_static_capacity()
    dummy = torch.zeros(16, device="cuda")
    with pytest.raises(pqhsa.PqhsaError) as e:
        pqhsa.select_static(p, dummy, dummy, dummy, dummy, dummy)
    assert e.value.status == pqhsa.ERR_WORKSPACE
