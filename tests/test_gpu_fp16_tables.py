"""The opt-in fp16-table modes of the scan (pqhsa_params.table_precision = PQHSA_TABLES_FP16 and
PQHSA_TABLES_FP16_RESCORE), -m gpu.

In this mode the approximate logits carry the rounding of fp16 table entries, so the scan stage is
NOT held to the 1e-4 logit tolerance.  What is checked instead, against the float64 oracle on the
same inputs:
  * every approximate logit is within the bound that the arithmetic gives: r_i * sum_m |entry| * 2^-9
    (entry rounding 2^-11 plus two levels of fp16 additions), far inside it on average;
  * the top-k is exact ON THE DEVICE'S SCORES (checked against a sort of those scores), and differs
    from the oracle's set only by tokens whose oracle logit is within that bound of the k-th score;
  * the output is within the usual tolerance of the oracle's hybrid output for the DEVICE's
    selection (the oracle's Eq. 4-5 evaluated with the device's set), and close to the oracle's own.
"""
import math

import numpy as np
import pytest
import torch

from oracle import pqhsa_oracle as O
from paper_2609_33746_b200 import pqhsa
from paper_2609_33746_b200.runner import DecodeOp

from helpers import make_case, oracle_arrays, run_oracle, selection_matches
from test_gpu_parity import LOGIT_RTOL, OUT_ATOL, out_tolerance, small

pytestmark = pytest.mark.gpu

CASES = {
    "g4": small("h_g4", seq_lens=(5000,)),
    "g8_ragged_sinks_window": small("h_g8", batch=3, n_q_heads=16, n_kv_heads=2, seq_lens=(3001, 0, 900),
                                    n_sink=4, n_local=64),
    "g3_padded_fp16_cache": small("h_g3", n_q_heads=6, n_kv_heads=2, seq_lens=(2777,), dtype="fp16"),
    "many_lists": small("h_l", seq_lens=(6000,), n_list=1024, n_q_heads=4, n_kv_heads=1, kmeans_iters=2),
}
FP32_TIE = 2e-5     # two scores this close (relative to max(1, |s_k|)) may swap between fp32 and fp64
# long enough for the threshold zone to hold tokens that the fp16 tables rank differently
LONG = small("h_long", seq_lens=(60000, 41000), batch=2, n_q_heads=8, n_kv_heads=2, n_list=256,
             budget_ppm=20000, kmeans_iters=1)


@pytest.mark.parametrize("key", list(CASES))
def test_fp16_tables_scores_selection_and_output(key):
    cfg = CASES[key]
    inp, idx = make_case(cfg, device="cuda")
    arrays = oracle_arrays(inp, idx)
    ref = run_oracle(inp, idx, arrays=arrays)
    op = DecodeOp(inp, idx, fp16_tables=True)
    op.alloc_stage_buffers()
    op.build_lut(); op.scan(); op.select()
    op.out_f32.fill_(5.0)
    op.hybrid_attend()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK
    N_max, k_max = op.params.max_seq_len, op.params.k_max
    scores = op.scores.view(cfg.batch, cfg.n_q_heads, N_max).cpu().double().numpy()
    sel = op.sel_idx.view(cfg.batch, cfg.n_q_heads, k_max).cpu().numpy()
    cnt = op.sel_count.view(cfg.batch, cfg.n_q_heads).cpu().numpy()
    y32 = op.out_f32.cpu().double().numpy()
    worst_ratio, mean_err = 0.0, []
    for (b, h), r in ref.items():
        R = r["R"]
        if len(R) == 0:
            continue
        r0, r1 = int(R[0]), int(R[-1]) + 1
        g = h // cfg.group
        got = scores[b, h, r0:r1]
        # the bound of the arithmetic, per token: |entries| looked up, times 2^-9, times r_q r_i / sqrt(d)
        codes = arrays["codes"][b, g, r0:r1].astype(np.int64)
        mag = np.abs(r["coarse"][arrays["list_ids"][b, g, r0:r1].astype(np.int64)]) * 0.0
        for m in range(cfg.pq_m):
            mag = mag + np.abs(r["lut"][m][codes[:, m]])
        bound = (r["r_q"] * arrays["key_norms"][b, g, r0:r1] / math.sqrt(128.0)) * mag * 2.0 ** -9 + 1e-4
        err = np.abs(got - r["approx"])
        assert np.all(err <= bound), f"{(b, h)}: {np.max(err / bound)} of the bound"
        worst_ratio = max(worst_ratio, float(np.max(err / bound)))
        mean_err.append(float(err.mean()))
        # exact top-k of the device's own scores (ties: lower position)
        k = r["k"]
        assert cnt[b, h] == k
        mine = sorted(sel[b, h, :k].tolist())
        want = (O.select_topk(got, k) + r0).tolist()
        assert mine == want
        # against the oracle's set: only tokens within the bound of the k-th score may differ
        if k:
            diff = set(mine) ^ set(int(x) for x in r["T"])
            for i in diff:
                assert abs(r["approx"][i - r0] - r["kth_score"]) <= 2 * bound[i - r0] + 1e-3
        # output: the oracle's Eq. 4-5 with the device's selection and the device's approximate
        # logits for the background
        S, L, _ = O.partition(int(arrays["seq_lens"][b]), cfg.n_sink, cfg.n_local)
        E = np.concatenate([S, L, np.array(mine, dtype=np.int64)])
        mask = np.ones(r1 - r0, dtype=bool)
        mask[np.array(mine, dtype=np.int64) - r0] = False
        keys = O.gather_rows(arrays["k_cache_flat"], arrays["block_table"][b], E, g, 128, cfg.page_size,
                             inp.stride_page, inp.stride_token, inp.stride_head)
        vals = O.gather_rows(arrays["v_cache_flat"], arrays["block_table"][b], E, g, 128, cfg.page_size,
                             inp.stride_page, inp.stride_token, inp.stride_head)
        y_dev_sel, _ = O.hybrid_output(arrays["q"][b, h], keys, vals, got[mask],
                                       arrays["list_ids"][b, g, r0:r1][mask], arrays["list_vmeans"][b, g],
                                       1.0 / math.sqrt(128.0))
        assert np.abs(y32[b, h] - y_dev_sel).max() <= OUT_ATOL
        assert np.abs(y32[b, h] - r["y"]).max() <= 5 * OUT_ATOL     # and near the fp32-table result
    assert worst_ratio <= 1.0 and np.mean(mean_err) > 1e-6          # approximate, inside its bound


@pytest.mark.parametrize("key", list(CASES) + ["long"])
def test_fp16_tables_with_rescore_select_what_fp32_tables_select(key):
    """With the fp32 re-score of the threshold zone the selected set is the oracle's up to ties at
    the level of fp32 rounding (2e-5 relative, far below the fp16 tables' error), the k-th score is
    the fp32 one, and the output meets the usual tolerance against the oracle's output; the fused
    call gives the staged calls' result."""
    cfg = LONG if key == "long" else CASES[key]
    inp, idx = make_case(cfg, device="cuda")
    arrays = oracle_arrays(inp, idx)
    ref = run_oracle(inp, idx, arrays=arrays)
    plain = DecodeOp(inp, idx, fp16_tables=True)
    plain.alloc_stage_buffers()
    plain.build_lut(); plain.scan(); plain.select()
    op = DecodeOp(inp, idx, fp16_tables="rescore")
    op.alloc_stage_buffers()
    op.build_lut(); op.scan()
    op.sel_idx.fill_(-1)
    op.select()                                   # top-k on the fp16-table scores, then the re-score
    op.out_f32.fill_(5.0)
    op.hybrid_attend()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK
    assert pqhsa.decode_launch_count(op.params) == pqhsa.decode_launch_count(plain.params) + 1
    k_max = op.params.k_max
    sel = op.sel_idx.view(cfg.batch, cfg.n_q_heads, k_max).cpu().numpy()
    sel_plain = plain.sel_idx.view(cfg.batch, cfg.n_q_heads, k_max).cpu().numpy()
    cnt = op.sel_count.view(cfg.batch, cfg.n_q_heads).cpu().numpy()
    kth = op.kth.view(cfg.batch, cfg.n_q_heads).cpu().numpy()
    y32 = op.out_f32.cpu().double().numpy()
    moved, plain_off = 0, 0
    for (b, h), r in ref.items():
        k = r["k"]
        assert cnt[b, h] == k
        ok, why = selection_matches(sel[b, h, :k], r, tol=FP32_TIE)
        assert ok, f"{(b, h)}: {why}"
        moved += len(set(sel[b, h, :k].tolist()) ^ set(sel_plain[b, h, :k].tolist()))
        plain_off += 0 if selection_matches(sel_plain[b, h, :k], r, tol=FP32_TIE)[0] else 1
        if k:
            assert abs(kth[b, h] - r["kth_score"]) <= LOGIT_RTOL * max(1.0, abs(r["kth_score"]))
        assert np.abs(y32[b, h] - r["y"]).max() <= OUT_ATOL
    print(f"{key}: the re-score moved {moved} positions; rows where the fp16 tables alone miss: {plain_off}")
    if key == "long":
        assert moved > 0 and plain_off > 0        # the case does exercise the re-score
    op.out.zero_()
    op.decode()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK
    fused_sel = op.decode_buffer(pqhsa.BUF_SEL_IDX, torch.int32).view(cfg.batch, cfg.n_q_heads, k_max).cpu().numpy()
    for (b, h), r in ref.items():
        assert sorted(fused_sel[b, h, :r["k"]].tolist()) == sorted(sel[b, h, :r["k"]].tolist())
    fused = op.out.cpu().double().numpy()
    for (b, h), r in ref.items():
        assert np.all(np.abs(fused[b, h] - r["y"]) <= out_tolerance(r["y"], cfg.dtype))


@pytest.mark.parametrize("factor", [20.0, 60.0, 150.0, 400.0, 3000.0])
def test_rescore_with_one_huge_key_norm(factor):
    """The error bound of a row scales with the largest key norm in it.  One token with a norm
    `factor` times the others' widens every row's threshold zone by that factor: first the zone
    still lies inside the top-k's candidate list, then it reaches below the list and is read off
    the score row, and finally it holds more tokens than the kernel's pool.  As long as the status
    word stays clear the re-score must land on the oracle's set; once a row reports that it was
    skipped (bit 64) it must have KEPT the exact top-k of the fp16-table scores -- nothing is
    dropped or duplicated either way."""
    cfg = small("h_norm", seq_lens=(30000,), n_q_heads=4, n_kv_heads=1, n_list=256,
                budget_ppm=20000, kmeans_iters=1)
    inp, idx = make_case(cfg, device="cuda")
    idx.key_norms[0, 0, 777] *= factor
    arrays = oracle_arrays(inp, idx)
    ref = run_oracle(inp, idx, arrays=arrays)
    op = DecodeOp(inp, idx, fp16_tables="rescore")
    op.alloc_stage_buffers()
    op.build_lut(); op.scan(); op.select()
    torch.cuda.synchronize()
    k_max = op.params.k_max
    sel = op.sel_idx.view(cfg.batch, cfg.n_q_heads, k_max).cpu().numpy()
    scores = op.scores.view(cfg.batch, cfg.n_q_heads, -1).cpu().double().numpy()
    status = op.device_status()
    assert status in (pqhsa.OK, pqhsa.ERR_DEVICE_CHECK)
    if factor <= 20.0:
        assert status == pqhsa.OK
    if factor >= 3000.0:
        assert status == pqhsa.ERR_DEVICE_CHECK
    for (b, h), r in ref.items():
        k = r["k"]
        assert len(set(sel[b, h, :k].tolist())) == k
        r0, r1 = int(r["R"][0]), int(r["R"][-1]) + 1
        approx_topk = (O.select_topk(scores[b, h, r0:r1], k) + r0).tolist()
        exact_ok, why = selection_matches(sel[b, h, :k], r, tol=FP32_TIE)
        if status == pqhsa.OK:
            assert exact_ok, f"{(b, h)}: {why}"
        else:       # some row was skipped: every row is either re-scored or untouched
            assert exact_ok or sorted(sel[b, h, :k].tolist()) == approx_topk, f"{(b, h)}: {why}"


def test_rescore_entry_point_is_refused_without_the_mode():
    cfg = small("h_plain", seq_lens=(1000,))
    inp, idx = make_case(cfg, device="cuda")
    op = DecodeOp(inp, idx, fp16_tables=True)
    op.alloc_stage_buffers()
    with pytest.raises(pqhsa.PqhsaError) as e:
        pqhsa.rescore(op.params, op.index, op.lut, op.coarse, op.scores, op.seq_lens, op.sel_idx,
                      op.sel_count, op.kth, op.ws)
    assert e.value.status == pqhsa.ERR_INVALID_ARG


def test_fp16_tables_are_refused_outside_the_supported_shape():
    cfg = small("h_m16", pq_m=16, n_q_heads=4, n_kv_heads=1, seq_lens=(1000,))
    inp, idx = make_case(cfg, device="cuda")
    op = DecodeOp(inp, idx, fp16_tables=True)
    with pytest.raises(pqhsa.PqhsaError) as e:
        op.decode()
    assert e.value.status == pqhsa.ERR_UNSUPPORTED
