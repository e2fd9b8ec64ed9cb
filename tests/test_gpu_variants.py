"""The mechanism variants of the paper's ablation (Table 2; App. B) and the per-sequence window
(Sec. 3.3) on the device, against the float64 oracle (-m gpu).

The variants share selector, budget and exact part and differ only in the background term, so
each case runs the first three stages once and the hybrid attention once per variant."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from paper_2609_33746_b200 import pqhsa
from paper_2609_33746_b200.runner import DecodeOp

from helpers import make_case, oracle_arrays, run_oracle, selection_matches
from test_gpu_parity import OUT_ATOL, LOGIT_RTOL, out_tolerance, small

pytestmark = pytest.mark.gpu

VARIANT_CASES = {
    "bf16_g4": small("v_g4", seq_lens=(5000,)),
    "sinks_window_ragged": small("v_swr", batch=3, seq_lens=(3000, 0, 1200), n_q_heads=4, n_kv_heads=1,
                                 n_sink=4, n_local=128, exact_set_multiple=16),
    "g8_fp16": small("v_g8", n_q_heads=16, n_kv_heads=2, seq_lens=(2500,), dtype="fp16"),
    "many_lists_few_members": small("v_l", seq_lens=(3000,), n_list=1024, n_q_heads=4, n_kv_heads=1,
                                    kmeans_iters=2, budget_ppm=100000),
    "four_bit_paper_index": small("v_p4", pq_m=8, pq_ncode=16, n_list=512, seq_lens=(6000,), n_sink=4,
                                  n_local=128, exact_set_multiple=16, kmeans_iters=2),
}
_cache = {}


def staged_case(key):
    if key not in _cache:
        inp, idx = make_case(VARIANT_CASES[key], device="cuda")
        arrays = oracle_arrays(inp, idx)
        _cache[key] = (inp, idx, arrays)
    return _cache[key]


@pytest.mark.parametrize("variant", ["B", "T", "Bx", "C", "C2", "C2b"])
@pytest.mark.parametrize("key", list(VARIANT_CASES))
def test_variant_outputs_match_the_oracle(key, variant):
    inp, idx, arrays = staged_case(key)
    cfg = inp.cfg
    ref = run_oracle(inp, idx, arrays=arrays, variant=variant)
    op = DecodeOp(inp, idx, variant=variant)
    op.alloc_stage_buffers()
    op.build_lut(); op.scan(); op.select()
    op.out.fill_(9.0)
    op.out_f32.fill_(9.0)
    op.hybrid_attend()
    torch.cuda.synchronize()
    y32 = op.out_f32.cpu().double().numpy()
    lse = op.lse.view(cfg.batch, cfg.n_q_heads).cpu().numpy()
    op.out.fill_(-9.0)
    op.decode()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK
    fused = op.out.cpu().double().numpy()
    assert pqhsa.decode_launch_count(op.params) == (7 if variant == "Bx" else 6)
    for (b, h), r in ref.items():
        err = np.abs(y32[b, h] - r["y"])
        assert err.max() <= OUT_ATOL, f"{variant} fp32 output {(b, h)}: max-abs {err.max()}"
        assert np.all(np.abs(fused[b, h] - r["y"]) <= out_tolerance(r["y"], cfg.dtype)), \
            f"{variant} fused output {(b, h)}"
        if "lse" in r:
            assert abs(lse[b, h] - r["lse"]) <= 2e-3 * max(1.0, abs(r["lse"]))


def test_variants_that_need_list_counts_reject_an_index_without_them():
    inp, idx, arrays = staged_case("bf16_g4")
    op = DecodeOp(inp, idx, variant="C")
    bare = pqhsa.make_index(op.centroids, op.codebooks, op.codes, op.list_ids, op.key_norms,
                            op.list_vmeans)
    with pytest.raises(pqhsa.PqhsaError) as e:
        pqhsa.decode(op.params, op.q, bare, op.kv, op.seq_lens, op.out, op.ws)
    assert e.value.status == pqhsa.ERR_INVALID_ARG


def test_background_term_beats_truncation_on_most_rows():
    """App. B reports the ordering err(B) < err(T) against full attention on almost every row.
    Sanity only (synthetic keys): against the library's own dense kernel, B is closer than T on
    most rows."""
    inp, idx, arrays = staged_case("bf16_g4")
    cfg = inp.cfg
    outs = {}
    for variant in ("B", "T"):
        op = DecodeOp(inp, idx, variant=variant)
        op.decode()
        torch.cuda.synchronize()
        outs[variant] = op.out.float().clone()
    ws = torch.empty(pqhsa.dense_workspace_bytes(op.params), dtype=torch.uint8, device="cuda")
    dense = torch.empty_like(op.q)
    pqhsa.dense_decode(op.params, op.q, op.kv, op.seq_lens, dense, ws)
    torch.cuda.synchronize()
    err = {v: (outs[v] - dense.float()).norm(dim=-1) for v in outs}
    # (the synthetic queries attend a few keys sharply: on many rows both errors are zero)
    assert (err["B"] <= err["T"] + 1e-6).float().mean().item() >= 0.75
    assert (err["B"] < err["T"]).sum().item() >= (err["T"] < err["B"]).sum().item()


# ----------------------------------------------------------------------------- per-sequence window
def _garble_unindexed(inp, idx):
    """What lies behind the indexed region was never encoded: make sure nobody relies on it."""
    for b, covered in enumerate(inp.cfg.indexed_lens):
        idx.codes[b, :, covered:] = 0xAB
        idx.list_ids[b, :, covered:] = inp.cfg.n_list - 1
        idx.key_norms[b, :, covered:] = 1e9


@pytest.mark.parametrize("extra", [(1, 100), (255, 0), (100, 255)])
def test_decode_between_two_index_updates(extra):
    """Sec. 3.3: tokens written since the last index update stay in the exactly-attended window
    until the next update encodes them.  Two sequences at different phases: the index covers
    N_b - 128 - extra_b positions, the rest (128 + extra_b tokens) is the window, and the arrays
    behind the covered part hold garbage."""
    lens = (4000 + extra[0], 2500 + extra[1])
    covered = tuple(n - 128 - e for n, e in zip(lens, extra))
    cfg = small("phase", batch=2, seq_lens=lens, n_q_heads=4, n_kv_heads=2, n_sink=4,
                indexed_lens=covered, exact_set_multiple=16)
    inp, idx = make_case(cfg, device="cuda")
    _garble_unindexed(inp, idx)
    arrays = oracle_arrays(inp, idx)
    ref = run_oracle(inp, idx, arrays=arrays)
    op = DecodeOp(inp, idx)
    op.alloc_stage_buffers()
    op.build_lut(); op.scan(); op.select(); op.hybrid_attend()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK
    N_max, k_max = op.params.max_seq_len, op.params.k_max
    scores = op.scores.view(cfg.batch, cfg.n_q_heads, N_max).cpu().double().numpy()
    sel = op.sel_idx.view(cfg.batch, cfg.n_q_heads, k_max).cpu().numpy()
    cnt = op.sel_count.view(cfg.batch, cfg.n_q_heads).cpu().numpy()
    y32 = op.out_f32.cpu().double().numpy()
    for (b, h), r in ref.items():
        r0, r1 = 4, covered[b]
        assert len(r["R"]) == r1 - r0 and len(r["E"]) - r["k"] == 4 + lens[b] - covered[b]
        got = scores[b, h, r0:r1]
        assert np.all(np.abs(got - r["approx"]) <= LOGIT_RTOL * np.maximum(np.abs(r["approx"]), 1.0))
        assert np.all(np.isneginf(scores[b, h, r1:lens[b]])) and np.all(np.isneginf(scores[b, h, :r0]))
        assert cnt[b, h] == r["k"]
        ok, why = selection_matches(sel[b, h, :cnt[b, h]], r)
        assert ok, why
        assert np.abs(y32[b, h] - r["y"]).max() <= OUT_ATOL
    op.out.fill_(3.0)
    op.decode()
    torch.cuda.synchronize()
    fused = op.out.cpu().double().numpy()
    for (b, h), r in ref.items():
        assert np.all(np.abs(fused[b, h] - r["y"]) <= out_tolerance(r["y"], cfg.dtype))
