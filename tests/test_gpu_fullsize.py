"""Parity at the full sizes of the benchmark's configs, in the launch configuration bench.py times
(-m gpu).  Each case checks (sequence, query head) rows end to end against the oracle:
approximate logits over the whole row, the selected set, and the output."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from paper_2609_33746_b200 import pqhsa
from paper_2609_33746_b200.index_builder import build_index
from paper_2609_33746_b200.runner import DecodeOp
from paper_2609_33746_b200.workload import generate, named_config

from helpers import oracle_arrays_for_sequence, run_oracle, selection_matches
from test_gpu_parity import LOGIT_RTOL, OUT_ATOL, half_ulp, out_tolerance

pytestmark = pytest.mark.gpu

ALL = range(32)        # every query head (all configs here have 32)
CASES = [
    # (workload, checked (sequence, query head) rows).  The oracle does a 128K row in well under
    # a second, so most configs are checked on EVERY row; the largest ones on every row of a few
    # sequences.
    ("c2", [(0, h) for h in ALL]),
    ("c3_b1_r1", [(0, h) for h in ALL]),
    ("c3_b1_r2", [(0, h) for h in ALL]),
    ("c3_b8_r1", [(b, h) for b in range(8) for h in ALL]),     # the benchmark's default workload
    ("c4", [(b, h) for b in (2, 11, 15) for h in ALL]),        # ragged batch of 16, G = 8
    ("c5_n512_b1", [(0, h) for h in ALL]),                     # 512K context, n_list = 4096
    # the paper's own partition at 128K: 4 sinks, 128-token window, exact set in whole pages
    # (1,456 tokens at 1 %, App. A)
    ("c3_b1_r1+sinks_window_pages", [(0, h) for h in ALL]),
    # ... and with the paper's own index on top: 512 lists, eight 4-bit subspaces
    ("c3p_b1_r1", [(0, h) for h in ALL]),
]


def config_of(name):
    base, _, extra = name.partition("+")
    cfg = named_config(base)
    if extra == "sinks_window_pages":
        cfg = dataclasses.replace(cfg, n_sink=4, n_local=128, exact_set_multiple=16)
    return cfg


@pytest.mark.parametrize("name,rows", CASES, ids=[c[0] for c in CASES])
def test_full_size_decode_on_sampled_rows(name, rows):
    cfg = dataclasses.replace(config_of(name), kmeans_iters=2)
    inp = generate(cfg, device="cuda")
    idx = build_index(inp)
    op = DecodeOp(inp, idx)
    out = op.decode()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK
    N_max, k_max = op.params.max_seq_len, op.params.k_max
    scores = op.decode_buffer(pqhsa.BUF_SCORES).view(cfg.batch, cfg.n_q_heads, N_max)
    sel = op.decode_buffer(pqhsa.BUF_SEL_IDX, torch.int32).view(cfg.batch, cfg.n_q_heads, k_max)
    cnt = op.decode_buffer(pqhsa.BUF_SEL_COUNT, torch.int32).view(cfg.batch, cfg.n_q_heads)
    out32 = op.decode_buffer(pqhsa.BUF_OUT_F32).view(cfg.batch, cfg.n_q_heads, -1)   # before the rounding
    by_seq = {}
    for b, h in rows:
        by_seq.setdefault(b, []).append(h)
    for b, heads in by_seq.items():
        arrays = oracle_arrays_for_sequence(inp, idx, b)
        sub = dataclasses.replace(inp, cfg=dataclasses.replace(cfg, batch=1, seq_lens=(cfg.seq_lens[b],)))
        ref = run_oracle(sub, None, heads=heads, batch_items=[0], arrays=arrays)
        n = cfg.seq_lens[b]
        r0, r1 = min(cfg.n_sink, n), max(min(cfg.n_sink, n), n - cfg.n_local)     # R = [r0, r1)
        for h in heads:
            r = ref[(0, h)]
            got = scores[b, h, r0:r1].cpu().double().numpy()
            assert np.all(np.abs(got - r["approx"]) <= LOGIT_RTOL * np.maximum(np.abs(r["approx"]), 1.0)), \
                f"{name} logits row {(b, h)}: {np.abs(got - r['approx']).max()}"
            c = int(cnt[b, h])
            assert c == r["k"]
            if cfg.exact_set_multiple > 1:
                assert (c + r0 + (n - r1)) % cfg.exact_set_multiple == 0
            ok, why = selection_matches(sel[b, h, :c].cpu().numpy(), r)
            assert ok, f"{name} selection row {(b, h)}: {why}"
            y32 = out32[b, h].cpu().double().numpy()
            assert np.abs(y32 - r["y"]).max() <= OUT_ATOL, \
                f"{name} output row {(b, h)} before rounding: max-abs {np.abs(y32 - r['y']).max()}"
            y = out[b, h].cpu().double().numpy()
            assert np.all(np.abs(y - y32) <= half_ulp(y32, cfg.dtype) * 1.0001), \
                f"{name} stored output row {(b, h)} is not the computed one rounded"
    del op, inp, idx
    torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", ["T", "Bx", "C", "C2", "C2b"])
def test_full_size_mechanism_variants(variant):
    """The ablation variants (Table 2, App. B) at 128K under the paper's own partition and index
    setting, every row: the output against the oracle's for that variant."""
    cfg = dataclasses.replace(config_of("c3p_b1_r1"), kmeans_iters=2)
    inp = generate(cfg, device="cuda")
    idx = build_index(inp)
    op = DecodeOp(inp, idx, variant=variant)
    out = op.decode()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK
    arrays = oracle_arrays_for_sequence(inp, idx, 0)
    ref = run_oracle(inp, None, heads=list(ALL), batch_items=[0], arrays=arrays, variant=variant)
    out32 = op.decode_buffer(pqhsa.BUF_OUT_F32).view(cfg.batch, cfg.n_q_heads, -1)
    for h in ALL:
        r = ref[(0, h)]
        y32 = out32[0, h].cpu().double().numpy()
        assert np.abs(y32 - r["y"]).max() <= OUT_ATOL, \
            f"variant {variant} output row {(0, h)} before rounding: max-abs {np.abs(y32 - r['y']).max()}"
        y = out[0, h].cpu().double().numpy()
        assert np.all(np.abs(y - r["y"]) <= out_tolerance(r["y"], cfg.dtype))
    del op, inp, idx
    torch.cuda.empty_cache()
