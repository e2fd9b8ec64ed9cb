"""Context-length sweep: PQ-HSA decode step against dense decode attention on the same paged
cache (the crossover study of the paper's Sec. 4.4, on B200 and synthetic data).

    python -m paper_2609_33746_b200.sweep [--contexts 16,32,64,128,256,512] [--batch 1] [--steps 50]

Prints one JSON line per point: context, batch, us/step of pqhsa_decode and of
pqhsa_dense_decode (CUDA events, L2 flushed between steps), their ratio, and bytes."""
from __future__ import annotations

import argparse
import os
import dataclasses
import json
import statistics

import torch

from . import pqhsa
from .index_builder import build_index
from .runner import DecodeOp
from .workload import generate, named_config


def time_call(fn, steps, flush):
    for _ in range(3):
        fn()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(steps)]
    torch.cuda.synchronize()
    for a, b in ev:
        flush.zero_()
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return statistics.median(a.elapsed_time(b) for a, b in ev) * 1000.0


def copy_bandwidth_gbs():
    """Measured device copy bandwidth if the repository carries the figure, else the pool's
    earlier measurement."""
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return 6650.0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--contexts", default="16,32,64,128,256,512", help="context lengths in K tokens")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--kmeans-iters", type=int, default=2)
    ap.add_argument("--paper-index", action="store_true",
                    help="the paper's own index setting: 512 lists, 8 subspaces of 4 bits, 4 sinks, "
                         "128-token window, exact set in whole pages")
    args = ap.parse_args()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    for ctx in (int(x) for x in args.contexts.split(",")):
        cfg = dataclasses.replace(named_config(f"c5_n{ctx}_b{args.batch}"),
                                  kmeans_iters=args.kmeans_iters)
        if args.paper_index:
            cfg = dataclasses.replace(cfg, n_list=512, pq_m=8, pq_ncode=16, n_sink=4, n_local=128,
                                      exact_set_multiple=16)
        inp = generate(cfg, device="cuda")
        idx = build_index(inp)
        op = DecodeOp(inp, idx)
        dws = torch.empty(pqhsa.dense_workspace_bytes(op.params), dtype=torch.uint8, device="cuda")
        dout = torch.empty_like(op.q)
        t_pq = time_call(op.decode, args.steps, flush)
        t_dense = time_call(lambda: pqhsa.dense_decode(op.params, op.q, op.kv, op.seq_lens, dout,
                                                       dws), args.steps, flush)
        dense_bytes = cfg.batch * cfg.n_kv_heads * cfg.max_seq_len * 2 * cfg.head_dim * 2
        t_ideal = dense_bytes / copy_bandwidth_gbs() / 1e3      # us: one read of K and V at copy speed
        print(json.dumps(dict(context=cfg.max_seq_len, batch=cfg.batch, n_list=cfg.n_list,
                              budget_ppm=cfg.budget_ppm, pqhsa_us=round(t_pq, 1),
                              dense_us=round(t_dense, 1), dense_over_pqhsa=round(t_dense / t_pq, 3),
                              dense_gbs=round(dense_bytes / t_dense / 1e3, 1),
                              ideal_dense_us=round(t_ideal, 1),
                              ideal_dense_over_pqhsa=round(t_ideal / t_pq, 3))), flush=True)
        del op, inp, idx, dws
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
