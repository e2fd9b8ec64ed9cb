"""The N>1 path on CPU: two gloo ranks each take their slice of a ragged batch, run it
independently (here with the oracle standing in for the GPU call), and the gathered outputs
equal a single-process run.  No collective is on the data path; the only reduction is the
max-over-ranks step time."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_33746_b200.sharding import max_over_ranks, rank_slice, shard_config
from paper_2609_33746_b200.workload import DecodeConfig

from helpers import make_case, run_oracle

CFG = DecodeConfig(name="shard", batch=5, n_q_heads=4, n_kv_heads=2, seq_lens=(300, 0, 257, 64, 129),
                   dtype="bf16", n_list=8, pq_m=16, budget_ppm=50000, seed=31, kmeans_iters=2)


def outputs(cfg, first_seq=0, full=None):
    """Oracle outputs [batch, Hq, d] of a (sub-)workload.  Sub-workloads are cut out of the
    full workload's tensors so that every rank sees the same keys it would see alone."""
    import dataclasses
    inp, idx = full
    lo, hi = first_seq, first_seq + cfg.batch
    sub_inp = dataclasses.replace(inp, cfg=cfg, q=inp.q[lo:hi], block_table=inp.block_table[lo:hi],
                                  seq_lens=inp.seq_lens[lo:hi])
    sub_idx = dataclasses.replace(idx, **{f.name: getattr(idx, f.name)[lo:hi]
                                          for f in dataclasses.fields(idx)})
    ref = run_oracle(sub_inp, sub_idx)
    out = np.zeros((cfg.batch, cfg.n_q_heads, cfg.head_dim))
    for (b, h), r in ref.items():
        out[b, h] = r["y"]
    return out


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        full = make_case(CFG)
        sub, first = shard_config(CFG, world, rank)
        mine = torch.from_numpy(outputs(sub, first, full))
        slowest = max_over_ranks(10.0 + rank)
        gathered = [None] * world
        dist.all_gather_object(gathered, (first, mine))
        if rank == 0:
            parts = [t for _, t in sorted(gathered, key=lambda p: p[0])]
            ret["out"] = torch.cat(parts).numpy()
            ret["slowest"] = slowest
    finally:
        dist.destroy_process_group()


def test_rank_slices_cover_every_item_once():
    for n in (0, 1, 5, 8, 17):
        for world in (1, 2, 3, 8):
            got = [i for r in range(world) for i in range(*rank_slice(n, world, r))]
            assert got == list(range(n))
            sizes = [b - a for a, b in (rank_slice(n, world, r) for r in range(world))]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        rank_slice(4, 2, 2)


def test_two_gloo_ranks_reproduce_the_single_process_result():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        ret = mgr.dict()
        procs = [ctx.Process(target=_worker, args=(r, 2, port, ret)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(timeout=240)
            assert p.exitcode == 0
        full = make_case(CFG)
        want = outputs(CFG, 0, full)
        assert ret["slowest"] == 11.0
        np.testing.assert_allclose(ret["out"], want, rtol=1e-12, atol=1e-14)
