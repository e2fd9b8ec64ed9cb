"""Shared test plumbing: build a workload + index, and hand the same arrays to the oracle."""
import math

import numpy as np
import torch

from oracle import pqhsa_oracle as O
from paper_2609_33746_b200.index_builder import build_index
from paper_2609_33746_b200.workload import DecodeConfig, generate


def make_case(cfg: DecodeConfig, device="cpu", pre_index=None):
    inp = generate(cfg, device=device)
    if pre_index is not None:
        pre_index(inp)
    idx = build_index(inp)
    return inp, idx


def oracle_arrays(inp, idx):
    """numpy views of the inputs in the oracle's (= the C ABI's) layouts, values in float64
    where they are floating point."""
    f64 = lambda t: t.detach().cpu().double().numpy()
    a = dict(
        q=f64(inp.q), centroids=f64(idx.centroids), codebooks=f64(idx.codebooks),
        codes=unpacked_codes(idx.codes.cpu().numpy(), inp.cfg),
        list_ids=idx.list_ids.cpu().numpy().view(np.uint16),
        key_norms=f64(idx.key_norms), list_vmeans=f64(idx.list_vmeans),
        k_cache_flat=f64(inp.k_cache.reshape(-1)), v_cache_flat=f64(inp.v_cache.reshape(-1)),
        block_table=inp.block_table.cpu().numpy(), seq_lens=inp.seq_lens.cpu().numpy())
    return a


def unpacked_codes(codes: np.ndarray, cfg) -> np.ndarray:
    """One code per byte for the oracle: 4-bit indices come two per byte (subspace 2j in the low
    nibble of byte j)."""
    if cfg.pq_ncode > 16:
        return codes
    out = np.empty(codes.shape[:-1] + (cfg.pq_m,), dtype=np.uint8)
    out[..., 0::2] = codes & 15
    out[..., 1::2] = codes >> 4
    return out


def oracle_arrays_for_sequence(inp, idx, b):
    """Same as oracle_arrays, but for one sequence of a large workload: only that sequence's
    index arrays and KV pages are copied to the host (pages re-packed contiguously with an
    identity block table; the oracle still reads rows through block table and strides)."""
    cfg = inp.cfg
    assert cfg.kv_layout == "split"
    f64 = lambda t: t.detach().cpu().double().numpy()
    n = int(inp.seq_lens[b])
    n_pages = max(1, (n + cfg.page_size - 1) // cfg.page_size)
    pages = inp.block_table[b, :n_pages].long()
    sl = slice(b, b + 1)
    return dict(
        q=f64(inp.q[sl]), centroids=f64(idx.centroids[sl]), codebooks=f64(idx.codebooks[sl]),
        codes=unpacked_codes(idx.codes[sl].cpu().numpy(), cfg),
        list_ids=idx.list_ids[sl].cpu().numpy().view(np.uint16),
        key_norms=f64(idx.key_norms[sl]), list_vmeans=f64(idx.list_vmeans[sl]),
        k_cache_flat=f64(inp.k_cache[pages].reshape(-1)),
        v_cache_flat=f64(inp.v_cache[pages].reshape(-1)),
        block_table=np.arange(n_pages, dtype=np.int32)[None, :],
        seq_lens=inp.seq_lens[sl].cpu().numpy())


def run_oracle(inp, idx, budget_ppm=None, heads=None, batch_items=None, arrays=None, variant=None,
               indexed_lens=None):
    cfg = inp.cfg
    a = arrays or oracle_arrays(inp, idx)
    return O.decode(a["q"], a["centroids"], a["codebooks"], a["codes"], a["list_ids"],
                    a["key_norms"], a["list_vmeans"], a["k_cache_flat"], a["v_cache_flat"],
                    a["block_table"], a["seq_lens"], n_kv_heads=cfg.n_kv_heads,
                    page_size=cfg.page_size, stride_page=inp.stride_page,
                    stride_token=inp.stride_token, stride_head=inp.stride_head,
                    budget_ppm=cfg.budget_ppm if budget_ppm is None else budget_ppm,
                    sm_scale=1.0 / math.sqrt(cfg.head_dim), heads=heads, batch_items=batch_items,
                    n_sink=cfg.n_sink, n_local=cfg.n_local,
                    variant=cfg.variant if variant is None else variant,
                    indexed_lens=cfg.indexed_lens if indexed_lens is None else indexed_lens,
                    round_exact_set_to_page=cfg.exact_set_multiple if cfg.exact_set_multiple > 1 else 0)


def selection_matches(gpu_sel, ref, tol=1e-3):
    """Selected sets are equal except for tokens whose approximate logit is within
    tol * max(1, |s_k|) of the k-th score s_k; the set size must be exactly k."""
    gpu = set(int(x) for x in gpu_sel)
    want = set(int(x) for x in ref["T"])
    if len(gpu) != ref["k"] or len(gpu_sel) != ref["k"]:
        return False, f"size {len(gpu_sel)} (unique {len(gpu)}) != k {ref['k']}"
    if ref["k"] == 0:
        return True, ""
    sk = ref["kth_score"]
    band = tol * max(1.0, abs(sk))
    approx = ref["approx"]
    r0 = int(ref["R"][0]) if len(ref["R"]) else 0
    for i in gpu ^ want:
        if abs(approx[i - r0] - sk) > band:
            return False, f"token {i} (score {approx[i - r0]}, kth {sk}) differs outside the tie band"
    return True, ""
