"""Seeded synthetic decode-step workloads (inputs only; none of the operator's arithmetic).

Everything here produces *inputs* of the PQ-HSA decode operator: queries, a paged
K/V cache with a shuffled block table, and sequence lengths.  The IVF-PQ index that
the operator also consumes is made from these keys/values by ``index_builder``.
Both the CUDA path and the CPU oracle read the arrays produced here; neither is
imported by this module.

Recipe (per sequence b and KV head g, one ``torch.Generator`` seeded from
(config seed, b, g); draws in this fixed order):
  1. 64 mixture centres  mu_c ~ N(0, I_d)
  2. token -> centre assignment  c_i ~ U{0..63}
  3. per-token offsets  0.3 * N(0, I_d)         keys  k_i = mu_{c_i} + offset_i
  4. 4 outlier channels (without replacement), multiplied by ``outlier_scale``
  5. values  v_i ~ N(0, I_d)
  6. per query head of the group: 3 key positions (uniform over the sequence)
  7. per query head: noise 0.1 * N(0, I_d);  q = k_a + k_b + k_c + noise
Keys, values and queries are rounded to the cache dtype (fp16 or bf16) before
anything else sees them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import torch

PAGE_SIZE = 16
N_MIXTURE_CENTERS = 64
N_OUTLIER_CHANNELS = 4


@dataclasses.dataclass(frozen=True)
class DecodeConfig:
    """Shape of one decode-step workload (names follow the paper's notation)."""
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    seq_lens: tuple                      # one length per sequence
    dtype: str                           # "fp16" | "bf16"  (q, K, V, out)
    n_list: int
    pq_m: int                            # M subspaces; dsub = head_dim / M
    budget_ppm: int                      # rho in parts per million
    head_dim: int = 128
    pq_ncode: int = 256
    page_size: int = PAGE_SIZE
    outlier_scale: float = 8.0
    kmeans_iters: int = 10
    pq_iters: Optional[int] = None       # Lloyd iterations of the codebooks (None: kmeans_iters)
    seed: int = 0
    kv_layout: str = "split"             # "split": K and V separate [page][tok][head][d]
                                         # "interleaved": one buffer [page][head][tok][2d]
    fit_sample: int = 0                  # >0: fit centroids/codebooks on this many tokens
    n_sink: int = 0                      # |S|: first tokens attended exactly (Sec. 3.2)
    n_local: int = 0                     # |L|: most recent tokens attended exactly
    exact_set_multiple: int = 0          # >1: |S|+|L|+k rounded up to this multiple (App. A)
    variant: str = "B"                   # background term: B (PQ-HSA), T, Bx, C, C2, C2b (Table 2)
    indexed_lens: Optional[tuple] = None # per sequence: positions the index covers; the rest of
                                         # the sequence is the exactly-attended window (Sec. 3.3)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def pq_dsub(self) -> int:
        return self.head_dim // self.pq_m

    @property
    def max_seq_len(self) -> int:
        return max(self.seq_lens) if self.seq_lens else 0

    def torch_dtype(self) -> torch.dtype:
        return {"fp16": torch.float16, "bf16": torch.bfloat16}[self.dtype]


def _ragged_lengths(batch: int, lo: int, hi: int, seed: int) -> tuple:
    g = torch.Generator().manual_seed(seed)
    return tuple(int(x) for x in torch.randint(lo, hi + 1, (batch,), generator=g))


def named_config(name: str) -> DecodeConfig:
    """The workloads of the benchmark plan, by name."""
    K = 1024
    if name == "c1":       # tiny single-KV-head case, seed 0
        return DecodeConfig("c1", 1, 4, 1, (4096,), "fp16", 64, 16, 20000, seed=0)
    if name == "c2":       # Llama-3.1-8B-shaped layer, 32K
        return DecodeConfig("c2", 1, 32, 8, (32 * K,), "bf16", 256, 32, 20000, seed=2000)
    if name.startswith("c3p"):  # c3p_b{B}_r{pct}: the same layer in the paper's own index setting
        _, b, r = name.split("_")  # (512 lists, 8 subspaces of 4 bits, 4 sinks, 128-token window,
        batch, pct = int(b[1:]), int(r[1:])          # exact set in whole pages; App. A)
        return DecodeConfig(name, batch, 32, 8, (128 * K,) * batch, "bf16", 512, 8, pct * 10000,
                            seed=3000, pq_ncode=16, n_sink=4, n_local=128, exact_set_multiple=16)
    if name.startswith("c3"):   # c3_b{1,8}_r{1,2}: Llama-3.1-8B-shaped layer, 128K
        _, b, r = name.split("_")
        batch, pct = int(b[1:]), int(r[1:])
        return DecodeConfig(name, batch, 32, 8, (128 * K,) * batch, "bf16", 1024, 32,
                            pct * 10000, seed=3000)
    if name == "c4":       # Qwen3-30B-A3B-shaped layer, ragged batch 16, G=8
        lens = _ragged_lengths(16, 96 * K, 128 * K, 4000)
        return DecodeConfig("c4", 16, 32, 4, lens, "bf16", 1024, 32, 10000,
                            outlier_scale=16.0, seed=4000)
    if name.startswith("c5"):   # c5_n{ctx in K}_b{batch}: context sweep, n_list = N/128
        _, n, b = name.split("_")
        ctx, batch = int(n[1:]) * K, int(b[1:])
        return DecodeConfig(name, batch, 32, 8, (ctx,) * batch, "bf16", ctx // 128, 32,
                            10000, seed=5000)
    raise KeyError(name)


@dataclasses.dataclass
class DecodeInputs:
    """Tensors of one workload, laid out as the C ABI expects them."""
    cfg: DecodeConfig
    q: torch.Tensor                # [B, Hq, d]            cache dtype
    k_cache: torch.Tensor          # paged, see kv_layout  cache dtype
    v_cache: torch.Tensor          # (a view into k_cache's buffer when interleaved)
    stride_page: int               # element strides of the paged view
    stride_token: int
    stride_head: int
    block_table: torch.Tensor      # [B, max_pages] int32
    seq_lens: torch.Tensor         # [B] int32
    max_pages_per_seq: int

    def gather_kv(self, b: int, g: int, device=None):
        """Contiguous [N_b, d] copies of one head's keys and values (used by the
        index builder and by tests; reads through the block table and strides)."""
        n = int(self.seq_lens[b])
        pos = torch.arange(n, device=self.block_table.device)
        page = self.block_table[b, pos // self.cfg.page_size].long()
        off = page * self.stride_page + (pos % self.cfg.page_size) * self.stride_token \
            + g * self.stride_head
        idx = off[:, None] + torch.arange(self.cfg.head_dim, device=off.device)[None, :]
        return self.k_cache.reshape(-1)[idx], self.v_cache.reshape(-1)[idx]


def generate(cfg: DecodeConfig, device: str = "cpu") -> DecodeInputs:
    """Draw one workload.  Deterministic for a given (cfg, device type)."""
    d, P = cfg.head_dim, cfg.page_size
    B, Hkv, G = cfg.batch, cfg.n_kv_heads, cfg.group
    dt = cfg.torch_dtype()
    dev = torch.device(device)
    pages_per_seq = [(n + P - 1) // P for n in cfg.seq_lens]
    max_pages = max(pages_per_seq) if pages_per_seq else 0
    total_pages = sum(pages_per_seq)

    # A real engine hands out pages in no particular order: shuffle the page ids.
    gperm = torch.Generator().manual_seed(cfg.seed * 7919 + 13)
    perm = torch.randperm(max(total_pages, 1), generator=gperm).to(torch.int32)
    block_table = torch.zeros((B, max(max_pages, 1)), dtype=torch.int32)
    o = 0
    for b in range(B):
        block_table[b, :pages_per_seq[b]] = perm[o:o + pages_per_seq[b]]
        o += pages_per_seq[b]
    block_table = block_table.to(dev)

    if cfg.kv_layout == "split":
        k_cache = torch.zeros((max(total_pages, 1), P, Hkv, d), dtype=dt, device=dev)
        v_cache = torch.zeros_like(k_cache)
        s_page, s_tok, s_head = P * Hkv * d, Hkv * d, d
        kflat, vflat = k_cache.view(-1), v_cache.view(-1)
    elif cfg.kv_layout == "interleaved":
        buf = torch.zeros((max(total_pages, 1), Hkv, P, 2 * d), dtype=dt, device=dev)
        k_cache = buf
        v_cache = buf.view(-1)[d:]
        s_page, s_tok, s_head = Hkv * P * 2 * d, 2 * d, P * 2 * d
        kflat, vflat = buf.view(-1), v_cache
    else:
        raise ValueError(cfg.kv_layout)

    q = torch.zeros((B, cfg.n_q_heads, d), dtype=dt, device=dev)
    ar_d = torch.arange(d, device=dev)
    for b in range(B):
        n = cfg.seq_lens[b]
        if n == 0:
            continue
        pos = torch.arange(n, device=dev)
        page = block_table[b, pos // P].long()
        for g in range(Hkv):
            gen = torch.Generator(device=dev).manual_seed(
                (cfg.seed * 1000003 + b * 4099 + g * 17 + 1) & 0x7FFFFFFF)
            mu = torch.randn((N_MIXTURE_CENTERS, d), generator=gen, device=dev)
            assign = torch.randint(0, N_MIXTURE_CENTERS, (n,), generator=gen, device=dev)
            keys = mu[assign] + 0.3 * torch.randn((n, d), generator=gen, device=dev)
            outl = torch.randperm(d, generator=gen, device=dev)[:N_OUTLIER_CHANNELS]
            keys[:, outl] *= cfg.outlier_scale
            vals = torch.randn((n, d), generator=gen, device=dev)
            keys, vals = keys.to(dt), vals.to(dt)
            off = page * s_page + (pos % P) * s_tok + g * s_head
            idx = off[:, None] + ar_d[None, :]
            kflat[idx] = keys
            vflat[idx] = vals
            picks = torch.randint(0, n, (G, 3), generator=gen, device=dev)
            noise = 0.1 * torch.randn((G, d), generator=gen, device=dev)
            qh = keys.float()[picks].sum(dim=1) + noise
            q[b, g * G:(g + 1) * G] = qh.to(dt)

    return DecodeInputs(cfg, q, k_cache, v_cache, s_page, s_tok, s_head, block_table,
                        torch.tensor(list(cfg.seq_lens), dtype=torch.int32, device=dev),
                        max(max_pages, 1))
