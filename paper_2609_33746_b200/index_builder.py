"""Seeded IVF-PQ index builder (direction-norm residual IVF-PQ over keys, Section 3.1).

This is input preparation, done once per prompt and *not* part of the decode hot
path: its output (centroids, codebooks, codes, list ids, key norms, list value
means) is handed unchanged to both the CUDA operator and the CPU oracle, so the
choices made here (Lloyd iterations, initialisation, empty-cluster rule) do not
enter any parity comparison.

Readings of Section 3.1 / Appendix A used here:
  * keys are split k_i = r_i u_i, the norm r_i is computed in fp32 from the stored
    (fp16/bf16) key and kept outside the quantiser;
  * coarse quantiser: Lloyd k-means (squared L2) on the unit directions u_i; a
    centroid is the arithmetic mean of its members and is *not* re-normalised,
    because Eq. 2 uses c_j as is;
  * residuals u_i - c_{a_i} are product-quantised in M contiguous subspaces of
    d/M dims, one 256-word codebook per (sequence, KV head, subspace), shared by
    all lists;
  * list value mean = mean of the stored values of ALL members of the list
    (selected or not), accumulated in float64, stored fp32; an empty list has mean 0;
  * initial centres = a seeded sample of the points without replacement; an empty
    cluster is re-seeded with the point farthest from its centre.
"""
from __future__ import annotations

import dataclasses

import torch

from .workload import DecodeConfig, DecodeInputs


@dataclasses.dataclass
class IvfPqIndex:
    """Index arrays in the layout the C ABI documents (all on one device)."""
    centroids: torch.Tensor     # [B, Hkv, n_list, d]        f32
    codebooks: torch.Tensor     # [B, Hkv, M, 256, dsub]     f32
    codes: torch.Tensor         # [B, Hkv, N_max, M] u8, or [.., M / 2] with two 4-bit codes per
                                # byte (subspace 2j in the low nibble) when pq_ncode == 16
    list_ids: torch.Tensor      # [B, Hkv, N_max]            int16 storage of uint16 ids
    key_norms: torch.Tensor     # [B, Hkv, N_max]            f32
    list_vmeans: torch.Tensor   # [B, Hkv, n_list, d]        f32
    list_counts: torch.Tensor = None   # [B, Hkv, n_list]    int32 members behind each mean


def _assign(x: torch.Tensor, c: torch.Tensor, chunk: int = 16384):
    """Nearest centre (squared L2) for every row of x; ties -> lowest index."""
    ids = torch.empty(x.shape[0], dtype=torch.long, device=x.device)
    dist = torch.empty(x.shape[0], dtype=x.dtype, device=x.device)
    cn = (c * c).sum(-1)
    for s in range(0, x.shape[0], chunk):
        xs = x[s:s + chunk]
        d2 = (xs * xs).sum(-1, keepdim=True) - 2.0 * (xs @ c.T) + cn[None, :]
        dmin, imin = d2.min(dim=1)
        ids[s:s + chunk] = imin
        dist[s:s + chunk] = dmin
    return ids, dist


def _kmeans(x: torch.Tensor, k: int, iters: int, gen: torch.Generator):
    """Lloyd's algorithm on the rows of x (fp32).  Returns centres [k, dim]."""
    n = x.shape[0]
    if n >= k:
        init = torch.randperm(n, generator=gen, device=x.device)[:k]
        c = x[init].clone()
    else:                       # fewer points than centres: pad with zeros
        c = torch.zeros((k, x.shape[1]), dtype=x.dtype, device=x.device)
        c[:n] = x
    for _ in range(iters):
        ids, dist = _assign(x, c)
        # sums in float64: the device adds in no fixed order, and at that precision the order
        # no longer reaches the fp32 centres, so two builds of one workload give one index
        sums = torch.zeros(c.shape, dtype=torch.float64, device=x.device).index_add_(0, ids, x.double())
        cnt = torch.zeros(k, dtype=torch.float64, device=x.device).index_add_(
            0, ids, torch.ones(n, dtype=torch.float64, device=x.device))
        nonempty = cnt > 0
        c[nonempty] = (sums[nonempty] / cnt[nonempty, None]).to(c.dtype)
        n_empty = int((~nonempty).sum())
        if n_empty and n > k:
            far = torch.topk(dist, n_empty).indices
            c[~nonempty] = x[far]
    return c


def _batched_pq_kmeans(res: torch.Tensor, ncode: int, iters: int, gen: torch.Generator,
                       chunk: int = 8192):
    """One k-means per subspace, run together.  res: [n, M, dsub] -> [M, ncode, dsub]."""
    n, M, dsub = res.shape
    x = res.permute(1, 0, 2).contiguous()                 # [M, n, dsub]
    if n >= ncode:
        init = torch.randperm(n, generator=gen, device=res.device)[:ncode]
        c = x[:, init].clone()
    else:
        c = torch.zeros((M, ncode, dsub), dtype=res.dtype, device=res.device)
        c[:, :n] = x
    ones = torch.ones((M, n), dtype=torch.float64, device=res.device)
    x64 = x.double()
    for _ in range(iters):
        ids = _pq_encode(x, c, chunk)                     # [M, n]
        # (float64 sums, as in _kmeans: the order of the device's additions stays below fp32)
        sums = torch.zeros(c.shape, dtype=torch.float64, device=res.device).scatter_add_(
            1, ids[..., None].expand(-1, -1, dsub), x64)
        cnt = torch.zeros((M, ncode), dtype=torch.float64, device=res.device).scatter_add_(1, ids, ones)
        ne = cnt > 0
        c = torch.where(ne[..., None], (sums / cnt.clamp(min=1)[..., None]).to(c.dtype), c)
    return c


def _pq_encode(x: torch.Tensor, c: torch.Tensor, chunk: int = 8192) -> torch.Tensor:
    """x: [M, n, dsub], c: [M, ncode, dsub] -> nearest codeword ids [M, n]."""
    M, n, _ = x.shape
    ids = torch.empty((M, n), dtype=torch.long, device=x.device)
    cn = (c * c).sum(-1)                                  # [M, ncode]
    for s in range(0, n, chunk):
        xs = x[:, s:s + chunk]
        d2 = (xs * xs).sum(-1, keepdim=True) - 2.0 * torch.bmm(xs, c.transpose(1, 2)) \
            + cn[:, None, :]
        ids[:, s:s + chunk] = d2.argmin(dim=2)
    return ids


def build_index(inp: DecodeInputs) -> IvfPqIndex:
    """Build the per-(sequence, KV head) IVF-PQ index of a workload."""
    cfg: DecodeConfig = inp.cfg
    dev = inp.q.device
    B, Hkv, d = cfg.batch, cfg.n_kv_heads, cfg.head_dim
    M, dsub, nl, nc = cfg.pq_m, cfg.pq_dsub, cfg.n_list, cfg.pq_ncode
    Nmax = max(16, (cfg.max_seq_len + 15) // 16 * 16)   # row stride, padded to whole pages
    out = IvfPqIndex(
        torch.zeros((B, Hkv, nl, d), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, M, nc, dsub), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, Nmax, M if nc > 16 else M // 2), dtype=torch.uint8, device=dev),
        torch.zeros((B, Hkv, Nmax), dtype=torch.int16, device=dev),
        torch.zeros((B, Hkv, Nmax), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, nl, d), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, nl), dtype=torch.int32, device=dev))
    for b in range(B):
        n = cfg.seq_lens[b]
        if n == 0:
            continue
        for g in range(Hkv):
            gen = torch.Generator(device=dev).manual_seed(_unit_seed(cfg, b, g))
            k, v = inp.gather_kv(b, g)
            k32 = k.float()
            r = k32.norm(dim=1)                                   # fp32 norms
            u = torch.where(r[:, None] > 0, k32 / r[:, None].clamp(min=1e-30),
                            torch.zeros_like(k32))
            fit = u
            if cfg.fit_sample and n > cfg.fit_sample:
                fit = u[torch.randperm(n, generator=gen, device=dev)[:cfg.fit_sample]]
            c = _kmeans(fit, nl, cfg.kmeans_iters, gen)
            ids, _ = _assign(u, c)
            res_fit = (fit - c[_assign(fit, c)[0]]) if fit is not u else (u - c[ids])
            cb = _batched_pq_kmeans(res_fit.view(-1, M, dsub), nc,
                                    cfg.kmeans_iters if cfg.pq_iters is None else cfg.pq_iters, gen)
            res = (u - c[ids]).view(n, M, dsub).permute(1, 0, 2).contiguous()
            codes = _pq_encode(res, cb)                           # [M, n]
            # list value means over the members inside the indexed region R (Sec. 3.2): sink
            # and window tokens are attended exactly and belong to no list's background
            r0 = min(cfg.n_sink, n)
            r1 = max(r0, n - cfg.n_local)
            if cfg.indexed_lens is not None:
                r1 = max(r0, min(n, cfg.indexed_lens[b]))
            vsum = torch.zeros((nl, d), dtype=torch.float64, device=dev).index_add_(
                0, ids[r0:r1], v[r0:r1].double())
            cnt = torch.zeros(nl, dtype=torch.float64, device=dev).index_add_(
                0, ids[r0:r1], torch.ones(r1 - r0, dtype=torch.float64, device=dev))
            vmean = torch.where(cnt[:, None] > 0, vsum / cnt.clamp(min=1)[:, None],
                                torch.zeros_like(vsum))
            out.centroids[b, g] = c
            out.codebooks[b, g] = cb
            ct = codes.T.to(torch.uint8)                          # [n, M]
            out.codes[b, g, :n] = ct if nc > 16 else (ct[:, 0::2] | (ct[:, 1::2] << 4))
            out.list_ids[b, g, :n] = ids.to(torch.int16)
            out.key_norms[b, g, :n] = r
            out.list_vmeans[b, g] = vmean.float()
            out.list_counts[b, g] = cnt.to(torch.int32)
    return out


def _unit_seed(cfg: DecodeConfig, b: int, g: int) -> int:
    return (cfg.seed * 1000003 + b * 4099 + g * 17 + 7) & 0x7FFFFFFF


def seed_positions(inp: DecodeInputs):
    """The random draws of build_index, on their own: for every (sequence, KV head) the
    positions of the tokens that seed the centroids [B, Hkv, n_list] and the codewords
    [B, Hkv, pq_ncode] (-1 where the sequence has fewer tokens than seeds).  Same generator,
    same order of draws as build_index (without fit_sample), so that another builder started
    from these positions trains the same problems."""
    cfg = inp.cfg
    dev = inp.q.device
    lists = torch.full((cfg.batch, cfg.n_kv_heads, cfg.n_list), -1, dtype=torch.int32, device=dev)
    words = torch.full((cfg.batch, cfg.n_kv_heads, cfg.pq_ncode), -1, dtype=torch.int32, device=dev)
    for b in range(cfg.batch):
        n = cfg.seq_lens[b]
        if n == 0:
            continue
        for g in range(cfg.n_kv_heads):
            gen = torch.Generator(device=dev).manual_seed(_unit_seed(cfg, b, g))
            if n >= cfg.n_list:
                lists[b, g] = torch.randperm(n, generator=gen, device=dev)[:cfg.n_list].int()
            else:
                lists[b, g, :n] = torch.arange(n, dtype=torch.int32, device=dev)
            if n >= cfg.pq_ncode:
                words[b, g] = torch.randperm(n, generator=gen, device=dev)[:cfg.pq_ncode].int()
            else:
                words[b, g, :n] = torch.arange(n, dtype=torch.int32, device=dev)
    return lists, words


def build_index_batched(inp: DecodeInputs, coarse_iters=None, pq_iters=None) -> IvfPqIndex:
    """The index of a workload trained by the library's batched build (pqhsa_index_build): all
    (sequence, KV head) problems in one call, from the same seed positions as build_index."""
    from . import pqhsa
    cfg = inp.cfg
    dev = inp.q.device
    B, Hkv, d = cfg.batch, cfg.n_kv_heads, cfg.head_dim
    M, dsub, nl, nc = cfg.pq_m, cfg.pq_dsub, cfg.n_list, cfg.pq_ncode
    Nmax = max(16, (cfg.max_seq_len + 15) // 16 * 16)
    out = IvfPqIndex(
        torch.zeros((B, Hkv, nl, d), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, M, nc, dsub), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, Nmax, M if nc > 16 else M // 2), dtype=torch.uint8, device=dev),
        torch.zeros((B, Hkv, Nmax), dtype=torch.int16, device=dev),
        torch.zeros((B, Hkv, Nmax), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, nl, d), dtype=torch.float32, device=dev),
        torch.zeros((B, Hkv, nl), dtype=torch.int32, device=dev))
    indexed = None
    if cfg.indexed_lens is not None:
        indexed = torch.tensor(list(cfg.indexed_lens), dtype=torch.int32, device=dev)
    params = pqhsa.make_params(
        batch=B, n_q_heads=cfg.n_q_heads, n_kv_heads=Hkv, n_list=nl, pq_m=M, max_seq_len=Nmax,
        max_pages_per_seq=inp.max_pages_per_seq, budget_ppm=cfg.budget_ppm, dtype=cfg.dtype,
        head_dim=d, pq_ncode=nc, page_size=cfg.page_size, n_sink=cfg.n_sink, n_local=cfg.n_local,
        exact_set_multiple=cfg.exact_set_multiple, indexed_lens=indexed)
    if cfg.kv_layout == "interleaved":
        k_cache, v_cache = inp.k_cache, inp.k_cache.view(-1)[d:]
    else:
        k_cache, v_cache = inp.k_cache, inp.v_cache
    kv = pqhsa.make_paged_kv(k_cache, v_cache, inp.stride_page, inp.stride_token, inp.stride_head,
                             inp.block_table)
    lists, words = seed_positions(inp)
    ws = torch.empty(pqhsa.index_build_workspace_bytes(params), dtype=torch.uint8, device=dev)
    it = cfg.kmeans_iters
    it_pq = it if cfg.pq_iters is None else cfg.pq_iters
    pqhsa.index_build(params, kv, inp.seq_lens, lists, words,
                      it if coarse_iters is None else coarse_iters,
                      it_pq if pq_iters is None else pq_iters,
                      out.centroids, out.codebooks, out.codes, out.list_ids, out.key_norms,
                      out.list_vmeans, out.list_counts, ws)
    torch.cuda.synchronize(dev)
    return out
