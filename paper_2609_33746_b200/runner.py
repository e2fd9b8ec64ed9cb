"""Glue between a generated workload and the C-ABI binding: owns the device buffers of one
decode step and calls the library.  No arithmetic of the method lives here."""
from __future__ import annotations

import torch

from . import pqhsa
from .index_builder import IvfPqIndex
from .workload import DecodeConfig, DecodeInputs


class DecodeOp:
    """Device buffers + marshalled structs of one workload; every method is one library call."""

    def __init__(self, inp: DecodeInputs, index: IvfPqIndex, device: str = "cuda:0",
                 budget_ppm: int | None = None, variant: str | None = None,
                 fp16_tables=False):
        cfg: DecodeConfig = inp.cfg
        self.cfg, self.device = cfg, torch.device(device)
        dev = self.device
        self.keep = []           # tensors whose storage the structs point into

        def put(t):
            t = t.to(dev).contiguous()
            self.keep.append(t)
            return t

        self.q = put(inp.q)
        if cfg.kv_layout == "interleaved":
            buf = put(inp.k_cache)
            self.k_cache, self.v_cache = buf, buf.view(-1)[cfg.head_dim:]
        else:
            self.k_cache, self.v_cache = put(inp.k_cache), put(inp.v_cache)
        self.block_table = put(inp.block_table)
        self.seq_lens = put(inp.seq_lens)
        self.centroids, self.codebooks = put(index.centroids), put(index.codebooks)
        self.codes, self.list_ids = put(index.codes), put(index.list_ids)
        self.key_norms, self.list_vmeans = put(index.key_norms), put(index.list_vmeans)
        self.list_counts = put(index.list_counts) if index.list_counts is not None else None
        self.indexed_lens = None
        if cfg.indexed_lens is not None:
            self.indexed_lens = put(torch.tensor(list(cfg.indexed_lens), dtype=torch.int32))

        ppm = cfg.budget_ppm if budget_ppm is None else budget_ppm
        self.params = pqhsa.make_params(
            batch=cfg.batch, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
            n_list=cfg.n_list, pq_m=cfg.pq_m, max_seq_len=self.codes.shape[2],
            max_pages_per_seq=inp.max_pages_per_seq, budget_ppm=ppm, dtype=cfg.dtype,
            head_dim=cfg.head_dim, pq_ncode=cfg.pq_ncode, page_size=cfg.page_size, n_sink=cfg.n_sink,
            n_local=cfg.n_local, exact_set_multiple=cfg.exact_set_multiple,
            variant=cfg.variant if variant is None else variant, indexed_lens=self.indexed_lens,
            fp16_tables=fp16_tables)
        self.index = pqhsa.make_index(self.centroids, self.codebooks, self.codes, self.list_ids,
                                      self.key_norms, self.list_vmeans, self.list_counts)
        self.kv = pqhsa.make_paged_kv(self.k_cache, self.v_cache, inp.stride_page,
                                      inp.stride_token, inp.stride_head, self.block_table)
        self.fp16_tables = fp16_tables
        self.ws = torch.empty(pqhsa.workspace_bytes(self.params), dtype=torch.uint8, device=dev)
        self.out = torch.zeros_like(self.q)

    # ---- intermediates for stage-by-stage calls
    def alloc_stage_buffers(self):
        p, dev = self.params, self.device
        f32 = lambda which: torch.empty(pqhsa.buffer_elems(p, which), dtype=torch.float32,
                                        device=dev)
        i32 = lambda which: torch.empty(pqhsa.buffer_elems(p, which), dtype=torch.int32,
                                        device=dev)
        self.lut, self.coarse = f32(pqhsa.BUF_LUT), f32(pqhsa.BUF_COARSE)
        self.scores = f32(pqhsa.BUF_SCORES)
        self.list_partials = f32(pqhsa.BUF_LIST_PARTIALS)
        self.sel_idx, self.sel_count = i32(pqhsa.BUF_SEL_IDX), i32(pqhsa.BUF_SEL_COUNT)
        self.kth = f32(pqhsa.BUF_KTH)
        self.lse = torch.empty(p.batch * p.n_q_heads, dtype=torch.float32, device=dev)
        self.out_f32 = torch.empty(self.q.shape, dtype=torch.float32, device=dev)

    def build_lut(self):
        pqhsa.build_lut(self.params, self.q, self.index, self.lut, self.coarse)

    def scan(self):
        pqhsa.scan(self.params, self.index, self.lut, self.coarse, self.seq_lens, self.scores,
                   self.list_partials, self.ws)

    def select(self):
        pqhsa.select(self.params, self.scores, self.seq_lens, self.sel_idx, self.sel_count,
                     self.kth, self.ws)
        if self.fp16_tables == "rescore":
            pqhsa.rescore(self.params, self.index, self.lut, self.coarse, self.scores, self.seq_lens,
                          self.sel_idx, self.sel_count, self.kth, self.ws)

    def hybrid_attend(self):
        pqhsa.hybrid_attend(self.params, self.q, self.kv, self.index, self.scores,
                            self.list_partials, self.sel_idx, self.sel_count, self.seq_lens,
                            self.out, self.lse, self.ws, out_f32=self.out_f32)

    def decode(self, q=None, out=None):
        pqhsa.decode(self.params, self.q if q is None else q, self.index, self.kv, self.seq_lens,
                     self.out if out is None else out, self.ws)
        return self.out if out is None else out

    def decode_buffer(self, which: int, dtype=torch.float32) -> torch.Tensor:
        """View of an intermediate that the last decode() left in the workspace."""
        off = pqhsa.decode_buffer_offset(self.params, which)
        n = pqhsa.buffer_elems(self.params, which)
        return self.ws[off:off + 4 * n].view(dtype)

    def device_status(self) -> int:
        return pqhsa.last_device_status(self.params, self.ws)
