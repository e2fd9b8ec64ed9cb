"""ctypes binding of libpqhsa.so: same entry points as include/pqhsa.h, argument marshalling only.

Every step of the decode path runs in the library's CUDA kernels.  PyTorch appears here
only as the owner of device memory and streams.  There is no fallback: if the shared
library is missing or a call fails, a ``PqhsaError`` is raised.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# PQHSA_LIBRARY selects another build of the same library, e.g. libpqhsa_debug.so (the build
# that records out-of-range indices in the status word)
LIB_PATH = os.environ.get("PQHSA_LIBRARY") or os.path.join(_HERE, "libpqhsa.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_CHECK = 0, -1, -2, -3, -4, -5
F16, BF16 = 0, 1
(BUF_LUT, BUF_COARSE, BUF_SCORES, BUF_LIST_PARTIALS, BUF_SEL_IDX, BUF_SEL_COUNT, BUF_KTH,
 BUF_BG_MASS, BUF_BG_MAX, BUF_OUT_F32) = range(10)
VARIANTS = {"B": 0, "T": 1, "Bx": 2, "C": 3, "C2": 4, "C2b": 5}      # pqhsa_variant

EXPORTS = [
    "pqhsa_heads_per_group", "pqhsa_num_partials", "pqhsa_buffer_elems", "pqhsa_workspace_bytes",
    "pqhsa_build_lut", "pqhsa_scan", "pqhsa_select", "pqhsa_hybrid_attend", "pqhsa_decode",
    "pqhsa_decode_events", "pqhsa_decode_host", "pqhsa_last_device_status", "pqhsa_decode_buffer_offset",
    "pqhsa_decode_launch_count", "pqhsa_status_string", "pqhsa_select_static",
    "pqhsa_select_static_bytes", "pqhsa_select_static_capacity", "pqhsa_dense_decode",
    "pqhsa_dense_workspace_bytes", "pqhsa_index_update", "pqhsa_debug_build",
    "pqhsa_debug_predicate", "pqhsa_index_build", "pqhsa_index_build_workspace_bytes",
    "pqhsa_rescore", "pqhsa_gather_probe",
]


class PqhsaError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status_string(status)} ({status})")


class Params(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "n_list", "pq_m", "pq_dsub", "pq_ncode",
        "max_seq_len", "page_size", "max_pages_per_seq", "n_sink", "n_local")] + [
        ("budget_ppm", ctypes.c_uint32), ("k_max", ctypes.c_int32), ("sm_scale", ctypes.c_float),
        ("dtype", ctypes.c_int32), ("exact_set_multiple", ctypes.c_int32),
        ("variant", ctypes.c_int32), ("table_precision", ctypes.c_int32),
        ("indexed_lens", ctypes.c_void_p)]


class Index(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "centroids", "codebooks", "codes", "list_ids", "key_norms", "list_vmeans", "list_counts")]


class IndexRW(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "centroids", "codebooks", "codes", "list_ids", "key_norms", "list_vmeans", "list_counts")]


class IndexOut(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "centroids", "codebooks", "codes", "list_ids", "key_norms", "list_vmeans", "list_counts")]


class PagedKV(ctypes.Structure):
    _fields_ = [("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
                ("stride_page", ctypes.c_int64), ("stride_token", ctypes.c_int64),
                ("stride_head", ctypes.c_int64), ("block_table", ctypes.c_void_p)]


_lib_handle = None


def lib() -> ctypes.CDLL:
    """The loaded shared library.  Raises if it has not been built."""
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(LIB_PATH):
            raise PqhsaError(f"loading {LIB_PATH} (build it with "
                             "`python -m paper_2609_33746_b200.build`)", ERR_CUDA)
        L = ctypes.CDLL(LIB_PATH)
        P, V, Z, I = ctypes.POINTER(Params), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        PI, PK = ctypes.POINTER(Index), ctypes.POINTER(PagedKV)
        sig = {
            "pqhsa_heads_per_group": (I, [P]),
            "pqhsa_num_partials": (I, [P]),
            "pqhsa_buffer_elems": (Z, [P, I]),
            "pqhsa_workspace_bytes": (Z, [P]),
            "pqhsa_build_lut": (I, [P, V, PI, V, V, V]),
            "pqhsa_scan": (I, [P, PI, V, V, V, V, V, V, Z, V]),
            "pqhsa_select": (I, [P, V, V, V, V, V, V, Z, V]),
            "pqhsa_rescore": (I, [P, PI, V, V, V, V, V, V, V, V, Z, V]),
            "pqhsa_hybrid_attend": (I, [P, V, PK, PI, V, V, V, V, V, V, V, V, V, Z, V]),
            "pqhsa_decode": (I, [P, V, PI, PK, V, V, V, Z, V]),
            "pqhsa_decode_events": (I, [P, V, PI, PK, V, V, V, Z, V, ctypes.POINTER(V)]),
            "pqhsa_decode_host": (I, [P, V, V, PI, PK, V, V, V, V, Z, V]),
            "pqhsa_last_device_status": (I, [P, V, V]),
            "pqhsa_decode_buffer_offset": (Z, [P, I]),
            "pqhsa_decode_launch_count": (I, [P]),
            "pqhsa_status_string": (ctypes.c_char_p, [I]),
            "pqhsa_select_static": (I, [P, V, V, V, V, V, V]),
            "pqhsa_select_static_bytes": (Z, [P]),
            "pqhsa_select_static_capacity": (Z, []),
            "pqhsa_dense_decode": (I, [P, V, PK, V, V, V, Z, V]),
            "pqhsa_dense_workspace_bytes": (Z, [P]),
            "pqhsa_gather_probe": (I, [P, PK, V, V, V, V, V]),
            "pqhsa_index_update": (I, [P, ctypes.POINTER(IndexRW), PK, V, V, I, V]),
            "pqhsa_index_build_workspace_bytes": (Z, [P]),
            "pqhsa_index_build": (I, [P, PK, V, V, V, I, I, ctypes.POINTER(IndexOut), V, Z, V]),
            "pqhsa_debug_build": (I, []),
            "pqhsa_debug_predicate": (I, [I, ctypes.c_longlong, ctypes.c_longlong, ctypes.c_longlong]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib_handle = L
    return _lib_handle


def status_string(status: int) -> str:
    try:
        return lib().pqhsa_status_string(int(status)).decode()
    except PqhsaError:
        return "library not loaded"


def _check(fn: str, status: int) -> None:
    if status != OK:
        raise PqhsaError(fn, status)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_params(*, batch, n_q_heads, n_kv_heads, n_list, pq_m, max_seq_len, max_pages_per_seq,
                budget_ppm, dtype, head_dim=128, pq_ncode=256, page_size=16, n_sink=0, n_local=0,
                k_max=None, sm_scale=None, exact_set_multiple=0, variant="B",
                indexed_lens=None, fp16_tables=False) -> Params:
    """`indexed_lens`: device int32 tensor [batch] or None; the caller keeps it alive.
    `fp16_tables`: False, True (fp16 tables in the scan) or "rescore" (fp16 tables and the fp32
    re-score of the top-k's threshold zone)."""
    if k_max is None:
        k_max = max(1, (max_seq_len * budget_ppm + 999_999) // 1_000_000)
        if exact_set_multiple > 1:
            k_max = min(max_seq_len, k_max + exact_set_multiple - 1)
    if sm_scale is None:
        sm_scale = 1.0 / math.sqrt(head_dim)
    code = {"fp16": F16, "bf16": BF16, torch.float16: F16, torch.bfloat16: BF16}[dtype]
    return Params(batch, n_q_heads, n_kv_heads, head_dim, n_list, pq_m, head_dim // pq_m, pq_ncode,
                  max_seq_len, page_size, max_pages_per_seq, n_sink, n_local, budget_ppm, k_max,
                  sm_scale, code, exact_set_multiple, VARIANTS[variant], {False: 0, True: 1, "rescore": 2}[fp16_tables],
                  _ptr(indexed_lens))


def make_index(centroids, codebooks, codes, list_ids, key_norms, list_vmeans,
               list_counts=None) -> Index:
    return Index(_ptr(centroids), _ptr(codebooks), _ptr(codes), _ptr(list_ids), _ptr(key_norms),
                 _ptr(list_vmeans), _ptr(list_counts))


def make_index_rw(centroids, codebooks, codes, list_ids, key_norms, list_vmeans,
                  list_counts) -> IndexRW:
    return IndexRW(_ptr(centroids), _ptr(codebooks), _ptr(codes), _ptr(list_ids), _ptr(key_norms),
                   _ptr(list_vmeans), _ptr(list_counts))


def make_paged_kv(k_cache, v_cache, stride_page, stride_token, stride_head, block_table) -> PagedKV:
    return PagedKV(_ptr(k_cache), _ptr(v_cache), stride_page, stride_token, stride_head,
                   _ptr(block_table))


# ------------------------------------------------------------------ host-only arithmetic
def heads_per_group(params: Params) -> int:
    r = lib().pqhsa_heads_per_group(ctypes.byref(params))
    _check("pqhsa_heads_per_group", min(r, 0))
    return r


def num_partials(params: Params) -> int:
    r = lib().pqhsa_num_partials(ctypes.byref(params))
    _check("pqhsa_num_partials", min(r, 0))
    return r


def buffer_elems(params: Params, which: int) -> int:
    return lib().pqhsa_buffer_elems(ctypes.byref(params), which)


def workspace_bytes(params: Params) -> int:
    return lib().pqhsa_workspace_bytes(ctypes.byref(params))


def decode_buffer_offset(params: Params, which: int) -> int:
    return lib().pqhsa_decode_buffer_offset(ctypes.byref(params), which)


def decode_launch_count(params: Params) -> int:
    return lib().pqhsa_decode_launch_count(ctypes.byref(params))


# ------------------------------------------------------------------ entry points
def build_lut(params, q, index: Index, lut, coarse, stream=None) -> None:
    _check("pqhsa_build_lut", lib().pqhsa_build_lut(
        ctypes.byref(params), _ptr(q), ctypes.byref(index), _ptr(lut), _ptr(coarse),
        _stream(stream)))


def scan(params, index: Index, lut, coarse, seq_lens, scores, list_partials, ws, stream=None) -> None:
    _check("pqhsa_scan", lib().pqhsa_scan(
        ctypes.byref(params), ctypes.byref(index), _ptr(lut), _ptr(coarse), _ptr(seq_lens),
        _ptr(scores), _ptr(list_partials), _ptr(ws), ws.numel() * ws.element_size(),
        _stream(stream)))


def select(params, scores, seq_lens, sel_idx, sel_count, kth_score, ws, stream=None) -> None:
    _check("pqhsa_select", lib().pqhsa_select(
        ctypes.byref(params), _ptr(scores), _ptr(seq_lens), _ptr(sel_idx), _ptr(sel_count),
        _ptr(kth_score), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def rescore(params, index, lut, coarse, scores, seq_lens, sel_idx, sel_count, kth_score, ws,
            stream=None) -> None:
    _check("pqhsa_rescore", lib().pqhsa_rescore(
        ctypes.byref(params), ctypes.byref(index), _ptr(lut), _ptr(coarse), _ptr(scores),
        _ptr(seq_lens), _ptr(sel_idx), _ptr(sel_count), _ptr(kth_score), _ptr(ws),
        ws.numel() * ws.element_size(), _stream(stream)))


def gather_probe(params, kv: PagedKV, sel_idx, sel_count, seq_lens, sink, stream=None) -> None:
    """Measurement aid: reads the selected tokens' K and V rows and computes nothing."""
    _check("pqhsa_gather_probe", lib().pqhsa_gather_probe(
        ctypes.byref(params), ctypes.byref(kv), _ptr(sel_idx), _ptr(sel_count), _ptr(seq_lens),
        _ptr(sink), _stream(stream)))


def select_static_capacity() -> int:
    return lib().pqhsa_select_static_capacity()


def select_static_bytes(params: Params) -> int:
    return lib().pqhsa_select_static_bytes(ctypes.byref(params))


def select_static(params, scores, seq_lens, sel_idx, sel_count, kth_score, stream=None) -> None:
    """pqhsa_select for callers that cannot allocate: the scratch is a fixed array inside the
    library (shared by all calls on the device; shapes beyond its capacity are rejected)."""
    _check("pqhsa_select_static", lib().pqhsa_select_static(
        ctypes.byref(params), _ptr(scores), _ptr(seq_lens), _ptr(sel_idx), _ptr(sel_count),
        _ptr(kth_score), _stream(stream)))


def hybrid_attend(params, q, kv: PagedKV, index: Index, scores, list_partials, sel_idx, sel_count,
                  seq_lens, out, lse, ws, out_f32=None, stream=None) -> None:
    _check("pqhsa_hybrid_attend", lib().pqhsa_hybrid_attend(
        ctypes.byref(params), _ptr(q), ctypes.byref(kv), ctypes.byref(index), _ptr(scores),
        _ptr(list_partials), _ptr(sel_idx), _ptr(sel_count), _ptr(seq_lens), _ptr(out), _ptr(lse),
        _ptr(out_f32), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def decode(params, q, index: Index, kv: PagedKV, seq_lens, out, ws, stream=None) -> None:
    _check("pqhsa_decode", lib().pqhsa_decode(
        ctypes.byref(params), _ptr(q), ctypes.byref(index), ctypes.byref(kv), _ptr(seq_lens),
        _ptr(out), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


N_STAGE_EVENTS = 5


def decode_events(params, q, index: Index, kv: PagedKV, seq_lens, out, ws, events, stream=None) -> None:
    """`events`: five torch.cuda.Event(enable_timing=True) that have been recorded once (so
    that their CUDA handles exist); the library re-records them around its stages."""
    arr = (ctypes.c_void_p * N_STAGE_EVENTS)(*[e.cuda_event for e in events])
    _check("pqhsa_decode_events", lib().pqhsa_decode_events(
        ctypes.byref(params), _ptr(q), ctypes.byref(index), ctypes.byref(kv), _ptr(seq_lens),
        _ptr(out), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream), arr))


def dense_workspace_bytes(params: Params) -> int:
    return lib().pqhsa_dense_workspace_bytes(ctypes.byref(params))


def dense_decode(params, q, kv: PagedKV, seq_lens, out, ws, stream=None) -> None:
    """Dense decode attention over the whole paged cache (the sweep's comparator)."""
    _check("pqhsa_dense_decode", lib().pqhsa_dense_decode(
        ctypes.byref(params), _ptr(q), ctypes.byref(kv), _ptr(seq_lens), _ptr(out), _ptr(ws),
        ws.numel() * ws.element_size(), _stream(stream)))


def decode_host(params, q_host, q_staging, index: Index, kv: PagedKV, seq_lens, out_staging,
                out_host, ws, stream=None) -> None:
    _check("pqhsa_decode_host", lib().pqhsa_decode_host(
        ctypes.byref(params), _ptr(q_host), _ptr(q_staging), ctypes.byref(index),
        ctypes.byref(kv), _ptr(seq_lens), _ptr(out_staging), _ptr(out_host), _ptr(ws),
        ws.numel() * ws.element_size(), _stream(stream)))


def index_build_workspace_bytes(params: Params) -> int:
    return lib().pqhsa_index_build_workspace_bytes(ctypes.byref(params))


def index_build(params, kv: PagedKV, seq_lens, seed_lists, seed_codes, coarse_iters: int, pq_iters: int,
                centroids, codebooks, codes, list_ids, key_norms, list_vmeans, list_counts, ws,
                stream=None) -> None:
    """Trains the index of every (sequence, KV head) at once from the paged cache; every index
    tensor is an output.  seed_lists / seed_codes: the positions whose tokens seed the centroids
    and the codewords (the method's random draws)."""
    out = IndexOut(_ptr(centroids), _ptr(codebooks), _ptr(codes), _ptr(list_ids), _ptr(key_norms),
                   _ptr(list_vmeans), _ptr(list_counts))
    _check("pqhsa_index_build", lib().pqhsa_index_build(
        ctypes.byref(params), ctypes.byref(kv), _ptr(seq_lens), _ptr(seed_lists), _ptr(seed_codes),
        int(coarse_iters), int(pq_iters), ctypes.byref(out), _ptr(ws),
        ws.numel() * ws.element_size(), _stream(stream)))


def debug_build() -> bool:
    """True if the loaded library was built with -DPQHSA_DEBUG."""
    return bool(lib().pqhsa_debug_build())


def debug_predicate(which: int, value: int, lo: int, hi: int) -> int:
    return lib().pqhsa_debug_predicate(which, value, lo, hi)


def last_device_status(params, ws, stream=None) -> int:
    return lib().pqhsa_last_device_status(ctypes.byref(params), _ptr(ws), _stream(stream))


def index_update(params, index_rw: IndexRW, kv: PagedKV, first_pos, n_new, max_new: int,
                 stream=None) -> None:
    """Encodes the tokens at positions first_pos[b] .. first_pos[b] + n_new[b] - 1 of every
    sequence into the existing lists and refreshes the list value means (in place)."""
    _check("pqhsa_index_update", lib().pqhsa_index_update(
        ctypes.byref(params), ctypes.byref(index_rw), ctypes.byref(kv), _ptr(first_pos),
        _ptr(n_new), int(max_new), _stream(stream)))
