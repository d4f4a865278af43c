"""Thin Python binding of libwar.so: argument marshalling only.

Every function here has the name and the meaning of the C entry point it wraps (see include/war.h); tensors are
torch CUDA tensors used as device buffers, and the current torch stream is the stream of the call.  Nothing is
computed on the Python side, and there is no fallback: if the library has not been built, importing this module
raises."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwar.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_17299_b200.build` "
                      "(there is no CPU or PyTorch fallback for this library)")
_lib = C.CDLL(LIB_PATH)

WAR_OK = 0
STATUS_NAMES = {0: "WAR_OK", 1: "WAR_ERR_INVALID_ARG", 2: "WAR_ERR_OOM", 3: "WAR_ERR_CAPACITY", 4: "WAR_ERR_CUDA",
                5: "WAR_ERR_TIMEOUT", 6: "WAR_ERR_UNSUPPORTED", 7: "WAR_ERR_BAD_TREE", 8: "WAR_ERR_BAD_PAGE"}

EXPORTS = ["war_index_build", "war_index_append", "war_index_append_async", "war_index_evict", "war_index_export_bytes", "war_index_export",
           "war_index_import", "war_index_info", "war_index_destroy", "war_draft", "war_draft_scored_workspace_bytes", "war_draft_scored", "war_draft_local", "war_draft_pick",
           "war_verify_attn_workspace_bytes", "war_verify_attn", "war_verify_attn_noalloc", "war_accept", "war_commit", "war_device_status",
           "war_selftest_bounded_wait",
           "war_status_string"]


class WarError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} returned {STATUS_NAMES.get(code, code)}: {status_string(code)}")


class IndexInfo(C.Structure):
    _fields_ = [("M", C.c_int64), ("capacity_tokens", C.c_int64), ("T", C.c_int32), ("vocab", C.c_int32),
                ("max_depth", C.c_int32), ("reserved", C.c_int32), ("d_corpus", C.c_void_p), ("d_sa", C.c_void_p),
                ("d_lcp", C.c_void_p), ("d_bucket", C.c_void_p)]


class DraftParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("P", C.c_int32), ("N", C.c_int32), ("topk", C.c_int32), ("min_match", C.c_int32),
                ("spec_batch_limit", C.c_int32), ("spec_factor_num", C.c_int32), ("spec_factor_den", C.c_int32),
                ("min_prob_num", C.c_int32), ("min_prob_den", C.c_int32)]


class AttnParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("D", C.c_int32),
                ("page_size", C.c_int32), ("max_pages_per_req", C.c_int32), ("kernel", C.c_int32),
                ("num_pages", C.c_int64), ("scale", C.c_float), ("reserved", C.c_int32),
                ("k_strides", C.c_int64 * 4), ("v_strides", C.c_int64 * 4)]


_lib.war_status_string.restype = C.c_char_p
_lib.war_status_string.argtypes = [C.c_int]
_lib.war_index_build.restype = C.c_int
_lib.war_index_build.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                 C.POINTER(C.c_void_p)]
_lib.war_index_append.restype = C.c_int
_lib.war_index_append.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
_lib.war_index_append_async.restype = C.c_int
_lib.war_index_append_async.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
_lib.war_index_evict.restype = C.c_int
_lib.war_index_evict.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
_lib.war_index_export_bytes.restype = C.c_size_t
_lib.war_index_export_bytes.argtypes = [C.c_void_p]
_lib.war_index_export.restype = C.c_int
_lib.war_index_export.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.war_index_import.restype = C.c_int
_lib.war_index_import.argtypes = [C.c_void_p, C.c_size_t, C.c_int64, C.c_void_p, C.POINTER(C.c_void_p)]
_lib.war_index_info.restype = C.c_int
_lib.war_index_info.argtypes = [C.c_void_p, C.POINTER(IndexInfo)]
_lib.war_index_destroy.restype = C.c_int
_lib.war_index_destroy.argtypes = [C.c_void_p]
_lib.war_draft.restype = C.c_int
_lib.war_draft.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(DraftParams)] + [C.c_void_p] * 6
_lib.war_verify_attn_workspace_bytes.restype = C.c_size_t
_lib.war_draft_scored_workspace_bytes.restype = C.c_size_t
_lib.war_draft_scored_workspace_bytes.argtypes = [C.POINTER(DraftParams), C.c_int32]
_lib.war_draft_scored.restype = C.c_int
_lib.war_draft_scored.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(DraftParams), C.c_int32] + [C.c_void_p] * 8
_lib.war_draft_local.restype = C.c_int
_lib.war_draft_local.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(DraftParams)] + [C.c_void_p] * 6
_lib.war_draft_pick.restype = C.c_int
_lib.war_draft_pick.argtypes = [C.c_int32, C.c_int32] + [C.c_void_p] * 17
_lib.war_verify_attn_workspace_bytes.argtypes = [C.POINTER(AttnParams)]
_lib.war_verify_attn.restype = C.c_int
_lib.war_verify_attn.argtypes = [C.c_void_p] * 7 + [C.POINTER(AttnParams)] + [C.c_void_p] * 4
_lib.war_verify_attn_noalloc.restype = C.c_int
_lib.war_verify_attn_noalloc.argtypes = [C.c_void_p] * 7 + [C.POINTER(AttnParams)] + [C.c_void_p] * 3
_lib.war_accept.restype = C.c_int
_lib.war_accept.argtypes = [C.c_void_p] * 4 + [C.c_int32] * 3 + [C.c_void_p] * 4
_lib.war_device_status.restype = C.c_int
_lib.war_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]


def status_string(code: int) -> str:
    return _lib.war_status_string(int(code)).decode()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device buffers must be contiguous CUDA tensors")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected {dtype}, got {t.dtype}")
    return t.data_ptr()


def _check(fn: str, code: int) -> None:
    if code != WAR_OK:
        raise WarError(fn, code)


class Index:
    """Owner of a war_index_t*."""

    def __init__(self, handle: int):
        self._h = C.c_void_p(handle)

    @property
    def handle(self) -> C.c_void_p:
        if not self._h:
            raise ValueError("index already destroyed")
        return self._h

    def destroy(self) -> None:
        if self._h:
            _lib.war_index_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def _offsets(h_offsets) -> np.ndarray:
    off = np.ascontiguousarray(np.asarray(h_offsets, dtype=np.int64))
    if off.ndim != 1 or len(off) < 1:
        raise ValueError("h_offsets must be int64 [T+1]")
    return off


def war_index_build(d_tokens: torch.Tensor, h_offsets, vocab: int, max_depth: int, capacity_tokens: int) -> Index:
    off = _offsets(h_offsets)
    out = C.c_void_p(None)
    code = _lib.war_index_build(_ptr(d_tokens, torch.int32), off.ctypes.data, len(off) - 1, vocab, max_depth,
                                capacity_tokens, _stream(), C.byref(out))
    _check("war_index_build", code)
    return Index(out.value)


def war_index_append(ix: Index, d_tokens: torch.Tensor, h_offsets) -> None:
    off = _offsets(h_offsets)
    _check("war_index_append", _lib.war_index_append(ix.handle, _ptr(d_tokens, torch.int32), off.ctypes.data,
                                                     len(off) - 1, _stream()))


def war_index_append_async(ix: Index, d_tokens: torch.Tensor, h_offsets) -> None:
    """Enqueues the append on the current stream and returns; keep d_tokens alive until that stream has run it."""
    off = _offsets(h_offsets)
    _check("war_index_append_async", _lib.war_index_append_async(ix.handle, _ptr(d_tokens, torch.int32), off.ctypes.data,
                                                                 len(off) - 1, _stream()))


def war_index_evict(ix: Index, n_oldest: int) -> None:
    _check("war_index_evict", _lib.war_index_evict(ix.handle, int(n_oldest), _stream()))


def war_index_export(ix: Index) -> np.ndarray:
    """The whole index as one host byte array (see war_index_import)."""
    n = int(_lib.war_index_export_bytes(ix.handle))
    buf = np.empty(n, dtype=np.uint8)
    _check("war_index_export", _lib.war_index_export(ix.handle, buf.ctypes.data, n, _stream()))
    return buf


def war_index_import(buf: np.ndarray, capacity_tokens: int) -> Index:
    buf = np.ascontiguousarray(buf, dtype=np.uint8)
    h = C.c_void_p()
    _check("war_index_import", _lib.war_index_import(buf.ctypes.data, buf.nbytes, int(capacity_tokens), _stream(), C.byref(h)))
    return Index(h.value)


def war_index_info(ix: Index) -> IndexInfo:
    info = IndexInfo()
    _check("war_index_info", _lib.war_index_info(ix.handle, C.byref(info)))
    return info


def war_index_destroy(ix: Index) -> None:
    ix.destroy()


def war_draft(ix: Index, d_tail: torch.Tensor, d_tail_len: torch.Tensor, N: int, topk: int, min_match: int,
              d_match_len: torch.Tensor, d_num_nodes: torch.Tensor, d_ids: torch.Tensor, d_parent: torch.Tensor,
              d_count: Optional[torch.Tensor], spec_batch_limit: int = 0, spec_factor=(0, 1), min_prob=(0, 1)) -> None:
    """spec_factor / min_prob are (numerator, denominator) pairs; a numerator of 0 switches the rule off."""
    B, P = d_tail.shape
    p = DraftParams(B, P, N, topk, min_match, spec_batch_limit, spec_factor[0], spec_factor[1], min_prob[0], min_prob[1])
    code = _lib.war_draft(ix.handle, _ptr(d_tail, torch.int32), _ptr(d_tail_len, torch.int32), C.byref(p),
                          _ptr(d_match_len, torch.int32), _ptr(d_num_nodes, torch.int32), _ptr(d_ids, torch.int32),
                          _ptr(d_parent, torch.int32), _ptr(d_count, torch.int32), _stream())
    _check("war_draft", code)


def war_draft_scored_workspace_bytes(B: int, P: int, N: int, topk: int, n_lengths: int) -> int:
    p = DraftParams(B, P, N, topk, 1, 0, 0, 1, 0, 1)
    return int(_lib.war_draft_scored_workspace_bytes(C.byref(p), n_lengths))


def war_draft_scored(ix: Index, d_tail: torch.Tensor, d_tail_len: torch.Tensor, N: int, topk: int, min_match: int,
                     n_lengths: int, d_workspace: torch.Tensor, d_match_len: torch.Tensor, d_used_len: torch.Tensor,
                     d_num_nodes: torch.Tensor, d_ids: torch.Tensor, d_parent: torch.Tensor, d_count: Optional[torch.Tensor],
                     spec_batch_limit: int = 0, spec_factor=(0, 1), min_prob=(0, 1)) -> None:
    """war_draft from the best-scoring of n_lengths suffix lengths; d_workspace is a uint8 CUDA tensor of at least
    war_draft_scored_workspace_bytes(...) bytes."""
    B, P = d_tail.shape
    p = DraftParams(B, P, N, topk, min_match, spec_batch_limit, spec_factor[0], spec_factor[1], min_prob[0], min_prob[1])
    need = int(_lib.war_draft_scored_workspace_bytes(C.byref(p), n_lengths))
    if need == 0 or d_workspace.dtype != torch.uint8 or not d_workspace.is_cuda or d_workspace.numel() < need:
        raise ValueError("workspace must be a uint8 CUDA tensor of war_draft_scored_workspace_bytes bytes")
    code = _lib.war_draft_scored(ix.handle, _ptr(d_tail, torch.int32), _ptr(d_tail_len, torch.int32), C.byref(p), n_lengths,
                                 d_workspace.data_ptr(), _ptr(d_match_len, torch.int32), _ptr(d_used_len, torch.int32),
                                 _ptr(d_num_nodes, torch.int32), _ptr(d_ids, torch.int32), _ptr(d_parent, torch.int32),
                                 _ptr(d_count, torch.int32), _stream())
    _check("war_draft_scored", code)


def war_draft_local(d_ctx: torch.Tensor, d_ctx_off: torch.Tensor, d_tail_len: torch.Tensor, P: int, N: int, topk: int,
                    min_match: int, d_match_len: torch.Tensor, d_num_nodes: torch.Tensor, d_ids: torch.Tensor,
                    d_parent: torch.Tensor, d_count: Optional[torch.Tensor], spec_batch_limit: int = 0, spec_factor=(0, 1),
                    min_prob=(0, 1)) -> None:
    """d_ctx: int32 tokens of all contexts back to back; d_ctx_off: int64 [B+1] bounds, both on the device."""
    B = d_ctx_off.numel() - 1
    p = DraftParams(B, P, N, topk, min_match, spec_batch_limit, spec_factor[0], spec_factor[1], min_prob[0], min_prob[1])
    code = _lib.war_draft_local(_ptr(d_ctx, torch.int32), _ptr(d_ctx_off, torch.int64), _ptr(d_tail_len, torch.int32),
                                C.byref(p), _ptr(d_match_len, torch.int32), _ptr(d_num_nodes, torch.int32),
                                _ptr(d_ids, torch.int32), _ptr(d_parent, torch.int32), _ptr(d_count, torch.int32), _stream())
    _check("war_draft_local", code)


def war_draft_pick(a, b, d_source: torch.Tensor, d_match_len: torch.Tensor, d_num_nodes: torch.Tensor, d_ids: torch.Tensor,
                   d_parent: torch.Tensor, d_count: Optional[torch.Tensor]) -> None:
    """a, b: (match_len, num_nodes, ids, parent, count) tensor tuples of the two trees."""
    B, N = a[2].shape
    args = [_ptr(t, torch.int32) for t in (*a, *b)]
    code = _lib.war_draft_pick(B, N, *args, _ptr(d_source, torch.int32), _ptr(d_match_len, torch.int32),
                               _ptr(d_num_nodes, torch.int32), _ptr(d_ids, torch.int32), _ptr(d_parent, torch.int32),
                               _ptr(d_count, torch.int32), _stream())
    _check("war_draft_pick", code)


def attn_params(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor, scale: float,
                kernel: int = 0) -> AttnParams:
    B, N, Hq, D = q.shape
    num_pages, Hkv, pg, _ = k_pool.shape
    p = AttnParams()
    p.B, p.N, p.Hq, p.Hkv, p.D, p.page_size = B, N, Hq, Hkv, D, pg
    p.max_pages_per_req = page_table.shape[1]
    p.kernel = kernel
    p.num_pages = num_pages
    p.scale = scale
    for i in range(4):
        p.k_strides[i] = k_pool.stride(i)
        p.v_strides[i] = v_pool.stride(i)
    return p


def war_verify_attn_workspace_bytes(params: AttnParams) -> int:
    return int(_lib.war_verify_attn_workspace_bytes(C.byref(params)))


def war_verify_attn(d_q: torch.Tensor, d_kpool: torch.Tensor, d_vpool: torch.Tensor, d_page_table: torch.Tensor,
                    d_prefix_len: torch.Tensor, d_num_nodes: torch.Tensor, d_parent: torch.Tensor, params: AttnParams,
                    d_workspace: torch.Tensor, d_out: torch.Tensor, d_lse: Optional[torch.Tensor]) -> None:
    for t in (d_kpool, d_vpool):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("pools must be bf16 CUDA tensors")
    code = _lib.war_verify_attn(_ptr(d_q, torch.bfloat16), d_kpool.data_ptr(), d_vpool.data_ptr(),
                                _ptr(d_page_table, torch.int32), _ptr(d_prefix_len, torch.int32),
                                _ptr(d_num_nodes, torch.int32), _ptr(d_parent, torch.int32), C.byref(params),
                                _ptr(d_workspace), _ptr(d_out, torch.bfloat16), _ptr(d_lse, torch.float32), _stream())
    _check("war_verify_attn", code)


NOALLOC_MAX_BYTES = 64 * 1024 * 1024


def war_verify_attn_noalloc(d_q: torch.Tensor, d_kpool: torch.Tensor, d_vpool: torch.Tensor, d_page_table: torch.Tensor,
                            d_prefix_len: torch.Tensor, d_num_nodes: torch.Tensor, d_parent: torch.Tensor,
                            params: AttnParams, d_out: torch.Tensor, d_lse: Optional[torch.Tensor]) -> None:
    """war_verify_attn without a workspace argument, for callers that cannot allocate device memory: the scratch
    is a fixed array inside the library (NOALLOC_MAX_BYTES).  Calls on one device share it, so keep them in stream
    order; make the first call on a device outside any stream capture."""
    for t in (d_kpool, d_vpool):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("pools must be bf16 CUDA tensors")
    code = _lib.war_verify_attn_noalloc(_ptr(d_q, torch.bfloat16), d_kpool.data_ptr(), d_vpool.data_ptr(),
                                        _ptr(d_page_table, torch.int32), _ptr(d_prefix_len, torch.int32),
                                        _ptr(d_num_nodes, torch.int32), _ptr(d_parent, torch.int32), C.byref(params),
                                        _ptr(d_out, torch.bfloat16), _ptr(d_lse, torch.float32), _stream())
    _check("war_verify_attn_noalloc", code)


def war_accept(d_ids: torch.Tensor, d_parent: torch.Tensor, d_num_nodes: torch.Tensor, d_target_ids: torch.Tensor,
               target_mode: int, d_accept_len: torch.Tensor, d_accept_path: torch.Tensor, d_bonus: torch.Tensor) -> None:
    B, N = d_ids.shape
    code = _lib.war_accept(_ptr(d_ids, torch.int32), _ptr(d_parent, torch.int32), _ptr(d_num_nodes, torch.int32),
                           _ptr(d_target_ids, torch.int32), B, N, target_mode, _ptr(d_accept_len, torch.int32),
                           _ptr(d_accept_path, torch.int32), _ptr(d_bonus, torch.int32), _stream())
    _check("war_accept", code)


class CommitParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("P", C.c_int32), ("Hkv", C.c_int32), ("D", C.c_int32),
                ("page_size", C.c_int32), ("max_pages_per_req", C.c_int32), ("reserved", C.c_int32),
                ("num_pages", C.c_int64), ("k_strides", C.c_int64 * 4), ("v_strides", C.c_int64 * 4)]


_lib.war_commit.restype = C.c_int
_lib.war_commit.argtypes = [C.c_void_p] * 7 + [C.POINTER(CommitParams)] + [C.c_void_p] * 4


def war_commit(d_ids: torch.Tensor, d_accept_len: torch.Tensor, d_accept_path: torch.Tensor, d_bonus: torch.Tensor,
               k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor, d_prefix_len: torch.Tensor,
               d_tail: torch.Tensor, d_tail_len: torch.Tensor) -> None:
    """Pools are [pages, Hkv, page_size, D] bf16 views (any strides the library accepts); updated in place."""
    B, N = d_ids.shape
    p = CommitParams()
    p.B, p.N, p.P = B, N, d_tail.shape[1]
    p.Hkv, p.D, p.page_size = k_pool.shape[1], k_pool.shape[3], k_pool.shape[2]
    p.max_pages_per_req, p.num_pages = page_table.shape[1], k_pool.shape[0]
    for i in range(4):
        p.k_strides[i] = k_pool.stride(i)
        p.v_strides[i] = v_pool.stride(i)
    code = _lib.war_commit(_ptr(d_ids, torch.int32), _ptr(d_accept_len, torch.int32), _ptr(d_accept_path, torch.int32),
                           _ptr(d_bonus, torch.int32), C.c_void_p(k_pool.data_ptr()), C.c_void_p(v_pool.data_ptr()),
                           _ptr(page_table, torch.int32), C.byref(p), _ptr(d_prefix_len, torch.int32),
                           _ptr(d_tail, torch.int32), _ptr(d_tail_len, torch.int32), _stream())
    _check("war_commit", code)


_lib.war_selftest_bounded_wait.restype = C.c_int
_lib.war_selftest_bounded_wait.argtypes = [C.c_int32, C.c_void_p, C.c_void_p]


def war_selftest_bounded_wait(budget_us: int, d_result: torch.Tensor) -> None:
    """d_result: int64 [4] CUDA tensor; see include/war.h."""
    _check("war_selftest_bounded_wait", _lib.war_selftest_bounded_wait(int(budget_us), _ptr(d_result, torch.int64), _stream()))


def war_device_status() -> int:
    v = C.c_int32(0)
    _check("war_device_status", _lib.war_device_status(_stream(), C.byref(v)))
    return int(v.value)


def new_workspace(params: AttnParams, device) -> torch.Tensor:
    """A device buffer of the size war_verify_attn asks for (torch's allocator returns 512-byte aligned blocks)."""
    n = war_verify_attn_workspace_bytes(params)
    if n == 0:
        raise WarError("war_verify_attn_workspace_bytes", 6)
    return torch.empty(n, dtype=torch.uint8, device=device)
