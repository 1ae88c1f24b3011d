"""Python binding of the C-ABI library declared in include/daf.h.

Argument marshalling only: every function here has the name and the argument
order of its C counterpart, takes torch tensors (or None) where the C function
takes pointers, and returns the C status.  No step of the method is computed
in Python.  There is no fallback: if libdaf_b200.so is missing or cannot be
loaded, the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdaf_b200.so")

DAF_OK = 0
DAF_ERR_INVALID_ARG = -1
DAF_ERR_UNSUPPORTED = -2
DAF_ERR_ALIGNMENT = -3
DAF_ERR_WORKSPACE = -4
DAF_ERR_CUDA = -5
DAF_ERR_TIMEOUT = -6
DAF_ERR_BOUNDS = -7

EXPORTS = [
    "daf_num_important", "daf_workspace_bytes", "daf_workspace_init", "daf_select", "daf_important_attn",
    "daf_qd_attn", "daf_fuse", "daf_full_causal_attn", "daf_layer", "daf_layer_host_arena_bytes",
    "daf_layer_host", "daf_layer_host_begin", "daf_layer_host_end", "daf_poll_status", "daf_strerror", "daf_last_cuda_error", "daf_launch_count",
    "daf_qd_attn_static", "daf_qd_attn_static_max_bytes", "daf_deviation_scores", "daf_blend_attn",
    "daf_imp_qd_attn", "daf_selftest_bounded_wait", "daf_qd_attn_static_poll_status",
    "daf_imp_qd_attn_launches", "daf_select_from_kv", "daf_expand_fp8_cache", "daf_layer_fp8", "daf_check_indices", "daf_select_topk",
]


class daf_params(ctypes.Structure):
    _fields_ = [
        ("L_d", ctypes.c_int32),
        ("L_q", ctypes.c_int32),
        ("r", ctypes.c_double),
        ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("fuse_mode", ctypes.c_int32),
        ("overwrite_doc_kv", ctypes.c_int32),
    ]


def make_params(L_d: int, L_q: int, r: float, n_q_heads: int, n_kv_heads: int, head_dim: int = 128,
                softmax_scale: float = 0.0, fuse_mode: int = 0, overwrite_doc_kv: int = 1) -> daf_params:
    return daf_params(L_d, L_q, r, n_q_heads, n_kv_heads, head_dim, softmax_scale, fuse_mode, overwrite_doc_kv)


class DafError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {daf_strerror(status)} (status {status}, cuda error {daf_last_cuda_error()})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libdaf_b200.so (built in-tree by paper_2607_21599_b200.build).  Raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_21599_b200.build` "
                "(there is no CPU or PyTorch fallback for this library)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        pp = ctypes.POINTER(daf_params)
        L.daf_num_important.restype = i32
        L.daf_num_important.argtypes = [i32, ctypes.c_double]
        L.daf_workspace_bytes.restype = sz
        L.daf_workspace_bytes.argtypes = [pp]
        L.daf_workspace_init.restype = ctypes.c_int
        L.daf_workspace_init.argtypes = [vp, sz, vp]
        L.daf_select.restype = ctypes.c_int
        L.daf_select.argtypes = [pp, vp, i32, vp] + [vp] * 3 + [vp] * 2 + [vp] * 4 + [vp, sz, vp]
        L.daf_select_from_kv.restype = ctypes.c_int
        L.daf_select_from_kv.argtypes = [pp, i32, vp, vp, vp, vp] + [vp] * 3 + [vp] * 2 + [vp] * 4 + [vp] + [vp, sz, vp]
        L.daf_important_attn.restype = ctypes.c_int
        L.daf_important_attn.argtypes = [pp, i32, vp, vp, vp, vp, i64, vp, vp, vp, sz, vp]
        L.daf_qd_attn.restype = ctypes.c_int
        L.daf_qd_attn.argtypes = [pp, vp, vp, vp, vp, i64, vp, vp, vp, sz, vp]
        L.daf_qd_attn_static.restype = ctypes.c_int
        L.daf_qd_attn_static.argtypes = [pp, vp, vp, vp, vp, i64, vp, vp, vp]
        L.daf_qd_attn_static_max_bytes.restype = sz
        L.daf_qd_attn_static_max_bytes.argtypes = []
        L.daf_qd_attn_static_poll_status.restype = ctypes.c_int
        L.daf_qd_attn_static_poll_status.argtypes = [vp]
        L.daf_imp_qd_attn.restype = ctypes.c_int
        L.daf_imp_qd_attn.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.daf_imp_qd_attn_launches.restype = ctypes.c_int
        L.daf_imp_qd_attn_launches.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, i32]
        L.daf_blend_attn.restype = ctypes.c_int
        L.daf_blend_attn.argtypes = [pp, i32, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
        L.daf_deviation_scores.restype = ctypes.c_int
        L.daf_deviation_scores.argtypes = [pp, vp, vp, vp, vp, vp, vp]
        L.daf_fuse.restype = ctypes.c_int
        L.daf_fuse.argtypes = [pp, i32, vp, vp, vp, vp, vp, vp]
        L.daf_full_causal_attn.restype = ctypes.c_int
        L.daf_full_causal_attn.argtypes = [pp, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.daf_layer.restype = ctypes.c_int
        L.daf_layer.argtypes = [pp, vp, i32, vp] + [vp] * 3 + [vp] * 2 + [vp] * 4 + [vp, vp] + [vp, sz, vp]
        L.daf_layer_fp8.restype = ctypes.c_int
        L.daf_layer_fp8.argtypes = [pp, vp, i32, vp] + [vp] * 3 + [vp] * 4 + [vp] * 2 + [vp] * 4 + [vp, vp] + [vp, sz, vp]
        L.daf_expand_fp8_cache.restype = ctypes.c_int
        L.daf_expand_fp8_cache.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
        L.daf_layer_host_arena_bytes.restype = sz
        L.daf_layer_host_arena_bytes.argtypes = [pp]
        L.daf_layer_host.restype = ctypes.c_int
        L.daf_layer_host.argtypes = [pp, vp, i32, vp] + [vp] * 3 + [vp, vp, i32] + [vp, vp] + [vp, sz, vp]
        L.daf_layer_host_begin.restype = ctypes.c_int
        L.daf_layer_host_begin.argtypes = [pp, vp, i32, vp] + [vp] * 3 + [vp, vp, i32] + [vp, vp] + [vp, sz, vp]
        L.daf_layer_host_end.restype = ctypes.c_int
        L.daf_layer_host_end.argtypes = [pp, vp, sz, vp]
        L.daf_select_topk.restype = ctypes.c_int
        L.daf_select_topk.argtypes = [pp, vp, i32, vp, vp, sz, vp]
        L.daf_check_indices.restype = ctypes.c_int
        L.daf_check_indices.argtypes = [pp, i32, vp, vp, sz, vp]
        L.daf_poll_status.restype = ctypes.c_int
        L.daf_poll_status.argtypes = [vp, vp]
        L.daf_selftest_bounded_wait.restype = ctypes.c_int
        L.daf_selftest_bounded_wait.argtypes = [vp, ctypes.c_size_t, ctypes.c_int32, vp]
        L.daf_strerror.restype = ctypes.c_char_p
        L.daf_strerror.argtypes = [ctypes.c_int]
        L.daf_last_cuda_error.restype = ctypes.c_int
        L.daf_last_cuda_error.argtypes = []
        L.daf_launch_count.restype = i64
        L.daf_launch_count.argtypes = []
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensors passed to the DAF library must be contiguous")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        if not torch.cuda.is_available():
            return None
        stream = torch.cuda.current_stream()
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


def _nbytes(t: Optional[torch.Tensor]) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def daf_strerror(status: int) -> str:
    return lib().daf_strerror(int(status)).decode()


def daf_last_cuda_error() -> int:
    return int(lib().daf_last_cuda_error())


def daf_launch_count() -> int:
    return int(lib().daf_launch_count())


def daf_num_important(L_d: int, r: float) -> int:
    return int(lib().daf_num_important(int(L_d), float(r)))


def daf_workspace_bytes(p: daf_params) -> int:
    return int(lib().daf_workspace_bytes(ctypes.byref(p)))


def daf_workspace_init(workspace: torch.Tensor, stream=None) -> int:
    return lib().daf_workspace_init(_ptr(workspace), _nbytes(workspace), _stream(stream))


def alloc_workspace(p: daf_params, device="cuda") -> torch.Tensor:
    """A zeroed device buffer of daf_workspace_bytes(p) bytes (torch owns the memory)."""
    n = daf_workspace_bytes(p)
    if n == 0:
        raise DafError(DAF_ERR_INVALID_ARG, "daf_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def daf_select(p, scores, n_sig, idx_in, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack, v_pack,
               workspace, stream=None) -> int:
    return lib().daf_select(ctypes.byref(p), _ptr(scores), int(n_sig), _ptr(idx_in), _ptr(q_fresh), _ptr(k_fresh),
                            _ptr(v_fresh), _ptr(kv_k), _ptr(kv_v), _ptr(idx_out), _ptr(q_pack), _ptr(k_pack),
                            _ptr(v_pack), _ptr(workspace), _nbytes(workspace), _stream(stream))


def _ptr_array(tensors):
    """A host array of device pointers (one per signal layer)."""
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = _ptr(t)
    return arr


def daf_select_from_kv(p, sig_k_fresh, sig_v_fresh, sig_k_cached, sig_v_cached, q_fresh, k_fresh, v_fresh, kv_k, kv_v,
                       idx_out, q_pack, k_pack, v_pack, signal_sum_out, workspace, stream=None) -> int:
    """sig_*: lists of n_sig device tensors (the signal layers' fresh and offline K/V)."""
    n_sig = len(sig_k_fresh)
    arrays = [_ptr_array(x) for x in (sig_k_fresh, sig_v_fresh, sig_k_cached, sig_v_cached)]
    return lib().daf_select_from_kv(ctypes.byref(p), n_sig, *arrays, _ptr(q_fresh), _ptr(k_fresh), _ptr(v_fresh),
                                    _ptr(kv_k), _ptr(kv_v), _ptr(idx_out), _ptr(q_pack), _ptr(k_pack), _ptr(v_pack),
                                    _ptr(signal_sum_out), _ptr(workspace), _nbytes(workspace), _stream(stream))


def daf_important_attn(p, k, q_pack, k_pack, v_pack, out, out_row_stride_bytes, dst_rows, lse, workspace,
                       stream=None, out_offset_bytes: int = 0) -> int:
    o = None if out is None else out.data_ptr() + out_offset_bytes
    return lib().daf_important_attn(ctypes.byref(p), int(k), _ptr(q_pack), _ptr(k_pack), _ptr(v_pack), o,
                                    int(out_row_stride_bytes), _ptr(dst_rows), _ptr(lse), _ptr(workspace),
                                    _nbytes(workspace), _stream(stream))


def daf_qd_attn(p, q_question, kv_k, kv_v, out, out_row_stride_bytes, dst_rows, lse, workspace, stream=None,
                out_offset_bytes: int = 0) -> int:
    o = None if out is None else out.data_ptr() + out_offset_bytes
    return lib().daf_qd_attn(ctypes.byref(p), _ptr(q_question), _ptr(kv_k), _ptr(kv_v), o,
                             int(out_row_stride_bytes), _ptr(dst_rows), _ptr(lse), _ptr(workspace),
                             _nbytes(workspace), _stream(stream))


def daf_qd_attn_static(p, q_question, kv_k, kv_v, out, out_row_stride_bytes, dst_rows, lse, stream=None) -> int:
    """Question-document attention without a workspace argument: the scratch is a fixed
    array inside the library, for callers that cannot hand over (or allocate) device memory.
    Calls on one device share that array, so they must not overlap on the GPU."""
    return lib().daf_qd_attn_static(ctypes.byref(p), _ptr(q_question), _ptr(kv_k), _ptr(kv_v), _ptr(out),
                                    int(out_row_stride_bytes), _ptr(dst_rows), _ptr(lse), _stream(stream))


def daf_qd_attn_static_max_bytes() -> int:
    return int(lib().daf_qd_attn_static_max_bytes())


def daf_qd_attn_static_poll_status(stream=None) -> int:
    return lib().daf_qd_attn_static_poll_status(_stream(stream))


def daf_imp_qd_attn(p, q_pack, q_fresh, k_pack, v_pack, q_question, kv_k, kv_v, idx, hidden, workspace, stream=None) -> int:
    return lib().daf_imp_qd_attn(ctypes.byref(p), _ptr(q_pack), _ptr(q_fresh), _ptr(k_pack), _ptr(v_pack), _ptr(q_question),
                                 _ptr(kv_k), _ptr(kv_v), _ptr(idx), _ptr(hidden), _ptr(workspace), _nbytes(workspace),
                                 _stream(stream))


def daf_imp_qd_attn_launches(p, q_pack, q_fresh, k_pack, v_pack, q_question, kv_k, kv_v, idx, hidden, workspace, launches,
                             stream=None) -> int:
    return lib().daf_imp_qd_attn_launches(ctypes.byref(p), _ptr(q_pack), _ptr(q_fresh), _ptr(k_pack), _ptr(v_pack),
                                          _ptr(q_question), _ptr(kv_k), _ptr(kv_v), _ptr(idx), _ptr(hidden), _ptr(workspace),
                                          _nbytes(workspace), _stream(stream), int(launches))


def daf_blend_attn(p, n_rows, q_rows, kv_k, kv_v, row_pos, out, out_row_stride_bytes, lse, workspace, stream=None) -> int:
    return lib().daf_blend_attn(ctypes.byref(p), int(n_rows), _ptr(q_rows), _ptr(kv_k), _ptr(kv_v), _ptr(row_pos),
                                _ptr(out), int(out_row_stride_bytes), _ptr(lse), _ptr(workspace), _nbytes(workspace),
                                _stream(stream))


def daf_deviation_scores(p, k_fresh, v_fresh, k_cached, v_cached, scores_row, stream=None) -> int:
    return lib().daf_deviation_scores(ctypes.byref(p), _ptr(k_fresh), _ptr(v_fresh), _ptr(k_cached), _ptr(v_cached),
                                      _ptr(scores_row), _stream(stream))


def daf_fuse(p, k, idx, o_imp, o_q, hidden, row_pos_out, stream=None) -> int:
    return lib().daf_fuse(ctypes.byref(p), int(k), _ptr(idx), _ptr(o_imp), _ptr(o_q), _ptr(hidden),
                          _ptr(row_pos_out), _stream(stream))


def daf_full_causal_attn(p, n_tokens, q, k, v, out, lse, workspace, stream=None) -> int:
    return lib().daf_full_causal_attn(ctypes.byref(p), int(n_tokens), _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                      _ptr(lse), _ptr(workspace), _nbytes(workspace), _stream(stream))


def daf_layer(p, scores, n_sig, idx_in, q_fresh, k_fresh, v_fresh, kv_k, kv_v, idx_out, q_pack, k_pack, v_pack,
              hidden, row_pos_out, workspace, stream=None) -> int:
    return lib().daf_layer(ctypes.byref(p), _ptr(scores), int(n_sig), _ptr(idx_in), _ptr(q_fresh), _ptr(k_fresh),
                           _ptr(v_fresh), _ptr(kv_k), _ptr(kv_v), _ptr(idx_out), _ptr(q_pack), _ptr(k_pack),
                           _ptr(v_pack), _ptr(hidden), _ptr(row_pos_out), _ptr(workspace), _nbytes(workspace),
                           _stream(stream))


def daf_layer_fp8(p, scores, n_sig, idx_in, q_fresh, k_fresh, v_fresh, k_cached_fp8, v_cached_fp8, k_scale, v_scale, kv_k, kv_v,
                  idx_out, q_pack, k_pack, v_pack, hidden, row_pos_out, workspace, stream=None) -> int:
    return lib().daf_layer_fp8(ctypes.byref(p), _ptr(scores), int(n_sig), _ptr(idx_in), _ptr(q_fresh), _ptr(k_fresh),
                               _ptr(v_fresh), _ptr(k_cached_fp8), _ptr(v_cached_fp8), _ptr(k_scale), _ptr(v_scale),
                               _ptr(kv_k), _ptr(kv_v), _ptr(idx_out), _ptr(q_pack), _ptr(k_pack), _ptr(v_pack), _ptr(hidden),
                               _ptr(row_pos_out), _ptr(workspace), _nbytes(workspace), _stream(stream))


def daf_expand_fp8_cache(p, k_cached_fp8, v_cached_fp8, k_scale, v_scale, kv_k, kv_v, stream=None) -> int:
    return lib().daf_expand_fp8_cache(ctypes.byref(p), _ptr(k_cached_fp8), _ptr(v_cached_fp8), _ptr(k_scale), _ptr(v_scale),
                                      _ptr(kv_k), _ptr(kv_v), _stream(stream))


def daf_layer_host_arena_bytes(p: daf_params) -> int:
    return int(lib().daf_layer_host_arena_bytes(ctypes.byref(p)))


def daf_layer_host(p, h_scores, n_sig, h_idx_in, h_q_fresh, h_k_fresh, h_v_fresh, h_kv_k, h_kv_v, copy_back_kv,
                   h_hidden, h_idx_out, arena, stream=None) -> int:
    """Host tensors in, host tensors out; `arena` is a device uint8 tensor of daf_layer_host_arena_bytes(p)."""
    for t in (h_scores, h_idx_in, h_q_fresh, h_k_fresh, h_v_fresh, h_kv_k, h_kv_v, h_hidden, h_idx_out):
        if t is not None and t.is_cuda:
            raise ValueError("daf_layer_host takes host tensors")
    return lib().daf_layer_host(ctypes.byref(p), _ptr(h_scores), int(n_sig), _ptr(h_idx_in), _ptr(h_q_fresh),
                                _ptr(h_k_fresh), _ptr(h_v_fresh), _ptr(h_kv_k), _ptr(h_kv_v), int(copy_back_kv),
                                _ptr(h_hidden), _ptr(h_idx_out), _ptr(arena), _nbytes(arena), _stream(stream))


def daf_layer_host_begin(p, h_scores, n_sig, h_idx_in, h_q_fresh, h_k_fresh, h_v_fresh, h_kv_k, h_kv_v, copy_back_kv,
                         h_hidden, h_idx_out, arena, stream=None) -> int:
    """daf_layer_host without the wait at its end (pinned host tensors); finish with daf_layer_host_end."""
    for t in (h_scores, h_idx_in, h_q_fresh, h_k_fresh, h_v_fresh, h_kv_k, h_kv_v, h_hidden, h_idx_out):
        if t is not None and t.is_cuda:
            raise ValueError("daf_layer_host_begin takes host tensors")
    return lib().daf_layer_host_begin(ctypes.byref(p), _ptr(h_scores), int(n_sig), _ptr(h_idx_in), _ptr(h_q_fresh),
                                      _ptr(h_k_fresh), _ptr(h_v_fresh), _ptr(h_kv_k), _ptr(h_kv_v), int(copy_back_kv),
                                      _ptr(h_hidden), _ptr(h_idx_out), _ptr(arena), _nbytes(arena), _stream(stream))


def daf_layer_host_end(p, arena, stream=None) -> int:
    return lib().daf_layer_host_end(ctypes.byref(p), _ptr(arena), _nbytes(arena), _stream(stream))


def daf_select_topk(p, scores, n_sig, idx_out, workspace, stream=None) -> int:
    return lib().daf_select_topk(ctypes.byref(p), _ptr(scores), int(n_sig), _ptr(idx_out), _ptr(workspace), _nbytes(workspace),
                                 _stream(stream))


def daf_check_indices(p, k, idx, workspace, stream=None) -> int:
    return lib().daf_check_indices(ctypes.byref(p), int(k), _ptr(idx), _ptr(workspace), _nbytes(workspace), _stream(stream))


def daf_poll_status(workspace, stream=None) -> int:
    return lib().daf_poll_status(_ptr(workspace), _stream(stream))


def daf_selftest_bounded_wait(workspace, limit_ms: int, stream=None) -> int:
    return lib().daf_selftest_bounded_wait(_ptr(workspace), _nbytes(workspace), int(limit_ms), _stream(stream))


def check(status: int, where: str = "daf") -> None:
    if status != DAF_OK:
        raise DafError(status, where)
