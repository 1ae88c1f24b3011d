"""ctypes front end of the C oracle (oracle/daf_oracle.c).  TEST INFRASTRUCTURE ONLY.

Marshals numpy arrays into the C routines; holds no arithmetic of its own
beyond calling them in the order the method states (see `daf_layer`).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "daf_oracle.c")
_LIB = os.path.join(_HERE, "libdaf_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) into oracle/libdaf_oracle.so."""
    stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_f = ctypes.POINTER(ctypes.c_float)
        c_d = ctypes.POINTER(ctypes.c_double)
        c_i = ctypes.POINTER(ctypes.c_int32)
        i32, i64, f64 = ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        lib.daf_oracle_num_important.restype = i64
        lib.daf_oracle_num_important.argtypes = [i64, f64]
        lib.daf_oracle_aggregate.restype = None
        lib.daf_oracle_aggregate.argtypes = [c_f, i32, i32, c_f]
        lib.daf_oracle_select.restype = i32
        lib.daf_oracle_select.argtypes = [c_f, i32, i32, i32, c_i]
        lib.daf_oracle_gather_rows.restype = None
        lib.daf_oracle_gather_rows.argtypes = [c_f, c_i, i32, i64, c_f]
        lib.daf_oracle_hybrid_kv.restype = None
        lib.daf_oracle_hybrid_kv.argtypes = [c_f, c_f, c_i, i32, i32, i32, i64, i32, c_f]
        for name in ("daf_oracle_important_attn",):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [c_f, c_f, c_f, i32, i32, i32, i32, f64, c_i, i32, c_d, c_d]
        lib.daf_oracle_qd_attn.restype = None
        lib.daf_oracle_qd_attn.argtypes = [c_f, c_f, c_f, i32, i32, i32, i32, i32, f64, c_i, i32, c_d, c_d]
        lib.daf_oracle_full_causal_attn.restype = None
        lib.daf_oracle_full_causal_attn.argtypes = [c_f, c_f, c_f, i32, i32, i32, i32, f64, c_i, i32, c_d, c_d]
        lib.daf_oracle_blend_attn.restype = None
        lib.daf_oracle_blend_attn.argtypes = [c_f, c_f, c_f, c_i, i32, i32, i32, i32, i32, f64, c_i, i32, c_d, c_d]
        lib.daf_oracle_deviation_scores.restype = None
        lib.daf_oracle_deviation_scores.argtypes = [c_f, c_f, c_f, c_f, i32, i64, c_d]
        lib.daf_oracle_fuse.restype = None
        lib.daf_oracle_fuse.argtypes = [c_d, c_d, c_i, i32, i32, i32, i64, i32, c_d, c_i]
        lib.daf_oracle_e4m3_decode.restype = ctypes.c_float
        lib.daf_oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
        lib.daf_oracle_dequant_fp8.restype = None
        lib.daf_oracle_dequant_fp8.argtypes = [ctypes.POINTER(ctypes.c_uint8), c_f, i64, i32, i32, c_f]
        lib.daf_oracle_num_threads.restype = i32
        lib.daf_oracle_num_threads.argtypes = []
        _lib = lib
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.float32)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    return int(_load().daf_oracle_num_threads())


def num_important(L_d: int, r: float) -> int:
    return int(_load().daf_oracle_num_important(int(L_d), float(r)))


def aggregate(scores) -> np.ndarray:
    S = _f32(scores)
    if S.ndim == 1:
        S = S[None, :]
    out = np.empty(S.shape[1], dtype=np.float32)
    _load().daf_oracle_aggregate(_p(S, ctypes.c_float), S.shape[0], S.shape[1], _p(out, ctypes.c_float))
    return out


def select(scores, k: int) -> np.ndarray:
    S = _f32(scores)
    if S.ndim == 1:
        S = S[None, :]
    idx = np.empty(max(int(k), 0), dtype=np.int32)
    rc = _load().daf_oracle_select(_p(S, ctypes.c_float), S.shape[0], S.shape[1], int(k), _p(idx, ctypes.c_int32))
    if rc != 0:
        raise ValueError(f"daf_oracle_select rejected its arguments (rc={rc})")
    return idx


def gather_rows(src, idx) -> np.ndarray:
    src = _f32(src)
    idx = _i32(idx)
    row_elems = int(np.prod(src.shape[1:]))
    dst = np.empty((idx.shape[0],) + src.shape[1:], dtype=np.float32)
    _load().daf_oracle_gather_rows(_p(src, ctypes.c_float), _p(idx, ctypes.c_int32), idx.shape[0], row_elems,
                                   _p(dst, ctypes.c_float))
    return dst


def hybrid_kv(cached, fresh, idx, L_d: int, L_q: int, overwrite: bool = True) -> np.ndarray:
    cached = _f32(cached)
    fresh = _f32(fresh)
    idx = _i32(idx)
    assert cached.shape[0] >= L_d and fresh.shape[0] == L_d + L_q
    row_elems = int(np.prod(fresh.shape[1:]))
    out = np.empty_like(fresh)
    _load().daf_oracle_hybrid_kv(_p(cached, ctypes.c_float), _p(fresh, ctypes.c_float), _p(idx, ctypes.c_int32),
                                 idx.shape[0], int(L_d), int(L_q), row_elems, int(bool(overwrite)),
                                 _p(out, ctypes.c_float))
    return out


def _rows_arg(rows: Optional[Sequence[int]], n_all: int):
    if rows is None:
        return None, n_all
    r = _i32(rows)
    return r, int(r.shape[0])


def _attn_shapes(q, k, v):
    q, k, v = _f32(q), _f32(k), _f32(v)
    assert q.ndim == 3 and k.ndim == 3 and v.shape == k.shape
    Hq, D = q.shape[1], q.shape[2]
    Hkv = k.shape[1]
    assert k.shape[2] == D and Hq % Hkv == 0
    return q, k, v, Hq, Hkv, D


def important_attn(q_pack, k_pack, v_pack, scale: float, rows=None, return_lse: bool = False):
    q, k, v, Hq, Hkv, D = _attn_shapes(q_pack, k_pack, v_pack)
    n = q.shape[0]
    assert k.shape[0] == n
    rows_a, n_rows = _rows_arg(rows, n)
    out = np.zeros((n_rows, Hq, D), dtype=np.float64)
    lse = np.zeros((n_rows, Hq), dtype=np.float64)
    _load().daf_oracle_important_attn(_p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(v, ctypes.c_float),
                                      n, Hq, Hkv, D, float(scale), _p(rows_a, ctypes.c_int32), n_rows,
                                      _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    return (out, lse) if return_lse else out


def qd_attn(q_question, kv_k, kv_v, L_d: int, scale: float, rows=None, return_lse: bool = False):
    q, k, v, Hq, Hkv, D = _attn_shapes(q_question, kv_k, kv_v)
    L_q = q.shape[0]
    assert k.shape[0] == L_d + L_q
    rows_a, n_rows = _rows_arg(rows, L_q)
    out = np.zeros((n_rows, Hq, D), dtype=np.float64)
    lse = np.zeros((n_rows, Hq), dtype=np.float64)
    _load().daf_oracle_qd_attn(_p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(v, ctypes.c_float),
                               int(L_d), L_q, Hq, Hkv, D, float(scale), _p(rows_a, ctypes.c_int32), n_rows,
                               _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    return (out, lse) if return_lse else out


def full_causal_attn(q, k, v, scale: float, rows=None, return_lse: bool = False):
    q, k, v, Hq, Hkv, D = _attn_shapes(q, k, v)
    n = q.shape[0]
    assert k.shape[0] == n
    rows_a, n_rows = _rows_arg(rows, n)
    out = np.zeros((n_rows, Hq, D), dtype=np.float64)
    lse = np.zeros((n_rows, Hq), dtype=np.float64)
    _load().daf_oracle_full_causal_attn(_p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(v, ctypes.c_float),
                                        n, Hq, Hkv, D, float(scale), _p(rows_a, ctypes.c_int32), n_rows,
                                        _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    return (out, lse) if return_lse else out


def blend_attn(q_rows, kv_k, kv_v, row_pos, scale: float, rows=None, return_lse: bool = False):
    """Compact rows (positions row_pos, ascending) attend every key t <= row_pos[j] of kv_k / kv_v."""
    q, k, v, Hq, Hkv, D = _attn_shapes(q_rows, kv_k, kv_v)
    pos = _i32(row_pos)
    n_q = q.shape[0]
    assert pos.shape[0] == n_q and (n_q == 0 or int(pos.max()) < k.shape[0])
    rows_a, n_rows = _rows_arg(rows, n_q)
    out = np.zeros((n_rows, Hq, D), dtype=np.float64)
    lse = np.zeros((n_rows, Hq), dtype=np.float64)
    _load().daf_oracle_blend_attn(_p(q, ctypes.c_float), _p(k, ctypes.c_float), _p(v, ctypes.c_float),
                                  _p(pos, ctypes.c_int32), n_q, k.shape[0], Hq, Hkv, D, float(scale),
                                  _p(rows_a, ctypes.c_int32), n_rows, _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    return (out, lse) if return_lse else out


def deviation_scores(k_fresh, v_fresh, k_cached, v_cached, L_d: int) -> np.ndarray:
    """fp64 [L_d]: squared deviation of each document token's fresh K/V rows from its cached rows."""
    kf, vf, kc, vc = _f32(k_fresh), _f32(v_fresh), _f32(k_cached), _f32(v_cached)
    assert kf.shape[0] >= L_d and kc.shape[0] >= L_d and kf.shape[1:] == kc.shape[1:] == vf.shape[1:] == vc.shape[1:]
    row_elems = int(np.prod(kf.shape[1:]))
    out = np.zeros(L_d, dtype=np.float64)
    _load().daf_oracle_deviation_scores(_p(kf, ctypes.c_float), _p(vf, ctypes.c_float), _p(kc, ctypes.c_float),
                                        _p(vc, ctypes.c_float), int(L_d), row_elems, _p(out, ctypes.c_double))
    return out


def e4m3_decode(byte: int) -> float:
    """Value of one byte of the 8-bit floating-point format (1 sign, 4 exponent, 3 mantissa bits; no infinities)."""
    return float(_load().daf_oracle_e4m3_decode(int(byte) & 0xFF))


def dequant_fp8(cache_bytes, scale=None) -> np.ndarray:
    """uint8 [tokens, heads, D] e4m3 bytes (+ optional fp32 [heads] scales) -> fp32 [tokens, heads, D] holding
    bf16(scale * decode(byte)): the offline cache as the rest of the path sees it."""
    b = np.ascontiguousarray(cache_bytes, dtype=np.uint8)
    tokens, heads, D = b.shape
    sc = None if scale is None else _f32(scale)
    out = np.empty(b.shape, dtype=np.float32)
    _load().daf_oracle_dequant_fp8(b.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)), _p(sc, ctypes.c_float), tokens, heads, D,
                                   _p(out, ctypes.c_float))
    return out


def fuse(o_imp, o_q, idx, L_d: int, mode: int = 0, hidden: Optional[np.ndarray] = None):
    """mode 0: compact [k+L_q, ...]; mode 1: scatter into `hidden` ([L_d+L_q, ...], modified in place)."""
    o_imp = np.ascontiguousarray(o_imp, dtype=np.float64)
    o_q = np.ascontiguousarray(o_q, dtype=np.float64)
    idx = _i32(idx)
    k, L_q = o_imp.shape[0], o_q.shape[0]
    tail = o_imp.shape[1:] if k else o_q.shape[1:]
    row_elems = int(np.prod(tail))
    if mode == 0:
        hidden = np.zeros((k + L_q,) + tuple(tail), dtype=np.float64)
    else:
        assert hidden is not None and hidden.dtype == np.float64 and hidden.flags.c_contiguous
        assert hidden.shape[0] == L_d + L_q
    row_pos = np.empty(k + L_q, dtype=np.int32)
    _load().daf_oracle_fuse(_p(o_imp, ctypes.c_double), _p(o_q, ctypes.c_double), _p(idx, ctypes.c_int32), k,
                            int(L_d), L_q, row_elems, int(mode), _p(hidden, ctypes.c_double),
                            _p(row_pos, ctypes.c_int32))
    return hidden, row_pos


def daf_layer(q_fresh, k_fresh, v_fresh, k_cached, v_cached, L_d: int, L_q: int, scale: float, *,
              scores=None, idx=None, r: Optional[float] = None, overwrite: bool = True, fuse_mode: int = 0,
              hidden: Optional[np.ndarray] = None):
    """One layer of the DAF path, steps in the paper's order: select, gather,
    hybrid-cache update, important-token attention, question-document
    attention, state fusion.  Returns a dict of every intermediate."""
    q_fresh, k_fresh, v_fresh = _f32(q_fresh), _f32(k_fresh), _f32(v_fresh)
    if idx is None:
        k = num_important(L_d, r)
        idx = select(scores, k)
    idx = _i32(idx)
    q_pack = gather_rows(q_fresh, idx)
    k_pack = gather_rows(k_fresh, idx)
    v_pack = gather_rows(v_fresh, idx)
    kv_k = hybrid_kv(k_cached, k_fresh, idx, L_d, L_q, overwrite)
    kv_v = hybrid_kv(v_cached, v_fresh, idx, L_d, L_q, overwrite)
    o_imp = important_attn(q_pack, k_pack, v_pack, scale)
    o_q = qd_attn(q_fresh[L_d:], kv_k, kv_v, L_d, scale)
    fused, row_pos = fuse(o_imp, o_q, idx, L_d, fuse_mode, hidden)
    return dict(idx=idx, q_pack=q_pack, k_pack=k_pack, v_pack=v_pack, kv_k=kv_k, kv_v=kv_v,
                o_imp=o_imp, o_q=o_q, hidden=fused, row_pos=row_pos)
