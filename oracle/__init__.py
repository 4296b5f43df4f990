"""CPU oracle for the paged-KV serving iteration (fp64, plain definition).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, ``__graft_entry__.smoke()``
and the CPU-baseline / reference legs of ``bench.py``.  The product package
never imports this module and this module never imports the product package.

``paged_attention_oracle.c`` holds the arithmetic (see its header for the
definition and the paper passages it follows); this file only compiles it with
gcc and marshals numpy arrays through ctypes.  bf16 tensors are ``uint16`` bit
patterns throughout.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "paged_attention_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib: Optional[ctypes.CDLL] = None


def compile_source(src: str, dst: str) -> str:
    """gcc -O2 -fopenmp -shared ``src`` -> ``dst`` (atomic replace)."""
    tmp = dst + f".{os.getpid()}.tmp"
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                           "-o", tmp, src, "-lm"])
    os.replace(tmp, dst)
    return dst


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        compile_source(_SRC, _LIB)
    return _LIB


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def bind(cdll: ctypes.CDLL) -> ctypes.CDLL:
    cdll.oracle_num_threads.restype = ctypes.c_int
    cdll.oracle_kv_append.restype = ctypes.c_int
    cdll.oracle_softmax_row.restype = ctypes.c_int
    cdll.oracle_copy_pages.restype = ctypes.c_int
    for name in ("oracle_attention", "oracle_attention_samples", "oracle_merge_partials",
                 "oracle_attention_range"):
        getattr(cdll, name).restype = None
    return cdll


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = bind(ctypes.CDLL(build()))
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def kv_append(k_pool: np.ndarray, v_pool: np.ndarray, q_lens, ctx_lens, block_tables,
              k_new: np.ndarray, v_new: np.ndarray) -> int:
    """In-place append into ``k_pool``/``v_pool`` ([num_pages][Hkv][16][d] uint16)."""
    assert k_pool.flags.c_contiguous and v_pool.flags.c_contiguous
    num_pages, hkv, page, d = k_pool.shape
    assert page == 16
    q_lens, ctx_lens, bt = _i32(q_lens), _i32(ctx_lens), _i32(block_tables)
    k_new, v_new = _u16(k_new), _u16(v_new)
    return int(lib().oracle_kv_append(
        _p(k_pool), _p(v_pool), ctypes.c_int(num_pages), ctypes.c_int(hkv), ctypes.c_int(d),
        ctypes.c_int(len(q_lens)), _p(q_lens), _p(ctx_lens), _p(bt), ctypes.c_int(bt.shape[1]),
        _p(k_new), _p(v_new)))


def copy_pages(k_dst: np.ndarray, v_dst: np.ndarray, k_src: np.ndarray, v_src: np.ndarray, dst_ids, src_ids) -> int:
    """In place: page ``src_ids[i]`` of the source planes -> page ``dst_ids[i]`` of the destination
    planes (all kv heads, K and V), simultaneously for all i.  The planes may be the same arrays."""
    assert k_dst.flags.c_contiguous and v_dst.flags.c_contiguous
    k_src, v_src = _u16(k_src), _u16(v_src)
    assert k_dst.shape[1:] == k_src.shape[1:] and k_dst.shape[2] == 16
    dst_ids, src_ids = _i32(dst_ids), _i32(src_ids)
    assert len(dst_ids) == len(src_ids)
    return int(lib().oracle_copy_pages(
        _p(k_dst), _p(v_dst), ctypes.c_int(k_dst.shape[0]), _p(k_src), _p(v_src), ctypes.c_int(k_src.shape[0]),
        ctypes.c_int(k_dst.shape[1]), ctypes.c_int(k_dst.shape[3]), ctypes.c_int(len(dst_ids)),
        _p(dst_ids), _p(src_ids)))


def attention(k_pool, v_pool, q_lens, ctx_lens, block_tables, q, scale: float = 0.0
              ) -> Tuple[np.ndarray, np.ndarray]:
    """All outputs of the iteration: (out [N_new][Hq][d] f64, lse [N_new][Hq] f64)."""
    k_pool, v_pool, q = _u16(k_pool), _u16(v_pool), _u16(q)
    _, hkv, _, d = k_pool.shape
    n_new, hq, _ = q.shape
    q_lens, ctx_lens, bt = _i32(q_lens), _i32(ctx_lens), _i32(block_tables)
    assert int(q_lens.sum()) == n_new
    out = np.zeros((n_new, hq, d), dtype=np.float64)
    lse = np.zeros((n_new, hq), dtype=np.float64)
    lib().oracle_attention(_p(k_pool), _p(v_pool), ctypes.c_int(hkv), ctypes.c_int(d),
                           ctypes.c_int(hq), ctypes.c_int(len(q_lens)), _p(q_lens), _p(ctx_lens),
                           _p(bt), ctypes.c_int(bt.shape[1]), _p(q), ctypes.c_double(scale),
                           _p(out), _p(lse))
    return out, lse


def attention_samples(k_pool, v_pool, q_lens, ctx_lens, block_tables, q, seq, tok, head,
                      scale: float = 0.0) -> Tuple[np.ndarray, np.ndarray]:
    """Selected outputs only: sample i = (sequence, new-token index, q head)."""
    k_pool, v_pool, q = _u16(k_pool), _u16(v_pool), _u16(q)
    _, hkv, _, d = k_pool.shape
    _, hq, _ = q.shape
    q_lens, ctx_lens, bt = _i32(q_lens), _i32(ctx_lens), _i32(block_tables)
    seq, tok, head = _i32(seq), _i32(tok), _i32(head)
    n = len(seq)
    out = np.zeros((n, d), dtype=np.float64)
    lse = np.zeros((n,), dtype=np.float64)
    lib().oracle_attention_samples(
        _p(k_pool), _p(v_pool), ctypes.c_int(hkv), ctypes.c_int(d), ctypes.c_int(hq),
        ctypes.c_int(len(q_lens)), _p(q_lens), _p(ctx_lens), _p(bt), ctypes.c_int(bt.shape[1]),
        _p(q), ctypes.c_double(scale), ctypes.c_int(n), _p(seq), _p(tok), _p(head), _p(out), _p(lse))
    return out, lse


def softmax_row(k_pool, v_pool, num_q_heads: int, bt_row, p: int, qv, head: int,
                scale: float = 0.0) -> np.ndarray:
    """Normalised softmax weights of one query over keys 0..p."""
    k_pool, v_pool, qv = _u16(k_pool), _u16(v_pool), _u16(qv)
    _, hkv, _, d = k_pool.shape
    bt_row = _i32(bt_row)
    w = np.zeros(p + 1, dtype=np.float64)
    lib().oracle_softmax_row(_p(k_pool), _p(v_pool), ctypes.c_int(hkv), ctypes.c_int(d),
                             ctypes.c_int(num_q_heads), _p(bt_row), ctypes.c_int(p), _p(qv),
                             ctypes.c_int(head), ctypes.c_double(scale), _p(w))
    return w


def attention_range(k_pool, v_pool, num_q_heads: int, bt_row, j0: int, j1: int, qv, head: int,
                    scale: float = 0.0) -> Tuple[np.ndarray, float]:
    """Attention of one query restricted to keys [j0, j1)."""
    k_pool, v_pool, qv = _u16(k_pool), _u16(v_pool), _u16(qv)
    _, hkv, _, d = k_pool.shape
    bt_row = _i32(bt_row)
    out = np.zeros(d, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    lib().oracle_attention_range(_p(k_pool), _p(v_pool), ctypes.c_int(hkv), ctypes.c_int(d),
                                 ctypes.c_int(num_q_heads), _p(bt_row), ctypes.c_int(j0),
                                 ctypes.c_int(j1), _p(qv), ctypes.c_int(head),
                                 ctypes.c_double(scale), _p(out), ctypes.byref(lse))
    return out, float(lse.value)


def merge_partials(o_parts: np.ndarray, lse_parts: np.ndarray) -> Tuple[np.ndarray, float]:
    """LSE merge of partial results over disjoint key ranges."""
    o_parts = np.ascontiguousarray(o_parts, dtype=np.float64)
    lse_parts = np.ascontiguousarray(lse_parts, dtype=np.float64)
    n, d = o_parts.shape
    o = np.zeros(d, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    lib().oracle_merge_partials(ctypes.c_int(n), ctypes.c_int(d), _p(o_parts), _p(lse_parts),
                                _p(o), ctypes.byref(lse))
    return o, float(lse.value)
