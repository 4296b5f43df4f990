"""Dense brute-force attention on contiguous tensors (numpy, fp64).

TEST INFRASTRUCTURE ONLY.  A second, structurally different statement of the
same definition, used to pin ``paged_attention_oracle.c``: for each sequence it
first gathers K and V into contiguous ``[ctx][Hkv][d]`` arrays, builds the whole
``q_len x ctx`` score matrix with an explicit boolean mask matrix, applies a row
softmax and multiplies by V with a dense matmul.  It has no notion of pages
beyond the initial gather, no per-row loops and no ``p``-bounded inner loop, so
an indexing, masking or normalisation mistake in the C oracle does not repeat
here.  Also holds an independent replay of the append as a dictionary.
"""
from __future__ import annotations

from typing import Dict, Tuple

import numpy as np

PAGE = 16


def _widen(b: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def gather_contiguous(pool: np.ndarray, bt_row: np.ndarray, ctx: int) -> np.ndarray:
    """[ctx][Hkv][d] float64 view of one sequence's logical K or V."""
    npg = (ctx + PAGE - 1) // PAGE
    pages = pool[np.asarray(bt_row[:npg], dtype=np.int64)]        # [npg][Hkv][16][d]
    seq = np.transpose(pages, (0, 2, 1, 3)).reshape(npg * PAGE, pool.shape[1], pool.shape[3])
    return _widen(seq[:ctx])


def dense_attention(k_pool, v_pool, q_lens, ctx_lens, block_tables, q, scale: float = 0.0
                    ) -> Tuple[np.ndarray, np.ndarray]:
    """(out [N_new][Hq][d], lse [N_new][Hq]) by dense masked softmax(QK^T)V."""
    _, hkv, _, d = k_pool.shape
    n_new, hq, _ = q.shape
    group = hq // hkv
    if scale <= 0.0:
        scale = 1.0 / np.sqrt(float(d))
    out = np.zeros((n_new, hq, d))
    lse = np.zeros((n_new, hq))
    row = 0
    for s, (ql, ctx) in enumerate(zip(q_lens, ctx_lens)):
        ql, ctx = int(ql), int(ctx)
        if ql == 0:
            continue
        kc = gather_contiguous(k_pool, block_tables[s], ctx)      # [ctx][Hkv][d]
        vc = gather_contiguous(v_pool, block_tables[s], ctx)
        qs = _widen(q[row:row + ql])                              # [ql][Hq][d]
        pos = ctx - ql + np.arange(ql)                            # position of each query
        mask = np.arange(ctx)[None, :] <= pos[:, None]            # [ql][ctx]
        for h in range(hq):
            g = h // group
            scores = (qs[:, h, :] @ kc[:, g, :].T) * scale         # [ql][ctx]
            scores = np.where(mask, scores, -np.inf)
            m = scores.max(axis=1, keepdims=True)
            e = np.exp(scores - m)
            z = e.sum(axis=1, keepdims=True)
            out[row:row + ql, h, :] = (e / z) @ vc[:, g, :]
            lse[row:row + ql, h] = (m + np.log(z))[:, 0]
        row += ql
    return out, lse


def append_as_dict(q_lens, ctx_lens, k_new, v_new) -> Dict[Tuple[int, int, int], Tuple[np.ndarray, np.ndarray]]:
    """{(sequence, position, kv_head): (k bits, v bits)} for every appended token."""
    rec = {}
    row = 0
    for s, (ql, ctx) in enumerate(zip(q_lens, ctx_lens)):
        for t in range(int(ql)):
            for g in range(k_new.shape[1]):
                rec[(s, int(ctx) - int(ql) + t, g)] = (k_new[row, g].copy(), v_new[row, g].copy())
            row += 1
    return rec
