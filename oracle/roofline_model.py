"""Oracle for the paper's operator cost model restricted to the attention sublayer.

TEST INFRASTRUCTURE ONLY (like everything under ``oracle/``): the product's
``ap_plan_predict`` is compared with it; it shares no code with the library.

App. B, "Roofline-Based Serve Cost": an operation with F flops that touches A
bytes has arithmetic intensity AI = F / A; on a GPU with memory bandwidth B_g and
peak F_g it achieves pi = min(AI * B_g, F_g) (Eq. "roofline") and takes
T_op = F / pi (Eq. "roofline-2").  Written out literally, in fp64.  The paper
applies it per sublayer; here the sublayers are the three kernels of one
serving iteration (append, decode attention, prefill-chunk attention), whose
work is counted from the definition of the operation by plain loops.

Pins (tests/test_oracle_pins.py): T_op = max(F / F_g, A / B_g); both branches
meet at the ridge AI* = F_g / B_g; the intensity of long-context grouped-query
decode tends to G = Hq / Hkv flop per byte; the pair count of a causal chunk
equals an explicit enumeration.
"""
from __future__ import annotations

import numpy as np

PAGE = 16


def achieved_rate(flops: float, bytes_: float, bandwidth: float, peak: float) -> float:
    """Eq. "roofline": pi(F, A, g) = min(F / A * B_g, F_g)."""
    ai = flops / bytes_
    return min(ai * bandwidth, peak)


def t_op(flops: float, bytes_: float, bandwidth: float, peak: float) -> float:
    """Eq. "roofline-2": T_op = F / pi.  An operation without flops (a copy) takes A / B_g."""
    if bytes_ <= 0:
        return 0.0
    if flops <= 0:
        return bytes_ / bandwidth
    return flops / achieved_rate(flops, bytes_, bandwidth, peak)


def iteration_work(q_lens, ctx_lens, num_q_heads: int, num_kv_heads: int, head_dim: int) -> dict:
    """Algorithmic bytes and flops of one iteration (one attention layer), sequence by sequence:
    every attended KV token's K and V once per kv head (bf16), q read, out (bf16) and lse (fp32)
    written, one int32 block-table entry per used page (decode), new K/V read and written once;
    4 * head_dim flop per (q head, query row, key the row attends)."""
    per_kv_token = 2 * num_kv_heads * head_dim * 2
    per_row = 2 * num_q_heads * head_dim * 2 + num_q_heads * 4
    w = dict(decode_bytes=0, decode_flops=0, prefill_bytes=0, prefill_flops=0, append_bytes=0)
    for ql, cl in zip(np.asarray(q_lens).tolist(), np.asarray(ctx_lens).tolist()):
        if ql <= 0:
            continue
        w["append_bytes"] += 2 * ql * per_kv_token
        if ql == 1:
            w["decode_bytes"] += cl * per_kv_token + per_row + ((cl + PAGE - 1) // PAGE) * 4
            w["decode_flops"] += 4 * num_q_heads * head_dim * cl
        else:
            pairs = 0
            for t in range(ql):                       # row t sits at position cl - ql + t and attends keys 0..position
                pairs += cl - ql + t + 1
            w["prefill_bytes"] += cl * per_kv_token + ql * per_row
            w["prefill_flops"] += 4 * num_q_heads * head_dim * pairs
    return {k: float(v) for k, v in w.items()}


def iteration_times_us(work: dict, hbm_gbs: float, tensor_tflops: float) -> dict:
    b, f = hbm_gbs * 1e9, tensor_tflops * 1e12
    return {"roofline_decode_us": 1e6 * t_op(work["decode_flops"], work["decode_bytes"], b, f),
            "roofline_prefill_us": 1e6 * t_op(work["prefill_flops"], work["prefill_bytes"], b, f),
            "roofline_append_us": 1e6 * t_op(0.0, work["append_bytes"], b, f)}
