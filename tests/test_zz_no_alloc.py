"""ap_attention_iteration_static: the attention call for users who cannot
allocate device memory.

Some integrations run attention from a place where cudaMalloc is off limits:
all device memory already belongs to a framework's caching allocator, or the
loop cannot afford cudaMalloc's device-wide synchronisation.  They have no
workspace to hand to ap_attention_iteration, so the library offers a variant
that keeps the split-K partials in a fixed 8 MiB array of its own.

This test drives that variant through the C ABI and requires the same output
as the ordinary entry point on two calls in a row (the second call sees the
scratch exactly as the first one left it, and a different batch in between
makes sure stale partials are never picked up); both are also held against
the CPU oracle, and the amount of free device memory must not move across the
calls.  It lives in the file pytest collects last, so a failure here cannot
hide the result of any other test.
"""
import numpy as np
import pytest

import paper_2604_07144_b200 as ap
from paper_2604_07144_b200 import binding as B
from paper_2604_07144_b200 import workloads as W

from harness import DeviceRun, LSE_RTOL, OUT_ATOL, oracle_pools, to_bits

pytestmark = pytest.mark.gpu


def _decode_batch(seed, ctx_lens):
    ctx = np.asarray(ctx_lens, np.int32)
    return W._assemble(f"static_ws_{seed}", W.SHAPE_8B, W.make_rng(seed), np.ones(len(ctx), np.int32), ctx, 1.3)


def _reference(run):
    """Output of the ordinary entry point (caller-provided workspace)."""
    run.append()
    run.attend()
    assert run.status() == 0
    n = run.batch.n_new
    return W.bf16_bits_to_f64(to_bits(run.out)[:n]), run.lse.cpu().numpy()[:n].astype(np.float64)


def _static(run):
    """Output of the no-allocation entry point, into poisoned output buffers."""
    run.out.fill_(float("nan"))
    run.lse.fill_(float("nan"))
    ap.attention_iteration_static(run.pool, run.plan, run.q, run.out, run.lse)
    assert run.status() == 0
    n = run.batch.n_new
    return W.bf16_bits_to_f64(to_bits(run.out)[:n]), run.lse.cpu().numpy()[:n].astype(np.float64)


def _oracle(batch):
    """The CPU oracle's result for the batch (append, then attention of every new token)."""
    import oracle
    k_ref, v_ref = oracle_pools(batch)
    return oracle.attention(k_ref, v_ref, batch.q_lens, batch.ctx_lens, batch.block_tables, batch.q)


def _same(got, ref):
    out, lse = got
    ref_out, ref_lse = ref
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    assert np.abs(out - ref_out).max() <= OUT_ATOL
    assert (np.abs(lse - ref_lse) / np.maximum(np.abs(ref_lse), 1.0)).max() <= LSE_RTOL


def test_static_workspace_matches_caller_workspace_twice_in_a_row():
    assert ap.static_workspace_bytes() == 8 << 20
    # long contexts: every (row, kv head) stream is cut, so partials and the merge are exercised
    a = DeviceRun(_decode_batch(901, [20000, 9001, 333, 64]))
    b = DeviceRun(_decode_batch(902, [15000, 12000, 17]))
    try:
        assert a.info["merge_entries"] > 0 and b.info["merge_entries"] > 0
        assert 0 < a.workspace_bytes <= ap.static_workspace_bytes()
        ref_a, ref_b = _reference(a), _reference(b)
        ora_a, ora_b = _oracle(a.batch), _oracle(b.batch)
        _same(ref_a, ora_a)
        _same(ref_b, ora_b)
        first = _static(a)                # first call on this pool
        _same(first, ref_a)
        _same(first, ora_a)
        import torch
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        second = _static(a)               # second call in a row, scratch holds the first call's partials
        _same(second, ref_a)
        _same(second, ora_a)
        other = _static(b)                # another batch over the same scratch
        _same(other, ref_b)
        _same(other, ora_b)
        _same(_static(a), ref_a)
        torch.cuda.synchronize()
        # nothing was allocated on the device by any of those calls (the comparisons above only
        # made host copies; torch's caching allocator serves them from blocks it already holds)
        assert torch.cuda.mem_get_info()[0] >= free_before
    finally:
        a.close()
        b.close()


def test_static_workspace_with_a_mixed_plan_run_side_by_side():
    # A plan whose decode part runs beside its prefill part (forced here) takes the same route
    # through the library's own scratch: the pool's second stream and events already exist, so
    # this entry point still allocates nothing.
    batch = W._assemble("static_ws_mixed", W.SHAPE_8B, W.make_rng(904), np.array([140, 1, 1, 1], np.int32),
                        np.array([500, 9000, 4000, 33], np.int32), 1.3)
    run = DeviceRun(batch, side_by_side=3)
    try:
        assert run.info["side_by_side"] == 1 and run.info["merge_entries"] > 0
        ref = _reference(run)
        ora = _oracle(batch)
        got = _static(run)
        _same(got, ref)
        _same(got, ora)
        _same(_static(run), ref)
    finally:
        run.close()


def test_static_workspace_small_plan_and_argument_checks():
    # A plan with no cut stream needs no scratch at all and must work too; bad
    # arguments are refused before anything is launched.  (A plan larger than
    # the 8 MiB array cannot be produced by the planner on 148 SMs, so the
    # size rule is checked on the plan's own number.)
    run = DeviceRun(_decode_batch(903, [40, 700]))
    try:
        assert run.workspace_bytes <= ap.static_workspace_bytes()
        run.append()
        ap.attention_iteration_static(run.pool, run.plan, run.q, run.out, run.lse)
        assert run.status() == 0
        with pytest.raises(ap.ApError) as e:       # misaligned q is refused before any launch
            ap.attention_iteration_static(run.pool, run.plan, run.q.data_ptr() + 2, run.out, run.lse)
        assert e.value.status == B.AP_ERR_INVALID_ARG
    finally:
        run.close()
