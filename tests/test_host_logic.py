"""Host logic of the library on a host-only pool (no GPU): page allocator,
batch validation, and coverage of the planner's work lists."""
import numpy as np
import pytest

import paper_2604_07144_b200 as ap
from paper_2604_07144_b200 import binding as B
from paper_2604_07144_b200 import workloads as W


def host_pool(num_pages=64, hkv=2, d=64):
    return ap.kv_pool_create(num_pages, hkv, d, device=-1)


def test_pool_create_rejects_bad_descriptions():
    for kw in (dict(num_pages=0, num_kv_heads=2, head_dim=64), dict(num_pages=4, num_kv_heads=0, head_dim=64)):
        with pytest.raises(ap.ApError) as e:
            ap.kv_pool_create(device=-1, **kw)
        assert e.value.status == B.AP_ERR_INVALID_ARG
    for kw in (dict(head_dim=96), dict(head_dim=64, page_size=32)):
        with pytest.raises(ap.ApError) as e:
            ap.kv_pool_create(4, 2, device=-1, **kw)
        assert e.value.status == B.AP_ERR_UNSUPPORTED


def test_allocator_all_or_nothing_and_double_free():
    pool = host_pool(10)
    a = ap.kv_pool_alloc_pages(pool, 4)
    assert list(a) == [0, 1, 2, 3] and ap.kv_pool_num_free(pool) == 6
    with pytest.raises(ap.ApError) as e:
        ap.kv_pool_alloc_pages(pool, 7)
    assert e.value.status == B.AP_ERR_OUT_OF_PAGES and ap.kv_pool_num_free(pool) == 6
    b = ap.kv_pool_alloc_pages(pool, 6)
    assert sorted(list(a) + list(b)) == list(range(10))
    ap.kv_pool_free_pages(pool, a[:2])
    for bad in ([int(a[0])], [int(a[2]), int(a[2])], [10], [-1]):
        with pytest.raises(ap.ApError) as e:
            ap.kv_pool_free_pages(pool, bad)
        assert e.value.status == B.AP_ERR_INVALID_ARG
    assert ap.kv_pool_num_free(pool) == 2
    ap.kv_pool_free_pages(pool, [int(a[2])])     # the rejected calls freed nothing
    assert sorted(ap.kv_pool_alloc_pages(pool, 3)) == sorted(int(x) for x in a[:3])
    ap.kv_pool_destroy(pool)


def test_seeded_free_list_is_a_permutation_and_deterministic():
    orders = []
    for _ in range(2):
        pool = host_pool(100)
        ap.kv_pool_seed_free_list(pool, 1234)
        orders.append(list(ap.kv_pool_alloc_pages(pool, 100)))
        ap.kv_pool_destroy(pool)
    assert orders[0] == orders[1]
    assert sorted(orders[0]) == list(range(100)) and orders[0] != list(range(100))


def test_plan_validation():
    pool = host_pool(8)
    bt = np.array([[0, 1, 2, -1]], np.int32)
    ok = ap.plan_create(pool, [1], [33], bt, 8)
    assert ap.plan_get_info(ok)["n_new"] == 1
    ap.plan_destroy(ok)
    cases = [
        (([2], [1], bt, 8), B.AP_ERR_INVALID_ARG),            # q_len > ctx_len
        (([-1], [5], bt, 8), B.AP_ERR_INVALID_ARG),
        (([1], [65], bt, 8), B.AP_ERR_INVALID_ARG),           # table too short
        (([1], [49], bt, 8), B.AP_ERR_BAD_BLOCK_TABLE),       # reaches the -1 entry
        (([1], [33], np.array([[0, 1, 8, 0]], np.int32), 8), B.AP_ERR_BAD_BLOCK_TABLE),  # page id == num_pages
        (([1], [33], bt, 7), B.AP_ERR_INVALID_ARG),           # heads not a multiple
        (([1], [33], bt, 32), B.AP_ERR_UNSUPPORTED),          # group of 16
    ]
    for args, status in cases:
        with pytest.raises(ap.ApError) as e:
            ap.plan_create(pool, *args)
        assert e.value.status == status, args
    # two sequences appending into the same slot
    bt2 = np.array([[3, -1], [3, -1]], np.int32)
    with pytest.raises(ap.ApError) as e:
        ap.plan_create(pool, [1, 1], [5, 5], bt2, 8)
    assert e.value.status == B.AP_ERR_BAD_BLOCK_TABLE
    # sharing a page for reading only is legal
    bt3 = np.array([[3, 4], [3, 5]], np.int32)
    ap.plan_destroy(ap.plan_create(pool, [1, 1], [17, 17], bt3, 8))
    # q_len 0 sequences are skipped, even with garbage tables
    p = ap.plan_create(pool, [0, 1], [40, 17], np.array([[-5, -5, -5], [3, 4, -1]], np.int32), 8)
    assert ap.plan_get_info(p)["kv_tokens"] == 17
    ap.plan_destroy(p)
    # a host-only pool cannot launch
    p = ap.plan_create(pool, [1], [33], bt, 8)
    with pytest.raises(ap.ApError) as e:
        ap.kv_append(pool, p, 0, 0)
    assert e.value.status == B.AP_ERR_CUDA
    ap.plan_destroy(p)
    ap.kv_pool_destroy(pool)


def check_plan_coverage(batch: W.Batch, side_by_side=None):
    """Every (decode row, kv head, page) appears in exactly one item (an item covers a block of
    HB = 4, 2 or 1 consecutive kv heads); merge entries and part slots are consistent; every prefill
    row/head is in one tile."""
    hq, hkv, d = batch.num_q_heads, batch.num_kv_heads, batch.head_dim
    pool = ap.kv_pool_create(batch.num_pages, hkv, d, device=-1)
    if side_by_side is not None:
        ap.kv_pool_set_side_by_side(pool, side_by_side)
    plan = ap.plan_create(pool, batch.q_lens, batch.ctx_lens, batch.block_tables, hq)
    ex = ap.plan_export(plan)
    info = ex["info"]
    rows = batch.q_indptr
    hb = info["decode_head_block"]
    # a block of kv heads per item when decode is confined to part of the GPU, and always at head_dim 64
    assert hb == ((4 if hkv % 4 == 0 else 2 if hkv % 2 == 0 else 1) if info["side_by_side"] or d < 128 else 1)
    assert info["n_new"] == batch.n_new and info["kv_tokens"] == batch.kv_tokens
    # append destinations
    exp = []
    for s in range(batch.batch):
        for t in range(int(batch.q_lens[s])):
            p = int(batch.ctx_lens[s]) - int(batch.q_lens[s]) + t
            exp.append(int(batch.block_tables[s, p // 16]) * 16 + p % 16)
    assert list(ex["append_dst"]) == exp
    # decode coverage
    items, cta = ex["decode_items"], ex["cta_begin"]
    seen = {}
    row_to_seq = {int(rows[s]): s for s in range(batch.batch) if batch.q_lens[s] == 1}
    for q_row, kvh, bt_off, pb, pc, kv_len, slot, _ in items:
        s = row_to_seq[int(q_row)]
        assert kv_len == batch.ctx_lens[s] and pc >= 1 and 0 <= kvh < hkv and kvh % hb == 0
        npages = (int(batch.ctx_lens[s]) + 15) // 16
        assert 0 <= pb and pb + pc <= npages
        if pb + pc < npages:
            assert pc % (4 // hb) == 0              # cuts fall on stage boundaries (4 tiles = 4 / HB pages)
        assert list(ex["bt_flat"][bt_off:bt_off + npages]) == list(batch.block_tables[s, :npages])
        for pg in range(pb, pb + pc):
            for head in range(int(kvh), int(kvh) + hb):
                assert (s, head, pg) not in seen
                seen[(s, head, pg)] = int(slot)
    want = {(s, g, pg) for s in row_to_seq.values() for g in range(hkv)
            for pg in range((int(batch.ctx_lens[s]) + 15) // 16)}
    assert set(seen) == want
    if len(items):
        assert cta[0] == 0 and cta[-1] == len(items) and (np.diff(cta) > 0).all()
        assert len(cta) - 1 == info["decode_ctas"] <= 148
        cost = [int(items[a:b, 4].sum()) * hb for a, b in zip(cta[:-1], cta[1:])]      # in (page, kv head) tiles
        if sum(cost) >= 148 * 64:                   # enough work to balance
            assert max(cost) <= 1.15 * (sum(cost) / len(cost)) + 8
    # merge entries
    slots = sorted(int(x) for x in items[:, 6] if x >= 0) if len(items) else []
    assert slots == list(range(len(slots)))
    covered = []
    for q_row, kvh, pb, pc in ex["merge_entries"]:
        assert pc >= 2
        its = items[(items[:, 0] == q_row) & (items[:, 1] == kvh)]
        assert sorted(int(x) for x in its[:, 6]) == list(range(pb, pb + pc))
        covered += list(range(pb, pb + pc))
    assert sorted(covered) == slots
    single = items[items[:, 6] < 0] if len(items) else items
    for it in single:
        assert it[3] == 0 and it[4] == (int(it[5]) + 15) // 16
    # prefill coverage
    seen_rows = set()
    for q_row0, nrows, qh, kvh, bt_off, pos0, ctx, qh_b in ex["prefill_tiles"]:
        assert 1 <= nrows <= 128 and kvh == qh // (hq // hkv)
        heads = [int(qh)]
        if qh_b >= 0:                                   # a second head of the same kv head shares the unit
            assert qh_b == qh + 1 and qh_b // (hq // hkv) == kvh
            heads.append(int(qh_b))
        for r in range(q_row0, q_row0 + nrows):
            for h in heads:
                assert (r, h) not in seen_rows
                seen_rows.add((r, h))
        s = int(np.searchsorted(rows, q_row0, side="right") - 1)
        assert ctx == batch.ctx_lens[s] and pos0 == ctx - batch.q_lens[s] + (q_row0 - rows[s])
    want_rows = {(r, h) for s in range(batch.batch) if batch.q_lens[s] > 1
                 for r in range(int(rows[s]), int(rows[s + 1])) for h in range(hq)}
    assert seen_rows == want_rows
    ends = [int(t[5] + t[1]) for t in ex["prefill_tiles"]]
    assert ends == sorted(ends, reverse=True)        # longest first
    ap.plan_destroy(plan)
    ap.kv_pool_destroy(pool)
    return info


def test_plan_coverage_small_and_ragged():
    for seed in range(20, 30):
        check_plan_coverage(W.random_ragged(seed, batch=9, max_ctx=700, max_q=3))
    check_plan_coverage(W.config1())
    info = check_plan_coverage(W.random_ragged(5, batch=6, max_ctx=900, max_q=300))
    assert info["prefill_tiles"] > 0


def test_plan_coverage_full_size_configs():
    i2 = check_plan_coverage(W.config2(with_pool=False))
    assert i2["decode_rows"] == 64 and i2["decode_ctas"] == 148
    i3 = check_plan_coverage(W.config3(with_pool=False))
    assert i3["prefill_seqs"] == 8 and i3["decode_rows"] == 120 and i3["prefill_tiles"] == 8 * 4 * 16
    i4 = check_plan_coverage(W.config4(with_pool=False))
    assert i4["decode_ctas"] == 148 and i4["merge_entries"] > 0


def test_side_by_side_planning():
    """Mixed iterations: the planner confines decode to k CTAs (cost model or forced) and the
    work lists still cover everything; pure decode / pure prefill plans stay sequential."""
    b3 = W.config3(with_pool=False)
    auto = check_plan_coverage(b3)                               # mode 1 is the default
    assert auto["side_by_side"] == 1 and 48 <= auto["decode_ctas"] <= 96
    off = check_plan_coverage(b3, side_by_side=0)
    assert off["side_by_side"] == 0 and off["decode_ctas"] == 148
    forced = check_plan_coverage(b3, side_by_side=40)
    assert forced["side_by_side"] == 1 and forced["decode_ctas"] <= 40
    assert forced["decode_items"] >= off["decode_rows"] * 2      # two blocks of four kv heads per row
    for b in (W.config2(with_pool=False), W.config4(with_pool=False)):
        assert check_plan_coverage(b, side_by_side=64)["side_by_side"] == 0
    # a mixed batch too small to gain anything stays sequential under the cost model
    small = W.random_ragged(5, batch=6, max_ctx=900, max_q=300)
    assert check_plan_coverage(small)["side_by_side"] == 0
    pool = host_pool()
    with pytest.raises(ap.ApError):
        ap.kv_pool_set_side_by_side(pool, -1)
    ap.kv_pool_destroy(pool)


def _mixed(shape, n_prefill, n_decode, dec_hi=4096, seed=77):
    rng = W.make_rng(seed)
    prefix = rng.g.integers(0, 4097, size=n_prefill)
    dec = rng.g.integers(256, dec_hi + 1, size=n_decode)
    q_lens = np.concatenate([np.full(n_prefill, 512), np.ones(n_decode)]).astype(np.int32)
    ctx = np.concatenate([prefix + 512, dec]).astype(np.int32)
    return W._assemble("mixed", shape, rng, q_lens, ctx, with_pool=False)


def test_side_by_side_decision_at_other_shapes_and_mixes():
    """The planner's decision for mixes other than config 3, as measured on B200 (the planner's choice beat
    the sequential dispatch by 7-11 % in each side-by-side case below, and sequential was right for d = 64):
    70B shape -> a few dozen decode CTAs; a decode-heavy 8B mix -> the cap of 0.7 #SM; a prefill-heavy one ->
    a handful of CTAs; the d = 64 shape, whose small TMA requests feed an SM too slowly, stays sequential."""
    def plan_info(batch):
        pool = ap.kv_pool_create(batch.num_pages, batch.num_kv_heads, batch.head_dim, device=-1)
        plan = ap.plan_create(pool, batch.q_lens, batch.ctx_lens, batch.block_tables, batch.num_q_heads)
        info, pred = ap.plan_get_info(plan), ap.plan_predict(plan)
        ap.plan_destroy(plan)
        ap.kv_pool_destroy(pool)
        return info, pred
    i, p = plan_info(_mixed(W.SHAPE_70B, 8, 120))
    assert i["side_by_side"] == 1 and 30 <= i["decode_ctas"] <= 60 and i["decode_head_block"] == 4
    assert 380 <= p["model_step_us"] <= 520                     # measured 457 us
    i, p = plan_info(_mixed(W.SHAPE_8B, 2, 300))
    assert i["side_by_side"] == 1 and i["decode_ctas"] == 103
    assert 340 <= p["model_step_us"] <= 520                     # measured 402 us
    i, p = plan_info(_mixed(W.SHAPE_8B, 14, 40))
    assert i["side_by_side"] == 1 and 12 <= i["decode_ctas"] <= 30
    assert 290 <= p["model_step_us"] <= 400                     # measured 342 us
    i, _ = plan_info(_mixed(W.SHAPE_S1, 8, 400, dec_hi=8192))
    assert i["side_by_side"] == 0 and i["decode_head_block"] == 2


def test_copy_pages_validation_on_host_pools():
    """ap_kv_copy_pages checks its lists on the host before anything is queued."""
    a, b = host_pool(20), host_pool(30)
    ap.kv_copy_pages(b, a, [], [])
    ap.kv_copy_pages(b, a, [29, 0, 7], [19, 19, 3])            # one source to several destinations is fine
    ap.kv_copy_pages(a, a, [5, 6], [5, 1])                     # a page onto itself is skipped
    for dst, src, status in (([30], [0], B.AP_ERR_BAD_BLOCK_TABLE), ([0], [20], B.AP_ERR_BAD_BLOCK_TABLE),
                             ([-1], [0], B.AP_ERR_BAD_BLOCK_TABLE), ([4, 4], [1, 2], B.AP_ERR_INVALID_ARG)):
        with pytest.raises(ap.ApError) as e:
            ap.kv_copy_pages(b, a, dst, src)
        assert e.value.status == status
    # inside one pool a destination may not be another pair's source (the copies run in parallel)
    with pytest.raises(ap.ApError) as e:
        ap.kv_copy_pages(a, a, [1, 2], [0, 1])
    assert e.value.status == B.AP_ERR_INVALID_ARG
    other_shape = ap.kv_pool_create(20, 4, 64, device=-1)
    with pytest.raises(ap.ApError) as e:
        ap.kv_copy_pages(other_shape, a, [0], [0])
    assert e.value.status == B.AP_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        ap.kv_copy_pages(b, a, [1, 2], [1])
    for p in (a, b, other_shape):
        ap.kv_pool_destroy(p)


def test_plan_predict_matches_the_cost_model_oracle():
    """ap_plan_predict: work figures equal the oracle's counts exactly, the paper-model times to rounding;
    the planner's own model is positive, additive when sequential and shorter when side by side."""
    from oracle import roofline_model as R
    batches = [W.config1(), W.config2(with_pool=False), W.config3(with_pool=False), W.config4(with_pool=False),
               W.random_ragged(5, batch=6, max_ctx=900, max_q=300), W.random_ragged(21, batch=9, max_ctx=700, max_q=3)]
    for b in batches:
        pool = ap.kv_pool_create(b.num_pages, b.num_kv_heads, b.head_dim, device=-1)
        plan = ap.plan_create(pool, b.q_lens, b.ctx_lens, b.block_tables, b.num_q_heads)
        for bw, tf in ((0.0, 0.0), (3350.0, 989.0)):
            got = ap.plan_predict(plan, bw, tf)
            work = R.iteration_work(b.q_lens, b.ctx_lens, b.num_q_heads, b.num_kv_heads, b.head_dim)
            for k, v in work.items():
                assert got[k] == v, (b.name, k)
            ref = R.iteration_times_us(work, bw or 6448.0, tf or 1642.0)
            for k, v in ref.items():
                assert np.isclose(got[k], v, rtol=1e-12, atol=0.0), (b.name, k)
        info = ap.plan_get_info(plan)
        assert (got["model_decode_us"] > 0) == (info["decode_rows"] > 0)
        assert (got["model_prefill_us"] > 0) == (info["prefill_seqs"] > 0)
        if not info["side_by_side"]:
            assert got["model_step_us"] >= got["model_decode_us"] + got["model_prefill_us"]
        ap.plan_destroy(plan)
        ap.kv_pool_destroy(pool)
    # config 3: side by side is predicted (and planned) to be shorter than decode then prefill
    b = W.config3(with_pool=False)
    steps = {}
    for mode in (0, 1):
        pool = ap.kv_pool_create(b.num_pages, b.num_kv_heads, b.head_dim, device=-1)
        ap.kv_pool_set_side_by_side(pool, mode)
        plan = ap.plan_create(pool, b.q_lens, b.ctx_lens, b.block_tables, b.num_q_heads)
        steps[mode] = ap.plan_predict(plan)["model_step_us"]
        ap.plan_destroy(plan)
        ap.kv_pool_destroy(pool)
    assert steps[1] < 0.95 * steps[0]


def test_execution_model_matches_its_oracle_and_the_papers_table():
    """paper_2604_07144_b200.execution_model against the oracle's term-by-term sum on random interval
    lists, and against the paper's printed artifact-feedback rows."""
    from oracle import execution_model as E
    from paper_2604_07144_b200 import execution_model as M
    from test_oracle_pins import _artifact_rows, _split
    rng = np.random.default_rng(2)
    for _ in range(50):
        n = int(rng.integers(1, 8))
        ivs = [M.Interval(*rng.random(4).tolist()) for _ in range(n)]
        ref = E.t_total([i.t_sched for i in ivs], [i.t_stale for i in ivs], [i.t_reconfig for i in ivs],
                        [i.t_serve for i in ivs])
        assert np.isclose(M.total_time(ivs), ref, rtol=1e-12)
    for name, n, stale, reconf, serve, total in _artifact_rows():
        serve_parts = _split(rng, serve, n + 1)
        ivs = [M.Interval(t_serve=serve_parts[0])] + [
            M.Interval(t_sched=5.0, t_stale=a, t_reconfig=b, t_serve=c)
            for a, b, c in zip(_split(rng, stale, n), _split(rng, reconf, n), serve_parts[1:])]
        fb = M.artifact_feedback(ivs)
        assert fb["N"] == n and abs(fb["T_total"] - total) < 0.05
        assert abs(fb["sum_t_stale"] - stale) < 1e-9 and abs(fb["sum_t_reconfig"] - reconf) < 1e-9
        assert abs(fb["sum_t_serve"] - serve) < 1e-9
    # measured iterations grouped into intervals
    times = [0.1] * 10
    ivs = M.intervals_from_iterations(times, reschedule_at=[4, 7], t_sched_first=0.5, t_stale=[1.0, 2.0],
                                      t_reconfig=[3.0])
    assert [round(i.t_serve, 6) for i in ivs] == [0.4, 0.3, 0.3]
    assert np.isclose(M.total_time(ivs), 0.5 + 1.0 + 1.0 + 2.0 + 3.0)
    assert M.artifact_feedback(M.intervals_from_iterations(times))["N"] == 0
    with pytest.raises(ValueError):
        M.intervals_from_iterations(times, reschedule_at=[5, 3])


def test_shared_pages_may_be_read_but_not_appended_to_twice():
    """Block tables may name the same page in several sequences as long as no slot is written by two of
    them: a shared read-only prefix plans fine, two sequences appending into the same slot are refused."""
    b = W._assemble("shared", W.SHAPE_S1, W.make_rng(71), np.array([1, 1], np.int32), np.array([100, 100], np.int32), 1.3,
                    with_pool=False)
    pool = ap.kv_pool_create(b.num_pages, b.num_kv_heads, b.head_dim, device=-1)
    bt = b.block_tables.copy()
    bt[1, :6] = bt[0, :6]                                   # positions 0..95 shared, position 99 in own pages
    ap.plan_destroy(ap.plan_create(pool, b.q_lens, b.ctx_lens, bt, b.num_q_heads))
    bt[1, 6] = bt[0, 6]                                     # now both append position 99 into the same slot
    with pytest.raises(ap.ApError) as e:
        ap.plan_create(pool, b.q_lens, b.ctx_lens, bt, b.num_q_heads)
    assert e.value.status == B.AP_ERR_BAD_BLOCK_TABLE
    ap.kv_pool_destroy(pool)


def test_empty_batch_plans_to_nothing():
    pool = host_pool()
    p = ap.plan_create(pool, [], [], np.zeros((0, 1), np.int32), 8)
    info = ap.plan_get_info(p)
    assert info["n_new"] == 0 and info["launches_attention"] == 0 and ap.plan_workspace_bytes(p) == 0
    ap.plan_destroy(p)
    ap.kv_pool_destroy(pool)


def test_trace_generator_invariants():
    reqs = W.trace_arrivals(iterations=120)
    peak = W.trace_peak_pages(reqs, iterations=120)
    alloc = W.FreeListAllocator(int(1.25 * peak) + 1)
    owner = {}
    done_tokens = 0
    for it in W.fcfs_trace(reqs, alloc.alloc, alloc.free, iterations=120):
        assert int(it.q_lens.sum()) <= 8192
        assert (it.q_lens >= 1).all() and (it.q_lens <= 512).all() and (it.ctx_lens >= it.q_lens).all()
        pf = it.q_lens > 1
        assert not pf[np.argmax(~pf):].any() if (~pf).any() else True     # prefill rows first
        used = set()
        for i, rid in enumerate(it.rids):
            n = (int(it.ctx_lens[i]) + 15) // 16
            pages = [int(p) for p in it.block_tables[i, :n]]
            assert all(p >= 0 for p in pages) and not (used & set(pages))
            used |= set(pages)
            assert owner.setdefault(int(rid), pages[:len(owner.get(int(rid), []))] or pages)[:1] == pages[:1]
        done_tokens += int(it.q_lens.sum())
    assert done_tokens > 0 and alloc.peak_used <= peak
