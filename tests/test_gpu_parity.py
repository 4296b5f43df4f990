"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Append and page indexing bit-exact; attention
output within 1e-2 max abs (bf16 out, N(0,1) inputs); lse within 1e-3 relative
(denominator max(|lse|, 1))."""
import numpy as np
import pytest

import paper_2604_07144_b200 as ap
from paper_2604_07144_b200 import binding as B
from paper_2604_07144_b200 import workloads as W

from harness import DeviceRun, check_batch_full, check_batch_sampled, to_bits

pytestmark = pytest.mark.gpu


def decode_batch(seed, shape, ctx_lens, pool_factor=1.3):
    ctx = np.asarray(ctx_lens, np.int32)
    return W._assemble(f"decode_{seed}", shape, W.make_rng(seed), np.ones(len(ctx), np.int32), ctx, pool_factor)


def test_config1_single_decode_both_readings():
    for post in (True, False):
        b = W.config1(post_append=post)
        err, lerr = check_batch_full(b)
        print(f"config1 post_append={post}: out err {err:.2e} lse err {lerr:.2e}")


def test_decode_page_boundaries_and_tiny_contexts():
    # first slot of a page, last slot, one token, exactly one stage, one stage + 1 ...
    ctx = [1, 2, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 1000]
    check_batch_full(decode_batch(101, W.SHAPE_S1, ctx))
    check_batch_full(decode_batch(102, W.SHAPE_8B, ctx))


@pytest.mark.parametrize("shape", [(8, 8, 64), (8, 4, 64), (6, 2, 128), (32, 8, 128), (64, 8, 128), (5, 1, 128)],
                         ids=lambda s: f"Hq{s[0]}_Hkv{s[1]}_d{s[2]}")
def test_decode_head_ratios(shape):
    rng = np.random.default_rng(7)
    ctx = rng.integers(1, 700, size=9)
    check_batch_full(decode_batch(103, shape, ctx))


def test_decode_split_and_merge_long_context():
    # few long sequences: every (row, kv head) stream is cut across many CTAs
    b = decode_batch(104, W.SHAPE_8B, [20000, 9001, 333])
    run = DeviceRun(b)
    assert run.info["merge_entries"] > 0 and run.info["decode_ctas"] > 100
    run.close()
    check_batch_full(b)


def test_decode_explicit_scale():
    check_batch_full(decode_batch(105, W.SHAPE_S1, [40, 300]), scale=0.05)


def test_mixed_ragged_small():
    for seed in (201, 202, 203):
        check_batch_full(W.random_ragged(seed, shape=W.SHAPE_S1, batch=7, max_ctx=400, max_q=40))
    check_batch_full(W.random_ragged(204, shape=W.SHAPE_8B, batch=5, max_ctx=900, max_q=300))


@pytest.mark.parametrize("mode,single", [(0, True), (3, True), (20, True), (3, False), (20, False)],
                         ids=["sequential", "k3_one_launch", "k20_one_launch", "k3_two_streams", "k20_two_streams"])
def test_mixed_iteration_side_by_side_modes(mode, single):
    """Decode confined to a few CTAs next to the prefill units (forced k) in one launch -- the decode
    CTAs are the first blocks of the grid, every later block a prefill unit -- or as two kernels on
    the caller's stream and the pool's second stream, and the sequential dispatch (mode 0): same
    results against the oracle, twice in a row on the same pool."""
    import oracle
    from harness import compare_outputs, oracle_pools
    batch = W._assemble("mixed_side_by_side", W.SHAPE_8B, W.make_rng(31),
                        np.array([200, 1, 1, 1, 130, 1], np.int32),
                        np.array([700, 333, 1500, 16, 130, 2049], np.int32), 1.3)
    run = DeviceRun(batch, side_by_side=mode, single_launch=single)
    try:
        assert run.info["side_by_side"] == (1 if mode else 0)
        assert run.info["launches_attention"] == (1 if mode and single else 2)
        if mode:
            assert run.info["decode_ctas"] <= mode
        run.append()
        k_ref, v_ref = oracle_pools(batch)
        ref_out, ref_lse = oracle.attention(k_ref, v_ref, batch.q_lens, batch.ctx_lens, batch.block_tables, batch.q)
        for _ in range(2):
            run.out.fill_(float("nan"))
            run.lse.fill_(float("nan"))
            run.attend()
            assert run.status() == 0
            compare_outputs(to_bits(run.out)[:batch.n_new], run.lse.cpu().numpy()[:batch.n_new], ref_out, ref_lse,
                            f"mode {mode}")
        assert np.array_equal(to_bits(run.k_pool), k_ref) and np.array_equal(to_bits(run.v_pool), v_ref)
    finally:
        run.close()


@pytest.mark.parametrize("mode,single", [(0, True), (3, True), (3, False)], ids=["sequential", "one_launch", "two_streams"])
def test_iteration_is_capturable_in_a_cuda_graph(mode, single):
    """Append + attention issue no host synchronisation and take every buffer by address, so the
    per-layer sequence of a model (here: the same layer four times) can be captured once into a CUDA
    graph and replayed; with decode beside prefill the fork / join through the pool's second stream
    is captured too.  The replayed result is checked against the oracle."""
    import torch
    import oracle
    from harness import compare_outputs, oracle_pools
    batch = W._assemble("graph_mixed", W.SHAPE_8B, W.make_rng(41), np.array([150, 1, 1, 1], np.int32),
                        np.array([400, 90, 1300, 17], np.int32), 1.3)
    run = DeviceRun(batch, side_by_side=mode, single_launch=single)
    try:
        assert run.info["side_by_side"] == (1 if mode else 0)
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            run.append()                       # warm-up outside the capture (first-launch attribute set-up)
            run.attend()
        stream.synchronize()
        assert run.status() == 0
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(4):
                run.append()
                run.attend()
        k_ref, v_ref = oracle_pools(batch)
        ref_out, ref_lse = oracle.attention(k_ref, v_ref, batch.q_lens, batch.ctx_lens, batch.block_tables, batch.q)
        for _ in range(2):
            run.out.fill_(float("nan"))
            run.lse.fill_(float("nan"))
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            assert run.status() == 0
            compare_outputs(to_bits(run.out)[:batch.n_new], run.lse.cpu().numpy()[:batch.n_new], ref_out, ref_lse,
                            f"graph replay, mode {mode}")
        assert np.array_equal(to_bits(run.k_pool), k_ref) and np.array_equal(to_bits(run.v_pool), v_ref)
        del graph
    finally:
        run.close()


def _used_pages(batch):
    return sorted({int(batch.block_tables[s, i]) for s in range(batch.batch)
                   for i in range((int(batch.ctx_lens[s]) + 15) // 16)})


@pytest.mark.parametrize("shape", [W.SHAPE_8B, (8, 2, 64)], ids=["8B", "S1"])
def test_page_copy_migration_and_copy_on_write(shape):
    """ap_kv_copy_pages against the oracle, bit for bit: every used page of a batch moves to a second
    pool (canaries elsewhere stay, the source is untouched), attention through the remapped block
    tables still matches the oracle; then pages are duplicated inside one pool."""
    import torch
    import oracle
    from harness import compare_outputs, to_dev
    batch = W._assemble("migrate", shape, W.make_rng(51), np.array([1, 70, 1, 1, 3], np.int32),
                        np.array([300, 200, 17, 1025, 64], np.int32), 1.3)
    run = DeviceRun(batch)
    try:
        run.append()
        used = _used_pages(batch)
        rng = np.random.default_rng(3)
        n_dst = batch.num_pages + 9
        new_of = dict(zip(used, rng.permutation(n_dst)[:len(used)].tolist()))
        src = np.array(used, np.int32)
        dst = np.array([new_of[p] for p in used], np.int32)
        canary = np.full((n_dst,) + batch.k_pool.shape[1:], 0x7FC1, np.uint16)
        k2, v2 = to_dev(canary), to_dev(canary)
        pool2 = ap.kv_pool_create(n_dst, batch.num_kv_heads, batch.head_dim, k2, v2)
        ap.kv_copy_pages(pool2, run.pool, dst, src)
        # the oracle's version of the same move
        k_src, v_src = to_bits(run.k_pool), to_bits(run.v_pool)
        k_ref, v_ref = canary.copy(), canary.copy()
        assert oracle.copy_pages(k_ref, v_ref, k_src, v_src, dst, src) == 0
        assert ap.last_device_status(pool2) == 0
        assert np.array_equal(to_bits(k2), k_ref) and np.array_equal(to_bits(v2), v_ref)
        assert np.array_equal(to_bits(run.k_pool), k_src) and np.array_equal(to_bits(run.v_pool), v_src)
        # attention on the migrated pages (no new tokens are appended again: same contexts, remapped tables)
        bt2 = batch.block_tables.copy()
        for s in range(batch.batch):
            for i in range((int(batch.ctx_lens[s]) + 15) // 16):
                bt2[s, i] = new_of[int(batch.block_tables[s, i])]
        plan2 = ap.plan_create(pool2, batch.q_lens, batch.ctx_lens, bt2, batch.num_q_heads)
        ws = torch.empty(max(ap.plan_workspace_bytes(plan2), 256), dtype=torch.uint8, device="cuda:0")
        ap.attention_iteration(pool2, plan2, run.q, run.out, run.lse, ws, ap.plan_workspace_bytes(plan2))
        assert ap.last_device_status(pool2) == 0
        ref_out, ref_lse = oracle.attention(k_ref, v_ref, batch.q_lens, batch.ctx_lens, bt2, batch.q)
        compare_outputs(to_bits(run.out)[:batch.n_new], run.lse.cpu().numpy()[:batch.n_new], ref_out, ref_lse, "migrated")
        ap.plan_destroy(plan2)
        # copy-on-write inside the second pool: duplicate some pages into free ones
        free = np.setdiff1d(np.arange(n_dst), dst).astype(np.int32)[:5]
        cow_src = dst[:len(free)]
        ap.kv_copy_pages(pool2, pool2, free, cow_src)
        assert oracle.copy_pages(k_ref, v_ref, k_ref, v_ref, free, cow_src) == 0
        assert np.array_equal(to_bits(k2), k_ref) and np.array_equal(to_bits(v2), v_ref)
        # a refused call queues nothing
        with pytest.raises(ap.ApError):
            ap.kv_copy_pages(pool2, pool2, [int(free[0]), int(free[1])], [int(cow_src[0]), int(free[0])])
        assert np.array_equal(to_bits(k2), k_ref)
        ap.kv_pool_destroy(pool2)
    finally:
        run.close()


def test_page_copy_full_size_config2():
    """All 8 k used pages of config 2 (534 MB) in one call, compared bit for bit with the oracle."""
    import oracle
    from harness import to_dev
    batch = W.config2()
    used = np.array(_used_pages(batch), np.int32)
    k1, v1 = to_dev(batch.k_pool), to_dev(batch.v_pool)
    pool1 = ap.kv_pool_create(batch.num_pages, batch.num_kv_heads, batch.head_dim, k1, v1)
    n_dst = len(used) + 3
    dst = np.random.default_rng(5).permutation(n_dst)[:len(used)].astype(np.int32)
    canary = np.full((n_dst,) + batch.k_pool.shape[1:], 0x7FC1, np.uint16)
    k2, v2 = to_dev(canary), to_dev(canary)
    pool2 = ap.kv_pool_create(n_dst, batch.num_kv_heads, batch.head_dim, k2, v2)
    ap.kv_copy_pages(pool2, pool1, dst, used)
    assert ap.last_device_status(pool2) == 0
    k_ref, v_ref = canary.copy(), canary.copy()
    assert oracle.copy_pages(k_ref, v_ref, batch.k_pool, batch.v_pool, dst, used) == 0
    assert np.array_equal(to_bits(k2), k_ref) and np.array_equal(to_bits(v2), v_ref)
    ap.kv_pool_destroy(pool1)
    ap.kv_pool_destroy(pool2)


@pytest.mark.parametrize("config", [2, 3, 4])
def test_plan_predict_tracks_the_measured_step(config):
    """The planner's calibrated model (ap_plan_predict.model_step_us) stays within -25 % / +35 % of the
    measured device time of append + attention on the full-size workloads, and the paper's roofline
    time is a lower bound of the measured attention time (up to the slack explained below)."""
    import torch
    batch = {2: W.config2, 3: W.config3, 4: W.config4}[config]()
    run = DeviceRun(batch)
    try:
        pred = ap.plan_predict(run.plan)
        for _ in range(3):
            run.append(); run.attend()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 10
        e0.record()
        for _ in range(n):
            run.append(); run.attend()
        e1.record()
        torch.cuda.synchronize()
        assert run.status() == 0
        us = 1e3 * e0.elapsed_time(e1) / n
        # measured on B200: model / measured = 1.12 (config 2), 0.92 (config 3, one launch), 1.08 (config 4)
        assert 0.75 * us <= pred["model_step_us"] <= 1.35 * us, (us, pred)
        # The paper's roofline time is a lower bound in principle, but its B_g here is the bandwidth of a
        # plain device-to-device copy (6468 GB/s) and the decode kernel, which only reads, streams at up to
        # 6.97 TB/s on config 4: 1.08x that "peak".  Hence 1.2 and not 1.0.  (These workloads are all much
        # larger than the L2, so no cache effect is involved.)
        assert max(pred["roofline_decode_us"], pred["roofline_prefill_us"]) <= 1.2 * us
    finally:
        run.close()


def test_page_copy_more_pairs_than_one_grid_dimension():
    """70,000 pairs in one call (the launch is sliced at 65,535 pairs per grid): every destination page
    must hold its source page, checked with torch on the device and on a sample against the oracle."""
    import torch
    import oracle
    n, hkv, d = 70000, 2, 64
    gen = torch.Generator(device="cuda").manual_seed(7)
    k1 = torch.randint(-32768, 32767, (n, hkv, 16, d), dtype=torch.int16, device="cuda", generator=gen).view(torch.bfloat16)
    v1 = torch.randint(-32768, 32767, (n, hkv, 16, d), dtype=torch.int16, device="cuda", generator=gen).view(torch.bfloat16)
    k2, v2 = torch.zeros_like(k1), torch.zeros_like(v1)
    src_pool = ap.kv_pool_create(n, hkv, d, k1, v1)
    dst_pool = ap.kv_pool_create(n, hkv, d, k2, v2)
    rng = np.random.default_rng(9)
    dst, src = rng.permutation(n).astype(np.int32), rng.integers(0, n, size=n).astype(np.int32)
    ap.kv_copy_pages(dst_pool, src_pool, dst, src)
    assert ap.last_device_status(dst_pool) == 0
    di, si = torch.from_numpy(dst.astype(np.int64)).cuda(), torch.from_numpy(src.astype(np.int64)).cuda()
    assert torch.equal(k2.view(torch.int16)[di], k1.view(torch.int16)[si])
    assert torch.equal(v2.view(torch.int16)[di], v1.view(torch.int16)[si])
    # the last pairs (second slice) once more against the oracle's copy
    tail = slice(n - 300, n)
    k_ref = np.zeros((n, hkv, 16, d), np.uint16)
    v_ref = np.zeros_like(k_ref)
    assert oracle.copy_pages(k_ref, v_ref, to_bits(k1), to_bits(v1), dst[tail], src[tail]) == 0
    assert np.array_equal(to_bits(k2)[dst[tail]], k_ref[dst[tail]]) and np.array_equal(to_bits(v2)[dst[tail]], v_ref[dst[tail]])
    ap.kv_pool_destroy(src_pool)
    ap.kv_pool_destroy(dst_pool)


def _shared_prefix_batch():
    """Three sequences reading the same six prefix pages (96 tokens) through their block tables: two
    decode rows and a prefill chunk; every sequence appends into pages of its own."""
    b = W._assemble("shared_prefix", W.SHAPE_8B, W.make_rng(61), np.array([1, 1, 40], np.int32),
                    np.array([300, 180, 96 + 40], np.int32), 1.3)
    b.block_tables[1, :6] = b.block_tables[0, :6]
    b.block_tables[2, :6] = b.block_tables[0, :6]
    return b


def test_shared_prefix_pages_are_read_by_several_sequences():
    check_batch_full(_shared_prefix_batch())


def test_fork_a_sequence_with_copy_on_write_of_its_last_page():
    """A sequence is forked: the fork's block table names the parent's full pages and a fresh page that
    ap_kv_copy_pages fills from the parent's partly filled last page; then parent and fork each append a
    different token and attend.  Against the oracle doing the same copy, append and attention."""
    import oracle
    from harness import compare_outputs
    base = W._assemble("fork_parent", W.SHAPE_8B, W.make_rng(62), np.array([1, 1], np.int32),
                       np.array([301, 301], np.int32), 1.5)          # row 1 is only a donor of pages and tokens
    n_pages = (301 + 15) // 16
    parent = base.block_tables[0, :n_pages].copy()
    fresh = int(base.block_tables[1, 0])                           # a page the parent does not use
    fork = parent.copy()
    fork[-1] = fresh
    base.block_tables[1, :n_pages] = fork
    run = DeviceRun(base)
    try:
        k_ref, v_ref = base.k_pool.copy(), base.v_pool.copy()
        ap.kv_copy_pages(run.pool, run.pool, [fresh], [int(parent[-1])])
        assert oracle.copy_pages(k_ref, v_ref, k_ref, v_ref, [fresh], [int(parent[-1])]) == 0
        run.append()
        run.attend()
        assert run.status() == 0
        assert oracle.kv_append(k_ref, v_ref, base.q_lens, base.ctx_lens, base.block_tables, base.k_new, base.v_new) == 0
        assert np.array_equal(to_bits(run.k_pool), k_ref) and np.array_equal(to_bits(run.v_pool), v_ref)
        ref_out, ref_lse = oracle.attention(k_ref, v_ref, base.q_lens, base.ctx_lens, base.block_tables, base.q)
        compare_outputs(to_bits(run.out)[:2], run.lse.cpu().numpy()[:2], ref_out, ref_lse, "fork")
        # same history, different new token and query: the two rows must differ
        assert not np.array_equal(to_bits(run.out)[0], to_bits(run.out)[1])
    finally:
        run.close()


def test_prefill_chunk_shapes():
    # whole prompt, chunk on a prefix, ragged last tile, several tiles, page-misaligned prefix
    cases = [([128], [128]), ([1 + 128], [129]), ([200], [777]), ([300], [300]), ([37], [1000]), ([512], [4096 + 512])]
    for i, (ql, cl) in enumerate(cases):
        b = W._assemble(f"prefill_{i}", W.SHAPE_8B, W.make_rng(300 + i), np.array(ql, np.int32), np.array(cl, np.int32), 1.3)
        check_batch_full(b)


def test_decode_stream_cut_into_more_than_32_partials():
    """One sequence, one kv head, 120 k tokens: the planner cuts the single (row, kv head) stream into
    one item per SM, so the in-kernel LSE merge takes its chunked path (more partials than a warp has
    lanes).  Every output against the oracle."""
    b = decode_batch(107, (8, 1, 128), [120000], pool_factor=1.05)
    run = DeviceRun(b)
    try:
        ex = ap.plan_export(run.plan)
        assert int(ex["merge_entries"][:, 3].max()) > 32, "the plan does not reach the chunked merge"
    finally:
        run.close()
    err, lerr = check_batch_full(b)
    print(f"148-way split: out err {err:.2e} lse err {lerr:.2e}")
    # two such streams (G = 4 and G = 8 take different batch sizes in the merge's fetch loop)
    check_batch_full(decode_batch(108, (8, 2, 128), [70000], pool_factor=1.05))
    check_batch_full(decode_batch(109, (2, 1, 64), [90000], pool_factor=1.05))


def test_decode_more_items_per_cta_than_the_shared_memory_list_holds():
    """1500 short decode rows x 8 kv heads = 12 000 items, ~81 per CTA: past the 32 item descriptors a
    CTA keeps in shared memory, so the rest come from global memory.  Every output against the oracle."""
    rng = np.random.default_rng(11)
    b = decode_batch(110, W.SHAPE_8B, rng.integers(1, 49, size=1500))
    run = DeviceRun(b)
    try:
        ex = ap.plan_export(run.plan)
        assert int(np.diff(ex["cta_begin"]).max()) > 32, "no CTA holds more than 32 items"
    finally:
        run.close()
    err, lerr = check_batch_full(b)
    print(f"12000 items: out err {err:.2e} lse err {lerr:.2e}")


def _prefill_rescales(batch, scale, head=0, seq=0):
    """How often the prefill kernel's rule "rescale O when some row of a 32-row group sees its running
    maximum rise by more than 8 (log2 units) after the first step" fires for one (sequence, q head),
    worked out from the inputs in fp64 (test-side bookkeeping of which inputs reach that path)."""
    from harness import oracle_pools
    k_ref, _ = oracle_pools(batch)
    hq, hkv, d = batch.num_q_heads, batch.num_kv_heads, batch.head_dim
    g = head // (hq // hkv)
    ql, cl = int(batch.q_lens[seq]), int(batch.ctx_lens[seq])
    pages = batch.block_tables[seq, :(cl + 15) // 16]
    k = W.bf16_bits_to_f64(k_ref[pages, g]).reshape(-1, d)[:cl]
    r0 = int(batch.q_indptr[seq])
    q = W.bf16_bits_to_f64(batch.q[r0:r0 + ql, head])
    s = (q @ k.T) * scale * np.log2(np.e)
    pos = cl - ql + np.arange(ql)
    s[np.arange(cl)[None, :] > pos[:, None]] = -np.inf
    fired = 0
    for t0 in range(0, ql, 128):
        rows = s[t0:t0 + 128]
        n_steps = (int(pos[min(t0 + 127, ql - 1)]) + 1 + 127) // 128
        for w0 in range(0, rows.shape[0], 32):
            blk = rows[w0:w0 + 32]
            m_used = np.full(blk.shape[0], -np.inf)
            for j in range(n_steps):
                mx = blk[:, j * 128:(j + 1) * 128].max(axis=1)
                m_new = np.maximum(m_used, mx)
                with np.errstate(invalid="ignore"):
                    moved = (m_new - m_used) > 8.0
                if moved.any():
                    m_used = m_new
                    fired += j > 0
    return fired


@pytest.mark.parametrize("shape,scale", [((4, 2, 64), 1.0), ((4, 2, 64), 0.5), (W.SHAPE_8B, 0.5), ((6, 2, 128), 0.7)],
                         ids=["d64_scale1", "d64_scale0.5", "8B_scale0.5", "G3_scale0.7"])
def test_prefill_explicit_scale_rescales_the_accumulator(shape, scale):
    """Prefill with an explicit softmax scale large enough that row maxima keep climbing after the
    first key step, so O is rescaled in tensor memory (the kernel's rare path); against the oracle at
    the same scale, same tolerances."""
    b = W._assemble("prefill_scale", shape, W.make_rng(320), np.array([384, 1, 200], np.int32),
                    np.array([1400, 300, 200], np.int32), 1.3)
    assert _prefill_rescales(b, scale) > 0, "these inputs never move the running maximum by more than 8"
    err, lerr = check_batch_full(b, scale=scale, peaked=True)
    print(f"prefill scale {scale}: out err {err:.2e} lse err {lerr:.2e}")


def test_prefill_keys_growing_along_the_context():
    """Default scale, but K grows with the position (norm x1 ... x4 over the context), so every row's
    maximum rises step after step and the O rescale fires at the standard 1/sqrt(d)."""
    b = W._assemble("prefill_growing_k", W.SHAPE_8B, W.make_rng(321), np.array([256, 1], np.int32),
                    np.array([2304, 500], np.int32), 1.3)
    cl, ql = int(b.ctx_lens[0]), int(b.q_lens[0])
    grow = lambda j: 1.0 + 3.0 * j / cl
    for j in range(cl - ql):                           # cached keys, through the block table
        page, slot = int(b.block_tables[0, j // 16]), j % 16
        b.k_pool[page, :, slot] = W.f32_to_bf16_bits((W.bf16_bits_to_f64(b.k_pool[page, :, slot]) * grow(j)).astype(np.float32))
    for t in range(ql):                                # this iteration's keys
        b.k_new[t] = W.f32_to_bf16_bits((W.bf16_bits_to_f64(b.k_new[t]) * grow(cl - ql + t)).astype(np.float32))
    b.q[:ql] = W.f32_to_bf16_bits((W.bf16_bits_to_f64(b.q[:ql]) * 1.5).astype(np.float32))
    assert _prefill_rescales(b, 1.0 / np.sqrt(b.head_dim)) > 0
    err, lerr = check_batch_full(b, peaked=True)
    print(f"prefill growing K: out err {err:.2e} lse err {lerr:.2e}")


def test_prefill_long_prefix_and_maximum_chunk():
    """The largest prefill work the configurations allow: a chunk deep inside a long context (485 key
    steps per unit, the K/V ring wraps ~190 times) and a whole 8192-token prompt in one iteration (the
    token budget), at the 70B and 8B shapes; sampled outputs against the oracle."""
    b = W._assemble("prefill_long_prefix", W.SHAPE_70B, W.make_rng(310), np.array([2048, 1], np.int32),
                    np.array([60000 + 2048, 70001], np.int32), 1.05)
    check_batch_sampled(b, 96, seed=1)
    b = W._assemble("prefill_whole_budget", W.SHAPE_8B, W.make_rng(311), np.array([8192], np.int32),
                    np.array([8192], np.int32), 1.05)
    check_batch_sampled(b, 96, seed=2)


def test_empty_and_skipped_sequences():
    b = W._assemble("skipped", W.SHAPE_S1, W.make_rng(400), np.array([0, 1, 0], np.int32), np.array([33, 70, 5], np.int32), 1.3)
    check_batch_full(b)
    b = W._assemble("all_skipped", W.SHAPE_S1, W.make_rng(401), np.array([0, 0], np.int32), np.array([33, 70], np.int32), 1.3)
    check_batch_full(b)


def test_workspace_too_small_is_reported():
    b = decode_batch(106, W.SHAPE_8B, [30000])
    run = DeviceRun(b)
    assert run.workspace_bytes > 0
    with pytest.raises(ap.ApError) as e:
        ap.attention_iteration(run.pool, run.plan, run.q, run.out, run.lse, run.workspace, run.workspace_bytes - 1)
    assert e.value.status == B.AP_ERR_WORKSPACE_TOO_SMALL
    run.close()


@pytest.mark.parametrize("config", [2, 3, 4])
def test_full_size_configs_every_output(config):
    """Configurations 2, 3 and 4 at full size, in the launch configuration the benchmark times (the
    planner's own dispatch mode): whole-pool bit comparison after the append and EVERY attention output
    and lse against the oracle."""
    batch = {2: W.config2, 3: W.config3, 4: W.config4}[config]()
    err, lerr = check_batch_full(batch)
    print(f"config{config}: every output, out err {err:.2e} lse err {lerr:.2e}")


def test_config3_sequential_dispatch_every_output():
    """Config 3 once more with decode and prefill one after the other (the mode the per-kernel
    roofline figures are taken in)."""
    err, lerr = check_batch_full(W.config3(), side_by_side=0)
    print(f"config3 sequential: out err {err:.2e} lse err {lerr:.2e}")


def test_host_buffer_iteration_against_the_oracle():
    """ap_serving_iteration_host (plan, copies in, append, attention, copies out, one sync) on a mixed
    batch with cut decode streams, from pinned host buffers: pool bit-exact and every output against
    the oracle; the device-buffer path on a second pool must give the same bits."""
    import torch
    import oracle
    from harness import compare_outputs, oracle_pools
    b = W._assemble("host_buffers", W.SHAPE_8B, W.make_rng(502), np.array([1, 1, 150, 1, 1], np.int32),
                    np.array([77, 9000, 400, 1300, 16], np.int32), 1.3)
    k_ref, v_ref = oracle_pools(b)
    ref_out, ref_lse = oracle.attention(k_ref, v_ref, b.q_lens, b.ctx_lens, b.block_tables, b.q)
    run = DeviceRun(b)
    try:
        assert run.info["merge_entries"] > 0
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
        q, kn, vn = pin(b.q), pin(b.k_new), pin(b.v_new)
        out = torch.empty((b.n_new, b.num_q_heads, b.head_dim), dtype=torch.int16).pin_memory()
        lse = torch.empty((b.n_new, b.num_q_heads), dtype=torch.float32).pin_memory()
        for _ in range(2):                               # the second call reuses the pool's staging buffers
            out.fill_(0x7FC1); lse.fill_(float("nan"))
            ap.serving_iteration_host(run.pool, b.q_lens, b.ctx_lens, b.block_tables, b.num_q_heads, q, kn, vn, out, lse)
            compare_outputs(out.numpy().view(np.uint16), lse.numpy(), ref_out, ref_lse, "host buffers")
        assert np.array_equal(to_bits(run.k_pool), k_ref) and np.array_equal(to_bits(run.v_pool), v_ref)
        host_out, host_lse = out.numpy().view(np.uint16).copy(), lse.numpy().copy()
    finally:
        run.close()
    run = DeviceRun(b)
    try:
        run.append(); run.attend()
        assert run.status() == 0
        assert np.array_equal(to_bits(run.out)[:b.n_new], host_out)
        assert np.array_equal(run.lse.cpu().numpy()[:b.n_new], host_lse)
    finally:
        run.close()


def _trace_full_check_iterations(budget, chunk, iterations=200):
    """Iterations of the trace whose every output is compared: the one with the largest plan (most
    decode work items), the one where a decode CTA's item list is longest, and the one with the most
    new tokens; found by a dry run of the scheduler on a host-only pool (which plans like a 148-SM GPU)."""
    from paper_2604_07144_b200 import binding as B_
    reqs = W.trace_arrivals(W.SEED_BASE + 5, iterations)
    alloc = W.FreeListAllocator(1 << 22)
    hq, hkv, d = W.SHAPE_8B
    pool = ap.kv_pool_create(1 << 22, hkv, d, device=-1)
    best_items, best_new, best_list = (-1, -1), (-1, -1), (-1, -1)
    for it in W.fcfs_trace(reqs, alloc.alloc, alloc.free, iterations=iterations, token_budget=budget, chunk=chunk):
        if int(it.q_lens.sum()) == 0:
            continue
        plan = ap.plan_create(pool, it.q_lens, it.ctx_lens, it.block_tables, hq)
        ex = ap.plan_export(plan)
        ap.plan_destroy(plan)
        per_cta = int(np.diff(ex["cta_begin"]).max()) if len(ex["cta_begin"]) > 1 else 0
        best_items = max(best_items, (ex["info"]["decode_items"], it.index))
        best_list = max(best_list, (per_cta, it.index))
        best_new = max(best_new, (int(it.q_lens.sum()), it.index))
    ap.kv_pool_destroy(pool)
    return {best_items[1], best_new[1], best_list[1]}, best_list[0]


@pytest.mark.parametrize("budget,chunk", [(8192, 512), (2048, 256)], ids=["budget8192_chunk512", "budget2048_chunk256"])
def test_config5_trace_parity(budget, chunk):
    """The whole 200-iteration workload-shift trace (both low-rate and both high-rate phases), under
    the configuration's scheduler and under a second fixed policy: pages come from the library's
    allocator and are freed per request; the pool must match the oracle's bit for bit at the end;
    every iteration is compared on sampled outputs, and the iterations with the largest plan and with
    the most new tokens on every output."""
    import oracle
    from harness import compare_outputs
    from paper_2604_07144_b200.trace_runner import TraceRun
    full_iters, longest_list = _trace_full_check_iterations(budget, chunk)
    if budget == 8192:
        assert longest_list > 32      # the trace's largest plan overflows a CTA's shared-memory item list
    run = TraceRun(iterations=200, token_budget=budget, chunk=chunk)
    hq, hkv, d = run.shape
    k_ref = np.full((run.num_pages, hkv, 16, d), W.CANARY, np.uint16)
    v_ref = k_ref.copy()
    rng = np.random.default_rng(55)
    seen_prefill = seen_decode = checked = full_checked = 0
    last_index = -1
    worst = (0.0, 0.0)
    try:
        for st in run.steps():
            last_index = st.index
            if st.q is None:
                continue
            assert oracle.kv_append(k_ref, v_ref, st.q_lens, st.ctx_lens, st.block_tables, st.k_new, st.v_new) == 0
            seen_prefill += st.n_prefill
            seen_decode += st.n_decode
            if st.index in full_iters:
                ref_out, ref_lse = oracle.attention(k_ref, v_ref, st.q_lens, st.ctx_lens, st.block_tables, st.q)
                e = compare_outputs(to_bits(st.out), st.lse.cpu().numpy(), ref_out, ref_lse,
                                    f"trace iteration {st.index}, every output")
                full_checked += 1
                checked += ref_lse.size
            else:
                n = 12
                seq = rng.integers(0, len(st.q_lens), size=n)
                tok = np.array([rng.integers(0, st.q_lens[s]) for s in seq], dtype=np.int32)
                head = rng.integers(0, hq, size=n).astype(np.int32)
                ref_out, ref_lse = oracle.attention_samples(k_ref, v_ref, st.q_lens, st.ctx_lens, st.block_tables,
                                                            st.q, seq, tok, head)
                rows = np.concatenate([[0], np.cumsum(st.q_lens)])[seq] + tok
                e = compare_outputs(to_bits(st.out)[rows, head], st.lse.cpu().numpy()[rows, head], ref_out, ref_lse,
                                    f"trace iteration {st.index}")
                checked += n
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        assert last_index == 199 and full_checked == len(full_iters)
        assert seen_prefill > 0 and seen_decode > 0 and checked > 2000
        assert np.array_equal(to_bits(run.k_pool), k_ref), "K plane differs after the trace"
        assert np.array_equal(to_bits(run.v_pool), v_ref), "V plane differs after the trace"
        print(f"config5 (200 iterations, {sorted(full_iters)} in full): {checked} outputs, out err {worst[0]:.2e} "
              f"lse err {worst[1]:.2e}")
    finally:
        run.close()


@pytest.mark.parametrize("shape", [(6, 2, 128), (4, 4, 64), (5, 1, 128), (8, 2, 64)],
                         ids=lambda s: f"Hq{s[0]}_Hkv{s[1]}_d{s[2]}")
def test_prefill_head_ratios(shape):
    # odd groups leave a head without a partner (single-tile units); G = 1 has no pairs at all
    b = W._assemble("prefill_heads", shape, W.make_rng(600), np.array([150, 1, 70], np.int32),
                    np.array([333, 90, 70], np.int32), 1.3)
    check_batch_full(b)


def test_bounded_wait_times_out_and_the_pool_recovers():
    """The kernels' failure path in the only form that harms nothing: a one-warp kernel waits, through
    the bounded-wait routine the attention kernels use, on a barrier nothing arrives on.  It must end by
    itself, leave AP_ERR_TIMEOUT in the pool's status word (returned once, then cleared) together with a
    raised split-K arrival counter (cleared with it), and the next ordinary iteration on the same pool,
    one with cut streams, must be right."""
    import time
    import torch
    import oracle
    from harness import compare_outputs, oracle_pools
    b = decode_batch(120, W.SHAPE_8B, [20000, 9001, 333])
    run = DeviceRun(b)
    try:
        assert run.info["merge_entries"] > 0
        with pytest.raises(ap.ApError):
            ap.selftest_wait_timeout(run.pool, 0)                    # a limit is required
        t0 = time.perf_counter()
        ap.selftest_wait_timeout(run.pool, 1_000_000, leave_counter=True)       # 1 ms
        assert run.status() == B.AP_ERR_TIMEOUT
        assert time.perf_counter() - t0 < 1.0
        assert run.status() == 0                                         # reported once
        ap.kv_pool_set_wait_limit(run.pool, 500_000_000)                 # a pool setting; kernels take it as an argument
        run.append(); run.attend()
        assert run.status() == 0
        k_ref, v_ref = oracle_pools(b)
        ref_out, ref_lse = oracle.attention(k_ref, v_ref, b.q_lens, b.ctx_lens, b.block_tables, b.q)
        compare_outputs(to_bits(run.out)[:b.n_new], run.lse.cpu().numpy()[:b.n_new], ref_out, ref_lse, "after a timeout")
        ap.kv_pool_set_wait_limit(run.pool, 0)
        run.attend()
        assert run.status() == 0
        assert torch.cuda.is_available()
    finally:
        run.close()
