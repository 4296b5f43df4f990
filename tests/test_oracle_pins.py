"""Pins for the CPU oracle: everything here is fixed by the definition of
attention and by mathematics, none of it by the oracle itself.

The paper prints no value for the attention / KV path, so the pins are closed
forms, invariants, a structurally different dense brute force
(``oracle/dense_reference.py``) and a dictionary replay of the append.  The last
test plants plausible mistakes into a copy of the C oracle and checks that the
pin suite rejects every one of them.
"""
import ctypes
import math
import os
import re

import numpy as np
import pytest

import oracle
from oracle import dense_reference as dense
from paper_2604_07144_b200 import workloads as W

TOL = 1e-12


def _bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _post_append(b: W.Batch):
    """Pool after the append, built by dictionary replay (not by the oracle)."""
    k, v = b.k_pool.copy(), b.v_pool.copy()
    for (s, p, g), (kb, vb) in dense.append_as_dict(b.q_lens, b.ctx_lens, b.k_new, b.v_new).items():
        page = int(b.block_tables[s, p // 16])
        k[page, g, p % 16] = kb
        v[page, g, p % 16] = vb
    return k, v


def _single_sequence(ctx, hq=8, hkv=2, d=64, seed=7, q_len=1, k_fn=None, v_fn=None, q_fn=None):
    """One sequence with hand-set K/V/Q (float arrays -> bf16), shuffled pages."""
    rng = W.make_rng(seed)
    q_lens = np.array([q_len], np.int32)
    ctx_lens = np.array([ctx], np.int32)
    bt, num_pages = W.shuffled_block_tables(rng, ctx_lens, 2.0)
    kf = rng.g.standard_normal((ctx, hkv, d)) if k_fn is None else k_fn(ctx, hkv, d)
    vf = rng.g.standard_normal((ctx, hkv, d)) if v_fn is None else v_fn(ctx, hkv, d)
    qf = rng.g.standard_normal((q_len, hq, d)) if q_fn is None else q_fn(q_len, hq, d)
    k_pool = np.full((num_pages, hkv, 16, d), W.CANARY, np.uint16)
    v_pool = np.full((num_pages, hkv, 16, d), W.CANARY, np.uint16)
    kb, vb = _bits(kf), _bits(vf)
    for j in range(ctx):
        k_pool[bt[0, j // 16], :, j % 16, :] = kb[j]
        v_pool[bt[0, j // 16], :, j % 16, :] = vb[j]
    return dict(k_pool=k_pool, v_pool=v_pool, q_lens=q_lens, ctx_lens=ctx_lens, bt=bt,
                q=_bits(qf), kb=kb, vb=vb, hq=hq, hkv=hkv, d=d)


# ---------------------------------------------------------------- the pins --

def pin_dense_bruteforce():
    for seed, shape in ((11, W.SHAPE_S1), (12, (4, 4, 64)), (13, (8, 1, 128)), (14, W.SHAPE_S1)):
        b = W.random_ragged(seed, shape=shape, batch=6, max_ctx=90, max_q=11)
        k, v = _post_append(b)
        o1, l1 = oracle.attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q)
        o2, l2 = dense.dense_attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q)
        assert np.isfinite(o1).all() and np.isfinite(l1).all()
        assert np.abs(o1 - o2).max() <= TOL
        assert np.abs(l1 - l2).max() <= TOL
        # an explicit scale, too
        o1, l1 = oracle.attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q, scale=0.3)
        o2, l2 = dense.dense_attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q, scale=0.3)
        assert np.abs(o1 - o2).max() <= TOL and np.abs(l1 - l2).max() <= TOL


def pin_rows_sum_to_one():
    c = _single_sequence(77, seed=21)
    for h in range(c["hq"]):
        for p in (0, 15, 16, 76):
            w = oracle.softmax_row(c["k_pool"], c["v_pool"], c["hq"], c["bt"][0], p, c["q"][0, h], h)
            assert w.shape == (p + 1,)
            assert (w >= 0).all()
            assert abs(w.sum() - 1.0) <= TOL


def pin_single_token_returns_v():
    c = _single_sequence(1, seed=22)
    out, lse = oracle.attention(c["k_pool"], c["v_pool"], c["q_lens"], c["ctx_lens"], c["bt"], c["q"])
    g = c["hq"] // c["hkv"]
    for h in range(c["hq"]):
        v0 = W.bf16_bits_to_f64(c["vb"][0, h // g])
        assert np.array_equal(out[0, h], v0)                      # exactly V
        dot = float(np.dot(W.bf16_bits_to_f64(c["q"][0, h]), W.bf16_bits_to_f64(c["kb"][0, h // g])))
        assert abs(lse[0, h] - dot / math.sqrt(c["d"])) <= TOL


def pin_identical_keys_give_mean_of_v():
    for ctx in (5, 16, 33):
        key = W.make_rng(23).g.standard_normal((1, 2, 64))
        c = _single_sequence(ctx, seed=24, k_fn=lambda n, hk, d: np.repeat(key, n, axis=0))
        out, lse = oracle.attention(c["k_pool"], c["v_pool"], c["q_lens"], c["ctx_lens"], c["bt"], c["q"])
        g = c["hq"] // c["hkv"]
        for h in range(c["hq"]):
            mean_v = W.bf16_bits_to_f64(c["vb"][:, h // g]).mean(axis=0)
            assert np.abs(out[0, h] - mean_v).max() <= TOL
            x = float(np.dot(W.bf16_bits_to_f64(c["q"][0, h]), W.bf16_bits_to_f64(c["kb"][0, h // g]))) / 8.0
            assert abs(lse[0, h] - (x + math.log(ctx))) <= TOL
        # q = 0: natural-log lse = ln(p+1), inclusive causal bound
        c = _single_sequence(ctx, seed=25, q_fn=lambda n, hq, d: np.zeros((n, hq, d)))
        out, lse = oracle.attention(c["k_pool"], c["v_pool"], c["q_lens"], c["ctx_lens"], c["bt"], c["q"])
        assert np.abs(lse - math.log(ctx)).max() <= TOL
        for h in range(c["hq"]):
            assert np.abs(out[0, h] - W.bf16_bits_to_f64(c["vb"][:, h // g]).mean(axis=0)).max() <= TOL


def pin_two_key_closed_form():
    """scale=1, q=e0, k0=0, k1=e0: weights 1/(1+e), e/(1+e)."""
    def kf(n, hk, d):
        k = np.zeros((n, hk, d)); k[1, :, 0] = 1.0; return k
    def qf(n, hq, d):
        q = np.zeros((n, hq, d)); q[:, :, 0] = 1.0; return q
    def vf(n, hk, d):
        v = np.zeros((n, hk, d)); v[0, :, :] = 2.0; v[1, :, :] = -1.0; return v
    c = _single_sequence(2, seed=26, k_fn=kf, q_fn=qf, v_fn=vf)
    out, lse = oracle.attention(c["k_pool"], c["v_pool"], c["q_lens"], c["ctx_lens"], c["bt"], c["q"], scale=1.0)
    w1 = math.e / (1.0 + math.e)
    assert np.abs(out - (2.0 * (1 - w1) - 1.0 * w1)).max() <= TOL
    assert np.abs(lse - math.log(1.0 + math.e)).max() <= TOL
    # default scale 1/sqrt(64): weights 1/(1+e^(1/8)), ...
    out, lse = oracle.attention(c["k_pool"], c["v_pool"], c["q_lens"], c["ctx_lens"], c["bt"], c["q"])
    assert np.abs(lse - math.log(1.0 + math.exp(0.125))).max() <= TOL


def pin_gqa_head_mapping():
    """K,V constant per kv head: q head h must see kv head h div G."""
    def vf(n, hk, d):
        return np.broadcast_to(np.arange(1, hk + 1, dtype=np.float64)[None, :, None], (n, hk, d)).copy()
    c = _single_sequence(20, hq=8, hkv=4, seed=27, v_fn=vf)
    out, _ = oracle.attention(c["k_pool"], c["v_pool"], c["q_lens"], c["ctx_lens"], c["bt"], c["q"])
    for h in range(8):
        assert np.abs(out[0, h] - (h // 2 + 1)).max() <= TOL


def pin_page_permutation_invariance():
    b = W.random_ragged(31, batch=4, max_ctx=120, max_q=5)
    k, v = _post_append(b)
    o1, l1 = oracle.attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q)
    perm = W.make_rng(32).g.permutation(b.num_pages)
    inv = np.empty_like(perm); inv[perm] = np.arange(b.num_pages)
    k2, v2 = k[perm], v[perm]                                   # new page i holds old page perm[i]
    bt2 = np.where(b.block_tables >= 0, inv[np.maximum(b.block_tables, 0)], -1).astype(np.int32)
    o2, l2 = oracle.attention(k2, v2, b.q_lens, b.ctx_lens, bt2, b.q)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


def pin_split_merge_identity():
    c = _single_sequence(150, seed=33)
    for h in (0, 3, 7):
        full, lse_full = oracle.attention_range(c["k_pool"], c["v_pool"], c["hq"], c["bt"][0], 0, 150, c["q"][0, h], h)
        ref, lse_ref = oracle.attention(c["k_pool"], c["v_pool"], c["q_lens"], c["ctx_lens"], c["bt"], c["q"])
        assert np.abs(full - ref[0, h]).max() <= TOL and abs(lse_full - lse_ref[0, h]) <= TOL
        for cuts in ((0, 37, 150), (0, 16, 64, 149, 150), (0, 1, 150)):
            parts = [oracle.attention_range(c["k_pool"], c["v_pool"], c["hq"], c["bt"][0], a, b_, c["q"][0, h], h)
                     for a, b_ in zip(cuts[:-1], cuts[1:])]
            o, lse = oracle.merge_partials(np.stack([p[0] for p in parts]), np.array([p[1] for p in parts]))
            assert np.abs(o - ref[0, h]).max() <= 1e-11
            assert abs(lse - lse_ref[0, h]) <= 1e-11
    # the merge formula against a hand-made case: two parts with lse ln1, ln3 -> weights 1/4, 3/4
    o, lse = oracle.merge_partials(np.array([[4.0, 0.0], [0.0, 8.0]]), np.array([0.0, math.log(3.0)]))
    assert np.abs(o - np.array([1.0, 6.0])).max() <= TOL and abs(lse - math.log(4.0)) <= TOL


def pin_chunking_identity():
    hq, hkv, d, n, n1 = 8, 2, 64, 45, 19
    rng = W.make_rng(34)
    ctx = np.array([n], np.int32)
    bt, num_pages = W.shuffled_block_tables(rng, ctx, 1.5)
    q = rng.normal_bf16((n, hq, d)); kn = rng.normal_bf16((n, hkv, d)); vn = rng.normal_bf16((n, hkv, d))
    empty = lambda: np.full((num_pages, hkv, 16, d), W.CANARY, np.uint16)
    # one prefill of n tokens
    k, v = empty(), empty()
    assert oracle.kv_append(k, v, [n], [n], bt, kn, vn) == 0
    o_full, l_full = oracle.attention(k, v, [n], [n], bt, q)
    # two chunks
    k2, v2 = empty(), empty()
    assert oracle.kv_append(k2, v2, [n1], [n1], bt, kn[:n1], vn[:n1]) == 0
    o_a, l_a = oracle.attention(k2, v2, [n1], [n1], bt, q[:n1])
    assert oracle.kv_append(k2, v2, [n - n1], [n], bt, kn[n1:], vn[n1:]) == 0
    o_b, l_b = oracle.attention(k2, v2, [n - n1], [n], bt, q[n1:])
    assert np.array_equal(k, k2) and np.array_equal(v, v2)
    assert np.abs(np.concatenate([o_a, o_b]) - o_full).max() <= TOL
    assert np.abs(np.concatenate([l_a, l_b]) - l_full).max() <= TOL
    # row t of the prefill == decode of token t on a context of t+1
    for t in (0, 15, 16, 44):
        o_d, l_d = oracle.attention(k, v, [1], [t + 1], bt, q[t:t + 1])
        assert np.abs(o_d[0] - o_full[t]).max() <= TOL and np.abs(l_d[0] - l_full[t]).max() <= TOL


def pin_append_replay():
    for seed in (41, 42, 43):
        b = W.random_ragged(seed, batch=7, max_ctx=70, max_q=20)
        k, v = b.k_pool.copy(), b.v_pool.copy()
        assert oracle.kv_append(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.k_new, b.v_new) == 0
        k_ref, v_ref = _post_append(b)
        assert np.array_equal(k, k_ref) and np.array_equal(v, v_ref)
        touched = np.zeros(k.shape[:3], bool)
        for (s, p, g) in dense.append_as_dict(b.q_lens, b.ctx_lens, b.k_new, b.v_new):
            touched[b.block_tables[s, p // 16], g, p % 16] = True
        assert np.array_equal(k[~touched], b.k_pool[~touched])     # untouched bytes unchanged
        assert np.array_equal(v[~touched], b.v_pool[~touched])
        assert touched.sum() == b.n_new * b.num_kv_heads
    # an out-of-range page id is reported, not written
    b = W.random_ragged(45, batch=3, max_ctx=40, max_q=4)
    assert b.n_new > 0
    bt = b.block_tables.copy(); bt[bt >= 0] = b.num_pages
    k, v = b.k_pool.copy(), b.v_pool.copy()
    assert oracle.kv_append(k, v, b.q_lens, b.ctx_lens, bt, b.k_new, b.v_new) == -1
    assert np.array_equal(k, b.k_pool)


def pin_page_copy_migration():
    """Page copy: (1) moving every used page of a batch into another pool and remapping the block
    tables leaves attention bit-identical, the source pool and the unused destination pages untouched;
    (2) it equals numpy's simultaneous gather/scatter, also for a rotation of pages inside one pool;
    (3) bad ids and repeated destinations are refused without writing."""
    b = W.random_ragged(61, batch=6, max_ctx=150, max_q=5)
    k, v = _post_append(b)
    o_ref, l_ref = oracle.attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q)
    used = sorted({int(b.block_tables[s, i]) for s in range(b.batch) for i in range((int(b.ctx_lens[s]) + 15) // 16)})
    rng = np.random.default_rng(7)
    n_dst = b.num_pages + 11
    new_of = dict(zip(used, rng.permutation(n_dst)[:len(used)].tolist()))
    canary = np.uint16(0x7FC1)
    k2 = np.full((n_dst,) + k.shape[1:], canary, np.uint16)
    v2 = np.full((n_dst,) + v.shape[1:], canary, np.uint16)
    src = np.array(used, np.int32)
    dst = np.array([new_of[p] for p in used], np.int32)
    k_before, v_before = k.copy(), v.copy()
    assert oracle.copy_pages(k2, v2, k, v, dst, src) == 0
    assert np.array_equal(k, k_before) and np.array_equal(v, v_before)
    assert np.array_equal(k2[dst], k[src]) and np.array_equal(v2[dst], v[src])
    rest = np.setdiff1d(np.arange(n_dst), dst)
    assert (k2[rest] == canary).all() and (v2[rest] == canary).all()
    bt2 = b.block_tables.copy()
    for s in range(b.batch):
        for i in range((int(b.ctx_lens[s]) + 15) // 16):
            bt2[s, i] = new_of[int(b.block_tables[s, i])]
    o2, l2 = oracle.attention(k2, v2, b.q_lens, b.ctx_lens, bt2, b.q)
    assert np.array_equal(o2, o_ref) and np.array_equal(l2, l_ref)
    # inside one pool the copies are simultaneous: a rotation a -> b -> c -> a
    a, bb, c = used[0], used[1], used[2]
    kr, vr = k.copy(), v.copy()
    assert oracle.copy_pages(kr, vr, kr, vr, [bb, c, a], [a, bb, c]) == 0
    ke, ve = k.copy(), v.copy()
    ke[[bb, c, a]] = k[[a, bb, c]]
    ve[[bb, c, a]] = v[[a, bb, c]]
    assert np.array_equal(kr, ke) and np.array_equal(vr, ve)
    assert not np.array_equal(k[a], v[a])                       # the planes differ, so a K/V mix-up shows
    # refusals write nothing
    for bad_dst, bad_src in (([n_dst], [used[0]]), ([0], [b.num_pages]), ([-1], [used[0]]), ([3, 3], [used[0], used[1]])):
        k3, v3 = k2.copy(), v2.copy()
        assert oracle.copy_pages(k3, v3, k, v, bad_dst, bad_src) == -1
        assert np.array_equal(k3, k2) and np.array_equal(v3, v2)
    assert oracle.copy_pages(k2, v2, k, v, [], []) == 0


def _artifact_rows():
    path = os.path.join(os.path.dirname(__file__), "golden", "table_artifact_feedback.txt")
    rows = []
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            name, n, stale, reconf, serve, total = line.split()
            rows.append((name, int(n), float(stale), float(reconf), float(serve), float(total)))
    assert len(rows) == 3
    return rows


def _split(rng, total, parts):
    """`parts` non-negative numbers adding up to `total`."""
    w = rng.random(parts) + 0.1
    return (w / w.sum() * total).tolist()


def test_execution_model_oracle_reproduces_the_papers_table():
    """Eq. "ttotal" against the printed rows: however the accumulated costs are spread over the
    N reschedulings, the total is the printed T_total; dropping a term is noticed."""
    from oracle import execution_model as E
    rng = np.random.default_rng(1)
    for name, n, stale, reconf, serve, total in _artifact_rows():
        for _ in range(5):
            t_serve = _split(rng, serve, n + 1)
            t_stale = [123.0] + _split(rng, stale, n)            # entry 0 does not exist in the model
            t_reconf = [456.0] + _split(rng, reconf, n)
            t_sched = [0.0] + [9.9] * n                          # later scheduling time is t_stale, not added again
            assert abs(E.t_total(t_sched, t_stale, t_reconf, t_serve) - total) < 0.05, name
            assert abs(E.t_total(t_sched, t_stale, [0.0] * (n + 1), t_serve) - total) > 1.0, name
    assert E.t_total([], [], [], []) == 0.0
    assert E.t_total([2.0], [7.0], [7.0], [3.0]) == 5.0          # cold start only: scheduling + serving


def test_roofline_model_pins():
    """The cost-model oracle (App. B Eq. "roofline") against what the mathematics fixes."""
    from oracle import roofline_model as R
    B, F = 6.0e12, 1.5e15
    rng = np.random.default_rng(0)
    for _ in range(200):
        fl, by = float(10 ** rng.uniform(3, 15)), float(10 ** rng.uniform(3, 12))
        # min over rates = max over times
        assert np.isclose(R.t_op(fl, by, B, F), max(fl / F, by / B), rtol=1e-12)
    ridge = F / B                                   # AI* = F_g / B_g: both branches meet
    assert np.isclose(R.t_op(ridge * 1e9, 1e9, B, F), 1e9 / B, rtol=1e-12)
    assert np.isclose(R.achieved_rate(ridge * 1e9, 1e9, B, F), F, rtol=1e-12)
    assert R.t_op(2.0 * ridge * 1e9, 1e9, B, F) == 2.0 * ridge * 1e9 / F          # compute-bound above the ridge
    assert R.t_op(0.5 * ridge * 1e9, 1e9, B, F) == 1e9 / B                        # memory-bound below it
    assert R.t_op(0.0, 1e9, B, F) == 1e9 / B and R.t_op(0.0, 0.0, B, F) == 0.0
    # long-context grouped-query decode: intensity tends to G = Hq / Hkv flop per byte
    for hq, hkv, d in ((32, 8, 128), (64, 8, 128), (8, 2, 64)):
        w = R.iteration_work([1], [1 << 20], hq, hkv, d)
        assert abs(w["decode_flops"] / w["decode_bytes"] - hq / hkv) < 1e-2
    # a causal chunk: the pair count against an explicit enumeration of (row, key) with key <= position
    ql, cl, hq, hkv, d = 37, 100, 4, 2, 64
    pairs = sum(1 for t in range(ql) for j in range(cl) if j <= cl - ql + t)
    w = R.iteration_work([ql], [cl], hq, hkv, d)
    assert w["prefill_flops"] == 4 * hq * d * pairs and pairs == ql * (cl - ql) + ql * (ql + 1) // 2
    assert w["append_bytes"] == 2 * ql * (2 * hkv * d * 2)
    assert w["prefill_bytes"] == cl * 2 * hkv * d * 2 + ql * (2 * hq * d * 2 + hq * 4)
    # config 2 at the 8B shape is on the memory side of the ridge, config 3's prefill on the compute side
    b2 = W.config2(with_pool=False)
    w2 = R.iteration_work(b2.q_lens, b2.ctx_lens, 32, 8, 128)
    assert w2["decode_flops"] / w2["decode_bytes"] < 5 < ridge
    b3 = W.config3(with_pool=False)
    w3 = R.iteration_work(b3.q_lens, b3.ctx_lens, 32, 8, 128)
    assert w3["prefill_flops"] / w3["prefill_bytes"] > ridge


PINS = [pin_dense_bruteforce, pin_rows_sum_to_one, pin_single_token_returns_v,
        pin_identical_keys_give_mean_of_v, pin_two_key_closed_form, pin_gqa_head_mapping,
        pin_page_permutation_invariance, pin_split_merge_identity, pin_chunking_identity,
        pin_append_replay, pin_page_copy_migration]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin()


def test_config1_matches_dense_bruteforce():
    b = W.config1()
    k, v = b.k_pool.copy(), b.v_pool.copy()
    assert oracle.kv_append(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.k_new, b.v_new) == 0
    o1, l1 = oracle.attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q)
    o2, l2 = dense.dense_attention(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q)
    assert np.abs(o1 - o2).max() <= TOL and np.abs(l1 - l2).max() <= TOL
    # sampled interface agrees with the full one
    seq = np.array([0, 1, 2, 3, 3]); tok = np.zeros(5, np.int32); head = np.array([0, 7, 3, 4, 5])
    os_, ls_ = oracle.attention_samples(k, v, b.q_lens, b.ctx_lens, b.block_tables, b.q, seq, tok, head)
    for i in range(5):
        assert np.array_equal(os_[i], o1[seq[i], head[i]]) and ls_[i] == l1[seq[i], head[i]]


# Plausible mistakes, planted into a copy of the C source.  Each must make at
# least one pin fail.
MUTATIONS = [
    ("causal bound excludes the query's own key", "for (int j = 0; j <= p; ++j) {\n        const uint16_t *kj",
     "for (int j = 0; j < p; ++j) {\n        const uint16_t *kj"),
    ("missing softmax scale", "x[j] = scale * dot;", "x[j] = dot;"),
    ("no normalisation by l", "for (int c = 0; c < d; ++c) out[c] /= l;\n    for (int j = 0; j <= p; ++j) x[j] /= l;",
     "for (int j = 0; j <= p; ++j) x[j] /= l;"),
    ("lse without the max", "*lse = m + log(l);\n}\n\n/*\n * Attention for every", "*lse = log(l);\n}\n\n/*\n * Attention for every"),
    ("log2 instead of ln", "*lse = m + log(l);\n}\n\n/*\n * Attention for every", "*lse = m + log2(l);\n}\n\n/*\n * Attention for every"),
    ("kv head = h mod Hkv", "q + o * d, h / G, scale, x,\n                               out + o * d",
     "q + o * d, h % Hkv, scale, x,\n                               out + o * d"),
    ("slot/page swapped in pool offset", "return (((size_t)page * Hkv + kv_head) * ORACLE_PAGE + slot) * (size_t)d;",
     "return (((size_t)page * ORACLE_PAGE + slot) * Hkv + kv_head) * (size_t)d;"),
    ("append position off by one", "int p = ctx_lens[s] - q_lens[s] + t;\n            if (p < 0",
     "int p = ctx_lens[s] - q_lens[s] + t + 1;\n            if (p < 0"),
    ("append writes V from K", "memcpy(V + dst, v_new + src", "memcpy(V + dst, k_new + src"),
    ("prefill rows all see the whole context", "int p = ctx_lens[s] - q_lens[s] + t;\n                    size_t o",
     "int p = ctx_lens[s] - 1;\n                    size_t o"),
    ("merge weights by exp(lse_k - m*) unnormalised", "double w = exp(lse_parts[k] - *lse);", "double w = exp(lse_parts[k] - mstar);"),
    ("V read from the K plane", "const uint16_t *vj = V + pool_off(bt[j / ORACLE_PAGE], g, j % ORACLE_PAGE, Hkv, d);\n        for (int c = 0; c < d; ++c) out[c] += x[j] * bf16_to_f64(vj[c]);",
     "const uint16_t *vj = K + pool_off(bt[j / ORACLE_PAGE], g, j % ORACLE_PAGE, Hkv, d);\n        for (int c = 0; c < d; ++c) out[c] += x[j] * bf16_to_f64(vj[c]);"),
    ("page copy takes V from the K plane", "V_src + (size_t)src_ids[i] * page_elems", "K_src + (size_t)src_ids[i] * page_elems"),
    ("page copy reads the destination's page number", "K_src + (size_t)src_ids[i] * page_elems", "K_src + (size_t)dst_ids[i] * page_elems"),
    ("page copy forgets the kv heads in the page size", "const size_t page_elems = (size_t)Hkv * ORACLE_PAGE * (size_t)d;",
     "const size_t page_elems = (size_t)ORACLE_PAGE * (size_t)d;"),
    ("page copy writes V pages into the K plane", "memcpy(V_dst + (size_t)dst_ids[i] * page_elems", "memcpy(K_dst + (size_t)dst_ids[i] * page_elems"),
    ("bf16 widened from the low half", "uint32_t u = (uint32_t)b << 16;", "uint32_t u = (uint32_t)b << 15;"),
]


@pytest.mark.parametrize("what,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(tmp_path, what, old, new):
    src = open(os.path.join(os.path.dirname(oracle.__file__), "paged_attention_oracle.c")).read()
    assert src.count(old) == 1, f"mutation anchor for '{what}' must match exactly once"
    mutated = tmp_path / "mutated.c"
    mutated.write_text(src.replace(old, new))
    so = oracle.compile_source(str(mutated), str(tmp_path / "mutated.so"))
    good = oracle.lib()
    oracle._lib = oracle.bind(ctypes.CDLL(so))
    try:
        failed = []
        for pin in PINS:
            try:
                pin()
            except AssertionError:
                failed.append(pin.__name__)
        assert failed, f"no pin noticed: {what}"
    finally:
        oracle._lib = good
