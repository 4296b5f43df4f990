"""Test harness: runs a workloads.Batch through the C ABI on a CUDA device and
through the CPU oracle, and compares them.  Test infrastructure only."""
from __future__ import annotations

import numpy as np

import oracle
import paper_2604_07144_b200 as ap
from paper_2604_07144_b200 import workloads as W

OUT_ATOL = 1e-2      # max abs error of the bf16 output against the fp64 oracle
LSE_RTOL = 1e-3      # |lse - ref| / max(|ref|, 1)


def to_dev(bits: np.ndarray, device="cuda:0"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def to_bits(t) -> np.ndarray:
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class GpuRun:
    """Pool + plan + device tensors of one batch."""

    def __init__(self, batch: W.Batch, device: int = 0, scale: float = 0.0, side_by_side=None):
        import torch
        self.torch = torch
        self.batch = batch
        dev = f"cuda:{device}"
        self.k_pool = to_dev(batch.k_pool, dev)
        self.v_pool = to_dev(batch.v_pool, dev)
        self.q = to_dev(batch.q, dev) if batch.n_new else torch.empty(0, dtype=torch.bfloat16, device=dev)
        self.k_new = to_dev(batch.k_new, dev) if batch.n_new else self.q
        self.v_new = to_dev(batch.v_new, dev) if batch.n_new else self.q
        self.out = torch.full((max(batch.n_new, 1), batch.num_q_heads, batch.head_dim), float("nan"),
                              dtype=torch.bfloat16, device=dev)
        self.lse = torch.full((max(batch.n_new, 1), batch.num_q_heads), float("nan"), dtype=torch.float32,
                              device=dev)
        self.pool = ap.kv_pool_create(batch.num_pages, batch.num_kv_heads, batch.head_dim, self.k_pool,
                                      self.v_pool, device=device)
        if side_by_side is not None:
            ap.kv_pool_set_side_by_side(self.pool, side_by_side)
        self.plan = ap.plan_create(self.pool, batch.q_lens, batch.ctx_lens, batch.block_tables,
                                   batch.num_q_heads, softmax_scale=scale)
        self.info = ap.plan_get_info(self.plan)
        nbytes = ap.plan_workspace_bytes(self.plan)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
        self.workspace_bytes = nbytes

    def append(self):
        ap.kv_append(self.pool, self.plan, self.k_new, self.v_new)

    def attend(self):
        ap.attention_iteration(self.pool, self.plan, self.q, self.out, self.lse, self.workspace,
                               self.workspace_bytes)

    def status(self) -> int:
        return ap.last_device_status(self.pool)

    def close(self):
        self.torch.cuda.synchronize()
        ap.plan_destroy(self.plan)
        ap.kv_pool_destroy(self.pool)


def oracle_pools(batch: W.Batch):
    k, v = batch.k_pool.copy(), batch.v_pool.copy()
    assert oracle.kv_append(k, v, batch.q_lens, batch.ctx_lens, batch.block_tables, batch.k_new, batch.v_new) == 0
    return k, v


def compare_outputs(out_bits: np.ndarray, lse: np.ndarray, ref_out: np.ndarray, ref_lse: np.ndarray, what=""):
    got = W.bf16_bits_to_f64(out_bits)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref_out).max() if got.size else 0.0
    lerr = (np.abs(lse.astype(np.float64) - ref_lse) / np.maximum(np.abs(ref_lse), 1.0)).max() if lse.size else 0.0
    assert err <= OUT_ATOL, f"{what}: out max abs err {err}"
    assert lerr <= LSE_RTOL, f"{what}: lse rel err {lerr}"
    return float(err), float(lerr)


def check_batch_full(batch: W.Batch, scale: float = 0.0, side_by_side=None):
    """Append + attention on the GPU against the oracle, every element."""
    run = GpuRun(batch, scale=scale, side_by_side=side_by_side)
    try:
        run.append()
        run.attend()
        assert run.status() == 0
        k_ref, v_ref = oracle_pools(batch)
        assert np.array_equal(to_bits(run.k_pool), k_ref), "K plane differs from the oracle (bit-exact)"
        assert np.array_equal(to_bits(run.v_pool), v_ref), "V plane differs from the oracle (bit-exact)"
        if batch.n_new == 0:
            return 0.0, 0.0
        ref_out, ref_lse = oracle.attention(k_ref, v_ref, batch.q_lens, batch.ctx_lens, batch.block_tables,
                                            batch.q, scale=scale)
        return compare_outputs(to_bits(run.out)[:batch.n_new], run.lse.cpu().numpy()[:batch.n_new], ref_out,
                               ref_lse, batch.name)
    finally:
        run.close()


def check_batch_sampled(batch: W.Batch, n_samples: int, seed: int = 0):
    """Full-size check: the append is compared bit-exactly on the whole pool,
    attention on randomly sampled (sequence, token, head) outputs."""
    run = GpuRun(batch)
    try:
        run.append()
        run.attend()
        assert run.status() == 0
        k_ref, v_ref = oracle_pools(batch)
        assert np.array_equal(to_bits(run.k_pool), k_ref)
        assert np.array_equal(to_bits(run.v_pool), v_ref)
        rng = np.random.default_rng(seed)
        active = np.nonzero(batch.q_lens > 0)[0]
        seq = rng.choice(active, size=n_samples)
        tok = np.array([rng.integers(0, batch.q_lens[s]) for s in seq], dtype=np.int32)
        head = rng.integers(0, batch.num_q_heads, size=n_samples).astype(np.int32)
        ref_out, ref_lse = oracle.attention_samples(k_ref, v_ref, batch.q_lens, batch.ctx_lens,
                                                    batch.block_tables, batch.q, seq, tok, head)
        rows = batch.q_indptr[seq] + tok
        out = to_bits(run.out)[rows, head]
        lse = run.lse.cpu().numpy()[rows, head]
        # every output must at least be finite and written
        assert np.isfinite(W.bf16_bits_to_f64(to_bits(run.out)[:batch.n_new])).all()
        return compare_outputs(out, lse, ref_out, ref_lse, batch.name)
    finally:
        run.close()
