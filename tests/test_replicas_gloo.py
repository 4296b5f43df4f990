"""The N > 1 path on CPU: two gloo ranks draw different replicas of the batch,
plan them independently on host-only pools, and aggregate their (fake) timings
the way bench.py does: sum of work, max of time."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import paper_2604_07144_b200 as ap
        from paper_2604_07144_b200 import replicas, workloads as W
        b = W.config2(seed=replicas.replica_seed(W.SEED_BASE + 2, rank), batch=16, with_pool=False)
        pool = ap.kv_pool_create(b.num_pages, b.num_kv_heads, b.head_dim, device=-1)
        plan = ap.plan_create(pool, b.q_lens, b.ctx_lens, b.block_tables, b.num_q_heads)
        info = ap.plan_get_info(plan)
        assert info["kv_tokens"] == b.kv_tokens
        fake_ms = 1.0 + rank                       # rank 1 is "slower"
        replicas.barrier()
        total, ms, rate = replicas.whole_job_throughput(b.kv_tokens, fake_ms)
        np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([b.kv_tokens, total, ms, rate], dtype=np.float64))
        ap.plan_destroy(plan)
        ap.kv_pool_destroy(pool)
    finally:
        dist.destroy_process_group()


def test_two_replicas_aggregate_sum_of_work_and_max_of_time(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [np.load(tmp_path / f"r{i}.npy") for i in range(world)]
    assert r[0][0] != r[1][0]                      # different batches per replica
    for i in range(world):
        assert r[i][1] == r[0][0] + r[1][0]        # whole-job work
        assert r[i][2] == 2.0                      # max over ranks
        assert abs(r[i][3] - (r[0][0] + r[1][0]) / 2e-3) < 1e-6


def test_single_process_needs_no_process_group():
    from paper_2604_07144_b200 import replicas
    assert replicas.reduce_max(3.5) == 3.5 and replicas.reduce_sum(2.0) == 2.0
    assert replicas.whole_job_throughput(10.0, 2.0) == (10.0, 2.0, 5000.0)
