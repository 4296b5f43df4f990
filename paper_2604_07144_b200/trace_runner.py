"""Drives the library over the workload-shift trace: a seeded bursty arrival
process served by the fixed FCFS continuous-batching scheduler of
``workloads.fcfs_trace``, with KV pages taken from and returned to the
library's own page allocator request by request.

Per iteration it builds the plan, appends the new tokens' K/V and runs
attention through the C ABI, and yields what happened (sizes, device time, and
the device tensors, so a caller can compare them with anything it likes).
It is a harness around the kernels: scheduling and input drawing live in
``workloads``; no arithmetic of the method happens here.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Iterator, Optional

import numpy as np

from . import binding as ap
from . import workloads as W


@dataclasses.dataclass
class TraceStep:
    index: int
    q_lens: np.ndarray
    ctx_lens: np.ndarray
    block_tables: np.ndarray
    q: Optional[np.ndarray]          # uint16 [n_new, Hq, d]   (None for an empty iteration)
    k_new: Optional[np.ndarray]
    v_new: Optional[np.ndarray]
    out: object                      # torch bf16 [n_new, Hq, d] (device)
    lse: object                      # torch fp32 [n_new, Hq]    (device)
    kv_tokens: int
    n_prefill: int
    n_decode: int
    gpu_ms: float                    # append + attention, CUDA events
    info: dict


class TraceRun:
    """Pool, allocator and device buffers for one replay of the trace."""

    def __init__(self, iterations: int = 200, seed: int = W.SEED_BASE + 5, shape=W.SHAPE_8B, device: int = 0,
                 pool_factor: float = 1.25, token_budget: int = 8192, chunk: int = 512):
        import torch
        self.torch = torch
        self.iterations = iterations
        self.seed = seed
        self.shape = shape
        self.device = device
        self.requests = W.trace_arrivals(seed, iterations)
        self.policy = {"token_budget": int(token_budget), "chunk": int(chunk)}     # the fixed scheduler's two knobs
        self.peak_pages = W.trace_peak_pages(self.requests, iterations=iterations, **self.policy)
        self.num_pages = max(16, int(math.ceil(pool_factor * self.peak_pages)))
        hq, hkv, d = shape
        dev = f"cuda:{device}"
        canary = torch.tensor([int(W.CANARY)], dtype=torch.int32).to(torch.int16)
        self.k_pool = canary.to(dev).view(torch.bfloat16).repeat(self.num_pages * hkv * 16 * d).view(
            self.num_pages, hkv, 16, d)
        self.v_pool = self.k_pool.clone()
        self.pool = ap.kv_pool_create(self.num_pages, hkv, d, self.k_pool, self.v_pool, device=device)
        ap.kv_pool_seed_free_list(self.pool, seed)
        self.max_new = 8192
        self.q = torch.empty((self.max_new, hq, d), dtype=torch.bfloat16, device=dev)
        self.k_new = torch.empty((self.max_new, hkv, d), dtype=torch.bfloat16, device=dev)
        self.v_new = torch.empty((self.max_new, hkv, d), dtype=torch.bfloat16, device=dev)
        self.out = torch.empty((self.max_new, hq, d), dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty((self.max_new, hq), dtype=torch.float32, device=dev)
        self.workspace = torch.empty(ap.static_workspace_bytes(), dtype=torch.uint8, device=dev)

    def _alloc(self, n):
        return ap.kv_pool_alloc_pages(self.pool, n)

    def _free(self, ids):
        ap.kv_pool_free_pages(self.pool, ids)

    def steps(self, draw_inputs: bool = True) -> Iterator[TraceStep]:
        torch = self.torch
        hq, hkv, d = self.shape
        rng = W.make_rng(self.seed + 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for it in W.fcfs_trace(self.requests, self._alloc, self._free, iterations=self.iterations, **self.policy):
            n = int(it.q_lens.sum())
            if n == 0:
                yield TraceStep(it.index, it.q_lens, it.ctx_lens, it.block_tables, None, None, None, None, None,
                                0, 0, 0, 0.0, {})
                continue
            q, kn, vn = W.trace_new_tokens(rng, it, self.shape)

            def up(dst, bits):
                dst[:n].copy_(torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16), non_blocking=False)
            up(self.q, q); up(self.k_new, kn); up(self.v_new, vn)
            plan = ap.plan_create(self.pool, it.q_lens, it.ctx_lens, it.block_tables, hq)
            info = ap.plan_get_info(plan)
            ws_bytes = ap.plan_workspace_bytes(plan)
            e0.record()
            ap.kv_append(self.pool, plan, self.k_new, self.v_new)
            ap.attention_iteration(self.pool, plan, self.q, self.out, self.lse, self.workspace, ws_bytes)
            e1.record()
            status = ap.last_device_status(self.pool)
            ap.plan_destroy(plan)
            if status != 0:
                raise ap.ApError(status, f"trace iteration {it.index}")
            yield TraceStep(it.index, it.q_lens, it.ctx_lens, it.block_tables, q, kn, vn, self.out[:n], self.lse[:n],
                            info["kv_tokens"], int((it.q_lens > 1).sum()), int((it.q_lens == 1).sum()),
                            float(e0.elapsed_time(e1)), info)

    def close(self):
        self.torch.cuda.synchronize()
        ap.kv_pool_destroy(self.pool)
