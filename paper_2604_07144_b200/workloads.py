"""Seeded synthetic inputs for the paged-KV serving iteration.

This module only *draws inputs*: sequence lengths, block tables, bf16 N(0,1)
tensors and an FCFS continuous-batching trace.  It contains none of the
arithmetic of the method (no append, no attention, no softmax), so both the
CUDA path and the CPU oracle can be fed from it without sharing any logic.

All tensors are numpy arrays; bf16 values are carried as ``uint16`` bit
patterns.  Randomness comes from numpy's counter-based Philox bit generator
keyed by ``SEED_BASE + config``.

The five generators follow the five serving workloads the project measures
(continuous batching over ragged batches whose composition a scheduling policy
decides; paper Sec. 5.3 "Serving simulator", App. B Eq. "serve-latency";
length scales as in the paper's trace tables in App. G).
"""
from __future__ import annotations

import dataclasses
import math
import os
from concurrent.futures import ThreadPoolExecutor
from typing import Callable, Dict, Iterator, List, Optional, Sequence, Tuple

import numpy as np

SEED_BASE = 0x5EED0000
PAGE_SIZE = 16
#: bf16 NaN bit pattern written to every pool slot that holds no token yet.
CANARY = np.uint16(0x7FC1)

#: attention shapes (num_q_heads, num_kv_heads, head_dim)
SHAPE_S1 = (8, 2, 64)
SHAPE_8B = (32, 8, 128)
SHAPE_70B = (64, 8, 128)


class SeededStream:
    """Source of all random inputs for one workload.

    ``g`` is a numpy Generator over Philox keyed by the seed (lengths,
    permutations, arrivals).  Large normal tensors are drawn chunk-wise, each
    chunk from its own Philox key ``[seed, (call << 32) | chunk]``, so the bits
    do not depend on how many threads fill the chunks.
    """

    CHUNK = 1 << 22

    def __init__(self, seed: int):
        self.seed = int(seed)
        self.g = np.random.Generator(np.random.Philox(key=self.seed))
        self._calls = 0

    def _chunk(self, out: np.ndarray, call: int, idx: int) -> None:
        lo = idx * self.CHUNK
        hi = min(out.shape[0], lo + self.CHUNK)
        g = np.random.Generator(np.random.Philox(key=[self.seed, (call << 32) | idx]))
        out[lo:hi] = f32_to_bf16_bits(g.standard_normal(hi - lo, dtype=np.float32))

    def normal_bf16(self, shape) -> np.ndarray:
        """bf16 bit patterns of N(0,1) samples (drawn in float32, rounded RNE)."""
        n = int(np.prod(shape))
        out = np.empty(n, dtype=np.uint16)
        call = self._calls
        self._calls += 1
        nchunks = (n + self.CHUNK - 1) // self.CHUNK
        if nchunks <= 1:
            if n:
                self._chunk(out, call, 0)
        else:
            with ThreadPoolExecutor(max_workers=_host_threads()) as ex:
                list(ex.map(lambda i: self._chunk(out, call, i), range(nchunks)))
        return out.reshape(shape)


def _host_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def make_rng(seed: int) -> SeededStream:
    return SeededStream(seed)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even), returned as uint16 bits."""
    u = np.array(x, dtype=np.float32, copy=True).reshape(-1).view(np.uint32)
    t = u >> np.uint32(16)
    t &= np.uint32(1)
    t += np.uint32(0x7FFF)
    u += t
    u >>= np.uint32(16)
    return u.astype(np.uint16).reshape(np.shape(x))


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def normal_bf16(rng: SeededStream, shape) -> np.ndarray:
    return rng.normal_bf16(shape)


@dataclasses.dataclass
class Batch:
    """One serving iteration's inputs (state *before* the append)."""

    name: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    num_pages: int
    q_lens: np.ndarray          # int32 [B]  new tokens this iteration
    ctx_lens: np.ndarray        # int32 [B]  context length including the new tokens
    block_tables: np.ndarray    # int32 [B, stride]; entries past ceil(ctx/16) are -1
    q: np.ndarray               # uint16 [N_new, Hq, d]
    k_new: np.ndarray           # uint16 [N_new, Hkv, d]
    v_new: np.ndarray           # uint16 [N_new, Hkv, d]
    k_pool: Optional[np.ndarray] = None   # uint16 [num_pages, Hkv, 16, d]
    v_pool: Optional[np.ndarray] = None
    page_size: int = PAGE_SIZE

    @property
    def batch(self) -> int:
        return int(self.q_lens.shape[0])

    @property
    def n_new(self) -> int:
        return int(self.q_lens.sum())

    @property
    def kv_tokens(self) -> int:
        """Unique KV tokens one attention layer must read this iteration."""
        return int(self.ctx_lens[self.q_lens > 0].astype(np.int64).sum())

    @property
    def q_indptr(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.q_lens, dtype=np.int64)])


def pages_needed(ctx_lens: np.ndarray) -> np.ndarray:
    return (np.asarray(ctx_lens, dtype=np.int64) + PAGE_SIZE - 1) // PAGE_SIZE


def shuffled_block_tables(rng, ctx_lens, pool_factor: float = 1.25, stride: Optional[int] = None
                          ) -> Tuple[np.ndarray, int]:
    """Sequences take pages, in batch order, from a Fisher-Yates-shuffled pool
    of ``ceil(pool_factor * total pages)`` pages."""
    need = pages_needed(ctx_lens)
    total = int(need.sum())
    num_pages = max(1, int(math.ceil(pool_factor * total)))
    perm = rng.g.permutation(num_pages).astype(np.int32)
    if stride is None:
        stride = max(1, int(need.max()) if len(need) else 1)
    bt = np.full((len(need), stride), -1, dtype=np.int32)
    pos = 0
    for s, n in enumerate(need):
        bt[s, :n] = perm[pos:pos + n]
        pos += int(n)
    return bt, num_pages


def fill_pool(rng, num_pages, num_kv_heads, head_dim, q_lens, ctx_lens, block_tables
              ) -> Tuple[np.ndarray, np.ndarray]:
    """Pool planes holding N(0,1) for every already-cached token and the NaN
    canary everywhere else (unused pages, slots still to be appended, page
    tails)."""
    shape = (num_pages, num_kv_heads, PAGE_SIZE, head_dim)
    old = np.maximum(np.asarray(ctx_lens, np.int64) - np.asarray(q_lens, np.int64), 0)
    npg = (old + PAGE_SIZE - 1) // PAGE_SIZE
    pages = np.concatenate([block_tables[s, :npg[s]] for s in range(len(old))] + [np.empty(0, np.int32)])
    last = np.cumsum(npg) - 1                       # index in `pages` of each sequence's last old page
    planes = []
    for _ in range(2):
        plane = np.full(shape, CANARY, dtype=np.uint16)
        vals = normal_bf16(rng, (len(pages), num_kv_heads, PAGE_SIZE, head_dim))
        for s in range(len(old)):
            tail = int(old[s] - (npg[s] - 1) * PAGE_SIZE) if npg[s] else PAGE_SIZE
            if tail < PAGE_SIZE:
                vals[last[s], :, tail:, :] = CANARY
        plane[pages] = vals
        planes.append(plane)
    k_pool, v_pool = planes
    return k_pool, v_pool


def _assemble(name, shape, rng, q_lens, ctx_lens, pool_factor=1.25, with_pool=True) -> Batch:
    hq, hkv, d = shape
    q_lens = np.asarray(q_lens, dtype=np.int32)
    ctx_lens = np.asarray(ctx_lens, dtype=np.int32)
    bt, num_pages = shuffled_block_tables(rng, ctx_lens, pool_factor)
    n_new = int(q_lens.sum())
    q = normal_bf16(rng, (n_new, hq, d))
    k_new = normal_bf16(rng, (n_new, hkv, d))
    v_new = normal_bf16(rng, (n_new, hkv, d))
    k_pool = v_pool = None
    if with_pool:
        k_pool, v_pool = fill_pool(rng, num_pages, hkv, d, q_lens, ctx_lens, bt)
    return Batch(name, hq, hkv, d, num_pages, q_lens, ctx_lens, bt, q, k_new, v_new, k_pool, v_pool)


def config1(seed: int = SEED_BASE + 1, post_append: bool = True) -> Batch:
    """Single decode iteration: 4 sequences, contexts 17/64/200/513 counted
    after the append (``post_append=False`` gives the other reading, 18/65/201/514)."""
    ctx = np.array([17, 64, 200, 513], dtype=np.int32)
    if not post_append:
        ctx = ctx + 1
    return _assemble("config1_single_decode", SHAPE_S1, make_rng(seed), np.ones(4, np.int32), ctx)


def config2(seed: int = SEED_BASE + 2, batch: int = 64, with_pool: bool = True) -> Batch:
    """Decode-heavy ragged batch, 8B attention shape: contexts log-uniform in [128, 8192]."""
    rng = make_rng(seed)
    u = rng.g.random(batch)
    ctx = np.floor(128.0 * np.exp(u * math.log(8192.0 / 128.0))).astype(np.int64)
    ctx = np.clip(ctx, 128, 8192).astype(np.int32)
    return _assemble("config2_decode_heavy_8b", SHAPE_8B, rng, np.ones(batch, np.int32), ctx,
                     with_pool=with_pool)


def config3(seed: int = SEED_BASE + 3, n_prefill: int = 8, n_decode: int = 120, chunk: int = 512,
            max_prefix: int = 4096, with_pool: bool = True) -> Batch:
    """Mixed iteration, 8B shape: prefill chunks on uniform prefixes, then decodes."""
    rng = make_rng(seed)
    prefix = rng.g.integers(0, max_prefix + 1, size=n_prefill)
    dec = rng.g.integers(256, 4096 + 1, size=n_decode)
    q_lens = np.concatenate([np.full(n_prefill, chunk), np.ones(n_decode)]).astype(np.int32)
    ctx = np.concatenate([prefix + chunk, dec]).astype(np.int32)
    return _assemble("config3_mixed_8b", SHAPE_8B, rng, q_lens, ctx, with_pool=with_pool)


def config4(seed: int = SEED_BASE + 4, batch: int = 16, lo: int = 32768, hi: int = 131072,
            with_pool: bool = True) -> Batch:
    """Long-context decode, 70B attention shape."""
    rng = make_rng(seed)
    ctx = rng.g.integers(lo, hi + 1, size=batch).astype(np.int32)
    return _assemble("config4_long_decode_70b", SHAPE_70B, rng, np.ones(batch, np.int32), ctx,
                     with_pool=with_pool)


def random_ragged(seed: int, shape=SHAPE_S1, batch: int = 5, max_ctx: int = 100, max_q: int = 9,
                  pool_factor: float = 1.5) -> Batch:
    """Small random mixed batch for tests: q_len in [0, max_q], ctx in [q_len, max_ctx]."""
    rng = make_rng(seed)
    q_lens = rng.g.integers(0, max_q + 1, size=batch).astype(np.int32)
    ctx = np.array([rng.g.integers(max(1, int(q)), max_ctx + 1) for q in q_lens], dtype=np.int32)
    ctx = np.where(q_lens == 0, np.maximum(ctx, 1), ctx).astype(np.int32)
    return _assemble(f"ragged_{seed}", shape, rng, q_lens, ctx, pool_factor)


# --------------------------------------------------------------------------
# Workload-shift trace (config 5): bursty arrivals + fixed FCFS continuous
# batching with a token budget and chunked prefill.  Scheduling only: which
# sequence contributes how many new tokens in which iteration, and which pages
# it owns.  Page ids come from an allocator passed in by the caller.
# --------------------------------------------------------------------------

class FreeListAllocator:
    """Plain LIFO free list over ``num_pages`` page ids (host-side stand-in
    used by CPU tests and by the dry run that sizes the pool)."""

    def __init__(self, num_pages: int):
        self.num_pages = int(num_pages)
        self._free = list(range(self.num_pages - 1, -1, -1))
        self.peak_used = 0

    def alloc(self, n: int) -> List[int]:
        if n > len(self._free):
            raise MemoryError("out of pages")
        ids = [self._free.pop() for _ in range(n)]
        self.peak_used = max(self.peak_used, self.num_pages - len(self._free))
        return ids

    def free(self, ids: Sequence[int]) -> None:
        self._free.extend(reversed(list(ids)))


@dataclasses.dataclass
class TraceRequest:
    rid: int
    arrival_iter: int
    prompt_len: int
    output_len: int
    done_prompt: int = 0
    decoded: int = 0
    pages: List[int] = dataclasses.field(default_factory=list)

    @property
    def ctx(self) -> int:
        return self.done_prompt + self.decoded


@dataclasses.dataclass
class TraceIteration:
    index: int
    rids: np.ndarray          # int64 [B] request id per batch row
    q_lens: np.ndarray        # int32 [B]
    ctx_lens: np.ndarray      # int32 [B] (post-append)
    block_tables: np.ndarray  # int32 [B, stride]
    freed_pages: int          # pages returned to the allocator after this iteration


def lognormal_lengths(rng, n, mean, sigma, lo, hi) -> np.ndarray:
    """Lognormal with the given *distribution mean*: mu = ln(mean) - sigma^2/2."""
    mu = math.log(mean) - 0.5 * sigma * sigma
    x = np.exp(mu + sigma * rng.g.standard_normal(n))
    return np.clip(np.rint(x), lo, hi).astype(np.int64)


def trace_arrivals(seed: int = SEED_BASE + 5, iterations: int = 200, dt: float = 0.25,
                   rates: Tuple[float, float] = (2.0, 20.0), switch_every: int = 50
                   ) -> List[TraceRequest]:
    """Poisson arrivals per iteration on a virtual clock of ``dt`` seconds per
    iteration; the rate alternates between ``rates`` every ``switch_every``
    iterations."""
    rng = make_rng(seed)
    reqs: List[TraceRequest] = []
    for it in range(iterations):
        rate = rates[(it // switch_every) % len(rates)]
        n = int(rng.g.poisson(rate * dt))
        if n == 0:
            continue
        prompts = lognormal_lengths(rng, n, 1024.0, 1.0, 1, 8192)
        outputs = lognormal_lengths(rng, n, 256.0, 0.8, 1, 2048)
        for p, o in zip(prompts, outputs):
            reqs.append(TraceRequest(len(reqs), it, int(p), int(o)))
    return reqs


def fcfs_trace(requests: Sequence[TraceRequest], alloc: Callable[[int], Sequence[int]],
               free: Callable[[Sequence[int]], None], iterations: int = 200,
               token_budget: int = 8192, chunk: int = 512) -> Iterator[TraceIteration]:
    """Fixed FCFS continuous-batching scheduler.

    Each iteration: (1) every running request decodes one token; (2) what is
    left of the token budget goes to waiting or partly prefilled requests in
    arrival order, at most one chunk of ``chunk`` tokens per request; (3) a
    request whose prompt completed this iteration decodes from the next one
    and finishes after ``output_len`` decode steps, when its pages are freed.
    Pages are taken lazily, when a position first crosses into a new page.
    Batch rows are ordered prefill chunks first, then decodes.
    """
    reqs = [dataclasses.replace(r, pages=[]) for r in requests]
    nxt = 0
    waiting: List[TraceRequest] = []
    running: List[TraceRequest] = []
    for it in range(iterations):
        while nxt < len(reqs) and reqs[nxt].arrival_iter <= it:
            waiting.append(reqs[nxt])
            nxt += 1
        budget = token_budget
        decodes = list(running)[:budget]
        budget -= len(decodes)
        prefills: List[Tuple[TraceRequest, int]] = []
        for r in waiting:
            if budget <= 0:
                break
            n = min(chunk, r.prompt_len - r.done_prompt, budget)
            prefills.append((r, n))
            budget -= n
        rows: List[Tuple[TraceRequest, int, bool]] = (
            [(r, n, False) for r, n in prefills] + [(r, 1, True) for r in decodes])
        rids, q_lens, ctx_lens = [], [], []
        for r, n, is_decode in rows:
            if is_decode:
                r.decoded += 1
            else:
                r.done_prompt += n
            need = (r.ctx + PAGE_SIZE - 1) // PAGE_SIZE - len(r.pages)
            if need > 0:
                r.pages.extend(int(p) for p in alloc(need))
            rids.append(r.rid)
            q_lens.append(n)
            ctx_lens.append(r.ctx)
        stride = max([len(r.pages) for r, _, _ in rows], default=1)
        bt = np.full((len(rows), max(1, stride)), -1, dtype=np.int32)
        for i, (r, _, _) in enumerate(rows):
            bt[i, :len(r.pages)] = r.pages
        freed = 0
        still_running: List[TraceRequest] = []
        for r in running:
            if r.decoded >= r.output_len:
                free(r.pages)
                freed += len(r.pages)
                r.pages = []
            else:
                still_running.append(r)
        running = still_running
        still_waiting: List[TraceRequest] = []
        for r in waiting:
            if r.done_prompt >= r.prompt_len:
                running.append(r)
            else:
                still_waiting.append(r)
        waiting = still_waiting
        yield TraceIteration(it, np.array(rids, dtype=np.int64), np.array(q_lens, dtype=np.int32),
                             np.array(ctx_lens, dtype=np.int32), bt, freed)


def trace_peak_pages(requests: Sequence[TraceRequest], **kw) -> int:
    """Dry run of :func:`fcfs_trace` against an unbounded free list; returns the
    peak number of pages in use (the pool is then sized 1.25x that)."""
    a = FreeListAllocator(1 << 22)
    for _ in fcfs_trace(requests, a.alloc, a.free, **kw):
        pass
    return a.peak_used


def trace_new_tokens(rng, it: TraceIteration, shape) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """q, k_new, v_new for one trace iteration."""
    hq, hkv, d = shape
    n = int(it.q_lens.sum())
    return (normal_bf16(rng, (n, hq, d)), normal_bf16(rng, (n, hkv, d)), normal_bf16(rng, (n, hkv, d)))
