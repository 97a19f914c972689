"""Seeded synthetic serving steps: mixed decode + interrupt-append batches over a paged KV pool.

This module only draws inputs (lengths, page tables, bf16 values).  It contains none of the
method's arithmetic: no append, no attention, no softmax.  Both the CUDA path and the CPU oracle
are fed from the arrays it returns.

The batches stand in for AsyncLM's serving traffic (Section 3.2 and Section 5.3 of the paper: a
returning function call makes the interrupt manager append a short token span to the end of one
sequence's context, and the next decoding step processes it together with the ordinary one-token
decodes of the other sequences).  Only the shape of that traffic is taken: short spans, sparse
arrivals, contexts of a few hundred to many thousand tokens.

Conventions
-----------
* bf16 tensors are carried as ``numpy.uint16`` bit patterns.
* ``kv_pool`` has layout ``[num_pages][2 (0=K, 1=V)][num_kv_heads][page_size][head_dim]``.
* ``q_indptr`` is a CSR over sequences: sequence ``b`` contributes ``q_indptr[b+1]-q_indptr[b]``
  new tokens this step (0 = paused by a trap, 1 = plain decode, >1 = interrupt append).
* ``kv_len_before[b]`` tokens of sequence ``b`` are already stored in its pages.
* ``page_indices[page_indptr[b] + j]`` is the physical page holding logical page ``j`` of ``b``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

BASE_SEED = 241207017


@dataclass(frozen=True)
class Shape:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int = 16

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2

    @property
    def page_elems(self) -> int:
        return 2 * self.num_kv_heads * self.page_size * self.head_dim


@dataclass
class Step:
    """One serving step's inputs (host arrays)."""
    q_indptr: np.ndarray        # int32 [B+1]
    kv_len_before: np.ndarray   # int32 [B]
    page_indptr: np.ndarray     # int32 [B+1]
    page_indices: np.ndarray    # int32 [page_indptr[-1]]
    q: np.ndarray               # uint16 [T, Hq, d]   bf16 bits
    k_new: np.ndarray           # uint16 [T, Hkv, d]  bf16 bits
    v_new: np.ndarray           # uint16 [T, Hkv, d]  bf16 bits

    @property
    def batch(self) -> int:
        return int(self.kv_len_before.shape[0])

    @property
    def total_q(self) -> int:
        return int(self.q_indptr[-1])

    @property
    def q_len(self) -> np.ndarray:
        return np.diff(self.q_indptr)


@dataclass
class Workload:
    name: str
    shape: Shape
    num_pages: int
    kv_pool: np.ndarray         # uint16 [num_pages, 2, Hkv, P, d]
    steps: List[Step] = field(default_factory=list)
    seed: int = 0
    note: str = ""


# --------------------------------------------------------------------------------------------
# value generation
# --------------------------------------------------------------------------------------------

def _rng(seed: int, stream: int) -> np.random.Generator:
    """Counter-based generator (Philox) keyed by (seed, stream) so any tensor can be redrawn."""
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round to nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float64 exactly."""
    u = b.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def normal_bf16(seed: int, stream: int, shape: Sequence[int], chunk: int = 1 << 22) -> np.ndarray:
    """N(0,1) samples rounded to bf16.  Chunk c of a tensor comes from its own Philox stream keyed by
    (seed, stream, c), so chunks can be drawn in parallel and any slice can be redrawn."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)

    def fill(c: int) -> None:
        s, e = c * chunk, min(n, (c + 1) * chunk)
        g = np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), (int(stream) << 24) | c]))
        out[s:e] = f32_to_bf16_bits(g.standard_normal(e - s, dtype=np.float32))

    nchunks = (n + chunk - 1) // chunk
    if nchunks <= 2:
        for c in range(nchunks):
            fill(c)
    else:
        from concurrent.futures import ThreadPoolExecutor
        import os
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, range(nchunks)))
    return out.reshape(tuple(shape))


# --------------------------------------------------------------------------------------------
# batch structure
# --------------------------------------------------------------------------------------------

def _ceil_div(a, b):
    return -(-a // b)


def build_step_tables(kv_len_before: np.ndarray, q_len: np.ndarray, page_size: int,
                      page_ids: np.ndarray, extra_pages: Optional[np.ndarray] = None):
    """CSR tables for a batch whose pages are taken, sequence by sequence, from ``page_ids``.

    ``extra_pages[b]`` (optional) pre-allocates that many unused pages after the needed ones.
    Returns (q_indptr, page_indptr, page_indices, pages_used).
    """
    kv_len_before = np.asarray(kv_len_before, dtype=np.int64)
    q_len = np.asarray(q_len, dtype=np.int64)
    need = _ceil_div(kv_len_before + q_len, page_size)
    if extra_pages is not None:
        need = need + np.asarray(extra_pages, dtype=np.int64)
    page_indptr = np.zeros(len(need) + 1, dtype=np.int64)
    page_indptr[1:] = np.cumsum(need)
    used = int(page_indptr[-1])
    assert used <= len(page_ids), "page pool too small for this batch"
    q_indptr = np.zeros(len(q_len) + 1, dtype=np.int64)
    q_indptr[1:] = np.cumsum(q_len)
    return (q_indptr.astype(np.int32), page_indptr.astype(np.int32),
            np.asarray(page_ids[:used], dtype=np.int32).copy(), used)


def make_single_step(name: str, shape: Shape, kv_len_before, q_len, seed: int,
                     spare_pages: int = 8, shuffle_pages: bool = True,
                     interleave_pages: bool = False, extra_pages=None,
                     poison_unused: bool = False) -> Workload:
    """A one-step workload with explicit per-sequence lengths.

    Physical page ids are a seeded permutation of the pool (``shuffle_pages``); with
    ``interleave_pages`` the pages of different sequences are additionally dealt round-robin.
    ``poison_unused`` overwrites every slot that no sequence owns after the append (tail slots of
    last pages, spare pages) with NaN / Inf / huge bf16 patterns.
    """
    kv_len_before = np.asarray(kv_len_before, dtype=np.int32)
    q_len = np.asarray(q_len, dtype=np.int32)
    P = shape.page_size
    need = _ceil_div(kv_len_before.astype(np.int64) + q_len, P)
    if extra_pages is not None:
        need = need + np.asarray(extra_pages, dtype=np.int64)
    total_pages = int(need.sum())
    num_pages = total_pages + int(spare_pages)
    g = _rng(seed, 1)
    ids = g.permutation(num_pages) if shuffle_pages else np.arange(num_pages)
    if interleave_pages:
        # deal pages one at a time to the sequences that still need one
        order = []
        left = need.copy()
        while left.sum() > 0:
            for b in np.nonzero(left > 0)[0]:
                order.append(b)
                left[b] -= 1
        order = np.asarray(order)
        dealt = ids[:total_pages]
        per_seq = [dealt[order == b] for b in range(len(need))]
        ids = np.concatenate(per_seq + [ids[total_pages:]]) if len(per_seq) else ids
    q_indptr, page_indptr, page_indices, _ = build_step_tables(
        kv_len_before, q_len, P, ids, extra_pages)
    T = int(q_indptr[-1])
    pool = normal_bf16(seed, 2, (num_pages, 2, shape.num_kv_heads, P, shape.head_dim))
    q = normal_bf16(seed, 3, (T, shape.num_q_heads, shape.head_dim))
    k_new = normal_bf16(seed, 4, (T, shape.num_kv_heads, shape.head_dim))
    v_new = normal_bf16(seed, 5, (T, shape.num_kv_heads, shape.head_dim))
    if poison_unused:
        owned = np.zeros((num_pages, P), dtype=bool)
        for b in range(len(need)):
            n_b = int(kv_len_before[b]) + int(q_len[b])
            pages = page_indices[page_indptr[b]:page_indptr[b + 1]]
            for j, pg in enumerate(pages):
                lo = j * P
                owned[pg, :max(0, min(P, n_b - lo))] = True
        patterns = np.array([0x7FC0, 0xFFC0, 0x7F80, 0xFF80, 0x7F7F, 0xFF7F], dtype=np.uint16)
        pg_idx, slot_idx = np.nonzero(~owned)
        fill = patterns[(pg_idx * 7 + slot_idx) % len(patterns)]
        pool[pg_idx, :, :, slot_idx, :] = fill[:, None, None, None]
    step = Step(q_indptr, kv_len_before, page_indptr, page_indices, q, k_new, v_new)
    return Workload(name, shape, num_pages, pool, [step], seed)


def _uniform_int(g: np.random.Generator, lo: int, hi: int, n: int) -> np.ndarray:
    """Integer-uniform on the closed range [lo, hi]."""
    return g.integers(lo, hi + 1, size=n, dtype=np.int64)


def _mixed_lengths(g, batch, ctx_lo, ctx_hi, n_interrupted, app_lo, app_hi):
    ctx = _uniform_int(g, ctx_lo, ctx_hi, batch)
    q_len = np.ones(batch, dtype=np.int64)
    who = g.permutation(batch)[:n_interrupted]
    q_len[who] = _uniform_int(g, app_lo, app_hi, n_interrupted)
    return ctx, q_len


def config_seed(c: int) -> int:
    return BASE_SEED + c


def make_config(c: int, seed: Optional[int] = None, scale: float = 1.0) -> Workload:
    """The five synthetic serving configurations.

    1 tiny mixed step, 2 Llama-3-8B attention shape, 3 large batch (GQA 8), 4 long context,
    5 interrupt-trace replay (see :func:`make_replay`).  ``scale`` < 1 shrinks context lengths
    (not the shape) for quick tests.
    """
    seed = config_seed(c) if seed is None else seed
    g = _rng(seed, 0)
    s = lambda x: max(1, int(round(x * scale)))
    if c == 1:
        shape = Shape(8, 2, 64, 16)
        ctx = _uniform_int(g, s(100), s(300), 4)
        q_len = np.array([12, 1, 1, 1])
        return make_single_step("tiny-mixed", shape, ctx, q_len, seed, spare_pages=8)
    if c == 2:
        shape = Shape(32, 8, 128, 16)
        ctx, q_len = _mixed_lengths(g, 32, s(512), s(4096), 8, 8, 64)
        return make_single_step("llama3-8b-mixed", shape, ctx, q_len, seed, spare_pages=64)
    if c == 3:
        shape = Shape(64, 8, 128, 16)
        ctx, q_len = _mixed_lengths(g, 128, s(2048), s(8192), 13, 16, 128)
        return make_single_step("large-batch", shape, ctx, q_len, seed, spare_pages=64)
    if c == 4:
        shape = Shape(32, 8, 128, 16)
        ctx = _uniform_int(g, s(32768), s(131072), 8)
        q_len = np.ones(8, dtype=np.int64)
        q_len[g.permutation(8)[:2]] = 256
        return make_single_step("long-context", shape, ctx, q_len, seed, spare_pages=64)
    if c == 5:
        return make_replay(seed=seed, scale=scale)
    raise ValueError(f"unknown config {c}")


def make_replay(seed: Optional[int] = None, batch: int = 256, steps: int = 200,
                ctx_lo: int = 256, ctx_hi: int = 2048, rate: float = 0.02,
                app_lo: int = 8, app_hi: int = 96, shape: Optional[Shape] = None,
                scale: float = 1.0, materialize: bool = True) -> Workload:
    """Interrupt-trace replay: ``steps`` consecutive decode steps over ``batch`` sequences.

    Every sequence decodes one token per step.  Interrupt arrivals are Poisson(``rate``) per
    sequence per step; each arrival carries a span of uniform [app_lo, app_hi] tokens and all
    arrivals of one sequence in one step are concatenated behind the sampled token (Section 5.3:
    every queued interrupt is appended together).  Pages come from a free list (a seeded
    permutation, popped from the end) one page at a time as sequences grow; the initial contexts
    are allocated round-robin so physical pages of different sequences interleave.  Nothing is
    freed during the trace.

    Each returned Step carries the full page table of that step.  The pool holds the initial
    contexts; later steps rely on earlier steps' appends having been applied in order.
    """
    seed = config_seed(5) if seed is None else seed
    shape = shape or Shape(32, 8, 128, 16)
    P = shape.page_size
    g = _rng(seed, 0)
    ctx0 = _uniform_int(g, max(1, int(ctx_lo * scale)), max(1, int(ctx_hi * scale)), batch)
    arrivals = g.poisson(rate, size=(steps, batch))
    q_lens = np.ones((steps, batch), dtype=np.int64)
    for t, b in zip(*np.nonzero(arrivals)):
        q_lens[t, b] += int(_uniform_int(g, app_lo, app_hi, int(arrivals[t, b])).sum())
    final = ctx0 + q_lens.sum(axis=0)
    num_pages = int(_ceil_div(final, P).sum()) + 64
    free = list(_rng(seed, 1).permutation(num_pages))
    tables: List[List[int]] = [[] for _ in range(batch)]
    need0 = _ceil_div(ctx0, P)
    for j in range(int(need0.max())):
        for b in range(batch):
            if j < need0[b]:
                tables[b].append(free.pop())
    pool = normal_bf16(seed, 2, (num_pages, 2, shape.num_kv_heads, P, shape.head_dim)) \
        if materialize else np.empty((0,), dtype=np.uint16)
    wl = Workload("interrupt-replay", shape, num_pages, pool, [], seed)
    ctx = ctx0.copy()
    for t in range(steps):
        ql = q_lens[t]
        for b in range(batch):
            while len(tables[b]) * P < ctx[b] + ql[b]:
                tables[b].append(free.pop())
        page_indptr = np.zeros(batch + 1, dtype=np.int32)
        page_indptr[1:] = np.cumsum([len(x) for x in tables])
        page_indices = np.fromiter((p for x in tables for p in x), dtype=np.int32,
                                   count=int(page_indptr[-1]))
        q_indptr = np.zeros(batch + 1, dtype=np.int32)
        q_indptr[1:] = np.cumsum(ql)
        T = int(q_indptr[-1])
        if materialize:
            q = normal_bf16(seed, 1000 + 3 * t, (T, shape.num_q_heads, shape.head_dim))
            kn = normal_bf16(seed, 1001 + 3 * t, (T, shape.num_kv_heads, shape.head_dim))
            vn = normal_bf16(seed, 1002 + 3 * t, (T, shape.num_kv_heads, shape.head_dim))
        else:
            q = kn = vn = np.empty((0,), dtype=np.uint16)
        wl.steps.append(Step(q_indptr, ctx.astype(np.int32), page_indptr, page_indices, q, kn, vn))
        ctx = ctx + ql
    return wl


# --------------------------------------------------------------------------------------------
# byte / flop accounting for reports (counts only; no attention arithmetic)
# --------------------------------------------------------------------------------------------

def algorithmic_bytes(shape: Shape, step: Step) -> dict:
    """Bytes one step must move, each counted once: the KV of every visible token, Q read, O
    written, the new K/V rows read and written, and the page ids."""
    n = step.kv_len_before.astype(np.int64) + step.q_len
    active = step.q_len > 0
    T = step.total_q
    kv = int(n[active].sum()) * shape.kv_bytes_per_token
    qo = 2 * T * shape.num_q_heads * shape.head_dim * 2
    app = 2 * T * shape.kv_bytes_per_token
    pages = 4 * int(_ceil_div(n[active], shape.page_size).sum())
    return {"kv": kv, "qo": qo, "append": app, "page_ids": pages, "total": kv + qo + app + pages}


def algorithmic_flops(shape: Shape, step: Step) -> int:
    """4 * d * Hq * (number of (query row, visible key) pairs)."""
    ctx = step.kv_len_before.astype(np.int64)
    ql = step.q_len.astype(np.int64)
    pairs = int((ql * ctx + ql * (ql + 1) // 2).sum())
    return 4 * shape.head_dim * shape.num_q_heads * pairs
