"""CPU oracle of the trap handler's data path and decision rule (TEST INFRASTRUCTURE ONLY).

What it follows (paper Section 5.4, "Trap Handler", and the example in Section 6.4, "Trap handling
strategy"): while a sequence waits for an interrupt its KV cache may stay in GPU memory, be swapped
to host memory (cost linear in the context length) or be dropped and recomputed (cost quadratic in
the context length).  The cache stays where it is if both the swap time and the recompute time are
longer than the estimated wait; otherwise the cheaper of the two is taken.

The data path is plain copying: swapping a sequence out gathers its pages, in logical order, into
one contiguous image; swapping it in scatters the image into whatever pages it is given then.
Nothing here imports, or is imported by, the CUDA package.

Pins (tests/test_trap_pins.py): a swap-out / swap-in round trip into other pages leaves the sequence's
logical view unchanged byte for byte and touches no other page; the rule's boundary cases and
monotonicity in the wait; the paper's own worked example (next interrupt in 100 ms, 300 tokens of
context: recompute on the smaller model, swap on the larger one) under cost models ordered as the
paper orders them.
"""
from __future__ import annotations

import numpy as np

KEEP, SWAP, RECOMPUTE = 0, 1, 2


def swap_out(kv_pool: np.ndarray, page_ids) -> np.ndarray:
    """Image of a sequence: its pages in logical order, [n_pages][2][Hkv][P][d] (a copy)."""
    return kv_pool[np.asarray(page_ids, dtype=np.int64)].copy()


def swap_in(kv_pool: np.ndarray, page_ids, image: np.ndarray) -> None:
    """Put an image back, logical page j into physical page page_ids[j] (in place)."""
    ids = np.asarray(page_ids, dtype=np.int64)
    assert image.shape[0] == len(ids) and len(set(ids.tolist())) == len(ids)
    kv_pool[ids] = image


def swap_us(model: dict, tokens: int) -> float:
    """Linear: fixed cost plus a cost per token of context."""
    return model["swap_fixed_us"] + model["swap_us_per_token"] * tokens


def recompute_us(model: dict, tokens: int) -> float:
    """Quadratic: fixed cost, a cost per token and a cost per pair of tokens."""
    return (model["recompute_fixed_us"] + model["recompute_us_per_token"] * tokens +
            model["recompute_us_per_token2"] * tokens * tokens)


def decide(model: dict, tokens: int, wait_us: float) -> int:
    """Section 5.4: keep if both alternatives take longer than the wait, else the cheaper one."""
    s, r = swap_us(model, tokens), recompute_us(model, tokens)
    if s > wait_us and r > wait_us:
        return KEEP
    return RECOMPUTE if r < s else SWAP
