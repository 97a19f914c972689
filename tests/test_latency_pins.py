"""Pins of the latency-model oracle (oracle/latency.py) and the library's calculator against it."""
import itertools

import numpy as np
import pytest

from oracle import latency as L
from paper_2412_07017_b200 import binding as B


def draws(seed, n):
    g = np.random.default_rng(seed)
    return g.uniform(0.05, 2.0, n), g.uniform(0.05, 5.0, n)


@pytest.mark.parametrize("seed", range(8))
def test_theorem_6_1_chain(seed):
    gen, exe = draws(seed, 2 + seed * 3)
    assert L.l_async(gen, exe) <= L.l_sync_par(gen, exe) + 1e-12
    assert L.l_sync_par(gen, exe) < L.l_sync(gen, exe)
    # hand-checkable case: two calls, G = (1, 2), E = (5, 1): LPT issues the long one first
    assert L.l_sync([1, 2], [5, 1]) == 9 and L.l_sync_par([1, 2], [5, 1]) == 8
    assert L.l_async(np.array([1.0, 2.0]), np.array([5.0, 1.0])) == 6          # max(1 + 5, 1 + 2 + 1)


@pytest.mark.parametrize("n", [2, 3, 5, 7])
def test_theorem_6_3_no_order_beats_lpt(n):
    gen, exe = draws(100 + n, n)
    best = min(L.schedule_latency(gen, exe, p) for p in itertools.permutations(range(n)))
    lpt = sorted(range(n), key=lambda i: -exe[i])
    assert L.schedule_latency(gen, exe, lpt) == pytest.approx(best, abs=1e-12)
    assert L.l_async(gen, exe) == pytest.approx(best, abs=1e-12)


def test_ties_in_execution_time():
    gen, exe = np.array([0.5, 1.5, 1.0, 2.0]), np.array([3.0, 3.0, 1.0, 3.0])
    best = min(L.schedule_latency(gen, exe, p) for p in itertools.permutations(range(4)))
    assert L.l_async(gen, exe) == pytest.approx(best)


def test_theorem_6_2_estimate_for_many_calls():
    g = np.random.default_rng(5)
    n = 4000
    gen = g.uniform(0.9, 1.1, n)
    exe = np.abs(g.normal(0.2, 0.05, n))
    ratio = L.l_sync(gen, exe) / L.l_async(gen, exe)
    est = L.speedup_estimate(gen, exe)
    assert abs(ratio - est) <= (np.mean(exe) / np.mean(gen)) ** 2 + 5.0 / n


@pytest.mark.parametrize("seed", range(6))
def test_library_calculator_matches_the_oracle(seed):
    gen, exe = draws(200 + seed, 1 + seed * 7)
    out = B.asynclm_latency_model(gen, exe)
    assert out["l_sync"] == pytest.approx(L.l_sync(gen, exe))
    assert out["l_sync_par"] == pytest.approx(L.l_sync_par(gen, exe))
    assert out["l_async"] == pytest.approx(L.l_async(gen, exe))
    assert out["speedup_estimate"] == pytest.approx(L.speedup_estimate(gen, exe))
    order = np.random.default_rng(seed).permutation(len(gen)).astype(np.int32)
    lat, done = B.asynclm_async_latency_of_order(gen, exe, order)
    assert lat == pytest.approx(L.schedule_latency(gen, exe, order))
    assert done.max() == pytest.approx(lat)
    # the LPT order the library reports attains the closed form
    assert B.asynclm_async_latency_of_order(gen, exe, out["lpt_order"])[0] == pytest.approx(out["l_async"])


def test_library_calculator_rejects_bad_input():
    with pytest.raises(B.AsynclmError):
        B.asynclm_latency_model([1.0, -1.0], [1.0, 1.0])
    with pytest.raises(B.AsynclmError):
        B.asynclm_async_latency_of_order([1.0, 1.0], [1.0, 1.0], np.array([0, 0], dtype=np.int32))
