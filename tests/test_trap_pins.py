"""Pins of the trap-handler oracle (oracle/trap.py): copy semantics and the decision rule."""
import numpy as np

from oracle import trap


def test_round_trip_into_other_pages_keeps_the_logical_view_and_nothing_else():
    g = np.random.default_rng(1)
    pool = g.integers(0, 1 << 16, size=(40, 2, 2, 16, 64), dtype=np.uint16)
    before = pool.copy()
    old = g.permutation(40)[:9]
    image = trap.swap_out(pool, old)
    # written independently of the function under test: one page at a time, by index
    for j, pg in enumerate(old):
        assert np.array_equal(image[j], before[pg])
    pool[old] = 0xFFFF                                  # the pages are given to someone else
    free = np.setdiff1d(np.arange(40), old)
    new = g.permutation(free)[:9]
    untouched = np.setdiff1d(np.arange(40), new)
    snapshot = pool.copy()
    trap.swap_in(pool, new, image)
    for j in range(9):
        assert np.array_equal(pool[new[j]], before[old[j]])
    assert np.array_equal(pool[untouched], snapshot[untouched])


def _model(swap_per_token, rec_per_token2):
    return dict(swap_fixed_us=50.0, swap_us_per_token=swap_per_token, recompute_fixed_us=20.0,
                recompute_us_per_token=1.0, recompute_us_per_token2=rec_per_token2)


def test_rule_boundaries_and_monotonicity():
    m = _model(10.0, 0.05)
    n = 200
    s, r = trap.swap_us(m, n), trap.recompute_us(m, n)
    assert s == 50.0 + 2000.0 and r == 20.0 + 200.0 + 0.05 * 40000
    assert r > s
    assert trap.decide(m, n, wait_us=min(s, r) - 1.0) == trap.KEEP          # both longer than the wait
    assert trap.decide(m, n, wait_us=min(s, r) + 1.0) == trap.SWAP          # the cheaper one fits
    assert trap.decide(m, n, wait_us=1e12) == trap.SWAP
    small = 20                                                              # few tokens: recompute is cheaper
    assert trap.recompute_us(m, small) < trap.swap_us(m, small)
    assert trap.decide(m, small, wait_us=1e12) == trap.RECOMPUTE
    # once the rule stops keeping, a longer wait never brings "keep" back
    kept = [trap.decide(m, n, w) == trap.KEEP for w in np.linspace(0, 2 * max(s, r), 200)]
    assert kept == sorted(kept, reverse=True)
    # the linear and the quadratic cost cross exactly once beyond the start
    choice = [trap.decide(m, k, 1e12) for k in range(1, 2000)]
    flips = sum(a != b for a, b in zip(choice[:-1], choice[1:]))
    assert choice[0] == trap.RECOMPUTE and choice[-1] == trap.SWAP and flips == 1


def test_papers_worked_example():
    with open(__file__.replace("test_trap_pins.py", "golden/trap_example.txt")) as f:
        row = [l.split() for l in f if l.strip() and not l.startswith("#")][0]
    wait_us, tokens = float(row[0]) * 1e3, int(row[1])
    names = {"keep": trap.KEEP, "swap": trap.SWAP, "recompute": trap.RECOMPUTE}
    # two cost models ordered as the paper orders its two models: the same swap slope per byte, more
    # bytes and far more recomputation on the larger model; both alternatives fit into the wait
    small = dict(swap_fixed_us=500.0, swap_us_per_token=60.0, recompute_fixed_us=3000.0,
                 recompute_us_per_token=30.0, recompute_us_per_token2=0.02)
    large = dict(swap_fixed_us=500.0, swap_us_per_token=110.0, recompute_fixed_us=6000.0,
                 recompute_us_per_token=120.0, recompute_us_per_token2=0.08)
    assert trap.recompute_us(large, tokens) > trap.recompute_us(small, tokens)
    assert max(trap.swap_us(large, tokens), trap.recompute_us(large, tokens)) < wait_us
    assert trap.decide(small, tokens, wait_us) == names[row[2]]
    assert trap.decide(large, tokens, wait_us) == names[row[3]]
