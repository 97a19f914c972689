"""Pins of the rotary-embedding oracle (oracle/rope.py)."""
import numpy as np

from oracle import rope


def test_identity_norm_composition_and_relative_position():
    g = np.random.default_rng(0)
    x = g.normal(size=(6, 3, 64))
    pos = np.array([0, 1, 5, 77, 1000, 4095])
    y = rope.rotate(x, pos, 500000.0)
    assert np.array_equal(y[0], x[0])                                             # position 0: nothing moves
    pair = lambda a: a[..., :32] ** 2 + a[..., 32:] ** 2
    assert np.allclose(pair(y), pair(x), rtol=1e-12)                               # rotations keep pair norms
    p, q = np.array([3, 3, 3, 3, 3, 3]), np.array([10, 0, 2, 5, 100, 7])
    assert np.allclose(rope.rotate(rope.rotate(x, p, 1e4), q, 1e4), rope.rotate(x, p + q, 1e4), atol=1e-12)
    # <R(m) a, R(n) b> depends on m - n only
    a, b = g.normal(size=(1, 1, 64)), g.normal(size=(1, 1, 64))
    dot = lambda m, n: float((rope.rotate(a, np.array([m]), 1e4) * rope.rotate(b, np.array([n]), 1e4)).sum())
    assert abs(dot(9, 4) - dot(105, 100)) < 1e-10 and abs(dot(9, 4) - dot(5, 0)) < 1e-10


def test_hand_computed_two_dimensional_case():
    # d = 2: one pair, angle = pos * theta^0 = pos radians; (1, 0) at position pi/2 would be (0, 1)
    x = np.array([[[1.0, 0.0]], [[0.0, 2.0]]])
    y = rope.rotate(x, np.array([1, 2]), 12345.0)
    assert np.allclose(y[0, 0], [np.cos(1.0), np.sin(1.0)])
    assert np.allclose(y[1, 0], [-2 * np.sin(2.0), 2 * np.cos(2.0)])
