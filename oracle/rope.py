"""CPU oracle of the rotary position embedding applied to new key rows (TEST INFRASTRUCTURE ONLY).

The paper serves Llama-3 models (Section 6, setup); their attention rotates every query and key by its
position before the keys are cached.  A multi-layer serving step therefore writes ROTATED key rows in
the interrupt append (Section 3.2: the block goes to the end of the context, so new token i of a
sequence has position ctx + i).  The rotation is the published rotary embedding in its "rotate-half"
form: with d the head dimension and theta the base,
    angle_j = pos * theta^(-2 j / d),                 j = 0 .. d/2 - 1
    out[j]       = x[j] cos(angle_j) - x[j + d/2] sin(angle_j)
    out[j + d/2] = x[j + d/2] cos(angle_j) + x[j] sin(angle_j)
evaluated in fp64 here and rounded to bf16 (nearest even) once at the end.  Values are untouched by
anything but that rotation.  Nothing here imports, or is imported by, the CUDA package.

Pins (tests/test_rope_pins.py): position 0 is the identity bit for bit; the rotation preserves the norm
of every (j, j + d/2) pair; rotating by p then by q equals rotating by p + q; the dot product of a
rotated query and key depends only on the position difference; a hand-computed 2-d case.
"""
from __future__ import annotations

import numpy as np


def rotate(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """x: float64 [..., T, H, d]; pos: int [T]; returns float64 of the same shape."""
    d = x.shape[-1]
    j = np.arange(d // 2, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * theta ** (-2.0 * j / d)      # [T, d/2]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)
