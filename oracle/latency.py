"""CPU oracle of the paper's latency model (TEST INFRASTRUCTURE ONLY).

Section 6.3 ("Latency Analysis") and Appendix A: for a set F of independent function calls with
token-generation latency G(f) and execution time E(f),

    L_Sync(F)    = sum G + sum E                      generate and execute one after the other
    L_SyncPar(F) = sum G + max E                      generate all, execute them concurrently
    L_Async(F)   = max_f ( E(f) + sum_{g in pred(f)} G(g) ),   pred(f) = { g : E(f) <= E(g) }

(the last under the longest-processing-time-first order), and the speed-up L_Sync / L_Async is about
1 + mean(E) / mean(G) for large F (Theorem 6.2).  `schedule_latency` is the appendix's completion-time
recurrence for an arbitrary generation order, C(f_i) = G(f_1) + ... + G(f_i) + E(f_i).

Pins (tests/test_latency_pins.py): Theorem 6.1's chain of inequalities on random draws; Theorem 6.3 by
brute force (no permutation of up to 7 calls beats the closed form, and the LPT order attains it); the
closed form against the recurrence under ties; Theorem 6.2's estimate on a large normal draw.
"""
from __future__ import annotations

import numpy as np


def l_sync(gen, exe) -> float:
    return float(np.sum(gen) + np.sum(exe))


def l_sync_par(gen, exe) -> float:
    return float(np.sum(gen) + np.max(exe))


def l_async(gen, exe) -> float:
    gen, exe = np.asarray(gen, dtype=np.float64), np.asarray(exe, dtype=np.float64)
    best = -np.inf
    for f in range(len(exe)):
        pred = exe[f] <= exe                       # every call at least as long as f, f included
        best = max(best, exe[f] + gen[pred].sum())
    return float(best)


def schedule_latency(gen, exe, order) -> float:
    """Generation in the given order, every call starts when its tokens are out."""
    t, worst = 0.0, 0.0
    for i in order:
        t += gen[i]
        worst = max(worst, t + exe[i])
    return float(worst)


def speedup_estimate(gen, exe) -> float:
    return float(1.0 + np.mean(exe) / np.mean(gen))
