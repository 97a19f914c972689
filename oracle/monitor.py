"""CPU oracle of the token monitor's sampling hook (TEST INFRASTRUCTURE ONLY).

Paper Section 5.1 ("Token Monitor"): a finite-state machine over CML (Section 3) constrains the
next-token distribution so that generated tokens follow CML syntax, and the model can never produce
[INTR] (interrupts are injected by the system, Section 3.2); after each token the monitor reports a
finished function call or trap and whether generation is inside a function-call block (the critical
section during which interrupts are deferred).

CML as the model may generate it (Section 3.1-3.2):
    [CALL] {function call} [END]          [CALL] {id} [HEAD] {function call} [END]          [TRAP] [END]
States: TEXT (outside a block), CALL (after [CALL], no [HEAD] yet), BODY (after [HEAD]), TRAP (after
[TRAP]).  Decoding here is greedy: the allowed token with the largest logit, the lowest id among equals;
NaN logits are never chosen; if no allowed token has a logit above -inf, the lowest allowed id is taken.  The paper does not fix a sampling rule; this reading is recorded in
the design doc.  Nothing here imports, or is imported by, the CUDA package.
"""
from __future__ import annotations

import numpy as np

TEXT, CALL, BODY, TRAP = 0, 1, 2, 3
EV_CALL, EV_TRAP, CRITICAL = 1, 2, 4          # flag bits: a call block closed, a trap closed, inside a call block


def allowed(state: int, special: dict, vocab: int) -> np.ndarray:
    """Boolean mask over the vocabulary for one state.  special: name -> token id."""
    ok = np.ones(vocab, dtype=bool)
    for t in special.values():
        ok[t] = False                              # specials only where the grammar says so
    if state == TEXT:
        ok[special["CALL"]] = ok[special["TRAP"]] = True
    elif state == CALL:
        ok[special["HEAD"]] = ok[special["END"]] = True
    elif state == BODY:
        ok[special["END"]] = True
    elif state == TRAP:
        ok[:] = False
        ok[special["END"]] = True
    return ok                                      # [INTR] is never allowed


def advance(state: int, token: int, special: dict):
    """(next state, flags) after `token` was generated in `state`."""
    nxt, flags = state, 0
    if state == TEXT:
        if token == special["CALL"]:
            nxt = CALL
        elif token == special["TRAP"]:
            nxt = TRAP
    elif state in (CALL, BODY):
        if token == special["HEAD"] and state == CALL:
            nxt = BODY
        elif token == special["END"]:
            nxt, flags = TEXT, EV_CALL
    elif state == TRAP:
        if token == special["END"]:
            nxt, flags = TEXT, EV_TRAP
    if nxt in (CALL, BODY):
        flags |= CRITICAL
    return nxt, flags


def step(logits: np.ndarray, states, special: dict):
    """One decoding step for a batch: (tokens, next states, flags)."""
    logits = np.asarray(logits, dtype=np.float64)
    B, V = logits.shape
    toks, nxts, flags = np.zeros(B, np.int32), np.zeros(B, np.int32), np.zeros(B, np.int32)
    for b in range(B):
        ok = allowed(int(states[b]), special, V) & ~np.isnan(logits[b])
        cand = np.where(ok, logits[b], -np.inf)
        if np.isneginf(cand).all():
            toks[b] = int(np.argmax(allowed(int(states[b]), special, V)))      # nothing to compare: lowest allowed id
        else:
            toks[b] = int(np.argmax(cand))         # first index of the maximum
        nxts[b], flags[b] = advance(int(states[b]), int(toks[b]), special)
    return toks, nxts, flags
