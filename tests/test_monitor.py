"""Token monitor kernel (paper Section 5.1) against the oracle: chosen tokens, states and flags are
integers, so the comparison is exact."""
import numpy as np
import pytest

from oracle import monitor as M
from paper_2412_07017_b200 import binding as B
from paper_2412_07017_b200 import workload as W

pytestmark = pytest.mark.gpu


def run(logits_bits_or_f32, states, special, bf16):
    import torch
    # rows start on 16-byte boundaries: the row stride is the vocabulary rounded up to 8 elements
    n, vocab = logits_bits_or_f32.shape
    stride = -(-vocab // 8) * 8
    if bf16:
        full = torch.zeros((n, stride), dtype=torch.bfloat16, device="cuda")
        full[:, :vocab] = torch.from_numpy(logits_bits_or_f32.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        full = torch.zeros((n, stride), dtype=torch.float32, device="cuda")
        full[:, :vocab] = torch.from_numpy(logits_bits_or_f32).cuda()
    logits = full[:, :vocab]
    st = torch.from_numpy(np.asarray(states, dtype=np.int32)).cuda()
    tok, nxt, fl = (torch.full_like(st, -7) for _ in range(3))
    ws = torch.zeros(B.token_monitor_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    B.asynclm_token_monitor_step(logits, special, st, tok, nxt, fl, ws)
    first = (tok.clone(), nxt.clone(), fl.clone())
    tok.fill_(-7)
    B.asynclm_token_monitor_step(logits, special, st, tok, nxt, fl, ws)      # the workspace came back zeroed
    torch.cuda.synchronize()
    assert int(ws.max()) == 0 and all(torch.equal(a, b) for a, b in zip(first, (tok, nxt, fl)))
    return tok.cpu().numpy(), nxt.cpu().numpy(), fl.cpu().numpy()


@pytest.mark.parametrize("vocab,bf16", [(128256, True), (32000, True), (1003, False), (50257, False)])
def test_batch_of_states_matches_the_oracle(vocab, bf16):
    g = np.random.default_rng(vocab)
    Bsz = 37
    special = dict(zip(("CALL", "INTR", "TRAP", "END", "HEAD"), g.permutation(vocab)[:5].tolist()))
    if bf16:
        bits = W.normal_bf16(5, 1, (Bsz, vocab))
        vals = W.bf16_bits_to_f64(bits)
    else:
        vals32 = g.normal(size=(Bsz, vocab)).astype(np.float32)
        bits, vals = vals32, vals32.astype(np.float64)
    states = g.integers(0, 4, Bsz)
    # push the interesting tokens to the top of some rows, ties and NaNs into others
    for b in range(Bsz):
        pick = [special["INTR"], special["END"], special["CALL"], special["HEAD"], special["TRAP"]][b % 5]
        if b % 3 == 0:
            vals[b, pick] = 30.0
        if b % 7 == 0:
            vals[b, special["INTR"]] = 40.0
        if b % 11 == 0:
            vals[b, [17, 900]] = 35.0
        if b % 13 == 0:
            vals[b, 5:50] = np.nan
    if bf16:
        bits = W.f32_to_bf16_bits(np.nan_to_num(vals, nan=0.0).astype(np.float32))
        nan_bits = np.uint16(0x7FC0)
        bits[np.isnan(vals)] = nan_bits
        vals = W.bf16_bits_to_f64(bits)
    else:
        bits = vals.astype(np.float32)
        vals = bits.astype(np.float64)
    tok, nxt, fl = run(bits, states, special, bf16)
    rt, rn, rf = M.step(vals, states, special)
    assert np.array_equal(tok, rt) and np.array_equal(nxt, rn) and np.array_equal(fl, rf)
    assert special["INTR"] not in tok


def test_a_cml_call_is_generated_token_by_token():
    """Logits that spell [CALL] id [HEAD] body [END] [TRAP] [END]: the device state machine walks the
    blocks, raises the call and the trap, and defers interrupts inside the call block."""
    vocab = 4096
    special = {"CALL": 100, "INTR": 101, "TRAP": 102, "END": 103, "HEAD": 104}
    want = [100, 7, 104, 8, 9, 103, 55, 102, 103]
    state = np.array([M.TEXT], dtype=np.int32)
    ref_state = M.TEXT
    seen = []
    for step, t in enumerate(want):
        vals = np.zeros((1, vocab), dtype=np.float32)
        vals[0, t] = 5.0
        vals[0, special["INTR"]] = 9.0          # always the largest logit, never allowed
        tok, nxt, fl = run(vals, state, special, False)
        ref_state, ref_fl = M.advance(ref_state, t, special)
        assert tok[0] == t and nxt[0] == ref_state and fl[0] == ref_fl
        seen.append(int(fl[0]))
        state = nxt
    assert seen == [4, 4, 4, 4, 4, 1, 0, 0, 2]


def test_degenerate_rows():
    vocab = 1024
    special = {"CALL": 3, "INTR": 0, "TRAP": 1, "END": 2, "HEAD": 9}
    vals = np.full((4, vocab), np.nan, dtype=np.float32)
    vals[1, :] = -np.inf
    states = [M.TEXT, M.CALL, M.BODY, M.TRAP]
    tok, nxt, fl = run(vals, states, special, False)
    rt, rn, rf = M.step(vals.astype(np.float64), states, special)
    assert np.array_equal(tok, rt) and np.array_equal(nxt, rn) and np.array_equal(fl, rf)
