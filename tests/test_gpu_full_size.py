"""GPU parity at the full sizes of the large configurations, in the default launch configuration.

The oracle cannot evaluate every row of these batches in reasonable time, so it is run on a seeded
sample of token rows (every interrupted sequence contributes rows from the start, middle and end of
its span; decode rows are drawn at random), all heads.  The KV pool is compared bit for bit in full.
Bars as everywhere: max |err| <= 1e-2, mean |err| <= 1e-3, lse within 1e-3.
"""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2412_07017_b200 import workload as W
from gpu_util import assert_close, gpu_step, to_bits, to_dev

pytestmark = pytest.mark.gpu


def sample_rows(st, n_decode, seed):
    rng = np.random.default_rng(seed)
    rows = []
    dec = []
    for b in range(st.batch):
        q0, q1 = int(st.q_indptr[b]), int(st.q_indptr[b + 1])
        if q1 - q0 > 1:
            rows += [q0, q0 + 1, (q0 + q1) // 2, q1 - 2, q1 - 1]
            # rows next to the query-tile boundaries of the tensor-core path (32 tokens at G = 4, 16 at G = 8)
            rows += [r for r in (q0 + 15, q0 + 16, q0 + 31, q0 + 32, q0 + 33, q0 + 63, q0 + 64, q0 + 127, q0 + 128)
                     if r < q1]
        elif q1 - q0 == 1:
            dec.append(q0)
    dec = np.array(dec)
    if len(dec):
        rows += list(rng.choice(dec, size=min(n_decode, len(dec)), replace=False))
    return np.unique(np.array(rows, dtype=np.int32))


def check_step(wl, st, pool_dev, ref_pool, rows, what):
    pool_dev, out, lse, plan = gpu_step(wl, st, pool_dev=pool_dev)
    oracle.kv_append(ref_pool, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                     st.k_new, st.v_new)
    ref_out, ref_lse = oracle.attn_mixed(ref_pool, st.q, st.q_indptr, st.kv_len_before, st.page_indptr,
                                         st.page_indices, sel_rows=rows)
    assert_close(out, lse, ref_out, ref_lse, rows=rows, what=what)
    assert np.isfinite(W.bf16_bits_to_f64(out)).all(), f"{what}: non-finite output outside the sample"
    return pool_dev, plan


def test_config3_large_batch_gqa8():
    wl = W.make_config(3)
    st = wl.steps[0]
    assert st.batch == 128 and (st.q_len > 1).sum() == 13 and wl.shape.group == 8
    ref_pool = wl.kv_pool.copy()
    pool_dev, plan = check_step(wl, st, None, ref_pool, sample_rows(st, 12, 3), "config3")
    assert np.array_equal(to_bits(pool_dev), ref_pool), "config3: pool differs after append"
    assert plan.info["num_items_tensor"] > 0


def test_config4_long_context_split_kv():
    wl = W.make_config(4)
    st = wl.steps[0]
    assert st.batch == 8 and sorted(st.q_len)[-2:] == [256, 256]
    assert st.kv_len_before.min() >= 32768
    ref_pool = wl.kv_pool.copy()
    pool_dev, plan = check_step(wl, st, None, ref_pool, sample_rows(st, 3, 4), "config4")
    assert np.array_equal(to_bits(pool_dev), ref_pool), "config4: pool differs after append"
    assert plan.info["num_split_units"] > 0 and plan.info["num_items_tensor"] > 0


def test_config5_interrupt_trace_replay():
    wl = W.make_replay()
    assert len(wl.steps) == 200 and wl.steps[0].batch == 256
    pool_dev = to_dev(wl.kv_pool)
    ref_pool = wl.kv_pool.copy()
    interrupted_steps = 0
    for t, st in enumerate(wl.steps):
        interrupted_steps += int((st.q_len > 1).any())
        if t % 40 == 0 or t == len(wl.steps) - 1:
            pool_dev, _ = check_step(wl, st, pool_dev, ref_pool, sample_rows(st, 6, 500 + t), f"replay step {t}")
        else:
            pool_dev, out, _, _ = gpu_step(wl, st, pool_dev=pool_dev, want_lse=False)
            oracle.kv_append(ref_pool, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                             st.k_new, st.v_new)
    assert interrupted_steps > 100
    assert np.array_equal(to_bits(pool_dev), ref_pool), "replay: pool differs after 200 steps"
