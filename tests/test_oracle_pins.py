"""Pins for the CPU oracle: it is checked against things other than itself.

Each test would fail under a plausible mistake in the oracle: a wrong causal limit, a dropped
scale, K and V swapped, a transposed page index, a wrong GQA head map, a missing normalisation.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2412_07017_b200 import workload as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def gather_dense(pool, st, b):
    """Logical K, V [n, Hkv, d] float64 of sequence b read through the page table (numpy)."""
    P = pool.shape[3]
    n = int(st.kv_len_before[b]) + int(st.q_len[b])
    pages = st.page_indices[st.page_indptr[b]:st.page_indptr[b + 1]]
    k = np.concatenate([pool[p, 0].transpose(1, 0, 2) for p in pages], axis=0)[:n]
    v = np.concatenate([pool[p, 1].transpose(1, 0, 2) for p in pages], axis=0)[:n]
    return W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(v)


def dense_twin(pool_after, st, shape, scale=None):
    """Separately written evaluation: explicit score matrix with -inf mask, numpy einsum."""
    Hq, Hkv, d = shape.num_q_heads, shape.num_kv_heads, shape.head_dim
    G = Hq // Hkv
    scale = scale or 1.0 / math.sqrt(d)
    T = st.total_q
    out = np.zeros((T, Hq, d))
    lse = np.zeros((T, Hq))
    for b in range(st.batch):
        ql = int(st.q_len[b])
        if ql == 0:
            continue
        ctx = int(st.kv_len_before[b])
        k, v = gather_dense(pool_after, st, b)                  # [n, Hkv, d]
        q = W.bf16_bits_to_f64(st.q[st.q_indptr[b]:st.q_indptr[b + 1]])   # [ql, Hq, d]
        kk = np.repeat(k, G, axis=1)                            # [n, Hq, d]
        vv = np.repeat(v, G, axis=1)
        s = np.einsum("ihd,jhd->hij", q, kk) * scale            # [Hq, ql, n]
        mask = np.arange(ctx + ql)[None, :] > (ctx + np.arange(ql))[:, None]
        s = np.where(mask[None], -np.inf, s)
        m = s.max(axis=-1, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=-1, keepdims=True)
        o = np.einsum("hij,jhd->ihd", e / z, vv)
        out[st.q_indptr[b]:st.q_indptr[b + 1]] = o
        lse[st.q_indptr[b]:st.q_indptr[b + 1]] = (m + np.log(z))[..., 0].T
    return out, lse


def run_oracle(wl, step_idx=0, scale=0.0):
    st = wl.steps[step_idx]
    pool = wl.kv_pool.copy()
    out, lse = oracle.step(pool, st, scale)
    return pool, out, lse


# ------------------------------------------------------------------------------------------
# append
# ------------------------------------------------------------------------------------------

def test_append_is_a_bit_copy_to_the_right_slots_only():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("t", shape, [5, 16, 31, 0, 40], [12, 1, 2, 7, 0], seed=11,
                            extra_pages=[0, 1, 0, 2, 1])
    st = wl.steps[0]
    pool = wl.kv_pool.copy()
    oracle.kv_append(pool, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                     st.k_new, st.v_new)
    expect = wl.kv_pool.copy()
    for b in range(st.batch):
        for i in range(int(st.q_len[b])):
            pos = int(st.kv_len_before[b]) + i
            pg = st.page_indices[st.page_indptr[b] + pos // 16]
            r = st.q_indptr[b] + i
            expect[pg, 0, :, pos % 16, :] = st.k_new[r]
            expect[pg, 1, :, pos % 16, :] = st.v_new[r]
    assert np.array_equal(pool, expect)
    assert (pool != wl.kv_pool).sum() > 0
    # idempotent
    again = pool.copy()
    oracle.kv_append(again, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                     st.k_new, st.v_new)
    assert np.array_equal(again, pool)


def test_append_rejects_short_page_table():
    shape = W.Shape(4, 2, 64, 16)
    wl = W.make_single_step("t", shape, [16], [1], seed=3)
    st = wl.steps[0]
    bad_indptr = st.page_indptr.copy()
    bad_indptr[1] -= 1
    with pytest.raises(ValueError):
        oracle.kv_append(wl.kv_pool.copy(), st.q_indptr, st.kv_len_before, bad_indptr,
                         st.page_indices, st.k_new, st.v_new)


# ------------------------------------------------------------------------------------------
# attention values
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("Hq,Hkv,d", [(8, 2, 64), (4, 4, 32), (8, 1, 128), (6, 2, 16)])
def test_matches_dense_numpy_evaluation(Hq, Hkv, d):
    shape = W.Shape(Hq, Hkv, d, 16)
    wl = W.make_single_step("t", shape, [37, 0, 16, 15, 90, 3], [12, 5, 1, 1, 0, 33], seed=7 + d,
                            interleave_pages=True)
    pool, out, lse = run_oracle(wl)
    out2, lse2 = dense_twin(pool, wl.steps[0], shape)
    assert np.abs(out - out2).max() < 1e-12
    assert np.abs(lse - lse2).max() < 1e-12


def test_custom_scale_is_used():
    shape = W.Shape(4, 2, 32, 16)
    wl = W.make_single_step("t", shape, [20, 3], [4, 1], seed=5)
    pool, out, lse = run_oracle(wl, scale=0.37)
    out2, lse2 = dense_twin(pool, wl.steps[0], shape, scale=0.37)
    assert np.abs(out - out2).max() < 1e-12 and np.abs(lse - lse2).max() < 1e-12
    _, out_default, _ = run_oracle(wl)
    assert np.abs(out - out_default).max() > 1e-3


@pytest.mark.parametrize("ctx,ql", [(0, 24), (19, 9), (48, 1)])
def test_matches_torch_sdpa_fp64(ctx, ql):
    """Library special case: contiguous K/V, boolean mask, fp64 scaled_dot_product_attention."""
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("t", shape, [ctx], [ql], seed=100 + ctx)
    st = wl.steps[0]
    pool, out, _ = run_oracle(wl)
    k, v = gather_dense(pool, st, 0)
    G = shape.group
    q_t = torch.from_numpy(W.bf16_bits_to_f64(st.q)).permute(1, 0, 2)[None]        # [1,Hq,ql,d]
    k_t = torch.from_numpy(np.repeat(k, G, axis=1)).permute(1, 0, 2)[None]
    v_t = torch.from_numpy(np.repeat(v, G, axis=1)).permute(1, 0, 2)[None]
    n = ctx + ql
    allowed = torch.arange(n)[None, :] <= (ctx + torch.arange(ql))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(q_t, k_t, v_t, attn_mask=allowed)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.abs(out - ref).max() < 1e-12
    if ctx == 0:
        ref2 = torch.nn.functional.scaled_dot_product_attention(q_t, k_t, v_t, is_causal=True)
        assert np.abs(out - ref2[0].permute(1, 0, 2).numpy()).max() < 1e-12


def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "two_key_softmax.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            vals[k] = float(v)
    return vals


def test_two_key_closed_form_fixture():
    g = _golden()
    assert abs(g["sigmoid1"] - 1 / (1 + math.exp(-1))) < 1e-15
    shape = W.Shape(1, 1, 64, 16)
    e0 = np.zeros(64); e0[0] = 1
    e1 = np.zeros(64); e1[1] = 1
    z = np.zeros(64)
    # decode row: ctx = 1 (K0, V0 cached), own key K1 = 0, V1 = e1
    pool = np.zeros((1, 2, 1, 16, 64), dtype=np.uint16)
    pool[0, 0, 0, 0] = bf(e0)
    pool[0, 1, 0, 0] = bf(e0)
    pool[0, :, 0, 2:] = 0x7FC0     # unused slots hold NaN patterns and must not matter
    q = bf(8 * e0).reshape(1, 1, 64)
    out, lse = oracle.attn_mixed(*_appended(pool, [0, 1], [1], [0, 1], [0],
                                            bf(z).reshape(1, 1, 64), bf(e1).reshape(1, 1, 64)),
                                 q, [0, 1], [1], [0, 1], [0])
    assert abs(out[0, 0, 0] - g["sigmoid1"]) < 1e-15
    assert abs(out[0, 0, 1] - g["one_minus_sigmoid1"]) < 1e-15
    assert np.abs(out[0, 0, 2:]).max() == 0
    assert abs(lse[0, 0] - g["lse_two_keys"]) < 1e-15
    # append: ctx = 0, two rows (K0,V0) then (K1,V1); both queries 8*e0
    pool2 = np.full((1, 2, 1, 16, 64), 0x7FC0, dtype=np.uint16)
    kn = np.stack([bf(e0), bf(z)]).reshape(2, 1, 64)
    vn = np.stack([bf(e0), bf(e1)]).reshape(2, 1, 64)
    qq = np.stack([bf(8 * e0), bf(8 * e0)]).reshape(2, 1, 64)
    out, lse = oracle.attn_mixed(*_appended(pool2, [0, 2], [0], [0, 1], [0], kn, vn),
                                 qq, [0, 2], [0], [0, 1], [0])
    assert np.array_equal(out[0, 0], e0) and abs(lse[0, 0] - g["lse_one_key"]) < 1e-15
    assert abs(out[1, 0, 0] - g["sigmoid1"]) < 1e-15
    assert abs(out[1, 0, 1] - g["one_minus_sigmoid1"]) < 1e-15
    assert abs(lse[1, 0] - g["lse_two_keys"]) < 1e-15


def _appended(pool, q_indptr, ctx, page_indptr, page_indices, kn, vn):
    pool = pool.copy()
    oracle.kv_append(pool, q_indptr, ctx, page_indptr, page_indices, kn, vn)
    return (pool,)


def test_zero_query_gives_mean_of_values_and_log_n():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("t", shape, [45, 7], [6, 1], seed=21)
    st = wl.steps[0]
    st.q[...] = 0
    pool, out, lse = run_oracle(wl)
    for b in range(2):
        k, v = gather_dense(pool, st, b)
        ctx = int(st.kv_len_before[b])
        for i in range(int(st.q_len[b])):
            n = ctx + i + 1
            r = st.q_indptr[b] + i
            mean = np.repeat(v[:n].mean(axis=0), shape.group, axis=0)
            assert np.abs(out[r] - mean).max() < 1e-13
            assert np.abs(lse[r] - math.log(n)).max() < 1e-13


def test_single_key_returns_v_exactly():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("t", shape, [0, 0, 0], [1, 1, 3], seed=22)
    st = wl.steps[0]
    pool, out, lse = run_oracle(wl)
    for r in (0, 1, 2):   # rows that see exactly one key: their own
        v = W.bf16_bits_to_f64(st.v_new[r])
        assert np.array_equal(out[r], np.repeat(v, shape.group, axis=0))
        q = W.bf16_bits_to_f64(st.q[r])
        k = np.repeat(W.bf16_bits_to_f64(st.k_new[r]), shape.group, axis=0)
        assert np.abs(lse[r] - (q * k).sum(-1) / 8.0).max() < 1e-13


def test_dominating_key_selects_its_value():
    shape = W.Shape(2, 1, 32, 16)
    wl = W.make_single_step("t", shape, [40], [1], seed=23)
    st = wl.steps[0]
    j = 17
    pg = st.page_indices[j // 16]
    st.q[0, :, :] = bf(np.full(32, 4.0))
    wl.kv_pool[pg, 0, 0, j % 16] = bf(np.full(32, 64.0))   # score ~ 32*4*64/sqrt(32) >> others
    pool, out, _ = run_oracle(wl)
    vj = W.bf16_bits_to_f64(pool[pg, 1, 0, j % 16])
    assert np.abs(out[0] - vj[None]).max() < 1e-12


# ------------------------------------------------------------------------------------------
# invariants of the method
# ------------------------------------------------------------------------------------------

def test_append_then_attend_equals_full_recomputation():
    """Section 3.2 (append in place) versus Section 5.5 (discard and recompute everything)."""
    shape = W.Shape(8, 2, 64, 16)
    ctx, ql = [70, 33, 16], [12, 1, 20]
    wl = W.make_single_step("t", shape, ctx, ql, seed=31)
    st = wl.steps[0]
    pool, out, lse = run_oracle(wl)
    for b in range(3):
        n = ctx[b] + ql[b]
        k, v = gather_dense(pool, st, b)
        # rebuild the whole sequence as one span on an empty context in a fresh pool
        k_all = np.zeros((n, 2, 64), dtype=np.uint16)
        v_all = np.zeros((n, 2, 64), dtype=np.uint16)
        P = 16
        pages = st.page_indices[st.page_indptr[b]:st.page_indptr[b + 1]]
        for j in range(n):
            k_all[j] = pool[pages[j // P], 0, :, j % P]
            v_all[j] = pool[pages[j // P], 1, :, j % P]
        q_all = W.normal_bf16(99, b, (n, 8, 64))
        q_all[ctx[b]:] = st.q[st.q_indptr[b]:st.q_indptr[b + 1]]
        npg = -(-n // P)
        fresh = np.full((npg + 2, 2, 2, P, 64), 0x7FC0, dtype=np.uint16)
        perm = np.random.default_rng(b).permutation(npg + 2)[:npg].astype(np.int32)
        o2, l2 = oracle.attn_mixed(*_appended(fresh, [0, n], [0], [0, npg], perm, k_all, v_all),
                                   q_all, [0, n], [0], [0, npg], perm)
        sl = slice(st.q_indptr[b], st.q_indptr[b + 1])
        assert np.array_equal(o2[ctx[b]:], out[sl])          # same sums in the same order
        assert np.array_equal(l2[ctx[b]:], lse[sl])


def test_two_spans_in_two_steps_equal_one_concatenated_span():
    """Section 5.3: all queued interrupts are appended together; order of arrival is kept."""
    shape = W.Shape(4, 2, 32, 16)
    ctx, a1, a2 = 21, 9, 14
    wl = W.make_single_step("t", shape, [ctx], [a1 + a2], seed=41)
    st = wl.steps[0]
    pool_one, out_one, _ = run_oracle(wl)
    pool = wl.kv_pool.copy()
    oracle.kv_append(pool, [0, a1], [ctx], st.page_indptr, st.page_indices,
                     st.k_new[:a1].copy(), st.v_new[:a1].copy())
    oracle.kv_append(pool, [0, a2], [ctx + a1], st.page_indptr, st.page_indices,
                     st.k_new[a1:].copy(), st.v_new[a1:].copy())
    assert np.array_equal(pool, pool_one)
    out_b, _ = oracle.attn_mixed(pool, st.q[a1:].copy(), [0, a2], [ctx + a1], st.page_indptr,
                                 st.page_indices)
    assert np.array_equal(out_b, out_one[a1:])


def test_output_is_invariant_to_physical_page_order():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("t", shape, [100, 37, 250], [12, 1, 1], seed=51)
    st = wl.steps[0]
    _, out, lse = run_oracle(wl)
    perm = np.random.default_rng(5).permutation(wl.num_pages)
    pool2 = np.empty_like(wl.kv_pool)
    pool2[perm] = wl.kv_pool                      # page p moves to perm[p]
    st2 = W.Step(st.q_indptr, st.kv_len_before, st.page_indptr,
                 perm[st.page_indices].astype(np.int32), st.q, st.k_new, st.v_new)
    out2, lse2 = oracle.step(pool2, st2)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_unused_slots_do_not_influence_the_result():
    shape = W.Shape(8, 2, 64, 16)
    args = dict(kv_len_before=[100, 37, 3], q_len=[12, 1, 1], seed=61, extra_pages=[1, 0, 2])
    clean = W.make_single_step("t", shape, **args)
    dirty = W.make_single_step("t", shape, poison_unused=True, **args)
    assert not np.array_equal(clean.kv_pool, dirty.kv_pool)
    _, o1, l1 = run_oracle(clean)
    _, o2, l2 = run_oracle(dirty)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)
    assert np.isfinite(o1).all()


def test_paused_sequences_contribute_nothing():
    shape = W.Shape(4, 2, 32, 16)
    wl = W.make_single_step("t", shape, [30, 50, 10], [0, 3, 0], seed=71)
    pool, out, lse = run_oracle(wl)
    assert out.shape[0] == 3 and np.isfinite(out).all()
    st = wl.steps[0]
    diff = np.nonzero((pool != wl.kv_pool).any(axis=(1, 2, 3, 4)))[0]
    assert set(diff) <= set(st.page_indices[st.page_indptr[1]:st.page_indptr[2]])


def test_split_kv_merge_reproduces_unsplit_result():
    """Merging per-chunk (O_c, LSE_c) by log-sum-exp equals attention over the whole range."""
    shape = W.Shape(4, 2, 32, 16)
    wl = W.make_single_step("t", shape, [150], [5], seed=81)
    st = wl.steps[0]
    pool, out, lse = run_oracle(wl)
    k, v = gather_dense(pool, st, 0)
    G = shape.group
    q = W.bf16_bits_to_f64(st.q)
    rng = np.random.default_rng(1)
    for cuts in ([0, 16, 155], [0, 1, 2, 150, 152, 155], sorted({0, 155, *rng.integers(1, 155, 6)})):
        parts_o, parts_l = [], []
        for lo, hi in zip(cuts[:-1], cuts[1:]):
            o_c = np.zeros((5, 4, 32)); l_c = np.full((5, 4), -np.inf)
            for i in range(5):
                top = min(hi, 150 + i + 1)
                if top <= lo:
                    continue
                for h in range(4):
                    s = (k[lo:top, h // G] @ q[i, h]) / math.sqrt(32)
                    m = s.max(); e = np.exp(s - m)
                    o_c[i, h] = (e[:, None] * v[lo:top, h // G]).sum(0) / e.sum()
                    l_c[i, h] = m + math.log(e.sum())
            parts_o.append(o_c); parts_l.append(l_c)
        o_m, l_m = oracle.lse_merge(np.stack(parts_o), np.stack(parts_l))
        assert np.abs(o_m - out).max() < 1e-12
        assert np.abs(l_m - lse).max() < 1e-12


def test_selected_rows_only():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("t", shape, [40, 20], [6, 1], seed=91)
    st = wl.steps[0]
    pool, out, lse = run_oracle(wl)
    o2, l2 = oracle.attn_mixed(pool, st.q, st.q_indptr, st.kv_len_before, st.page_indptr,
                               st.page_indices, sel_rows=[6, 2])
    assert np.array_equal(o2[[2, 6]], out[[2, 6]]) and np.array_equal(l2[[2, 6]], lse[[2, 6]])
    assert np.isnan(o2[[0, 1, 3, 4, 5]]).all()
