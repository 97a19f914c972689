"""asynclm_attn_mixed_static: attention without caller-provided scratch memory.

Some users of the library cannot allocate device memory for it (all of HBM already committed to
the KV pool, a host application that owns the allocator, a loop where cudaMalloc is forbidden).
This entry point keeps the split-KV partial results in an array compiled into the library.  It must
give what asynclm_attn_mixed gives, call after call, although all calls share that one array, and
it must refuse plans whose partial results do not fit.

This file is named so that pytest collects it after every other test file.
"""
import numpy as np
import pytest
import torch

from paper_2412_07017_b200 import binding as B
from paper_2412_07017_b200 import workload as W
from gpu_util import assert_close, oracle_step, to_bits, to_dev

pytestmark = pytest.mark.gpu


def _both_ways(wl, **opts):
    """Run the ordinary call and the static-scratch call on the same appended pool."""
    st = wl.steps[0]
    shape = wl.shape
    pool = to_dev(wl.kv_pool)
    q, kn, vn = to_dev(st.q), to_dev(st.k_new), to_dev(st.v_new)
    plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr,
                          st.page_indices, **opts)
    B.asynclm_kv_append(plan, kn, vn, pool)
    res = []
    for fn in (B.asynclm_attn_mixed, B.asynclm_attn_mixed_static):
        out = torch.full((st.total_q, shape.num_q_heads, shape.head_dim), float("nan"),
                         dtype=torch.bfloat16, device="cuda")
        lse = torch.full((st.total_q, shape.num_q_heads), float("nan"), dtype=torch.float32,
                         device="cuda")
        fn(plan, q, pool, out, lse)
        torch.cuda.synchronize()
        assert B.last_device_status(plan) == 0
        res.append((to_bits(out), lse.cpu().numpy()))
    _, ref_out, ref_lse = oracle_step(wl, st)
    return plan, res, (ref_out, ref_lse)


def _assert_same(res, ref):
    """Same kernels, same plan, same chunk order: the two calls must agree bit for bit (a tolerance
    would hide a stale value leaking out of the shared array), and both must match the oracle."""
    (o_ref, l_ref), (o_new, l_new) = res
    assert np.array_equal(o_new, o_ref) and np.array_equal(l_new, l_ref)
    assert_close(o_new, l_new, ref[0], ref[1], what="static scratch against the oracle")


def test_static_scratch_matches_the_ordinary_call_twice_in_a_row():
    # first call: many split units (fixed 128-token chunks), Llama head shape
    a = W.make_single_step("a", W.Shape(32, 8, 128, 16), [1500, 64, 700, 900], [1, 1, 9, 3], seed=301)
    plan, res, ref = _both_ways(a, kv_chunk_tokens=128)
    assert plan.info["partial_rows"] > 0
    _assert_same(res, ref)
    # second call straight after, different shape and lengths: the shared array still holds the
    # first call's partial results and must not leak into this one
    b = W.make_single_step("b", W.Shape(8, 2, 64, 16), [333, 2000, 15], [1, 2, 1], seed=302)
    plan, res, ref = _both_ways(b, kv_chunk_tokens=64)
    assert plan.info["partial_rows"] > 0
    _assert_same(res, ref)
    # and a plan with nothing split at all
    plan, res, ref = _both_ways(b, kv_chunk_tokens=1 << 20)
    assert plan.info["partial_rows"] == 0
    _assert_same(res, ref)
    # the default policy: chunks handed out at run time, split units merged inside the attention kernel
    c = W.make_single_step("c", W.Shape(32, 8, 128, 16), [3000, 2500, 900, 1800] * 3, [1, 1, 40, 1] * 3, seed=304)
    plan, res, ref = _both_ways(c)
    assert plan.info["partial_rows"] > 0
    _assert_same(res, ref)


def test_plans_beyond_the_fixed_array_are_refused():
    shape = W.Shape(64, 8, 128, 16)
    wl = W.make_single_step("big", shape, [9000], [6], seed=303)
    st = wl.steps[0]
    plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr,
                          st.page_indices, kv_chunk_tokens=64)
    need = plan.info["partial_rows"] * shape.group * (shape.head_dim + 1) * 4
    assert need > B.static_scratch_bytes()
    out = torch.zeros((st.total_q, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16,
                      device="cuda")
    with pytest.raises(B.AsynclmError) as e:
        B.asynclm_attn_mixed_static(plan, to_dev(st.q), to_dev(wl.kv_pool), out)
    assert e.value.status == -8
    assert "scratch" in str(e.value)
