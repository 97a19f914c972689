"""GPU parity: the CUDA path through the C ABI against the fp64 CPU oracle, element by element.

Bars: KV append bit-exact over the whole pool; attention max |err| <= 1e-2 and mean |err| <= 1e-3
(bf16 inputs, fp32 accumulation, bf16 output); lse within 1e-3.
"""
import numpy as np
import pytest
import torch

from paper_2412_07017_b200 import binding as B
from paper_2412_07017_b200 import workload as W
import gpu_util
from gpu_util import (assert_close, gpu_step, oracle_step, to_bits, to_dev)

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["calls", "step"])
def api(request):
    """Every test runs through the three calls and through asynclm_step."""
    gpu_util.API = request.param
    yield request.param
    gpu_util.API = "calls"


def run_and_check(wl, st=None, what="", **opts):
    st = st or wl.steps[0]
    pool_dev, out_bits, lse, plan = gpu_step(wl, st, **opts)
    ref_pool, ref_out, ref_lse = oracle_step(wl, st)
    assert np.array_equal(to_bits(pool_dev), ref_pool), f"{what}: pool differs after append"
    assert_close(out_bits, lse, ref_out, ref_lse, what=what)
    return out_bits, lse, plan


def test_config1_tiny_mixed_step():
    wl = W.make_config(1)
    _, _, plan = run_and_check(wl, what="config1")
    assert plan.info["total_q"] == 15


@pytest.mark.parametrize("Hq,Hkv,d", [(8, 2, 64), (4, 4, 64), (8, 1, 64), (2, 1, 128), (32, 8, 128),
                                      (16, 2, 128), (4, 2, 128), (8, 8, 128)])
def test_shapes_and_ragged_lengths(Hq, Hkv, d):
    shape = W.Shape(Hq, Hkv, d, 16)
    ctx = [0, 1, 15, 16, 17, 129, 700, 0, 300, 47]
    ql = [1, 1, 1, 1, 12, 5, 1, 33, 0, 70]
    wl = W.make_single_step("ragged", shape, ctx, ql, seed=1000 + Hq * 7 + d,
                            extra_pages=[0, 1, 0, 0, 2, 0, 0, 1, 3, 0], interleave_pages=True)
    run_and_check(wl, what=f"ragged {Hq}/{Hkv}/{d}")


@pytest.mark.parametrize("chunk", [64, 128, 512, 1 << 20])
def test_fixed_chunk_lengths_agree_with_oracle(chunk):
    shape = W.Shape(8, 2, 128, 16)
    wl = W.make_single_step("chunks", shape, [1500, 64, 127, 900], [1, 1, 40, 7], seed=77)
    _, _, plan = run_and_check(wl, what=f"chunk {chunk}", kv_chunk_tokens=chunk)
    if chunk < 1 << 20:
        assert plan.info["num_split_units"] > 0
    # fixed chunks are dealt to the CTAs statically, and some CTA gets span tiles and warp-body
    # items: the fused kernel runs both bodies there, one after the other
    if chunk <= 128:
        items = plan.items()
        assert set(items[items["path"] == 1]["cta"].tolist()) & set(items[items["path"] == 0]["cta"].tolist())


@pytest.mark.parametrize("Hq", [8, 16])
def test_cuda_core_path_handles_spans_too(Hq):
    """Every row on the CUDA-core kernel (4 and 8 heads per kv head; with 8 the planner would send
    even decode rows to the tensor cores by default)."""
    shape = W.Shape(Hq, 2, 128, 16)
    wl = W.make_single_step("spans", shape, [300, 0, 40, 700], [64, 130, 9, 1], seed=78)
    _, _, plan = run_and_check(wl, what="cuda-core spans", flags=B.PLAN_NO_TENSOR_PATH)
    assert plan.info["num_items_tensor"] == 0


def test_eight_heads_per_kv_head():
    """Default routing with 8 heads per kv head: decode rows (8 columns of the warp body's MMAs) stay on
    the warp body, the 20-token span (160 rows) takes the span body; tensor_min_rows = 8 sends the
    decode rows to the span body as well."""
    shape = W.Shape(16, 2, 128, 16)
    wl = W.make_single_step("gqa8", shape, [300, 0, 1500, 77], [1, 1, 1, 20], seed=79)
    _, _, plan = run_and_check(wl, what="gqa8, default routing")
    assert 0 < plan.info["num_items_tensor"] < plan.info["num_items"]
    items = plan.items()
    assert (items[items["path"] == 0]["ntok"] == 1).all() and (items[items["path"] == 1]["seq"] == 3).all()
    _, _, plan = run_and_check(wl, what="gqa8, every row on the span body", tensor_min_rows=8)
    assert plan.info["num_items_tensor"] == plan.info["num_items"]


def test_decode_rows_beside_spans_on_few_sms():
    """Default policy with 12 CTAs: span units on the first CTAs, decode rows queued for whichever CTA
    is free (span CTAs join the queue when their span tiles are done)."""
    shape = W.Shape(8, 2, 128, 16)
    ctx = [1900, 40, 2500, 3, 700, 1200, 0, 333] + [900 + 37 * i for i in range(24)]
    ql = [40, 1, 1, 9, 1, 64, 1, 1] + [1] * 24
    wl = W.make_single_step("hybrid", shape, ctx, ql, seed=83)
    _, _, plan = run_and_check(wl, what="decode rows beside spans", num_sms=12)
    items = plan.items()
    tens, warp = items[items["path"] == 1], items[items["path"] == 0]
    assert len(tens) > 0 and (warp["cta"] < 0).sum() > 0
    assert plan.info["num_split_units"] > 0          # short chunks at the end of the queue: merged in the kernel
    run_and_check(wl, what="all rows on the warp body", flags=B.PLAN_NO_TENSOR_PATH)
    run_and_check(wl, what="all rows on the span body", tensor_min_rows=1)


def test_short_spans_share_the_columns_of_a_warp_body_unit():
    """Spans below 32 rows run on the warp body, 8 / G tokens to a unit (2 at 4 heads per kv head, 8 at
    one), each column with its own causal limit; odd span lengths leave a unit partly empty."""
    for Hq, Hkv, d in [(8, 2, 128), (4, 4, 64), (2, 1, 128), (16, 2, 64)]:
        shape = W.Shape(Hq, Hkv, d, 16)
        wl = W.make_single_step("short", shape, [0, 5, 130, 1000, 16, 255], [3, 7, 2, 5, 1, 6], seed=500 + Hq)
        _, _, plan = run_and_check(wl, what=f"short spans {Hq}/{Hkv}/{d}")
        items = plan.items()
        assert (items["path"] == 0).all() and items["ntok"].max() == min(7, 8 // shape.group)


def test_results_are_bitwise_reproducible():
    wl = W.make_config(1)
    a = gpu_step(wl, wl.steps[0])
    b = gpu_step(wl, wl.steps[0])
    assert np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])


def test_physical_page_order_does_not_change_a_single_bit():
    wl = W.make_config(1)
    st = wl.steps[0]
    _, out, lse, _ = gpu_step(wl, st)
    perm = np.random.default_rng(9).permutation(wl.num_pages)
    pool2 = np.empty_like(wl.kv_pool)
    pool2[perm] = wl.kv_pool
    wl2 = W.Workload("perm", wl.shape, wl.num_pages, pool2)
    st2 = W.Step(st.q_indptr, st.kv_len_before, st.page_indptr,
                 perm[st.page_indices].astype(np.int32), st.q, st.k_new, st.v_new)
    _, out2, lse2, _ = gpu_step(wl2, st2)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_unused_slots_and_pages_may_hold_nan_patterns():
    shape = W.Shape(8, 2, 128, 16)
    args = dict(kv_len_before=[100, 37, 3, 260], q_len=[12, 1, 1, 35], seed=61,
                extra_pages=[1, 0, 2, 0])
    clean = W.make_single_step("clean", shape, **args)
    dirty = W.make_single_step("dirty", shape, poison_unused=True, **args)
    _, out_c, lse_c, _ = gpu_step(clean, clean.steps[0])
    out_d, lse_d, _ = run_and_check(dirty, what="poisoned")
    assert np.array_equal(out_c, out_d) and np.array_equal(lse_c, lse_d)


def test_single_visible_key_returns_v_exactly():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("one", shape, [0, 0, 0], [1, 1, 3], seed=22)
    st = wl.steps[0]
    _, out, _, _ = gpu_step(wl, st)
    for r in (0, 1, 2):
        assert np.array_equal(out[r], np.repeat(st.v_new[r], shape.group, axis=0))


def test_append_only_touches_its_slots_and_is_idempotent():
    shape = W.Shape(8, 2, 128, 16)
    wl = W.make_single_step("app", shape, [5, 16, 31, 0, 40], [12, 1, 2, 7, 0], seed=11,
                            extra_pages=[0, 1, 0, 2, 1], poison_unused=True)
    st = wl.steps[0]
    pool_dev, _, _, plan = gpu_step(wl, st)
    ref_pool, _, _ = oracle_step(wl, st)
    assert np.array_equal(to_bits(pool_dev), ref_pool)
    B.asynclm_kv_append(plan, to_dev(st.k_new), to_dev(st.v_new), pool_dev)
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(pool_dev), ref_pool)


def test_two_spans_in_two_steps_equal_one_concatenated_span():
    shape = W.Shape(8, 2, 128, 16)
    ctx, a1, a2 = 210, 9, 14
    wl = W.make_single_step("cat", shape, [ctx], [a1 + a2], seed=41)
    st = wl.steps[0]
    pool_one, out_one, _, _ = gpu_step(wl, st)
    s1 = W.Step(np.array([0, a1], np.int32), np.array([ctx], np.int32), st.page_indptr,
                st.page_indices, st.q[:a1].copy(), st.k_new[:a1].copy(), st.v_new[:a1].copy())
    s2 = W.Step(np.array([0, a2], np.int32), np.array([ctx + a1], np.int32), st.page_indptr,
                st.page_indices, st.q[a1:].copy(), st.k_new[a1:].copy(), st.v_new[a1:].copy())
    pool, _, _, _ = gpu_step(wl, s1)
    pool, out_b, _, _ = gpu_step(wl, s2, pool_dev=pool)
    assert np.array_equal(to_bits(pool), to_bits(pool_one))
    ref_pool, ref_out, ref_lse = oracle_step(wl, st)
    assert_close(out_b, None, ref_out[a1:], None, what="second span")


def test_custom_softmax_scale():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("scale", shape, [90, 10], [5, 1], seed=5)
    st = wl.steps[0]
    _, out, lse, _ = gpu_step(wl, st, sm_scale=0.05)
    _, ref_out, ref_lse = oracle_step(wl, st, sm_scale=0.05)
    assert_close(out, lse, ref_out, ref_lse, what="scale")


def test_empty_and_all_paused_batches_are_no_ops():
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("paused", shape, [30, 50], [0, 0], seed=71)
    st = wl.steps[0]
    pool_dev, out, _, plan = gpu_step(wl, st)
    assert out.shape[0] == 0 and np.array_equal(to_bits(pool_dev), wl.kv_pool)


def test_replay_steps_keep_state_across_steps():
    wl = W.make_replay(batch=24, steps=6, ctx_lo=40, ctx_hi=400, rate=0.2,
                       shape=W.Shape(32, 8, 128, 16))
    pool_dev = to_dev(wl.kv_pool)
    ref_pool = wl.kv_pool.copy()
    for t, st in enumerate(wl.steps):
        pool_dev, out, lse, _ = gpu_step(wl, st, pool_dev=pool_dev)
        ref_pool, ref_out, ref_lse = oracle_step(wl, st, pool=ref_pool)
        assert np.array_equal(to_bits(pool_dev), ref_pool), f"step {t}"
        assert_close(out, lse, ref_out, ref_lse, what=f"replay step {t}")


@pytest.mark.parametrize("Hq,Hkv,ctx,ql", [
    (32, 8, [700, 64, 0, 129], [64, 33, 64, 40]),       # two full row tiles per (sequence, kv head), ragged second tile
    (32, 8, [1000], [200]),                              # a span longer than one work item: several units per head
    (16, 2, [300, 55], [32, 17]),                        # 8 heads per kv head: 256 rows from 32 tokens
    (4, 4, [500, 20], [256, 130]),                       # one head per kv head: the row tiles are all tokens
    (8, 2, [48, 64, 65, 127, 128, 193], [40, 40, 40, 40, 40, 40]),   # last KV tile with 1..8 pages
])
def test_span_row_tile_pairs(Hq, Hkv, ctx, ql):
    """Spans whose (token, head) rows fill one row tile, exactly two, two with a ragged end, or more
    than one work item, across the KV-tile tail lengths the two-half softmax distinguishes."""
    shape = W.Shape(Hq, Hkv, 128, 16)
    wl = W.make_single_step("pairs", shape, ctx, ql, seed=300 + Hq + len(ctx), interleave_pages=True)
    run_and_check(wl, what=f"row tile pairs {Hq}/{Hkv}")
    run_and_check(wl, what=f"row tile pairs {Hq}/{Hkv}, fixed chunks", kv_chunk_tokens=128)


def test_scores_that_keep_growing_move_the_reference_maximum():
    """Keys whose scores rise steadily along the context: the lazily updated softmax reference of
    both attention paths has to move again and again (and rescale what it has accumulated)."""
    shape = W.Shape(8, 2, 128, 16)
    ctx, ql = [1200, 1200, 900], [40, 1, 70]
    wl = W.make_single_step("growing", shape, ctx, ql, seed=91)
    st = wl.steps[0]
    d = shape.head_dim
    u = np.ones(d, dtype=np.float32)
    for b in range(len(ctx)):
        n = ctx[b] + ql[b]
        # q . k / sqrt(d) runs from about -40 to +40 over the sequence
        alpha = np.linspace(-40.0, 40.0, n, dtype=np.float32) * np.sqrt(d) / d
        for pos in range(ctx[b]):
            pg = st.page_indices[st.page_indptr[b] + pos // 16]
            wl.kv_pool[pg, 0, :, pos % 16, :] = W.f32_to_bf16_bits(alpha[pos] * u)[None, :]
        for i in range(ql[b]):
            st.k_new[st.q_indptr[b] + i] = W.f32_to_bf16_bits(alpha[ctx[b] + i] * u)[None, :]
    st.q[:] = W.f32_to_bf16_bits(u)[None, None, :]
    run_and_check(wl, what="growing scores")
    run_and_check(wl, what="growing scores, split", kv_chunk_tokens=256)


def test_config2_llama_batch_full_size():
    """Full-size Llama-3-8B-shaped mixed batch, default planning (the benchmarked configuration)."""
    wl = W.make_config(2)
    st = wl.steps[0]
    pool_dev, out, lse, plan = gpu_step(wl, st)
    ref_pool, ref_out, ref_lse = oracle_step(wl, st)
    assert np.array_equal(to_bits(pool_dev), ref_pool)
    is_app = np.repeat(st.q_len > 1, st.q_len)
    assert_close(out, lse, ref_out, ref_lse, rows=np.nonzero(~is_app)[0], what="config2 decode rows")
    assert_close(out, lse, ref_out, ref_lse, rows=np.nonzero(is_app)[0], what="config2 append rows")
    assert_close(out, lse, ref_out, ref_lse, what="config2")


def test_page_ids_whose_offsets_need_64_bits():
    """Pages high in a pool of 70 000 pages (4.6 GB): element offsets beyond 2^31 and byte offsets beyond
    2^32 in the append, in the span body's 16-byte copies and in the warp body's tensor-map
    coordinates.  Only the pages in use are written on the device; the oracle works on a compact copy
    of those pages under renumbered ids."""
    shape = W.Shape(32, 8, 128, 16)
    small = W.make_single_step("high", shape, [300, 200, 77, 1030], [1, 40, 2, 1], seed=88, spare_pages=0)
    st = small.steps[0]
    num_pages = 70000
    high = (np.random.default_rng(5).permutation(num_pages - 66000)[:small.num_pages] + 66000).astype(np.int32)
    assert int(high.min()) * shape.page_elems > 2**31
    pool_dev = torch.empty((num_pages,) + small.kv_pool.shape[1:], dtype=torch.bfloat16, device="cuda")
    pool_dev[torch.from_numpy(high.astype(np.int64)).cuda()] = to_dev(small.kv_pool)
    big = W.Workload("high", shape, num_pages, small.kv_pool)
    st_big = W.Step(st.q_indptr, st.kv_len_before, st.page_indptr, high[st.page_indices], st.q, st.k_new, st.v_new)
    pool_dev, out, lse, plan = gpu_step(big, st_big, pool_dev=pool_dev)
    assert 0 < plan.info["num_items_tensor"] < plan.info["num_items"]
    ref_pool, ref_out, ref_lse = oracle_step(small, st)
    got = to_bits(pool_dev[torch.from_numpy(high.astype(np.int64)).cuda()])
    assert np.array_equal(got, ref_pool), "pool differs after append"
    assert_close(out, lse, ref_out, ref_lse, what="high page ids")


def test_sequences_that_share_prefix_pages():
    """Two sequences (a fork after a common prompt) whose page tables name the same physical pages for
    their first 20 full pages; each appends into pages of its own.  Reads of shared pages are legal."""
    shape = W.Shape(8, 2, 128, 16)
    wl = W.make_single_step("fork", shape, [400, 520, 333, 700], [1, 24, 1, 3], seed=97)
    st = wl.steps[0]
    shared = 20
    for b in (1, 3):      # sequences 1 and 3 start with sequence 0's first 20 pages
        st.page_indices[st.page_indptr[b]:st.page_indptr[b] + shared] = \
            st.page_indices[st.page_indptr[0]:st.page_indptr[0] + shared]
    _, _, plan = run_and_check(wl, what="shared prefix pages", flags=B.PLAN_REJECT_ALIASED_WRITES)
    assert plan.info["num_items_tensor"] > 0
