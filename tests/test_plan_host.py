"""Host planner (integer work only, no GPU): coverage, balance and validation."""
import numpy as np
import pytest

from paper_2412_07017_b200 import binding as B
from paper_2412_07017_b200 import workload as W


def plan(wl, st=None, **kw):
    st = st or wl.steps[0]
    return B.plan_host(wl.shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr,
                       st.page_indices, **kw)


def check_cover(wl, p, st=None):
    """Every (sequence, kv head, new token, visible key) is covered by exactly one item."""
    st = st or wl.steps[0]
    items = p.items()
    cover = {}
    for it in items:
        for t in range(it["ntok"]):
            i = it["tok0"] + t
            lim = int(st.kv_len_before[it["seq"]]) + i + 1
            lo, hi = int(it["kv0"]), min(int(it["kv1"]), lim)
            key = (int(it["seq"]), int(it["kv_head"]), i)
            cover.setdefault(key, []).append((lo, hi))
    want = set()
    for b in range(st.batch):
        for i in range(int(st.q_len[b])):
            for h in range(wl.shape.num_kv_heads):
                want.add((b, h, i))
    assert set(cover) == want
    for (b, h, i), segs in cover.items():
        segs = sorted(s for s in segs if s[1] > s[0])
        assert segs[0][0] == 0
        for a, c in zip(segs[:-1], segs[1:]):
            assert a[1] == c[0]
        assert segs[-1][1] == int(st.kv_len_before[b]) + i + 1
    # chunk boundaries are page aligned
    assert (items["kv0"] % 16 == 0).all()
    return items


@pytest.mark.parametrize("chunk", [0, 64, 128, 512, 1 << 20])
def test_items_partition_the_causal_work(chunk):
    wl = W.make_config(1)
    p = plan(wl, kv_chunk_tokens=chunk)
    items = check_cover(wl, p)
    assert p.info["total_q"] == 15 and p.info["num_items"] == len(items)
    if chunk >= 1 << 20:
        assert p.info["num_split_units"] == 0 and p.info["partial_rows"] == 0


@pytest.mark.parametrize("sms", [1, 4, 148])
def test_cover_with_paused_and_empty_context_sequences(sms):
    shape = W.Shape(8, 2, 64, 16)
    wl = W.make_single_step("t", shape, [0, 700, 33, 0, 5], [40, 0, 1, 1, 3], seed=2)
    p = plan(wl, num_sms=sms)
    check_cover(wl, p)


def _queue_checks(p, items, n_sms):
    """Properties of the run-time queue of warp-body chunks under the default policy."""
    warp = items[items["path"] == 0]
    own = warp[warp["cta"] >= 0]
    queue = warp[warp["cta"] < 0]
    # a CTA starts on at most one chunk of its own; everything else is handed out at run time
    assert len(set(own["cta"].tolist())) == len(own) and (queue["cta"] == -1).all()
    # the list holds the own chunks first, then the queue in the order it is handed out
    n_own = len(own)
    assert (warp["cta"][:n_own] >= 0).all()
    # the long pieces come longest first, the short chunks (cut from few units) at the end
    tiles = -(-(warp["kv1"] - warp["kv0"]) // 128)
    units = {}
    for it, t in zip(warp, tiles):
        units.setdefault((int(it["seq"]), int(it["kv_head"]), int(it["tok0"])), []).append(int(t))
    split = {k: v for k, v in units.items() if len(v) > 1}
    whole_or_long = np.array([t for it, t in zip(warp, tiles)
                              if len(units[(int(it["seq"]), int(it["kv_head"]), int(it["tok0"]))]) <= 3])
    assert (np.diff(whole_or_long) <= 0).all()
    return own, queue, tiles, units, split


def test_decode_work_goes_to_a_queue_of_long_pieces_and_short_tail_chunks():
    g = np.random.default_rng(0)
    ctx = g.integers(512, 4097, 32)
    ql = np.ones(32, dtype=np.int64); ql[:8] = g.integers(8, 65, 8)
    shape = W.Shape(32, 8, 128, 16)
    need = -(-(ctx + ql) // 16)
    ids = np.arange(need.sum())
    q_indptr, page_indptr, page_indices, _ = W.build_step_tables(ctx, ql, 16, ids)
    p = B.plan_host(shape, int(need.sum()), q_indptr, ctx, page_indptr, page_indices, num_sms=148,
                    flags=B.PLAN_NO_TENSOR_PATH)
    items = p.items()
    assert (items["path"] == 0).all()
    own, queue, tiles, units, split = _queue_checks(p, items, 148)
    assert len(own) == 148 and len(queue) > 0
    # about a sixth of the tiles is cut into short chunks; the rest stays in long pieces
    short = sum(sum(v) for v in split.values() if len(v) > 3)
    assert 0.1 * tiles.sum() <= short <= 0.3 * tiles.sum()
    assert len(split) < 0.35 * len(units)


def test_plan_is_a_function_of_lengths_only():
    wl = W.make_config(1)
    st = wl.steps[0]
    a = plan(wl).items()
    perm = np.random.default_rng(3).permutation(wl.num_pages).astype(np.int32)
    b = B.plan_host(wl.shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr,
                    perm[st.page_indices]).items()
    assert np.array_equal(a, b)


def test_empty_batch_and_all_paused():
    shape = W.Shape(8, 2, 64, 16)
    p = B.plan_host(shape, 4, [0], [], [0], [])
    assert p.info["num_items"] == 0 and p.info["total_q"] == 0
    p = B.plan_host(shape, 4, [0, 0, 0], [5, 9], [0, 1, 2], [0, 1])
    assert p.info["num_items"] == 0


def _expect(status, fn):
    with pytest.raises(B.AsynclmError) as e:
        fn()
    assert e.value.status == status


def test_validation_errors():
    shape = W.Shape(8, 2, 64, 16)
    ok = dict(q_indptr=[0, 1], kv_len_before=[20], page_indptr=[0, 2], page_indices=[1, 0])
    B.plan_host(shape, 2, **ok)
    _expect(-3, lambda: B.plan_host(shape, 2, **{**ok, "page_indptr": [0, 1]}))       # too few pages
    _expect(-3, lambda: B.plan_host(shape, 2, **{**ok, "page_indices": [1, 2]}))      # id outside pool
    _expect(-3, lambda: B.plan_host(shape, 2, **{**ok, "page_indices": [-1, 0]}))
    _expect(-1, lambda: B.plan_host(shape, 2, **{**ok, "q_indptr": [0, -1]}))         # negative q_len
    _expect(-1, lambda: B.plan_host(shape, 2, **{**ok, "kv_len_before": [-2]}))
    _expect(-1, lambda: B.plan_host(shape, 2, **{**ok, "q_indptr": [1, 2]}))          # indptr[0] != 0
    _expect(-1, lambda: B.plan_host(shape, 2, kv_chunk_tokens=100, **ok))             # not a multiple of 64
    _expect(-2, lambda: B.plan_host(W.Shape(8, 2, 96, 16), 2, **ok))                  # head_dim
    _expect(-2, lambda: B.plan_host(W.Shape(8, 2, 64, 32), 2, **ok))                  # page size
    _expect(-2, lambda: B.plan_host(W.Shape(6, 2, 64, 16), 2, **ok))                  # group 3
    _expect(-2, lambda: B.plan_host(W.Shape(7, 2, 64, 16), 2, **ok))


def test_paused_sequence_page_ids_are_not_checked():
    shape = W.Shape(8, 2, 64, 16)
    B.plan_host(shape, 2, [0, 0, 1], [40, 3], [0, 3, 4], [99, -5, 7, 1])


def test_aliased_write_detection_is_optional():
    shape = W.Shape(8, 2, 64, 16)
    args = dict(q_indptr=[0, 1, 2], kv_len_before=[3, 3], page_indptr=[0, 1, 2], page_indices=[0, 0])
    B.plan_host(shape, 1, **args)
    _expect(-3, lambda: B.plan_host(shape, 1, flags=B.PLAN_REJECT_ALIASED_WRITES, **args))
    # sharing a fully read-only prefix page is fine
    args = dict(q_indptr=[0, 1, 2], kv_len_before=[16, 16], page_indptr=[0, 2, 4],
                page_indices=[0, 1, 0, 2])
    B.plan_host(shape, 3, flags=B.PLAN_REJECT_ALIASED_WRITES, **args)


def test_workspace_size_bounds_actual_use():
    wl = W.make_config(1)
    st = wl.steps[0]
    p = plan(wl)
    hb, db = B.workspace_size(wl.shape, wl.num_pages, st.batch, st.total_q, len(st.page_indices),
                              num_sms=148)
    assert hb >= p.info["host_bytes_used"] and db >= p.info["device_bytes_used"]
    p = plan(wl, kv_chunk_tokens=64)
    hb, db = B.workspace_size(wl.shape, wl.num_pages, st.batch, st.total_q, len(st.page_indices),
                              num_sms=148, kv_chunk_tokens=64)
    assert hb >= p.info["host_bytes_used"] and db >= p.info["device_bytes_used"]


def _llama_lengths(seed=0):
    g = np.random.default_rng(seed)
    ctx = g.integers(512, 4097, 32)
    ql = np.ones(32, dtype=np.int64)
    ql[:8] = g.integers(8, 65, 8)
    need = -(-(ctx + ql) // 16)
    q_indptr, page_indptr, page_indices, _ = W.build_step_tables(ctx, ql, 16, np.arange(need.sum()))
    return ctx, ql, int(need.sum()), q_indptr, page_indptr, page_indices


def test_mixed_batch_spans_stay_whole_on_few_ctas_and_decode_rows_are_queued():
    """Default policy on the Llama-shaped mixed batch: every (token, key) pair is covered once; span
    units are packed whole onto the first CTAs (a unit of two row tiles that would not fit is divided
    by rows first, so that few span units need partial rows); the CTAs without span work start
    on one decode chunk each and the rest of the decode work is queued."""
    ctx, ql, num_pages, q_indptr, page_indptr, page_indices = _llama_lengths()
    shape = W.Shape(32, 8, 128, 16)
    p = B.plan_host(shape, num_pages, q_indptr, ctx, page_indptr, page_indices, num_sms=148)
    items = p.items()
    # coverage, per (sequence, kv head, token)
    for b in range(32):
        for h in (0, 7):
            for i in {0, int(ql[b]) - 1}:
                segs = sorted((int(it["kv0"]), min(int(it["kv1"]), int(ctx[b]) + i + 1)) for it in items
                              if it["seq"] == b and it["kv_head"] == h and it["tok0"] <= i < it["tok0"] + it["ntok"])
                segs = [s for s in segs if s[1] > s[0]]
                assert segs[0][0] == 0 and segs[-1][1] == int(ctx[b]) + i + 1
                assert all(a[1] == c[0] for a, c in zip(segs[:-1], segs[1:]))
    span = items[items["path"] == 1]
    dec = items[items["path"] == 0]
    assert len(span) and len(dec)
    assert (span["kv0"] % 128 == 0).all() and (dec["kv0"] % 128 == 0).all()
    # span work sits on CTAs 0 .. used-1, the own decode chunks on the others
    used = int(span["cta"].max()) + 1
    assert set(span["cta"].tolist()) == set(range(used)) and 0 < used < 148
    own = dec[dec["cta"] >= 0]
    assert set(own["cta"].tolist()) == set(range(used, 148))
    # span units: at most 256 (token, head) rows, i.e. 64 tokens at 4 heads per kv head, and whole
    assert span["ntok"].max() <= 64
    keys = [(int(it["seq"]), int(it["kv_head"]), int(it["tok0"])) for it in span]
    assert len(keys) < 1.3 * len(set(keys))      # only the longest units are cut by keys as well
    # decode rows: one token per unit, never on the span body
    assert (dec["ntok"] == 1).all() and (span["ntok"] * 4 >= 32).all()
    _queue_checks(p, items, 148)
    # split decode units are merged inside the attention kernel; only span units cut by keys need
    # the merge kernel
    assert p.info["launches_attn"] == (2 if len(keys) > len(set(keys)) else 1) and p.info["num_split_units"] > 0


@pytest.mark.parametrize("seed", range(6))
def test_random_mixed_batches_are_covered_once_under_the_default_policy(seed):
    """Spans, decode rows, paused and empty-context sequences at head_dim 128 (both kernel bodies in
    play): every (sequence, kv head, token, key) is covered by exactly one item, whatever the SM count."""
    g = np.random.default_rng(100 + seed)
    n = int(g.integers(3, 40))
    ctx = g.integers(0, 3000, n)
    ctx[g.random(n) < 0.15] = 0
    ql = np.ones(n, dtype=np.int64)
    spans = g.random(n) < 0.3
    ql[spans] = g.integers(2, 80, int(spans.sum()))
    ql[g.random(n) < 0.1] = 0
    ql[(ctx == 0) & (ql == 0)] = 1
    heads = [(8, 2), (4, 1), (16, 2), (4, 4)][seed % 4]
    shape = W.Shape(heads[0], heads[1], 128, 16)
    wl = W.make_single_step("rnd", shape, ctx.tolist(), ql.tolist(), seed=seed)
    for sms in (3, 20, 148):
        p = plan(wl, num_sms=sms)
        items = check_cover(wl, p)
        assert items["cta"].max() < sms


def test_decode_only_batch_has_no_span_items():
    ctx, ql, num_pages, q_indptr, page_indptr, page_indices = _llama_lengths(1)
    ql[:] = 1
    need = -(-(ctx + ql) // 16)
    q_indptr, page_indptr, page_indices, _ = W.build_step_tables(ctx, ql, 16, np.arange(need.sum()))
    p = B.plan_host(W.Shape(32, 8, 128, 16), int(need.sum()), q_indptr, ctx, page_indptr, page_indices, num_sms=148)
    items = p.items()
    assert (items["path"] == 0).all() and p.info["num_items_tensor"] == 0
    own, queue, tiles, units, split = _queue_checks(p, items, 148)
    assert len(own) == 148 and p.info["launches_attn"] == 1


def test_long_span_units_are_cut_by_keys_and_merged_by_the_merge_kernel():
    """A span over a context far longer than a CTA's share has to be cut by keys as well."""
    shape = W.Shape(32, 8, 128, 16)
    ctx, ql = np.array([60000, 900]), np.array([64, 1])
    need = -(-(ctx + ql) // 16)
    q_indptr, page_indptr, page_indices, _ = W.build_step_tables(ctx, ql, 16, np.arange(need.sum()))
    p = B.plan_host(shape, int(need.sum()), q_indptr, ctx, page_indptr, page_indices, num_sms=148)
    items = p.items()
    span = items[items["path"] == 1]
    keys = [(int(it["seq"]), int(it["kv_head"]), int(it["tok0"])) for it in span]
    assert len(set(keys)) < len(keys)            # some unit has several chunks
    assert (span["ntok"] * 4 <= 128).all()      # and the row tiles were divided first
    assert p.info["launches_attn"] == 2


def test_host_workspace_must_be_16_byte_aligned():
    shape = W.Shape(8, 2, 64, 16)
    lib = B.load()
    import ctypes
    cs, co = B._cshape(shape, 2), B._copts(num_sms=148)
    cb, keep = B._cbatch([0, 1], [20], [0, 2], [1, 0])
    ws = np.zeros(1 << 14, dtype=np.int64)
    base = ws.ctypes.data
    out = ctypes.c_void_p()
    ok = base + (-base % 16)
    assert lib.asynclm_plan(ctypes.byref(cs), ctypes.byref(co), ctypes.byref(cb), ok, 1 << 16, None, 0,
                            None, ctypes.byref(out)) == 0
    assert lib.asynclm_plan(ctypes.byref(cs), ctypes.byref(co), ctypes.byref(cb), ok + 8, 1 << 16, None, 0,
                            None, ctypes.byref(out)) == -1
