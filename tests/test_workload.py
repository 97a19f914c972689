"""The seeded input generators: determinism, shapes and table consistency (no arithmetic)."""
import numpy as np

from paper_2412_07017_b200 import workload as W


def _check_tables(wl, st):
    P = wl.shape.page_size
    n = st.kv_len_before.astype(np.int64) + st.q_len
    have = np.diff(st.page_indptr)
    assert (have * P >= n).all()
    assert st.page_indices.min() >= 0 and st.page_indices.max() < wl.num_pages
    assert len(np.unique(st.page_indices)) == len(st.page_indices)
    assert st.q.shape == (st.total_q, wl.shape.num_q_heads, wl.shape.head_dim)
    assert st.k_new.shape == (st.total_q, wl.shape.num_kv_heads, wl.shape.head_dim)


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38], dtype=np.float32)
    b = W.f32_to_bf16_bits(x)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up
    assert list(b[:4]) == [0x3F80, 0x3F80, 0x3F82, 0xC020]
    back = W.bf16_bits_to_f64(b)
    assert back[0] == 1.0 and back[3] == -2.5


def test_config1_shape_and_determinism():
    a = W.make_config(1)
    b = W.make_config(1)
    st = a.steps[0]
    assert a.shape == W.Shape(8, 2, 64, 16) and st.batch == 4
    assert list(st.q_len) == [12, 1, 1, 1]
    assert ((st.kv_len_before >= 100) & (st.kv_len_before <= 300)).all()
    assert np.array_equal(a.kv_pool, b.kv_pool) and np.array_equal(st.q, b.steps[0].q)
    _check_tables(a, st)
    c = W.make_config(1, seed=5)
    assert not np.array_equal(c.steps[0].q, st.q)


def test_config2_lengths():
    wl = W.make_config(2, scale=0.05)
    st = wl.steps[0]
    assert st.batch == 32 and (st.q_len > 1).sum() == 8
    app = st.q_len[st.q_len > 1]
    assert app.min() >= 8 and app.max() <= 64
    _check_tables(wl, st)
    by = W.algorithmic_bytes(wl.shape, st)
    n = (st.kv_len_before + st.q_len).sum()
    assert by["kv"] == int(n) * 4096


def test_values_look_standard_normal():
    x = W.bf16_bits_to_f64(W.normal_bf16(1, 2, (1 << 16,)))
    assert abs(x.mean()) < 0.02 and abs(x.std() - 1) < 0.02


def test_replay_grows_consistently():
    wl = W.make_replay(batch=16, steps=30, ctx_lo=20, ctx_hi=80, rate=0.1,
                       shape=W.Shape(4, 2, 32, 16))
    ctx = wl.steps[0].kv_len_before.astype(np.int64)
    seen_append = False
    for st in wl.steps:
        assert np.array_equal(st.kv_len_before, ctx)
        assert (st.q_len >= 1).all()
        seen_append |= bool((st.q_len > 1).any())
        _check_tables(wl, st)
        ctx = ctx + st.q_len
    assert seen_append
    # a sequence's page list only ever grows by appending
    a, b = wl.steps[0], wl.steps[-1]
    for s in range(16):
        pa = a.page_indices[a.page_indptr[s]:a.page_indptr[s + 1]]
        pb = b.page_indices[b.page_indptr[s]:b.page_indptr[s + 1]]
        assert np.array_equal(pb[:len(pa)], pa)
