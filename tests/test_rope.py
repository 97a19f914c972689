"""asynclm_kv_append_rope against the oracle: V rows and every untouched byte bit-exact; rotated K and Q
rows equal to the fp64 rotation rounded once to bf16, up to a rounding tie here and there (the two sides
evaluate pow / sin / cos with different libraries)."""
import numpy as np
import pytest

from oracle import oracle, rope
from paper_2412_07017_b200 import binding as B
from paper_2412_07017_b200 import workload as W

pytestmark = pytest.mark.gpu


def ulp_diff(a_bits, b_bits):
    """Distance in bf16 steps between two arrays of finite bf16 bit patterns."""
    key = lambda x: np.where(x & 0x8000, 0x8000 - (x & 0x7FFF).astype(np.int32), 0x8000 + (x & 0x7FFF).astype(np.int32))
    return np.abs(key(a_bits) - key(b_bits))


@pytest.mark.parametrize("Hq,Hkv,d,theta", [(32, 8, 128, 500000.0), (8, 2, 64, 10000.0)])
def test_rotated_append(Hq, Hkv, d, theta):
    import torch
    from gpu_util import to_bits, to_dev
    shape = W.Shape(Hq, Hkv, d, 16)
    wl = W.make_single_step("rope", shape, [5, 16, 31, 0, 4000, 70000], [12, 1, 2, 7, 40, 3], seed=31,
                            extra_pages=[0, 1, 0, 2, 1, 0], poison_unused=True)
    st = wl.steps[0]
    pool_dev = to_dev(wl.kv_pool)
    q_dev = to_dev(st.q)
    plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices)
    B.asynclm_kv_append_rope(plan, to_dev(st.k_new), to_dev(st.v_new), pool_dev, q_dev, theta)
    torch.cuda.synchronize()
    # oracle: rotate in fp64, round once, then the plain bit-copy append of the rotated rows
    pos = np.concatenate([np.arange(c, c + n) for c, n in zip(st.kv_len_before, st.q_len)])
    rot = lambda bits: W.f32_to_bf16_bits(rope.rotate(W.bf16_bits_to_f64(bits), pos, theta).astype(np.float32))
    k_rot, q_rot = rot(st.k_new), rot(st.q)
    ref_pool = wl.kv_pool.copy()
    oracle.kv_append(ref_pool, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices, k_rot, st.v_new)
    got_pool, got_q = to_bits(pool_dev), to_bits(q_dev)
    assert np.array_equal(got_pool[:, 1], ref_pool[:, 1])                        # V and all untouched V slots: exact
    differs = got_pool[:, 0] != ref_pool[:, 0]
    assert differs.mean() < 1e-4                                                  # untouched K slots are exact too
    assert ulp_diff(got_pool[:, 0][differs], ref_pool[:, 0][differs]).max(initial=0) <= 1
    dq = got_q != q_rot
    assert dq.mean() < 1e-3 and ulp_diff(got_q[dq], q_rot[dq]).max(initial=0) <= 1
