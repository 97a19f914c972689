"""Trap handler (paper Section 5.4): the library's decision rule and swap kernels against the oracle."""
import numpy as np
import pytest

from oracle import trap
from paper_2412_07017_b200 import binding as B
from paper_2412_07017_b200 import workload as W


def test_decision_rule_matches_the_oracle_on_a_grid():
    g = np.random.default_rng(0)
    for _ in range(20):
        m = dict(swap_fixed_us=g.uniform(0, 500), swap_us_per_token=g.uniform(0.1, 100),
                 recompute_fixed_us=g.uniform(0, 5000), recompute_us_per_token=g.uniform(0, 100),
                 recompute_us_per_token2=g.uniform(0, 0.2))
        for n in (0, 1, 17, 300, 4096, 100000):
            for w in (0.0, 10.0, 1e3, 1e5, 1e9):
                dec, s, r = B.asynclm_trap_decide(m, n, w)
                assert dec == trap.decide(m, n, w)
                assert s == pytest.approx(trap.swap_us(m, n)) and r == pytest.approx(trap.recompute_us(m, n))
    assert (B.TRAP_KEEP, B.TRAP_SWAP, B.TRAP_RECOMPUTE) == (trap.KEEP, trap.SWAP, trap.RECOMPUTE)


def test_swap_argument_checks_need_no_gpu():
    import ctypes
    lib = B.load()
    cs = B._cshape(W.Shape(8, 2, 64, 16), 10)
    ids = np.array([1, 2, 12], dtype=np.int32)
    buf = np.zeros(1 << 16, dtype=np.uint8)
    a = buf.ctypes.data + (-buf.ctypes.data % 256)
    assert lib.asynclm_kv_swap_out(ctypes.byref(cs), ids.ctypes.data, 3, a, a, a, None) == -3      # id outside the pool
    ids[2] = 2
    assert lib.asynclm_kv_swap_in(ctypes.byref(cs), ids.ctypes.data, 3, a, a, a, None) == -3       # duplicate destination
    assert lib.asynclm_kv_swap_in(ctypes.byref(cs), ids.ctypes.data, 3, a, a + 8, a, None) == -1   # misaligned
    assert lib.asynclm_kv_swap_out(ctypes.byref(cs), None, 0, None, None, None, None) == 0
    assert B.kv_swap_staging_bytes(W.Shape(8, 2, 64, 16), 10, 3) >= 3 * 2 * 2 * 16 * 64 * 2 + 12


@pytest.mark.gpu
@pytest.mark.parametrize("Hq,Hkv,d", [(32, 8, 128), (8, 2, 64)])
def test_swap_out_and_in_are_bit_copies(Hq, Hkv, d):
    """A paused sequence's pages go to pinned host memory and come back into other pages: the image,
    the pool after the swap-in and every untouched page agree with the oracle byte for byte."""
    import torch
    from gpu_util import to_bits, to_dev
    shape = W.Shape(Hq, Hkv, d, 16)
    wl = W.make_single_step("swap", shape, [700, 333, 90], [1, 0, 1], seed=21, spare_pages=60)
    st = wl.steps[0]
    pool_dev = to_dev(wl.kv_pool)
    ref_pool = wl.kv_pool.copy()
    b = 1                                                     # the paused sequence
    old = st.page_indices[st.page_indptr[b]:st.page_indptr[b + 1]]
    n = len(old)
    staging = torch.empty(B.kv_swap_staging_bytes(shape, wl.num_pages, n), dtype=torch.uint8, device="cuda")
    image = torch.zeros((n,) + wl.kv_pool.shape[1:], dtype=torch.int16).pin_memory()
    B.asynclm_kv_swap_out(shape, wl.num_pages, old, pool_dev, staging, image)
    torch.cuda.synchronize()
    ref_image = trap.swap_out(ref_pool, old)
    assert np.array_equal(image.numpy().view(np.uint16), ref_image)
    assert np.array_equal(to_bits(pool_dev), ref_pool)                      # swap-out does not write the pool
    # the old pages are reused by someone else, the sequence comes back into pages nobody owns
    pool_dev[torch.from_numpy(old.astype(np.int64)).cuda()] = 0
    ref_pool[old] = 0
    used = set(st.page_indices.tolist())
    new = np.array([p for p in np.random.default_rng(3).permutation(wl.num_pages) if p not in used][:n], dtype=np.int32)
    B.asynclm_kv_swap_in(shape, wl.num_pages, new, pool_dev, staging, image)
    torch.cuda.synchronize()
    trap.swap_in(ref_pool, new, ref_image)
    assert np.array_equal(to_bits(pool_dev), ref_pool)
