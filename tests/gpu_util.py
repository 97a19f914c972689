"""Helpers for the GPU parity tests: run one step through the C ABI and bring the results back."""
import numpy as np
import torch

from oracle import oracle
from paper_2412_07017_b200 import binding as B
from paper_2412_07017_b200 import workload as W

MAX_ABS = 1e-2      # bf16 in, fp32 accumulate, bf16 out: max |gpu - oracle|
MEAN_ABS = 1e-3     # mean |gpu - oracle| over all output elements of a step
LSE_ABS = 1e-3

# "calls": asynclm_kv_append + asynclm_attn_mixed; "step": asynclm_step (one launch).  The parity
# module runs every test both ways.
API = "calls"


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> cuda bfloat16 tensor of the same shape."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def gpu_step(wl, st, pool_dev=None, want_lse=True, sm_scale=0.0, **opts):
    """plan + kv_append + attn_mixed on the current device; returns (pool_dev, out bits, lse, plan)."""
    if pool_dev is None:
        pool_dev = to_dev(wl.kv_pool)
    q, kn, vn = to_dev(st.q), to_dev(st.k_new), to_dev(st.v_new)
    T = st.total_q
    out = torch.full((T, wl.shape.num_q_heads, wl.shape.head_dim), float("nan"),
                     dtype=torch.bfloat16, device="cuda")
    lse = torch.full((T, wl.shape.num_q_heads), float("nan"), dtype=torch.float32,
                     device="cuda") if want_lse else None
    plan = B.asynclm_plan(wl.shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr,
                          st.page_indices, sm_scale=sm_scale, **opts)
    if API == "step":
        B.asynclm_step(plan, q, kn, vn, pool_dev, out, lse)
    else:
        B.asynclm_kv_append(plan, kn, vn, pool_dev)
        B.asynclm_attn_mixed(plan, q, pool_dev, out, lse)
    torch.cuda.synchronize()
    assert B.last_device_status(plan) == 0
    return pool_dev, to_bits(out), (lse.cpu().numpy() if want_lse else None), plan


def oracle_step(wl, st, pool=None, sm_scale=0.0, sel_rows=None):
    pool = wl.kv_pool.copy() if pool is None else pool
    out, lse = oracle.step(pool, st, sm_scale, sel_rows)
    return pool, out, lse


def assert_close(out_bits, lse, ref_out, ref_lse, rows=None, what=""):
    got = W.bf16_bits_to_f64(out_bits)
    if rows is not None:
        got, ref_out = got[rows], ref_out[rows]
        if lse is not None:
            lse, ref_lse = lse[rows], ref_lse[rows]
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    if got.size == 0:
        return 0.0, 0.0
    err = np.abs(got - ref_out)
    assert err.max() <= MAX_ABS, f"{what}: max abs err {err.max():.4g}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean abs err {err.mean():.4g}"
    if lse is not None:
        le = np.abs(lse.astype(np.float64) - ref_lse)
        assert le.max() <= LSE_ABS, f"{what}: lse err {le.max():.4g}"
    return float(err.max()), float(err.mean())
