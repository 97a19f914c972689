"""Child process of test_checked_build.py: runs with ASYNCLM_LIBRARY pointing at the checked build
(-DASYNCLM_DEBUG) of the library, so that the page-id checks are compiled in before anything is made
to depend on them.  Prints one JSON line."""
import json
import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(HERE))
sys.path.insert(0, HERE)

from paper_2412_07017_b200 import binding as B  # noqa: E402
from paper_2412_07017_b200 import workload as W  # noqa: E402
from gpu_util import assert_close, oracle_step, to_bits, to_dev  # noqa: E402


def find_page_table(plan, page_indices):
    """Word offset of the step's page_indices array inside the plan's device workspace."""
    n = plan.dev_ws.numel() // 4 * 4
    words = plan.dev_ws[:n].view(torch.int32).cpu().numpy()
    pat = np.asarray(page_indices, dtype=np.int32)
    first = np.flatnonzero(words[: len(words) - len(pat) + 1] == pat[0])
    hits = [int(i) for i in first if np.array_equal(words[i:i + len(pat)], pat)]
    assert len(hits) == 1, hits
    return hits[0]


def main():
    assert "debug" in os.path.basename(os.environ.get("ASYNCLM_LIBRARY", "")), "the checked build must be the one loaded"
    torch.cuda.set_device(0)
    shape = W.Shape(32, 8, 128, 16)
    # a decode row over 44 pages, a 40-token span (160 rows per kv head: the span body) over 59 pages, a short row
    wl = W.make_single_step("checked", shape, [700, 900, 300], [1, 40, 1], seed=77)
    st = wl.steps[0]
    pool = to_dev(wl.kv_pool)
    q, kn, vn = to_dev(st.q), to_dev(st.k_new), to_dev(st.v_new)
    _, ref_out, ref_lse = oracle_step(wl, st)
    bad = wl.num_pages + 7
    result = {}

    def run(corrupt_seq):
        out = torch.zeros((st.total_q, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((st.total_q, shape.num_q_heads), dtype=torch.float32, device="cuda")
        # whole units, dealt statically: every item starts at key 0, so its page 36 is read from the table
        plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                              kv_chunk_tokens=1 << 20)
        B.asynclm_kv_append(plan, kn, vn, pool)
        if corrupt_seq is not None:
            torch.cuda.synchronize()
            off = find_page_table(plan, st.page_indices)
            n = plan.dev_ws.numel() // 4 * 4
            words = plan.dev_ws[:n].view(torch.int32)
            words[off + int(st.page_indptr[corrupt_seq]) + 36] = bad
        B.asynclm_attn_mixed(plan, q, pool, out, lse)
        torch.cuda.synchronize()
        return B.last_device_status(plan), to_bits(out), lse.cpu().numpy(), plan

    status, out, lse, plan = run(None)
    assert status == 0, status
    assert plan.info["num_items_tensor"] > 0
    assert_close(out, lse, ref_out, ref_lse, what="checked build, untouched plan")
    result["clean"] = status
    # a page id beyond the pool in the decode row's table: the warp body reports it and reads page 0 instead
    status, out, lse, _ = run(0)
    result["bad_id_warp_body"] = status
    # the rows of the other sequences do not depend on it
    rows = np.arange(int(st.q_indptr[1]), st.total_q)
    assert_close(out[rows], lse[rows], ref_out[rows], ref_lse[rows], what="checked build, other sequences")
    # the same in the span's table: the span body reports it and takes zeros for the page
    status, out, lse, _ = run(1)
    result["bad_id_span_body"] = status
    keep = np.r_[0, np.arange(int(st.q_indptr[2]), st.total_q)]
    assert_close(out[keep], lse[keep], ref_out[keep], ref_lse[keep], what="checked build, other sequences")
    print(json.dumps(result))


def wait_expiry():
    """A hand-off that never comes: the bounded waits run out, the status word names one of them, the
    context stays usable and the next step is correct."""
    import ctypes
    torch.cuda.set_device(0)
    shape = W.Shape(32, 8, 128, 16)
    wl = W.make_single_step("stall", shape, [1500, 1200], [64, 64], seed=78)      # spans only: the span kernel alone
    st = wl.steps[0]
    pool = to_dev(wl.kv_pool)
    q, kn, vn = to_dev(st.q), to_dev(st.k_new), to_dev(st.v_new)
    _, ref_out, ref_lse = oracle_step(wl, st)
    lib = B.load()
    lib.asynclm_debug_stall_span_tile.argtypes = [ctypes.c_void_p, ctypes.c_int32]
    lib.asynclm_debug_stall_span_tile.restype = ctypes.c_int

    def run(stall):
        out = torch.zeros((st.total_q, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((st.total_q, shape.num_q_heads), dtype=torch.float32, device="cuda")
        plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices)
        assert plan.info["num_items_tensor"] == plan.info["num_items"] > 0
        assert lib.asynclm_debug_stall_span_tile(ctypes.c_void_p(plan.handle), stall) == 0
        B.asynclm_kv_append(plan, kn, vn, pool)
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        B.asynclm_attn_mixed(plan, q, pool, out, lse)
        t1.record()
        torch.cuda.synchronize()
        return B.last_device_status(plan), to_bits(out), lse.cpu().numpy(), t0.elapsed_time(t1)

    status, _, _, ms = run(2)
    res = {"stalled_status": status, "stalled_ms": ms}
    status, out, lse, ms = run(0)
    assert_close(out, lse, ref_out, ref_lse, what="the step after a wait ran out")
    res.update({"next_status": status, "next_ms": ms})
    print(json.dumps(res))


if __name__ == "__main__":
    wait_expiry() if sys.argv[1:] == ["wait"] else main()
