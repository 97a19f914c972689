"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Wraps ``asynclm_oracle.c`` (fp64, plain definition) through ctypes and adds the plain statement
of the split-KV merge.  Nothing here imports, or is imported by, the CUDA package; only tests, the
smoke check and the CPU-baseline leg of the benchmark may use it.

What it follows: an interrupt's tokens are appended at the end of the sequence's context and are
processed in the next decoding step together with the other sequences' decodes (paper Section 3.2
and Section 5.3); recomputing the whole context instead is the Section 5.5 variant, which the
append path must equal.

Pins (tests/test_oracle_pins.py): a separately written dense numpy evaluation with an explicit
mask, torch's scaled_dot_product_attention in fp64, closed forms (zero query -> mean of V and
lse = ln n; single key -> V exactly; a dominating key -> its V), append-then-attend == full
recomputation, invariance to physical page order, and the merge identity over arbitrary splits.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "asynclm_oracle.c")
_LIB = os.path.join(_HERE, "libasynclm_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_kv_append.restype = ctypes.c_int
        lib.oracle_kv_append.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                         ctypes.c_int, i32p, i32p, i32p, i32p, u16p, u16p, u16p]
        lib.oracle_attn_mixed.restype = ctypes.c_int
        lib.oracle_attn_mixed.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, i32p, i32p, i32p, i32p, u16p, u16p,
                                          ctypes.c_double, ctypes.c_int, i32p, f64p, f64p]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _u16(a):
    assert a.dtype == np.uint16 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def kv_append(kv_pool: np.ndarray, q_indptr, kv_len_before, page_indptr, page_indices,
              k_new: np.ndarray, v_new: np.ndarray) -> None:
    """Step 1: copy each new K/V row, bit for bit, to slot (ctx_b + i) of its sequence (in place)."""
    num_pages, two, Hkv, P, d = kv_pool.shape
    assert two == 2
    qi, qip = _i32(q_indptr)
    kb, kbp = _i32(kv_len_before)
    pi, pip_ = _i32(page_indptr)
    px, pxp = _i32(page_indices)
    rc = _load().oracle_kv_append(Hkv, d, P, num_pages, len(kb), qip, kbp, pip_, pxp,
                                  _u16(k_new), _u16(v_new), _u16(kv_pool))
    if rc != 0:
        raise ValueError("oracle_kv_append: page table does not cover the appended rows")


def attn_mixed(kv_pool: np.ndarray, q: np.ndarray, q_indptr, kv_len_before, page_indptr,
               page_indices, sm_scale: float = 0.0,
               sel_rows: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Step 2: fp64 attention of every new row over keys [0, ctx_b + i] of the post-append pool.

    Returns (out [T, Hq, d] float64, lse [T, Hq] float64, natural log).  With ``sel_rows`` only
    those token rows are computed; the rest of the returned arrays is NaN.
    """
    num_pages, two, Hkv, P, d = kv_pool.shape
    T, Hq, d2 = q.shape
    assert d2 == d and Hq % Hkv == 0
    qi, qip = _i32(q_indptr)
    kb, kbp = _i32(kv_len_before)
    pi, pip_ = _i32(page_indptr)
    px, pxp = _i32(page_indices)
    assert int(qi[-1]) == T
    out = np.full((T, Hq, d), np.nan, dtype=np.float64)
    lse = np.full((T, Hq), np.nan, dtype=np.float64)
    if sel_rows is None:
        n_sel, sel, selp = 0, None, None
    else:
        sel, selp = _i32(sel_rows)
        n_sel = len(sel)
        if n_sel == 0:
            return out, lse
    if T == 0:
        return out, lse
    f64p = ctypes.POINTER(ctypes.c_double)
    rc = _load().oracle_attn_mixed(Hq, Hkv, d, P, len(kb), qip, kbp, pip_, pxp, _u16(q),
                                   _u16(kv_pool), float(sm_scale), n_sel, selp,
                                   out.ctypes.data_as(f64p), lse.ctypes.data_as(f64p))
    if rc != 0:
        raise MemoryError("oracle_attn_mixed failed")
    return out, lse


def step(kv_pool: np.ndarray, st, sm_scale: float = 0.0, sel_rows=None):
    """Append then attend for one workload step (``st`` has the Step fields).  Mutates kv_pool."""
    kv_append(kv_pool, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
              st.k_new, st.v_new)
    return attn_mixed(kv_pool, st.q, st.q_indptr, st.kv_len_before, st.page_indptr,
                      st.page_indices, sm_scale, sel_rows)


def lse_merge(o_parts: np.ndarray, lse_parts: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Plain statement of the split-KV merge over chunks c (axis 0):

        LSE = ln sum_c exp(LSE_c),   O = sum_c exp(LSE_c - LSE) O_c

    where O_c is the softmax-weighted average inside chunk c and LSE_c its log-sum-exp.  A chunk
    with no visible key has LSE_c = -inf and weight 0.
    """
    o_parts = np.asarray(o_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    m = np.max(lse_parts, axis=0)
    w = np.exp(lse_parts - m)
    tot = w.sum(axis=0)
    o = (w[..., None] * np.where(w[..., None] > 0, o_parts, 0.0)).sum(axis=0) / tot[..., None]
    return o, m + np.log(tot)
