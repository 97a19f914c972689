"""ctypes binding of libasynclm.so: argument marshalling only.

Every step of the path (planning, append, attention, merge) runs inside the shared library; this
module converts Python objects to the C structs of include/asynclm.h and owns the two workspaces a
plan lives in.  torch is used for device memory, pinned host memory and streams.  There is no
fallback: if the library cannot be loaded, every entry point raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np

from . import build as _build

EXPORTS = [
    "asynclm_version", "asynclm_strerror", "asynclm_plan_workspace_size", "asynclm_plan",
    "asynclm_plan_get_info", "asynclm_plan_get_items", "asynclm_kv_append", "asynclm_attn_mixed",
    "asynclm_last_device_status", "asynclm_last_cuda_error", "asynclm_attn_mixed_static",
    "asynclm_static_scratch_bytes", "asynclm_step", "asynclm_read_ceiling", "asynclm_kv_swap_staging_bytes",
    "asynclm_kv_swap_out", "asynclm_kv_swap_in", "asynclm_trap_decide", "asynclm_latency_model",
    "asynclm_async_latency_of_order", "asynclm_token_monitor_step", "asynclm_token_monitor_workspace_bytes",
    "asynclm_kv_append_rope",
]

TRAP_KEEP, TRAP_SWAP, TRAP_RECOMPUTE = 0, 1, 2

PLAN_REJECT_ALIASED_WRITES = 1
PLAN_NO_TENSOR_PATH = 2


class AsynclmError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        detail = f" [{load().asynclm_last_cuda_error().decode()}]" if status == -5 else ""
        super().__init__(f"{what}: {strerror(status)} ({status}){detail}")


class CShape(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("num_pages", ctypes.c_int64), ("sm_scale", ctypes.c_float),
                ("reserved", ctypes.c_int32)]


class CPlanOptions(ctypes.Structure):
    _fields_ = [("num_sms", ctypes.c_int32), ("kv_chunk_tokens", ctypes.c_int32),
                ("tensor_min_rows", ctypes.c_int32), ("flags", ctypes.c_int32)]


class CTrapModel(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("swap_fixed_us", "swap_us_per_token", "recompute_fixed_us",
                                               "recompute_us_per_token", "recompute_us_per_token2")]


class CCmlTokens(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("call", "intr", "trap", "end", "head")]


class CLatency(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("l_sync", "l_sync_par", "l_async", "speedup_estimate")]


class CBatch(ctypes.Structure):
    # the four arrays are `const int32_t*` in C; plain addresses marshal faster than typed pointers
    _fields_ = [("batch", ctypes.c_int32),
                ("q_indptr", ctypes.c_void_p),
                ("kv_len_before", ctypes.c_void_p),
                ("page_indptr", ctypes.c_void_p),
                ("page_indices", ctypes.c_void_p)]


class CPlanInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "total_q", "num_units", "num_items", "num_split_units", "partial_rows", "kv_chunk_tokens",
        "num_ctas_cuda", "num_ctas_tensor", "num_items_tensor", "launches_append", "launches_attn",
        "num_sms")] + [("total_kv_tokens", ctypes.c_int64), ("device_bytes_used", ctypes.c_uint64),
                       ("host_bytes_used", ctypes.c_uint64)]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


ITEM_DTYPE = np.dtype([(n, np.int32) for n in
                       ("seq", "kv_head", "tok0", "ntok", "kv0", "kv1", "path", "cta")])

_lib = None


def load(rebuild_if_stale: bool = True):
    """Load libasynclm.so, building it first when the sources are newer (needs nvcc)."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("ASYNCLM_LIBRARY") or _build.LIB      # e.g. the time-stamp build of build.py
    if path == _build.LIB and rebuild_if_stale and _build.find_nvcc() is not None and _build.is_stale():
        _build.build()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing and could not be built; the CUDA library is required "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(path)
    vp, i32, i64, szp = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.POINTER(ctypes.c_size_t)
    lib.asynclm_version.restype = ctypes.c_int
    lib.asynclm_strerror.restype = ctypes.c_char_p
    lib.asynclm_strerror.argtypes = [ctypes.c_int]
    lib.asynclm_last_cuda_error.restype = ctypes.c_char_p
    lib.asynclm_plan_workspace_size.argtypes = [ctypes.POINTER(CShape), ctypes.POINTER(CPlanOptions),
                                                i32, i32, i64, szp, szp]
    lib.asynclm_plan.argtypes = [ctypes.POINTER(CShape), ctypes.POINTER(CPlanOptions),
                                 ctypes.POINTER(CBatch), vp, ctypes.c_size_t, vp, ctypes.c_size_t,
                                 vp, ctypes.POINTER(vp)]
    lib.asynclm_plan_get_info.argtypes = [vp, ctypes.POINTER(CPlanInfo)]
    lib.asynclm_plan_get_items.argtypes = [vp, vp, i32]
    lib.asynclm_kv_append.argtypes = [vp, vp, vp, vp, vp]
    lib.asynclm_attn_mixed.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.asynclm_kv_append_rope.argtypes = [vp, vp, vp, vp, vp, ctypes.c_double, vp]
    lib.asynclm_attn_mixed_static.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.asynclm_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.asynclm_read_ceiling.argtypes = [vp, vp, i64, i64, i32, vp, vp]
    lib.asynclm_kv_swap_staging_bytes.argtypes = [ctypes.POINTER(CShape), i32]
    lib.asynclm_kv_swap_out.argtypes = [ctypes.POINTER(CShape), vp, i32, vp, vp, vp, vp]
    lib.asynclm_kv_swap_in.argtypes = [ctypes.POINTER(CShape), vp, i32, vp, vp, vp, vp]
    lib.asynclm_latency_model.argtypes = [vp, vp, i32, ctypes.POINTER(CLatency), vp]
    lib.asynclm_async_latency_of_order.argtypes = [vp, vp, vp, i32, ctypes.POINTER(ctypes.c_double), vp]
    lib.asynclm_token_monitor_step.argtypes = [vp, i32, i32, i32, i64, ctypes.POINTER(CCmlTokens), vp, vp, vp, vp, vp, vp]
    lib.asynclm_token_monitor_workspace_bytes.argtypes = [i32]
    lib.asynclm_trap_decide.argtypes = [ctypes.POINTER(CTrapModel), i32, ctypes.c_double,
                                        ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double),
                                        ctypes.POINTER(ctypes.c_double)]
    lib.asynclm_static_scratch_bytes.argtypes = []
    lib.asynclm_last_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
    for name in EXPORTS:
        if name not in ("asynclm_strerror", "asynclm_last_cuda_error", "asynclm_static_scratch_bytes",
                        "asynclm_kv_swap_staging_bytes", "asynclm_token_monitor_workspace_bytes"):
            getattr(lib, name).restype = ctypes.c_int
    lib.asynclm_static_scratch_bytes.restype = ctypes.c_size_t
    lib.asynclm_kv_swap_staging_bytes.restype = ctypes.c_size_t
    lib.asynclm_token_monitor_workspace_bytes.restype = ctypes.c_size_t
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().asynclm_strerror(int(status)).decode()


def _check(rc: int, what: str):
    if rc != 0:
        raise AsynclmError(rc, what)


def _cshape(shape, num_pages: int, sm_scale: float = 0.0) -> CShape:
    return CShape(shape.num_q_heads, shape.num_kv_heads, shape.head_dim, shape.page_size,
                  int(num_pages), float(sm_scale), 0)


def _copts(num_sms=0, kv_chunk_tokens=0, tensor_min_rows=0, flags=0) -> CPlanOptions:
    return CPlanOptions(int(num_sms), int(kv_chunk_tokens), int(tensor_min_rows), int(flags))


def _i32(a):
    if not (isinstance(a, np.ndarray) and a.dtype == np.int32 and a.flags.c_contiguous):
        a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data


def _cbatch(q_indptr, kv_len_before, page_indptr, page_indices):
    keep = [_i32(q_indptr), _i32(kv_len_before), _i32(page_indptr), _i32(page_indices)]
    b = CBatch(len(keep[1][0]), keep[0][1], keep[1][1], keep[2][1], keep[3][1])
    return b, keep


def workspace_size(shape, num_pages, max_batch, max_total_q, max_total_pages, **opts):
    """Upper bounds (host_bytes, device_bytes) for any batch within the given maxima."""
    hs, ds = ctypes.c_size_t(0), ctypes.c_size_t(0)
    cs, co = _cshape(shape, num_pages), _copts(**opts)
    _check(load().asynclm_plan_workspace_size(ctypes.byref(cs), ctypes.byref(co), max_batch,
                                              max_total_q, max_total_pages, ctypes.byref(hs),
                                              ctypes.byref(ds)), "asynclm_plan_workspace_size")
    return int(hs.value), int(ds.value)


@dataclass
class Plan:
    """A plan handle with the workspaces it lives in.  `info` (what the planner decided) is read from
    the plan on first access, so look at it before the workspaces are reused for another plan."""
    handle: int
    host_ws: object
    dev_ws: object
    keepalive: object = None
    _info: Optional[dict] = None

    @property
    def info(self) -> dict:
        if self._info is None:
            self._info = _get_info(self.handle)
        return self._info

    def items(self) -> np.ndarray:
        n = self.info["num_items"]
        arr = np.zeros(max(n, 1), dtype=ITEM_DTYPE)
        rc = load().asynclm_plan_get_items(self.handle, arr.ctypes.data, n)
        if rc < 0:
            raise AsynclmError(rc, "asynclm_plan_get_items")
        return arr[:n]


def _get_info(handle) -> dict:
    info = CPlanInfo()
    _check(load().asynclm_plan_get_info(handle, ctypes.byref(info)), "asynclm_plan_get_info")
    return info.as_dict()


def plan_host(shape, num_pages, q_indptr, kv_len_before, page_indptr, page_indices, num_sms=148,
              sm_scale=0.0, **opts) -> Plan:
    """Host-only planning (no CUDA call): for inspection, sizing and CPU tests."""
    lib = load()
    cs, co = _cshape(shape, num_pages, sm_scale), _copts(num_sms=num_sms, **opts)
    cb, keep = _cbatch(q_indptr, kv_len_before, page_indptr, page_indices)
    T = int(keep[0][0][-1]) if len(keep[0][0]) else 0
    hbytes = 1 << 16
    while True:
        ws = np.zeros(hbytes // 8, dtype=np.int64)
        out = ctypes.c_void_p()
        rc = lib.asynclm_plan(ctypes.byref(cs), ctypes.byref(co), ctypes.byref(cb), ws.ctypes.data,
                              ws.nbytes, None, 0, None, ctypes.byref(out))
        if rc == -4 and hbytes < (1 << 32):
            hbytes *= 4
            continue
        _check(rc, "asynclm_plan")
        return Plan(out.value, ws, None, keep)


def asynclm_plan(shape, num_pages, q_indptr, kv_len_before, page_indptr, page_indices,
                 stream=None, sm_scale=0.0, host_ws=None, dev_ws=None, **opts) -> Plan:
    """Plan one step on the current CUDA device; uploads the plan on `stream`.

    host_ws (pinned uint8 tensor) and dev_ws (cuda uint8 tensor) may be supplied for reuse;
    otherwise they are sized exactly by a host-only dry run and allocated here.
    """
    import torch
    lib = load()
    cs, co = _cshape(shape, num_pages, sm_scale), _copts(**opts)
    cb, keep = _cbatch(q_indptr, kv_len_before, page_indptr, page_indices)
    if host_ws is None or dev_ws is None:
        sms = opts.get("num_sms") or torch.cuda.get_device_properties(
            torch.cuda.current_device()).multi_processor_count
        dry_opts = dict(opts)
        dry_opts.pop("num_sms", None)
        dry = plan_host(shape, num_pages, q_indptr, kv_len_before, page_indptr, page_indices,
                        num_sms=sms, sm_scale=sm_scale, **dry_opts)
        if host_ws is None:
            host_ws = torch.empty(dry.info["host_bytes_used"] + 256, dtype=torch.uint8).pin_memory()
        if dev_ws is None:
            dev_ws = torch.empty(dry.info["device_bytes_used"] + 256, dtype=torch.uint8, device="cuda")
    s = _stream_ptr(stream)
    out = ctypes.c_void_p()
    _check(lib.asynclm_plan(ctypes.byref(cs), ctypes.byref(co), ctypes.byref(cb),
                            host_ws.data_ptr(), host_ws.numel(), dev_ws.data_ptr(), dev_ws.numel(),
                            s, ctypes.byref(out)), "asynclm_plan")
    return Plan(out.value, host_ws, dev_ws, None)


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def asynclm_kv_append(plan: Plan, k_new, v_new, kv_pool, stream=None) -> None:
    """Scatter the step's new K/V rows (device tensors) into kv_pool through the page table."""
    _check(load().asynclm_kv_append(plan.handle, k_new.data_ptr(), v_new.data_ptr(),
                                    kv_pool.data_ptr(), _stream_ptr(stream)), "asynclm_kv_append")


def asynclm_kv_append_rope(plan: Plan, k_new, v_new, kv_pool, q_inout=None, rope_theta=500000.0, stream=None) -> None:
    """asynclm_kv_append with the keys (and, if given, the queries, in place) rotated by their positions."""
    _check(load().asynclm_kv_append_rope(plan.handle, k_new.data_ptr(), v_new.data_ptr(), kv_pool.data_ptr(),
                                         None if q_inout is None else q_inout.data_ptr(), float(rope_theta),
                                         _stream_ptr(stream)), "asynclm_kv_append_rope")


def asynclm_attn_mixed(plan: Plan, q, kv_pool, out, lse=None, stream=None) -> None:
    """Attention of every new row over its sequence's pages; writes `out` (bf16) and `lse` (fp32)."""
    _check(load().asynclm_attn_mixed(plan.handle, q.data_ptr(), kv_pool.data_ptr(), out.data_ptr(),
                                     None if lse is None else lse.data_ptr(), _stream_ptr(stream)),
           "asynclm_attn_mixed")


def asynclm_step(plan: Plan, q, k_new, v_new, kv_pool, out, lse=None, stream=None) -> None:
    """Append and attention in one launch (asynclm_kv_append + asynclm_attn_mixed)."""
    _check(load().asynclm_step(plan.handle, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                               kv_pool.data_ptr(), out.data_ptr(),
                               None if lse is None else lse.data_ptr(), _stream_ptr(stream)),
           "asynclm_step")


def kv_swap_staging_bytes(shape, num_pages: int, n_pages: int) -> int:
    cs = _cshape(shape, num_pages)
    return int(load().asynclm_kv_swap_staging_bytes(ctypes.byref(cs), int(n_pages)))


def asynclm_kv_swap_out(shape, num_pages: int, page_ids, kv_pool, staging, host_image, stream=None) -> None:
    """Gather the pages `page_ids` (host ints) of kv_pool into host_image (pinned tensor) via `staging`."""
    ids, ptr = _i32(page_ids)
    cs = _cshape(shape, num_pages)
    _check(load().asynclm_kv_swap_out(ctypes.byref(cs), ptr, len(ids), kv_pool.data_ptr(), staging.data_ptr(),
                                      host_image.data_ptr(), _stream_ptr(stream)), "asynclm_kv_swap_out")


def asynclm_kv_swap_in(shape, num_pages: int, page_ids, kv_pool, staging, host_image, stream=None) -> None:
    """Scatter host_image (pinned tensor) into the pages `page_ids` (host ints) of kv_pool via `staging`."""
    ids, ptr = _i32(page_ids)
    cs = _cshape(shape, num_pages)
    _check(load().asynclm_kv_swap_in(ctypes.byref(cs), ptr, len(ids), kv_pool.data_ptr(), staging.data_ptr(),
                                     host_image.data_ptr(), _stream_ptr(stream)), "asynclm_kv_swap_in")


def asynclm_trap_decide(model: dict, context_tokens: int, wait_us: float):
    """(decision, swap_us, recompute_us) of the keep / swap / recompute rule."""
    cm = CTrapModel(*(float(model[n]) for n, _ in CTrapModel._fields_))
    dec, s, r = ctypes.c_int32(-1), ctypes.c_double(0), ctypes.c_double(0)
    _check(load().asynclm_trap_decide(ctypes.byref(cm), int(context_tokens), float(wait_us), ctypes.byref(dec),
                                      ctypes.byref(s), ctypes.byref(r)), "asynclm_trap_decide")
    return int(dec.value), float(s.value), float(r.value)


def token_monitor_workspace_bytes(batch: int) -> int:
    return int(load().asynclm_token_monitor_workspace_bytes(int(batch)))


def asynclm_token_monitor_step(logits, special: dict, state_in, token_out, state_out, flags_out, workspace,
                               stream=None) -> None:
    """Masked greedy next token and CML state advance for a batch (device tensors; logits bf16 or fp32,
    [batch][vocab]); special: {"CALL", "INTR", "TRAP", "END", "HEAD"} -> token id; workspace: zeroed
    uint8 device tensor of token_monitor_workspace_bytes(batch) bytes (left zeroed)."""
    import torch
    ct = CCmlTokens(*(int(special[k]) for k in ("CALL", "INTR", "TRAP", "END", "HEAD")))
    dtype = 0 if logits.dtype == torch.bfloat16 else 1
    _check(load().asynclm_token_monitor_step(logits.data_ptr(), dtype, logits.shape[0], logits.shape[1],
                                             logits.stride(0), ctypes.byref(ct), state_in.data_ptr(),
                                             token_out.data_ptr(), state_out.data_ptr(), flags_out.data_ptr(),
                                             workspace.data_ptr(), _stream_ptr(stream)), "asynclm_token_monitor_step")


def asynclm_latency_model(gen, exe) -> dict:
    """Closed forms of Section 6.3 for independent calls (gen, exe: positive floats per call)."""
    g = np.ascontiguousarray(gen, dtype=np.float64)
    e = np.ascontiguousarray(exe, dtype=np.float64)
    out = CLatency()
    order = np.zeros(max(len(g), 1), dtype=np.int32)
    _check(load().asynclm_latency_model(g.ctypes.data, e.ctypes.data, len(g), ctypes.byref(out), order.ctypes.data),
           "asynclm_latency_model")
    return {"l_sync": out.l_sync, "l_sync_par": out.l_sync_par, "l_async": out.l_async,
            "speedup_estimate": out.speedup_estimate, "lpt_order": order[:len(g)]}


def asynclm_async_latency_of_order(gen, exe, order):
    """(latency, completion time of every call) when the calls are generated in `order`."""
    g = np.ascontiguousarray(gen, dtype=np.float64)
    e = np.ascontiguousarray(exe, dtype=np.float64)
    o = np.ascontiguousarray(order, dtype=np.int32)
    lat = ctypes.c_double(0)
    done = np.zeros(max(len(g), 1), dtype=np.float64)
    _check(load().asynclm_async_latency_of_order(g.ctypes.data, e.ctypes.data, o.ctypes.data, len(g),
                                                 ctypes.byref(lat), done.ctypes.data),
           "asynclm_async_latency_of_order")
    return float(lat.value), done[:len(g)]


def asynclm_read_ceiling(kv_pool, k_block_offsets, v_delta_bytes: int, block_bytes: int, sink, stream=None) -> None:
    """Read-only ceiling probe: plain loads of the listed K/V block pairs (see include/asynclm.h)."""
    _check(load().asynclm_read_ceiling(kv_pool.data_ptr(), k_block_offsets.data_ptr(),
                                       int(k_block_offsets.numel()), int(v_delta_bytes), int(block_bytes),
                                       sink.data_ptr(), _stream_ptr(stream)), "asynclm_read_ceiling")


def asynclm_attn_mixed_static(plan: Plan, q, kv_pool, out, lse=None, stream=None) -> None:
    """asynclm_attn_mixed for callers that cannot hand the library scratch memory: split-KV
    partial results go to the fixed array inside the library (see include/asynclm.h)."""
    _check(load().asynclm_attn_mixed_static(plan.handle, q.data_ptr(), kv_pool.data_ptr(),
                                            out.data_ptr(), None if lse is None else lse.data_ptr(),
                                            _stream_ptr(stream)), "asynclm_attn_mixed_static")


def static_scratch_bytes() -> int:
    return int(load().asynclm_static_scratch_bytes())


def last_device_status(plan: Plan, stream=None) -> int:
    val = ctypes.c_int32(0)
    rc = load().asynclm_last_device_status(plan.handle, _stream_ptr(stream), ctypes.byref(val))
    if rc not in (0, -7):
        raise AsynclmError(rc, "asynclm_last_device_status")
    return int(val.value)
