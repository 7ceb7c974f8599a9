"""ctypes binding of libcompact_attn: argument marshalling only.

Every function has the name and argument order of its C entry point in
``include/compact_attn.h``; device buffers are passed as torch tensors (their
``data_ptr()`` is taken) or as raw integer addresses.  There is no fallback:
if the shared library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
# CPA_LIB_PATH points at another build of the library (same ABI), e.g. one made with other compile-time options
LIB_PATH = os.environ.get("CPA_LIB_PATH") or os.path.join(_PKG, "libcompact_attn.so")

CPA_OK, CPA_EINVAL, CPA_ENOSPC, CPA_EUNSUPPORTED, CPA_ECUDA, CPA_ETIMEOUT, CPA_ESTATE = 0, -1, -2, -3, -4, -5, -6

ARR_CU_SEQLENS, ARR_PAGE_INDPTR, ARR_PAGE_INDICES, ARR_SEQ_LENS = 0, 1, 2, 3
ARR_SLOT_MAPPING, ARR_PREFILL_ITEMS, ARR_DECODE_ITEMS, ARR_SPLIT_INDPTR = 4, 5, 6, 7
ARR_SPLIT_PAGES = 8
ARR_PREFILL_SCHED = 9
ARR_DEC_START, ARR_CHUNK_ROWS = 10, 11
ARR_PAGES_ASSIGNED, ARR_FREE_RING = 12, 13
ARR_SPLIT_RANGES = 14
_ARR_WIDTH = {ARR_PREFILL_ITEMS: 2, ARR_DECODE_ITEMS: 3, 14: 2}

PARAM_NUM_BLOCKS, PARAM_TOTAL_TOKENS, PARAM_Q_TILE_ROWS, PARAM_PAGES_PER_SPLIT = 0, 1, 2, 3
PARAM_PAGES_USED, PARAM_INDEX_BYTES, PARAM_DECODE_WORKSPACE_BYTES, PARAM_TOTAL_SPLITS = 4, 5, 6, 7
PARAM_MAX_NEW_TOKENS = 8
PARAM_PREFILL_CTAS = 9
PARAM_SHARED_CHUNK_PAGES = 10
PARAM_CHUNK_TOKENS, PARAM_NUM_STEPS, PARAM_CHUNK_STEPS, PARAM_DECODE_SMS, PARAM_NUM_SMS = 11, 12, 13, 14, 15
PARAM_DECODE_STEPS_PER_CHUNK = 16
PARAM_DECODE_EVEN_CUT, PARAM_DECODE_CTAS, PARAM_HOST_STAGE_BYTES = 17, 18, 19


class cpa_config(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("scale", ctypes.c_float), ("q_tile_rows", ctypes.c_int32),
                ("pages_per_split", ctypes.c_int32), ("num_sms", ctypes.c_int32)]


class CpaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {cpa_strerror(status)} ({status})")


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2605_23296_b200.build` "
        "(there is no fallback implementation)")
_lib = ctypes.CDLL(LIB_PATH)

_vp, _i32p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)
_lib.cpa_plan_create.argtypes = [ctypes.POINTER(cpa_config), ctypes.c_int32, _i32p, ctypes.c_int32,
                                 _i32p, ctypes.c_int32, ctypes.POINTER(_vp)]
_lib.cpa_plan_create.restype = ctypes.c_int
_lib.cpa_plan_create_prefix.argtypes = [ctypes.POINTER(cpa_config), ctypes.c_int32, _i32p, _i32p, _i32p, ctypes.c_int32,
                                        ctypes.c_int32, _i32p, ctypes.c_int32, ctypes.POINTER(_vp)]
_lib.cpa_plan_create_prefix.restype = ctypes.c_int
_lib.cpa_plan_create_chunked.argtypes = [ctypes.POINTER(cpa_config), ctypes.c_int32, _i32p, ctypes.c_int32, ctypes.c_int32,
                                         ctypes.c_int32, ctypes.c_int32, _i32p, ctypes.c_int32, ctypes.POINTER(_vp)]
_lib.cpa_plan_create_chunked.restype = ctypes.c_int
_lib.cpa_plan_create_prefix_chunked.argtypes = [ctypes.POINTER(cpa_config), ctypes.c_int32, _i32p, _i32p, _i32p,
                                                ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                                ctypes.c_int32, _i32p, ctypes.c_int32, ctypes.POINTER(_vp)]
_lib.cpa_plan_create_prefix_chunked.restype = ctypes.c_int
_lib.cpa_plan_create_dynamic.argtypes = [ctypes.POINTER(cpa_config), ctypes.c_int32, _i32p, ctypes.c_int32, _i32p,
                                         ctypes.c_int32, ctypes.POINTER(_vp)]
_lib.cpa_plan_create_dynamic.restype = ctypes.c_int
_lib.cpa_plan_sync.argtypes = [_vp, _vp]
_lib.cpa_plan_sync.restype = ctypes.c_int
_lib.cpa_decode_append_dynamic.argtypes = [_vp] * 10
_lib.cpa_decode_append_dynamic.restype = ctypes.c_int
_lib.cpa_release_blocks.argtypes = [_vp, _vp, _vp]
_lib.cpa_release_blocks.restype = ctypes.c_int
_lib.cpa_step_mixed.argtypes = [_vp, ctypes.c_int32] + [_vp] * 12
_lib.cpa_step_mixed.restype = ctypes.c_int
_lib.cpa_event_host.argtypes = [_vp] * 14
_lib.cpa_step_mixed_range.argtypes = [_vp, ctypes.c_int32, ctypes.c_int32] + [_vp] * 12
_lib.cpa_step_mixed_range.restype = ctypes.c_int
_lib.cpa_decode_append_steps.argtypes = [_vp] * 8 + [ctypes.c_int32, _vp]
_lib.cpa_decode_append_steps.restype = ctypes.c_int
_lib.cpa_partition.argtypes = [ctypes.c_int64, ctypes.c_int32, _i32p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)]
_lib.cpa_partition.restype = ctypes.c_int
_lib.cpa_event_host.restype = ctypes.c_int
_lib.cpa_plan_export.argtypes = [_vp, ctypes.c_int, ctypes.POINTER(_i32p), ctypes.POINTER(ctypes.c_int64)]
_lib.cpa_plan_export.restype = ctypes.c_int
_lib.cpa_plan_param.argtypes = [_vp, ctypes.c_int]
_lib.cpa_plan_param.restype = ctypes.c_int64
_lib.cpa_plan_upload.argtypes = [_vp, _vp, ctypes.c_int64, _vp]
_lib.cpa_plan_upload.restype = ctypes.c_int
_lib.cpa_plan_status.argtypes = [_vp, _vp]
_lib.cpa_plan_status.restype = ctypes.c_int
_lib.cpa_plan_destroy.argtypes = [_vp]
_lib.cpa_plan_destroy.restype = None
_lib.cpa_prefill.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.cpa_prefill.restype = ctypes.c_int
_lib.cpa_prefill_prefix.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.cpa_prefill_prefix.restype = ctypes.c_int
_lib.cpa_prefill_variant.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_int]
_lib.cpa_prefill_variant.restype = ctypes.c_int
_lib.cpa_kv_append.argtypes = [_vp, _vp, _vp, _i32p, _vp, _vp, _vp]
_lib.cpa_kv_append.restype = ctypes.c_int
_lib.cpa_decode.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.cpa_decode.restype = ctypes.c_int
_lib.cpa_decode_append.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.cpa_decode_append.restype = ctypes.c_int
_lib.cpa_decode_static.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp]
_lib.cpa_decode_static.restype = ctypes.c_int
_lib.cpa_strerror.argtypes = [ctypes.c_int]
_lib.cpa_strerror.restype = ctypes.c_char_p


def _ptr(x) -> Optional[int]:
    """Device/host address of a tensor-like, or the integer itself."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return int(x.data_ptr())


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def cpa_strerror(status: int) -> str:
    return _lib.cpa_strerror(int(status)).decode()


def cpa_plan_create(cfg: cpa_config, block_lens: Sequence[int], max_new_tokens: int,
                    free_pages: Sequence[int], check: bool = True):
    """Returns the plan handle (int); raises CpaError unless check=False, then (status, handle)."""
    lens, free = _i32(block_lens), _i32(free_pages)
    out = _vp()
    rc = _lib.cpa_plan_create(ctypes.byref(cfg), lens.shape[0], lens.ctypes.data_as(_i32p),
                              int(max_new_tokens), free.ctypes.data_as(_i32p), free.shape[0],
                              ctypes.byref(out))
    if not check:
        return rc, out.value
    if rc != CPA_OK:
        raise CpaError(rc, "cpa_plan_create")
    return out.value


def cpa_partition(history_tokens: int, block_tokens: int, capacity: int = 1 << 16, check: bool = True):
    """Block lengths of a history cut into blocks of `block_tokens` (the last one may be short)."""
    lens = np.zeros(max(capacity, 1), dtype=np.int32)
    n = ctypes.c_int32(0)
    rc = _lib.cpa_partition(int(history_tokens), int(block_tokens), lens.ctypes.data_as(_i32p), int(capacity),
                            ctypes.byref(n))
    if not check:
        return rc, n.value
    if rc != CPA_OK:
        raise CpaError(rc, "cpa_partition")
    return lens[:n.value].copy()


def cpa_plan_create_prefix(cfg: cpa_config, own_lens: Sequence[int], prefix_lens: Sequence[int],
                           shared_pages: Sequence[int], max_new_tokens: int, free_pages: Sequence[int],
                           check: bool = True):
    """Plan of the prefix-aware layout; returns the handle, or (status, handle) with check=False."""
    lens, pre, shared, free = _i32(own_lens), _i32(prefix_lens), _i32(shared_pages), _i32(free_pages)
    out = _vp()
    rc = _lib.cpa_plan_create_prefix(ctypes.byref(cfg), lens.shape[0], lens.ctypes.data_as(_i32p),
                                     pre.ctypes.data_as(_i32p), shared.ctypes.data_as(_i32p), shared.shape[0],
                                     int(max_new_tokens), free.ctypes.data_as(_i32p), free.shape[0],
                                     ctypes.byref(out))
    if not check:
        return rc, out.value
    if rc != CPA_OK:
        raise CpaError(rc, "cpa_plan_create_prefix")
    return out.value


def cpa_plan_create_chunked(cfg: cpa_config, block_lens: Sequence[int], max_new_tokens: int, chunk_tokens: int,
                            free_pages: Sequence[int], decode_sms: int = 0, decode_steps_per_chunk: int = 1,
                            check: bool = True):
    """Plan of an event with chunked prefill; returns the handle, or (status, handle) with check=False."""
    lens, free = _i32(block_lens), _i32(free_pages)
    out = _vp()
    rc = _lib.cpa_plan_create_chunked(ctypes.byref(cfg), lens.shape[0], lens.ctypes.data_as(_i32p), int(max_new_tokens),
                                      int(chunk_tokens), int(decode_steps_per_chunk), int(decode_sms),
                                      free.ctypes.data_as(_i32p), free.shape[0],
                                      ctypes.byref(out))
    if not check:
        return rc, out.value
    if rc != CPA_OK:
        raise CpaError(rc, "cpa_plan_create_chunked")
    return out.value


def cpa_plan_create_prefix_chunked(cfg: cpa_config, own_lens: Sequence[int], prefix_lens: Sequence[int],
                                   shared_pages: Sequence[int], max_new_tokens: int, chunk_tokens: int,
                                   free_pages: Sequence[int], decode_sms: int = 0, decode_steps_per_chunk: int = 1,
                                   check: bool = True):
    """Plan of the prefix-aware layout with chunked prefill; the handle, or (status, handle) with check=False."""
    lens, pre, shared, free = _i32(own_lens), _i32(prefix_lens), _i32(shared_pages), _i32(free_pages)
    out = _vp()
    rc = _lib.cpa_plan_create_prefix_chunked(ctypes.byref(cfg), lens.shape[0], lens.ctypes.data_as(_i32p),
                                             pre.ctypes.data_as(_i32p), shared.ctypes.data_as(_i32p), shared.shape[0],
                                             int(max_new_tokens), int(chunk_tokens), int(decode_steps_per_chunk),
                                             int(decode_sms), free.ctypes.data_as(_i32p), free.shape[0],
                                             ctypes.byref(out))
    if not check:
        return rc, out.value
    if rc != CPA_OK:
        raise CpaError(rc, "cpa_plan_create_prefix_chunked")
    return out.value


def cpa_plan_create_dynamic(cfg: cpa_config, block_lens: Sequence[int], max_new_tokens: int,
                            free_pages: Sequence[int], check: bool = True):
    """Plan with pages on demand; returns the handle, or (status, handle) with check=False."""
    lens, free = _i32(block_lens), _i32(free_pages)
    out = _vp()
    rc = _lib.cpa_plan_create_dynamic(ctypes.byref(cfg), lens.shape[0], lens.ctypes.data_as(_i32p), int(max_new_tokens),
                                      free.ctypes.data_as(_i32p), free.shape[0], ctypes.byref(out))
    if not check:
        return rc, out.value
    if rc != CPA_OK:
        raise CpaError(rc, "cpa_plan_create_dynamic")
    return out.value


def cpa_plan_sync(plan: int, stream: int = 0) -> int:
    return _lib.cpa_plan_sync(plan, stream or None)


def cpa_decode_append_dynamic(plan: int, q, k_new, v_new, d_active, k_pool, v_pool, o, d_workspace, stream: int = 0) -> int:
    return _lib.cpa_decode_append_dynamic(plan, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(d_active), _ptr(k_pool),
                                          _ptr(v_pool), _ptr(o), _ptr(d_workspace), stream or None)


def cpa_release_blocks(plan: int, d_active, stream: int = 0) -> int:
    return _lib.cpa_release_blocks(plan, _ptr(d_active), stream or None)


def cpa_plan_export(plan: int, which: int) -> np.ndarray:
    """Copy of one host index array; item lists come back as [n, width]."""
    ptr, n = _i32p(), ctypes.c_int64()
    rc = _lib.cpa_plan_export(plan, which, ctypes.byref(ptr), ctypes.byref(n))
    if rc != CPA_OK:
        raise CpaError(rc, "cpa_plan_export")
    w = _ARR_WIDTH.get(which, 1)
    if n.value == 0:
        return np.zeros((0, w) if w > 1 else (0,), dtype=np.int32)
    a = np.ctypeslib.as_array(ptr, shape=(n.value * w,)).copy()
    return a.reshape(n.value, w) if w > 1 else a


def cpa_plan_param(plan: int, which: int) -> int:
    return int(_lib.cpa_plan_param(plan, which))


def cpa_plan_upload(plan: int, d_index_buf, nbytes: int, stream: int = 0) -> int:
    return _lib.cpa_plan_upload(plan, _ptr(d_index_buf), int(nbytes), stream or None)


def cpa_plan_status(plan: int, stream: int = 0) -> int:
    return _lib.cpa_plan_status(plan, stream or None)


def cpa_plan_destroy(plan: int) -> None:
    _lib.cpa_plan_destroy(plan)


def cpa_prefill(plan: int, q, k, v, o, d_workspace=None, stream: int = 0) -> int:
    return _lib.cpa_prefill(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_workspace), stream or None)


PREFILL_TENSOR_CORE, PREFILL_WARP_MMA = 0, 1


def cpa_prefill_prefix(plan: int, q, k, v, k_pool, v_pool, o, stream: int = 0) -> int:
    return _lib.cpa_prefill_prefix(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(k_pool), _ptr(v_pool), _ptr(o), stream)


def cpa_prefill_variant(plan: int, q, k, v, o, stream: int = 0, variant: int = 0) -> int:
    return _lib.cpa_prefill_variant(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(o), stream or None, int(variant))


def cpa_kv_append(plan: int, k_new, v_new, new_lens, k_pool, v_pool, stream: int = 0) -> int:
    if new_lens is None:
        lens_p = None
    else:
        lens = _i32(new_lens)
        lens_p = lens.ctypes.data_as(_i32p)
    return _lib.cpa_kv_append(plan, _ptr(k_new), _ptr(v_new), lens_p, _ptr(k_pool), _ptr(v_pool),
                              stream or None)


def cpa_decode(plan: int, q, k_pool, v_pool, o, d_workspace, stream: int = 0) -> int:
    return _lib.cpa_decode(plan, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(o), _ptr(d_workspace),
                           stream or None)


def cpa_decode_append(plan: int, q, k_new, v_new, k_pool, v_pool, o, d_workspace, stream: int = 0) -> int:
    return _lib.cpa_decode_append(plan, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(o),
                                  _ptr(d_workspace), stream or None)


def cpa_step_mixed(plan: int, step: int, q, k, v, o, q_dec, k_new, v_new, o_dec, k_pool, v_pool, d_workspace,
                   stream: int = 0) -> int:
    return _lib.cpa_step_mixed(plan, int(step), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(q_dec), _ptr(k_new),
                               _ptr(v_new), _ptr(o_dec), _ptr(k_pool), _ptr(v_pool), _ptr(d_workspace), stream or None)


def cpa_decode_append_steps(plan: int, q, k_new, v_new, k_pool, v_pool, o, d_workspace, num_steps: int,
                            stream: int = 0) -> int:
    return _lib.cpa_decode_append_steps(plan, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(o),
                                        _ptr(d_workspace), int(num_steps), stream or None)


def cpa_event_host(plan: int, h_q, h_k, h_v, h_o, h_q_dec, h_k_dec, h_v_dec, h_o_dec, d_stage, k_pool, v_pool,
                   d_workspace, stream: int = 0) -> int:
    """A whole event from host tensors (page-locked for overlap); the results are in place after a stream sync."""
    return _lib.cpa_event_host(plan, _ptr(h_q), _ptr(h_k), _ptr(h_v), _ptr(h_o), _ptr(h_q_dec), _ptr(h_k_dec),
                               _ptr(h_v_dec), _ptr(h_o_dec), _ptr(d_stage), _ptr(k_pool), _ptr(v_pool),
                               _ptr(d_workspace), stream or None)


def cpa_step_mixed_range(plan: int, first_step: int, num_steps: int, q, k, v, o, q_dec, k_new, v_new, o_dec, k_pool,
                         v_pool, d_workspace, stream: int = 0) -> int:
    return _lib.cpa_step_mixed_range(plan, int(first_step), int(num_steps), _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                     _ptr(q_dec), _ptr(k_new), _ptr(v_new), _ptr(o_dec), _ptr(k_pool), _ptr(v_pool),
                                     _ptr(d_workspace), stream or None)


STATIC_SCRATCH_BYTES = 16 << 20


def cpa_decode_static(plan: int, q, k_pool, v_pool, o, stream: int = 0) -> int:
    """cpa_decode with the split partials in the library's own fixed 16 MiB device array.

    For callers that cannot allocate or pass scratch memory (a plugin behind a framework
    that hands out fixed buffers, a service with a fully budgeted device).  Returns
    CPA_ENOSPC if the plan needs more than STATIC_SCRATCH_BYTES.  Calls that overlap on
    the device race on the shared array; the first call per device should happen outside
    stream capture.
    """
    return _lib.cpa_decode_static(plan, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(o), stream or None)
