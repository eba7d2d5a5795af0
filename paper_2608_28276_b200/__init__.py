"""Thin Python binding of libpask (include/pask.h): argument marshalling only.

Every step of the path runs inside the CUDA library; this module just turns torch tensors into
pointers and sizes. PyTorch is used for device memory and streams. There is no CPU fallback: if
libpask.so has not been built (python paper_2608_28276_b200/build.py) importing this package
fails.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpask.so")

OK = 0
ERR_INVALID_ARG, ERR_BAD_POLICY, ERR_UNSUPPORTED_SHAPE, ERR_POOL_EXHAUSTED = -1, -2, -3, -4
ERR_BAD_SEQ, ERR_CUDA, ERR_TIMEOUT, ERR_WORKSPACE, ERR_NO_MEMORY, ERR_STALE_PLAN = -5, -6, -7, -8, -9, -10
DEV_POOL_EXHAUSTED, DEV_BAD_SEQ, DEV_SEQ_OVERFLOW, DEV_BAD_RAGGED, DEV_TIMEOUT, DEV_RANGE, DEV_INTERNAL = 1, 2, 4, 8, 16, 32, 64
DEV_BAD_ACTION, DEV_STALE_PLAN = 128, 256
ACTION_RELEASE, ACTION_RETAIN_LOW, ACTION_RETAIN_HIGH = 0, 1, 2
TAG_PROTECTED = 0xFF
MAX_GROUPS = 8
MAX_WINDOW = 256

EXPORTS = [
    "pask_load_policy", "pask_free_policy", "pask_policy_action", "pask_cache_sizes", "pask_cache_create",
    "pask_cache_destroy", "pask_cache_reset", "pask_seq_reset", "pask_append_kv", "pask_decide",
    "pask_append_kv_decided", "pask_append_attend", "pask_plan_area_bytes", "pask_plan_ahead", "pask_decode_step_ahead", "pask_decode_attention",
    "pask_decode_attention_full", "pask_decode_attention_static", "pask_workspace_bytes", "pask_decode_step_host", "pask_step_staging_bytes", "pask_step_packed_layout", "pask_decode_step_packed", "pask_decode_step_pipelined", "pask_decode_step_pipelined_ahead", "pask_decode_step_drain",
    "pask_budget_state", "pask_distortion", "pask_cache_set_timing_events", "pask_cache_set_timing_span", "pask_debug_stream_len", "pask_debug_dump_high",
    "pask_debug_dump_low", "pask_debug_pool_state", "pask_debug_ctrl_words", "pask_debug_page_order", "pask_debug_page_ids", "pask_debug_partition", "pask_debug_set_attention_ctas", "pask_debug_set_wait", "pask_debug_plan_order_span", "pask_status_string",
]


class CacheDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("page_tokens", C.c_int32), ("max_seqs", C.c_int32),
                ("max_tokens_per_seq", C.c_int32), ("max_append_tokens", C.c_int32),
                ("pool_high_pages", C.c_uint32), ("pool_low_pages", C.c_uint32), ("recent_window", C.c_int32),
                ("low_bits", C.c_int32)]


class CacheSizes(C.Structure):
    _fields_ = [("pool_high_bytes", C.c_size_t), ("pool_low_bytes", C.c_size_t), ("meta_bytes", C.c_size_t),
                ("high_page_bytes", C.c_size_t), ("low_page_bytes", C.c_size_t)]


class BudgetState(C.Structure):
    _fields_ = [("n_seen", C.c_uint64 * MAX_GROUPS), ("n_high", C.c_uint64 * MAX_GROUPS),
                ("n_low", C.c_uint64 * MAX_GROUPS), ("n_drop", C.c_uint64 * MAX_GROUPS),
                ("retained_bytes", C.c_uint64), ("full_bytes", C.c_uint64), ("remaining_bytes", C.c_int64),
                ("bad_tags", C.c_uint64), ("pages_high", C.c_uint32), ("pages_low", C.c_uint32),
                ("device_status", C.c_uint32), ("reserved", C.c_uint32),
                ("decided_full_bytes", C.c_uint64), ("decided_retained_bytes", C.c_uint64),
                ("n_demoted", C.c_uint64), ("n_promoted", C.c_uint64), ("n_floor_conflicts", C.c_uint64)]


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python paper_2608_28276_b200/build.py` "
                      "(there is no fallback path)")
_lib = C.CDLL(LIB_PATH)

_vp, _i32, _sz = C.c_void_p, C.c_int32, C.c_size_t
_lib.pask_load_policy.argtypes = [C.c_char_p, _sz, C.POINTER(_vp)]
_lib.pask_free_policy.argtypes = [_vp]
_lib.pask_free_policy.restype = None
_lib.pask_policy_action.argtypes = [_vp, _i32, _i32]
_lib.pask_cache_sizes.argtypes = [C.POINTER(CacheDesc), C.POINTER(CacheSizes)]
_lib.pask_cache_create.argtypes = [C.POINTER(CacheDesc), _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]
_lib.pask_cache_destroy.argtypes = [_vp]
_lib.pask_cache_destroy.restype = None
_lib.pask_cache_reset.argtypes = [_vp, _vp]
_lib.pask_seq_reset.argtypes = [_vp, _i32, _vp]
_lib.pask_append_kv.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.pask_decide.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.pask_append_kv_decided.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.pask_append_attend.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.pask_decode_attention.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.pask_plan_area_bytes.argtypes = [_vp, _i32]
_lib.pask_plan_area_bytes.restype = _sz
_lib.pask_plan_ahead.argtypes = [_vp, _i32, _i32, _vp, _vp, _sz, _vp]
_lib.pask_decode_step_ahead.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]
_lib.pask_decode_attention_full.argtypes = _lib.pask_decode_attention.argtypes
_lib.pask_decode_attention_static.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.pask_workspace_bytes.argtypes = [_vp, _i32]
_lib.pask_workspace_bytes.restype = _sz
_lib.pask_decode_step_host.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]
_lib.pask_step_packed_layout.argtypes = [_vp, _i32, C.POINTER(_sz * 6), C.POINTER(_sz)]
_lib.pask_decode_step_packed.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _sz, _vp, _sz, _vp]
_lib.pask_decode_step_pipelined.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _sz, _vp, _sz, _vp]
_lib.pask_decode_step_pipelined_ahead.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _sz, _vp, _sz, _vp, _sz, _vp]
_lib.pask_decode_step_drain.argtypes = [_vp]
_lib.pask_step_staging_bytes.argtypes = [_vp, _i32]
_lib.pask_step_staging_bytes.restype = _sz
_lib.pask_distortion.argtypes = [_i32, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.pask_budget_state.argtypes = [_vp, _i32, C.POINTER(BudgetState), _vp]
_lib.pask_cache_set_timing_events.argtypes = [_vp, _vp, _vp]
_lib.pask_debug_stream_len.argtypes = [_vp, _i32, _i32, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), _vp]
_lib.pask_debug_dump_high.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp]
_lib.pask_debug_dump_low.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.pask_debug_pool_state.argtypes = [_vp, _vp, _vp]
_lib.pask_debug_page_ids.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp]
_lib.pask_debug_ctrl_words.argtypes = [_vp, _vp, _i32, _vp]
_lib.pask_debug_partition.argtypes = [_i32, _vp, _vp, _i32, _vp]
_lib.pask_debug_page_order.argtypes = [C.c_uint32, C.c_uint32, _vp]
_lib.pask_debug_set_attention_ctas.argtypes = [_vp, _i32]
_lib.pask_cache_set_timing_span.argtypes = [_vp, _vp]
_lib.pask_debug_set_wait.argtypes = [_vp, C.c_int64, C.c_uint32]
_lib.pask_debug_plan_order_span.argtypes = [_vp, _i32, _i32, _i32, C.POINTER(_sz), C.POINTER(_sz)]
_lib.pask_status_string.argtypes = [_i32]
_lib.pask_status_string.restype = C.c_char_p


class PaskError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {pask_status_string(status)} ({status})")


def _check(status: int, where: str):
    if status != OK:
        raise PaskError(status, where)


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _dptr(t, dtype=None):
    """Device pointer of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return t.data_ptr()


def pask_status_string(status: int) -> str:
    return _lib.pask_status_string(status).decode()


def pask_load_policy(blob: bytes) -> int:
    h = _vp()
    _check(_lib.pask_load_policy(blob, len(blob), C.byref(h)), "pask_load_policy")
    return h.value


def pask_free_policy(policy: int):
    _lib.pask_free_policy(policy)


def pask_policy_action(policy: int, tag: int, group: int) -> int:
    return int(_lib.pask_policy_action(policy, tag, group))


def pask_cache_sizes(desc: CacheDesc) -> CacheSizes:
    out = CacheSizes()
    _check(_lib.pask_cache_sizes(C.byref(desc), C.byref(out)), "pask_cache_sizes")
    return out


def pask_cache_create(desc: CacheDesc, policy: int, pool_high, pool_low, meta, stream=None) -> int:
    h = _vp()
    _check(_lib.pask_cache_create(C.byref(desc), policy, _dptr(pool_high), _dptr(pool_low), _dptr(meta),
                                  _stream(stream), C.byref(h)), "pask_cache_create")
    return h.value


def pask_cache_destroy(cache: int):
    _lib.pask_cache_destroy(cache)


def pask_cache_reset(cache: int, stream=None):
    _check(_lib.pask_cache_reset(cache, _stream(stream)), "pask_cache_reset")


def pask_seq_reset(cache: int, seq: int, stream=None):
    _check(_lib.pask_seq_reset(cache, seq, _stream(stream)), "pask_seq_reset")


def pask_append_kv(cache: int, layer: int, seq_ids, cu_tokens, k, v, tags, states=None, actions_out=None,
                   stream=None, total_tokens=None):
    n_seqs = seq_ids.numel()
    total = k.shape[0] if total_tokens is None else total_tokens
    _check(_lib.pask_append_kv(cache, layer, n_seqs, total, _dptr(seq_ids, torch.int32), _dptr(cu_tokens, torch.int32),
                               _dptr(k, torch.bfloat16), _dptr(v, torch.bfloat16), _dptr(tags, torch.uint8),
                               _dptr(states), _dptr(actions_out, torch.uint8), _stream(stream)), "pask_append_kv")


def pask_decide(cache: int, seq_ids, cu_tokens, tags, states, actions_out, stream=None):
    """Algorithm 2 steps 1-6 and 8: tags u8 [total], states u16/i16 [total] or None,
    actions_out u8 [total][n_groups]."""
    _check(_lib.pask_decide(cache, seq_ids.numel(), tags.numel(), _dptr(seq_ids, torch.int32),
                            _dptr(cu_tokens, torch.int32), _dptr(tags, torch.uint8), _dptr(states),
                            _dptr(actions_out, torch.uint8), _stream(stream)), "pask_decide")


def pask_append_kv_decided(cache: int, layer: int, seq_ids, cu_tokens, k, v, tags, actions, actions_out=None,
                           stream=None, total_tokens=None):
    n_seqs = seq_ids.numel()
    total = k.shape[0] if total_tokens is None else total_tokens
    _check(_lib.pask_append_kv_decided(cache, layer, n_seqs, total, _dptr(seq_ids, torch.int32),
                                       _dptr(cu_tokens, torch.int32), _dptr(k, torch.bfloat16),
                                       _dptr(v, torch.bfloat16), _dptr(tags, torch.uint8),
                                       _dptr(actions, torch.uint8), _dptr(actions_out, torch.uint8),
                                       _stream(stream)), "pask_append_kv_decided")


def pask_append_attend(cache: int, layer: int, seq_ids, cu_tokens, k, v, tags, q, out, lse, workspace, actions=None,
                       actions_out=None, stream=None, total_tokens=None):
    """One layer of a decode step: append (table actions, or `actions` from pask_decide) then attention."""
    total = k.shape[0] if total_tokens is None else total_tokens
    _check(_lib.pask_append_attend(cache, layer, seq_ids.numel(), total, _dptr(seq_ids, torch.int32),
                                   _dptr(cu_tokens, torch.int32), _dptr(k, torch.bfloat16), _dptr(v, torch.bfloat16),
                                   _dptr(tags, torch.uint8), _dptr(actions, torch.uint8), _dptr(actions_out, torch.uint8),
                                   _dptr(q, torch.bfloat16), _dptr(out, torch.float32), _dptr(lse, torch.float32),
                                   _dptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "pask_append_attend")


def pask_plan_area_bytes(cache: int, n_seqs: int) -> int:
    return int(_lib.pask_plan_area_bytes(cache, n_seqs))


def pask_plan_ahead(cache: int, layer: int, seq_ids, plan_area, stream=None):
    """Write the layer's decode-attention plan for this batch from the cache as it stands (see pask.h)."""
    _check(_lib.pask_plan_ahead(cache, layer, seq_ids.numel(), _dptr(seq_ids, torch.int32), _dptr(plan_area),
                                plan_area.numel() * plan_area.element_size(), _stream(stream)), "pask_plan_ahead")


def pask_decode_step_ahead(cache: int, layer: int, seq_ids, k, v, tags, q, out, lse, workspace, plan_area, actions=None,
                           actions_out=None, stream=None):
    """One layer of a decode step, one new token per sequence, from the plan made ahead: the streaming kernel starts at
    once, the append runs beside it and leaves the next step's plan, the merge attends the new token from k / v."""
    _check(_lib.pask_decode_step_ahead(cache, layer, seq_ids.numel(), _dptr(seq_ids, torch.int32), _dptr(k, torch.bfloat16),
                                       _dptr(v, torch.bfloat16), _dptr(tags, torch.uint8), _dptr(actions, torch.uint8),
                                       _dptr(actions_out, torch.uint8), _dptr(q, torch.bfloat16), _dptr(out, torch.float32),
                                       _dptr(lse, torch.float32), _dptr(workspace), workspace.numel() * workspace.element_size(),
                                       _dptr(plan_area), plan_area.numel() * plan_area.element_size(), _stream(stream)),
           "pask_decode_step_ahead")


def pask_workspace_bytes(cache: int, n_seqs: int) -> int:
    return int(_lib.pask_workspace_bytes(cache, n_seqs))


def _attention(fn, name, cache, layer, seq_ids, q, out, lse, workspace, stream):
    _check(fn(cache, layer, seq_ids.numel(), _dptr(seq_ids, torch.int32), _dptr(q, torch.bfloat16),
              _dptr(out, torch.float32), _dptr(lse, torch.float32), _dptr(workspace),
              workspace.numel() * workspace.element_size(), _stream(stream)), name)


def pask_decode_attention(cache: int, layer: int, seq_ids, q, out, lse, workspace, stream=None):
    _attention(_lib.pask_decode_attention, "pask_decode_attention", cache, layer, seq_ids, q, out, lse, workspace, stream)


def pask_decode_attention_full(cache: int, layer: int, seq_ids, q, out, lse, workspace, stream=None):
    _attention(_lib.pask_decode_attention_full, "pask_decode_attention_full", cache, layer, seq_ids, q, out, lse,
               workspace, stream)


STATIC_WORKSPACE_BYTES = 8 << 20


def pask_decode_attention_static(cache: int, layer: int, seq_ids, q, out, lse, stream=None):
    """pask_decode_attention without a workspace argument: the library's built-in scratch is used
    (for callers that cannot allocate one; see include/pask.h for the limits)."""
    _check(_lib.pask_decode_attention_static(cache, layer, seq_ids.numel(), _dptr(seq_ids, torch.int32),
                                             _dptr(q, torch.bfloat16), _dptr(out, torch.float32),
                                             _dptr(lse, torch.float32), _stream(stream)), "pask_decode_attention_static")


def pask_step_staging_bytes(cache: int, n_seqs: int) -> int:
    return int(_lib.pask_step_staging_bytes(cache, n_seqs))


def pask_decode_step_host(cache: int, layer: int, seq_ids_host, k_host, v_host, tags_host, q_host, out_host, staging,
                          workspace, stream=None):
    """All *_host arguments are CPU tensors (pinned for real asynchrony); staging / workspace CUDA."""
    for t in (seq_ids_host, k_host, v_host, tags_host, q_host, out_host):
        assert not t.is_cuda and t.is_contiguous()
    _check(_lib.pask_decode_step_host(cache, layer, seq_ids_host.numel(), seq_ids_host.data_ptr(), k_host.data_ptr(),
                                      v_host.data_ptr(), tags_host.data_ptr(), q_host.data_ptr(), out_host.data_ptr(),
                                      _dptr(staging), staging.numel() * staging.element_size(), _dptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream(stream)),
           "pask_decode_step_host")


def pask_distortion(o_ref, o_test, per_row_out=None, sum_inout=None, stream=None):
    """Eq. 4's inner term: per row max over heads of the squared distance of two attention outputs
    [rows][n_q][128] fp32; per_row_out fp32 [rows] and / or sum_inout fp64 [1] (added to)."""
    assert o_ref.shape == o_test.shape and o_ref.shape[-1] == 128
    _check(_lib.pask_distortion(o_ref.shape[0], o_ref.shape[1], _dptr(o_ref, torch.float32), _dptr(o_test, torch.float32),
                                _dptr(per_row_out, torch.float32), _dptr(sum_inout, torch.float64), _stream(stream)),
           "pask_distortion")


def pask_step_packed_layout(cache: int, n_seqs: int):
    """(offsets of seq_ids, cu_tokens, k, v, tags, q in the packed host block; its size in bytes)."""
    off, n = (_sz * 6)(), _sz(0)
    _check(_lib.pask_step_packed_layout(cache, n_seqs, C.byref(off), C.byref(n)), "pask_step_packed_layout")
    return [int(x) for x in off], int(n.value)


def pask_decode_step_packed(cache: int, layer: int, n_seqs: int, packed_host, out_host, staging, workspace, stream=None):
    """packed_host: CPU uint8 tensor (pinned) laid out per pask_step_packed_layout; out_host CPU fp32."""
    assert not packed_host.is_cuda and packed_host.is_contiguous() and not out_host.is_cuda and out_host.is_contiguous()
    _check(_lib.pask_decode_step_packed(cache, layer, n_seqs, packed_host.data_ptr(), out_host.data_ptr(), _dptr(staging),
                                        staging.numel() * staging.element_size(), _dptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)),
           "pask_decode_step_packed")


def pask_decode_step_pipelined(cache: int, layer: int, n_seqs: int, packed_host, out_host, staging, workspace, stream=None):
    """pask_decode_step_packed with the copies on the cache's own copy streams (staging: two slots).
    out_host is valid only after pask_decode_step_drain."""
    assert not packed_host.is_cuda and packed_host.is_contiguous() and not out_host.is_cuda and out_host.is_contiguous()
    _check(_lib.pask_decode_step_pipelined(cache, layer, n_seqs, packed_host.data_ptr(), out_host.data_ptr(), _dptr(staging),
                                           staging.numel() * staging.element_size(), _dptr(workspace),
                                           workspace.numel() * workspace.element_size(), _stream(stream)),
           "pask_decode_step_pipelined")


def pask_decode_step_pipelined_ahead(cache: int, layer: int, n_seqs: int, packed_host, out_host, staging, workspace, plan_area,
                                     stream=None):
    """pask_decode_step_pipelined with the layer's step issued as pask_decode_step_ahead."""
    assert not packed_host.is_cuda and packed_host.is_contiguous() and not out_host.is_cuda and out_host.is_contiguous()
    _check(_lib.pask_decode_step_pipelined_ahead(cache, layer, n_seqs, packed_host.data_ptr(), out_host.data_ptr(), _dptr(staging),
                                                 staging.numel() * staging.element_size(), _dptr(workspace),
                                                 workspace.numel() * workspace.element_size(), _dptr(plan_area),
                                                 plan_area.numel() * plan_area.element_size(), _stream(stream)),
           "pask_decode_step_pipelined_ahead")


def pask_decode_step_drain(cache: int):
    _check(_lib.pask_decode_step_drain(cache), "pask_decode_step_drain")


def pask_budget_state(cache: int, seq: int, stream=None) -> BudgetState:
    out = BudgetState()
    _check(_lib.pask_budget_state(cache, seq, C.byref(out), _stream(stream)), "pask_budget_state")
    return out


def pask_cache_set_timing_events(cache: int, start, stop):
    """start / stop: torch.cuda.Event(enable_timing=True) that have been recorded at least once
    (so that their CUDA handles exist), or None."""
    a = None if start is None else start.cuda_event
    b = None if stop is None else stop.cuda_event
    _check(_lib.pask_cache_set_timing_events(cache, a, b), "pask_cache_set_timing_events")


def pask_debug_stream_len(cache: int, layer: int, seq: int, stream=None):
    a, b = C.c_uint32(0), C.c_uint32(0)
    _check(_lib.pask_debug_stream_len(cache, layer, seq, C.byref(a), C.byref(b), _stream(stream)), "pask_debug_stream_len")
    return a.value, b.value


def pask_debug_dump_high(cache: int, layer: int, seq: int, n_kv: int, stream=None):
    import numpy as np
    nh, _ = pask_debug_stream_len(cache, layer, seq, stream)
    k = np.zeros((nh, n_kv, 128), np.uint16)
    v = np.zeros_like(k)
    pages = np.zeros((nh + 15) // 16, np.uint32)
    _check(_lib.pask_debug_dump_high(cache, layer, seq, k.ctypes.data, v.ctypes.data, pages.ctypes.data, _stream(stream)),
           "pask_debug_dump_high")
    return k, v, pages


def pask_debug_dump_low(cache: int, layer: int, seq: int, n_kv: int, stream=None):
    import numpy as np
    _, nl = pask_debug_stream_len(cache, layer, seq, stream)
    kc = np.zeros((nl, n_kv, 128), np.uint8)
    vc = np.zeros_like(kc)
    ks = np.zeros((nl, n_kv, 4), np.uint16)
    vs = np.zeros_like(ks)
    pages = np.zeros((nl + 15) // 16, np.uint32)
    _check(_lib.pask_debug_dump_low(cache, layer, seq, kc.ctypes.data, ks.ctypes.data, vc.ctypes.data, vs.ctypes.data,
                                    pages.ctypes.data, _stream(stream)), "pask_debug_dump_low")
    return kc, ks, vc, vs, pages


def pask_debug_page_ids(cache: int, layer: int, seq: int, stream=None):
    import numpy as np
    nh, nl = pask_debug_stream_len(cache, layer, seq, stream)
    hi, lo = np.zeros((nh + 15) // 16, np.uint32), np.zeros((nl + 15) // 16, np.uint32)
    _check(_lib.pask_debug_page_ids(cache, layer, seq, hi.ctypes.data, lo.ctypes.data, _stream(stream)), "pask_debug_page_ids")
    return hi, lo


def pask_debug_pool_state(cache: int, stream=None):
    import numpy as np
    out = np.zeros(4, np.uint32)
    _check(_lib.pask_debug_pool_state(cache, out.ctypes.data, _stream(stream)), "pask_debug_pool_state")
    return tuple(int(x) for x in out)


def pask_debug_ctrl_words(cache: int, count: int = 64, stream=None):
    import numpy as np
    out = np.zeros(count, np.uint32)
    _check(_lib.pask_debug_ctrl_words(cache, out.ctypes.data, count, _stream(stream)), "pask_debug_ctrl_words")
    return out


def pask_debug_partition(pages_high, pages_low, n_ctas: int):
    """Host-only: ranges [n_ctas][n_seqs][2] of positions in each sequence's page order that the
    CTAs of the decode-attention grid would process."""
    import numpy as np
    ph = np.ascontiguousarray(pages_high, dtype=np.uint32)
    pl = np.ascontiguousarray(pages_low, dtype=np.uint32)
    out = np.zeros((n_ctas, len(ph), 2), np.uint32)
    _check(_lib.pask_debug_partition(len(ph), ph.ctypes.data, pl.ctypes.data, n_ctas, out.ctypes.data),
           "pask_debug_partition")
    return out


def pask_debug_page_order(pages_high: int, pages_low: int):
    """Host-only: the order a sequence's pages are visited in: (is_high bool array, page index array)."""
    import numpy as np
    out = np.zeros(pages_high + pages_low, np.uint32)
    _check(_lib.pask_debug_page_order(pages_high, pages_low, out.ctypes.data), "pask_debug_page_order")
    return (out >> 31).astype(bool), (out & 0x7FFFFFFF).astype(np.int64)


def pask_cache_set_timing_span(cache: int, span):
    """span: int64 device tensor [2] preset to (-1, 0) (all ones, zero), or None: the next streaming kernel leaves its
    earliest CTA start and latest CTA end there (GPU global timer, ns)."""
    _check(_lib.pask_cache_set_timing_span(cache, None if span is None else span.data_ptr()), "pask_cache_set_timing_span")


def pask_debug_set_attention_ctas(cache: int, n_ctas: int):
    _check(_lib.pask_debug_set_attention_ctas(cache, n_ctas), "pask_debug_set_attention_ctas")


def pask_debug_plan_order_span(cache: int, n_seqs: int, layer: int, parity: int):
    """(byte offset, byte length) of the page-order list of (layer, parity) inside a plan area for n_seqs sequences."""
    off, n = _sz(0), _sz(0)
    _check(_lib.pask_debug_plan_order_span(cache, n_seqs, layer, parity, C.byref(off), C.byref(n)), "pask_debug_plan_order_span")
    return int(off.value), int(n.value)


def pask_debug_set_wait(cache: int, limit_cycles: int = 2_000_000_000, surplus_bytes: int = 0):
    """Bound of the decode-attention kernel's waits for its bulk copies, and the test aid that makes one run out."""
    _check(_lib.pask_debug_set_wait(cache, limit_cycles, surplus_bytes), "pask_debug_set_wait")


class Cache:
    """Convenience owner of the device buffers a cache needs (torch allocations) plus its handle."""

    def __init__(self, blob: bytes, n_layers, n_q, n_kv, max_seqs, max_tokens_per_seq, max_append_tokens,
                 pool_high_pages, pool_low_pages, device="cuda", recent_window=0, low_bits=4):
        self.policy = pask_load_policy(blob)
        self.desc = CacheDesc(n_layers, n_q, n_kv, 128, 16, max_seqs, max_tokens_per_seq, max_append_tokens,
                              pool_high_pages, pool_low_pages, recent_window, low_bits)
        self.sizes = pask_cache_sizes(self.desc)
        self.n_q, self.n_kv, self.n_layers = n_q, n_kv, n_layers
        self.pool_high = torch.empty(max(256, self.sizes.pool_high_bytes), dtype=torch.uint8, device=device)
        self.pool_low = torch.empty(max(256, self.sizes.pool_low_bytes), dtype=torch.uint8, device=device)
        self.meta = torch.empty(self.sizes.meta_bytes, dtype=torch.uint8, device=device)
        self.handle = pask_cache_create(self.desc, self.policy, self.pool_high, self.pool_low, self.meta)
        self._ws = None

    def workspace(self, n_seqs: int):
        need = pask_workspace_bytes(self.handle, n_seqs)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.meta.device)
        return self._ws

    def close(self):
        if getattr(self, "handle", None):
            pask_cache_destroy(self.handle)
            self.handle = None
        if getattr(self, "policy", None):
            pask_free_policy(self.policy)
            self.policy = None

    def __del__(self):
        try:
            self.close()
        except Exception:       # interpreter shutdown: the module's globals may already be gone
            pass
