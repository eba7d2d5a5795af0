"""ctypes view of the CPU oracle (oracle/pask_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package. It never
imports the CUDA package and the CUDA package never imports it.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from .build import build as _build

OK, ERR_ARG, ERR_POLICY, ERR_POOL, ERR_SEQ = 0, -1, -2, -4, -5
MAX_GROUPS = 8


class Budget(C.Structure):
    _fields_ = [("n_seen", C.c_uint64 * MAX_GROUPS), ("n_high", C.c_uint64 * MAX_GROUPS),
                ("n_low", C.c_uint64 * MAX_GROUPS), ("n_drop", C.c_uint64 * MAX_GROUPS),
                ("retained_bytes", C.c_uint64), ("full_bytes", C.c_uint64),
                ("remaining_bytes", C.c_int64), ("bad_tags", C.c_uint64),
                ("pages_high", C.c_uint32), ("pages_low", C.c_uint32),
                ("decided_full_bytes", C.c_uint64), ("decided_retained_bytes", C.c_uint64),
                ("n_demoted", C.c_uint64), ("n_promoted", C.c_uint64), ("n_floor_conflicts", C.c_uint64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        vp, i32, u32 = C.c_void_p, C.c_int, C.c_uint32
        L.orc_f32_to_f16_rne.restype = C.c_uint16
        L.orc_f32_to_f16_rne.argtypes = [C.c_float]
        L.orc_f16_to_f32.restype = C.c_float
        L.orc_f16_to_f32.argtypes = [C.c_uint16]
        L.orc_quantize_group.argtypes = [vp, vp, vp]
        L.orc_quantize_group.restype = None
        L.orc_quantize_group_bits.argtypes = [vp, vp, vp, i32]
        L.orc_quantize_group_bits.restype = None
        L.orc_lut_fold.argtypes = [i32, i32]
        L.orc_policy_load.restype = vp
        L.orc_policy_load.argtypes = [C.c_char_p, C.c_size_t, C.POINTER(C.c_int)]
        L.orc_policy_free.argtypes = [vp]
        L.orc_policy_free.restype = None
        L.orc_policy_action.argtypes = [vp, i32, i32]
        L.orc_cache_create.restype = vp
        L.orc_cache_create.argtypes = [vp, i32, i32, i32, u32, u32]
        L.orc_cache_destroy.argtypes = [vp]
        L.orc_cache_destroy.restype = None
        L.orc_seq_reset.argtypes = [vp, i32]
        L.orc_append.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
        L.orc_append_decided.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.orc_decide.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        L.orc_stream_len.argtypes = [vp, i32, i32, C.POINTER(u32), C.POINTER(u32)]
        L.orc_dump_high.argtypes = [vp, i32, i32, vp, vp, vp]
        L.orc_dump_low.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
        L.orc_budget_state.argtypes = [vp, i32, C.POINTER(Budget)]
        L.orc_pool_state.argtypes = [vp] + [C.POINTER(u32)] * 4
        L.orc_pool_state.restype = None
        L.orc_attention.argtypes = [vp, i32, i32, vp, vp, vp]
        L.orc_attention_batch.argtypes = [vp, i32, i32, vp, vp, vp, vp]
        L.orc_distortion.restype = C.c_double
        L.orc_distortion.argtypes = [i32, i32, vp, vp, vp]
        assert L.orc_sizeof_budget() == C.sizeof(Budget)
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def f32_to_f16_bits(x: float) -> int:
    return int(lib().orc_f32_to_f16_rne(C.c_float(x)))


def f16_bits_to_f32(h: int) -> float:
    return float(lib().orc_f16_to_f32(C.c_uint16(h)))


def quantize_group(x_bits: np.ndarray, bits: int = 4):
    """32 bf16 bit patterns -> (fp16 scale bit pattern, 32 codes); bits = 2, 4 or 8."""
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    assert x.shape == (32,)
    s = np.zeros(1, np.uint16)
    c = np.zeros(32, np.uint8)
    lib().orc_quantize_group_bits(_ptr(x), _ptr(s), _ptr(c), bits)
    return int(s[0]), c


def lut_fold(a0: int, a_floor: int) -> int:
    return int(lib().orc_lut_fold(a0, a_floor))


class Policy:
    def __init__(self, blob: bytes):
        err = C.c_int(0)
        self.h = lib().orc_policy_load(blob, len(blob), C.byref(err))
        self.err = err.value
        if not self.h:
            raise ValueError(f"oracle rejected the policy blob ({self.err})")

    def action(self, tag: int, group: int) -> int:
        return int(lib().orc_policy_action(self.h, tag, group))

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_policy_free(self.h)
            self.h = None


class Cache:
    """The oracle's cache: per (sequence, layer) two arrival-ordered streams plus page ids."""

    def __init__(self, policy: Policy, n_q: int, n_kv: int, max_seqs: int, pool_high_pages: int,
                 pool_low_pages: int):
        self.policy = policy
        self.n_q, self.n_kv = n_q, n_kv
        self.h = lib().orc_cache_create(policy.h, n_q, n_kv, max_seqs, pool_high_pages, pool_low_pages)
        if not self.h:
            raise ValueError("oracle rejected the cache shape")

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_cache_destroy(self.h)
            self.h = None

    def decide(self, seq_ids, cu_tokens, tags, states=None, n_groups=None):
        """Algorithm 2 steps 1-6 and 8; returns (status, actions u8 [total][n_groups])."""
        seq_ids = np.ascontiguousarray(seq_ids, dtype=np.int32)
        cu = np.ascontiguousarray(cu_tokens, dtype=np.int32)
        tags = np.ascontiguousarray(tags, dtype=np.uint8)
        total = int(cu[-1])
        assert tags.size == total
        st = None
        if states is not None:
            st = np.ascontiguousarray(states, dtype=np.uint16)
            assert st.size == total
        actions = np.full((total, n_groups), 0xEE, dtype=np.uint8)
        rc = lib().orc_decide(self.h, len(seq_ids), _ptr(seq_ids), _ptr(cu), _ptr(tags),
                              _ptr(st) if st is not None else None, _ptr(actions))
        return rc, actions

    def append(self, layer, seq_ids, cu_tokens, k_bits, v_bits, tags, decided=None):
        """k_bits / v_bits: int16/uint16 [total][n_kv][128]; returns (status, actions u8 [total]).
        decided: u8 [total][n_groups] from decide(), persisted instead of the table's actions."""
        seq_ids = np.ascontiguousarray(seq_ids, dtype=np.int32)
        cu = np.ascontiguousarray(cu_tokens, dtype=np.int32)
        k = np.ascontiguousarray(k_bits).view(np.uint16)
        v = np.ascontiguousarray(v_bits).view(np.uint16)
        tags = np.ascontiguousarray(tags, dtype=np.uint8)
        total = int(cu[-1])
        assert k.size == total * self.n_kv * 128 and v.size == k.size and tags.size == total
        actions = np.full(total, 0xEE, dtype=np.uint8)
        dec = None
        if decided is not None:
            dec = np.ascontiguousarray(decided, dtype=np.uint8)
            assert dec.ndim == 2 and dec.shape[0] == total
        rc = lib().orc_append_decided(self.h, layer, len(seq_ids), _ptr(seq_ids), _ptr(cu), _ptr(k), _ptr(v),
                                      _ptr(tags), _ptr(dec) if dec is not None else None, _ptr(actions))
        return rc, actions

    def stream_len(self, layer, seq):
        a, b = C.c_uint32(0), C.c_uint32(0)
        rc = lib().orc_stream_len(self.h, layer, seq, C.byref(a), C.byref(b))
        assert rc == 0
        return a.value, b.value

    def dump_high(self, layer, seq):
        nh, _ = self.stream_len(layer, seq)
        k = np.zeros((nh, self.n_kv, 128), np.uint16)
        v = np.zeros_like(k)
        pages = np.zeros((nh + 15) // 16, np.uint32)
        n = lib().orc_dump_high(self.h, layer, seq, _ptr(k), _ptr(v), _ptr(pages))
        assert n == pages.shape[0]
        return k, v, pages

    def dump_low(self, layer, seq):
        _, nl = self.stream_len(layer, seq)
        kc = np.zeros((nl, self.n_kv, 128), np.uint8)
        vc = np.zeros_like(kc)
        ks = np.zeros((nl, self.n_kv, 4), np.uint16)
        vs = np.zeros_like(ks)
        pages = np.zeros((nl + 15) // 16, np.uint32)
        n = lib().orc_dump_low(self.h, layer, seq, _ptr(kc), _ptr(ks), _ptr(vc), _ptr(vs), _ptr(pages))
        assert n == pages.shape[0]
        return kc, ks, vc, vs, pages

    def budget(self, seq) -> Budget:
        b = Budget()
        rc = lib().orc_budget_state(self.h, seq, C.byref(b))
        assert rc == 0
        return b

    def pool_state(self):
        v = [C.c_uint32(0) for _ in range(4)]
        lib().orc_pool_state(self.h, *[C.byref(x) for x in v])
        return tuple(x.value for x in v)   # high_next, high_free, low_next, low_free

    def seq_reset(self, seq):
        return lib().orc_seq_reset(self.h, seq)

    def attention(self, layer, seq, q_bits):
        """q_bits [n_q][128] bf16 bit patterns -> (out f64 [n_q][128], lse f64 [n_q])."""
        q = np.ascontiguousarray(q_bits).view(np.uint16)
        out = np.zeros((self.n_q, 128), np.float64)
        lse = np.zeros(self.n_q, np.float64)
        rc = lib().orc_attention(self.h, layer, seq, _ptr(q), _ptr(out), _ptr(lse))
        assert rc == 0
        return out, lse

    def attention_batch(self, layer, seq_ids, q_bits):
        seq_ids = np.ascontiguousarray(seq_ids, dtype=np.int32)
        q = np.ascontiguousarray(q_bits).view(np.uint16)
        n = len(seq_ids)
        out = np.zeros((n, self.n_q, 128), np.float64)
        lse = np.zeros((n, self.n_q), np.float64)
        rc = lib().orc_attention_batch(self.h, layer, n, _ptr(seq_ids), _ptr(q), _ptr(out), _ptr(lse))
        assert rc == 0
        return out, lse


def distortion(o_ref: np.ndarray, o_test: np.ndarray):
    """Eq. 4's inner term: (per-row max over heads of the squared distance, their sum). fp32 [rows][n_q][128] in."""
    a = np.ascontiguousarray(o_ref, dtype=np.float32)
    b = np.ascontiguousarray(o_test, dtype=np.float32)
    assert a.shape == b.shape and a.ndim == 3 and a.shape[2] == 128
    per = np.zeros(a.shape[0], np.float64)
    total = lib().orc_distortion(a.shape[0], a.shape[1], _ptr(a), _ptr(b), _ptr(per))
    return per, float(total)


def max_threads() -> int:
    return int(lib().orc_max_threads())


def set_threads(n: int) -> None:
    """Threads of the oracle's parallel loops (torchrun pins OMP_NUM_THREADS to 1 per rank)."""
    lib().orc_set_threads(int(n))
