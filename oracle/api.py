"""ctypes wrapper over the C oracle (oracle/pevlm_oracle.c).  TEST INFRASTRUCTURE ONLY.

Arrays of bf16 values are numpy uint16 bit patterns; results are fp64.
"""
from __future__ import annotations

import ctypes as C
import numpy as np

from .build import build

_lib = None


class Shape(C.Structure):
    _fields_ = [("S", C.c_int64), ("B", C.c_int64), ("N", C.c_int64), ("Q", C.c_int64),
                ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32), ("full_causal", C.c_int32),
                ("B_last", C.c_int64)]

    @property
    def n_video(self):
        if self.N <= 0:
            return self.S
        return self.S + (self.N - 1) * self.B + (self.B_last if self.B_last > 0 else self.B)

    @property
    def L(self):
        return self.n_video + self.Q


def make_shape(S, B, N, Q, Hq, Hkv, d, full_causal=False, B_last=0) -> Shape:
    """B_last: length of the last context block when the video does not divide evenly (0 = B)."""
    assert 0 <= B_last <= B
    return Shape(S, B, N, Q, Hq, Hkv, d, 1 if full_causal else 0, B_last)


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_num_threads.restype = C.c_int
        _lib.oracle_visible.restype = C.c_int
        _lib.oracle_count_pairs.restype = C.c_int64
        _lib.oracle_round_bf16.restype = C.c_uint16
        _lib.oracle_round_bf16.argtypes = [C.c_double]
        _lib.oracle_count_rect_pairs.restype = C.c_int64
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16
    return a


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().oracle_set_num_threads(C.c_int(int(n)))


def round_bf16(x: float) -> int:
    """bf16 bit pattern of the two-step rounding fp64 -> fp32 -> bf16 (both to nearest even) the RoPE ends with."""
    return int(lib().oracle_round_bf16(float(x)))


def visible(sh: Shape, t: int):
    lo = (C.c_int64 * 2)()
    hi = (C.c_int64 * 2)()
    n = lib().oracle_visible(C.byref(sh), C.c_int64(t), lo, hi)
    return [(int(lo[i]), int(hi[i])) for i in range(n)]


def rope(x_bits, theta: float, pos=None, first_pos: int = 0, want_f64: bool = False):
    """x_bits [n, heads, d] uint16 -> roped bf16 bits (and the fp64 values before rounding)."""
    x = _u16(x_bits)
    n, heads, d = x.shape
    out = np.empty_like(x)
    f64 = np.empty(x.shape, dtype=np.float64) if want_f64 else None
    posa = np.ascontiguousarray(pos, dtype=np.int64) if pos is not None else None
    lib().oracle_rope(_p(x), C.c_int64(n), C.c_int32(heads), C.c_int32(d), C.c_double(theta),
                      _p(posa), C.c_int64(first_pos), _p(out), _p(f64))
    return (out, f64) if want_f64 else out


def rope_mrope(x_bits, theta: float, pos3, sections, want_f64: bool = False):
    """Multimodal RoPE: pos3 [3, n] (temporal, height, width), sections = pairs per component."""
    x = _u16(x_bits)
    n, heads, d = x.shape
    pos3 = np.ascontiguousarray(pos3, dtype=np.int64)
    assert pos3.shape == (3, n) and sum(sections) == d // 2
    sec = np.ascontiguousarray(sections, dtype=np.int32)
    out = np.empty_like(x)
    f64 = np.empty(x.shape, dtype=np.float64) if want_f64 else None
    lib().oracle_rope_mrope(_p(x), C.c_int64(n), C.c_int32(heads), C.c_int32(d), C.c_double(theta),
                            _p(pos3), _p(sec), _p(out), _p(f64))
    return (out, f64) if want_f64 else out


def attn_rows(sh: Shape, q_bits, k_bits, v_bits, rows, scale: float = 0.0, key_lo: int = -1, key_hi: int = -1):
    """Rows of masked softmax attention.  Returns (o [n,Hq,d] fp64, lse [n,Hq] fp64)."""
    q, k, v = _u16(q_bits), _u16(k_bits), _u16(v_bits)
    L = sh.L
    assert q.shape == (L, sh.Hq, sh.d) and k.shape == (L, sh.Hkv, sh.d) and v.shape == k.shape
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < L)
    o = np.empty((rows.size, sh.Hq, sh.d), dtype=np.float64)
    lse = np.empty((rows.size, sh.Hq), dtype=np.float64)
    lib().oracle_attn_rows(C.byref(sh), _p(q), _p(k), _p(v), C.c_double(scale), _p(rows),
                           C.c_int64(rows.size), C.c_int64(key_lo), C.c_int64(key_hi), _p(o), _p(lse))
    return o, lse


def weights_row(sh: Shape, q_bits, k_bits, t: int, h: int, scale: float = 0.0):
    q, k = _u16(q_bits), _u16(k_bits)
    w = np.empty(sh.L, dtype=np.float64)
    lib().oracle_weights_row(C.byref(sh), _p(q), _p(k), C.c_double(scale), C.c_int64(t), C.c_int32(h), _p(w))
    return w


def merge_lse(o_parts, lse_parts):
    """o_parts [splits, n, d], lse_parts [splits, n] -> (o [n,d], lse [n])."""
    o_parts = np.ascontiguousarray(o_parts, dtype=np.float64)
    lse_parts = np.ascontiguousarray(lse_parts, dtype=np.float64)
    s, n, d = o_parts.shape
    o = np.empty((n, d), dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    lib().oracle_merge_lse(_p(o_parts), _p(lse_parts), C.c_int64(s), C.c_int64(n), C.c_int32(d), _p(o), _p(lse))
    return o, lse


def assemble_kv(sh: Shape, video_bits, question_bits):
    v, qn = _u16(video_bits), _u16(question_bits)
    cache = np.empty((sh.L, sh.Hkv, sh.d), dtype=np.uint16)
    lib().oracle_assemble_kv(C.byref(sh), _p(v), _p(qn), _p(cache))
    return cache


def count_pairs(sh: Shape) -> int:
    return int(lib().oracle_count_pairs(C.byref(sh)))


def count_rect_pairs(sh: Shape) -> int:
    return int(lib().oracle_count_rect_pairs(C.byref(sh)))
