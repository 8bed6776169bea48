"""Thin ctypes binding over the C ABI of libpevlm.so (include/pevlm.h), same names.

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
Tensors are torch CUDA tensors (torch is used for device memory and streams); a call
enqueues work on torch's current stream and returns.  There is no CPU fallback: if the
library has not been built, `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_DIR, "libpevlm.so")

PEVLM_OK = 0
PEVLM_EINVAL, PEVLM_EALIGN, PEVLM_EUNSUPPORTED, PEVLM_EWORKSPACE, PEVLM_ECUDA, PEVLM_ETIMEOUT = -1, -2, -3, -4, -5, -6
MASK_PEVLM, MASK_FULL_CAUSAL = 0, 1
WS_PREFILL, WS_QUERY = 0, 1

NOALLOC_SCRATCH_BYTES = 32 << 20

EXPORTS = ["pevlm_rope_qk", "pevlm_rope_qk_mrope", "pevlm_parallel_prefill_attn", "pevlm_block_attn", "pevlm_assemble_kv", "pevlm_query_attn",
           "pevlm_query_attn_noalloc",
           "pevlm_workspace_bytes", "pevlm_read_status", "pevlm_selftest_wait_expiry", "pevlm_tile_stats", "pevlm_strerror",
           "pevlm_last_cuda_error"]


class Shape(C.Structure):
    """pevlm_shape_t"""
    _fields_ = [("batch", C.c_int32), ("sink_len", C.c_int32), ("block_len", C.c_int32),
                ("num_blocks", C.c_int32), ("query_len", C.c_int32), ("num_q_heads", C.c_int32),
                ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("rope_theta", C.c_float),
                ("softmax_scale", C.c_float), ("mask_mode", C.c_int32)]

    @property
    def n_video(self):
        return self.sink_len + self.num_blocks * self.block_len

    @property
    def L(self):
        return self.n_video + self.query_len


def make_shape(S, B, N, Q, Hq, Hkv, d, theta=1e4, scale=0.0, mask_mode=MASK_PEVLM, batch=1) -> Shape:
    return Shape(batch, S, B, N, Q, Hq, Hkv, d, theta, scale, mask_mode)


class PevlmError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        text = lib().pevlm_strerror(code).decode()
        extra = lib().pevlm_last_cuda_error().decode() if code == PEVLM_ECUDA else ""
        super().__init__(f"{where}: {text} ({code}) {extra}".strip())


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_19651_b200.build` "
                               "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        vp, sp = C.c_void_p, C.POINTER(Shape)
        l.pevlm_rope_qk.argtypes = [sp, vp, vp, vp, vp, C.c_int64, C.c_int64, vp, vp]
        l.pevlm_rope_qk_mrope.argtypes = [sp, vp, vp, vp, vp, C.c_int64, vp, C.POINTER(C.c_int32), vp]
        l.pevlm_rope_qk_mrope.restype = C.c_int
        l.pevlm_parallel_prefill_attn.argtypes = [sp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        l.pevlm_block_attn.argtypes = [sp, vp, vp, vp, C.c_int64, C.c_int64, vp, vp, vp, C.c_size_t, vp]
        l.pevlm_block_attn.restype = C.c_int
        l.pevlm_assemble_kv.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp]
        l.pevlm_query_attn.argtypes = [sp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        l.pevlm_query_attn_noalloc.argtypes = [sp, vp, vp, vp, vp, vp, vp]
        l.pevlm_query_attn_noalloc.restype = C.c_int
        l.pevlm_workspace_bytes.argtypes = [sp, C.c_int]
        l.pevlm_workspace_bytes.restype = C.c_size_t
        l.pevlm_read_status.argtypes = [vp, vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        l.pevlm_selftest_wait_expiry.argtypes = [vp, C.c_size_t, C.c_int64, vp]
        l.pevlm_selftest_wait_expiry.restype = C.c_int
        l.pevlm_tile_stats.argtypes = [sp, C.c_int, C.POINTER(C.c_int64), C.POINTER(C.c_double)]
        l.pevlm_strerror.argtypes = [C.c_int]
        l.pevlm_strerror.restype = C.c_char_p
        l.pevlm_last_cuda_error.restype = C.c_char_p
        for name in ("pevlm_rope_qk", "pevlm_parallel_prefill_attn", "pevlm_assemble_kv", "pevlm_query_attn",
                     "pevlm_read_status", "pevlm_tile_stats"):
            getattr(l, name).restype = C.c_int
        _lib = l
    return _lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, where):
    if rc != PEVLM_OK:
        raise PevlmError(rc, where)


def pevlm_workspace_bytes(shape: Shape, which: int) -> int:
    return int(lib().pevlm_workspace_bytes(C.byref(shape), which))


def pevlm_rope_qk(shape: Shape, q_in, k_in, q_out, k_out, first_token: int, n_tokens: int, pos_ids=None):
    _check(lib().pevlm_rope_qk(C.byref(shape), _ptr(q_in), _ptr(k_in), _ptr(q_out), _ptr(k_out),
                               first_token, n_tokens, _ptr(pos_ids), _stream()), "pevlm_rope_qk")


def pevlm_rope_qk_mrope(shape: Shape, q_in, k_in, q_out, k_out, n_tokens: int, pos_ids3, sections):
    sec = (C.c_int32 * 3)(*sections)
    _check(lib().pevlm_rope_qk_mrope(C.byref(shape), _ptr(q_in), _ptr(k_in), _ptr(q_out), _ptr(k_out),
                                     n_tokens, _ptr(pos_ids3), sec, _stream()), "pevlm_rope_qk_mrope")


def pevlm_parallel_prefill_attn(shape: Shape, q, k, v, o, lse, workspace):
    _check(lib().pevlm_parallel_prefill_attn(C.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                             _ptr(workspace), workspace.numel() * workspace.element_size(),
                                             _stream()), "pevlm_parallel_prefill_attn")


def pevlm_block_attn(shape: Shape, q_blocks, k_cache, v_cache, first_key_row: int, cache_rows: int, o, lse, workspace):
    _check(lib().pevlm_block_attn(C.byref(shape), _ptr(q_blocks), _ptr(k_cache), _ptr(v_cache), first_key_row,
                                  cache_rows, _ptr(o), _ptr(lse), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream()), "pevlm_block_attn")


def pevlm_assemble_kv(shape: Shape, k_video, v_video, k_question, v_question, k_cache, v_cache):
    _check(lib().pevlm_assemble_kv(C.byref(shape), _ptr(k_video), _ptr(v_video), _ptr(k_question),
                                   _ptr(v_question), _ptr(k_cache), _ptr(v_cache), _stream()), "pevlm_assemble_kv")


def pevlm_query_attn(shape: Shape, q_question, k_cache, v_cache, o, lse, workspace):
    _check(lib().pevlm_query_attn(C.byref(shape), _ptr(q_question), _ptr(k_cache), _ptr(v_cache), _ptr(o),
                                  _ptr(lse), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                  _stream()), "pevlm_query_attn")


def pevlm_query_attn_noalloc(shape: Shape, q_question, k_cache, v_cache, o, lse):
    """Question attention for callers that cannot allocate device memory: no workspace argument,
    the partials go to the library's built-in scratch array (see include/pevlm.h for its limits)."""
    _check(lib().pevlm_query_attn_noalloc(C.byref(shape), _ptr(q_question), _ptr(k_cache), _ptr(v_cache), _ptr(o),
                                          _ptr(lse), _stream()), "pevlm_query_attn_noalloc")


def pevlm_selftest_wait_expiry(workspace, limit_ns: int):
    _check(lib().pevlm_selftest_wait_expiry(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                            limit_ns, _stream()), "pevlm_selftest_wait_expiry")


def pevlm_read_status(workspace):
    """workspace = None reads the built-in array of pevlm_query_attn_noalloc on the current device."""
    st, det = C.c_int32(0), C.c_int32(0)
    _check(lib().pevlm_read_status(_ptr(workspace), _stream(), C.byref(st), C.byref(det)), "pevlm_read_status")
    return st.value, det.value


@dataclass
class TileStats:
    tiles: int
    flops: float


def pevlm_tile_stats(shape: Shape, which: int) -> TileStats:
    t, f = C.c_int64(0), C.c_double(0.0)
    _check(lib().pevlm_tile_stats(C.byref(shape), which, C.byref(t), C.byref(f)), "pevlm_tile_stats")
    return TileStats(t.value, f.value)
