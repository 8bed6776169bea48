"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, sizes workspaces, counts tiles and rejects bad arguments before any launch."""
import ctypes as C
import os
import re

import pytest

from paper_2506_19651_b200 import binding as pb
from paper_2506_19651_b200 import build as pbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pbuild.build()
    return pb.lib()


def test_exports_match_header(lib):
    header = open(os.path.join(ROOT, "include", "pevlm.h")).read()
    declared = set(re.findall(r"\b(pevlm_[a-z_]+)\s*\(", header))
    assert declared == set(pb.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_strerror(lib):
    assert lib.pevlm_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert len(lib.pevlm_strerror(code)) > 3


def test_workspace_sizes(lib):
    s = pb.make_shape(1568, 1568, 31, 128, 28, 4, 128, 1e6)
    assert pb.pevlm_workspace_bytes(s, pb.WS_PREFILL) >= 256
    q = pb.pevlm_workspace_bytes(s, pb.WS_QUERY)
    assert q > 128 * 28 * 129 * 4          # at least one split of fp32 partials
    assert q < 1 << 30
    bad = pb.make_shape(10, 10, 1, 1, 3, 2, 128)   # Hq % Hkv != 0
    assert pb.pevlm_workspace_bytes(bad, pb.WS_QUERY) == 0


def test_tile_stats_closed_form(lib):
    # sizes that are multiples of 128: tiles = Hq * (tri(S/128) + N * (B/128) * (S/128) + N * tri(B/128))
    S, B, N, Hq = 256, 384, 3, 4
    s = pb.make_shape(S, B, N, 0, Hq, 2, 128)
    st = pb.pevlm_tile_stats(s, pb.WS_PREFILL)
    tri = lambda n: n * (n + 1) // 2
    tiles = Hq * (tri(S // 128) + N * ((B // 128) * (S // 128) + tri(B // 128)))
    assert st.tiles == tiles
    assert st.flops == 4.0 * 128 * 128 * 128 * tiles
    full = pb.make_shape(S, B, N, 0, Hq, 2, 128, mask_mode=pb.MASK_FULL_CAUSAL)
    assert pb.pevlm_tile_stats(full, pb.WS_PREFILL).tiles == Hq * tri((S + N * B) // 128)
    # ragged: 784 = 6 * 128 + 16 -> the last key tile issues 16 columns
    r = pb.make_shape(784, 784, 1, 0, 1, 1, 128)
    st = pb.pevlm_tile_stats(r, pb.WS_PREFILL)
    assert st.tiles == tri(7) + 7 * 7 + tri(7)
    cols_tri = sum(sum(min(128, min(784, (q + 1) * 128) - j * 128) for j in range(q + 1)) for q in range(7))
    assert st.flops == 4.0 * 128 * 128 * (cols_tri + 7 * 784 + cols_tri)


def test_tile_stats_packed_ragged_tails(lib):
    # 1568 = 12 * 128 + 32: the 32-row tails of 4 of the 7 q heads of a kv group share one query tile,
    # so a (segment, kv head) has 12 * 7 full tiles and ceil(7 / 4) = 2 tail tiles
    S = B = 1568
    N, Hq, Hkv = 2, 28, 4
    st = pb.pevlm_tile_stats(pb.make_shape(S, B, N, 0, Hq, Hkv, 128), pb.WS_PREFILL)
    G = Hq // Hkv
    sink_tiles = sum((qt + 1) * G for qt in range(12)) + 13 * 2          # key tiles per query tile: qt + 1
    block_tiles = sum((13 + qt + 1) * G for qt in range(12)) + (13 + 13) * 2
    assert st.tiles == Hkv * (sink_tiles + N * block_tiles)
    # more than 64 tail rows: no packing (every head keeps its own ragged tile)
    st2 = pb.pevlm_tile_stats(pb.make_shape(200, 200, 1, 0, 4, 2, 128), pb.WS_PREFILL)
    assert st2.tiles == 4 * ((1 + 2) + (2 + 1) + (2 + 2))


def test_argument_errors_before_launch(lib):
    good = pb.make_shape(64, 128, 4, 32, 4, 2, 64)
    ws = C.c_void_p(256 * 4)
    p16 = C.c_void_p(4096)
    odd = C.c_void_p(4098)
    f = lib.pevlm_parallel_prefill_attn
    assert f(C.byref(good), None, p16, p16, p16, None, ws, 1 << 20, None) == pb.PEVLM_EINVAL
    assert f(C.byref(good), odd, p16, p16, p16, None, ws, 1 << 20, None) == pb.PEVLM_EALIGN
    # the attention outputs are written with 32-byte vector stores: an `o` at 16 mod 32 is refused on the
    # host (nothing is launched), for every call that writes one
    o16 = C.c_void_p(4096 + 16)
    assert f(C.byref(good), p16, p16, p16, o16, None, ws, 1 << 20, None) == pb.PEVLM_EALIGN
    assert lib.pevlm_block_attn(C.byref(good), p16, p16, p16, 64, 64 + 512, o16, None, ws, 1 << 20, None) == pb.PEVLM_EALIGN
    assert lib.pevlm_query_attn(C.byref(good), p16, p16, p16, o16, None, ws, 1 << 30, None) == pb.PEVLM_EALIGN
    assert lib.pevlm_query_attn_noalloc(C.byref(good), p16, p16, p16, o16, None, None) == pb.PEVLM_EALIGN
    assert f(C.byref(good), p16, p16, p16, p16, None, C.c_void_p(4096 + 128), 1 << 20, None) == pb.PEVLM_EALIGN
    assert f(C.byref(good), p16, p16, p16, p16, None, None, 1 << 20, None) == pb.PEVLM_EWORKSPACE
    assert f(C.byref(good), p16, p16, p16, p16, None, ws, 8, None) == pb.PEVLM_EWORKSPACE
    assert f(None, p16, p16, p16, p16, None, ws, 1 << 20, None) == pb.PEVLM_EINVAL
    for field, val, code in [("head_dim", 96, pb.PEVLM_EUNSUPPORTED), ("num_kv_heads", 3, pb.PEVLM_EINVAL),
                             ("sink_len", -1, pb.PEVLM_EINVAL), ("batch", 0, pb.PEVLM_EINVAL),
                             ("mask_mode", 7, pb.PEVLM_EINVAL), ("rope_theta", 0.0, pb.PEVLM_EINVAL)]:
        bad = pb.make_shape(64, 128, 4, 32, 4, 2, 64)
        setattr(bad, field, val)
        assert f(C.byref(bad), p16, p16, p16, p16, None, ws, 1 << 20, None) == code, field
        assert lib.pevlm_query_attn(C.byref(bad), p16, p16, p16, p16, None, ws, 1 << 30, None) == code, field
        assert lib.pevlm_rope_qk(C.byref(bad), p16, p16, p16, p16, 0, 8, None, None) == code, field
        assert lib.pevlm_assemble_kv(C.byref(bad), p16, p16, p16, p16, p16, p16, None) == code, field
        # the no-workspace entry point names the same error, before it touches the device
        assert lib.pevlm_query_attn_noalloc(C.byref(bad), p16, p16, p16, p16, None, None) == code, field
    assert lib.pevlm_rope_qk(C.byref(good), p16, None, None, None, 0, 8, None, None) == pb.PEVLM_EINVAL
    assert lib.pevlm_rope_qk(C.byref(good), odd, None, odd, None, 0, 8, None, None) == pb.PEVLM_EALIGN
    assert lib.pevlm_rope_qk(C.byref(good), p16, None, p16, None, -1, 8, None, None) == pb.PEVLM_EINVAL
    sec_bad = (C.c_int32 * 3)(16, 24, 23)
    sec_ok = (C.c_int32 * 3)(8, 12, 12)
    assert lib.pevlm_rope_qk_mrope(C.byref(good), p16, None, p16, None, 8, p16, sec_bad, None) == pb.PEVLM_EINVAL
    assert lib.pevlm_rope_qk_mrope(C.byref(good), p16, None, p16, None, 8, None, sec_ok, None) == pb.PEVLM_EINVAL
    assert lib.pevlm_rope_qk_mrope(C.byref(good), odd, None, odd, None, 8, p16, sec_ok, None) == pb.PEVLM_EALIGN
    assert lib.pevlm_assemble_kv(C.byref(good), p16, None, None, None, None, None, None) == pb.PEVLM_EINVAL
    assert lib.pevlm_query_attn(C.byref(good), p16, p16, p16, p16, None, ws, 16, None) == pb.PEVLM_EWORKSPACE
    # block range: must start at or after the sink and end inside the cache; PEVLM mask only
    g = lib.pevlm_block_attn
    nb = good.num_blocks * good.block_len
    assert g(C.byref(good), p16, p16, p16, 63, 64 + nb, p16, None, ws, 1 << 20, None) == pb.PEVLM_EINVAL
    assert g(C.byref(good), p16, p16, p16, 64, 64 + nb - 1, p16, None, ws, 1 << 20, None) == pb.PEVLM_EINVAL
    assert g(C.byref(good), p16, p16, odd, 64, 64 + nb, p16, None, ws, 1 << 20, None) == pb.PEVLM_EALIGN
    assert g(C.byref(good), p16, p16, p16, 64, 64 + nb, p16, None, None, 0, None) == pb.PEVLM_EWORKSPACE
    fc = pb.make_shape(64, 128, 4, 32, 4, 2, 64, mask_mode=pb.MASK_FULL_CAUSAL)
    assert g(C.byref(fc), p16, p16, p16, 64, 64 + nb, p16, None, ws, 1 << 20, None) == pb.PEVLM_EINVAL
    assert lib.pevlm_query_attn_noalloc(C.byref(good), None, p16, p16, p16, None, None) == pb.PEVLM_EINVAL
    # wait self-test: workspace, alignment and the range of the limit are checked on the host
    t = lib.pevlm_selftest_wait_expiry
    assert t(None, 256, 1000000, None) == pb.PEVLM_EWORKSPACE
    assert t(ws, 16, 1000000, None) == pb.PEVLM_EWORKSPACE
    assert t(C.c_void_p(1024 + 8), 256, 1000000, None) == pb.PEVLM_EALIGN
    assert t(ws, 256, 10, None) == pb.PEVLM_EINVAL
    assert t(ws, 256, 10 ** 10, None) == pb.PEVLM_EINVAL


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(pb, "_lib", None)
    monkeypatch.setattr(pb, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        pb.lib()
