"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test cites the passage it pins.  The oracle under test is oracle/pevlm_oracle.c
(through oracle.api); the independent comparisons are oracle/dense.py (a dense-mask numpy
evaluation), closed forms, and a literal pure-Python loop written in this file.
"""
import math
import os
import struct

import numpy as np
import pytest

from oracle import api, dense
from paper_2506_19651_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_stream(S, B, N, Q, Hq, Hkv, d, seed=11, theta=1e4, outliers=False, pos=None):
    w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, theta, outliers, seed)
    q, k, v = inputs.make_qkv(w)
    qr = api.rope(q, theta, pos=pos)
    kr = api.rope(k, theta, pos=pos)
    return w, q, k, v, qr, kr


def all_rows(L):
    return np.arange(L, dtype=np.int64)


# ---- P1: with N <= 1 the PEVLM mask is plain causal attention (Eq. 1, Eq. 3-5) --------

@pytest.mark.parametrize("S,B,N,Q", [(5, 7, 1, 3), (9, 1, 0, 4), (0, 6, 1, 2), (4, 3, 1, 0)])
def test_p1_single_block_is_full_causal(S, B, N, Q):
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, 4, 2, 8)
    sh = api.make_shape(S, B, N, Q, 4, 2, 8)
    o, lse = api.attn_rows(sh, qr, kr, v, all_rows(w.L))
    tril = np.tril(np.ones((w.L, w.L), dtype=bool))     # textbook causal mask
    o_ref, lse_ref, _ = dense.dense_attention(qr, kr, v, tril)
    np.testing.assert_allclose(o, o_ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref, rtol=0, atol=1e-12)


def test_p1_full_causal_mode_any_n():
    S, B, N, Q = 6, 5, 3, 4
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, 2, 2, 16)
    sh = api.make_shape(S, B, N, Q, 2, 2, 16, full_causal=True)
    o, lse = api.attn_rows(sh, qr, kr, v, all_rows(w.L))
    tril = np.tril(np.ones((w.L, w.L), dtype=bool))
    o_ref, lse_ref, _ = dense.dense_attention(qr, kr, v, tril)
    np.testing.assert_allclose(o, o_ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref, rtol=0, atol=1e-12)


# ---- whole mask against the dense-mask evaluation (Eq. 3-5, Sec. 3.2.1) --------------

@pytest.mark.parametrize("S,B,N,Q,Hq,Hkv,d", [(3, 4, 2, 2, 2, 1, 4), (8, 16, 3, 5, 4, 2, 8), (0, 4, 3, 2, 2, 2, 4),
                                              (5, 3, 4, 0, 6, 2, 8), (64, 128, 4, 32, 4, 2, 64)])
def test_oracle_vs_dense_mask(S, B, N, Q, Hq, Hkv, d):
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, Hq, Hkv, d)
    sh = api.make_shape(S, B, N, Q, Hq, Hkv, d)
    o, lse = api.attn_rows(sh, qr, kr, v, all_rows(w.L))
    mask = dense.dense_mask(S, B, N, Q)
    o_ref, lse_ref, _ = dense.dense_attention(qr, kr, v, mask)
    np.testing.assert_allclose(o, o_ref, rtol=0, atol=1e-11)
    np.testing.assert_allclose(lse, lse_ref, rtol=0, atol=1e-11)


# ---- shorter last context block (a video that does not divide evenly; Sec. 3.2.1 is silent) ----

@pytest.mark.parametrize("S,B,N,Q,B_last,Hq,Hkv,d", [(3, 4, 3, 2, 1, 2, 1, 4), (8, 16, 3, 5, 7, 4, 2, 8),
                                                     (0, 5, 2, 3, 4, 2, 2, 4), (6, 9, 1, 2, 5, 2, 1, 8)])
def test_ragged_last_block_vs_dense_mask_and_counts(S, B, N, Q, B_last, Hq, Hkv, d):
    w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, 1e4, False, 13, B_last=B_last)
    assert w.n_video == S + (N - 1) * B + B_last
    q, k, v = inputs.make_qkv(w)
    qr, kr = api.rope(q, 1e4), api.rope(k, 1e4)
    sh = api.make_shape(S, B, N, Q, Hq, Hkv, d, B_last=B_last)
    assert sh.L == w.L
    o, lse = api.attn_rows(sh, qr, kr, v, all_rows(w.L))
    mask = dense.dense_mask(S, B, N, Q, B_last=B_last)
    assert mask.shape == (w.L, w.L)
    o_ref, lse_ref, _ = dense.dense_attention(qr, kr, v, mask)
    np.testing.assert_allclose(o, o_ref, rtol=0, atol=1e-11)
    np.testing.assert_allclose(lse, lse_ref, rtol=0, atol=1e-11)
    # closed-form pair counts: the last block contributes B_last*S + tri(B_last) (Eq. 8 with its own length)
    tri = lambda n: n * (n + 1) // 2
    nv = w.n_video
    want = tri(S) + (N - 1) * (B * S + tri(B)) + B_last * S + tri(B_last) + Q * nv + tri(Q)
    assert api.count_pairs(sh) == want == int(mask.sum())
    want_rect = S * S + (N - 1) * B * (S + B) + B_last * (S + B_last) + Q * w.L
    assert api.count_rect_pairs(sh) == want_rect
    # zero keys: LSE = ln(#visible) (row r of the last block sees S + r + 1 keys)
    o0, lse0 = api.attn_rows(sh, q, np.zeros_like(k), v, all_rows(w.L))
    first_last = S + (N - 1) * B
    for t in range(first_last, nv):
        assert abs(lse0[t, 0] - math.log(S + (t - first_last) + 1)) < 1e-12
    for t in range(nv, w.L):
        assert abs(lse0[t, 0] - math.log(t + 1)) < 1e-12


def test_ragged_last_block_equal_to_uniform_when_lengths_agree():
    S, B, N, Q, Hq, Hkv, d = 4, 6, 3, 2, 2, 1, 4
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, Hq, Hkv, d)
    a = api.attn_rows(api.make_shape(S, B, N, Q, Hq, Hkv, d), qr, kr, v, all_rows(w.L))
    b = api.attn_rows(api.make_shape(S, B, N, Q, Hq, Hkv, d, B_last=B), qr, kr, v, all_rows(w.L))
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


# ---- P2: sink rows equal full-attention rows (Eq. 3) ---------------------------------

def test_p2_sink_rows_equal_full_attention():
    S, B, N, Q = 10, 6, 3, 4
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, 4, 2, 8)
    rows = all_rows(S)
    o_p, lse_p = api.attn_rows(api.make_shape(S, B, N, Q, 4, 2, 8), qr, kr, v, rows)
    tril = np.tril(np.ones((w.L, w.L), dtype=bool))
    o_f, lse_f, _ = dense.dense_attention(qr, kr, v, tril)
    np.testing.assert_allclose(o_p, o_f[:S], rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse_p, lse_f[:S], rtol=0, atol=1e-12)


# ---- P3: softmax weights sum to 1, lie in (0,1], vanish across blocks (Sec. 1) -------

def test_p3_weights_sum_to_one_and_block_isolation():
    S, B, N, Q = 6, 5, 4, 3
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, 2, 1, 8)
    sh = api.make_shape(S, B, N, Q, 2, 1, 8)
    seg = dense.segment_ids(S, B, N, Q)
    for t in range(w.L):
        for h in range(2):
            wt = api.weights_row(sh, qr, kr, t, h)
            assert abs(wt.sum() - 1.0) < 1e-12
            assert (wt >= 0).all() and wt.max() <= 1.0
            assert (wt[t + 1:] == 0).all()              # causal
            if 0 <= seg[t] < N:                          # context row: nothing from other blocks
                other = (seg >= 0) & (seg < N) & (seg != seg[t])
                assert (wt[other] == 0).all()
                assert (wt[:S] > 0).all()                # the whole sink is visible
            # o equals the weighted sum of V
            o, _ = api.attn_rows(sh, qr, kr, v, np.array([t]))
            ref = wt @ dense.bits_to_f64(v)[:, 0, :]
            np.testing.assert_allclose(o[0, h], ref, rtol=0, atol=1e-12)


# ---- P4: block independence and sequential positions (Sec. 3.2.2, Sec. 1) ------------

def test_p4_block_permutation_with_carried_positions():
    S, B, N, Q = 4, 6, 3, 0
    Hq, Hkv, d, theta = 2, 1, 8, 1e4
    w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, theta, False, 5)
    q, k, v = inputs.make_qkv(w)
    pos = np.arange(w.L, dtype=np.int64)
    sh = api.make_shape(S, B, N, Q, Hq, Hkv, d)
    o0, lse0 = api.attn_rows(sh, api.rope(q, theta, pos=pos), api.rope(k, theta, pos=pos), v, all_rows(w.L))

    # swap the contents of blocks 0 and 2
    perm = np.arange(w.L)
    a = slice(S, S + B)
    c = slice(S + 2 * B, S + 3 * B)
    perm[a], perm[c] = np.arange(c.start, c.stop), np.arange(a.start, a.stop)
    q2, k2, v2 = q[perm], k[perm], v[perm]
    # positions carried with the content: outputs of the moved rows are unchanged
    pos2 = pos[perm]
    o1, lse1 = api.attn_rows(sh, api.rope(q2, theta, pos=pos2), api.rope(k2, theta, pos=pos2), v2, all_rows(w.L))
    np.testing.assert_array_equal(o1, o0[perm])
    np.testing.assert_array_equal(lse1, lse0[perm])
    # positions NOT carried (content moved, slots keep sequential positions): the moved blocks'
    # outputs change (only through RoPE), the untouched block's and the sink's do not
    o2, lse2 = api.attn_rows(sh, api.rope(q2, theta, pos=pos), api.rope(k2, theta, pos=pos), v2, all_rows(w.L))
    moved = np.r_[a, c]
    assert np.abs(o2[moved] - o0[perm][moved]).max() > 1e-3
    keep = np.r_[0:S, S + B:S + 2 * B]
    np.testing.assert_array_equal(o2[keep], o0[keep])


# ---- P5: closed forms with K = 0 or constant V (mask counted exactly; Eq. 3-5) -------

def test_p5_zero_keys_closed_form():
    S, B, N, Q, Hq, Hkv, d = 7, 5, 3, 4, 4, 2, 8
    w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, 1e4, False, 3)
    q, k, v = inputs.make_qkv(w)
    k0 = np.zeros_like(k)
    sh = api.make_shape(S, B, N, Q, Hq, Hkv, d)
    o, lse = api.attn_rows(sh, q, k0, v, all_rows(w.L))
    vf = dense.bits_to_f64(v)
    G = Hq // Hkv
    nv = S + N * B
    for t in range(w.L):
        if t < S or t >= nv:
            vis = list(range(t + 1))
            count = t + 1
        else:
            r = (t - S) % B
            start = t - r
            vis = list(range(S)) + list(range(start, t + 1))
            count = S + r + 1
        assert len(vis) == count
        for h in range(Hq):
            assert abs(lse[t, h] - math.log(count)) < 1e-12
            np.testing.assert_allclose(o[t, h], vf[vis, h // G, :].mean(axis=0), rtol=0, atol=1e-12)


def test_p5_constant_values():
    S, B, N, Q, Hq, Hkv, d = 5, 4, 2, 3, 2, 1, 8
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, Hq, Hkv, d)
    vconst = np.broadcast_to(v[0:1], v.shape).copy()
    o, _ = api.attn_rows(api.make_shape(S, B, N, Q, Hq, Hkv, d), qr, kr, vconst, all_rows(w.L))
    ref = dense.bits_to_f64(v[0, 0])
    np.testing.assert_allclose(o, np.broadcast_to(ref, o.shape), rtol=0, atol=1e-12)


# ---- P6: partition structure against the paper's operation model (Eq. 6-10) ----------

def test_p6_pair_counts_match_eq10_golden():
    for line in open(os.path.join(GOLDEN, "op_count_eq10.txt")):
        if line.startswith("#") or not line.strip():
            continue
        S, B, N, Q, eq10, full = (int(x) for x in line.split())
        sh = api.make_shape(S, B, N, Q, 1, 1, 2)
        assert api.count_rect_pairs(sh) == eq10
        L = S + N * B + Q
        assert api.count_rect_pairs(api.make_shape(0, 1, 0, L, 1, 1, 2)) == full  # one segment: L^2
        # causal counts: triangular numbers per segment
        tri = lambda n: n * (n + 1) // 2
        assert api.count_pairs(sh) == tri(S) + N * (B * S + tri(B)) + Q * (S + N * B) + tri(Q)
        assert api.count_pairs(api.make_shape(S, B, N, Q, 1, 1, 2, full_causal=True)) == tri(L)


def test_p6_speedup_ratio_consistent_with_paper():
    # The abstract's "up to 7.47x" attention speed-up (and 7.79x in Sec. 4.2) was measured at ~100k
    # tokens with 16-frame (~4k token) sink and blocks.  Under the mask read as "sink + own
    # block" the visible-pair ratio full/PEVLM at that scale is close to 8; reading Eq. 4
    # literally (all earlier blocks visible) would give about 1.
    S = B = 4096
    N, Q = 23, 256
    sh = api.make_shape(S, B, N, Q, 1, 1, 2)
    ratio = api.count_pairs(api.make_shape(S, B, N, Q, 1, 1, 2, full_causal=True)) / api.count_pairs(sh)
    assert 7.0 < ratio < 8.5


# ---- P7: RoPE convention and exactness (Sec. 3.2.2) ----------------------------------

def _bf16_bits_of(x: float) -> int:
    """Independent fp64 -> fp32 -> bf16 (RNE) rounding with struct, for scalar pins."""
    u = struct.unpack("<I", struct.pack("<f", x))[0]
    return (u + 0x7FFF + ((u >> 16) & 1)) >> 16


def _bits(vals):
    return np.array([_bf16_bits_of(v) for v in vals], dtype=np.uint16)


COS1, SIN1 = 0.5403023058681398, 0.8414709848078965   # cos(1), sin(1), typed from tables


def test_p7_rope_hand_values_pairing_and_frequency():
    # d = 4: pairs are (0,2) and (1,3); inv_freq = [1, theta^(-1/2)].  theta = 1e4 -> 0.01.
    # At position 100 the angles are 100 and 1.0.
    x = _bits([0.0, 1.0, 0.0, 0.0]).reshape(1, 1, 4)      # only element 1 set: pair (1,3), angle 1.0
    out, f64 = api.rope(x, 1e4, first_pos=100, want_f64=True)
    np.testing.assert_allclose(f64[0, 0], [0.0, COS1, 0.0, SIN1], rtol=0, atol=1e-15)
    np.testing.assert_array_equal(out[0, 0], _bits([0.0, COS1, 0.0, SIN1]))
    x = _bits([0.0, 0.0, 0.0, 2.0]).reshape(1, 1, 4)      # element 3: x'[1] = -2 sin, x'[3] = 2 cos
    _, f64 = api.rope(x, 1e4, first_pos=100, want_f64=True)
    np.testing.assert_allclose(f64[0, 0], [0.0, -2 * SIN1, 0.0, 2 * COS1], rtol=0, atol=1e-15)
    x = _bits([1.0, 0.0, 0.0, 0.0]).reshape(1, 1, 4)      # element 0: pair (0,2), angle = position = 1
    _, f64 = api.rope(x, 1e4, first_pos=1, want_f64=True)
    np.testing.assert_allclose(f64[0, 0], [COS1, 0.0, SIN1, 0.0], rtol=0, atol=1e-15)


def test_p7_bf16_rounding_is_nearest_even():
    # a = 1, b = 0 at angle 1: outputs cos(1), sin(1); compare bits with the struct-based rounding
    x = _bits([1.0, 0.0]).reshape(1, 1, 2)
    out = api.rope(x, 1e4, first_pos=1)
    assert int(out[0, 0, 0]) == _bf16_bits_of(COS1) == 0x3F0A
    assert int(out[0, 0, 1]) == _bf16_bits_of(SIN1) == 0x3F57
    # ties: 1 + 2^-8 -> 1.0 (even), 1 + 3*2^-8 -> 1 + 2^-6 (even); via position 0 (identity) on fp64
    assert _bf16_bits_of(1 + 2 ** -8) == 0x3F80 and _bf16_bits_of(1 + 3 * 2 ** -8) == 0x3F82


# R1, the one rounding of the oracle (fp64 -> fp32 -> bf16, both to nearest even), pinned on bit patterns
# worked out by hand from the binary expansions; the comments give the fp32 word before the second step.
R1_HAND = [
    (0.3, 0x3E9A),                        # 0x3E99999A: low half 0x999A > 0x8000, rounds UP
    (-0.3, 0xBE9A),                       # sign does not change the magnitude rounding
    (1 + 2.0 ** -9, 0x3F80),              # 0x3F804000: below half, rounds down
    (1 + 2.0 ** -8, 0x3F80),              # 0x3F808000: exact tie, 0x3F80 is even, stays
    (1 + 3 * 2.0 ** -8, 0x3F82),          # 0x3F818000: exact tie, 0x3F81 is odd, goes up to even
    (-(1 + 3 * 2.0 ** -8), 0xBF82),
    (1 + 2.0 ** -8 + 2.0 ** -20, 0x3F81),  # 0x3F808008: just above the tie, rounds up
    (1 + 2.0 ** -8 + 2.0 ** -30, 0x3F80),  # two steps: fp32 drops 2^-30 (tie 0x3F808000 -> even); one step would give 0x3F81
    (1 + 2.0 ** -7 - 2.0 ** -30, 0x3F81),  # fp32 rounds up to 0x3F810000 exactly: 0x3F81
    (1 + 3 * 2.0 ** -8 - 2.0 ** -30, 0x3F82),  # fp32 gives the tie 0x3F818000 -> even 0x3F82; one step would give 0x3F81
    (0.0, 0x0000), (1.0, 0x3F80), (-2.0, 0xC000), (3.140625, 0x4049),
    (65280.0, 0x477F), (65408.0, 0x4780),  # 0x477F8000: tie with odd upper half, carries into the exponent
]


@pytest.mark.parametrize("x,bits", R1_HAND)
def test_r1_rounding_hand_values(x, bits):
    assert api.round_bf16(x) == bits


def test_r1_rounding_through_rope_matches_fp64_output():
    # the bits the RoPE emits are the scalar rounding of the fp64 values it reports, and both agree with an
    # independent integer formulation of the two-step rounding, on a few thousand roped elements
    w = inputs.Workload("t", 40, 1, 0, 0, 3, 3, 32, 1e6, False, 77)
    q, _, _ = inputs.make_qkv(w)
    out, f64 = api.rope(q, 1e6, first_pos=50000, want_f64=True)
    flat_bits, flat = out.reshape(-1), f64.reshape(-1)
    assert flat.size >= 3000
    f32_words = flat.astype(np.float32).view(np.uint32).astype(np.uint64)    # step 1 by numpy's cast (RNE)
    low, upper = f32_words & 0xFFFF, f32_words >> 16
    up = (low > 0x8000) | ((low == 0x8000) & ((upper & 1) == 1))             # step 2 spelled out as a comparison
    expect = ((upper + up.astype(np.uint64)) & 0xFFFF).astype(np.uint16)
    np.testing.assert_array_equal(flat_bits, expect)
    assert up.sum() > 1000 and (~up).sum() > 1000                           # both directions occur
    for i in range(0, flat.size, 97):
        assert api.round_bf16(float(flat[i])) == int(flat_bits[i])
    # position 0 is the identity on fp64, so bf16 inputs come back bit for bit (no rounding error at all)
    mrope_bits = api.rope_mrope(q, 1e6, np.zeros((3, 40), dtype=np.int64), (4, 6, 6))
    np.testing.assert_array_equal(mrope_bits, q)


def test_p7_rope_position_zero_identity_and_norm():
    w = inputs.Workload("t", 16, 1, 0, 0, 3, 3, 16, 1e6, False, 9)
    q, _, _ = inputs.make_qkv(w)
    out0 = api.rope(q, 1e6, pos=np.zeros(16, dtype=np.int64))
    np.testing.assert_array_equal(out0, q)
    _, f64 = api.rope(q, 1e6, first_pos=50000, want_f64=True)
    x = dense.bits_to_f64(q)
    h = 8
    np.testing.assert_allclose(f64[..., :h] ** 2 + f64[..., h:] ** 2, x[..., :h] ** 2 + x[..., h:] ** 2, rtol=1e-13)


def test_p7_rope_scores_depend_on_relative_position_only():
    d, theta = 16, 1e4
    w = inputs.Workload("t", 12, 1, 0, 0, 1, 1, d, theta, False, 21)
    q, k, _ = inputs.make_qkv(w)
    _, qa = api.rope(q, theta, first_pos=0, want_f64=True)
    _, ka = api.rope(k, theta, first_pos=0, want_f64=True)
    _, qb = api.rope(q, theta, first_pos=4321, want_f64=True)
    _, kb = api.rope(k, theta, first_pos=4321, want_f64=True)
    sa = qa[:, 0, :] @ ka[:, 0, :].T
    sb = qb[:, 0, :] @ kb[:, 0, :].T
    np.testing.assert_allclose(sa, sb, rtol=0, atol=1e-9)
    # closed form: <rope(q,m), rope(k,n)> = sum_i Re[(q_i + i q_{i+d/2}) conj(k_i + i k_{i+d/2}) e^{i(m-n)f_i}]
    x, y = dense.bits_to_f64(q)[:, 0, :], dense.bits_to_f64(k)[:, 0, :]
    f = theta ** (-2.0 * np.arange(d // 2) / d)
    qc = x[:, :d // 2] + 1j * x[:, d // 2:]
    kc = y[:, :d // 2] + 1j * y[:, d // 2:]
    for m in (0, 5, 11):
        for n in (0, 3, 11):
            ref = np.real(qc[m] * np.conj(kc[n]) * np.exp(1j * (m - n) * f)).sum()
            assert abs(sa[m, n] - ref) < 1e-12


def test_p7_huge_theta_rotates_only_first_pair():
    d = 8
    w = inputs.Workload("t", 4, 1, 0, 0, 1, 1, d, 1e300, False, 2)
    q, _, _ = inputs.make_qkv(w)
    _, f64 = api.rope(q, 1e300, first_pos=3, want_f64=True)
    x = dense.bits_to_f64(q)
    keep = [1, 2, 3, 5, 6, 7]
    np.testing.assert_allclose(f64[..., keep], x[..., keep], rtol=0, atol=1e-60)
    assert np.abs(f64[..., [0, 4]] - x[..., [0, 4]]).max() > 1e-3


def test_p7_mrope_reduces_to_rope_and_uses_the_right_component():
    # three equal components: bit-identical to plain RoPE at those positions
    w = inputs.Workload("t", 9, 1, 0, 0, 2, 2, 16, 1e6, False, 4)
    q, _, _ = inputs.make_qkv(w)
    pos = np.array([0, 5, 77, 1234, 70000, 3, 3, 9, 12], dtype=np.int64)
    np.testing.assert_array_equal(api.rope_mrope(q, 1e6, np.stack([pos, pos, pos]), [3, 3, 2]), api.rope(q, 1e6, pos=pos))
    # d = 4, sections [1, 1, 0]: pair (0,2) turns by the temporal position, pair (1,3) by the height position
    # times theta^(-1/2) = 0.01; hand values with cos(1), sin(1)
    x = _bits([1.0, 1.0, 0.0, 0.0]).reshape(1, 1, 4)
    _, f64 = api.rope_mrope(x, 1e4, np.array([[1], [100], [555]]), [1, 1, 0], want_f64=True)
    np.testing.assert_allclose(f64[0, 0], [COS1, COS1, SIN1, SIN1], rtol=0, atol=1e-15)
    # sections [0, 1, 1]: pair 0 by height (angle 100: not cos 1), pair 1 by width 100 * 0.01 = 1
    _, f64 = api.rope_mrope(x, 1e4, np.array([[1], [100], [100]]), [0, 1, 1], want_f64=True)
    np.testing.assert_allclose(f64[0, 0, [1, 3]], [COS1, SIN1], rtol=0, atol=1e-15)
    np.testing.assert_allclose(f64[0, 0, [0, 2]], [math.cos(100.0), math.sin(100.0)], rtol=0, atol=1e-14)


# ---- P8: LSE merge of key-range partials reproduces the unsplit result ---------------

@pytest.mark.parametrize("cuts", [[0, 9, 20, 31], [0, 31], [0, 0, 5, 5, 31], [0, 1, 2, 30, 31, 40]])
def test_p8_merge_equals_unsplit(cuts):
    S, B, N, Q, Hq, Hkv, d = 6, 5, 4, 5, 4, 2, 8
    w, _, _, v, qr, kr = small_stream(S, B, N, Q, Hq, Hkv, d)
    sh = api.make_shape(S, B, N, Q, Hq, Hkv, d)
    rows = np.arange(S + N * B, w.L, dtype=np.int64)           # question rows
    o_full, lse_full = api.attn_rows(sh, qr, kr, v, rows)
    parts_o, parts_l = [], []
    for a, e in zip(cuts[:-1], cuts[1:]):
        o, l = api.attn_rows(sh, qr, kr, v, rows, key_lo=a, key_hi=e)
        parts_o.append(o.reshape(-1, d))
        parts_l.append(l.reshape(-1))
    o_m, lse_m = api.merge_lse(np.stack(parts_o), np.stack(parts_l))
    np.testing.assert_allclose(o_m.reshape(o_full.shape), o_full, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse_m.reshape(lse_full.shape), lse_full, rtol=0, atol=1e-12)


def test_p8_merge_all_empty_is_minus_inf():
    o, lse = api.merge_lse(np.zeros((2, 3, 4)), np.full((2, 3), -np.inf))
    assert np.isneginf(lse).all() and (o == 0).all()


# ---- P9: literal triple loop on a tiny shape (Eq. 1, Eq. 3-5) ------------------------

def _literal(S, B, N, Q, Hq, Hkv, d, q, k, v, B_last=0):
    nv = S + (N - 1) * B + (B_last or B) if N > 0 else S
    L = nv + Q
    G = Hq // Hkv
    o = [[[0.0] * d for _ in range(Hq)] for _ in range(L)]
    lse = [[0.0] * Hq for _ in range(L)]
    for t in range(L):
        if t < S:
            keys = [j for j in range(S) if j <= t]                          # Eq. 3
        elif t < nv:
            i = (t - S) // B
            own = range(S + i * B, min(S + (i + 1) * B, nv))
            keys = list(range(S)) + [j for j in own if j <= t]              # Eq. 4
        else:
            keys = [j for j in range(L) if j <= t]                          # Eq. 5
        for h in range(Hq):
            g = h // G
            sc = [sum(q[t][h][c] * k[j][g][c] for c in range(d)) / math.sqrt(d) for j in keys]
            z = sum(math.exp(x) for x in sc)
            lse[t][h] = math.log(z)
            for c in range(d):
                o[t][h][c] = sum(math.exp(x) / z * v[j][g][c] for x, j in zip(sc, keys))
    return np.array(o), np.array(lse)


@pytest.mark.parametrize("S,B,N,Q,Hq,Hkv,d,B_last", [(3, 4, 2, 2, 2, 1, 4, 0), (2, 3, 3, 1, 4, 2, 2, 0),
                                                     (3, 4, 3, 2, 2, 1, 4, 2)])
def test_p9_literal_loops(S, B, N, Q, Hq, Hkv, d, B_last):
    w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, 1e4, False, 11, B_last=B_last)
    _, k, v = inputs.make_qkv(w)
    qr, kr = api.rope(inputs.make_qkv(w)[0], 1e4), api.rope(k, 1e4)
    o, lse = api.attn_rows(api.make_shape(S, B, N, Q, Hq, Hkv, d, B_last=B_last), qr, kr, v, all_rows(w.L))
    o_ref, lse_ref = _literal(S, B, N, Q, Hq, Hkv, d, dense.bits_to_f64(qr).tolist(),
                              dense.bits_to_f64(kr).tolist(), dense.bits_to_f64(v).tolist(), B_last)
    np.testing.assert_allclose(o, o_ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref, rtol=0, atol=1e-12)
    # first row sees one key: O = V[0], LSE = its score
    vf, qf, kf = dense.bits_to_f64(v), dense.bits_to_f64(qr), dense.bits_to_f64(kr)
    G = Hq // Hkv
    for h in range(Hq):
        np.testing.assert_allclose(o[0, h], vf[0, h // G], rtol=0, atol=1e-15)
        assert abs(lse[0, h] - (qf[0, h] @ kf[0, h // G]) / math.sqrt(d)) < 1e-14


# ---- KV assembly and sampling helpers -------------------------------------------------

def test_assemble_kv_is_concatenation():
    S, B, N, Q, Hkv, d = 3, 2, 2, 2, 2, 4
    w = inputs.Workload("t", S, B, N, Q, 2, Hkv, d, 1e4, False, 1)
    _, k, _ = inputs.make_qkv(w)
    nv = S + N * B
    cache = api.assemble_kv(api.make_shape(S, B, N, Q, 2, Hkv, d), k[:nv], k[nv:])
    np.testing.assert_array_equal(cache, np.concatenate([k[:nv], k[nv:]], axis=0))


def test_inputs_are_chunk_consistent_and_outliers_applied():
    a = inputs.normal_bf16(5, 2, 5000, 2, 4)
    b = inputs.normal_bf16(5, 2, 300, 2, 4, first_token=4000)
    np.testing.assert_array_equal(a[4000:4300], b)
    w = inputs.WORKLOADS["c2_qwen"].with_(N=0, Q=0)
    _, k, _ = inputs.make_qkv(w)
    kf = inputs.bf16_bits_to_f32(k)
    assert kf[:4].std() > 6 and abs(kf[4:].std() - 1) < 0.05
    rows = inputs.sample_rows(inputs.WORKLOADS["c1_tiny"], 10)
    assert rows.max() < 608 and set(range(576, 608)) <= set(rows.tolist())
