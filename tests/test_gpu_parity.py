"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the
same seeded inputs.  Tolerances: 2e-2 max-abs on outputs, 1e-3 on per-row LSE; RoPE and the
KV assembly are compared bit for bit."""
import numpy as np
import pytest

from oracle import api as oracle
from paper_2506_19651_b200 import inputs
from helpers import (LSE_TOL, O_TOL, bits_to_f64, check_against_oracle, gpu_shape, run_gpu_layer, to_bits, to_dev)

pytestmark = pytest.mark.gpu


def wl(S, B, N, Q, Hq, Hkv, d, theta=1e6, outliers=False, seed=1234):
    return inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, theta, outliers, seed)


# ---------------------------------------------------------------- RoPE (Sec. 3.2.2)

@pytest.mark.parametrize("n,Hq,Hkv,d,theta,first", [
    (37, 4, 2, 64, 1e4, 0), (130, 28, 4, 128, 1e6, 0), (65, 8, 8, 128, 1e6, 70000), (5, 2, 1, 64, 1e6, 123456)])
def test_rope_bit_exact(n, Hq, Hkv, d, theta, first):
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(n, 1, 0, 0, Hq, Hkv, d, theta)
    q, k, _ = inputs.make_qkv(w)
    s = gpu_shape(w)
    qd, kd = to_dev(q), to_dev(k)
    qo, ko = torch.empty_like(qd), torch.empty_like(kd)
    pb.pevlm_rope_qk(s, qd, kd, qo, ko, first, n)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_bits(qo), oracle.rope(q, theta, first_pos=first))
    np.testing.assert_array_equal(to_bits(ko), oracle.rope(k, theta, first_pos=first))
    # in place, K only, explicit position ids
    pos = np.random.default_rng(0).integers(0, 80000, size=n).astype(np.int32)
    pb.pevlm_rope_qk(s, None, kd, None, kd, 0, n, torch.from_numpy(pos).cuda())
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_bits(kd), oracle.rope(k, theta, pos=pos.astype(np.int64)))
    np.testing.assert_array_equal(to_bits(qd), q)  # untouched


def test_rope_bit_exact_on_edge_values():
    """Zeros of both signs, the smallest and largest finite bf16 values and subnormals in every position of a
    rotation pair: the kernel widens bf16 to fp64 with integer arithmetic on the common path and must still
    agree with the oracle bit for bit."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    special = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x0080, 0x8080, 0x7F7F, 0xFF7F, 0x3F80, 0xBF80,
                        0x0100, 0x3F81, 0x4049, 0x00FF, 0x7F00], dtype=np.uint16)
    n, Hq, Hkv, d = 64, 4, 2, 128
    rng = np.random.default_rng(11)
    q = special[rng.integers(0, special.size, size=(n, Hq, d))]
    k = special[rng.integers(0, special.size, size=(n, Hkv, d))]
    w = wl(n, 1, 0, 0, Hq, Hkv, d, 1e6)
    s = gpu_shape(w)
    qd, kd = to_dev(q), to_dev(k)
    qo, ko = torch.empty_like(qd), torch.empty_like(kd)
    pb.pevlm_rope_qk(s, qd, kd, qo, ko, 12345, n)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_bits(qo), oracle.rope(q, 1e6, first_pos=12345))
    np.testing.assert_array_equal(to_bits(ko), oracle.rope(k, 1e6, first_pos=12345))


# ---------------------------------------------------------------- KV assembly (Eq. 5 key set)

def test_assemble_kv_bit_exact():
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(100, 77, 3, 19, 4, 2, 64)
    _, k, v = inputs.make_qkv(w)
    nv = w.n_video
    s = gpu_shape(w)
    kc = torch.zeros((w.L, w.Hkv, w.d), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    pb.pevlm_assemble_kv(s, to_dev(k[:nv]), to_dev(v[:nv]), to_dev(k[nv:]), to_dev(v[nv:]), kc, vc)
    torch.cuda.synchronize()
    sh = oracle.make_shape(w.S, w.B, w.N, w.Q, w.Hq, w.Hkv, w.d)
    np.testing.assert_array_equal(to_bits(kc), oracle.assemble_kv(sh, k[:nv], k[nv:]))
    np.testing.assert_array_equal(to_bits(vc), oracle.assemble_kv(sh, v[:nv], v[nv:]))
    # partial call: only the question V rows
    vc.zero_()
    pb.pevlm_assemble_kv(s, None, None, None, to_dev(v[nv:]), kc, vc)
    torch.cuda.synchronize()
    got = to_bits(vc)
    np.testing.assert_array_equal(got[nv:], v[nv:])
    assert (got[:nv] == 0).all()


# ---------------------------------------------------------------- whole path, small shapes

SMALL = [
    # S, B, N, Q, Hq, Hkv, d, theta, outliers
    (64, 128, 4, 32, 4, 2, 64, 1e4, False),      # the tiny correctness configuration
    (200, 300, 3, 20, 4, 2, 128, 1e6, True),     # several tiles, ragged tails, outlier sink keys
    (16, 16, 5, 3, 2, 1, 128, 1e6, False),       # everything smaller than a tile
    (0, 150, 2, 9, 7, 1, 128, 1e6, False),       # no sink (block attention without sink), G = 7
    (129, 1, 3, 1, 2, 2, 64, 1e4, False),        # blocks of one token
    (257, 384, 2, 130, 8, 2, 128, 1e6, True),    # question longer than a tile's worth of tokens
    (130, 0, 0, 0, 4, 4, 128, 1e6, False),       # sink only
    (700, 900, 3, 70, 8, 2, 64, 1e6, True),      # head_dim 64 over many tiles: 6 sink + up to 8 block key tiles per item
    (100, 100, 1, 4800, 8, 8, 64, 1e6, True),    # a question block so long that its tiles alone exceed the SM count:
                                                 # one key split, more work items than CTAs in the question launch
    (0, 0, 0, 40, 4, 2, 64, 1e4, False),         # question only
]


@pytest.mark.parametrize("S,B,N,Q,Hq,Hkv,d,theta,outl", SMALL)
def test_layer_matches_oracle_small(S, B, N, Q, Hq, Hkv, d, theta, outl):
    w = wl(S, B, N, Q, Hq, Hkv, d, theta, outl)
    q, k, v = inputs.make_qkv(w)
    res = run_gpu_layer(w, q, k, v)
    errs, qr, kr = check_against_oracle(w, q, k, v, res, np.arange(w.L))
    nv = w.n_video
    # RoPE outputs and the assembled cache, bit for bit
    np.testing.assert_array_equal(res["q_video"], qr[:nv])
    np.testing.assert_array_equal(res["q_question"], qr[nv:])
    np.testing.assert_array_equal(res["k_cache"], kr)
    np.testing.assert_array_equal(res["v_cache"], v)
    for name, e in errs.items():
        assert e <= (LSE_TOL if name.startswith("lse") else O_TOL), (name, e, errs)


@pytest.mark.parametrize("S,B,N,Q,Hq,Hkv,d", [(100, 200, 2, 10, 4, 2, 128), (64, 128, 4, 32, 4, 2, 64)])
def test_full_causal_mode_matches_oracle(S, B, N, Q, Hq, Hkv, d):
    w = wl(S, B, N, Q, Hq, Hkv, d)
    q, k, v = inputs.make_qkv(w)
    res = run_gpu_layer(w, q, k, v, full_causal=True)
    errs, _, _ = check_against_oracle(w, q, k, v, res, np.arange(w.L), full_causal=True)
    for name, e in errs.items():
        assert e <= (LSE_TOL if name.startswith("lse") else O_TOL), (name, e, errs)


def test_run_twice_is_bit_identical():
    w = wl(200, 300, 3, 20, 4, 2, 128, outliers=True)
    q, k, v = inputs.make_qkv(w)
    a = run_gpu_layer(w, q, k, v)
    b = run_gpu_layer(w, q, k, v)
    for name in ("o_video", "lse_video", "o_question", "lse_question"):
        np.testing.assert_array_equal(a[name], b[name])


def test_softmax_scale_and_null_lse():
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(70, 90, 2, 0, 2, 1, 64, 1e4)
    q, k, v = inputs.make_qkv(w)
    qr, kr = oracle.rope(q, w.theta), oracle.rope(k, w.theta)
    s = gpu_shape(w, scale=0.3)
    o = torch.empty((w.L, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
    pb.pevlm_parallel_prefill_attn(s, to_dev(qr), to_dev(kr), to_dev(v), o, None, ws)
    torch.cuda.synchronize()
    ref, _ = oracle.attn_rows(oracle.make_shape(w.S, w.B, w.N, 0, w.Hq, w.Hkv, w.d), qr, kr, v, np.arange(w.L), scale=0.3)
    assert np.abs(bits_to_f64(to_bits(o)) - ref).max() <= O_TOL


# ---------------------------------------------------------------- full-size workloads, sampled rows

def assert_rope_bits(got, want, allowed):
    """Bit-exact up to `allowed` elements, and each of those off by exactly one bf16 ulp (neighbouring bit
    patterns of the same sign): the device's and the host libm's fp64 sin/cos may differ in the last place,
    which after the rounding to bf16 flips about one element in 1e8."""
    bad = np.flatnonzero(got.reshape(-1) != want.reshape(-1))
    assert bad.size <= allowed, bad.size
    for i in bad:
        a, b = int(got.reshape(-1)[i]), int(want.reshape(-1)[i])
        assert abs(a - b) == 1 and (a >> 15) == (b >> 15), (hex(a), hex(b))


@pytest.mark.parametrize("name,n_random", [("c2_qwen", None), ("c3_long", 2000)])
def test_full_size_sampled_rows(name, n_random):
    """c2_qwen: EVERY row of the layer; c3_long: the edges of every block and tile, the question block and
    2,000 random rows."""
    w = inputs.WORKLOADS[name]
    q, k, v = inputs.make_qkv(w)
    res = run_gpu_layer(w, q, k, v)
    rows = np.arange(w.L) if n_random is None else inputs.sample_rows(w, n_random)
    errs, qr, kr = check_against_oracle(w, q, k, v, res, rows)
    assert_rope_bits(res["q_video"], qr[:w.n_video], 4)
    assert_rope_bits(res["k_cache"], kr, 2)
    np.testing.assert_array_equal(res["v_cache"], v)
    for key, e in errs.items():
        assert e <= (LSE_TOL if key.startswith("lse") else O_TOL), (key, e, errs)


# ---------------------------------------------------------------- batch > 1 (independent sequences)

def test_batch_of_two_sequences():
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(96, 160, 2, 24, 4, 2, 128, outliers=True)
    nv = w.n_video
    seqs = [inputs.make_qkv(w.with_(seed=w.seed + i)) for i in range(2)]
    s = gpu_shape(w)
    s.batch = 2
    cat = lambda idx, sl: to_dev(np.concatenate([seqs[b][idx][sl] for b in range(2)], axis=0))
    q_v, k_v, v_v = cat(0, slice(0, nv)), cat(1, slice(0, nv)), cat(2, slice(0, nv))
    q_q, k_q, v_q = cat(0, slice(nv, None)), cat(1, slice(nv, None)), cat(2, slice(nv, None))
    pb.pevlm_rope_qk(s, q_v, k_v, q_v, k_v, 0, nv)
    pb.pevlm_rope_qk(s, q_q, k_q, q_q, k_q, nv, w.Q)
    kc = torch.empty((2 * w.L, w.Hkv, w.d), dtype=torch.bfloat16, device="cuda")
    vc = torch.empty_like(kc)
    pb.pevlm_assemble_kv(s, k_v, v_v, k_q, v_q, kc, vc)
    o_v = torch.empty_like(q_v)
    lse_v = torch.empty((2, w.Hq, nv), dtype=torch.float32, device="cuda")
    ws = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
    pb.pevlm_parallel_prefill_attn(s, q_v, k_v, v_v, o_v, lse_v, ws)
    o_q = torch.empty_like(q_q)
    lse_q = torch.empty((2, w.Hq, w.Q), dtype=torch.float32, device="cuda")
    wq = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_QUERY), dtype=torch.uint8, device="cuda")
    pb.pevlm_query_attn(s, q_q, kc, vc, o_q, lse_q, wq)
    torch.cuda.synchronize()
    assert pb.pevlm_read_status(ws)[0] == 0 and pb.pevlm_read_status(wq)[0] == 0
    for b in range(2):
        q, k, v = seqs[b]
        qr, kr = oracle.rope(q, w.theta), oracle.rope(k, w.theta)
        np.testing.assert_array_equal(to_bits(kc[b * w.L:(b + 1) * w.L]), kr)
        np.testing.assert_array_equal(to_bits(vc[b * w.L:(b + 1) * w.L]), v)
        sh = oracle.make_shape(w.S, w.B, w.N, w.Q, w.Hq, w.Hkv, w.d)
        o_ref, lse_ref = oracle.attn_rows(sh, qr, kr, v, np.arange(w.L))
        got_o = np.concatenate([bits_to_f64(to_bits(o_v[b * nv:(b + 1) * nv])), bits_to_f64(to_bits(o_q[b * w.Q:(b + 1) * w.Q]))])
        got_l = np.concatenate([lse_v[b].double().cpu().numpy().T, lse_q[b].double().cpu().numpy().T])
        assert np.abs(got_o - o_ref).max() <= O_TOL
        assert np.abs(got_l - lse_ref).max() <= LSE_TOL


# ---------------------------------------------------------------- the other full-size configurations

@pytest.mark.parametrize("name,layer,n_random", [
    ("c4_sweep_F1", 0, 2000), ("c4_sweep_F2", 0, 1000), ("c4_sweep_F4", 0, 1000), ("c4_sweep_F8", 0, 1000),
    ("c4_sweep_F16", 0, 600), ("c4_sweep_F32", 0, 400),
    ("c5_stack", 0, 2000), ("c5_stack", 13, 2000), ("c5_stack", 27, 2000)])
def test_sweep_and_stack_sampled_rows(name, layer, n_random):
    """Every point of the block-size sweep (1 to 32 query tiles per block: the whole range of the work-item
    ordering rules) and three layers of the 28-layer stack: block and tile edges of every block, the question
    block, and seeded random rows."""
    w = inputs.WORKLOADS[name]
    q, k, v = inputs.make_qkv(w, layer=layer)
    res = run_gpu_layer(w, q, k, v)
    rows = inputs.sample_rows(w, n_random)
    errs, qr, kr = check_against_oracle(w, q, k, v, res, rows)
    assert_rope_bits(res["k_cache"], kr, 2)
    assert_rope_bits(res["q_video"], qr[:w.n_video], 4)
    for key, e in errs.items():
        assert e <= (LSE_TOL if key.startswith("lse") else O_TOL), (key, e, errs)


def test_full_causal_mode_full_size_sampled_rows():
    # the speed-up baseline: plain causal attention over the 12,544 video tokens of the Qwen-shaped layer
    w = inputs.WORKLOADS["c2_qwen"]
    q, k, v = inputs.make_qkv(w)
    res = run_gpu_layer(w, q, k, v, full_causal=True)
    rows = inputs.sample_rows(w, 100)
    errs, _, _ = check_against_oracle(w, q, k, v, res, rows[rows < w.n_video], full_causal=True)
    for key, e in errs.items():
        assert e <= (LSE_TOL if key.startswith("lse") else O_TOL), (key, e, errs)


# ---------------------------------------------------------------- position and mask variants (no new kernels)

def test_reused_positions_per_block_variant():
    """The comparison the paper draws in Sec. 3.2.2 / Sec. 5.1: positions restarting in every block (what
    prior parallel-encoding methods do) instead of sequential ones.  Only the position ids change."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(96, 160, 3, 0, 4, 2, 128)
    q, k, v = inputs.make_qkv(w)
    t = np.arange(w.L)
    pos = np.where(t < w.S, t, w.S + (t - w.S) % w.B).astype(np.int32)      # every block restarts after the sink
    s = gpu_shape(w)
    qd, kd = to_dev(q), to_dev(k)
    pb.pevlm_rope_qk(s, qd, kd, qd, kd, 0, w.L, torch.from_numpy(pos).cuda())
    o = torch.empty_like(qd)
    lse = torch.empty((w.Hq, w.L), dtype=torch.float32, device="cuda")
    ws = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
    pb.pevlm_parallel_prefill_attn(s, qd, kd, to_dev(v), o, lse, ws)
    torch.cuda.synchronize()
    qr, kr = oracle.rope(q, w.theta, pos=pos.astype(np.int64)), oracle.rope(k, w.theta, pos=pos.astype(np.int64))
    np.testing.assert_array_equal(to_bits(qd), qr)
    o_ref, lse_ref = oracle.attn_rows(oracle.make_shape(w.S, w.B, w.N, 0, w.Hq, w.Hkv, w.d), qr, kr, v, np.arange(w.L))
    assert np.abs(bits_to_f64(to_bits(o)) - o_ref).max() <= O_TOL
    assert np.abs(lse.double().cpu().numpy().T - lse_ref).max() <= LSE_TOL
    # and it differs from the sequential-position result on the context rows (the method's point)
    o_seq, _ = oracle.attn_rows(oracle.make_shape(w.S, w.B, w.N, 0, w.Hq, w.Hkv, w.d), oracle.rope(q, w.theta),
                                oracle.rope(k, w.theta), v, np.arange(w.S + w.B, w.L))
    assert np.abs(o_seq - o_ref[w.S + w.B:]).max() > 1e-2


@pytest.mark.parametrize("Q", [1, 2, 5])
def test_decode_sized_question_blocks(Q):
    """A few new rows against the assembled cache (the step after prefill): the question attention with
    1 to 5 query tokens, i.e. 7 to 35 rows of a 128-row tile."""
    w = wl(300, 260, 3, Q, 28, 4, 128, outliers=True)
    q, k, v = inputs.make_qkv(w)
    res = run_gpu_layer(w, q, k, v)
    errs, _, _ = check_against_oracle(w, q, k, v, res, np.arange(w.n_video, w.L))
    for key, e in errs.items():
        assert e <= (LSE_TOL if key.startswith("lse") else O_TOL), (key, e, errs)


# ---------------------------------------------------------------- multimodal RoPE (three position components)

@pytest.mark.parametrize("n,Hq,Hkv,d,sections", [(300, 28, 4, 128, (16, 24, 24)), (77, 4, 2, 64, (8, 12, 12)), (5, 2, 2, 128, (64, 0, 0))])
def test_mrope_bit_exact(n, Hq, Hkv, d, sections):
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(n, 1, 0, 0, Hq, Hkv, d, 1e6)
    q, k, _ = inputs.make_qkv(w)
    rng = np.random.default_rng(5)
    # a video-like id grid: temporal id per frame, height/width ids inside the frame, all offset by a text prefix
    t_id = 40 + np.arange(n) // 16
    pos3 = np.stack([t_id, 40 + (np.arange(n) % 16) // 4, 40 + np.arange(n) % 4]).astype(np.int32)
    pos3[:, :3] = rng.integers(0, 70000, size=(1, 3))            # text tokens: equal components, large values
    s = gpu_shape(w)
    qd, kd = to_dev(q), to_dev(k)
    qo, ko = torch.empty_like(qd), torch.empty_like(kd)
    pb.pevlm_rope_qk_mrope(s, qd, kd, qo, ko, n, torch.from_numpy(pos3).cuda(), sections)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_bits(qo), oracle.rope_mrope(q, 1e6, pos3, sections))
    np.testing.assert_array_equal(to_bits(ko), oracle.rope_mrope(k, 1e6, pos3, sections))


# ---------------------------------------------------------------- many launches: no expired wait, identical results

@pytest.mark.parametrize("S,B,N,Q,Hq,Hkv,d", [(64, 64, 40, 5, 14, 2, 128), (200, 300, 9, 17, 8, 2, 128), (0, 512, 6, 64, 28, 4, 128)])
def test_many_launches_identical(S, B, N, Q, Hq, Hkv, d):
    """The persistent kernel hands work out through an atomic counter, so which CTA runs which item differs from
    launch to launch; every item's arithmetic does not.  500 layer passes: status word clear, bit-identical outputs."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    from paper_2506_19651_b200.layer import LayerBuffers, layer_forward
    w = wl(S, B, N, Q, Hq, Hkv, d, outliers=S > 0)
    q, k, v = (to_dev(a) for a in inputs.make_qkv(w))
    buf = LayerBuffers(gpu_shape(w))
    ref = None
    for i in range(500):
        layer_forward(buf, q, k, v)
        if i % 100 == 99 or i == 0:
            torch.cuda.synchronize()
            for ws in (buf.ws_prefill, buf.ws_query):
                st, det = pb.pevlm_read_status(ws)
                assert st == 0, (i, st, det)
            got = (to_bits(buf.o_video).copy(), buf.lse_video.cpu().numpy().copy(), to_bits(buf.o_question).copy())
            if ref is None:
                ref = got
            for a, b in zip(got, ref):
                np.testing.assert_array_equal(a, b)


# ---------------------------------------------------------------- failure path: a bounded wait that runs out

def test_bounded_wait_expires_and_the_context_stays_usable():
    """One thread block waits, with the library's bounded wait, on a barrier nothing arrives on; the wait
    gives up after 1 ms, the kernel ends normally and reports PEVLM_ETIMEOUT with the id of the wait through
    the workspace header.  A normal call on the same workspace then clears the status and is correct."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(70, 90, 2, 0, 2, 1, 64, 1e4)
    s = gpu_shape(w)
    ws = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    pb.pevlm_selftest_wait_expiry(ws, 1_000_000)
    t1.record()
    st, det = pb.pevlm_read_status(ws)
    assert st == pb.PEVLM_ETIMEOUT and det == 99 * 1000000, (st, det)
    assert 0.9 <= t0.elapsed_time(t1) <= 50.0        # the limit, then the short grace period of the second wait
    q, k, v = inputs.make_qkv(w)
    qr, kr = oracle.rope(q, w.theta), oracle.rope(k, w.theta)
    o = torch.empty((w.L, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.Hq, w.L), dtype=torch.float32, device="cuda")
    pb.pevlm_parallel_prefill_attn(s, to_dev(qr), to_dev(kr), to_dev(v), o, lse, ws)
    assert pb.pevlm_read_status(ws) == (0, 0)
    ref, lref = oracle.attn_rows(oracle.make_shape(w.S, w.B, w.N, 0, w.Hq, w.Hkv, w.d), qr, kr, v, np.arange(w.L))
    assert np.abs(bits_to_f64(to_bits(o)) - ref).max() <= O_TOL
    assert np.abs(lse.double().cpu().numpy().T - lref).max() <= LSE_TOL


# ---------------------------------------------------------------- seeded random shapes (all rows, canary bytes)

def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        d = int(rng.choice([64, 128]))
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 3, 4, 7, 8]))
        S = int(rng.choice([0, int(rng.integers(1, 40)), int(rng.integers(40, 300)), 128, 256]))
        N = int(rng.integers(0, 5))
        B = int(rng.choice([int(rng.integers(1, 20)), int(rng.integers(20, 400)), 128, 192])) if N > 0 else 0
        Q = int(rng.choice([0, 1, int(rng.integers(2, 70))]))
        if S + N * B + Q == 0:
            S = 17
        out.append((S, B, N, Q, Hkv * G, Hkv, d, bool(rng.integers(0, 2)) and S > 0))
    return out


@pytest.mark.parametrize("S,B,N,Q,Hq,Hkv,d,outl", _random_shapes(40, seed=20250619))
def test_random_shapes_match_oracle(S, B, N, Q, Hq, Hkv, d, outl):
    """Forty seeded shapes drawn over the ranges where the tiling changes form (segments shorter than a tile,
    ragged tails that are or are not packed across the heads of a group, group sizes 1 to 8, both head
    dimensions, empty sink / no blocks / no question): every row against the oracle, RoPE and cache bit for bit,
    canary bytes around every buffer (inside run_gpu_layer)."""
    w = wl(S, B, N, Q, Hq, Hkv, d, 1e6, outl, seed=4242 + S + 7 * B + 13 * N + Q)
    q, k, v = inputs.make_qkv(w)
    res = run_gpu_layer(w, q, k, v)
    errs, qr, kr = check_against_oracle(w, q, k, v, res, np.arange(w.L))
    nv = w.n_video
    np.testing.assert_array_equal(res["q_video"], qr[:nv])
    np.testing.assert_array_equal(res["q_question"], qr[nv:])
    np.testing.assert_array_equal(res["k_cache"], kr)
    np.testing.assert_array_equal(res["v_cache"], v)
    for name, e in errs.items():
        assert e <= (LSE_TOL if name.startswith("lse") else O_TOL), (name, e, errs)


# ---------------------------------------------------------------- the rare in-place rescale of the accumulator

@pytest.mark.parametrize("S,B,N,Q,Hq,Hkv,d", [(300, 400, 2, 40, 8, 2, 128), (140, 520, 1, 9, 4, 2, 64)])
def test_late_outlier_keys_force_the_accumulator_rescale(S, B, N, Q, Hq, Hkv, d):
    """The kernel moves a row's reference maximum only when the maximum grows by more than 2^8 and then rescales
    the row of the output accumulator in place.  With N(0,1) inputs, or outliers among the first sink keys only,
    that never happens after a row's first key tile.  Here key rows late in the sink, in the middle of the blocks
    and in the question are scaled by 12 to 40, so the reference maximum jumps in the 2nd, 3rd, ... key tile of
    rows that follow them (several times for some rows).  Every row against the oracle."""
    w = wl(S, B, N, Q, Hq, Hkv, d, 1e6, False, seed=31337)
    late = {S - 7: 12.0, S - 1: 25.0, S + 5: 16.0, S + 131: 30.0, S + B // 2: 20.0, S + B - 2: 40.0}
    if N > 1:
        late.update({S + B + 129: 18.0, S + B + 300: 35.0})
    late.update({w.n_video + Q // 2: 28.0})
    q = inputs.normal_bf16(w.seed, 1, w.L, Hq, d)
    k = inputs.normal_bf16(w.seed, 2, w.L, Hkv, d, scale_rows=late)
    v = inputs.normal_bf16(w.seed, 3, w.L, Hkv, d)
    res = run_gpu_layer(w, q, k, v)
    errs, qr, kr = check_against_oracle(w, q, k, v, res, np.arange(w.L))
    np.testing.assert_array_equal(res["k_cache"], kr)
    for name, e in errs.items():
        assert e <= (LSE_TOL if name.startswith("lse") else O_TOL), (name, e, errs)


# ---------------------------------------------------------------- RoPE, long-range form of every instantiation

@pytest.mark.parametrize("n,Hq,Hkv,d,sections", [
    (40000, 2, 1, 64, None),                # plain positions, head_dim 64
    (10000, 3, 1, 128, (16, 24, 24)),       # multimodal, section boundaries on multiples of 8 pairs
    (10000, 3, 1, 128, (10, 27, 27)),       # multimodal, a position component per pair
    (40000, 2, 1, 64, (8, 12, 12)),         # multimodal at head_dim 64
])
def test_rope_long_range_forms_bit_exact(n, Hq, Hkv, d, sections):
    """Token ranges long enough for the RoPE launch to take its long-range form (pairs in shared memory, loads
    issued ahead), for each instantiation the full-size layer tests do not reach: bit for bit against the oracle."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    w = wl(n, 1, 0, 0, Hq, Hkv, d, 1e6, seed=808)
    q, k, _ = inputs.make_qkv(w)
    s = gpu_shape(w)
    qd, kd = to_dev(q), to_dev(k)
    qo, ko = torch.empty_like(qd), torch.empty_like(kd)
    if sections is None:
        pb.pevlm_rope_qk(s, qd, kd, qo, ko, 1000, n)
        want_q, want_k = oracle.rope(q, 1e6, first_pos=1000), oracle.rope(k, 1e6, first_pos=1000)
    else:
        idx = np.arange(n)
        pos3 = np.stack([50 + idx // 256, 50 + (idx % 256) // 16, 50 + idx % 16]).astype(np.int32)
        pb.pevlm_rope_qk_mrope(s, qd, kd, qo, ko, n, torch.from_numpy(pos3).cuda(), sections)
        want_q, want_k = oracle.rope_mrope(q, 1e6, pos3, sections), oracle.rope_mrope(k, 1e6, pos3, sections)
    torch.cuda.synchronize()
    assert_rope_bits(to_bits(qo), want_q, 1)
    assert_rope_bits(to_bits(ko), want_k, 1)
