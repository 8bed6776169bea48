"""GPU parity of the block-range attention call and of what is composed from it: a shorter last context
block, and a sliding window of blocks over a fixed sink.  Oracle: the fp64 definition (Eq. 3-5)."""
import numpy as np
import pytest

from oracle import api as oracle
from paper_2506_19651_b200 import inputs
from helpers import LSE_TOL, O_TOL, bits_to_f64, to_bits, to_dev

pytestmark = pytest.mark.gpu


def _status_ok(*workspaces):
    from paper_2506_19651_b200 import binding as pb
    for ws in workspaces:
        st, det = pb.pevlm_read_status(ws)
        assert st == 0, f"device wait expired: status {st} detail {det}"


@pytest.mark.parametrize("S,B,N,Q,B_last,Hq,Hkv,d", [
    (64, 128, 3, 32, 50, 4, 2, 64),        # last block shorter than a tile
    (200, 300, 4, 17, 129, 8, 2, 128),     # ragged everywhere, last block one row past a tile
    (0, 256, 2, 8, 255, 4, 4, 128),        # no sink
    (130, 260, 1, 5, 7, 14, 2, 128),       # the only block is the short one, G = 7 (packed tails)
    (784, 784, 5, 64, 392, 28, 4, 128),    # Qwen-shaped, half a block left over
    (1568, 1568, 31, 128, 980, 28, 4, 128),  # the 50K-token shape with 5 of the last block's 8 frames (sampled rows)
])
def test_ragged_last_block(S, B, N, Q, B_last, Hq, Hkv, d):
    import torch
    from paper_2506_19651_b200.layer import ragged_layer_forward
    theta = 1e6
    w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, theta, S > 0, 4321, B_last=B_last)
    q, k, v = inputs.make_qkv(w)
    from helpers import GuardedAllocator
    guard = GuardedAllocator()
    o_v, lse_v, o_q, lse_q, ws = ragged_layer_forward(to_dev(q), to_dev(k), to_dev(v), S, B, N, B_last, Q, theta, alloc=guard)
    torch.cuda.synchronize()
    _status_ok(*ws)
    guard.check()   # canary bytes around every buffer of the pass, the block-range call's o and lse included
    nv = w.n_video
    qr, kr = oracle.rope(q, theta), oracle.rope(k, theta)
    sh = oracle.make_shape(S, B, N, Q, Hq, Hkv, d, B_last=B_last)
    rows = np.arange(w.L, dtype=np.int64) if w.L <= 1500 else np.unique(np.concatenate([
        np.random.default_rng(5).integers(0, w.L, size=300), np.arange(nv - B_last - 2, w.L)]))
    o, lse = oracle.attn_rows(sh, qr, kr, v, rows)
    vid, que = rows < nv, rows >= nv
    o_gpu = np.concatenate([bits_to_f64(to_bits(o_v)), bits_to_f64(to_bits(o_q[:Q]))])[rows]
    lse_gpu = np.concatenate([lse_v.double().cpu().numpy().T, lse_q[:, :Q].double().cpu().numpy().T])[rows]
    assert np.abs(o_gpu - o).max() <= O_TOL
    assert np.abs(lse_gpu - lse).max() <= LSE_TOL
    assert vid.any() and que.any()


def test_block_range_in_the_middle_of_a_cache():
    """Blocks 1..2 of a 4-block stream recomputed alone from the resident cache equal the rows of the
    whole-stream call bit for bit (same kernel, same tiles), and the oracle within tolerance."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    S, B, N, Hq, Hkv, d, theta = 96, 160, 4, 8, 4, 64, 1e4
    w = inputs.Workload("t", S, B, N, 0, Hq, Hkv, d, theta, False, 99)
    q, k, v = inputs.make_qkv(w)
    nv = w.n_video
    s = pb.make_shape(S, B, N, 0, Hq, Hkv, d, theta=theta)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    pb.pevlm_rope_qk(s, qd, kd, qd, kd, 0, nv)
    o_all = torch.empty_like(qd)
    lse_all = torch.empty((Hq, nv), dtype=torch.float32, device="cuda")
    ws = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
    pb.pevlm_parallel_prefill_attn(s, qd, kd, vd, o_all, lse_all, ws)
    s2 = pb.make_shape(S, B, 2, 0, Hq, Hkv, d, theta=theta)
    lo, hi = S + B, S + 3 * B
    o_mid = torch.empty((2 * B, Hq, d), dtype=torch.bfloat16, device="cuda")
    lse_mid = torch.empty((Hq, 2 * B), dtype=torch.float32, device="cuda")
    ws2 = torch.zeros_like(ws)
    pb.pevlm_block_attn(s2, qd[lo:hi], kd, vd, lo, nv, o_mid, lse_mid, ws2)
    torch.cuda.synchronize()
    _status_ok(ws, ws2)
    np.testing.assert_array_equal(to_bits(o_mid), to_bits(o_all[lo:hi]))
    np.testing.assert_array_equal(lse_mid.cpu().numpy(), lse_all[:, lo:hi].cpu().numpy())
    rows = np.arange(lo, hi, dtype=np.int64)
    o, lse = oracle.attn_rows(oracle.make_shape(S, B, N, 0, Hq, Hkv, d), to_bits(qd), to_bits(kd), v, rows)
    assert np.abs(bits_to_f64(to_bits(o_mid)) - o).max() <= O_TOL
    assert np.abs(lse_mid.double().cpu().numpy().T - lse).max() <= LSE_TOL


def test_block_attn_rejects_bad_ranges():
    import torch
    from paper_2506_19651_b200 import binding as pb
    s = pb.make_shape(64, 128, 1, 0, 4, 2, 64)
    t = torch.zeros((256, 4, 64), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((256, 2, 64), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for first, rows in ((63, 256), (129, 256), (64, 191)):
        with pytest.raises(pb.PevlmError) as e:
            pb.pevlm_block_attn(s, t, kv, kv, first, rows, t, None, ws)
        assert e.value.code == pb.PEVLM_EINVAL
    sf = pb.make_shape(64, 128, 1, 0, 4, 2, 64, mask_mode=pb.MASK_FULL_CAUSAL)
    with pytest.raises(pb.PevlmError):
        pb.pevlm_block_attn(sf, t, kv, kv, 64, 256, t, None, ws)


@pytest.mark.parametrize("S,B,W,T,Q,Hq,Hkv,d", [(100, 200, 3, 7, 9, 4, 2, 64), (256, 384, 2, 3, 40, 14, 2, 128),
                                                (128, 128, 4, 2, 1, 8, 8, 128)])
def test_streaming_window(S, B, W, T, Q, Hq, Hkv, d):
    """T blocks stream through a window of W slots.  Every block's output equals the oracle's Eq. 4 rows on
    [sink | that block] at its global positions; the question equals the oracle's Eq. 5 rows on the stream
    [sink | blocks now in the window, in slot order | question] with the positions carried along."""
    import torch
    from paper_2506_19651_b200.layer import StreamingWindow
    theta = 1e6
    w = inputs.Workload("t", S, B, T, Q, Hq, Hkv, d, theta, True, 777)
    q, k, v = inputs.make_qkv(w)   # the whole stream [sink | T blocks | question], un-roped
    win = StreamingWindow(S, B, W, Q, Hq, Hkv, d, theta)
    o_s, lse_s = win.set_sink(to_dev(q[:S]), to_dev(k[:S]), to_dev(v[:S]))
    outs = []
    for t in range(T):
        a, b = S + t * B, S + (t + 1) * B
        outs.append(win.append_block(to_dev(q[a:b]), to_dev(k[a:b]), to_dev(v[a:b])))
    nv = S + T * B
    o_q, lse_q = win.ask(to_dev(q[nv:]), to_dev(k[nv:]), to_dev(v[nv:]))
    torch.cuda.synchronize()
    _status_ok(win.ws_sink, win.ws_block, win.ws_query)
    qr, kr = oracle.rope(q, theta), oracle.rope(k, theta)   # global sequential positions
    # sink
    o, lse = oracle.attn_rows(oracle.make_shape(S, 1, 0, 0, Hq, Hkv, d), qr[:S], kr[:S], v[:S], np.arange(S, dtype=np.int64))
    assert np.abs(bits_to_f64(to_bits(o_s)) - o).max() <= O_TOL
    assert np.abs(lse_s.double().cpu().numpy().T - lse).max() <= LSE_TOL
    # every block as it arrived
    for t in range(T):
        a, b = S + t * B, S + (t + 1) * B
        idx = np.concatenate([np.arange(S), np.arange(a, b)])
        o, lse = oracle.attn_rows(oracle.make_shape(S, B, 1, 0, Hq, Hkv, d), qr[idx], kr[idx], v[idx],
                                  np.arange(S, S + B, dtype=np.int64))
        assert np.abs(bits_to_f64(to_bits(outs[t][0])) - o).max() <= O_TOL, t
        assert np.abs(outs[t][1].double().cpu().numpy().T - lse).max() <= LSE_TOL, t
    # the question over the window's content, slots in cache order
    held = min(T, W)
    slot_block = {t % W: t for t in range(T)}   # the last writer of each slot
    idx = np.concatenate([np.arange(S)] + [np.arange(S + slot_block[j] * B, S + (slot_block[j] + 1) * B) for j in range(held)] +
                         [np.arange(nv, nv + Q)])
    sh = oracle.make_shape(S, B, held, Q, Hq, Hkv, d)
    o, lse = oracle.attn_rows(sh, qr[idx], kr[idx], v[idx], np.arange(S + held * B, S + held * B + Q, dtype=np.int64))
    assert np.abs(bits_to_f64(to_bits(o_q)) - o).max() <= O_TOL
    assert np.abs(lse_q.double().cpu().numpy().T - lse).max() <= LSE_TOL
    # the cache holds exactly those roped keys
    np.testing.assert_array_equal(to_bits(win.k_cache[:S + held * B + Q]), kr[idx])


def test_sequences_of_different_shapes_share_one_cache_buffer():
    """Per-sequence shapes: three streams with different (S, B, N, Q) packed back to back in one K/V cache buffer,
    one group of calls per stream on slices of the shared buffers, all on one CUDA stream without a sync in between."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    Hq, Hkv, d, theta = 8, 2, 128, 1e6
    seqs = [(64, 128, 3, 8), (96, 160, 2, 5), (0, 256, 2, 4)]
    ws_list, outs, streams = [], [], []
    total = sum(S + N * B + Q for S, B, N, Q in seqs)
    k_cache = torch.zeros((total, Hkv, d), dtype=torch.bfloat16, device="cuda")
    v_cache = torch.zeros_like(k_cache)
    row = 0
    for i, (S, B, N, Q) in enumerate(seqs):
        w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, theta, S > 0, 900 + i)
        q, k, v = inputs.make_qkv(w)
        streams.append((w, q, k, v))
        s = pb.make_shape(S, B, N, Q, Hq, Hkv, d, theta=theta)
        nv, L = w.n_video, w.L
        kc, vc = k_cache[row:row + L], v_cache[row:row + L]
        qd = to_dev(q)
        pb.pevlm_rope_qk(s, qd, to_dev(k), qd, kc, 0, L)
        pb.pevlm_assemble_kv(s, None, to_dev(v[:nv]), None, to_dev(v[nv:]), kc, vc)
        o_v = torch.empty((nv, Hq, d), dtype=torch.bfloat16, device="cuda")
        lse_v = torch.empty((Hq, nv), dtype=torch.float32, device="cuda")
        o_q = torch.empty((Q, Hq, d), dtype=torch.bfloat16, device="cuda")
        lse_q = torch.empty((Hq, Q), dtype=torch.float32, device="cuda")
        ws_p = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
        ws_q = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_QUERY), dtype=torch.uint8, device="cuda")
        pb.pevlm_parallel_prefill_attn(s, qd[:nv], kc[:nv], vc[:nv], o_v, lse_v, ws_p)
        pb.pevlm_query_attn(s, qd[nv:], kc, vc, o_q, lse_q, ws_q)
        ws_list += [ws_p, ws_q]
        outs.append((o_v, lse_v, o_q, lse_q))
        row += L
    torch.cuda.synchronize()
    _status_ok(*ws_list)
    for (w, q, k, v), (o_v, lse_v, o_q, lse_q) in zip(streams, outs):
        qr, kr = oracle.rope(q, theta), oracle.rope(k, theta)
        sh = oracle.make_shape(w.S, w.B, w.N, w.Q, Hq, Hkv, d)
        o, lse = oracle.attn_rows(sh, qr, kr, v, np.arange(w.L, dtype=np.int64))
        o_gpu = np.concatenate([bits_to_f64(to_bits(o_v)), bits_to_f64(to_bits(o_q))])
        lse_gpu = np.concatenate([lse_v.double().cpu().numpy().T, lse_q.double().cpu().numpy().T])
        assert np.abs(o_gpu - o).max() <= O_TOL
        assert np.abs(lse_gpu - lse).max() <= LSE_TOL


@pytest.mark.parametrize("S,B,N,Hq,Hkv,d", [(100, 75, 2, 4, 2, 128), (37, 130, 1, 14, 2, 128), (200, 333, 3, 8, 4, 64)])
def test_block_range_ignores_the_rest_of_the_cache(S, B, N, Hq, Hkv, d):
    """The cache outside the sink rows and the block range holds NaN bit patterns (an uninitialised slot of a
    streaming window); S and B are not multiples of 16, so the ragged last key tiles end inside a 16-row MMA
    step.  The outputs must be those of the oracle (a zero probability times a NaN value row would be NaN),
    and nothing may be written outside o and lse (canary bytes around both)."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    from helpers import GuardedAllocator
    theta = 1e6
    w = inputs.Workload("t", S, B, N, 0, Hq, Hkv, d, theta, True, 555)
    q, k, v = inputs.make_qkv(w)
    qr, kr = oracle.rope(q, theta), oracle.rope(k, theta)
    gap, tail = 53, 91                              # unused rows between the sink and the blocks, and after them
    first = S + gap
    rows = first + N * B + tail
    nan = torch.full((rows, Hkv, d), -1, dtype=torch.int16, device="cuda").view(torch.bfloat16)   # 0xFFFF = NaN
    kc, vc = nan.clone(), nan.clone()
    kc[:S], vc[:S] = to_dev(kr[:S]), to_dev(v[:S])
    kc[first:first + N * B], vc[first:first + N * B] = to_dev(kr[S:]), to_dev(v[S:])
    s = pb.make_shape(S, B, N, 0, Hq, Hkv, d, theta=theta)
    guard = GuardedAllocator()
    o = guard((N * B, Hq, d), torch.bfloat16)
    lse = guard((Hq, N * B), torch.float32)
    ws = guard((pb.pevlm_workspace_bytes(s, pb.WS_PREFILL),), torch.uint8, zero=True)
    pb.pevlm_block_attn(s, to_dev(qr[S:]), kc, vc, first, rows, o, lse, ws)
    torch.cuda.synchronize()
    _status_ok(ws)
    guard.check()
    o_ref, lse_ref = oracle.attn_rows(oracle.make_shape(S, B, N, 0, Hq, Hkv, d), qr, kr, v, np.arange(S, w.L, dtype=np.int64))
    got = bits_to_f64(to_bits(o))
    assert np.isfinite(got).all()
    assert np.abs(got - o_ref).max() <= O_TOL
    assert np.abs(lse.double().cpu().numpy().T - lse_ref).max() <= LSE_TOL
