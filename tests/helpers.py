"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding and
the oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np

from oracle import api as oracle
from paper_2506_19651_b200 import inputs

O_TOL = 2e-2     # max-abs error on outputs (bf16 inputs, fp32 accumulation)
LSE_TOL = 1e-3   # max-abs error on per-row log-sum-exp


def to_dev(bits):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t):
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bits_to_f64(b):
    return inputs.bf16_bits_to_f64(b)


class GuardedAllocator:
    """Device buffers with canary bytes before and after each one (the stand-in for a memory checker): every
    buffer sits inside a larger allocation whose first and last 4 KiB (the tail guard starts at the buffer's
    last byte + 1) hold a known pattern; check() asserts that no kernel wrote there."""
    GUARD = 4096
    PATTERN = 0xA5

    def __init__(self):
        self.items = []

    def __call__(self, shape, dtype, zero=False):
        import torch
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((2 * self.GUARD + (n + 255) // 256 * 256,), self.PATTERN, dtype=torch.uint8, device="cuda")
        view = raw[self.GUARD:self.GUARD + n].view(dtype).view(shape)
        if zero:
            view.zero_()
        self.items.append((raw, n))
        return view

    def check(self):
        for raw, n in self.items:
            assert bool((raw[:self.GUARD] == self.PATTERN).all()), "write before the start of a buffer"
            assert bool((raw[self.GUARD + n:] == self.PATTERN).all()), "write past the end of a buffer"


def gpu_shape(w: inputs.Workload, full_causal=False, scale=0.0):
    from paper_2506_19651_b200 import binding as pb
    return pb.make_shape(w.S, w.B, w.N, w.Q, w.Hq, w.Hkv, w.d, theta=w.theta, scale=scale,
                         mask_mode=pb.MASK_FULL_CAUSAL if full_causal else pb.MASK_PEVLM)


def oracle_shape(w: inputs.Workload, full_causal=False, drop_question=False):
    return oracle.make_shape(w.S, w.B, w.N, 0 if drop_question else w.Q, w.Hq, w.Hkv, w.d, full_causal=full_causal)


def run_gpu_layer(w: inputs.Workload, q, k, v, full_causal=False):
    """Whole hot path on the GPU.  Returns dict of numpy results."""
    import torch
    from paper_2506_19651_b200 import binding as pb
    from paper_2506_19651_b200.layer import LayerBuffers, layer_forward
    s = gpu_shape(w, full_causal)
    guard = GuardedAllocator()
    buf = LayerBuffers(s, alloc=guard)
    layer_forward(buf, to_dev(q), to_dev(k), to_dev(v))
    torch.cuda.synchronize()
    for ws in (buf.ws_prefill, buf.ws_query):
        st, det = pb.pevlm_read_status(ws)
        assert st == 0, f"device wait expired: status {st} detail {det}"
    guard.check()   # no store outside q_video, the caches, o, lse or the workspaces (partials included)
    nv = w.n_video
    return {
        "q_video": to_bits(buf.q_video[:nv]), "q_question": to_bits(buf.q_question[:w.Q]),
        "k_cache": to_bits(buf.k_cache), "v_cache": to_bits(buf.v_cache),
        "o_video": bits_to_f64(to_bits(buf.o_video[:nv])), "lse_video": buf.lse_video[:, :nv].double().cpu().numpy().T,
        "o_question": bits_to_f64(to_bits(buf.o_question[:w.Q])),
        "lse_question": buf.lse_question[:, :w.Q].double().cpu().numpy().T,
    }


def check_against_oracle(w: inputs.Workload, q, k, v, res, rows, full_causal=False):
    """Compare GPU results with the oracle on the given global token rows.  Returns max errors."""
    nv = w.n_video
    qr = oracle.rope(q, w.theta)
    kr = oracle.rope(k, w.theta)
    errs = {}
    rows = np.asarray(rows, dtype=np.int64)
    vid = rows[rows < nv]
    que = rows[rows >= nv]
    if vid.size:
        # video rows never see the question: evaluate them on the video-only stream so that
        # full-causal mode means "causal over the video tokens"
        sh = oracle_shape(w, full_causal, drop_question=True)
        o, lse = oracle.attn_rows(sh, qr[:nv], kr[:nv], v[:nv], vid)
        errs["o_video"] = float(np.abs(res["o_video"][vid] - o).max())
        errs["lse_video"] = float(np.abs(res["lse_video"][vid] - lse).max())
    if que.size:
        sh = oracle_shape(w, False)
        o, lse = oracle.attn_rows(sh, qr, kr, v, que)
        errs["o_question"] = float(np.abs(res["o_question"][que - nv] - o).max())
        errs["lse_question"] = float(np.abs(res["lse_question"][que - nv] - lse).max())
    return errs, qr, kr
