"""One pass of the whole hot path over one layer's tensors, as a user of the library calls it.

Host-side orchestration only (buffer allocation through torch, then the C-ABI calls in the
order of the method): RoPE of the video Q/K at global positions -> parallel prefill attention
(Eq. 3-4) -> RoPE of the question Q/K -> KV-cache assembly -> question attention (Eq. 5).
"""
from __future__ import annotations

from . import binding as pb


class LayerBuffers:
    """Device buffers of one layer pass, allocated once and reused across steps."""

    def __init__(self, shape: pb.Shape, device="cuda"):
        import torch
        s = shape
        nv, Q, L = s.n_video, s.query_len, s.L
        Hq, Hkv, d = s.num_q_heads, s.num_kv_heads, s.head_dim
        bf, f32 = torch.bfloat16, torch.float32
        self.shape = s
        self.q_video = torch.empty((max(nv, 1), Hq, d), dtype=bf, device=device)   # roped in place
        self.q_question = torch.empty((max(Q, 1), Hq, d), dtype=bf, device=device)
        self.k_cache = torch.empty((L, Hkv, d), dtype=bf, device=device)
        self.v_cache = torch.empty((L, Hkv, d), dtype=bf, device=device)
        self.o_video = torch.empty((max(nv, 1), Hq, d), dtype=bf, device=device)
        self.lse_video = torch.empty((Hq, max(nv, 1)), dtype=f32, device=device)
        self.o_question = torch.empty((max(Q, 1), Hq, d), dtype=bf, device=device)
        self.lse_question = torch.empty((Hq, max(Q, 1)), dtype=f32, device=device)
        self.ws_prefill = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device=device)
        self.ws_query = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_QUERY), dtype=torch.uint8, device=device)


KERNELS_PER_PASS = 7  # rope, V copy, prefill attention, rope, V copy, question attention, merge


def layer_forward(buf: LayerBuffers, q, k, v, mark=None):
    """q [L,Hq,d], k, v [L,Hkv,d]: un-roped bf16 device tensors of the whole stream.
    Leaves O/LSE of the video rows and of the question rows in `buf`.  `mark(name)`, if
    given, is called before the first call and after each C-ABI call (for event timing)."""
    s = buf.shape
    nv, Q = s.n_video, s.query_len
    mark = mark or (lambda name: None)
    mark("start")
    if nv > 0:
        # K goes straight into its cache slot; Q is roped into a scratch copy
        pb.pevlm_rope_qk(s, q[:nv], k[:nv], buf.q_video, buf.k_cache[:nv], 0, nv)
        mark("rope_video")
        pb.pevlm_assemble_kv(s, None, v[:nv], None, None, buf.k_cache, buf.v_cache)
        mark("assemble_video")
        pb.pevlm_parallel_prefill_attn(s, buf.q_video, buf.k_cache[:nv], buf.v_cache[:nv], buf.o_video,
                                       buf.lse_video, buf.ws_prefill)
        mark("prefill_attn")
    if Q > 0:
        pb.pevlm_rope_qk(s, q[nv:], k[nv:], buf.q_question, buf.k_cache[nv:], nv, Q)
        mark("rope_question")
        pb.pevlm_assemble_kv(s, None, None, None, v[nv:], buf.k_cache, buf.v_cache)
        mark("assemble_question")
        pb.pevlm_query_attn(s, buf.q_question, buf.k_cache, buf.v_cache, buf.o_question, buf.lse_question,
                            buf.ws_query)
        mark("query_attn")
    return buf
