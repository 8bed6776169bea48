"""One pass of the whole hot path over one layer's tensors, as a user of the library calls it.

Host-side orchestration only (buffer allocation through torch, then the C-ABI calls in the
order of the method): RoPE of the video Q/K at global positions -> parallel prefill attention
(Eq. 3-4) -> RoPE of the question Q/K -> KV-cache assembly -> question attention (Eq. 5).
"""
from __future__ import annotations

from . import binding as pb


class LayerBuffers:
    """Device buffers of one layer pass, allocated once and reused across steps."""

    def __init__(self, shape: pb.Shape, device="cuda", alloc=None):
        """`alloc(shape, dtype, zero)` replaces torch.empty / torch.zeros (the tests pass an allocator that puts
        guard bytes around every buffer)."""
        import torch
        s = shape
        nv, Q, L = s.n_video, s.query_len, s.L
        Hq, Hkv, d = s.num_q_heads, s.num_kv_heads, s.head_dim
        bf, f32 = torch.bfloat16, torch.float32
        if alloc is None:
            def alloc(shp, dtype, zero=False):
                return (torch.zeros if zero else torch.empty)(shp, dtype=dtype, device=device)
        self.shape = s
        self.q_video = alloc((max(nv, 1), Hq, d), bf)   # roped copy of the video queries
        self.q_question = alloc((max(Q, 1), Hq, d), bf)
        self.k_cache = alloc((L, Hkv, d), bf)
        self.v_cache = alloc((L, Hkv, d), bf)
        self.o_video = alloc((max(nv, 1), Hq, d), bf)
        self.lse_video = alloc((Hq, max(nv, 1)), f32)
        self.o_question = alloc((max(Q, 1), Hq, d), bf)
        self.lse_question = alloc((Hq, max(Q, 1)), f32)
        self.ws_prefill = alloc((pb.pevlm_workspace_bytes(s, pb.WS_PREFILL),), torch.uint8, zero=True)
        self.ws_query = alloc((pb.pevlm_workspace_bytes(s, pb.WS_QUERY),), torch.uint8, zero=True)


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


def ragged_layer_forward(q, k, v, S, B, N, B_last, Q, theta, scale=0.0, alloc=None):
    """Layer pass over a video whose length is not a multiple of the block length: N context blocks, the
    first N-1 of B tokens, the last one of B_last < B tokens (the uniform partition of Sec. 3.2.1 with the
    remainder as one shorter block).  q [L,Hq,d], k, v [L,Hkv,d] un-roped device tensors of the whole
    stream, L = S + (N-1)*B + B_last + Q.  Returns (o_video, lse_video, o_question, lse_question, workspaces).

    The uniform prefix runs through pevlm_parallel_prefill_attn, the last block through pevlm_block_attn
    against the same cache, the question through pevlm_query_attn; positions are the global ones.
    `alloc(shape, dtype, zero)` replaces torch.empty / torch.zeros (see LayerBuffers).
    """
    import torch
    Hq, Hkv, d = q.shape[1], k.shape[1], q.shape[2]
    nv_full = S + (N - 1) * B
    nv = nv_full + B_last
    L = nv + Q
    assert N >= 1 and 1 <= B_last <= B and q.shape[0] == L
    dev, bf, f32 = q.device, torch.bfloat16, torch.float32
    s_all = pb.make_shape(nv, 1, 0, Q, Hq, Hkv, d, theta=theta, scale=scale)          # [video | question]
    s_full = pb.make_shape(S, B, N - 1, 0, Hq, Hkv, d, theta=theta, scale=scale)      # uniform prefix
    s_last = pb.make_shape(S, B_last, 1, 0, Hq, Hkv, d, theta=theta, scale=scale)     # the shorter last block
    if alloc is None:
        def alloc(shp, dtype, zero=False):
            return (torch.zeros if zero else torch.empty)(shp, dtype=dtype, device=dev)
    q_roped = alloc((L, Hq, d), bf)
    k_cache = alloc((L, Hkv, d), bf)
    v_cache = alloc((L, Hkv, d), bf)
    o_video = alloc((nv, Hq, d), bf)
    lse_video = alloc((Hq, nv), f32)
    lse_last = alloc((Hq, B_last), f32)
    o_question = alloc((max(Q, 1), Hq, d), bf)
    lse_question = alloc((Hq, max(Q, 1)), f32)
    ws = [alloc((pb.pevlm_workspace_bytes(s, which),), torch.uint8, zero=True)
          for s, which in ((s_full, pb.WS_PREFILL), (s_last, pb.WS_PREFILL), (s_all, pb.WS_QUERY))]
    pb.pevlm_rope_qk(s_all, q, k, q_roped, k_cache, 0, L)
    pb.pevlm_assemble_kv(s_all, None, v[:nv], None, v[nv:] if Q > 0 else None, k_cache, v_cache)
    lse_full = alloc((Hq, max(nv_full, 1)), f32)
    if nv_full > 0:
        pb.pevlm_parallel_prefill_attn(s_full, q_roped[:nv_full], k_cache[:nv_full], v_cache[:nv_full],
                                       o_video[:nv_full], lse_full, ws[0])
        lse_video[:, :nv_full] = lse_full
    pb.pevlm_block_attn(s_last, q_roped[nv_full:nv], k_cache, v_cache, nv_full, L, o_video[nv_full:nv], lse_last, ws[1])
    lse_video[:, nv_full:] = lse_last
    if Q > 0:
        pb.pevlm_query_attn(s_all, q_roped[nv:], k_cache, v_cache, o_question, lse_question, ws[2])
    return o_video, lse_video, o_question, lse_question, ws


class StreamingWindow:
    """A sliding window of W context blocks over a fixed sink (the streaming use the paper names as
    future work, Sec. 5).  The cache is [sink | W block slots | question]; block t of the stream is encoded
    once, at its global positions S + t*B ..., against the sink alone (Eq. 4) and replaces the oldest
    block (slot t mod W).  A question attends to the sink and the blocks now in the window (Eq. 5 over the
    window); key order inside the cache does not matter to it because every key carries its own position.
    """

    def __init__(self, S, B, W, Q_max, Hq, Hkv, d, theta, scale=0.0, device="cuda"):
        import torch
        self.S, self.B, self.W, self.Q_max, self.theta, self.scale = S, B, W, Q_max, theta, scale
        self.Hq, self.Hkv, self.d = Hq, Hkv, d
        self.rows = S + W * B + Q_max
        bf, f32 = torch.bfloat16, torch.float32
        self.k_cache = torch.zeros((self.rows, Hkv, d), dtype=bf, device=device)
        self.v_cache = torch.zeros((self.rows, Hkv, d), dtype=bf, device=device)
        self.q_buf = torch.empty((max(S, B, Q_max), Hq, d), dtype=bf, device=device)
        self.s_sink = self._shape(S, 1, 0, 0)
        self.s_block = self._shape(S, B, 1, 0)
        self.ws_sink = torch.zeros(pb.pevlm_workspace_bytes(self.s_sink, pb.WS_PREFILL), dtype=torch.uint8, device=device)
        self.ws_block = torch.zeros(pb.pevlm_workspace_bytes(self.s_block, pb.WS_PREFILL), dtype=torch.uint8, device=device)
        self.ws_query = torch.zeros(pb.pevlm_workspace_bytes(self._shape(S + W * B, 1, 0, Q_max), pb.WS_QUERY),
                                    dtype=torch.uint8, device=device)
        self.blocks_seen = 0
        self._f32, self._bf, self._dev = f32, bf, device

    def _shape(self, S, B, N, Q):
        return pb.make_shape(S, B, N, Q, self.Hq, self.Hkv, self.d, theta=self.theta, scale=self.scale)

    def set_sink(self, q, k, v):
        """Encode the sink (Eq. 3).  Returns (o [S,Hq,d], lse [Hq,S])."""
        import torch
        S = self.S
        o = torch.empty((S, self.Hq, self.d), dtype=self._bf, device=self._dev)
        lse = torch.empty((self.Hq, S), dtype=self._f32, device=self._dev)
        pb.pevlm_rope_qk(self.s_sink, q, k, self.q_buf[:S], self.k_cache[:S], 0, S)
        pb.pevlm_assemble_kv(self.s_sink, None, v, None, None, self.k_cache, self.v_cache)
        pb.pevlm_parallel_prefill_attn(self.s_sink, self.q_buf[:S], self.k_cache[:S], self.v_cache[:S], o, lse, self.ws_sink)
        return o, lse

    def append_block(self, q, k, v):
        """Encode the next block of the stream into the slot of the oldest one.  Returns (o [B,Hq,d], lse [Hq,B])."""
        import torch
        S, B = self.S, self.B
        t = self.blocks_seen
        row0 = S + (t % self.W) * B
        o = torch.empty((B, self.Hq, self.d), dtype=self._bf, device=self._dev)
        lse = torch.empty((self.Hq, B), dtype=self._f32, device=self._dev)
        pb.pevlm_rope_qk(self.s_block, q, k, self.q_buf[:B], self.k_cache[row0:row0 + B], S + t * B, B)
        # the V rows go to cache rows [row0, row0 + B): the copy call with those rows as its trailing segment
        pb.pevlm_assemble_kv(self._shape(row0, 1, 0, B), None, None, None, v, self.k_cache, self.v_cache)
        pb.pevlm_block_attn(self.s_block, self.q_buf[:B], self.k_cache, self.v_cache, row0, self.rows, o, lse, self.ws_block)
        self.blocks_seen = t + 1
        return o, lse

    def ask(self, q, k, v):
        """Question of Qn <= Q_max tokens at the positions that follow the stream so far, against the sink
        and the blocks in the window (Eq. 5).  Returns (o [Qn,Hq,d], lse [Hq,Qn])."""
        import torch
        Qn = q.shape[0]
        held = min(self.blocks_seen, self.W)
        nv = self.S + held * self.B
        s = self._shape(nv, 1, 0, Qn)
        o = torch.empty((Qn, self.Hq, self.d), dtype=self._bf, device=self._dev)
        lse = torch.empty((self.Hq, Qn), dtype=self._f32, device=self._dev)
        pb.pevlm_rope_qk(s, q, k, self.q_buf[:Qn], self.k_cache[nv:nv + Qn], self.S + self.blocks_seen * self.B, Qn)
        pb.pevlm_assemble_kv(s, None, None, None, v, self.k_cache, self.v_cache)
        pb.pevlm_query_attn(s, self.q_buf[:Qn], self.k_cache[:nv + Qn], self.v_cache[:nv + Qn], o, lse, self.ws_query)
        return o, lse
