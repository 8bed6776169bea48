"""Second, independent evaluation of the PEVLM definition through a materialised dense
mask, in numpy fp64.  TEST INFRASTRUCTURE ONLY; small shapes only (L x L memory).

The mask is built from the sentence-level statement of the method (Sec. 3.2.1, Eq. 3-5):
a sink token sees the sink tokens up to itself; a token of a context block sees every sink
token and the tokens of its own block up to itself; a question token sees every token up to
itself.  Nothing here shares code with oracle/pevlm_oracle.c.
"""
from __future__ import annotations

import numpy as np


def segment_ids(S, B, N, Q, B_last=0):
    """-1 for sink tokens, block index for context tokens, N for question tokens.  The last
    context block may be shorter than the others (B_last tokens; 0 = B)."""
    lens = [B] * N
    if N > 0 and B_last > 0:
        lens[-1] = B_last
    seg = np.concatenate([np.full(S, -1, dtype=np.int64)] +
                         [np.full(n, b, dtype=np.int64) for b, n in enumerate(lens)] +
                         [np.full(Q, N, dtype=np.int64)])
    return seg


def dense_mask(S, B, N, Q, full_causal=False, B_last=0):
    seg = segment_ids(S, B, N, Q, B_last)
    L = len(seg)
    row = np.arange(L)[:, None]
    col = np.arange(L)[None, :]
    causal = col <= row
    if full_causal:
        return causal
    is_sink_col = (seg == -1)[None, :]
    same_seg = seg[:, None] == seg[None, :]
    is_question_row = (seg == N)[:, None]
    return causal & (is_sink_col | same_seg | is_question_row)


def bits_to_f64(b):
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def dense_attention(q_bits, k_bits, v_bits, mask, scale=None):
    """softmax(mask(Q K^T * scale)) V per head (Eq. 1); q [L,Hq,d], k,v [L,Hkv,d] bf16 bits,
    already roped.  Returns o [L,Hq,d], lse [L,Hq], weights [Hq,L,L]."""
    q, k, v = bits_to_f64(q_bits), bits_to_f64(k_bits), bits_to_f64(v_bits)
    L, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    o = np.empty((L, Hq, d))
    lse = np.empty((L, Hq))
    w_all = np.empty((Hq, L, L))
    for h in range(Hq):
        g = h // G
        s = (q[:, h, :] @ k[:, g, :].T) * scale
        s = np.where(mask, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        l = e.sum(axis=1, keepdims=True)
        w = e / l
        o[:, h, :] = w @ v[:, g, :]
        lse[:, h] = (m + np.log(l))[:, 0]
        w_all[h] = w
    return o, lse, w_all
