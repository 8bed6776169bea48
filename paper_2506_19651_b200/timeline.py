"""Timeline of the attention kernel's hand-offs in steady state (a profiling aid, not part of the hot path).

    PEVLM_TRACE=1 python -m paper_2506_19651_b200.build --force && python -m paper_2506_19651_b200.timeline

Runs the prefill attention in full-causal mode on c3_long-sized random tensors (long work items) with a library
built with time stamps, and prints, for 16 consecutive key tiles of CTA 0's first work item, the SM-clock
cycles between the hand-offs of the two query tiles: scores seen by the softmax, probabilities handed to the
MMA warp, PV and QK issue.  Then the same launch under the PEVLM mask (c3_long and the 256-token blocks of the
sweep): the events at the boundaries between CTA 0's work items.  Rebuild without PEVLM_TRACE afterwards.
"""
from __future__ import annotations

import ctypes as C

import numpy as np


def main():
    import torch
    from . import binding as pb, inputs
    lib = pb.lib()
    if not hasattr(lib, "pevlm_debug_trace"):
        raise SystemExit("library built without PEVLM_TRACE=1")
    w = inputs.WORKLOADS["c3_long"]
    s = pb.make_shape(w.S, w.B, w.N, w.Q, w.Hq, w.Hkv, w.d, theta=w.theta, mask_mode=pb.MASK_FULL_CAUSAL)
    nv = w.n_video
    q = torch.randn(nv, w.Hq, w.d, device="cuda", dtype=torch.bfloat16)
    k = torch.randn(nv, w.Hkv, w.d, device="cuda", dtype=torch.bfloat16)
    v = torch.randn_like(k)
    o = torch.empty_like(q)
    lse = torch.empty(w.Hq, nv, device="cuda")
    ws = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
    for _ in range(3):
        pb.pevlm_parallel_prefill_attn(s, q, k, v, o, lse, ws)
    torch.cuda.synchronize()
    buf = (C.c_uint32 * 128)()
    assert lib.pevlm_debug_trace(buf) == 0
    t = np.array(buf, dtype=np.int64).reshape(8, 16)
    t = (t - t[0, 0]) & 0xFFFFFFFF

    def med(a):
        return int(np.median(a))
    print("cycles (median over 15-16 key tiles; each stamp itself costs some tens of cycles)")
    print("period of query tile 0 (scores seen -> next scores seen):", med(np.diff(t[0])))
    print("softmax of one tile (scores seen -> probabilities handed over): tile 0", med(t[2] - t[0]), " tile 1", med(t[3] - t[1]))
    print("lag of tile 1 behind tile 0 (probabilities handed over):", med(t[3] - t[2]))
    print("probabilities handed over -> seen by the MMA warp:", med(t[6] - t[2]))
    print("seen -> PV issued (fence + 8 MMAs, A from TMEM):", med(t[7] - t[6]))
    print("PV issued -> next QK issue starts:", med(t[4, 1:] - t[7, :-1]))
    print("QK issue (8 MMAs, both operands from shared memory):", med(t[5] - t[4]))
    print("QK issued -> scores seen by the softmax:", med((t[0] - t[5])[1:]))
    print("chain: probabilities handed over -> next scores seen:", med(t[0, 1:] - t[2, :-1]),
          " (tensor work in it: PV 512 + QK 512)")
    del q, k, v, o, lse
    for name in ("c3_long", "c4_sweep_F1"):
        item_boundaries(name)


def item_boundaries(name):
    import torch
    from . import binding as pb, inputs
    w = inputs.WORKLOADS[name]
    s = pb.make_shape(w.S, w.B, w.N, w.Q, w.Hq, w.Hkv, w.d, theta=w.theta)
    nv = w.n_video
    q = torch.randn(nv, w.Hq, w.d, device="cuda", dtype=torch.bfloat16)
    k = torch.randn(nv, w.Hkv, w.d, device="cuda", dtype=torch.bfloat16)
    v = torch.randn_like(k)
    o = torch.empty_like(q)
    lse = torch.empty(w.Hq, nv, device="cuda")
    ws = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_PREFILL), dtype=torch.uint8, device="cuda")
    for _ in range(3):
        pb.pevlm_parallel_prefill_attn(s, q, k, v, o, lse, ws)
    torch.cuda.synchronize()
    buf = (C.c_uint32 * 128)()
    assert pb.lib().pevlm_debug_trace_items(buf) == 0
    t = np.array(buf, dtype=np.int64).reshape(8, 16)[:, :12]   # items 2..13 of CTA 0

    def med(a):
        return int(np.median(a & 0xFFFFFFFF))
    print(f"-- work-item boundaries, {name} under the PEVLM mask (medians over 11-12 items of CTA 0, cycles)")
    print("item (first scores seen -> next item's first scores seen):", med(t[3, 1:] - t[3, :-1]))
    print("last probabilities of tile 0 handed over -> accumulator complete:", med(t[5] - t[4]))
    print("accumulator complete -> released:", med(t[6] - t[5]))
    print("released -> output stored:", med(t[7] - t[6]))
    print("last probabilities of tile 0 -> MMA warp has issued the item's last PV and commits:", med(t[2] - t[4]))
    print("MMA warp: end of item -> next item taken:", med(t[0, 1:] - t[2, :-1]))
    print("next item taken -> its first QK goes out:", med(t[1] - t[0]))
    print("first QK goes out -> first scores seen:", med(t[3] - t[1]))
    print("last probabilities of tile 0 -> next item's first scores seen:", med(t[3, 1:] - t[4, :-1]))


if __name__ == "__main__":
    main()
