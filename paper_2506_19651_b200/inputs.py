"""Seeded synthetic inputs and workload shapes for the PEVLM prefill-attention path.

This module holds no arithmetic of the method (no RoPE, no masks, no softmax): it only
produces bf16 bit patterns from a seeded generator and names the workload shapes.  Both
the CUDA path's tests/bench and the CPU oracle's tests are fed from here, so the two
sides always see identical bits.

Token stream layout (Sec. 3.2.1, Sec. 3.2.3): [sink | c_0 | ... | c_{N-1} | question]
with lengths S, B (uniform), N blocks, Q; L = S + N*B + Q.

The paper's measurements used real video benchmarks and trained weights; the tensors
made here are synthetic stand-ins that keep only the shapes (frames x tokens per
frame, block sizes, head counts) and the one statistical feature the paper stresses:
a few early sink keys with outsized attention (Sec. 2), modelled as the first four
sink K rows scaled by 8.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np

TOKENS_PER_CHUNK = 4096  # every chunk of tokens has its own Philox key


@dataclass(frozen=True)
class Workload:
    name: str
    S: int            # sink length
    B: int            # context block length
    N: int            # number of context blocks
    Q: int            # question length
    Hq: int
    Hkv: int
    d: int
    theta: float
    outliers: bool    # first 4 sink K rows x8
    seed: int
    layers: int = 1
    B_last: int = 0   # length of the last context block when the video does not divide evenly (0 = B)

    @property
    def n_video(self) -> int:
        if self.N <= 0:
            return self.S
        return self.S + (self.N - 1) * self.B + (self.B_last or self.B)

    @property
    def L(self) -> int:
        return self.n_video + self.Q

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


_BASE_SEED = 20250619 * 1000


def _wl(idx, name, S, B, N, Q, Hq, Hkv, d, theta, outliers, layers=1):
    return Workload(name, S, B, N, Q, Hq, Hkv, d, theta, outliers, _BASE_SEED + idx * 100, layers)


def sweep_workload(frames_per_block: int) -> Workload:
    """Block-size sweep point: 128 frames x 256 tokens, sink = the first block."""
    F = frames_per_block
    assert 128 % F == 0
    return _wl(4, f"c4_sweep_F{F}", 256 * F, 256 * F, 128 // F - 1, 64, 32, 8, 128, 1e6, False)


# The sink is taken from the video's first F frames (Sec. 3.2.1: the sink holds the first
# several frames, the context blocks hold the remaining video), so N = T/F - 1.
WORKLOADS = {
    "c1_tiny": _wl(1, "c1_tiny", 64, 128, 4, 32, 4, 2, 64, 1e4, False),
    "c2_qwen": _wl(2, "c2_qwen", 784, 784, 15, 64, 28, 4, 128, 1e6, True),
    "c3_long": _wl(3, "c3_long", 1568, 1568, 31, 128, 28, 4, 128, 1e6, True),
    "c5_stack": _wl(5, "c5_stack", 1152, 1152, 63, 256, 28, 4, 128, 1e6, True, layers=28),
}
for _F in (1, 2, 4, 8, 16, 32):
    WORKLOADS[f"c4_sweep_F{_F}"] = sweep_workload(_F)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even. Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def normal_bf16(seed: int, tensor_id: int, n_tokens: int, heads: int, d: int,
                first_token: int = 0, scale_rows: dict | None = None) -> np.ndarray:
    """bf16 bits of N(0,1) samples, shape [n_tokens, heads, d], for tokens
    first_token .. first_token+n_tokens-1 of tensor `tensor_id`.  Any token range gives the
    same bits as the matching slice of the whole tensor.  `scale_rows` maps a global token
    index to a factor applied before the bf16 rounding."""
    out = np.empty((n_tokens, heads, d), dtype=np.uint16)
    t = first_token
    end = first_token + n_tokens
    while t < end:
        chunk = t // TOKENS_PER_CHUNK
        c0 = chunk * TOKENS_PER_CHUNK
        c1 = min(c0 + TOKENS_PER_CHUNK, end)
        gen = np.random.Generator(np.random.Philox(key=[(seed << 8) | tensor_id, chunk]))
        vals = gen.standard_normal(size=(TOKENS_PER_CHUNK, heads, d), dtype=np.float32)
        lo, hi = t - c0, c1 - c0
        block = vals[lo:hi]
        if scale_rows:
            for row, factor in scale_rows.items():
                if t <= row < c1:
                    block[row - t] *= np.float32(factor)
        out[t - first_token:c1 - first_token] = f32_to_bf16_bits(block)
        t = c1
    return out


def make_qkv(w: Workload, layer: int = 0):
    """Un-roped Q [L,Hq,d], K [L,Hkv,d], V [L,Hkv,d] as bf16 bit patterns (uint16)."""
    seed = w.seed + layer
    outl = {r: 8.0 for r in range(min(4, w.S))} if w.outliers else None
    q = normal_bf16(seed, 1, w.L, w.Hq, w.d)
    k = normal_bf16(seed, 2, w.L, w.Hkv, w.d, scale_rows=outl)
    v = normal_bf16(seed, 3, w.L, w.Hkv, w.d)
    return q, k, v


def sample_rows(w: Workload, n_random: int, seed: int = 7, tile: int = 128) -> np.ndarray:
    """A stratified sample of token rows: the first and last two rows and every tile edge (edge - 1, edge,
    edge + 1) of the sink and of EVERY context block, the whole question block, plus seeded random rows.
    Sorted, unique, all < L."""
    rows = set()
    nv = w.n_video
    segs = [(0, w.S)] + [(w.S + b * w.B, w.S + (b + 1) * w.B) for b in range(w.N)]
    for si in range(len(segs)):
        a, e = segs[si]
        if e <= a:
            continue
        for r in (a, a + 1, e - 2, e - 1):
            if a <= r < e:
                rows.add(r)
        for edge in range(a, e, tile):
            for r in (edge - 1, edge, edge + 1):
                if a <= r < e:
                    rows.add(r)
    rows.update(range(nv, w.L))
    rng = np.random.Generator(np.random.Philox(key=[seed, w.seed]))
    if n_random > 0 and w.L > 0:
        rows.update(int(x) for x in rng.integers(0, w.L, size=n_random))
    return np.array(sorted(rows), dtype=np.int64)
