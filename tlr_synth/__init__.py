"""Seeded synthetic inputs for the token-routing step.

Holds input generation only -- none of the routing arithmetic (no logits, no
softmax, no threshold).  Both the tests of the CPU oracle and the callers of
the CUDA library draw their inputs from here so that they see the same bytes.

The tensors imitate the shapes and value distributions of a small language
model's LM head during decoding (Sec. 4: a 0.5B-class model; Sec. 4.2 mentions
the 1.5B-class model of the routing method's original paper):

  W  [V, d]  bf16, i.i.d. N(0, 0.02^2)            -- output embedding, row v = token v
  h  [n, d]  bf16, i.i.d. N(0, 1) rows, each divided by its own root-mean-square
             (no gain vector, epsilon 0), rounded to bf16 (nearest even)
  optional "planted" rows: before normalisation, 8*u is added to the row where
             u = W[v]/rms(W[v]) for a random token v, which makes token v dominate
             that row's distribution (confidence near 1).  The planted rows are a
             seeded random subset, so they are scattered over the batch.

Each tensor uses its own generator sub-stream, so changing n does not change W.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

_STREAM_W, _STREAM_G, _STREAM_ROWS, _STREAM_TARGETS = 1, 2, 3, 4


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) * 1_000_003 + stream)
    return g


@dataclass(frozen=True)
class Workload:
    """One named configuration.  tau=None means "threshold at the 7th-percentile confidence"."""
    name: str
    n: int
    d: int
    V: int
    tau: float | None
    planted_fraction: float = 0.0
    note: str = ""


# The five benchmark configurations (the sweep is expanded over n; tau is swept by the caller).
WORKLOADS = {
    "decode16": Workload("decode16", 16, 896, 151936, None, note="n=16 rows, 0.5B-class head, tau at 7th percentile"),
    "decode256": Workload("decode256", 256, 896, 151936, 0.5, note="256 sessions x 1 token, tau=0.5"),
    "prefill8192": Workload("prefill8192", 8192, 896, 151936, 0.5, planted_fraction=0.05,
                            note="16 sequences x 512 tokens, 5% planted rows, tau=0.5"),
    "head1p5b": Workload("head1p5b", 4096, 1536, 151936, None, note="1.5B-class head, tau at 7th percentile"),
}
SWEEP_N = (1, 8, 64, 512, 4096, 16384)
SWEEP_TAU = (0.3, 0.5, 0.9)
for _n in SWEEP_N:
    WORKLOADS["sweep%d" % _n] = Workload("sweep%d" % _n, _n, 2048, 128256, 0.5, note="batch sweep, d=2048, V=128256")


def make_W(d: int, V: int, seed: int = 0, std: float = 0.02) -> torch.Tensor:
    """bf16 [V, d] output-embedding matrix, i.i.d. N(0, std^2), generated in fp32 then rounded."""
    g = _gen(seed, _STREAM_W)
    W = torch.empty((V, d), dtype=torch.bfloat16)
    rows_per_chunk = max(1, (1 << 24) // max(d, 1))
    for r0 in range(0, V, rows_per_chunk):
        r1 = min(V, r0 + rows_per_chunk)
        W[r0:r1] = (torch.randn((r1 - r0, d), generator=g, dtype=torch.float32) * std).to(torch.bfloat16)
    return W


@dataclass
class Hidden:
    h: torch.Tensor                                  # bf16 [n, d]
    planted_rows: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int64))
    planted_tokens: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int64))


def make_h(n: int, d: int, seed: int = 0, W: torch.Tensor | None = None,
           planted_fraction: float = 0.0, planted_scale: float = 8.0) -> Hidden:
    """bf16 [n, d] unit-RMS hidden states, optionally with planted dominant-token rows."""
    g = torch.randn((n, d), generator=_gen(seed, _STREAM_G), dtype=torch.float32).double()
    rows = np.zeros(0, np.int64)
    toks = np.zeros(0, np.int64)
    k = int(np.floor(planted_fraction * n))
    if k > 0:
        if W is None:
            raise ValueError("planted rows need W")
        V = W.shape[0]
        rows = torch.randperm(n, generator=_gen(seed, _STREAM_ROWS))[:k].numpy().astype(np.int64)
        toks = torch.randint(0, V, (k,), generator=_gen(seed, _STREAM_TARGETS)).numpy().astype(np.int64)
        w = W[torch.from_numpy(toks)].double()
        u = w / w.pow(2).mean(dim=1, keepdim=True).sqrt()
        g[torch.from_numpy(rows)] += planted_scale * u
    if n > 0:
        g = g / g.pow(2).mean(dim=1, keepdim=True).sqrt()
    return Hidden(g.to(torch.bfloat16), rows, toks)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The uint16 bit patterns of a CPU bf16 tensor (a view, no copy)."""
    if t.dtype != torch.bfloat16 or t.device.type != "cpu":
        raise TypeError("expected a CPU bf16 tensor")
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bf16_from_values(values) -> torch.Tensor:
    """bf16 tensor from exactly representable numbers (small integers and the like)."""
    t = torch.tensor(values, dtype=torch.float64)
    b = t.to(torch.bfloat16)
    if not torch.equal(b.double(), t):
        raise ValueError("values are not exactly representable in bf16")
    return b


# ---------------------------------------------------------------- 8-bit copy of W (decode batches)

def _e4m3_magnitudes() -> np.ndarray:
    """The 127 finite magnitudes of the OCP e4m3 format in code order (code 0..126): 1 sign bit,
    4 exponent bits (bias 7), 3 mantissa bits; exponent 0 is subnormal (m/8 * 2^-6); no infinities,
    and code 127 (0x7f) is NaN, so the largest finite magnitude is 448.  Used here only to CHOOSE
    codes; what the codes mean to the routing step is defined by the callee."""
    out = np.empty(127, np.float64)
    for c in range(127):
        e, m = c >> 3, c & 7
        out[c] = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return out


def make_W8(d: int, V: int, seed: int = 0, std: float = 0.02):
    """An 8-bit LM head: (codes uint8 [V, d], scale float32 [V]) with W[v][k] = scale[v] * e4m3(codes[v][k]).

    Recipe: the same N(0, std^2) draw as make_W (in fp32, not rounded to bf16), one scale per row
    that maps the row's largest magnitude to 448, and for every element the nearest e4m3 code of
    value / scale (ties to the even code)."""
    g = _gen(seed, _STREAM_W)
    mags = _e4m3_magnitudes()
    mid = (mags[1:] + mags[:-1]) / 2.0
    codes = np.empty((V, d), np.uint8)
    scale = np.empty(V, np.float32)
    rows_per_chunk = max(1, (1 << 22) // max(d, 1))
    for r0 in range(0, V, rows_per_chunk):
        r1 = min(V, r0 + rows_per_chunk)
        w = (torch.randn((r1 - r0, d), generator=g, dtype=torch.float32) * std).numpy().astype(np.float64)
        amax = np.abs(w).max(axis=1)
        s = np.where(amax > 0, amax / 448.0, 1.0).astype(np.float32)
        x = w / s.astype(np.float64)[:, None]
        a = np.minimum(np.abs(x), 448.0)
        c = np.searchsorted(mid, a, side="left")                 # nearest magnitude; exact ties go down ...
        tie = (c < 126) & (a == mid[np.minimum(c, 125)]) & (c % 2 == 1)
        c = np.where(tie, c + 1, c)                               # ... unless the upper neighbour is the even code
        codes[r0:r1] = (c.astype(np.uint8) | np.where(x < 0, 0x80, 0).astype(np.uint8))
        scale[r0:r1] = s
    return torch.from_numpy(codes), torch.from_numpy(scale)
