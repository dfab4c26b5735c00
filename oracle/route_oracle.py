"""CPU fp64 oracle for the per-token routing step.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain definition the CUDA path is checked against.
It is imported by the tests, by the smoke check and by the CPU-baseline leg of
the benchmark, and by nothing on the product path.  It shares no code with the
CUDA sources and imports nothing from the package that wraps them.

What it computes, per decoding position i (one row of ``h``):

  1. logits   z_v = sum_k h[i,k] * W[v,k]                      (LM head on the small
     model's last-layer hidden state -- Sec. 3.3 "Backend": the hidden state the
     router consumes is the LM head's input)
  2. token    = lowest v attaining max_v z_v                     (the small model's
     own next token)
  3. p        = softmax(z); conf = p[token]                      ("confidence score",
     Sec. 3.1 "Front End"; the max-softmax-probability reading of it)
  4. entropy  = -sum_v p_v ln p_v   (nats, 0*ln 0 := 0)
  5. route    = conf < tau   (strict: a token is routed when its score "falls
     below" the threshold, Sec. 3.1; Sec. 2.1: routing scores against a
     predefined threshold tau)
  6. routed_idx = ascending positions with route set; routed_count = how many
  Variants of steps 5-6: one threshold per row, the opposite polarity (Sec. 2.2:
  defer when the score exceeds the threshold), and the first routed position of
  every sequence (Sec. 4.1: where the re-processing of a returned context stops).
  8-bit copy of W (decode batches): e4m3 codes and one scale per row; the step is
  defined as the step on the de-quantised matrix (dequantize_e4m3).
  Vocabulary-sharded form (several GPUs, each a contiguous range of W's rows):
  shard_summary is what one range reports per row, merge_summaries combines the
  ranges; together they must reproduce steps 2-4 (pinned against them).

All arithmetic is fp64 on the exact values of the bf16 inputs.  The only
library primitive used as a step is the dense matrix product of step 1.  Rows
are independent, so they are processed in blocks of rows purely to bound
memory; nothing inside a row is blocked, fused or reordered.

Parity pins (tests/test_oracle_pins.py): hand-worked integer logits, textbook
softmax values, the closed forms of the all-equal and one-hot-plus-flat logit
vectors, an independent library softmax/entropy, a pure-Python brute force,
threshold invariants (tau=0, tau=1, monotone count -- Table 1 "Routing
Number"), and distributional closed forms of the synthetic workload.
Parity unpinned: anything tied to the paper's dataset or trained router
(accuracy and routed-ratio curves, Figs. 7-8) -- neither is available; and
mlp_router_score, whose shape the paper does not give (pinned by closed forms
and a library cross-check only).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class RouteResult:
    token: np.ndarray         # int32 [n]   argmax (lowest index on ties)
    conf: np.ndarray          # float64 [n] max softmax probability
    entropy: np.ndarray       # float64 [n] Shannon entropy, nats
    route_mask: np.ndarray    # uint8 [n]   1 = send this position to the large model
    routed_idx: np.ndarray    # int32 [routed_count] ascending
    routed_count: int
    top2_gap: np.ndarray      # float64 [n] z_(1) - z_(2); 0 on an exact tie
    tau: float                # the fp32 threshold actually compared against, widened


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp64 exactly.

    A bf16 value is the upper half of an IEEE fp32; placing the 16 bits in the
    high half of a 32-bit word gives that fp32 exactly, and fp32 -> fp64 is exact.
    """
    bits = np.ascontiguousarray(bits)
    if bits.dtype != np.uint16:
        raise TypeError("expected uint16 bf16 bit patterns, got %s" % bits.dtype)
    as_f32 = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return as_f32.astype(np.float64)


def logits_fp64(h64: np.ndarray, W64: np.ndarray) -> np.ndarray:
    """Step 1: z[i,v] = sum_k h[i,k] W[v,k].  W is [V,d]: row v is token v's output embedding."""
    if h64.ndim != 2 or W64.ndim != 2 or h64.shape[1] != W64.shape[1]:
        raise ValueError("h must be [n,d] and W [V,d]")
    return h64 @ W64.T


def row_statistics(z: np.ndarray):
    """Steps 2-4 on a block of logit rows z [r,V]: token, conf, entropy, top-2 gap."""
    r, V = z.shape
    rows = np.arange(r)
    m = z.max(axis=1)
    token = z.argmax(axis=1)                    # numpy returns the first (lowest) maximiser
    e = np.exp(z - m[:, None])
    p = e / e.sum(axis=1)[:, None]
    conf = p[rows, token]
    safe = np.where(p > 0.0, p, 1.0)            # 0 * ln 0 := 0
    entropy = -(p * np.log(safe)).sum(axis=1)
    if V > 1:
        rest = z.copy()
        rest[rows, token] = -np.inf
        gap = m - rest.max(axis=1)
    else:
        gap = np.full(r, np.inf)
    return token.astype(np.int32), conf, entropy, gap


def route_decision(conf: np.ndarray, tau, route_above: bool = False):
    """Steps 5-6.  ``tau`` is rounded to fp32 first: that is the value the C-ABI carries.

    ``tau`` is a scalar or one threshold per row (the threshold is a per-user
    setting in the front end, Sec. 3.1).  ``route_above`` switches to the
    polarity of the deferral rule of Sec. 2.2 (defer when the score exceeds
    the threshold).  A row whose confidence is not a number is routed under
    either polarity (fail-safe to the large model): the tests are
    "not (conf >= tau)" and "not (conf <= tau)", which equal "conf < tau" and
    "conf > tau" for every finite confidence.
    """
    tau32 = np.asarray(tau, dtype=np.float32).astype(np.float64)
    if route_above:
        mask = np.logical_not(conf <= tau32).astype(np.uint8)
    else:
        mask = np.logical_not(conf >= tau32).astype(np.uint8)
    idx = np.flatnonzero(mask).astype(np.int32)
    return mask, idx, int(idx.size), (float(tau32) if tau32.ndim == 0 else tau32)


def first_routed(route_mask: np.ndarray, seq_len: int) -> np.ndarray:
    """Per sequence of ``seq_len`` consecutive rows: position of its first routed row, or seq_len.

    After the large model has supplied a token the small model re-processes the whole
    context (Sec. 4.1; the multi-round prefill of Sec. 3): this is where it stops next.
    """
    n = route_mask.shape[0]
    if seq_len <= 0 or n % seq_len != 0:
        raise ValueError("n must be a positive multiple of seq_len")
    out = np.full(n // seq_len, seq_len, dtype=np.int32)
    for b in range(n // seq_len):
        hits = np.flatnonzero(route_mask[b * seq_len:(b + 1) * seq_len])
        if hits.size:
            out[b] = hits[0]
    return out


def route_oracle(h_bits: np.ndarray, W_bits: np.ndarray, tau: float,
                 row_block: int = 128, W64: np.ndarray | None = None) -> RouteResult:
    """The whole path on bf16 inputs given as uint16 bit patterns.

    ``W64`` may carry an already widened W so repeated calls on one W do not
    pay the widening again; it must equal bf16_bits_to_f64(W_bits).
    """
    h64 = bf16_bits_to_f64(h_bits)
    if W64 is None:
        W64 = bf16_bits_to_f64(W_bits)
    n = h64.shape[0]
    token = np.empty(n, np.int32)
    conf = np.empty(n, np.float64)
    entropy = np.empty(n, np.float64)
    gap = np.empty(n, np.float64)
    for r0 in range(0, n, row_block):
        r1 = min(n, r0 + row_block)
        z = logits_fp64(h64[r0:r1], W64)
        token[r0:r1], conf[r0:r1], entropy[r0:r1], gap[r0:r1] = row_statistics(z)
    mask, idx, count, tau32 = route_decision(conf, tau)
    return RouteResult(token, conf, entropy, mask, idx, count, gap, tau32)


def with_threshold(result: RouteResult, tau, route_above: bool = False) -> RouteResult:
    """The same per-row scores with steps 5-6 redone for another threshold or polarity."""
    mask, idx, count, tau32 = route_decision(result.conf, tau, route_above)
    return RouteResult(result.token, result.conf, result.entropy, mask, idx, count, result.top2_gap, tau32)


def e4m3_value(codes: np.ndarray) -> np.ndarray:
    """Values of OCP 8-bit floats "e4m3": bit 7 sign, bits 6..3 exponent E (bias 7), bits 2..0
    mantissa M.  E = 0: (M/8) * 2^-6 (subnormal);  otherwise (1 + M/8) * 2^(E-7); there are no
    infinities and E = 15 with M = 7 (0x7f, 0xff) is NaN.  fp64 out."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    E = (c >> 3) & 15
    M = (c & 7).astype(np.float64)
    mag = np.where(E == 0, (M / 8.0) * 2.0 ** -6, (1.0 + M / 8.0) * np.exp2((E - 7).astype(np.float64)))
    mag = np.where((E == 15) & ((c & 7) == 7), np.nan, mag)
    return np.where(c & 0x80, -mag, mag)


def dequantize_e4m3(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """The LM head an 8-bit copy stands for: W[v][k] = scale[v] * e4m3_value(codes[v][k]), fp64.
    The routing step on an 8-bit W is, by definition, the step on this matrix (route_oracle with
    W64 = dequantize_e4m3(...)); the hidden states stay bf16."""
    return e4m3_value(codes) * np.asarray(scale, dtype=np.float64)[:, None]


def shard_summary(h_bits: np.ndarray, W_shard_bits: np.ndarray, v_offset: int):
    """Per-row summary of a contiguous range of the vocabulary (rows v_offset.. of the full W).

    What one GPU of a vocabulary-sharded step reports for a row with shard logits z:
        m = max z,  idx = v_offset + lowest position attaining it,
        s = sum exp(z - m),  t = sum exp(z - m) * (z - m).
    Returned as four arrays (m, idx, s, t), fp64 / int64.
    """
    z = logits_fp64(bf16_bits_to_f64(h_bits), bf16_bits_to_f64(W_shard_bits))
    m = z.max(axis=1)
    idx = z.argmax(axis=1).astype(np.int64) + int(v_offset)
    e = np.exp(z - m[:, None])
    return m, idx, e.sum(axis=1), (e * (z - m[:, None])).sum(axis=1)


def merge_summaries(parts):
    """Combines per-row summaries of disjoint vocabulary ranges into token, conf, entropy.

    With M the largest of the ranges' maxima: token = the lowest index among the ranges that
    attain M; S = sum_g s_g exp(m_g - M); T = sum_g exp(m_g - M) (t_g + (m_g - M) s_g);
    conf = 1/S and entropy = ln S - T/S.  (Both follow from p_v = exp(z_v - M)/S:
    p_token = 1/S, and -sum p ln p = ln S - (1/S) sum exp(z_v - M)(z_v - M).)
    """
    ms = np.stack([p[0] for p in parts])            # [G, n]
    idxs = np.stack([p[1] for p in parts])
    M = ms.max(axis=0)
    at_max = ms == M[None, :]
    token = np.where(at_max, idxs, np.iinfo(np.int64).max).min(axis=0)
    S = np.zeros_like(M)
    T = np.zeros_like(M)
    for m, _, s, t in parts:
        w = np.exp(m - M)
        S += s * w
        T += w * (t + (m - M) * s)
    return token.astype(np.int32), 1.0 / S, np.log(S) - T / S


def mlp_router_score(h_bits: np.ndarray, W1_bits: np.ndarray, b1, w2, b2: float) -> np.ndarray:
    """Learned routing score sigmoid(w2 . relu(W1 h + b1) + b2), fp64, one value per row.

    The paper routes on the output of a small learned classifier (an MLP) fed with the
    last-layer hidden state (Sec. 3.1; Sec. 2.1) without giving its shape; one hidden layer with ReLU
    and a sigmoid output is this repository's assumption, so this function is pinned
    only by mathematics (closed forms, a library cross-check), not by the paper:
    parity unpinned by the paper.  W1 is bf16 bits [d_hidden, d]; b1, w2 are fp32.
    """
    h64 = bf16_bits_to_f64(h_bits)
    W1 = bf16_bits_to_f64(W1_bits)
    b1 = np.asarray(b1, dtype=np.float32).astype(np.float64)
    w2 = np.asarray(w2, dtype=np.float32).astype(np.float64)
    hidden = np.maximum(h64 @ W1.T + b1[None, :], 0.0)
    logit = hidden @ w2 + float(np.float32(b2))
    return 1.0 / (1.0 + np.exp(-logit))


def percentile_tau(conf: np.ndarray, fraction: float = 0.07) -> float:
    """Threshold that routes exactly the k = max(1, floor(fraction*n)) least confident rows.

    Imitates the paper's operating point of under 7% of tokens routed (abstract,
    conclusion).  tau is placed halfway between the k-th and (k+1)-th smallest
    confidence, so no row sits on the threshold; the fp32 rounding of that
    midpoint is checked to still separate the two.
    """
    c = np.sort(np.asarray(conf, dtype=np.float64))
    n = c.size
    k = max(1, int(np.floor(fraction * n)))
    if k >= n:
        return float(np.float32(1.0))
    tau = float(np.float32(0.5 * (c[k - 1] + c[k])))
    if not (c[k - 1] < tau <= c[k]):
        raise ValueError("fp32 midpoint does not separate the k-th and (k+1)-th confidences")
    return tau


def route_bruteforce(h_vals, W_vals, tau: float):
    """Pure-Python restatement for tiny inputs (nested lists of floats).  Used only as a pin."""
    import math
    n, V, d = len(h_vals), len(W_vals), len(W_vals[0])
    tau32 = float(np.float32(tau))
    out = []
    routed = []
    for i in range(n):
        z = [math.fsum(h_vals[i][k] * W_vals[v][k] for k in range(d)) for v in range(V)]
        best = 0
        for v in range(1, V):
            if z[v] > z[best]:
                best = v
        denom = math.fsum(math.exp(zv - z[best]) for zv in z)
        p = [math.exp(zv - z[best]) / denom for zv in z]
        H = -math.fsum(pv * math.log(pv) for pv in p if pv > 0.0)
        flag = 1 if p[best] < tau32 else 0
        if flag:
            routed.append(i)
        out.append((best, p[best], H, flag))
    return out, routed
