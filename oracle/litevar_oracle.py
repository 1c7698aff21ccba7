"""CPU fp64 oracle for LiteVAR's multi-diagonal windowed attention (MDWA) with
attention sharing across CFG (ASC).

TEST INFRASTRUCTURE ONLY.  This file is the plain definition the CUDA path is checked
against.  It is imported by tests, by the smoke check and by the benchmark's
cpu-baseline leg, never by the product path, and it shares no code with the CUDA
kernels.  It is slow on purpose: every step is written the way the paper states it.

What follows the paper, and where:

* schedule  -- Section 2: K scales, scale k holds s_k^2 tokens; at step k the current
  scale's s_k^2 queries attend to all sum_{i<=k} s_i^2 tokens generated so far
  (worked example: k=2 gives a [4,5] map).
* parts     -- Section 2, step (2): the step-k map is cut into k-2 parts; the first
  part holds the columns of scales 1..3 together, every later scale is a part of
  its own.
* window    -- Section 2 / Fig. 2(a) caption: inside every part only a local window of
  width w around the part's diagonal is kept.  Reading used here (the paper's
  figure is not available): the "diagonal" of part j is the key cell of scale j that
  contains the centre of the query cell, and the window is the square of
  Chebyshev radius w around it, clipped at the image border.
* global parts -- "MDWA implementation details": the first parts stay full attention
  (attention sinks).  Reading: key scales 1..n_global_scales (default 3).
* R_0 = 1   -- Section 2: the mask degenerates to full attention.
* ASC       -- Section 3: the unconditional CFG branch reuses the conditional branch's
  attention output.
* QKV8      -- Section 4: Q, K and V are quantised to 8-bit integers with a scale s and a
  zero point z taken online from the maximum and minimum of the data (dynamic
  quantisation), x_q = round(clamp((x - z) / s, -2^(B-1), 2^(B-1))), z = (max + min) / 2.
  Readings: one (s, z) per token row of a head (64 values); s = (max - min) / (2^B - 1),
  the step that makes the stated clamp range the range of the data (the printed
  s = max(abs(x)) does not match the printed clamp bounds); the upper clamp bound is
  2^(B-1) - 1 so that the code fits B bits; round = to nearest, ties to even; the
  attention then runs on the dequantised values x_q * s + z, rounded to bf16.

Parity status: mask, schedule, softmax-attention and ASC are pinned by the CPU tests
(paper's worked shapes, Table 1's saving, library softmax attention, brute force in
exact rationals, closed-form counts).  The numeric window widths that the paper
obtains by calibrating on VAR activations are NOT reproducible here (needs weights
and ImageNet): for those, parity unpinned; the default rule below is a stand-in.
The row quantiser is pinned by a hand-worked row, the classical unsigned min-max
formula, its error bound and its invariances; which granularity and step the authors
used is a reading (see above), not something the paper fixes.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

GLOBAL = -1  # radius value meaning "every key of this scale is live"


# ----------------------------------------------------------------------------- schedule
def tokens(scales: Sequence[int]) -> List[int]:
    """n_k = s_k^2 (Section 2)."""
    return [int(s) ** 2 for s in scales]


def offsets(scales: Sequence[int]) -> List[int]:
    """off_j = sum_{i<j} n_i, with one trailing entry: offsets[K] = total tokens."""
    out = [0]
    for n in tokens(scales):
        out.append(out[-1] + n)
    return out


def map_shape(scales: Sequence[int], k: int) -> Tuple[int, int]:
    """Shape [s_k^2, sum_{i<=k} s_i^2] of the attention map at 1-based step k (Section 2)."""
    return tokens(scales)[k - 1], offsets(scales)[k]


def parts(scales: Sequence[int], k: int, n_merged: int = 3) -> List[Tuple[int, int]]:
    """Column ranges [c0, c1) of the parts of the step-k map (Section 2, step (2)).

    The first part merges scales 1..n_merged; each later scale j <= k is its own part,
    which gives k-2 parts for k > 3 (and a single part for k <= 3).
    """
    off = offsets(scales)
    first_end = min(k, n_merged)
    out = [(0, off[first_end])]
    for j in range(first_end + 1, k + 1):
        out.append((off[j - 1], off[j]))
    return out


# ----------------------------------------------------------------------------- window
def default_radius(s_j: int, rho_num: int, rho_den: int) -> int:
    """Stand-in for the calibrated width: w_j = round-half-up(rho * s_j), integer arithmetic."""
    return (2 * rho_num * s_j + rho_den) // (2 * rho_den)


def window_table(scales: Sequence[int], rho: Tuple[int, int] = (1, 4),
                 n_global_scales: int = 3) -> np.ndarray:
    """w[k-1][j-1] for every step k and key scale j <= k; GLOBAL (-1) = whole part live.

    Entries with j > k are unused and set to GLOBAL.
    """
    K = len(scales)
    w = np.full((K, K), GLOBAL, dtype=np.int64)
    for k in range(1, K + 1):
        for j in range(1, k + 1):
            if j > n_global_scales:
                w[k - 1, j - 1] = default_radius(int(scales[j - 1]), rho[0], rho[1])
    return w


def full_table(scales: Sequence[int]) -> np.ndarray:
    """The R_0 = 1 case (Section 2): every part is global."""
    K = len(scales)
    return np.full((K, K), GLOBAL, dtype=np.int64)


def centre(x: int, s_j: int, s_k: int) -> int:
    """Index of the scale-j cell containing the centre of cell x of scale k (one axis).

    Cell x of an s_k grid spans [x/s_k, (x+1)/s_k); its centre is (x + 1/2)/s_k; the
    scale-j cell containing it is floor((x + 1/2) * s_j / s_k).
    """
    return ((2 * x + 1) * s_j) // (2 * s_k)


def live(scales: Sequence[int], k: int, w_row: Sequence[int], q: int, t: int) -> bool:
    """Is key t live for query q at step k?  One (q, t) pair, straight from the definition."""
    s_k = int(scales[k - 1])
    off = offsets(scales)
    j = 1
    while not (off[j - 1] <= t < off[j]):
        j += 1
    s_j = int(scales[j - 1])
    w = int(w_row[j - 1])
    if w == GLOBAL:
        return True
    r, c = divmod(q, s_k)
    rk, ck = divmod(t - off[j - 1], s_j)
    return abs(rk - centre(r, s_j, s_k)) <= w and abs(ck - centre(c, s_j, s_k)) <= w


def mask(scales: Sequence[int], k: int, w_row: Sequence[int],
         q_rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Boolean live mask [n_k (or len(q_rows)), L_k] of step k.

    Same predicate as `live`, evaluated for all pairs at once with array broadcasting
    (one comparison per (q, t) pair; no intervals, no tiles).
    """
    s_k = int(scales[k - 1])
    n_k, L_k = map_shape(scales, k)
    off = offsets(scales)
    q = np.arange(n_k, dtype=np.int64) if q_rows is None else np.asarray(q_rows, dtype=np.int64)
    r = q // s_k
    c = q % s_k
    out = np.zeros((q.shape[0], L_k), dtype=bool)
    for j in range(1, k + 1):
        s_j = int(scales[j - 1])
        w = int(w_row[j - 1])
        t = np.arange(off[j - 1], off[j], dtype=np.int64) - off[j - 1]
        if w == GLOBAL:
            out[:, off[j - 1]:off[j]] = True
            continue
        rk = t // s_j
        ck = t % s_j
        cr = ((2 * r + 1) * s_j) // (2 * s_k)
        cc = ((2 * c + 1) * s_j) // (2 * s_k)
        ok_r = np.abs(rk[None, :] - cr[:, None]) <= w
        ok_c = np.abs(ck[None, :] - cc[:, None]) <= w
        out[:, off[j - 1]:off[j]] = ok_r & ok_c
    return out


def live_count(scales: Sequence[int], k: int, w_row: Sequence[int]) -> int:
    return int(mask(scales, k, w_row).sum())


# ----------------------------------------------------------------------------- band window
# Second reading of "window width w" around "the diagonal" of a part (Section 2, Fig. 2(a) caption):
# taken literally in the flattened attention map, the diagonal of the [n_k, n_j] part joins its corners,
# and the window is the band of key tokens within w of it.
def band_centre(q: int, n_j: int, n_k: int) -> int:
    """Key token of a part with n_j columns under the centre of query row q of n_k rows:
    floor((q + 1/2) * n_j / n_k)."""
    return ((2 * q + 1) * n_j) // (2 * n_k)


def band_table(scales: Sequence[int], rho: Tuple[int, int] = (1, 7), n_global_scales: int = 3) -> np.ndarray:
    """Half-widths b[k-1][j-1] = round-half-up(rho * n_j) in key tokens; GLOBAL for the first scales."""
    K = len(scales)
    w = np.full((K, K), GLOBAL, dtype=np.int64)
    for k in range(1, K + 1):
        for j in range(1, k + 1):
            if j > n_global_scales:
                w[k - 1, j - 1] = default_radius(int(scales[j - 1]) ** 2, rho[0], rho[1])
    return w


def mask_band(scales: Sequence[int], k: int, w_row: Sequence[int],
              q_rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Boolean live mask of step k under the band reading: key token t' of scale j is live for query q
    iff |t' - band_centre(q)| <= w_row[j-1] (or the part is GLOBAL).  One comparison per pair."""
    n_k, L_k = map_shape(scales, k)
    off = offsets(scales)
    q = np.arange(n_k, dtype=np.int64) if q_rows is None else np.asarray(q_rows, dtype=np.int64)
    out = np.zeros((q.shape[0], L_k), dtype=bool)
    for j in range(1, k + 1):
        n_j = int(scales[j - 1]) ** 2
        w = int(w_row[j - 1])
        if w == GLOBAL:
            out[:, off[j - 1]:off[j]] = True
            continue
        t = np.arange(n_j, dtype=np.int64)
        ctr = ((2 * q + 1) * n_j) // (2 * n_k)
        out[:, off[j - 1]:off[j]] = np.abs(t[None, :] - ctr[:, None]) <= w
    return out


def schedule_saving(scales: Sequence[int], w: np.ndarray) -> float:
    """Fraction of attention-map entries (hence of QK^T + PV FLOPs) removed over all steps."""
    dense = 0
    kept = 0
    for k in range(1, len(scales) + 1):
        n_k, L_k = map_shape(scales, k)
        dense += n_k * L_k
        kept += live_count(scales, k, w[k - 1])
    return 1.0 - kept / dense


# ----------------------------------------------------------------------------- window calibration
def window_ratio(scales: Sequence[int], k: int, j: int, w: int, maps: np.ndarray) -> float:
    """R_w of part j of the step-k maps (Section 2): the sum of all attention values inside the window of
    radius w divided by the sum of all values of the part.  maps: [n_maps, n_k, L_k], post-softmax."""
    off = offsets(scales)
    w_row = [GLOBAL] * len(scales)
    w_row[j - 1] = w
    inside = mask(scales, k, w_row)[:, off[j - 1]:off[j]]
    part = np.asarray(maps, dtype=np.float64)[:, :, off[j - 1]:off[j]]
    return float((part * inside[None]).sum() / part.sum())


def calibrate_radius(scales: Sequence[int], k: int, maps: np.ndarray, r0: float,
                     n_global_scales: int = 3) -> np.ndarray:
    """Window design of Section 2, steps (1)-(3), for one step: for every part after the global ones the
    window grows from zero until R_w reaches the threshold R_0; returns the radius row (GLOBAL for the
    global parts and for unused entries j > k).  The decision is taken as inside >= R_0 * total in fp64."""
    off = offsets(scales)
    m = np.asarray(maps, dtype=np.float64)
    out = np.full(len(scales), GLOBAL, dtype=np.int64)
    for j in range(n_global_scales + 1, k + 1):
        part = m[:, :, off[j - 1]:off[j]]
        total = part.sum()
        w = 0
        while True:
            w_row = [GLOBAL] * len(scales)
            w_row[j - 1] = w
            inside = (part * mask(scales, k, w_row)[None, :, off[j - 1]:off[j]]).sum()
            if inside >= np.float64(r0) * total or w >= int(scales[j - 1]) - 1:
                break
            w += 1
        out[j - 1] = w
    return out


# ----------------------------------------------------------------------------- 8-bit Q/K/V
def round_to_bf16(x32: np.ndarray) -> np.ndarray:
    """fp32 -> nearest bf16 (ties to even), returned as fp32 holding the bf16 value."""
    u = np.asarray(x32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16 << 16
    return u.astype(np.uint32).view(np.float32)


def quantize_rows(x: np.ndarray, bits: int = 8):
    """Dynamic min-max quantisation of Section 4, one (s, z) per row (last axis).

    The decision which integer a value becomes is taken in fp32, one IEEE operation at a time, in the
    order written here: z = (max + min) * 0.5; s = (max - min) / (2^B - 1);
    code = clamp(rint((x - z) / s), -2^(B-1), 2^(B-1) - 1); dequantised = bf16(code * s + z).
    The quotient (x - z) / s is the division the section's formula prints, rounded once to fp32.
    A constant row (s = 0) has code 0 everywhere and dequantises to z.
    Returns (codes int32, s fp32 [..., 1], z fp32 [..., 1], dequantised fp32 holding bf16 values)."""
    x = np.asarray(x, dtype=np.float32)
    mx = x.max(axis=-1, keepdims=True)
    mn = x.min(axis=-1, keepdims=True)
    z = (mx + mn) * np.float32(0.5)
    s = (mx - mn) / np.float32(2 ** bits - 1)
    safe = np.where(s > 0, s, np.float32(1))
    code = np.rint((x - z) / safe)
    code = np.clip(code, -(2 ** (bits - 1)), 2 ** (bits - 1) - 1)
    code = np.where(s > 0, code, np.float32(0)).astype(np.float32)
    deq = round_to_bf16((code * s).astype(np.float32) + z)
    return code.astype(np.int32), s, z, deq


# ----------------------------------------------------------------------------- attention
def bf16_to_f64(x) -> np.ndarray:
    """Widen a torch bf16/fp32 tensor or numpy array to fp64 exactly."""
    if hasattr(x, "detach"):
        return x.detach().to("cpu").double().numpy()
    return np.asarray(x, dtype=np.float64)


def attention_rows(Qr: np.ndarray, K: np.ndarray, V: np.ndarray, live_rows: np.ndarray,
                   sm_scale: float, return_weights: bool = False):
    """Masked softmax attention for a block of query rows of ONE (batch, head).

    Qr [m, d], K [L, d], V [L, d] fp64; live_rows [m, L] bool.
    z = sm_scale * Q K^T; masked scores are -inf, so the weights renormalise over the
    live keys; out = softmax(z) V.  All in fp64.
    """
    z = sm_scale * (Qr @ K.T)
    z = np.where(live_rows, z, -np.inf)
    m = z.max(axis=1, keepdims=True)
    p = np.where(live_rows, np.exp(z - m), 0.0)
    wgt = p / p.sum(axis=1, keepdims=True)
    out = wgt @ V
    return (out, wgt) if return_weights else out


def attention_step(scales: Sequence[int], k: int, w_row: Sequence[int], Q, Kc, Vc,
                   sm_scale: Optional[float] = None, share_cfg: bool = False,
                   return_weights: bool = False, band: bool = False):
    """Step-k MDWA attention for the whole batch.

    Q [2B, H, n_k, d]; Kc, Vc [2B, H, >=L_k, d] (only the first L_k rows are read).
    With share_cfg (ASC, Section 3) rows b < B are computed and rows b + B are copies of
    them; the unconditional half of Q/K/V is never read.
    `band` selects the band reading of the window (mask_band) instead of the square one.
    Returns out [2B, H, n_k, d] fp64 (and the weights [2B, H, n_k, L_k] if asked).
    """
    Qd, Kd, Vd = bf16_to_f64(Q), bf16_to_f64(Kc), bf16_to_f64(Vc)
    n_k, L_k = map_shape(scales, k)
    rows, H, nq, d = Qd.shape
    assert nq == n_k and Kd.shape[2] >= L_k and Vd.shape[2] >= L_k
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(d)
    lv = mask_band(scales, k, w_row) if band else mask(scales, k, w_row)
    out = np.empty((rows, H, n_k, d), dtype=np.float64)
    wts = np.empty((rows, H, n_k, L_k), dtype=np.float64) if return_weights else None
    if share_cfg:
        assert rows % 2 == 0
    computed = rows // 2 if share_cfg else rows
    for b in range(computed):
        for h in range(H):
            res = attention_rows(Qd[b, h], Kd[b, h, :L_k], Vd[b, h, :L_k], lv, sm_scale,
                                 return_weights)
            if return_weights:
                out[b, h], wts[b, h] = res
            else:
                out[b, h] = res
    if share_cfg:
        B = rows // 2
        out[B:] = out[:B]
        if return_weights:
            wts[B:] = wts[:B]
    return (out, wts) if return_weights else out


def attention_sampled(scales: Sequence[int], k: int, w_row: Sequence[int], Q, Kc, Vc,
                      samples: Sequence[Tuple[int, int, int]], sm_scale: Optional[float] = None,
                      share_cfg: bool = False, band: bool = False) -> np.ndarray:
    """Outputs for selected (batch row, head, query) triples only: [len(samples), d] fp64.

    Used at sizes where evaluating every row is out of reach.  With share_cfg a sample in
    the unconditional half is computed from the conditional row b - B, as ASC defines it.
    Samples of one (batch row, head) are evaluated together (one widening of that unit's K and V);
    every row still goes through `mask` / `mask_band` and `attention_rows` as in `attention_step`.
    """
    n_k, L_k = map_shape(scales, k)
    rows = Q.shape[0]
    d = Q.shape[-1]
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(d)
    B = rows // 2
    out = np.empty((len(samples), d), dtype=np.float64)
    groups = {}
    for i, (b, h, q) in enumerate(samples):
        src = b - B if (share_cfg and b >= B) else b
        groups.setdefault((src, h), []).append((i, q))
    for (src, h), items in groups.items():
        qs = [q for _, q in items]
        lv = mask_band(scales, k, w_row, q_rows=qs) if band else mask(scales, k, w_row, q_rows=qs)
        Qr = bf16_to_f64(Q[src, h])[qs]
        res = attention_rows(Qr, bf16_to_f64(Kc[src, h, :L_k]), bf16_to_f64(Vc[src, h, :L_k]), lv, sm_scale)
        for (i, _), row in zip(items, res):
            out[i] = row
    return out


def flops_saving_with_asc(mdwa_saving: float) -> float:
    """ASC skips the whole unconditional half of what MDWA leaves (Section 3 + abstract)."""
    return 1.0 - (1.0 - mdwa_saving) / 2.0
