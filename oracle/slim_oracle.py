"""CPU fp64 oracle for K-cache-only ("slim") multi-head decode attention.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is checked against.  It is imported by the tests, by the smoke
check and by the benchmark's CPU-baseline leg, never by the product path, and
it imports nothing from the CUDA package.  Everything is numpy float64; the
loops are over heads (and, in the ``*_loops`` functions, over scalars) exactly
as the paper states the operations, with no tiling, fusion or reordering.

Paper passages followed (arxiv 2503.05840):
  Eq. 4, Eq. 5, Eq. 2   vanilla MHA: Q = X W_Q, K = X W_K, V = X W_V,
                        head_i = softmax(Q_i K_i^T / sqrt(d_k)) V_i
  Eq. 6                 W_KV = W_K^{-1} W_V,  V = K W_KV,  V_i = K W_KV,i
  Eq. 7                 Option 1: softmax(.) [K W_KV,i]
                        Option 2: [softmax(.) K] W_KV,i
  Appendix "Support for RoPE"   encoding / decoding rotation formulas, and
                        Option 1 of that appendix: raw keys are cached and
                        rotated after they are read
  Appendix "MHA complexity"     OP counts 2 n d_k (scores) and 2 n d
                        (weighted sum of K) per head
  Section "Support for non-square weight matrices", Option 2 (X-cache) and
  section "Support for encoder-decoder transformers", Option 2 (E-cache)
                        A_i = ((x_n W_Q,i + b) W_K,i^T) X^T; the values are
                        recomputed as well: head_i = [softmax(.) X] W_V,i.
                        No RoPE in this scheme.
  Section "Support for non-square weight matrices", Option 1
                        right inverse W_K^{-1} = W_K^T (W_K W_K^T)^{-1} for
                        W_K in R^{d x e}, e = d_k h > d;  W_KV = W_K^{-1} W_V
                        is e x e

  Appendix "Taking advantage of softmax sparsities" with appendix "Support for
  RoPE", Option 2     the cache holds RoPE'd keys; attention scores below a
                        threshold are skipped in the weighted sum, and only the
                        key rows that are kept are RoPE-decoded before they
                        enter it (oracle_rotated_cache).  Not exact: the skipped
                        scores are simply left out, nothing is renormalised.

  Introduction, memory-size example ("1 byte per value")  8-bit K-cache: the paper only counts
                        the bytes; the format is a reading (e4m3_* and quantize_keys_e4m3 below):
                        OCP FP8 E4M3 codes with one power-of-two exponent per (row, head)

Readings where the paper is silent (the CUDA path takes the same ones):
  * RoPE pairs element j with j + d_k/2 inside a head, frequency
    theta_j = rope_theta ** (-2 j / d_k), angle = position * theta_j;
    the rotation sign is the one printed in the appendix
    (y1 = x1 cos + x2 sin, y2 = -x1 sin + x2 cos).  rope_theta == 0 means
    "no positional rotation".
  * The single decode query sits at position T-1 (the newest key is already
    in the cache), key t sits at position t.  No causal mask is needed.
  * d_v = d_k, head i owns columns i*d_k .. (i+1)*d_k-1 of every projection.
  * A sequence of length 0 produces a zero output row.
  * W_KV is obtained with a linear solve W_K W_KV = W_V rather than by
    forming the inverse explicitly (same matrix up to rounding).

Pins: tests/test_oracle_pins.py (closed forms, identities, brute force).
"""
from __future__ import annotations

import math

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# RoPE (appendix "Support for RoPE")
# --------------------------------------------------------------------------
def rope_frequencies(d_k: int, rope_theta: float) -> np.ndarray:
    """theta_j for j = 0 .. d_k/2 - 1 (float64)."""
    if d_k % 2:
        raise ValueError("d_k must be even for RoPE")
    j = np.arange(d_k // 2, dtype=F64)
    return np.power(F64(rope_theta), -2.0 * j / F64(d_k))


def rope_encode(x: np.ndarray, positions, rope_theta: float) -> np.ndarray:
    """Rotate head vectors x[..., d_k] sitting at `positions` (broadcast over
    the leading axes of x).  Appendix formulas, pair (j, j + d_k/2):
        y1 =  x1 cos(m theta) + x2 sin(m theta)
        y2 = -x1 sin(m theta) + x2 cos(m theta)
    """
    x = np.asarray(x, dtype=F64)
    if rope_theta == 0:
        return x.copy()
    d_k = x.shape[-1]
    half = d_k // 2
    ang = np.asarray(positions, dtype=F64)[..., None] * rope_frequencies(d_k, rope_theta)
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c + x2 * s, -x1 * s + x2 * c], axis=-1)


def rope_decode(y: np.ndarray, positions, rope_theta: float) -> np.ndarray:
    """Inverse rotation (appendix "RoPE decoding"), same cos/sin table:
        x1 = y1 cos - y2 sin,   x2 = y1 sin + y2 cos
    """
    y = np.asarray(y, dtype=F64)
    if rope_theta == 0:
        return y.copy()
    d_k = y.shape[-1]
    half = d_k // 2
    ang = np.asarray(positions, dtype=F64)[..., None] * rope_frequencies(d_k, rope_theta)
    c, s = np.cos(ang), np.sin(ang)
    y1, y2 = y[..., :half], y[..., half:]
    return np.concatenate([y1 * c - y2 * s, y1 * s + y2 * c], axis=-1)


# --------------------------------------------------------------------------
# softmax (Eq. 2)
# --------------------------------------------------------------------------
def softmax(z: np.ndarray) -> np.ndarray:
    """Softmax over the last axis: subtract the exact row maximum, exp, divide
    by the sum.  float64 throughout."""
    z = np.asarray(z, dtype=F64)
    e = np.exp(z - np.max(z, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def attention_weights(q_i: np.ndarray, K_i: np.ndarray, rope_theta: float) -> np.ndarray:
    """s = softmax(RoPE_{T-1}(q_i) . RoPE_t(K_i[t])^T / sqrt(d_k)) for one head.
    q_i: [d_k], K_i: [T, d_k] (raw, un-rotated keys).  Returns [T]."""
    T, d_k = K_i.shape
    qr = rope_encode(q_i, T - 1, rope_theta)
    Kr = rope_encode(K_i, np.arange(T), rope_theta)
    return softmax(Kr @ qr / math.sqrt(d_k))


# --------------------------------------------------------------------------
# Eq. 6: W_KV
# --------------------------------------------------------------------------
def oracle_wkv(W_K: np.ndarray, W_V: np.ndarray) -> np.ndarray:
    """W_KV = W_K^{-1} W_V in float64 (Eq. 6), by solving W_K W_KV = W_V."""
    W_K = np.asarray(W_K, dtype=F64)
    W_V = np.asarray(W_V, dtype=F64)
    if W_K.ndim != 2 or W_K.shape[0] != W_K.shape[1]:
        raise ValueError("W_K must be square (MHA with d = h d_k)")
    return np.linalg.solve(W_K, W_V)


def oracle_wkv_right_inverse(W_K: np.ndarray, W_V: np.ndarray) -> np.ndarray:
    """Non-square projections, Option 1: W_K, W_V are [d, e] with e > d.
    W_K^{-1} = W_K^T (W_K W_K^T)^{-1} (so that W_K W_K^{-1} = I_d) and
    W_KV = W_K^{-1} W_V, an [e, e] matrix.  float64; the d x d inverse is
    applied as a linear solve."""
    W_K = np.asarray(W_K, dtype=F64)
    W_V = np.asarray(W_V, dtype=F64)
    if W_K.ndim != 2 or W_K.shape != W_V.shape or W_K.shape[0] > W_K.shape[1]:
        raise ValueError("W_K and W_V must be [d, e] with e >= d")
    G = W_K @ W_K.T                                   # d x d
    return W_K.T @ np.linalg.solve(G, W_V)            # e x e


def oracle_prompt_values(K: np.ndarray, W_KV: np.ndarray) -> np.ndarray:
    """Prompt phase (Fig. 3(a), Eq. 6): the values of all prompt tokens from their keys,
    V = K W_KV.  K: [n, d] raw keys, returns [n, d]."""
    return np.asarray(K, dtype=F64) @ np.asarray(W_KV, dtype=F64)


# --------------------------------------------------------------------------
# Eq. 4, 5, 2: vanilla MHA decode with an explicit V cache
# --------------------------------------------------------------------------
def oracle_vanilla(X: np.ndarray, W_Q: np.ndarray, W_K: np.ndarray, W_V: np.ndarray,
                   H: int, rope_theta: float = 0.0, q: np.ndarray | None = None) -> np.ndarray:
    """Output concat(head_1..head_h) (no W_O) for the LAST token of X attending
    over all T = len(X) tokens.  X: [T, d].  If q is given it replaces
    X[-1] W_Q (used where the query carries a bias)."""
    X = np.asarray(X, dtype=F64)
    T = X.shape[0]
    e = np.asarray(W_K).shape[1]                 # width of K and V: d for square MHA, d_k h > d otherwise
    d_k = e // H
    K = X @ np.asarray(W_K, dtype=F64)           # Eq. 4
    V = X @ np.asarray(W_V, dtype=F64)           # Eq. 5
    if q is None:
        q = X[-1] @ np.asarray(W_Q, dtype=F64)   # Eq. 4, one query row
    q = np.asarray(q, dtype=F64)
    out = np.empty(e, dtype=F64)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        s = attention_weights(q[sl], K[:, sl], rope_theta)
        out[sl] = s @ V[:, sl]                   # Eq. 2
    return out


# --------------------------------------------------------------------------
# Eq. 7: slim attention, one sequence
# --------------------------------------------------------------------------
def oracle_slim(q: np.ndarray, K: np.ndarray, W_KV: np.ndarray, H: int,
                rope_theta: float = 0.0) -> np.ndarray:
    """Eq. 7, Option 2: head_i = [softmax(.) K] W_KV,i with the FULL d-wide raw
    keys in the weighted sum.  q: [d], K: [T, d] raw keys, W_KV: [d, d]."""
    q = np.asarray(q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    W_KV = np.asarray(W_KV, dtype=F64)
    T, d = K.shape
    d_k = d // H
    out = np.empty(d, dtype=F64)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        s = attention_weights(q[sl], K[:, sl], rope_theta)   # [T]
        u = s @ K                                            # [d]   weighted sum of K
        out[sl] = u @ W_KV[:, sl]                            # [d_k]
    return out


def oracle_slim_option1(q: np.ndarray, K: np.ndarray, W_KV: np.ndarray, H: int,
                        rope_theta: float = 0.0) -> np.ndarray:
    """Eq. 7, Option 1: V_i = K W_KV,i first, then softmax(.) V_i."""
    q = np.asarray(q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    W_KV = np.asarray(W_KV, dtype=F64)
    T, d = K.shape
    d_k = d // H
    out = np.empty(d, dtype=F64)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        s = attention_weights(q[sl], K[:, sl], rope_theta)
        V_i = K @ W_KV[:, sl]                                # Eq. 6
        out[sl] = s @ V_i
    return out


def oracle_xcache(q: np.ndarray, X: np.ndarray, W_K: np.ndarray, W_V: np.ndarray, H: int) -> np.ndarray:
    """X-cache / E-cache scheme for one decode token.  q: [e] = x_n W_Q (+ query bias),
    X: [T, d] cached layer inputs (or encoder outputs), W_K, W_V: [d, e].  Per head i:
    q~_i = q_i W_K,i^T (a d-vector), A_i = q~_i X^T, s_i = softmax(A_i / sqrt(d_k)),
    u_i = s_i X, head_i = u_i W_V,i.  Returns concat(head_1 .. head_h), [e]."""
    q = np.asarray(q, dtype=F64)
    X = np.asarray(X, dtype=F64)
    W_K = np.asarray(W_K, dtype=F64)
    W_V = np.asarray(W_V, dtype=F64)
    e = W_K.shape[1]
    d_k = e // H
    out = np.empty(e, dtype=F64)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        qt = q[sl] @ W_K[:, sl].T                     # [d]
        s = softmax(X @ qt / math.sqrt(d_k))          # [T]
        u = s @ X                                     # [d]
        out[sl] = u @ W_V[:, sl]                      # [d_k]
    return out


def oracle_rotated_cache(q: np.ndarray, K_rot: np.ndarray, W_KV: np.ndarray, H: int, rope_theta: float,
                         threshold: float):
    """Sparsity appendix + RoPE appendix Option 2.  K_rot: [T, d] keys stored ALREADY rotated
    (head slice i of row t encoded at position t).  Per head i:
      s = softmax(RoPE_{T-1}(q_i) . K_rot,i^T / sqrt(d_k))         (no rotation at read time)
      keep = { t : s_t > threshold }                               (scores at or below it are skipped)
      u_i = sum_{t in keep} s_t * RoPE-decode_t(K_rot[t, :])       (full-width row, every head slice decoded)
      head_i = u_i W_KV,i
    The kept scores are used as they are (the paper skips vectors, it does not renormalise), so with
    threshold < min s the result is oracle_slim on the raw keys, and the error of a larger threshold is
    bounded by the skipped probability mass times the largest value row.
    Returns (out [d], kept [H] number of rows decoded per head)."""
    q = np.asarray(q, dtype=F64)
    K_rot = np.asarray(K_rot, dtype=F64)
    W_KV = np.asarray(W_KV, dtype=F64)
    T, d = K_rot.shape
    d_k = d // H
    pos = np.arange(T)
    out = np.empty(d, dtype=F64)
    kept = np.zeros(H, dtype=np.int64)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        qr = rope_encode(q[sl], T - 1, rope_theta)
        s = softmax(K_rot[:, sl] @ qr / math.sqrt(d_k))                 # [T]
        keep = np.nonzero(s > threshold)[0]
        kept[i] = keep.size
        u = np.zeros(d, dtype=F64)
        if keep.size:
            rows = K_rot[keep].reshape(keep.size, H, d_k)               # decode every head slice of the kept rows
            raw = rope_decode(rows, pos[keep][:, None], rope_theta).reshape(keep.size, d)
            u = s[keep] @ raw
        out[sl] = u @ W_KV[:, sl]
    return out, kept


# --------------------------------------------------------------------------
# 8-bit K-cache: OCP FP8 E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities,
# S.1111.111 is NaN, largest finite value 448, subnormals k * 2^-9) with a power-of-two exponent per
# (row, head).  Written from the published format definition.
# --------------------------------------------------------------------------
def e4m3_decode_table() -> np.ndarray:
    """Value of each of the 256 codes (NaN for 0x7f and 0xff)."""
    v = np.empty(256, dtype=F64)
    for c in range(256):
        sign = -1.0 if c & 0x80 else 1.0
        ex, man = (c >> 3) & 0xF, c & 7
        if ex == 0xF and man == 7:
            v[c] = np.nan
        elif ex == 0:
            v[c] = sign * man * 2.0 ** -9                       # subnormal: 0.mmm * 2^-6
        else:
            v[c] = sign * (1.0 + man / 8.0) * 2.0 ** (ex - 7)
    return v


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """Round to the nearest E4M3 value, ties to the even code, saturating at +-448.  Brute force over
    the 127 finite magnitudes: the definition of rounding, not a bit trick."""
    x = np.asarray(x, dtype=F64)
    mags = e4m3_decode_table()[:0x7F]                            # codes 0x00 .. 0x7e, increasing in value
    a = np.minimum(np.abs(x), 448.0)
    hi = np.searchsorted(mags, a, side="left")                   # first code with value >= a
    hi = np.minimum(hi, 0x7E)
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = mags[hi] - a, a - mags[lo]
    pick_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(pick_lo, lo, hi).astype(np.uint8)
    return np.where(np.signbit(x), code | 0x80, code).astype(np.uint8)


def quantize_keys_e4m3(K: np.ndarray, H: int):
    """K: [T, d] key rows (bf16-representable values).  Per (row, head): exponent e = the smallest
    integer with max|k| * 2^-e <= 448 (0 for an all-zero slice, clamped to [-126, 127]), codes =
    e4m3_encode(k * 2^-e).  Returns (codes uint8 [T, d], exps int8 [T, H], dequantised keys [T, d])."""
    K = np.asarray(K, dtype=F64)
    T, d = K.shape
    d_k = d // H
    Kh = K.reshape(T, H, d_k)
    amax = np.max(np.abs(Kh), axis=2)                            # [T, H]
    e = np.zeros((T, H), dtype=np.int64)
    nz = amax > 0
    e[nz] = np.ceil(np.log2(amax[nz] / 448.0)).astype(np.int64)
    # log2 can be off by one ulp at exact powers of two: fix up so that e is the smallest that fits
    e = np.where(nz & (amax * np.exp2(-(e - 1).astype(F64)) <= 448.0), e - 1, e)
    e = np.where(nz & (amax * np.exp2(-e.astype(F64)) > 448.0), e + 1, e)
    e = np.clip(e, -126, 127)
    scale = np.exp2(e.astype(F64))[:, :, None]
    codes = e4m3_encode(Kh / scale)
    deq = (e4m3_decode_table()[codes] * scale).reshape(T, d)
    return codes.reshape(T, d), e.astype(np.int8), deq


def oracle_slim_fp8(q: np.ndarray, K: np.ndarray, W_KV: np.ndarray, H: int, rope_theta: float = 0.0) -> np.ndarray:
    """Slim attention over an 8-bit K-cache: the keys are quantised (quantize_keys_e4m3) and Eq. 7
    Option 2 is evaluated on the stored (dequantised) keys."""
    return oracle_slim(q, quantize_keys_e4m3(K, H)[2], W_KV, H, rope_theta)


# --------------------------------------------------------------------------
# One context split into slices (several GPUs): per-slice partial results and their join
# --------------------------------------------------------------------------
def oracle_slim_partial(q: np.ndarray, K_slice: np.ndarray, first_pos: int, q_pos: int, H: int, rope_theta: float = 0.0):
    """Rows K_slice [n, d] sit at absolute positions first_pos .. first_pos + n - 1, the query at q_pos.
    Per head: z_t = RoPE_{q_pos}(q_i) . RoPE_t(k_{t,i}) / sqrt(d_k) (natural-log units),
    lse = log2 sum_t e^{z_t}  (reported in log2 units, as the library does), u = sum_t e^{z_t} K[t, :] / sum_t e^{z_t}.
    An empty slice gives lse = -inf and u = 0.  Returns (lse [H], u [H, d])."""
    q = np.asarray(q, dtype=F64)
    K_slice = np.asarray(K_slice, dtype=F64)
    n, d = K_slice.shape
    d_k = d // H
    lse = np.full(H, -np.inf)
    u = np.zeros((H, d), dtype=F64)
    if n == 0:
        return lse, u
    pos = first_pos + np.arange(n)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        z = rope_encode(K_slice[:, sl], pos, rope_theta) @ rope_encode(q[sl], q_pos, rope_theta) / math.sqrt(d_k)
        zmax = np.max(z)
        e = np.exp(z - zmax)
        lse[i] = (zmax + math.log(np.sum(e))) / math.log(2.0)
        u[i] = (e @ K_slice) / np.sum(e)
    return lse, u


def oracle_combine_partials(lse_all: np.ndarray, u_all: np.ndarray, W_KV: np.ndarray) -> np.ndarray:
    """Join of R slices: lse_all [R, H] (log2 units), u_all [R, H, d].  Per head w_r = 2^lse_r / sum_r' 2^lse_r',
    u = sum_r w_r u_r, head_i = u W_KV,i (Eq. 7 Option 2).  All slices empty gives zeros."""
    lse_all = np.asarray(lse_all, dtype=F64)
    u_all = np.asarray(u_all, dtype=F64)
    W_KV = np.asarray(W_KV, dtype=F64)
    R, H, d = u_all.shape
    d_k = d // H
    out = np.zeros(d, dtype=F64)
    for i in range(H):
        if not np.any(np.isfinite(lse_all[:, i])):
            continue
        w = np.exp2(lse_all[:, i] - np.max(lse_all[:, i]))
        w = w / np.sum(w)
        out[i * d_k:(i + 1) * d_k] = (w @ u_all[:, i, :]) @ W_KV[:, i * d_k:(i + 1) * d_k]
    return out


def oracle_slim_batch(q: np.ndarray, K: np.ndarray, lengths, W_KV: np.ndarray, H: int,
                      rope_theta: float = 0.0) -> np.ndarray:
    """Ragged batch: q [B, d], K [B, T_cap, d], lengths[b] rows valid.
    Sequence b attends over K[b, :lengths[b]]; length 0 gives a zero row."""
    q = np.asarray(q, dtype=F64)
    B, d = q.shape
    out = np.zeros((B, d), dtype=F64)
    for b in range(B):
        n = int(lengths[b])
        if n > 0:
            out[b] = oracle_slim(q[b], np.asarray(K[b][:n], dtype=F64), W_KV, H, rope_theta)
    return out


# --------------------------------------------------------------------------
# Scalar-loop version with an operation counter (appendix "MHA complexity")
# --------------------------------------------------------------------------
def oracle_slim_loops(q, K, W_KV, H: int, rope_theta: float = 0.0):
    """Same result as oracle_slim, written as scalar loops, for tiny inputs.
    Returns (out, macs) where macs counts the multiply-accumulates of the two
    attention products only (scores: T d_k per head; weighted sum of K: T d
    per head), which the paper totals as 2 n d (h + 1) OPs = n d (h + 1) MACs."""
    q = [float(v) for v in q]
    K = [[float(v) for v in row] for row in K]
    T, d = len(K), len(q)
    d_k = d // H
    half = d_k // 2
    macs = 0
    out = [0.0] * d
    for i in range(H):
        base = i * d_k
        # rotate the query of this head to position T-1
        qr = list(q[base:base + d_k])
        if rope_theta != 0:
            for j in range(half):
                ang = (T - 1) * rope_theta ** (-2.0 * j / d_k)
                c, s = math.cos(ang), math.sin(ang)
                x1, x2 = q[base + j], q[base + j + half]
                qr[j] = x1 * c + x2 * s
                qr[j + half] = -x1 * s + x2 * c
        z = []
        for t in range(T):
            kr = list(K[t][base:base + d_k])
            if rope_theta != 0:
                for j in range(half):
                    ang = t * rope_theta ** (-2.0 * j / d_k)
                    c, s = math.cos(ang), math.sin(ang)
                    x1, x2 = K[t][base + j], K[t][base + j + half]
                    kr[j] = x1 * c + x2 * s
                    kr[j + half] = -x1 * s + x2 * c
            acc = 0.0
            for e in range(d_k):
                acc += qr[e] * kr[e]
                macs += 1
            z.append(acc / math.sqrt(d_k))
        zmax = max(z)
        ez = [math.exp(v - zmax) for v in z]
        tot = sum(ez)
        s_w = [v / tot for v in ez]
        u = [0.0] * d
        for t in range(T):
            for c_ in range(d):
                u[c_] += s_w[t] * K[t][c_]
                macs += 1
        for c_ in range(d_k):
            acc = 0.0
            for r in range(d):
                acc += u[r] * float(W_KV[r][base + c_])
            out[base + c_] = acc
    return np.array(out, dtype=F64), macs


# --------------------------------------------------------------------------
# Error norms used by the parity tests (the two stated tolerances: fp32 and bf16 caches)
# --------------------------------------------------------------------------
def err_fp32_norm(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i |got_i - ref_i| / max(|ref_i|, RMS(ref)) over one output row."""
    got = np.asarray(got, dtype=F64)
    ref = np.asarray(ref, dtype=F64)
    rms = math.sqrt(float(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), rms if rms > 0 else 1.0)
    return float(np.max(np.abs(got - ref) / den))


def err_rms_norm(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i |got_i - ref_i| / RMS(ref) over one output row."""
    got = np.asarray(got, dtype=F64)
    ref = np.asarray(ref, dtype=F64)
    rms = math.sqrt(float(np.mean(ref * ref)))
    return float(np.max(np.abs(got - ref)) / (rms if rms > 0 else 1.0))
