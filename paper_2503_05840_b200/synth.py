"""Seeded synthetic inputs shaped like the paper's MHA models.

This module only *draws data*: random activations, random projection weights
with a controlled condition number, and their rounding to the cache dtype.
It contains none of the attention arithmetic; both the CUDA library and the
CPU oracle are fed from it so that they see identical bits.

The shapes follow Table 1 of the paper (CodeLlama-7B d=4096 / 32 layers / 16k
context, Phi-3-mini d=3072 / 32 layers, Whisper-tiny d=384, Whisper-large-v3
d=1280 / 32 layers / 1500 encoder tokens); head counts come from the public
model cards.  The checkpoints themselves are not used: weights are random.

Recipe (per layer, seed = SEED_BASE + 1000*config + layer):
  X      rows ~ N(0, 1)            (config 4: rows RMS-normalised)
  W_K    = Q diag(s),  Q Haar-orthogonal (sign-fixed QR of a Gaussian),
           s ~ U[0.5, 2]  =>  cond(W_K) <= 4
  W_V, W_Q ~ N(0, 1/d)
  K      = X W_K rounded once to the cache dtype
  q      = x_n W_Q rounded to the cache dtype  (x_n = last context row)
  config 2 lengths ~ U{8192..16384}; other configs use the full context.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

SEED_BASE = 0x51A77E00


@dataclass(frozen=True)
class SlimConfig:
    name: str
    d: int
    H: int
    d_k: int
    batch: int
    context: int          # T_cap
    layers: int
    rope_theta: float     # 0 => no RoPE
    dtype: str            # "f32" | "bf16"
    ragged_min: int = 0   # 0 => all sequences use the full context
    rmsnorm_x: bool = False

    def scaled(self, **kw) -> "SlimConfig":
        return replace(self, **kw)


CONFIGS = [
    SlimConfig("whisper-tiny-shaped", 384, 6, 64, 1, 1500, 1, 0.0, "f32"),
    SlimConfig("phi-3-mini-shaped", 3072, 32, 96, 1, 4096, 1, 1.0e4, "bf16"),
    SlimConfig("codellama-7b-shaped", 4096, 32, 128, 16, 16384, 32, 1.0e6, "bf16", ragged_min=8192),
    SlimConfig("whisper-large-v3-cross-shaped", 1280, 20, 64, 64, 1500, 32, 0.0, "bf16"),
    SlimConfig("long-context-stress", 4096, 32, 128, 1, 131072, 1, 1.0e6, "bf16", rmsnorm_x=True),
]


def layer_seed(config_index: int, layer: int) -> int:
    return SEED_BASE + 1000 * config_index + layer


def _rng(seed: int) -> np.random.Generator:
    # Philox is counter-based: the stream depends on the seed only.
    return np.random.Generator(np.random.Philox(seed))


# ---------------------------------------------------------------- rounding
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even) and return
    them as float32 (every result is exactly representable in bf16)."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bf16-representable."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round to the cache dtype; result held as float32 (f32) values."""
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(dtype)


# ---------------------------------------------------------------- weights
def make_weights(d: int, seed: int):
    """(W_Q, W_K, W_V, Qorth, s) in float64; W_K = Qorth diag(s)."""
    g = _rng(seed)
    G = g.standard_normal((d, d))
    Qo, R = np.linalg.qr(G)
    Qo = Qo * np.sign(np.diag(R))[None, :]        # Haar measure: fix column signs
    s = g.uniform(0.5, 2.0, size=d)
    W_K = Qo * s[None, :]
    W_V = g.standard_normal((d, d)) / np.sqrt(d)
    W_Q = g.standard_normal((d, d)) / np.sqrt(d)
    return W_Q, W_K, W_V, Qo, s


def make_weights_nonsquare(d_model: int, e: int, seed: int):
    """Non-square projections [d_model, e], e > d_model: W_K = diag(s) Q[:d_model, :] with Q an
    e x e Haar-orthogonal matrix and s ~ U[0.5, 2] (orthogonal rows, cond <= 4);
    W_V, W_Q ~ N(0, 1/d_model).  Returns (W_Q, W_K, W_V, Qrows, s) in float64."""
    g = _rng(seed)
    G = g.standard_normal((e, e))
    Qo, R = np.linalg.qr(G)
    Qo = Qo * np.sign(np.diag(R))[None, :]
    Qrows = Qo[:d_model, :]
    s = g.uniform(0.5, 2.0, size=d_model)
    W_K = s[:, None] * Qrows
    W_V = g.standard_normal((d_model, e)) / np.sqrt(d_model)
    W_Q = g.standard_normal((d_model, e)) / np.sqrt(d_model)
    return W_Q, W_K, W_V, Qrows, s


def make_lengths(cfg: SlimConfig, seed: int) -> np.ndarray:
    if cfg.ragged_min and cfg.ragged_min < cfg.context:
        g = _rng(seed ^ 0x5EED)
        return g.integers(cfg.ragged_min, cfg.context + 1, size=cfg.batch).astype(np.int32)
    return np.full(cfg.batch, cfg.context, dtype=np.int32)


@dataclass
class LayerInputs:
    cfg: SlimConfig
    W_Q: np.ndarray        # [d, d] f64
    W_K: np.ndarray        # [d, d] f64
    W_V: np.ndarray        # [d, d] f64
    Qorth: np.ndarray      # [d, d] f64   (W_K = Qorth diag(s))
    s: np.ndarray          # [d]    f64
    X: list                # B arrays [len_b, d] f64 (unrounded activations)
    K: np.ndarray          # [B, T_cap, d] f32 holding cache-dtype values; rows >= len_b are zero
    q: np.ndarray          # [B, d] f32 holding cache-dtype values
    lengths: np.ndarray    # [B] int32


def make_layer(cfg: SlimConfig, seed: int, lengths: np.ndarray | None = None) -> LayerInputs:
    """Draw one attention layer's inputs on the host (small / medium sizes)."""
    W_Q, W_K, W_V, Qo, s = make_weights(cfg.d, seed)
    if lengths is None:
        lengths = make_lengths(cfg, seed)
    lengths = np.asarray(lengths, dtype=np.int32)
    g = _rng(seed + 7)
    K = np.zeros((cfg.batch, cfg.context, cfg.d), dtype=np.float32)
    q = np.zeros((cfg.batch, cfg.d), dtype=np.float32)
    Xs = []
    for b in range(cfg.batch):
        n = int(lengths[b])
        X = g.standard_normal((n, cfg.d))
        if cfg.rmsnorm_x and n:
            X = X / np.sqrt(np.mean(X * X, axis=1, keepdims=True))
        Xs.append(X)
        if n:
            K[b, :n] = round_to_dtype(X @ W_K, cfg.dtype)
            q[b] = round_to_dtype(X[-1] @ W_Q, cfg.dtype)
    return LayerInputs(cfg, W_Q, W_K, W_V, Qo, s, Xs, K, q, lengths)


# ---------------------------------------------------------------- byte accounting
def kcache_values(d: int, layers: int, tokens: int) -> int:
    """Number of cached key activations: d * layers * tokens (half of the
    2 d layers tokens the paper gives for a KV-cache under Table 1)."""
    return d * layers * tokens


def kcache_bytes_per_step(cfg: SlimConfig, lengths: np.ndarray) -> int:
    """Algorithmic K bytes one decode step reads: layers * sum(lengths) * d *
    sizeof(dtype)  (the 'n d reads' of Table 2, per layer and sequence)."""
    rows = int(cfg.layers) * int(np.sum(lengths, dtype=np.int64))
    if cfg.dtype == "fp8":                       # one byte per value plus one exponent byte per (row, head)
        return rows * (cfg.d + cfg.H)
    size = 2 if cfg.dtype == "bf16" else 4
    return rows * cfg.d * size


# ---------------------------------------------------------------- device-side drawing (full-size configs)
def make_weights_torch(d: int, seed: int, device):
    """Same recipe as make_weights, drawn and factorised on `device` in float64
    (used where the host QR of a 4096 x 4096 matrix per layer would dominate
    set-up).  Returns (W_Q, W_K, W_V, Qorth, s) as float64 tensors."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    G = torch.randn((d, d), generator=g, dtype=torch.float64, device=device)
    Qo, R = torch.linalg.qr(G)
    Qo = Qo * torch.sign(torch.diagonal(R))[None, :]
    s = torch.rand(d, generator=g, dtype=torch.float64, device=device) * 1.5 + 0.5
    W_K = Qo * s[None, :]
    W_V = torch.randn((d, d), generator=g, dtype=torch.float64, device=device) / d ** 0.5
    W_Q = torch.randn((d, d), generator=g, dtype=torch.float64, device=device) / d ** 0.5
    return W_Q, W_K, W_V, Qo, s


def fill_layer_torch(cfg: SlimConfig, seed: int, W_Q, W_K, lengths, k_out, q_out) -> None:
    """Draw X per sequence on the device, write K = X W_K (rounded to the cache
    dtype) into k_out[b, :len_b] and q = x_n W_Q into q_out[b].  Rows beyond
    len_b are left as they are."""
    import torch
    g = torch.Generator(device=k_out.device)
    g.manual_seed(seed + 7)
    for b in range(cfg.batch):
        n = int(lengths[b])
        if n == 0:
            continue
        X = torch.randn((n, cfg.d), generator=g, dtype=torch.float64, device=k_out.device)
        if cfg.rmsnorm_x:
            X = X / torch.sqrt(torch.mean(X * X, dim=1, keepdim=True))
        k_out[b, :n] = (X @ W_K).to(k_out.dtype)
        q_out[b] = (X[-1] @ W_Q).to(q_out.dtype)
        del X
