"""How much of the context a rotated-key cache with skipped scores could skip (sparsity appendix and
RoPE appendix, Option 2) on the synthetic workloads: a CPU survey that calls only the oracle and the
seeded input generators.  TEST / MEASUREMENT INFRASTRUCTURE, not part of the product path.

For one sequence per workload shape and for every head, the attention scores are sorted and the
largest set of smallest scores whose sum stays below `eps` is marked skippable (an error contract:
leaving them out changes a head's output by at most eps times the largest value row).  Reported:
  S_rows_heads  share of (row, head) scores that are skippable  (the paper's sparsity factor S)
  rows_all      share of rows skippable for ALL heads at once   (a key row is read once for all heads)
  tiles_all     share of 16-row tiles whose rows are all skippable for all heads (what a kernel that
                feeds whole tiles to the tensor core could leave out)
`sharp` multiplies the query (1 = the workload's recipe; larger = more peaked softmax).

    python -m oracle.sparsity_survey            # prints one line per workload shape and query sharpness
"""
from __future__ import annotations

import sys

import numpy as np

from oracle import slim_oracle as so
from paper_2503_05840_b200 import synth


def survey_sequence(q, K, H, theta, eps, tile=16):
    T, d = K.shape
    d_k = d // H
    skip = np.zeros((H, T), dtype=bool)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        s = so.attention_weights(q[sl], K[:, sl], theta)
        order = np.argsort(s)
        n = int(np.searchsorted(np.cumsum(s[order]), eps, side="right"))
        skip[i, order[:n]] = True
    rows_all = np.all(skip, axis=0)
    nt = T // tile
    tiles_all = np.all(rows_all[:nt * tile].reshape(nt, tile), axis=1)
    return float(skip.mean()), float(rows_all.mean()), float(tiles_all.mean())


def main(argv):
    eps = 1e-3
    shapes = [(0, 1500), (1, 4096), (2, 12288), (3, 1500), (4, 32768)]     # config index, context rows surveyed
    print(f"eps = {eps}: skipped probability mass per head")
    print("config                          T      sharp  S_rows_heads  rows_all  tiles_all")
    for ci, T in shapes:
        cfg = synth.CONFIGS[ci].scaled(batch=1, context=T, ragged_min=0)
        g = np.random.Generator(np.random.Philox(synth.layer_seed(ci, 0)))
        # keys with the recipe's statistics (X W_K with orthogonal-times-diagonal W_K has independent
        # N(0, s_j^2) columns), drawn directly so that a 4096-wide QR is not needed here
        s = g.uniform(0.5, 2.0, size=cfg.d)
        X = g.standard_normal((T, cfg.d))
        if cfg.rmsnorm_x:
            X /= np.sqrt(np.mean(X * X, axis=1, keepdims=True))
        K = synth.round_to_dtype(X * s[None, :], cfg.dtype).astype(np.float64)
        q0 = synth.round_to_dtype(g.standard_normal(cfg.d), cfg.dtype).astype(np.float64)
        for sharp in (1.0, 4.0, 16.0):
            a, b, c = survey_sequence(q0 * sharp, K, cfg.H, cfg.rope_theta, eps)
            print(f"{ci} {cfg.name:28s} {T:6d}  {sharp:5.1f}  {a:12.3f}  {b:8.3f}  {c:9.3f}")


if __name__ == "__main__":
    main(sys.argv[1:])
