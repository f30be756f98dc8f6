"""Per-tile timing of the tensor-core decode kernel, from the instrumented build of the library.

    python -m paper_2503_05840_b200.trace [--config 2] [--layers 1]

Builds libslim_trace.so (the library compiled with -DSLIM_TC_TRACE: one thread of each role of
slim_tc_kernel stores the SM clock at fixed points of its per-tile loop), runs decode steps of one
layer of the chosen workload shape on random keys, reads the trace back and prints, in SM clocks
(medians over the steady-state tiles of all CTAs, with the 10th and 90th percentile):

  period        producer: load issued for tile i -> load issued for tile i+1
  stage wait    producer: top of its loop -> the stage is free (time the producer is held up)
  load          load issued -> score warp 0 sees the keys
  scores        keys seen -> probabilities computed (score warp 0)
  P-stage wait  probabilities computed -> P stage free
  ship          P stage free -> shipped to both CTAs and released
  MMA wait      score warp 0 released -> MMA thread sees the tile complete (the other warps and the peer CTA)
  MMA issue     tile complete -> all MMAs and the commit issued
  hold          load issued -> the same stage free again (one stage's round trip)

The numbers describe this kernel only; they are a tool for reading its pipeline, not a benchmark.
Needs a B200.  The environment variable SLIM_LIBRARY is set for this process before the binding loads."""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np


def main(argv=None) -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--steps", type=int, default=4)
    ap.add_argument("--library", default="", help="an instrumented library built by hand (e.g. with -DSLIM_TC_TRACE_WARP=7)")
    args = ap.parse_args(argv)

    from . import build as _build
    os.environ["SLIM_LIBRARY"] = args.library or _build.build(trace=True)
    import torch
    from . import binding as B
    from . import synth
    from .layer import SlimLayer

    cfg = synth.CONFIGS[args.config].scaled(layers=1)
    assert cfg.dtype == "bf16", "the tensor-core kernel takes bf16 caches"
    dev = "cuda:0"
    torch.cuda.set_device(0)
    lengths = synth.make_lengths(cfg, synth.layer_seed(args.config, 0))
    lay = SlimLayer(cfg.d, cfg.H, cfg.d_k, cfg.rope_theta, cfg.dtype, cfg.batch, cfg.context, dev)
    g = torch.Generator(device=dev); g.manual_seed(1)
    for b in range(cfg.batch):                    # random keys: the pipeline's timing does not depend on their values
        lay.k[b].copy_(torch.randn((cfg.context, cfg.d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16))
    lay.set_wkv(np.eye(cfg.d))
    q = torch.randn((cfg.batch, cfg.d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    ld = torch.from_numpy(lengths).to(dev)
    n_cta = 2 * lay.query(B.SLIM_Q_WORKERS)
    TILES = 192
    buf = torch.zeros((n_cta, TILES, 8), dtype=torch.int64, device=dev)
    for _ in range(3):
        lay.decode(q, ld)
    B.slim_set_trace(lay.ctx, buf)
    for _ in range(args.steps):
        buf.zero_()
        lay.decode(q, ld)
    torch.cuda.synchronize()
    assert lay.device_status() == B.SLIM_OK
    t = buf.cpu().numpy().astype(np.int64)
    lay.close()

    ok = np.all(t[:, :, :] > 0, axis=2)          # tiles every role recorded
    lo, hi = 8, TILES - 4                         # steady state: past the ramp, short of the end

    def stat(name, a):
        a = a[np.isfinite(a)]
        a = a[(a > -1e7) & (a < 1e7)]
        print(f"  {name:13s} median {np.median(a):8.0f}   p10 {np.percentile(a, 10):8.0f}   p90 {np.percentile(a, 90):8.0f}   (n = {a.size})")

    def sel(x):
        m = ok[:, lo:hi]
        return x[:, lo:hi][m].astype(np.float64)

    def sel_next(x_next, x):                      # tile i+1 minus tile i
        m = ok[:, lo:hi] & ok[:, lo + 1:hi + 1]
        return (x_next[:, lo + 1:hi + 1] - x[:, lo:hi])[m].astype(np.float64)

    print(f"config {args.config}: d={cfg.d} H={cfg.H} d_k={cfg.d_k} batch={cfg.batch}, {n_cta} CTAs, tiles {lo}..{hi} of each CTA, SM clocks")
    stat("period", sel_next(t[:, :, 1], t[:, :, 1]))
    stat("stage wait", sel(t[:, :, 1] - t[:, :, 0]))
    stat("load", sel(t[:, :, 2] - t[:, :, 1]))
    stat("scores", sel(t[:, :, 3] - t[:, :, 2]))
    stat("P-stage wait", sel(t[:, :, 4] - t[:, :, 3]))
    stat("ship", sel(t[:, :, 5] - t[:, :, 4]))
    stat("MMA wait", sel(t[:, :, 6] - t[:, :, 5]))
    stat("MMA issue", sel(t[:, :, 7] - t[:, :, 6]))
    ns = 3 if cfg.d_k != 64 else 4
    m = ok[:, lo:hi] & ok[:, lo + ns:hi + ns]
    stat(f"hold ({ns} st.)", (t[:, lo + ns:hi + ns, 1] - t[:, lo:hi, 1])[m].astype(np.float64))


if __name__ == "__main__":
    main(sys.argv[1:])
