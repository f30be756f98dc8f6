#!/usr/bin/env python
"""Benchmark of the slim-attention decode path (one process per GPU).

A *step* is one decode token for every sequence of the batch through all
layers of the workload: per layer slim_append_k (the new key row) followed by
slim_decode.  The default workload is the CodeLlama-7B-shaped configuration
(32 layers, d=4096, H=32, d_k=128, batch 16, ragged contexts U[8192,16384],
bf16 K-cache, RoPE theta 1e6) with seeded synthetic data.

  value      decode tokens/s with all inputs resident in HBM (CUDA events)
  e2e        the same through host buffers: per step the queries and new keys
             are copied from pinned host memory and the outputs copied back
  roofline   K-cache bytes per main-kernel launch / its CUDA-event duration,
             against the measured HBM copy rate
  cpu_baseline  the fp64 oracle timed on the host cores on a bounded sample

`--impl reference` times the oracle alone (there is no reference code to run).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="index into the five workload shapes")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (0 = the config's)")
    ap.add_argument("--path", default="auto", choices=["auto", "generic", "tc"])
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (0 = the config's)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--variant", default="kcache", choices=["kcache", "xcache", "prompt", "fp8"],
                    help="xcache: the X/E-cache scheme, one cache shared by all layers (configs without RoPE); "
                         "prompt: the prompt-phase V = K W_KV of the config's shape; "
                         "fp8: the K-cache path with an 8-bit cache")
    ap.add_argument("--paged", type=int, default=0, help="K-cache in a shuffled pool of pages of this many rows (0 = contiguous)")
    return ap.parse_args()


# DRAM bytes (read + write) of one main-kernel launch on the benchmarked workload, from an
# ncu capture (profiles/), keyed by the hash of the kernel source it was taken with.  A kernel
# that has changed since reports no traffic.
NCU_TRAFFIC = {"7d1c1e8701d6f306": 1636218000 + 6251776}


def ncu_traffic(config_index, layers_ignored=None):
    import hashlib
    if config_index != 2:
        return None
    src = os.path.join(ROOT, "paper_2503_05840_b200", "csrc", "slim_tc.cu")
    try:
        with open(src, "rb") as f:
            return NCU_TRAFFIC.get(hashlib.sha256(f.read()).hexdigest()[:16])
    except OSError:
        return None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def hbm_read_probe(dev):
    """Read-only HBM stream rate of this GPU, for context beside the copy figure: a library reduction
    (torch.sum) over 4 GiB of float32, best of 5, CUDA events.  Harness only."""
    import torch
    x = torch.ones(1 << 30, dtype=torch.float32, device=dev)
    best = None
    for _ in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); x.sum(); e1.record(); torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        best = ms if best is None else min(best, ms)
    del x
    return {"gbs": 4 * (1 << 30) / (best * 1e-3) / 1e9, "how": "torch.sum over 4 GiB of float32, best of 6 (first is warm-up), CUDA events"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thr = threading.Thread(target=self._read, daemon=True)
            self.thr.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for ts, line in self.rows:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            inside = t0 <= ts <= t1 + 0.1
            try:
                if inside:
                    sm.append(float(parts[1]))
                mx = float(parts[2])
            except ValueError:
                continue
            if inside:
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        if not sm:      # timed region shorter than the sampling period: use every sample
            for ts, line in self.rows:
                parts = [x.strip() for x in line.split(",")]
                try:
                    sm.append(float(parts[1]))
                except (ValueError, IndexError):
                    pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample_seconds(cfg, lengths, get_seq, W_KV):
    """Time the oracle, as it stands, on one (layer, sequence) of the workload."""
    from oracle import slim_oracle as so
    b = int(np.argmin(np.abs(lengths - np.mean(lengths))))
    q, K = get_seq(b)
    t0 = time.perf_counter()
    so.oracle_slim(q, K, W_KV, cfg.H, cfg.rope_theta)
    dt = time.perf_counter() - t0
    return b, dt


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The CPU oracle as the reference arm: one step = one (layer, sequence)
    sample of the workload; throughput is scaled to whole decode tokens."""
    from oracle import slim_oracle as so
    from paper_2503_05840_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = synth.CONFIGS[args.config]
    layers = args.layers or cfg.layers
    seed = synth.layer_seed(args.config, 0)
    lengths = synth.make_lengths(cfg, seed)
    # bounded sample: one sequence of one layer, context capped so a step stays in seconds
    n = int(min(int(np.mean(lengths)), 4096))
    g = np.random.Generator(np.random.Philox(seed))
    s = g.uniform(0.5, 2.0, size=cfg.d)
    K = synth.round_to_dtype(g.standard_normal((n, cfg.d)) * s[None, :], cfg.dtype).astype(np.float64)
    q = synth.round_to_dtype(g.standard_normal(cfg.d), cfg.dtype).astype(np.float64)
    W_KV = g.standard_normal((cfg.d, cfg.d)) / np.sqrt(cfg.d)
    for _ in range(max(1, min(args.warmup, 1))):
        so.oracle_slim(q, K, W_KV, cfg.H, cfg.rope_theta)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        so.oracle_slim(q, K, W_KV, cfg.H, cfg.rope_theta)
    dt = (time.perf_counter() - t0) / args.steps
    # seconds per (layer, sequence) at the mean context, then per decode token (all layers)
    per_token = dt * (float(np.mean(lengths)) / n) * layers
    value = 1.0 / per_token
    cores = host_threads()
    sample = f"oracle_slim on 1 layer x 1 sequence x {n} context rows per step, scaled to {layers} layers and mean context {int(np.mean(lengths))}"
    line = {"impl": "reference", "metric": "decode_attention_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config{args.config}:{cfg.name}", "layers": layers, "batch": cfg.batch,
                       "context": cfg.context, "d": cfg.d, "H": cfg.H, "d_k": cfg.d_k},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_xcache(args):
    """X/E-cache scheme on a config without RoPE: one cache of layer inputs shared by all layers,
    per layer slim_xcache_decode.  Reported beside the K-cache numbers; not the default line."""
    import torch
    from paper_2503_05840_b200 import binding as B
    from paper_2503_05840_b200 import build as _build
    from paper_2503_05840_b200 import synth
    _build.build()
    cfg = synth.CONFIGS[args.config]
    if args.batch:
        cfg = cfg.scaled(batch=args.batch)
    assert cfg.rope_theta == 0.0, "the X-cache scheme has no RoPE: use --config 0 or 3"
    layers_n = args.layers or cfg.layers
    dev = "cuda:0"
    torch.cuda.set_device(0)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    g = torch.Generator(device=dev); g.manual_seed(synth.layer_seed(args.config, 0))
    X = torch.randn((cfg.batch, cfg.context, cfg.d), generator=g, device=dev, dtype=torch.float32).to(tdt)
    lengths = torch.full((cfg.batch,), cfg.context, dtype=torch.int32, device=dev)
    q = torch.randn((layers_n, cfg.batch, cfg.d), generator=g, device=dev, dtype=torch.float32).to(tdt)
    o = torch.empty((layers_n, cfg.batch, cfg.d), dtype=torch.float32, device=dev)
    ctxs, caches = [], []
    ws = None
    for li in range(layers_n):
        ctx = B.slim_create(cfg.d, cfg.H, cfg.d_k, 0.0, B.SLIM_BF16 if cfg.dtype == "bf16" else B.SLIM_F32)
        W_Q, W_K, W_V, _, _ = synth.make_weights_torch(cfg.d, synth.layer_seed(args.config, li), dev)
        B.slim_xcache_set_weights(ctx, W_K.cpu().numpy(), W_V.cpu().numpy())
        ctxs.append(ctx); caches.append(B.slim_cache_create(ctx, X, cfg.batch, cfg.context))
        if ws is None:
            ws = torch.empty(B.slim_xcache_workspace_bytes(ctx, cfg.batch, cfg.context), dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream().cuda_stream

    def step():
        for li in range(layers_n):
            B.slim_xcache_decode(ctxs[li], q[li], caches[li], lengths, o[li], ws, st)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record(); torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    cache_bytes = X.numel() * X.element_size()
    # parity of what was timed: sampled sequences of the last layer against the oracle
    parity = None
    if not args.no_cpu_baseline:
        from oracle import slim_oracle as so
        W_Q, W_K, W_V, _, _ = synth.make_weights_torch(cfg.d, synth.layer_seed(args.config, layers_n - 1), dev)
        W_K_h, W_V_h = W_K.cpu().numpy(), W_V.cpu().numpy()
        got = o[layers_n - 1].cpu().numpy().astype(np.float64)
        worst = 0.0
        for b in sorted({0, cfg.batch // 3, cfg.batch - 1}):
            ref = so.oracle_xcache(q[layers_n - 1, b].float().cpu().numpy(), X[b].float().cpu().numpy(), W_K_h, W_V_h, cfg.H)
            worst = max(worst, so.err_rms_norm(got[b], ref) if cfg.dtype == "bf16" else so.err_fp32_norm(got[b], ref))
        tol = 2e-2 if cfg.dtype == "bf16" else 1e-4
        parity = {"err": worst, "tolerance": tol, "parity": "green" if worst <= tol else "FAILED",
                  "sample": "3 sequences of the last layer against oracle_xcache"}
    peak, peak_kind = measured_peaks()
    # algorithmic bytes: the cache is needed once per layer (the kernels read it twice)
    gbs = cache_bytes * layers_n / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "decode_attention_tokens_per_s", "variant": "xcache", "value": cfg.batch / (ms * 1e-3),
                      "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "dtype": cfg.dtype, "data": "synthetic",
                      "config": {"workload": f"config{args.config}:{cfg.name} (X/E-cache scheme)", "layers": layers_n,
                                 "batch": cfg.batch, "context": cfg.context, "d": cfg.d, "H": cfg.H, "d_k": cfg.d_k},
                      "cache_bytes_shared_by_all_layers": cache_bytes,
                      "kcache_bytes_equivalent": cache_bytes * layers_n,
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak, "traffic": None,
                                   "peak_kind": peak_kind, "kernel": "whole step (dense scores + weighted sum + tail); algorithmic "
                                   "bytes = one pass over the shared cache per layer"},
                      "parity": parity,
                      "device_status": int(B.slim_device_status(ctxs[0], st))}))
    if parity is not None and parity["parity"] != "green":
        raise SystemExit("parity check against the oracle FAILED on the timed X-cache workload")


def run_prompt(args):
    """Prompt phase: V = K W_KV for all prompt rows of one layer of the config (batch x context rows)."""
    import torch
    from paper_2503_05840_b200 import binding as B
    from paper_2503_05840_b200 import build as _build
    from paper_2503_05840_b200 import synth
    _build.build()
    cfg = synth.CONFIGS[args.config]
    dev = "cuda:0"
    torch.cuda.set_device(0)
    n = min((args.batch or cfg.batch) * cfg.context, 262144)
    ctx = B.slim_create(cfg.d, cfg.H, cfg.d_k, 0.0, B.SLIM_BF16 if cfg.dtype == "bf16" else B.SLIM_F32)
    B.slim_set_wkv(ctx, np.random.default_rng(0).standard_normal((cfg.d, cfg.d)) / np.sqrt(cfg.d))
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    K = torch.randn((n, cfg.d), device=dev).to(tdt)
    V = torch.empty((n, cfg.d), dtype=torch.float32, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    for _ in range(max(args.warmup, 3)):
        B.slim_values_from_keys(ctx, K, n, V, st)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        B.slim_values_from_keys(ctx, K, n, V, st)
    e1.record(); torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    tf = 2.0 * n * cfg.d * cfg.d / (ms * 1e-3) / 1e12
    peak, sustained = 1590.0, 1400.0
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    kind = "fallback"
    if os.path.exists(pk):
        with open(pk) as f:
            pkd = json.load(f)
        peak = float(pkd["bf16_tflops"]); sustained = float(pkd.get("bf16_tflops_sustained", peak)); kind = "measured"
    print(json.dumps({"metric": "prompt_value_rows_per_s", "variant": "prompt", "value": n / (ms * 1e-3), "unit": "rows/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
                      "dtype": cfg.dtype, "data": "synthetic",
                      "config": {"workload": f"config{args.config}:{cfg.name} (prompt phase V = K W_KV)", "rows": n, "d": cfg.d,
                                 "H": cfg.H, "d_k": cfg.d_k},
                      "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                                   "traffic": None, "peak_kind": kind, "frac_of_sustained_peak": tf / sustained},
                      "device_status": int(B.slim_device_status(ctx, st))}))
    B.slim_destroy(ctx)


def _rank_entry(rank, world, argv):
    """Body of one spawned replica: the launcher environment is set, run the benchmark as that rank."""
    sys.argv = [os.path.abspath(__file__)] + list(argv)
    main()


def main():
    args = parse()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.variant in ("kcache", "fp8"):
        # no launcher around us: start one process per GPU ourselves (same rendezvous a launcher would set up)
        from paper_2503_05840_b200 import replicas
        import torch
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus} asked for, {torch.cuda.device_count()} CUDA device(s) visible")
        return replicas.spawn_replicas(_rank_entry, args.gpus, (sys.argv[1:],))
    if args.variant == "xcache":
        return run_xcache(args)
    if args.variant == "prompt":
        return run_prompt(args)

    import torch
    from paper_2503_05840_b200 import binding as B
    from paper_2503_05840_b200 import build as _build
    from paper_2503_05840_b200 import synth
    from paper_2503_05840_b200.layer import SlimLayer

    from paper_2503_05840_b200 import replicas
    rank, world, local = replicas.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    if rank == 0:
        _build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("NCCL_DEBUG", "INFO")           # the rank count of the job shows in NCCL's own log (stderr)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
        dist.barrier()
    dev = f"cuda:{local}"
    torch.cuda.set_device(local)

    cfg = synth.CONFIGS[args.config]
    if args.batch:
        cfg = cfg.scaled(batch=args.batch)
    layers_n = args.layers or cfg.layers
    cfg = cfg.scaled(layers=layers_n)
    fp8 = args.variant == "fp8"
    cfg_draw = cfg                               # the keys are drawn in the config's own type ...
    if fp8:
        assert cfg.dtype == "bf16", "the 8-bit cache takes bf16 keys"
        cfg = cfg.scaled(dtype="fp8")            # ... and quantised by the library when they are appended
    path = {"auto": B.SLIM_PATH_AUTO, "generic": B.SLIM_PATH_GENERIC, "tc": B.SLIM_PATH_TC}[args.path]

    # ---- set-up (untimed): per-layer weights, W_KV solve, K-cache fill -----------
    seed0 = replicas.replica_seed(synth.layer_seed(args.config, 0), rank)
    lengths = synth.make_lengths(cfg, synth.layer_seed(args.config, 0))      # same ragged mix on every rank
    lens_dev = torch.from_numpy(lengths).to(dev)
    pos_dev = (lens_dev - 1).clamp(min=0).to(torch.int32)
    layers = []
    ws = None
    paged_tables = []

    def seq_rows(li, lay, b, n):
        """Context rows 0..n-1 of sequence b of a layer, whatever the cache arrangement."""
        if fp8:                                  # stored key = code * 2^exponent, decoded with the oracle's table of the format
            from oracle import slim_oracle as so
            nb = cfg.batch * cfg.context * cfg.d
            codes = lay.k[:nb].view(cfg.batch, cfg.context, cfg.d)[b, :n].cpu().numpy()
            off = (nb + 15) // 16 * 16
            exps = lay.k[off:off + cfg.batch * cfg.context * cfg.H].view(torch.int8).view(cfg.batch, cfg.context, cfg.H)[b, :n].cpu().numpy()
            vals = so.e4m3_decode_table()[codes].reshape(n, cfg.H, cfg.d_k) * np.exp2(exps.astype(np.float64))[:, :, None]
            return torch.from_numpy(vals.reshape(n, cfg.d))
        if not args.paged:
            return lay.k[b, :n]
        pr = args.paged
        pages = paged_tables[li][b, :(n + pr - 1) // pr].long()
        return lay.k.reshape(-1, pr, cfg.d)[pages].reshape(-1, cfg.d)[:n]

    def make_paged(lay, page_rows, li):
        # the layer's own storage is the pool: [batch * pages][page_rows][d]; sequence b uses pages in a rotated order,
        # so rows must be written through the table (slim_append_k) -- done below by re-appending the drawn keys
        assert cfg.context % page_rows == 0
        mp = cfg.context // page_rows
        tab = (torch.arange(cfg.batch * mp, dtype=torch.int32, device=dev).reshape(cfg.batch, mp) + 7 * (li + 1)) % (cfg.batch * mp)
        B.slim_cache_destroy(lay.cache)
        lay.cache = B.slim_cache_create_paged(lay.ctx, lay.k, cfg.batch * mp, page_rows, tab, cfg.batch, mp)
        return tab
    q_all = torch.zeros((layers_n, cfg.batch, cfg.d), dtype=torch.float32 if cfg.dtype == "f32" else torch.bfloat16,
                        device=dev)
    knew_all = torch.zeros_like(q_all)
    o_all = torch.zeros((layers_n, cfg.batch, cfg.d), dtype=torch.float32, device=dev)
    wkv_last = None
    wkv_all = []
    small_keys = synth.kcache_bytes_per_step(cfg, lengths) < 512e6 and not fp8 and not args.paged
    t_setup = time.time()
    for li in range(layers_n):
        lay = SlimLayer(cfg.d, cfg.H, cfg.d_k, cfg.rope_theta, cfg.dtype, cfg.batch, cfg.context, dev, workspace=ws)
        ws = lay.workspace
        lay.set_path(path)
        W_Q, W_K, W_V, _, _ = synth.make_weights_torch(cfg.d, seed0 + li, dev)
        if fp8:                             # bf16 keys into a scratch tensor, then through slim_append_k (which quantises)
            tmp = torch.zeros((cfg.batch, cfg.context, cfg.d), dtype=torch.bfloat16, device=dev)
            synth.fill_layer_torch(cfg_draw, seed0 + li, W_Q, W_K, lengths, tmp, q_all[li])
            lay.append_k(tmp, torch.zeros(cfg.batch, dtype=torch.int32, device=dev))
            for b in range(cfg.batch):
                if lengths[b] > 0:
                    knew_all[li, b] = tmp[b, int(lengths[b]) - 1]
            torch.cuda.synchronize()
            del tmp
        else:
            synth.fill_layer_torch(cfg, seed0 + li, W_Q, W_K, lengths, lay.k, q_all[li])
        if args.paged:                      # move the drawn keys into the paged arrangement through slim_append_k
            tmp = lay.k.clone()
            paged_tables.append(make_paged(lay, args.paged, li))
            lay.append_k(tmp, torch.zeros(cfg.batch, dtype=torch.int32, device=dev))
            torch.cuda.synchronize()
            del tmp
        want = (li == layers_n - 1) or small_keys
        res, wkv = lay.set_weights(W_K.cpu().numpy(), W_V.cpu().numpy(), want_wkv=want)
        if small_keys:
            wkv_all.append(wkv)
        if li == layers_n - 1:
            wkv_last = wkv
        assert res < 1e-8, f"W_KV residual {res}"
        for b in range(cfg.batch):          # the step re-appends the newest key row
            if lengths[b] > 0 and not fp8:
                knew_all[li, b] = seq_rows(li, lay, b, int(lengths[b]))[-1]
        del W_Q, W_K, W_V
        layers.append(lay)
    torch.cuda.synchronize()
    # Cold-cache timing for workloads whose keys would otherwise stay in L2 (126 MB): the step rotates
    # over enough distinct copies of the caches that at least 512 MB of keys lie between two visits
    # of the same copy.  Copies share the data and W_KV; only their storage differs.
    k_bytes_step = synth.kcache_bytes_per_step(cfg, lengths)
    n_sets = 1
    if k_bytes_step < 512e6 and not fp8 and not args.paged:
        n_sets = int(min(512, -(-512e6 // max(k_bytes_step, 1)) + 1))
    layer_sets = [layers]
    for _ in range(n_sets - 1):
        clone = []
        for li, lay in enumerate(layers):
            c = SlimLayer(cfg.d, cfg.H, cfg.d_k, cfg.rope_theta, cfg.dtype, cfg.batch, cfg.context, dev, workspace=ws)
            c.set_path(path)
            c.k.copy_(lay.k)
            c.set_wkv(wkv_all[li])
            clone.append(c)
        layer_sets.append(clone)
    torch.cuda.synchronize()
    t_setup = time.time() - t_setup
    stream = torch.cuda.current_stream()
    turn = [0]

    def step():
        cur = layer_sets[turn[0] % n_sets]
        turn[0] += 1
        for li, lay in enumerate(cur):
            lay.decode_step(q_all[li], knew_all[li], lens_dev, o_all[li])

    def step_warm():
        for li, lay in enumerate(layers):
            lay.decode_step(q_all[li], knew_all[li], lens_dev, o_all[li])

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = replicas.max_over_ranks(e0.elapsed_time(e1), dist, dev)
        barrier()
        return ms

    def timed_blocks(fn, steps):
        """The timed region: `steps` steps bracketed by barrier + synchronize.  A region under a second
        is repeated (up to 5 blocks of `steps` steps, back to back) and the median block is reported,
        so that one slow or fast block (clock ramp, a neighbour on the host) does not decide the line."""
        first = timed(fn, steps)
        blocks = [first]
        if first < 1000.0:
            n_more = int(min(4, max(0, 2000.0 // max(first, 1.0))))
            blocks += [timed(fn, steps) for _ in range(n_more)]
        return float(np.median(blocks)), blocks

    # ---- device-resident timing ------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step()
    for lay in layers[:1]:
        assert lay.device_status() == B.SLIM_OK, f"device status {lay.device_status()} after warm-up"
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    t0 = time.time()
    ms_total, ms_blocks = timed_blocks(step, args.steps)
    ms_step = ms_total / args.steps
    tokens = cfg.batch * world
    value = replicas.job_throughput(cfg.batch, world, ms_step)

    # ---- attribution inside a sustained loop: the library records CUDA events around the main
    # kernel and the tail of every decode; the loop runs like the timed one (no synchronisation
    # between steps, same clocks and power state) and the events of its last step are read once,
    # after it.  The events cost a little, so this loop's own step time is reported beside it.
    for lset in layer_sets:
        for lay in lset:
            lay.profile(True)
    turn_prof = turn[0]
    ms_prof = timed(step, args.steps) / args.steps
    main_list, tail_list = [], []
    for i in range(min(n_sets, args.steps)):          # the copies this loop visited (each holds its last step's events)
        for lay in layer_sets[(turn_prof + i) % n_sets]:
            a, b = lay.profile_read()
            main_list.append(a); tail_list.append(b)
    for lset in layer_sets:
        for lay in lset:
            lay.profile(False)
    warm_ms = None
    if n_sets > 1:                                   # the same step on ONE copy: keys served from L2
        for _ in range(3):
            step_warm()
        warm_ms = timed(step_warm, args.steps) / args.steps
    probe = hbm_read_probe(dev) if rank == 0 else None
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    main_ms, tail_ms = float(np.mean(main_list)), float(np.mean(tail_list))
    k_bytes_layer = synth.kcache_bytes_per_step(cfg.scaled(layers=1), lengths)
    peak, peak_kind = measured_peaks()
    achieved = k_bytes_layer / (main_ms * 1e-3) / 1e9
    step_gbs = k_bytes_layer * layers_n / (ms_step * 1e-3) / 1e9

    # ---- end to end through host buffers -----------------------------------------
    e2e = None
    if not args.no_e2e:
        q_host = q_all.cpu().pin_memory()
        k_host = knew_all.cpu().pin_memory()
        o_host = torch.empty(o_all.shape, dtype=torch.float32).pin_memory()

        # Per layer: inputs in on a copy stream, append + decode on the compute stream, output out
        # on a third stream, chained with events, so that the transfers of one layer run beside the
        # kernels of its neighbours.  The compute stream joins both copy streams at the step's end,
        # so the timed events on it bracket every byte moved.
        h2d_s, d2h_s = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in layers]
        ev_dec = [torch.cuda.Event() for _ in layers]
        ev_free, ev_h2d_end, ev_d2h_end = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()

        def step_e2e():
            ev_free.record(stream)                       # the last step no longer reads q_all / knew_all
            h2d_s.wait_event(ev_free)
            with torch.cuda.stream(h2d_s):
                for li in range(layers_n):
                    q_all[li].copy_(q_host[li], non_blocking=True)
                    knew_all[li].copy_(k_host[li], non_blocking=True)
                    ev_in[li].record(h2d_s)
                ev_h2d_end.record(h2d_s)
            cur = layer_sets[turn[0] % n_sets]
            turn[0] += 1
            for li, lay in enumerate(cur):
                stream.wait_event(ev_in[li])
                lay.decode_step(q_all[li], knew_all[li], lens_dev, o_all[li])
                ev_dec[li].record(stream)
                d2h_s.wait_event(ev_dec[li])
                with torch.cuda.stream(d2h_s):
                    o_host[li].copy_(o_all[li], non_blocking=True)
            ev_d2h_end.record(d2h_s)
            stream.wait_event(ev_h2d_end)
            stream.wait_event(ev_d2h_end)

        for _ in range(3):
            step_e2e()
        ms_e2e = timed_blocks(step_e2e, args.steps)[0] / args.steps
        assert torch.equal(o_host, o_all.cpu()), "end-to-end outputs differ from the resident ones"
        e2e = {"value": tokens / (ms_e2e * 1e-3), "unit": "tokens/s",
               "h2d_bytes_per_step": int(q_host.numel() * q_host.element_size() * 2),
               "d2h_bytes_per_step": int(o_host.numel() * 4), "ms_per_step": ms_e2e}

    # ---- CPU oracle baseline on a bounded sample (rank 0, N=1 only) ----------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import slim_oracle as so
        lay = layers[-1]
        W_KV = wkv_last
        # bounded sample: whole sequences of the last layer, longest-first order does not matter;
        # stop once ~20 s of host time are spent
        rows_done, dt, worst, n_seq = 0, 0.0, 0.0, 0
        got_all = lay.decode(q_all[-1], lens_dev).cpu().numpy().astype(np.float64)
        for b in range(cfg.batch):
            n = int(lengths[b])
            if n == 0:
                continue
            Kb = seq_rows(layers_n - 1, lay, b, n).double().cpu().numpy()
            qb = q_all[-1, b].float().cpu().numpy().astype(np.float64)
            tt = time.perf_counter()
            ref = so.oracle_slim(qb, Kb, W_KV, cfg.H, cfg.rope_theta)
            dt += time.perf_counter() - tt
            rows_done += n; n_seq += 1
            err = so.err_fp32_norm(got_all[b], ref) if cfg.dtype == "f32" else so.err_rms_norm(got_all[b], ref)
            worst = max(worst, err)          # the same sample doubles as a live parity check of what was timed
            if dt > 20.0:
                break
        per_step = dt * (float(np.sum(lengths)) / rows_done) * layers_n      # all sequences, all layers
        tol = 1e-4 if cfg.dtype == "f32" else 2e-2
        parity_ok = worst <= tol
        cpu = {"value": cfg.batch / per_step, "unit": "tokens/s", "cores": host_threads(), "kind": "oracle",
               "parity_tolerance": tol, "parity": "green" if parity_ok else "FAILED",
               "sample": f"oracle_slim on layer {layers_n - 1}, {n_seq} full sequences ({rows_done} context rows, "
                         f"{dt:.1f} s), scaled by rows to {int(np.sum(lengths))} rows x {layers_n} layers",
               "parity_err_on_sample": worst}

    status = max(int(lay.device_status()) for lay in layers)      # worst status over all layers
    if rank == 0:
        launches = sum(lay.query(B.SLIM_Q_LAUNCHES_PER_DECODE) for lay in layers)
        line = {
            "metric": "decode_attention_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": {"bf16": "bf16", "f32": "f32", "fp8": "e4m3 cache decoded exactly to bf16, then the bf16 path (bf16 queries and W_KV)"}[cfg.dtype],
            "data": "synthetic",
            "config": {"workload": f"config{args.config}:{cfg.name}" + (" (8-bit K-cache)" if fp8 else ""), "layers": layers_n, "batch_per_gpu": cfg.batch,
                       "global_batch": tokens, "context": cfg.context, "sum_lengths": int(lengths.sum()),
                       "d": cfg.d, "H": cfg.H, "d_k": cfg.d_k, "rope_theta": cfg.rope_theta,
                       "parallelism": f"replicas x{world} (batch-sharded, no collective)",
                       "l2": "inputs larger than L2 (K-cache per step >> 126 MB)" if n_sets == 1
                             else f"cold: the step rotates over {n_sets} distinct copies of the cache "
                                  f"({n_sets * k_bytes_step / 1e6:.0f} MB of keys between two visits of a copy)",
                       "path": {1: "generic", 2: "tc"}[layers[0].query(B.SLIM_Q_PATH_IN_USE)],
                       "cache": f"paged, {args.paged} rows per page" if args.paged else "contiguous"},
            "kcache_gbs": step_gbs, "kcache_frac_of_8000": step_gbs / 8000.0, "kcache_frac_of_measured": step_gbs / peak,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": ncu_traffic(args.config) if not fp8 else None, "peak_kind": peak_kind,
                         "kernel": "main decode kernel (per layer launch)" if not fp8 else
                                   ("decode of the 8-bit rows into the bf16 scratch + main decode kernel on the scratch "
                                    "(1 + 2 + 2 bytes of DRAM traffic per key element)"
                                    if layers[0].query(B.SLIM_Q_PATH_IN_USE) == 2 else
                                    "score + accumulation kernels (CUDA cores; the 8-bit keys are read twice per layer)"),
                         "main_ms": main_ms, "tail_ms": tail_ms, "bytes_per_launch": k_bytes_layer,
                         "timing": "CUDA events recorded by the library inside a sustained loop of the same step "
                                   "(last step, mean over layers); that loop ran at %.4f ms per step" % ms_prof},
            "ms_per_step_blocks": [b / args.steps for b in ms_blocks],
            "warm_cache_ms_per_step": warm_ms, "hbm_read_probe": probe,
            "e2e": e2e, "cpu_baseline": cpu, "gpu_launches": launches, "clocks": clocks,
            "device_status": int(status), "setup_s": t_setup,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if cpu is not None and cpu["parity"] != "green":
        raise SystemExit(f"parity check against the oracle FAILED on the timed workload: {cpu['parity_err_on_sample']:.3e} "
                         f"> {cpu['parity_tolerance']}")


if __name__ == "__main__":
    main()
