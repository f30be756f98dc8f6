"""World-size-2 check (gloo, CPU) of the replica logic bench.py uses for N > 1:
distinct per-rank seeds, identical length mix, max-over-ranks timing, whole-job
throughput.  No GPU and no CUDA library is touched."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2503_05840_b200 import replicas, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, w, _ = replicas.rank_info()
    cfg = synth.CONFIGS[2].scaled(batch=4, context=256, ragged_min=128, d=64, H=2, d_k=32)
    base = synth.layer_seed(2, 0)
    lengths = synth.make_lengths(cfg, base)                       # same on every rank
    L = synth.make_layer(cfg, replicas.replica_seed(base, r), lengths=lengths)
    ms = replicas.max_over_ranks(10.0 + 5.0 * r, dist)            # rank 1 is the slow one
    dist.barrier()
    out.put((r, w, lengths.tolist(), float(L.K[0, 0, 0]), ms, replicas.job_throughput(cfg.batch, w, ms)))
    dist.destroy_process_group()


def test_two_replicas_share_only_timing():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (r0, w0, len0, k0, ms0, v0), (r1, w1, len1, k1, ms1, v1) = res
    assert (r0, r1) == (0, 1) and w0 == w1 == 2
    assert len0 == len1                                  # equal work per rank
    assert k0 != k1                                      # different data per rank
    assert ms0 == ms1 == 15.0                            # slowest rank's time on both
    assert np.isclose(v0, 4 * 2 / 15e-3) and v0 == v1    # units of all ranks / that time


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2503_05840_b200 import replicas
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.replica_seed(7, 0) == 7 and replicas.replica_seed(7, 3) != replicas.replica_seed(7, 2)


def _stub_rank(rank, world, out_dir):
    """What bench.py does per rank, with the GPU step replaced by a stub: rendezvous from the
    launcher environment, barrier, max-over-ranks of a per-rank time, one line from rank 0."""
    sys.path.insert(0, ROOT)
    import json
    import torch.distributed as dist
    from paper_2503_05840_b200 import replicas
    r, w, local = replicas.rank_info()
    assert (r, w, local) == (rank, world, rank)
    dist.init_process_group("gloo")
    dist.barrier()
    ms = replicas.max_over_ranks(4.0 + 2.0 * r, dist)
    dist.barrier()
    if r == 0:
        with open(os.path.join(out_dir, "line.json"), "w") as f:
            json.dump({"n_gpus": w, "ms_per_step": ms, "value": replicas.job_throughput(16, w, ms), "scaling": "weak"}, f)
    dist.destroy_process_group()


def test_spawn_replicas_starts_one_process_per_rank(tmp_path):
    """The path bench.py --gpus N takes when no launcher started it: N processes, launcher-style
    environment, one result line from rank 0 that carries the whole job."""
    import json
    sys.path.insert(0, ROOT)
    from paper_2503_05840_b200 import replicas
    replicas.spawn_replicas(_stub_rank, 2, (str(tmp_path),))
    with open(tmp_path / "line.json") as f:
        line = json.load(f)
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 6.0 and line["scaling"] == "weak"
    assert np.isclose(line["value"], 16 * 2 / 6e-3)


def _split_rank(rank, world, out_dir):
    """One rank of a split context on CPU: its slice's partial comes from the oracle (the CUDA kernels
    need a GPU), the exchange and the index logic are the package's own."""
    sys.path.insert(0, ROOT)
    import json
    import torch
    import torch.distributed as dist
    from oracle import slim_oracle as so
    from paper_2503_05840_b200 import context_split as cs
    from paper_2503_05840_b200 import synth
    dist.init_process_group("gloo")
    cfg = synth.SlimConfig("split", 32, 2, 16, 3, 100, 1, 1.0e4, "f32")
    lengths = np.array([100, 37, 0], dtype=np.int32)
    L = synth.make_layer(cfg, 2468, lengths=lengths)                  # same seed on every rank: the same context
    W_KV = so.oracle_wkv(L.W_K, L.W_V)
    first, count = cs.shard_batch(lengths, world, rank)
    lse = np.empty((cfg.batch, cfg.H)); u = np.empty((cfg.batch, cfg.H, cfg.d))
    for b in range(cfg.batch):
        a = first[b] * cs.TILE
        lse[b], u[b] = so.oracle_slim_partial(L.q[b], L.K[b, a:a + count[b]], a, int(lengths[b]) - 1, cfg.H, cfg.rope_theta)
    lse_all, u_all = cs.gather_partials(torch.from_numpy(lse), torch.from_numpy(u), dist)
    assert tuple(lse_all.shape) == (world, cfg.batch, cfg.H) and tuple(u_all.shape) == (world, cfg.batch, cfg.H, cfg.d)
    worst = 0.0
    for b in range(cfg.batch):
        out = so.oracle_combine_partials(lse_all[:, b].numpy(), u_all[:, b].numpy(), W_KV)
        ref = so.oracle_slim_batch(L.q, L.K, lengths, W_KV, cfg.H, cfg.rope_theta)[b]
        worst = max(worst, float(np.max(np.abs(out - ref))))
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"worst": worst, "count": count, "first": first}, f)
    dist.destroy_process_group()


def test_context_split_two_ranks_exchange_and_join(tmp_path):
    import json
    sys.path.insert(0, ROOT)
    from paper_2503_05840_b200 import context_split as cs
    from paper_2503_05840_b200 import replicas
    # slices are whole tiles, cover the context once, and the ragged tail goes to the last non-empty slice
    for n in (0, 1, 15, 16, 17, 100, 131072):
        for world in (1, 2, 3, 8):
            cuts = [cs.shard_rows(n, world, r) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(cuts[:-1], cuts[1:]))
            assert all(a % cs.TILE == 0 for a, _ in cuts if a < n)
    replicas.spawn_replicas(_split_rank, 2, (str(tmp_path),))
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(2)]
    assert all(r["worst"] < 1e-12 for r in res)                       # every rank holds the whole-context result
    assert [a + b for a, b in zip(res[0]["count"], res[1]["count"])] == [100, 37, 0]
