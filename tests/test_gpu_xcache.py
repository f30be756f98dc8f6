"""X-cache / E-cache scheme through the C ABI against the oracle: the cache holds the
layer inputs X, scores use the dense per-head query (x_n W_Q,i + b) W_K,i^T, values are
recomputed as [softmax X] W_V,i.  Same tolerances as the K-cache path."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2503_05840_b200 import binding as B
from paper_2503_05840_b200 import synth
from paper_2503_05840_b200.layer import to_device_keys

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {"f32": 1e-4, "bf16": 2e-2}


class XLayer:
    """One decoder layer's X-cache context over caller-owned (possibly shared) storage."""
    def __init__(self, d, H, d_k, dtype, batch, t_cap, storage):
        self.ctx = B.slim_create(d, H, d_k, 0.0, B.SLIM_BF16 if dtype == "bf16" else B.SLIM_F32)
        self.cache = B.slim_cache_create(self.ctx, storage, batch, t_cap)
        self.ws = torch.empty(B.slim_xcache_workspace_bytes(self.ctx, batch, t_cap), dtype=torch.uint8, device=DEV)
        self.o = torch.empty((batch, d), dtype=torch.float32, device=DEV)

    def decode(self, q, lengths):
        B.slim_xcache_decode(self.ctx, q, self.cache, lengths, self.o, self.ws, torch.cuda.current_stream().cuda_stream)
        return self.o

    def close(self):
        B.slim_cache_destroy(self.cache); B.slim_destroy(self.ctx)


def _err(got, ref, dtype):
    return so.err_fp32_norm(got, ref) if dtype == "f32" else so.err_rms_norm(got, ref)


@pytest.mark.parametrize("d,H,d_k,dtype", [(256, 4, 64, "f32"), (512, 4, 128, "bf16"), (1280, 20, 64, "bf16"), (384, 4, 96, "bf16")])
def test_xcache_decode_matches_oracle_and_layers_share_one_cache(d, H, d_k, dtype):
    g = np.random.default_rng(d + H)
    lengths = np.array([700, 333, 0, 17, 1], dtype=np.int32)
    batch, t_cap = len(lengths), 700
    X = np.zeros((batch, t_cap, d), dtype=np.float32)
    for b in range(batch):
        X[b, :lengths[b]] = synth.round_to_dtype(g.standard_normal((int(lengths[b]), d)), dtype)
    with torch.cuda.device(DEV):
        storage = to_device_keys(X, dtype, DEV)
        storage[1, lengths[1]:] = float("nan")                     # rows past the end must not matter
        layers = []
        try:
            for li in range(2):                                    # two layers, one shared E-cache
                W_Q, W_K, W_V, _, _ = synth.make_weights(d, 100 + li)
                bias = g.standard_normal(d) * 0.1
                q = np.zeros((batch, d), dtype=np.float32)
                for b in range(batch):
                    if lengths[b]:
                        q[b] = synth.round_to_dtype(X[b, lengths[b] - 1].astype(np.float64) @ W_Q + bias, dtype)
                lay = XLayer(d, H, d_k, dtype, batch, t_cap, storage)
                layers.append(lay)
                B.slim_xcache_set_weights(lay.ctx, W_K, W_V)
                got = lay.decode(to_device_keys(q, dtype, DEV), torch.from_numpy(lengths).to(DEV)).cpu().numpy().astype(np.float64)
                assert B.slim_device_status(lay.ctx, torch.cuda.current_stream().cuda_stream) == B.SLIM_OK
                assert np.all(np.isfinite(got))
                for b in range(batch):
                    n = int(lengths[b])
                    if n == 0:
                        assert np.all(got[b] == 0)
                        continue
                    ref = so.oracle_xcache(q[b], X[b, :n], W_K, W_V, H)
                    e = _err(got[b], ref, dtype)
                    assert e <= TOL[dtype], f"layer {li} seq {b}: {e:.3e}"
        finally:
            for lay in layers:
                lay.close()


def test_xcache_needs_its_weights_and_refuses_rope():
    with torch.cuda.device(DEV):
        storage = torch.zeros((1, 32, 128), dtype=torch.bfloat16, device=DEV)
        lay = XLayer(128, 2, 64, "bf16", 1, 32, storage)
        try:
            q = torch.zeros((1, 128), dtype=torch.bfloat16, device=DEV)
            with pytest.raises(B.SlimError) as ei:
                lay.decode(q, torch.ones(1, dtype=torch.int32, device=DEV))
            assert ei.value.status == B.SLIM_ERR_NO_WEIGHTS
        finally:
            lay.close()
        ctx = B.slim_create(128, 2, 64, 1.0e4, B.SLIM_BF16)
        try:
            with pytest.raises(B.SlimError) as ei:
                B.slim_xcache_set_weights(ctx, np.eye(128), np.eye(128))
            assert ei.value.status == B.SLIM_ERR_UNSUPPORTED
        finally:
            B.slim_destroy(ctx)


def _xcache_device_case(d, H, d_k, batch, t_cap, lengths, sample, seed):
    """Inputs drawn on the device (bf16), weights from the seeded host recipe; the stored bits of
    the sampled sequences go back to the host for the oracle."""
    with torch.cuda.device(DEV):
        g = torch.Generator(device=DEV); g.manual_seed(seed)
        storage = torch.randn((batch, t_cap, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
        W_Q, W_K, W_V, _, _ = synth.make_weights(d, seed)
        bias = np.random.default_rng(seed).standard_normal(d) * 0.1
        lens = torch.from_numpy(lengths).to(DEV)
        x_last = storage[torch.arange(batch, device=DEV), (lens.long() - 1).clamp(min=0)].double()
        q = (x_last @ torch.from_numpy(W_Q).to(DEV) + torch.from_numpy(bias).to(DEV)).to(torch.bfloat16)
        for b in range(batch):
            if lengths[b] < t_cap:
                storage[b, int(lengths[b]):] = float("nan")         # rows past the end must not matter
        lay = XLayer(d, H, d_k, "bf16", batch, t_cap, storage)
        try:
            B.slim_xcache_set_weights(lay.ctx, W_K, W_V)
            got = lay.decode(q, lens).cpu().numpy().astype(np.float64)
            assert B.slim_device_status(lay.ctx, torch.cuda.current_stream().cuda_stream) == B.SLIM_OK
            assert np.all(np.isfinite(got))
            worst = 0.0
            for b in sample:
                n = int(lengths[b])
                if n == 0:
                    assert np.all(got[b] == 0)
                    continue
                ref = so.oracle_xcache(q[b].float().cpu().numpy(), storage[b, :n].float().cpu().numpy(), W_K, W_V, H)
                e = so.err_rms_norm(got[b], ref)
                worst = max(worst, e)
                assert e <= TOL["bf16"], f"seq {b}: {e:.3e}"
            return worst
        finally:
            lay.close()


def test_xcache_whisper_large_shape_full_batch_sampled_sequences():
    """The shape the X-cache variant is benchmarked on (batch 64, 1500 encoder rows, d = 1280, 20 heads):
    the dense query transform walks the batch in four passes of 16 sequences; one sequence of each pass
    and both ends of the batch are checked."""
    lengths = np.full(64, 1500, dtype=np.int32)
    worst = _xcache_device_case(1280, 20, 64, 64, 1500, lengths, [0, 15, 16, 37, 48, 63], 3003)
    print(f"X-cache, Whisper-large shape: worst error {worst:.3e}")


def test_xcache_batch_above_sixteen_small_ragged():
    """More than 16 sequences at a small size: several passes of the query transform, ragged lengths,
    an empty sequence and single rows; every sequence is checked."""
    g = np.random.default_rng(5)
    lengths = g.integers(1, 120, size=40).astype(np.int32)
    lengths[[3, 17, 33]] = [0, 1, 119]
    _xcache_device_case(256, 4, 64, 40, 119, lengths, list(range(40)), 3004)


@pytest.mark.parametrize("d,H,d_k,dtype", [(512, 8, 128, "bf16"),      # e = 1024 > d, tensor-core kernels (a T5-style widening)
                                           (512, 2, 128, "bf16"),      # e = 256 < d
                                           (1280, 10, 64, "bf16"),     # e = 640, two heads per projection MMA
                                           (192, 4, 64, "f32"),        # CUDA-core kernels, e = 256
                                           (320, 6, 100, "f32")])      # a head width outside the vector paths, e = 600
def test_xcache_nonsquare_projections_match_oracle(d, H, d_k, dtype):
    """Non-square projections (section "Support for non-square weight matrices", Option 2): the cache
    holds d-wide inputs, W_K and W_V are d x e with e = H d_k != d, queries and outputs are e wide."""
    e = H * d_k
    g = np.random.default_rng(d + e)
    lengths = np.array([700, 333, 0, 17, 1, 129], dtype=np.int32)
    batch, t_cap = len(lengths), 700
    X = np.zeros((batch, t_cap, d), dtype=np.float32)
    for b in range(batch):
        X[b, :lengths[b]] = synth.round_to_dtype(g.standard_normal((int(lengths[b]), d)), dtype)
    if e > d:
        W_Q, W_K, W_V, _, _ = synth.make_weights_nonsquare(d, e, 500 + d)
    else:
        W_Q, W_K, W_V = (g.standard_normal((d, e)) / np.sqrt(d) for _ in range(3))
    bias = g.standard_normal(e) * 0.1
    q = np.zeros((batch, e), dtype=np.float32)
    for b in range(batch):
        if lengths[b]:
            q[b] = synth.round_to_dtype(X[b, lengths[b] - 1].astype(np.float64) @ W_Q + bias, dtype)
    with torch.cuda.device(DEV):
        storage = to_device_keys(X, dtype, DEV)
        storage[1, lengths[1]:] = float("nan")
        ctx = B.slim_xcache_create(d, H, d_k, B.SLIM_BF16 if dtype == "bf16" else B.SLIM_F32)
        cache = None
        try:
            cache = B.slim_cache_create(ctx, storage, batch, t_cap)
            ws = torch.empty(B.slim_xcache_workspace_bytes(ctx, batch, t_cap), dtype=torch.uint8, device=DEV)
            o = torch.full((batch, e), float("nan"), dtype=torch.float32, device=DEV)
            st = torch.cuda.current_stream().cuda_stream
            B.slim_xcache_set_weights(ctx, W_K, W_V)
            B.slim_xcache_decode(ctx, to_device_keys(q, dtype, DEV), cache, torch.from_numpy(lengths).to(DEV), o, ws, st)
            assert B.slim_device_status(ctx, st) == B.SLIM_OK
            got = o.cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(got))
            for b in range(batch):
                n = int(lengths[b])
                if n == 0:
                    assert np.all(got[b] == 0)
                    continue
                ref = so.oracle_xcache(q[b], X[b, :n], W_K, W_V, H)
                err = _err(got[b], ref, dtype)
                assert err <= TOL[dtype], f"seq {b}: {err:.3e}"
            # the K-cache calls have no meaning on such a context (W_K is not square)
            if e != d:
                with pytest.raises(B.SlimError) as ei:
                    B.slim_decode(ctx, to_device_keys(q, dtype, DEV), cache, torch.from_numpy(lengths).to(DEV), o, ws, st)
                assert ei.value.status == B.SLIM_ERR_UNSUPPORTED
        finally:
            if cache:
                B.slim_cache_destroy(cache)
            B.slim_destroy(ctx)
