"""Paged K-cache: keys live in a pool of pages addressed through a block table.  slim_decode and
slim_append_k must give exactly what they give on a contiguous cache holding the same rows."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2503_05840_b200 import binding as B
from paper_2503_05840_b200 import synth
from paper_2503_05840_b200.layer import SlimLayer, to_device_keys

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("d,H,d_k,theta,dtype,page_rows", [
    (512, 4, 128, 1.0e6, "bf16", 16), (512, 4, 128, 1.0e4, "bf16", 64), (1280, 20, 64, 0.0, "bf16", 32), (256, 4, 64, 1.0e4, "f32", 16)])
def test_paged_cache_equals_contiguous_cache(d, H, d_k, theta, dtype, page_rows):
    lengths = np.array([333, 0, 640, 17, 257], dtype=np.int32)
    batch, t_cap = len(lengths), 640
    max_pages = t_cap // page_rows
    cfg = synth.SlimConfig("paged", d, H, d_k, batch, t_cap, 1, theta, dtype)
    L = synth.make_layer(cfg, 77, lengths=lengths)
    W_KV = so.oracle_wkv(L.W_K, L.W_V)
    g = np.random.default_rng(1)
    num_pages = batch * max_pages + 7
    perm = g.permutation(num_pages)[:batch * max_pages].astype(np.int32).reshape(batch, max_pages)
    ref_layer = SlimLayer(d, H, d_k, theta, dtype, batch, t_cap, DEV)
    ctx = B.slim_create(d, H, d_k, theta, B.SLIM_BF16 if dtype == "bf16" else B.SLIM_F32)
    cache = None
    try:
        with torch.cuda.device(DEV):
            Kd = to_device_keys(L.K, dtype, DEV)
            ref_layer.k.copy_(Kd)
            ref_layer.set_wkv(W_KV)
            B.slim_set_wkv(ctx, W_KV)
            pool = torch.full((num_pages, page_rows, d), float("nan"), dtype=Kd.dtype, device=DEV)   # unused pages are poison
            table = torch.from_numpy(perm).to(DEV)
            cache = B.slim_cache_create_paged(ctx, pool, num_pages, page_rows, table, batch, max_pages)
            ws = torch.empty(B.slim_workspace_bytes(ctx, batch, t_cap), dtype=torch.uint8, device=DEV)
            st = torch.cuda.current_stream().cuda_stream
            # fill the pool through slim_append_k: all but the last row in bulk, then the last row
            for b in range(batch):
                for pg in range(max_pages):
                    pool[perm[b, pg]] = 0
            bulk = int(lengths[lengths > 0].min()) - 1
            pos0 = torch.zeros(batch, dtype=torch.int32, device=DEV)
            B.slim_append_k(ctx, cache, Kd[:, :bulk].contiguous(), pos0, bulk, st)
            for b in range(batch):                                  # the rest row-wise through the table on the host side
                for t in range(bulk, int(lengths[b])):
                    pool[perm[b, t // page_rows], t % page_rows] = Kd[b, t]
                if lengths[b] < bulk:
                    pass
            q = to_device_keys(L.q, dtype, DEV)
            ld = torch.from_numpy(lengths).to(DEV)
            for path in (B.SLIM_PATH_AUTO, B.SLIM_PATH_GENERIC):
                ref_layer.set_path(path); B.slim_set_path(ctx, path)
                want = ref_layer.decode(q, ld).clone()
                o = torch.full((batch, d), float("nan"), dtype=torch.float32, device=DEV)
                B.slim_decode(ctx, q, cache, ld, o, ws, st)
                assert B.slim_device_status(ctx, st) == B.SLIM_OK
                assert torch.equal(o, want), f"path {path}"
            ref = so.oracle_slim_batch(L.q, L.K, lengths, W_KV, H, theta)
            got = o.cpu().numpy().astype(np.float64)
            for b in range(batch):
                if lengths[b]:
                    e = so.err_rms_norm(got[b], ref[b]) if dtype == "bf16" else so.err_fp32_norm(got[b], ref[b])
                    assert e <= (2e-2 if dtype == "bf16" else 1e-4)
            # a page id outside the pool is reported, not followed
            bad = table.clone(); bad[0, 0] = num_pages + 3
            cache_bad = B.slim_cache_create_paged(ctx, pool, num_pages, page_rows, bad, batch, max_pages)
            B.slim_decode(ctx, q, cache_bad, ld, o, ws, st)
            assert B.slim_device_status(ctx, st) == B.SLIM_ERR_CAPACITY
            B.slim_cache_destroy(cache_bad)
    finally:
        if cache:
            B.slim_cache_destroy(cache)
        B.slim_destroy(ctx)
        ref_layer.close()


def test_paged_cache_argument_checks():
    ctx = B.slim_create(128, 2, 64, 0.0, B.SLIM_BF16)
    try:
        with torch.cuda.device(DEV):
            pool = torch.zeros((4, 24, 128), dtype=torch.bfloat16, device=DEV)
            table = torch.zeros((1, 2), dtype=torch.int32, device=DEV)
            with pytest.raises(B.SlimError) as ei:                       # page_rows must be a multiple of 16
                B.slim_cache_create_paged(ctx, pool, 4, 24, table, 1, 2)
            assert ei.value.status == B.SLIM_ERR_UNSUPPORTED
            with pytest.raises(B.SlimError) as ei:
                B.slim_cache_create_paged(ctx, pool, 0, 16, table, 1, 2)
            assert ei.value.status == B.SLIM_ERR_INVALID_ARG
    finally:
        B.slim_destroy(ctx)
